// Offline conversion of a full gate matrix into a LoPA gate (architecture casting, Sec. 3.4 "LoPA approximation"):
// minimise || W - M - U V ||_F^2 over M (one +-1 per row), U, V by alternating two exact half-steps.  The two
// element-wise / row-wise parts are here; the truncated SVD of the UV-step and the product U V are library routines
// called by the Python driver.
//
//   lopa_m_step_kernel    R = W - P row by row (P = U V, or absent for the first step): position of the largest
//                         |R_ij| (first one on ties), the sign of that entry, max |R_ij| and sum_j R_ij^2
//   lopa_residual_kernel  A = W - M, the matrix whose truncated SVD is the best U V for that M
#include "cast_kernels.cuh"

#include "common.cuh"

namespace sffn {

// One warp per row.  A lane walks its columns in ascending order and keeps the first maximum; the lanes are then
// combined so that equal magnitudes resolve to the lower column: the result does not depend on the lane layout.
__global__ void __launch_bounds__(256) lopa_m_step_kernel(const float* W, const float* P, int H, int D, int32_t* g_idx,
                                                           int8_t* g_sign, double* row_energy, float* row_best) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= H) return;
  const float* w = W + (size_t)row * D;
  const float* p = P ? P + (size_t)row * D : nullptr;
  float best = -1.f, best_val = 0.f;
  int best_j = 0;
  double energy = 0.0;
  for (int j = lane; j < D; j += 32) {
    const float r = p ? w[j] - p[j] : w[j];
    energy += (double)r * (double)r;
    const float a = fabsf(r);
    if (a > best) { best = a; best_j = j; best_val = r; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const float ov = __shfl_xor_sync(0xffffffffu, best_val, o);
    const int oj = __shfl_xor_sync(0xffffffffu, best_j, o);
    energy += __shfl_xor_sync(0xffffffffu, energy, o);
    if (ob > best || (ob == best && oj < best_j)) { best = ob; best_j = oj; best_val = ov; }
  }
  if (lane == 0) {
    g_idx[row] = best_j;
    g_sign[row] = best_val < 0.f ? -1 : 1;
    if (row_energy) row_energy[row] = energy;
    if (row_best) row_best[row] = best;
  }
}

// One CTA per row: 16-byte copies where the row allows them, and the one entry of M taken off.
__global__ void __launch_bounds__(256) lopa_residual_kernel(const float* W, const int32_t* g_idx, const int8_t* g_sign,
                                                             int H, int D, float* A) {
  const int row = blockIdx.x;
  const float* w = W + (size_t)row * D;
  float* a = A + (size_t)row * D;
  const int col = g_idx[row];
  const float m = (float)g_sign[row];
  const bool vec = D % 4 == 0 && ((reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(A)) & 15u) == 0;
  if (vec) {
    for (int q = threadIdx.x; q < D / 4; q += blockDim.x) {
      float4 v = reinterpret_cast<const float4*>(w)[q];
      if (q == col / 4) {
        const int e = col & 3;
        if (e == 0) v.x -= m; else if (e == 1) v.y -= m; else if (e == 2) v.z -= m; else v.w -= m;
      }
      reinterpret_cast<float4*>(a)[q] = v;
    }
  } else {
    for (int j = threadIdx.x; j < D; j += blockDim.x) a[j] = w[j] - (j == col ? m : 0.f);
  }
}

cudaError_t launch_lopa_m_step(const float* W, const float* P, int H, int D, int32_t* g_idx, int8_t* g_sign,
                               double* row_energy, float* row_best, cudaStream_t s) {
  lopa_m_step_kernel<<<(H + 7) / 8, 256, 0, s>>>(W, P, H, D, g_idx, g_sign, row_energy, row_best);
  return cudaGetLastError();
}

cudaError_t launch_lopa_residual(const float* W, const int32_t* g_idx, const int8_t* g_sign, int H, int D, float* A,
                                 cudaStream_t s) {
  lopa_residual_kernel<<<H, 256, 0, s>>>(W, g_idx, g_sign, H, D, A);
  return cudaGetLastError();
}

}  // namespace sffn
