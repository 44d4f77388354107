// Batched path on the warp-level tensor cores (mma.sync m16n8k16, bf16 x bf16 -> fp32), for B >= 2 tokens:
//
//   rows_mma_kernel<GATE>  Z[H, B] = W[H, K] X[B, K]^T (+ bias + fixed-matrix term), activation, gate values
//                          and per-neuron "any token fires" flags              (Eq. 1 gate / LoPA U stage)
//   rows_mma_kernel<UP>    over the union list of fired neurons (Sec. 5.4): Up[u, B] = W_up[idx[u]] X^T,
//                          Hm = a . Up, written as bf16 HmT[b][u] for the next contraction
//   down_mma_kernel        Y^T[D, B] = W_down[idx]^T Hm, split over D-slices and union chunks; the split
//                          partials are summed afterwards in fixed order (deterministic)
//
// Weight rows go from global memory straight into A fragments: a lane loads 16 contiguous bytes of row g
// and of row g+8, and the contraction index inside each 32-wide block is permuted identically for the
// token operand, so no shared-memory staging or ldmatrix is needed for the streamed matrix.
// The LoPA vector n = RMSNorm(Vx) is fp32; it enters as two bf16 columns per token (high and low part),
// which keeps 16 bits of mantissa through the bf16 tensor-core inputs.
#include "batched_kernels.cuh"

#include "common.cuh"

namespace sffn {

namespace {

constexpr int kDownStages = 8;      // cp.async stages of the down projection (16 union rows each)
constexpr int kKC = 128;            // contraction elements staged per step
constexpr int kXPitch = kKC + 32;   // bf16 elements; 320 bytes = 64 mod 128 -> conflict-free 16-byte reads

__device__ __forceinline__ void mma_bf16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool valid) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const int n = valid ? 16 : 0;  // src-size 0: zero fill
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// ------------------------------------------------------------------------------------------------
// One CTA = 8 warps x 16 rows.  NT = number of 8-column tiles of the token operand.
template <int NT, bool UP>
__global__ void __launch_bounds__(256) rows_mma_kernel(const RowsMmaParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [3][NT*8][kXPitch]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int K = p.K;
  const int n_rows = p.count ? *p.count : p.R;
  const int n_tiles = (n_rows + 127) / 128;
  const int ncols = NT * 8;
  const int chunks_per_stage = ncols * (kKC / 8);

  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int i0 = tile * 128 + warp * 16 + g;  // list positions of this lane's two rows
    const int i1 = i0 + 8;
    int j0 = p.idx ? p.idx[min(i0, n_rows - 1)] : min(i0, n_rows - 1);
    int j1 = p.idx ? p.idx[min(i1, n_rows - 1)] : min(i1, n_rows - 1);
    if (!SFFN_IN_BOUNDS(j0 >= 0 && j0 < p.R && j1 >= 0 && j1 < p.R, p.status, 30)) j0 = j1 = 0;
    const uint4* w0 = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.W) + (size_t)j0 * K) + t;
    const uint4* w1 = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.W) + (size_t)j1 * K) + t;

    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[n][q] = 0.f;

    auto stage = [&](int kc, int buf) {
      __nv_bfloat16* dst = xs + (size_t)buf * ncols * kXPitch;
      for (int c = tid; c < chunks_per_stage; c += 256) {
        const int col = c / (kKC / 8), kk = (c % (kKC / 8)) * 8;
        const bool valid = col < p.ncols_valid && kc + kk < K;
        const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(p.X) + (size_t)(valid ? col : 0) * p.x_stride +
                                   (valid ? kc + kk : 0);
        cp_async16(dst + (size_t)col * kXPitch + kk, src, valid);
      }
      cp_async_commit();
    };

    const int n_steps = (K + kKC - 1) / kKC;
    constexpr int KB = kKC / 32;  // 32-wide blocks per step
    // Weight fragments are double-buffered in registers (two steps ahead of the tensor cores) and the
    // token operand is triple-buffered in shared memory, so the loads of steps s+1 and s+2 are in
    // flight while step s is multiplied.
    uint4 a0[3][KB], a1[3][KB];
    auto load_a = [&](int step, int buf) {
      const int kc = step * kKC;
      const int kblocks = min(kKC, K - kc) / 32;
#pragma unroll
      for (int kb = 0; kb < KB; ++kb) {
        if (kb < kblocks) {
          a0[buf][kb] = ld_stream16(w0 + (kc / 8) + kb * 4);
          a1[buf][kb] = ld_stream16(w1 + (kc / 8) + kb * 4);
        }
      }
    };
    __syncthreads();  // previous tile's readers are done with the staging buffers
    stage(0, 0);
    load_a(0, 0);
    if (n_steps > 1) { stage(kKC, 1); load_a(1, 1); }
#pragma unroll 1
    for (int s3 = 0; s3 < n_steps; s3 += 3) {
#pragma unroll
      for (int u = 0; u < 3; ++u) {
        const int s = s3 + u;
        if (s < n_steps) {
          if (s + 2 < n_steps) { stage((s + 2) * kKC, (u + 2) % 3); load_a(s + 2, (u + 2) % 3); }
          if (s + 2 < n_steps) cp_async_wait<2>(); else if (s + 1 < n_steps) cp_async_wait<1>(); else cp_async_wait<0>();
          __syncthreads();
          const int kblocks = min(kKC, K - s * kKC) / 32;
          const __nv_bfloat16* xb = xs + (size_t)u * ncols * kXPitch;
#pragma unroll
          for (int kb = 0; kb < KB; ++kb) {
            if (kb < kblocks) {
#pragma unroll
              for (int n = 0; n < NT; ++n) {
                const uint4 b = *reinterpret_cast<const uint4*>(xb + (size_t)(n * 8 + g) * kXPitch + kb * 32 + t * 8);
                mma_bf16(acc[n], a0[u][kb].x, a1[u][kb].x, a0[u][kb].y, a1[u][kb].y, b.x, b.y);
                mma_bf16(acc[n], a0[u][kb].z, a1[u][kb].z, a0[u][kb].w, a1[u][kb].w, b.z, b.w);
              }
            }
          }
          __syncthreads();
        }
      }
    }

    // ---- epilogue: lane (g, t) holds rows i0 (acc[.][0..1]) and i1 (acc[.][2..3]), columns 2t, 2t+1
    const int B = p.B;
    if (UP) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int i = half ? i1 : i0;
        const int j = half ? j1 : j0;
        if (i < n_rows) {
#pragma unroll
          for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int col = n * 8 + 2 * t + q;
              if (col < B) {
                const float h = p.a[(size_t)col * p.a_stride + j] * activation(p.act_up, acc[n][half * 2 + q]);
                static_cast<__nv_bfloat16*>(p.hmT)[(size_t)col * p.hm_stride + i] = __float2bfloat16(h);
              }
            }
        }
      }
    }
    if (!UP) {
      // Gate epilogue.  With split columns (LoPA) the value of token b is column b plus column b + B.
      // Tokens are spread over the accumulator tiles, so exchange through shared memory:
      // zt[row_in_tile][col] (fp32), one 128 x ncols tile per CTA, reusing the token staging buffer.
      float* zt = reinterpret_cast<float*>(smem_raw);
      const int pitch = ncols + 1;
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int q = 0; q < 4; ++q)
          zt[(size_t)(warp * 16 + g + (q >> 1) * 8) * pitch + n * 8 + 2 * t + (q & 1)] = acc[n][q];
      __syncthreads();
      // thread r < 128 finishes row r of the tile
      if (tid < 128) {
        const int i = tile * 128 + tid;
        if (i < n_rows) {
          const int j = i;  // the gate runs over all neurons in order
          const float bias = p.b_g ? p.b_g[j] : 0.f;
          const int gi = p.g_idx ? p.g_idx[j] : -1;
          const float sg = (p.g_sign && p.g_sign[j] < 0) ? -1.f : 1.f;
          bool fired = false;
          for (int b = 0; b < B; ++b) {
            float z = zt[(size_t)tid * pitch + b];
            if (p.split_cols) z += zt[(size_t)tid * pitch + b + B];
            if (gi >= 0) z += sg * __bfloat162float(static_cast<const __nv_bfloat16*>(p.xtok)[(size_t)b * p.xtok_stride + gi]);
            z += bias;
            fired |= z > 0.f;
            p.a_out[(size_t)b * p.a_stride + j] = activation(p.act, z);
          }
          if (p.flag) p.flag[j] = fired ? 1 : 0;
        }
      }
      __syncthreads();
    }
  }
}

// ------------------------------------------------------------------------------------------------
// n (fp32, [B][r]) -> bf16 high parts in columns [0, B) and low parts in columns [B, 2B) of X2 [2B][r].
__global__ void split_bf16_kernel(const float* n, int B, int r, int n_stride, __nv_bfloat16* x2) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  if (k >= r) return;
  const float v = n[(size_t)b * n_stride + k];
  const __nv_bfloat16 hi = __float2bfloat16(v);
  const __nv_bfloat16 lo = __float2bfloat16(v - __bfloat162float(hi));
  x2[(size_t)b * r + k] = hi;
  x2[(size_t)(B + b) * r + k] = lo;
}

// ------------------------------------------------------------------------------------------------
// Down projection.  grid = (D / 256, splits).  CTA (ds, sp) owns columns [256 ds, 256 ds + 256) and the
// union rows [lo, hi) of split sp; warp w owns columns 32 w .. 32 w + 31 (two 16-row M tiles of Y^T).
// Per step: 16 union rows x 256 columns of W_down (cp.async, 3 stages) and the matching 16 columns of
// HmT; A fragments come from ldmatrix.trans (the staged tile is [u][d], the operand is [d][u]).
template <int NT>
__global__ void __launch_bounds__(256) down_mma_kernel(const DownMmaParams p) {
  constexpr int kStages = kDownStages;
  constexpr int kWPitch = 256 + 8;  // bf16 elements: 528 bytes, odd multiple of 16 -> conflict-free ldmatrix
  constexpr int kHPitch = 16 + 8;   // bf16 elements per token row of the Hm stage (48 bytes)
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* ws = reinterpret_cast<__nv_bfloat16*>(smem_raw);                  // [kStages][16][kWPitch]
  __nv_bfloat16* hs = ws + (size_t)kStages * 16 * kWPitch;                          // [kStages][NT*8][kHPitch]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n_rows = p.count ? *p.count : p.R;
  const int d0 = blockIdx.x * 256;
  const int steps_total = (n_rows + 15) / 16;
  const int steps_per = (steps_total + gridDim.y - 1) / gridDim.y;
  const int s_lo = blockIdx.y * steps_per, s_hi = min(steps_total, s_lo + steps_per);
  const int ncols = NT * 8;

  float acc[2][NT][4];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[m][n][q] = 0.f;

  auto stage = [&](int s, int buf) {
    const int u0 = s * 16;
    // W_down rows: 16 rows x 512 bytes = 512 chunks of 16 bytes, two per thread
    for (int c = tid; c < 512; c += 256) {
      const int r = c >> 5, cc = c & 31;
      const int u = u0 + r;
      const bool valid = u < n_rows;
      int j = valid ? (p.idx ? p.idx[u] : u) : 0;
      if (!SFFN_IN_BOUNDS(j >= 0 && j < p.R, p.status, 31)) j = 0;
      cp_async16(ws + ((size_t)buf * 16 + r) * kWPitch + cc * 8,
                 static_cast<const __nv_bfloat16*>(p.W_down) + (size_t)j * p.D + d0 + cc * 8, valid);
    }
    // HmT columns u0..u0+15 for every token: ncols rows x 32 bytes = 2 chunks each
    for (int c = tid; c < ncols * 2; c += 256) {
      const int b = c >> 1, half = c & 1;
      const bool valid = b < p.B && u0 + half * 8 < n_rows;  // HmT is zero beyond n_rows (padded to 16)
      cp_async16(hs + ((size_t)buf * ncols + b) * kHPitch + half * 8,
                 static_cast<const __nv_bfloat16*>(p.hmT) + (size_t)(valid ? b : 0) * p.hm_stride + u0 + half * 8, valid);
    }
    cp_async_commit();
  };

  // One commit group per step, real or empty, so that "all but the newest kStages-1 groups are
  // complete" always means "step s has landed".
  for (int q = 0; q < kStages - 1; ++q) {
    if (s_lo + q < s_hi) stage(s_lo + q, q); else cp_async_commit();
  }
  for (int s = s_lo; s < s_hi; ++s) {
    const int buf = (s - s_lo) % kStages;
    if (s + kStages - 1 < s_hi) stage(s + kStages - 1, (s - s_lo + kStages - 1) % kStages); else cp_async_commit();
    cp_async_wait<kStages - 1>();
    __syncthreads();
    // B fragments: (k = u: 2t, 2t+1 | 2t+8, 2t+9 ; n = token g of tile n)
    uint32_t bf[NT][2];
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const __nv_bfloat16* hrow = hs + ((size_t)buf * ncols + n * 8 + g) * kHPitch;
      bf[n][0] = *reinterpret_cast<const uint32_t*>(hrow + 2 * t);
      bf[n][1] = *reinterpret_cast<const uint32_t*>(hrow + 2 * t + 8);
    }
#pragma unroll
    for (int m = 0; m < 2; ++m) {
      // A = transpose of the staged [16 u][16 d] block at columns warp*32 + m*16
      const int dcol = warp * 32 + m * 16;
      const int mat = lane >> 3, r8 = lane & 7;
      const __nv_bfloat16* src = ws + ((size_t)buf * 16 + (mat >> 1) * 8 + r8) * kWPitch + dcol + (mat & 1) * 8;
      uint32_t a0, a1, a2, a3;
      const uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(src));
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                   : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3)
                   : "r"(addr));
#pragma unroll
      for (int n = 0; n < NT; ++n) mma_bf16(acc[m][n], a0, a1, a2, a3, bf[n][0], bf[n][1]);
    }
    __syncthreads();
  }
  // partial[(split * B + b) * D + d]: lane holds d = dcol + g (+8), tokens 2t, 2t+1 of tile n
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int d = d0 + warp * 32 + m * 16 + g + (q >> 1) * 8;
        const int b = n * 8 + 2 * t + (q & 1);
        if (b < p.B && d < p.D) p.partial[((size_t)blockIdx.y * p.B + b) * p.D + d] = acc[m][n][q];
      }
}

template <int NT>
cudaError_t launch_rows_nt(bool up, const RowsMmaParams& p, int grid, cudaStream_t s) {
  const size_t stage_bytes = (size_t)3 * NT * 8 * kXPitch * sizeof(__nv_bfloat16);
  const size_t z_bytes = (size_t)128 * (NT * 8 + 1) * sizeof(float);
  const size_t smem = stage_bytes > z_bytes ? stage_bytes : z_bytes;
  if (up) {
    auto k = rows_mma_kernel<NT, true>;
    if (smem > 48 * 1024) cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    k<<<grid, 256, smem, s>>>(p);
  } else {
    auto k = rows_mma_kernel<NT, false>;
    if (smem > 48 * 1024) cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    k<<<grid, 256, smem, s>>>(p);
  }
  return cudaGetLastError();
}

template <int NT>
cudaError_t launch_down_nt(const DownMmaParams& p, dim3 grid, cudaStream_t s) {
  const size_t smem = (size_t)kDownStages * (16 * (256 + 8) + NT * 8 * (16 + 8)) * sizeof(__nv_bfloat16);
  auto k = down_mma_kernel<NT>;
  if (smem > 48 * 1024) cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  k<<<grid, 256, smem, s>>>(p);
  return cudaGetLastError();
}

int tiles_for(int cols) { return cols <= 8 ? 1 : cols <= 16 ? 2 : cols <= 32 ? 4 : cols <= 64 ? 8 : 16; }

}  // namespace

bool batched_mma_supported(int D, int K, int cols) { return D % 256 == 0 && K % 32 == 0 && cols >= 1 && cols <= 128; }

cudaError_t launch_rows_mma(bool up, const RowsMmaParams& p, int cols, int grid, cudaStream_t s) {
  switch (tiles_for(cols)) {
    case 1: return launch_rows_nt<1>(up, p, grid, s);
    case 2: return launch_rows_nt<2>(up, p, grid, s);
    case 4: return launch_rows_nt<4>(up, p, grid, s);
    case 8: return launch_rows_nt<8>(up, p, grid, s);
    default: return launch_rows_nt<16>(up, p, grid, s);
  }
}

cudaError_t launch_split_bf16(const float* n, int B, int r, int n_stride, void* x2, cudaStream_t s) {
  split_bf16_kernel<<<dim3((r + 255) / 256, B), 256, 0, s>>>(n, B, r, n_stride, static_cast<__nv_bfloat16*>(x2));
  return cudaGetLastError();
}

cudaError_t launch_down_mma(const DownMmaParams& p, int splits, cudaStream_t s) {
  const dim3 grid(p.D / 256, splits);
  switch (tiles_for(p.B)) {
    case 1: return launch_down_nt<1>(p, grid, s);
    case 2: return launch_down_nt<2>(p, grid, s);
    case 4: return launch_down_nt<4>(p, grid, s);
    default: return launch_down_nt<8>(p, grid, s);
  }
}

}  // namespace sffn
