// General multi-kernel path of the sparse gated FFN: any batch size, fp32 or bf16 storage.
//
//   rowdot_kernel   z = W vec (+ bias + fixed-matrix term), activation, per-neuron "fires" flag
//                   (Eq. 1 gate; also the two stages of the LoPA gate, Eq. 3)
//   rmsnorm_kernel  n = gain * v / sqrt(mean(v^2) + eps)          (LoPA in practice, Sec. 3.3)
//   compact_kernel  ascending list of the neurons whose flag is set (16 flags per thread, block scan)
//   updown_kernel   u_j = W_up[j].x, h_j = a_j u_j, y_part += h_j W_down[j] over the listed rows only
//                   (sparse execution, Sec. 3.1; union of the batch's active sets, Sec. 5.4)
//   reduce_kernel   y = sum of the per-CTA partials in CTA order (deterministic)
//
// All accumulation is fp32.  No atomics on floating-point data anywhere.
#include "general_kernels.cuh"

#include "common.cuh"

namespace sffn {

// ------------------------------------------------------------------------------------------------
// Row-times-vector kernel.  One warp owns two rows at a time and walks them in 16-byte steps with
// four steps in flight per row; the NB vectors sit in shared memory as fp32.
template <typename T, typename VT, int NB, bool GATE>
__global__ void __launch_bounds__(256) rowdot_kernel(const RowDotParams p) {
  extern __shared__ float svec[];  // [NB][K]
  constexpr int EPV = Elem<T>::kPerVec;
  using X = typename TokenOf<T>::type;  // storage type of the tokens
  const int K = p.K;
  pdl_launch_dependents();
  pdl_wait();  // the vectors (and, for the gate, the flag / value buffers) belong to earlier kernels until here
  for (int b = 0; b < NB; ++b) {
    const VT* v = static_cast<const VT*>(p.vec) + (size_t)b * p.vec_stride;
    for (int k = threadIdx.x; k < K; k += blockDim.x) svec[b * K + k] = Elem<VT>::to_float(v[k]);
  }
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = K / EPV;
  const size_t row_bytes = row_bytes_of<T>(K);
  const char* Wb = static_cast<const char*>(p.W);
  constexpr int UNROLL = 4;

  for (int pair = blockIdx.x * 8 + warp; pair * 2 < p.R; pair += gridDim.x * 8) {
    const int j0 = pair * 2;
    const bool has1 = j0 + 1 < p.R;
    const uint4* w0 = reinterpret_cast<const uint4*>(Wb + (size_t)j0 * row_bytes);
    const uint4* w1 = reinterpret_cast<const uint4*>(Wb + (size_t)(has1 ? j0 + 1 : j0) * row_bytes);
    float acc0[NB], acc1[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc0[b] = acc1[b] = 0.f;

    for (int c0 = lane; c0 < nvec; c0 += 32 * UNROLL) {
      uint4 a[UNROLL], c[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int cc = c0 + u * 32;
        if (cc < nvec) {
          a[u] = ld_stream16(w0 + cc);
          c[u] = ld_stream16(w1 + cc);
        } else {
          a[u] = make_uint4(0, 0, 0, 0);
          c[u] = make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int cc = c0 + u * 32;
        if (cc < nvec) {
          float fa[EPV], fc[EPV];
          Elem<T>::unpack(a[u], fa);
          Elem<T>::unpack(c[u], fc);
#pragma unroll
          for (int b = 0; b < NB; ++b) {
            const float4* xs = reinterpret_cast<const float4*>(svec + b * K + cc * EPV);
#pragma unroll
            for (int q = 0; q < EPV / 4; ++q) {
              const float4 xv = xs[q];
              acc0[b] = fmaf(fa[4 * q + 0], xv.x, acc0[b]);
              acc0[b] = fmaf(fa[4 * q + 1], xv.y, acc0[b]);
              acc0[b] = fmaf(fa[4 * q + 2], xv.z, acc0[b]);
              acc0[b] = fmaf(fa[4 * q + 3], xv.w, acc0[b]);
              acc1[b] = fmaf(fc[4 * q + 0], xv.x, acc1[b]);
              acc1[b] = fmaf(fc[4 * q + 1], xv.y, acc1[b]);
              acc1[b] = fmaf(fc[4 * q + 2], xv.z, acc1[b]);
              acc1[b] = fmaf(fc[4 * q + 3], xv.w, acc1[b]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      acc0[b] = warp_sum(acc0[b]);
      acc1[b] = warp_sum(acc1[b]);
    }
    if (lane == 0) {
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int j = j0 + rr;
        if (j >= p.R) break;
        // int8 rows: the dot product of the codes times the row's scale
        const float sc = (TokenOf<T>::kScaled && p.row_scale) ? p.row_scale[j] : 1.f;
        if (!GATE) {
#pragma unroll
          for (int b = 0; b < NB; ++b) p.out[(size_t)b * p.out_stride + j] = (rr ? acc1[b] : acc0[b]) * sc;
        } else {
          const float bias = p.b_g ? p.b_g[j] : 0.f;
          const int gi = p.g_idx ? p.g_idx[j] : -1;
          const float sg = (p.g_sign && p.g_sign[j] < 0) ? -1.f : 1.f;
          bool any = false;
#pragma unroll
          for (int b = 0; b < NB; ++b) {
            float z = (rr ? acc1[b] : acc0[b]) * sc;
            if (gi >= 0)
              z += sg * Elem<X>::to_float(static_cast<const X*>(p.x)[(size_t)b * p.x_stride + gi]);
            z += bias;
            any |= z > 0.f;
            p.out[(size_t)b * p.out_stride + j] = activation(p.act, z);
          }
          if (p.flag) p.flag[j] = (p.flag_or ? p.flag[j] : 0) | (any ? 1 : 0);
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// RMSNorm over the r entries of v, one CTA per token.
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* v, float* n, const float* gain,
                                                      int r, int stride, float eps) {
  __shared__ float red[8];
  pdl_launch_dependents();
  pdl_wait();
  const float* vb = v + (size_t)blockIdx.x * stride;
  float* nb = n + (size_t)blockIdx.x * stride;
  float ss = 0.f;
  for (int k = threadIdx.x; k < r; k += blockDim.x) ss = fmaf(vb[k], vb[k], ss);
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float inv = rsqrtf(tot / (float)r + eps);
  for (int k = threadIdx.x; k < r; k += blockDim.x) nb[k] = (gain ? gain[k] : 1.f) * vb[k] * inv;
}

// ------------------------------------------------------------------------------------------------
// Stream compaction of the flags into an ascending index list.  One CTA of 1024 threads walks the
// flags in chunks of 16384: a thread reads its 16 consecutive flags with one 16-byte load, a warp scan
// and a scan over the 32 warp totals give its first position, and it writes its set indices in order.
__global__ void __launch_bounds__(1024) compact_kernel(const uint8_t* flag, int H, int32_t* idx,
                                                       int32_t* count) {
  __shared__ int warp_total[32];
  pdl_launch_dependents();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(flag) & 15u) == 0;
  int base = 0;
  for (int c0 = 0; c0 < H; c0 += 16384) {
    const int j0 = c0 + threadIdx.x * 16;
    uint32_t bits = 0;  // bit q: flag[j0 + q] is set
    if (vec_ok && j0 + 16 <= H) {
      const uint4 v = *reinterpret_cast<const uint4*>(flag + j0);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int b = 0; b < 4; ++b)
          if ((w[i] >> (8 * b)) & 0xffu) bits |= 1u << (4 * i + b);
    } else {
      for (int q = 0; q < 16; ++q)
        if (j0 + q < H && flag[j0 + q] != 0) bits |= 1u << q;
    }
    const int c = __popc(bits);
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += t;
    }
    if (lane == 31) warp_total[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < 32; ++w) {
      const int t = warp_total[w];
      before += w < warp ? t : 0;
      total += t;
    }
    int pos = base + before + incl - c;
    while (bits) {
      const int q = __ffs(bits) - 1;
      bits &= bits - 1;
      idx[pos++] = j0 + q;
    }
    base += total;
    __syncthreads();  // warp_total is reused by the next chunk
  }
  if (threadIdx.x == 0) *count = base;
}

// ------------------------------------------------------------------------------------------------
// Fused up / down projection over a list of rows.  CTA g owns the contiguous slice
// [n*g/G, n*(g+1)/G) of the list.  16 warps: each takes one listed row, dots W_up[j] with the NB
// tokens, scales by the gate values and parks h in shared memory; then all 512 threads stream the
// same 16 rows of W_down, each thread owning CPT 16-byte column chunks of y for all NB tokens.
template <typename T, int NB, int CPT>
__global__ void __launch_bounds__(512) updown_kernel(const UpDownParams p) {
  extern __shared__ float svec[];  // [NB][D] tokens as fp32
  __shared__ float hbuf[16][NB];
  __shared__ int lbuf[16];  // row contributes (some token has h != 0): otherwise its W_down row is not read
  __shared__ int jbuf[16];
  constexpr int EPV = Elem<T>::kPerVec;
  const int D = p.D;
  pdl_launch_dependents();
  pdl_wait();
  using X = typename TokenOf<T>::type;
  for (int b = 0; b < NB; ++b) {
    const X* xb = static_cast<const X*>(p.x) + (size_t)b * p.x_stride;
    for (int k = threadIdx.x; k < D; k += blockDim.x) svec[b * D + k] = Elem<X>::to_float(xb[k]);
  }
  const int n = p.count ? *p.count : p.H;
  const int lo = (int)((long long)n * blockIdx.x / gridDim.x);
  const int hi = (int)((long long)n * (blockIdx.x + 1) / gridDim.x);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = D / EPV;
  const size_t row_bytes = row_bytes_of<T>(D);
  const char* Wu = static_cast<const char*>(p.W_up);
  const char* Wd = static_cast<const char*>(p.W_down);

  float acc[CPT][EPV][NB];
#pragma unroll
  for (int c = 0; c < CPT; ++c)
#pragma unroll
    for (int e = 0; e < EPV; ++e)
#pragma unroll
      for (int b = 0; b < NB; ++b) acc[c][e][b] = 0.f;
  __syncthreads();

  for (int base = lo; base < hi; base += 16) {
    const int i = base + warp;
    const bool valid = i < hi;
    int j = valid ? (p.idx ? p.idx[i] : i) : 0;
    if (!SFFN_IN_BOUNDS(j >= 0 && j < p.H, p.status, 10)) j = 0;
    float u[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) u[b] = 0.f;
    if (valid) {
      const uint4* w = reinterpret_cast<const uint4*>(Wu + (size_t)j * row_bytes);
      for (int c0 = lane; c0 < nvec; c0 += 32 * 4) {
        uint4 a[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          a[q] = (c0 + q * 32 < nvec) ? ld_stream16(w + c0 + q * 32) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int cc = c0 + q * 32;
          if (cc < nvec) {
            float fa[EPV];
            Elem<T>::unpack(a[q], fa);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
              const float* xs = svec + b * D + cc * EPV;
#pragma unroll
              for (int e = 0; e < EPV; ++e) u[b] = fmaf(fa[e], xs[e], u[b]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) u[b] = warp_sum(u[b]);
    if (lane == 0) {
      jbuf[warp] = j;
      bool live = false;
      // int8 rows: u = s_up[j] (codes . x); the scale of the W_down row rides on the coefficient h
      const float su = (TokenOf<T>::kScaled && valid) ? p.s_up[j] : 1.f;
      const float sd = (TokenOf<T>::kScaled && valid) ? p.s_down[j] : 1.f;
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        // h = A(z) * A_3(u): double activation of Sec. 3.3 when act_up names one, Eq. 1 otherwise
        const float h = valid ? p.a[(size_t)b * p.a_stride + j] * activation(p.act_up, u[b] * su) * sd : 0.f;
        hbuf[warp][b] = h;
        live |= h != 0.f;
      }
      lbuf[warp] = live ? 1 : 0;
    }
    __syncthreads();
    const int rows = min(16, hi - base);
    for (int r0 = 0; r0 < rows; r0 += 4) {
      uint4 wv[4][CPT];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4* w = reinterpret_cast<const uint4*>(Wd + (size_t)jbuf[min(r0 + q, 15)] * row_bytes);
#pragma unroll
        for (int c = 0; c < CPT; ++c) {
          const int cc = threadIdx.x + c * 512;
          wv[q][c] = (r0 + q < rows && lbuf[r0 + q] && cc < nvec) ? ld_stream16(w + cc) : make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (r0 + q < rows && lbuf[r0 + q]) {
#pragma unroll
          for (int c = 0; c < CPT; ++c) {
            float fw[EPV];
            Elem<T>::unpack(wv[q][c], fw);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
              const float h = hbuf[r0 + q][b];
#pragma unroll
              for (int e = 0; e < EPV; ++e) acc[c][e][b] = fmaf(h, fw[e], acc[c][e][b]);
            }
          }
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int c = 0; c < CPT; ++c) {
    const int cc = threadIdx.x + c * 512;
    if (cc < nvec) {
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        float* dst = p.partial + ((size_t)blockIdx.x * NB + b) * D + (size_t)cc * EPV;
#pragma unroll
        for (int e = 0; e < EPV; e += 4)
          *reinterpret_cast<float4*>(dst + e) =
              make_float4(acc[c][e][b], acc[c][e + 1][b], acc[c][e + 2][b], acc[c][e + 3][b]);
      }
    }
  }
}

// y[b][d] = sum_g partial[g][b][d], g ascending.  One thread per four columns.
__global__ void __launch_bounds__(256) reduce_kernel(const float* partial, int G, int NB, int D,
                                                     float* y, int y_stride) {
  pdl_launch_dependents();
  pdl_wait();
  const int q = blockIdx.x * blockDim.x + threadIdx.x;  // float4 index within [NB][D/4]
  const int per = D / 4;
  if (q >= NB * per) return;
  const int b = q / per, d4 = q % per;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  const float4* src = reinterpret_cast<const float4*>(partial) + (size_t)b * per + d4;
  const size_t step = (size_t)NB * per;
#pragma unroll 8
  for (int g = 0; g < G; ++g) {
    const float4 v = src[(size_t)g * step];
    s.x += v.x;
    s.y += v.y;
    s.z += v.z;
    s.w += v.w;
  }
  *reinterpret_cast<float4*>(y + (size_t)b * y_stride + (size_t)d4 * 4) = s;
}

// Copy of n16 16-byte units from mapped pinned host memory into a staging buffer of the workspace, without a
// copy-engine operation between two kernels of the stream.  The source is host data that was complete when
// the call was made, so its first 4 units per thread are read into registers at once, while the predecessors
// in the stream still run; nothing is written before they have finished.
__global__ void __launch_bounds__(256) copy16_kernel(const uint4* src, uint4* dst, size_t n16) {
  pdl_launch_dependents();
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint4 v[4];
#pragma unroll
  for (int k = 0; k < 4; ++k)
    if (i0 + k * stride < n16) v[k] = src[i0 + k * stride];
  pdl_wait();
#pragma unroll
  for (int k = 0; k < 4; ++k)
    if (i0 + k * stride < n16) dst[i0 + k * stride] = v[k];
  for (size_t i = i0 + 4 * stride; i < n16; i += stride) dst[i] = src[i];
}

// Glue between two FFN calls of a layer loop: out = T(resid + alpha * y), four elements per thread.
template <typename T>
__global__ void __launch_bounds__(256) residual_cast_kernel(const float* y, const T* resid, float alpha, T* out, int n4) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float4 v = reinterpret_cast<const float4*>(y)[i];
  float r[4];
  if (sizeof(T) == 4) {
    const float4 q = reinterpret_cast<const float4*>(resid)[i];
    r[0] = q.x; r[1] = q.y; r[2] = q.z; r[3] = q.w;
  } else {
    const uint2 q = reinterpret_cast<const uint2*>(resid)[i];
    r[0] = __uint_as_float(q.x << 16); r[1] = __uint_as_float(q.x & 0xffff0000u);
    r[2] = __uint_as_float(q.y << 16); r[3] = __uint_as_float(q.y & 0xffff0000u);
  }
  const float o[4] = {fmaf(alpha, v.x, r[0]), fmaf(alpha, v.y, r[1]), fmaf(alpha, v.z, r[2]), fmaf(alpha, v.w, r[3])};
  if (sizeof(T) == 4) {
    reinterpret_cast<float4*>(out)[i] = make_float4(o[0], o[1], o[2], o[3]);
  } else {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(o[0], o[1]), hi = __floats2bfloat162_rn(o[2], o[3]);
    uint2 w;
    w.x = *reinterpret_cast<const uint32_t*>(&lo);
    w.y = *reinterpret_cast<const uint32_t*>(&hi);
    reinterpret_cast<uint2*>(out)[i] = w;
  }
}

// ------------------------------------------------------------------------------------------------
// Host-side launchers.
template <typename T, typename VT, int NB>
static cudaError_t launch_rowdot_t(const RowDotParams& p, bool gate, int grid, cudaStream_t s) {
  const size_t smem = (size_t)NB * p.K * sizeof(float);
  if (gate) {
    auto k = rowdot_kernel<T, VT, NB, true>;
    if (smem > 48 * 1024) {
      const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    return launch_pdl(k, dim3(grid), dim3(256), smem, s, p);
  } else {
    auto k = rowdot_kernel<T, VT, NB, false>;
    if (smem > 48 * 1024) {
      const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    return launch_pdl(k, dim3(grid), dim3(256), smem, s, p);
  }
}

template <typename T, typename VT>
static cudaError_t launch_rowdot_nb(const RowDotParams& p, int nb, bool gate, int grid, cudaStream_t s) {
  switch (nb) {
    case 1: return launch_rowdot_t<T, VT, 1>(p, gate, grid, s);
    case 2: return launch_rowdot_t<T, VT, 2>(p, gate, grid, s);
    default: return launch_rowdot_t<T, VT, 4>(p, gate, grid, s);
  }
}

cudaError_t launch_rowdot(int wkind, bool vec_is_f32, int nb, bool gate, const RowDotParams& p,
                          int sm_count, cudaStream_t s) {
  const int blocks_needed = (p.R + 15) / 16;  // 8 warps x 2 rows per pass
  const int grid = blocks_needed < sm_count * 4 ? (blocks_needed > 0 ? blocks_needed : 1) : sm_count * 4;
  if (wkind == kWQ8) {
    return vec_is_f32 ? launch_rowdot_nb<int8_t, float>(p, nb, gate, grid, s)
                      : launch_rowdot_nb<int8_t, __nv_bfloat16>(p, nb, gate, grid, s);
  }
  if (wkind == kWQ4) {
    return vec_is_f32 ? launch_rowdot_nb<q4_t, float>(p, nb, gate, grid, s)
                      : launch_rowdot_nb<q4_t, __nv_bfloat16>(p, nb, gate, grid, s);
  }
  if (wkind == kWBF16) {
    return vec_is_f32 ? launch_rowdot_nb<__nv_bfloat16, float>(p, nb, gate, grid, s)
                      : launch_rowdot_nb<__nv_bfloat16, __nv_bfloat16>(p, nb, gate, grid, s);
  }
  return launch_rowdot_nb<float, float>(p, nb, gate, grid, s);
}

cudaError_t launch_rmsnorm(const float* v, float* n, const float* gain, int r, int stride, float eps,
                           int B, cudaStream_t s) {
  return launch_pdl(rmsnorm_kernel, dim3(B), dim3(256), 0, s, v, n, gain, r, stride, eps);
}

// union[idx[i]] = 1 for the listed neurons: accumulates the fired sets of the chunks of a batch that is run in parts.
__global__ void __launch_bounds__(256) mark_union_kernel(const int32_t* idx, const int32_t* count, int H, uint8_t* u) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = *count;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int j = idx[i];
    if (j >= 0 && j < H) u[j] = 1;
  }
}

cudaError_t launch_mark_union(const int32_t* idx, const int32_t* count, int H, uint8_t* u, cudaStream_t s) {
  return launch_pdl(mark_union_kernel, dim3(32), dim3(256), 0, s, idx, count, H, u);
}

cudaError_t launch_compact(const uint8_t* flag, int H, int32_t* idx, int32_t* count, cudaStream_t s) {
  return launch_pdl(compact_kernel, dim3(1), dim3(1024), 0, s, flag, H, idx, count);
}

template <typename T, int NB, int CPT>
static cudaError_t launch_updown_t(const UpDownParams& p, int grid, cudaStream_t s) {
  const size_t smem = (size_t)NB * p.D * sizeof(float);
  auto k = updown_kernel<T, NB, CPT>;
  if (smem > 48 * 1024) {
    const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  return launch_pdl(k, dim3(grid), dim3(512), smem, s, p);
}

template <typename T>
static cudaError_t launch_updown_d(const UpDownParams& p, int nb, int grid, cudaStream_t s) {
  const int nvec = p.D / Elem<T>::kPerVec;
  const int cpt = nvec <= 512 ? 1 : nvec <= 1024 ? 2 : 4;
#define SFFN_UD(NBV, CPTV) \
  if (nb == NBV && cpt == CPTV) return launch_updown_t<T, NBV, CPTV>(p, grid, s);
  SFFN_UD(1, 1) SFFN_UD(1, 2) SFFN_UD(1, 4) SFFN_UD(2, 1) SFFN_UD(2, 2) SFFN_UD(2, 4)
  SFFN_UD(4, 1) SFFN_UD(4, 2)
#undef SFFN_UD
  return cudaErrorInvalidValue;
}

int updown_max_tokens(int wkind, int D) {
  const int nvec = D / weight_epv(wkind);
  if (wkind == kWQ8) return nvec > 1024 ? 0 : nvec > 512 ? 2 : 4;  // 16 accumulators per chunk and token
  if (wkind == kWQ4) return nvec > 512 ? 0 : 2;                    // 32 accumulators per chunk and token
  if (nvec > 2048) return 0;
  return nvec > 1024 ? 2 : 4;
}

cudaError_t launch_updown(int wkind, int nb, const UpDownParams& p, int grid, cudaStream_t s) {
  if (wkind == kWQ8) {
    const int nvec = p.D / 16;
    if (nvec <= 512) {
      if (nb == 1) return launch_updown_t<int8_t, 1, 1>(p, grid, s);
      if (nb == 2) return launch_updown_t<int8_t, 2, 1>(p, grid, s);
      if (nb == 4) return launch_updown_t<int8_t, 4, 1>(p, grid, s);
    } else if (nvec <= 1024) {
      if (nb == 1) return launch_updown_t<int8_t, 1, 2>(p, grid, s);
      if (nb == 2) return launch_updown_t<int8_t, 2, 2>(p, grid, s);
    }
    return cudaErrorInvalidValue;
  }
  if (wkind == kWQ4) {
    if (p.D / 32 <= 512) {
      if (nb == 1) return launch_updown_t<q4_t, 1, 1>(p, grid, s);
      if (nb == 2) return launch_updown_t<q4_t, 2, 1>(p, grid, s);
    }
    return cudaErrorInvalidValue;
  }
  return wkind == kWBF16 ? launch_updown_d<__nv_bfloat16>(p, nb, grid, s) : launch_updown_d<float>(p, nb, grid, s);
}

cudaError_t launch_residual_cast(bool bf16, const float* y, const void* resid, float alpha, void* out, int n,
                                 cudaStream_t s) {
  const int n4 = n / 4;
  const dim3 grid((n4 + 255) / 256);
  if (bf16)
    return launch_pdl(residual_cast_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, y,
                      static_cast<const __nv_bfloat16*>(resid), alpha, static_cast<__nv_bfloat16*>(out), n4);
  return launch_pdl(residual_cast_kernel<float>, grid, dim3(256), 0, s, y, static_cast<const float*>(resid), alpha,
                    static_cast<float*>(out), n4);
}

cudaError_t launch_copy16(const void* src, void* dst, size_t bytes, cudaStream_t s) {
  const size_t n16 = bytes / 16;
  const int grid = (int)((n16 + 255) / 256 < 64 ? (n16 + 255) / 256 : 64);
  return launch_pdl(copy16_kernel, dim3(grid < 1 ? 1 : grid), dim3(256), 0, s, static_cast<const uint4*>(src),
                    static_cast<uint4*>(dst), n16);
}

cudaError_t launch_reduce(const float* partial, int G, int NB, int D, float* y, int y_stride,
                          cudaStream_t s) {
  const int total = NB * (D / 4);
  return launch_pdl(reduce_kernel, dim3((total + 255) / 256), dim3(256), 0, s, partial, G, NB, D, y, y_stride);
}

}  // namespace sffn
