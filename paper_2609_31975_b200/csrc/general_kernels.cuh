// Launchers of the general multi-kernel path (see general_kernels.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sffn {

struct RowDotParams {
  const void* W;     // [R, K] storage dtype
  int R, K;
  const void* vec;   // [NB][K] with stride vec_stride (elements); storage dtype or fp32
  int vec_stride;
  float* out;        // out[b * out_stride + j]
  int out_stride;
  // gate epilogue only
  const float* b_g;       // [R] or null
  const int32_t* g_idx;   // [R] or null: column of x added to the pre-activation
  const int8_t* g_sign;   // [R] or null
  const void* x;          // [NB][.] tokens in storage dtype (fixed-matrix term)
  int x_stride;
  int act;
  uint8_t* flag;          // [R] or null: 1 where any of the NB tokens fires
  int flag_or;            // 0: overwrite flag, 1: OR into it (later token chunks)
  const float* row_scale; // int8 rows: [R] scale of each row; null = 1
};

struct UpDownParams {
  const void* W_up;    // [H, D]
  const void* W_down;  // [H, D]
  const void* x;       // [NB][D] storage dtype, stride x_stride
  int x_stride;
  const float* a;      // gate values a[b * a_stride + j]
  int a_stride;
  const int32_t* idx;  // list of rows, or null = all rows 0..H-1
  const int32_t* count;  // device length of idx, or null = H
  int H, D;
  float* partial;      // [grid][NB][D]
  int act_up;          // activation on the up projection (double activation), kActNone = none
  const float* s_up;   // int8 rows: [H] row scales of W_up and W_down
  const float* s_down;
  int32_t* status;     // device status block (debug builds record a row index outside [0, H) here), or null
};

// wkind: kWF32 / kWBF16 / kWQ8 (common.cuh); tokens are fp32, bf16, bf16 respectively.
cudaError_t launch_rowdot(int wkind, bool vec_is_f32, int nb, bool gate, const RowDotParams& p,
                          int sm_count, cudaStream_t s);
cudaError_t launch_rmsnorm(const float* v, float* n, const float* gain, int r, int stride, float eps,
                           int B, cudaStream_t s);
cudaError_t launch_compact(const uint8_t* flag, int H, int32_t* idx, int32_t* count, cudaStream_t s);
cudaError_t launch_mark_union(const int32_t* idx, const int32_t* count, int H, uint8_t* union_flags, cudaStream_t s);
// Largest token chunk (4, 2 or 0 = unsupported D) the up/down kernel takes at this D.
int updown_max_tokens(int wkind, int D);
cudaError_t launch_updown(int wkind, int nb, const UpDownParams& p, int grid, cudaStream_t s);
cudaError_t launch_residual_cast(bool bf16, const float* y, const void* resid, float alpha, void* out, int n,
                                 cudaStream_t s);
cudaError_t launch_copy16(const void* src, void* dst, size_t bytes, cudaStream_t s);
cudaError_t launch_reduce(const float* partial, int G, int NB, int D, float* y, int y_stride,
                          cudaStream_t s);

}  // namespace sffn
