// Launchers of the batched tensor-core path (see batched_kernels.cu).  bf16 storage only.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sffn {

struct RowsMmaParams {
  const void* W;         // [*, K] bf16, rows selected by idx (or 0..R-1)
  int R, K;
  const int32_t* idx;    // UP: list of rows, or null
  const int32_t* count;  // UP: device length of the list, or null (= R)
  const void* X;         // token operand [cols][K] bf16, row stride x_stride
  int x_stride;
  int ncols_valid;       // columns of X that exist (others are zero-filled)
  int B;                 // tokens
  int split_cols;        // GATE: 1 = columns [B, 2B) are low parts to add onto columns [0, B)
  // GATE epilogue
  const float* b_g;
  const int32_t* g_idx;
  const int8_t* g_sign;
  const void* xtok;      // tokens [B][.] bf16 for the fixed-matrix term
  int xtok_stride;
  int act;
  float* a_out;          // gate values a_out[b * a_stride + j]
  uint8_t* flag;         // [R] any token fires, or null
  // UP epilogue
  const float* a;        // gate values a[b * a_stride + j]
  int a_stride;
  void* hmT;             // bf16 [B][hm_stride]: h of token b for list position u
  int hm_stride;
  int act_up;            // activation on the up projection (double activation), kActNone = none
  int32_t* status;       // device status block (debug builds record a list entry outside [0, R) here), or null
};

struct DownMmaParams {
  const void* W_down;    // [H, D] bf16
  int R, D;
  const int32_t* idx;
  const int32_t* count;
  const void* hmT;       // bf16 [B][hm_stride]
  int hm_stride;
  int B;
  float* partial;        // [splits][B][D]
  int32_t* status;       // device status block (debug builds), or null
};

bool batched_mma_supported(int D, int K, int cols);
cudaError_t launch_rows_mma(bool up, const RowsMmaParams& p, int cols, int grid, cudaStream_t s);
cudaError_t launch_split_bf16(const float* n, int B, int r, int n_stride, void* x2, cudaStream_t s);
cudaError_t launch_down_mma(const DownMmaParams& p, int splits, cudaStream_t s);

}  // namespace sffn
