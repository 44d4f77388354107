// Launchers of the tcgen05 (TMEM accumulator) kernels of the batched path (see umma_kernels.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sffn {

// Value of UmmaRowsParams::act that stores the raw products (no bias is usually given, no activation).
constexpr int kUmmaActIdentity = 3;

struct UmmaRowsParams {
  const void* W;         // [*, K] bf16 (or int8 / packed int4 codes, see qbits), rows selected by idx (or 0..R-1)
  int R, K;
  int qbits;             // 0: bf16 rows; 8 / 4: rows of weight codes, K * qbits / 8 bytes each, expanded to bf16 in
                         // shared memory; 1: int8 rows multiplied as int8 -- X then holds the tokens as int8 limbs (four
                         // rows per token, launch_token_limbs) and tok_scale their scales; 2: the same for int4 rows,
                         // whose nibbles are expanded to int8 (16 x the code) in shared memory
  const float* tok_scale;  // qbits = 1: scale of each token's limbs
  const float* w_scale;  // quantised rows: scale of row j of W (applied to its accumulator row), or null
  const float* out_scale;  // UP, quantised rows: scale of row j of the down matrix, folded into Hm, or null
  const int32_t* idx;    // UP: list of rows, or null
  const int32_t* count;  // UP: device length of the list, or null (= R)
  const uint32_t* words_in;  // UP, instead of idx / count: the gate kernel's "fired" bit masks (n_words of
  int n_words;               //   them, 4 per gate tile of gate_tile_rows rows); the kernel compacts them itself
  int gate_tile_rows;
  int gate_rows_per_word;    //   rows covered by one mask word: 32 for gate tiles of more than 64 rows, else 16
  int32_t* idx_out;          //   ... and writes the ascending list
  int32_t* count_out;        //   ... and its length
  int32_t* walk_all;         //   ... and 1 here when it walked every row instead of the list (the down kernel must too), else 0
  const void* X;         // token operand [cols][K] bf16, row stride x_stride (elements)
  int x_stride;
  int ncols_valid;
  int B;                 // tokens
  int split_cols;        // GATE: 1 = columns 2b, 2b+1 are the high / low bf16 parts of token b's vector
  const float* b_g;
  const int32_t* g_idx;
  const int8_t* g_sign;
  const void* xtok;      // tokens [B][.] bf16 for the fixed-matrix term
  int xtok_stride;
  int act;
  float* a_out;          // GATE: gate values a_out[b * a_stride + j]
  uint8_t* flag;         // GATE: [R] any token fires, or null
  uint32_t* words_out;   // GATE: the same as bit masks, word 4 * tile + epilogue warp, or null
  const float* a;        // UP: gate values
  int a_stride;
  void* hmT;             // UP: bf16 [B][hm_stride]
  int hm_stride;
  int act_up;            // UP: activation on the up projection (double activation), kUmmaActIdentity = none
  int32_t* status;       // device status word
  int npad, ring_bytes;  // filled by the launcher
  long long wait_cycles; // budget of every device-side wait (filled by the launcher)
  int drop_stage;        // test hook: CTA 0 of the gate kernel never copies the weights of this stage (-1: none)
};

struct UmmaDownParams {
  const void* W_down;    // [R, D] bf16 (or codes, see qbits; their row scales are already folded into hmT)
  int R, D;
  int qbits;             // 0: bf16 rows; 8 / 4: rows of weight codes
  const int32_t* idx;    // list of rows (readable up to the next multiple of 64 past its length), or null = all R rows
  const int32_t* count;  // device length of the list, or null (= R)
  const void* hmT;       // bf16 [B][hm_stride]; entries from the list's end to the next multiple of 64 are zero
  int hm_stride;         // multiple of 64
  int B;
  int splits;            // the list is cut into this many runs of 64-row blocks
  const int32_t* walk_all;  // device word: nonzero = walk every row of W_down instead of the list (set by the up kernel), or null
  float* partial;        // [splits][B][D]
  int32_t* status;
  int npad, stages;      // filled by the launcher
  long long wait_cycles; // budget of every device-side wait (filled by the launcher)
};

int umma_down_splits(int D, int sm_count, int max_splits);
bool umma_down_supported(int D, int cols);
cudaError_t launch_umma_down(UmmaDownParams p, cudaStream_t s);
bool umma_rows_supported(int K, int cols);
// Batches wide enough for the up kernel to consider walking every row instead of the union list.
bool umma_may_walk(int B);
bool umma_own_list_supported(int R, int sm_count);
void umma_gate_tiling(int R, int sm_count, int* tile_rows, int* n_tiles);
cudaError_t launch_umma_rows(bool up, UmmaRowsParams p, int cols, int sm_count, cudaStream_t s);
bool umma_rows_native_i8_supported(int K, int tokens);
// Tokens [B][K] bf16 as four int8 limbs each ([4 B][K], most significant first, 7 bits apart) and one scale per token.
cudaError_t launch_token_limbs(const void* x, int B, int K, int x_stride, void* limbs, float* scale, cudaStream_t s);
// The same for the LoPA vector n = RMSNorm(v) (or v), from fp32.
cudaError_t launch_rmsnorm_limbs(const float* v, int B, int r, int v_stride, const float* gain, float eps, bool use_rms,
                                 void* limbs, float* scale, cudaStream_t s);
cudaError_t launch_rmsnorm_split(const float* v, int B, int r, int v_stride, const float* gain, float eps,
                                 bool use_rms, void* x2, cudaStream_t s);

}  // namespace sffn
