// Fused single-launch sparse FFN for one token (see fused_kernel.cu).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "sparse_ffn.h"

namespace sffn {

struct FusedCall {
  int wkind;  // kWF32 / kWBF16 / kWQ8: storage of the weights (tokens: fp32, bf16, bf16)
  const float* s_gate;  // kWQ8: row scales of the gate matrix (W_g or U), of V, of W_up and of W_down
  const float* s_V;
  const float* s_up;
  const float* s_down;
  int D, H;
  const void* x;
  const sffn_gate* gate;
  const float* b_g;
  const void* W_up;
  const void* W_down;
  int act;
  int act_up;
  bool gated_skip;       // double activation on the sparse route: W_down rows only where h != 0
  float* y;
  bool dense;
  int engine;        // sffn_gate_engine of the handle
  int r_max;         // the handle's largest LoPA rank (workspace layout)
  void* workspace;   // fused_workspace_bytes() bytes, zeroed at handle creation
  int32_t* status;   // device status word
  uint8_t* flag;     // [H] "neuron fired" bytes (sparse calls)
  bool flag_or;      // the bytes are only ever set (a batch run token by token: the union of the tokens' fired sets)
  int sm_count;
};

size_t fused_workspace_bytes(int D, int H, int r_max);
size_t fused_tagged_partials_offset(int D, int r_max);  // where the tensor-core kernel's tagged partials start
bool fused_supported(int wkind, int D, int H, int B, const sffn_gate* gate, int sm_count);
void debug_fused_plan(int wkind, int D, int H, int K, bool lopa, int sm_count, int* out);
cudaError_t launch_fused(const FusedCall& c, cudaStream_t s, int* launched);

// The same call with the gate on the tensor cores (fused_tc_kernel.cu): bf16 rows, standard gate, D a multiple of
// 64 and at least 1024.  launch_fused takes this route by itself when it applies.
bool fused_tc_supported(int wkind, int D, int H, int B, const sffn_gate* gate, int sm_count);
cudaError_t launch_fused_tc(const FusedCall& c, cudaStream_t s, int* launched);

// Test hooks (see the "test hooks" section of sparse_ffn.h).
struct FusedTestKnobs {
  bool pdl = true;               // programmatic dependent launch between calls
  int tensor_gate = -1;          // 1 / 0: tensor-core gate wherever it applies / nowhere; -1: the handle's engine decides
  long long wait_cycles = 1LL << 31;  // budget of every device-side wait (about one second)
  bool poison_list = false;      // debug builds: the CUDA-core path corrupts its list's first entry (bounds-check test)
  int drop_stage = -1;           // batched gate kernel: CTA 0 never copies this stage's weights (its wait runs out)
  int skip_arrival_cta = -1;     // this CTA does not count itself as finished: the summing CTAs' wait runs out
  int ring_S = 0, ring_NA = 0;   // tensor-core gate: ring split override (0 = planned)
  int l2_hints = 2;              // tensor-core gate: bit 0 weights evict-first, bit 1 partials evict-last
  int ring_E = -1;               // tensor-core gate: gate stages parked in the act ring at the start (-1 = planned)
  long long* trace = nullptr;    // SFFN_TRACE builds: [grid][16] time stamps
};
FusedTestKnobs& fused_test_knobs();

}  // namespace sffn
