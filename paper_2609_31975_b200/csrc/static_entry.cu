// sparse_ffn_forward_static: the sparse FFN for callers that can neither allocate device memory nor
// bring a workspace.  Its scratch (gate values, fired flags, index list, per-CTA partial sums) lives
// in a file-scope __device__ array inside this library; every GPU that loads the library holds those
// ~4.3 MB until the process exits.  The work itself is done by the general-path kernels.
#include <cuda_runtime.h>

#include <mutex>

#include "general_kernels.cuh"
#include "sparse_ffn.h"

namespace {

constexpr int kMaxD = SFFN_STATIC_MAX_D;
constexpr int kMaxH = SFFN_STATIC_MAX_H;
constexpr int kGrid = 128;  // CTAs of the up/down kernel = number of partial sums
constexpr int kMaxDevices = 64;

// Carve-up of the scratch array (all offsets multiples of 256 bytes).
constexpr size_t kOffCount = 0;                                   // int32: length of the index list
constexpr size_t kOffAct = 256;                                   // float [kMaxH]: gate values a_j
constexpr size_t kOffFlag = kOffAct + (size_t)kMaxH * 4;          // uint8 [kMaxH]: neuron fired
constexpr size_t kOffIdx = kOffFlag + (size_t)kMaxH;              // int32 [kMaxH]: ascending list
constexpr size_t kOffPartial = kOffIdx + (size_t)kMaxH * 4;       // float [kGrid][kMaxD]
constexpr size_t kScratchBytes = kOffPartial + (size_t)kGrid * kMaxD * 4;

// In host code this name is only a handle for the runtime's symbol table, not a device address:
// the address every kernel receives comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

std::mutex g_setup_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {};
int g_sm_count[kMaxDevices] = {};

// Once per device, with that device current: resolve the array's device address.
int setup_current_device(int* dev_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SFFN_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return SFFN_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      return SFFN_ERR_CUDA;
    g_sm_count[dev] = sms;
    g_scratch_ptr[dev] = static_cast<unsigned char*>(ptr);
  }
  *dev_out = dev;
  return SFFN_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int sparse_ffn_forward_static(const void* x, const void* W_g, const float* b_g, const void* W_up,
                                         const void* W_down, int D, int H, int dtype, int act, float* y,
                                         void* stream) {
  using namespace sffn;
  if (!x || !W_g || !W_up || !W_down || !y) return SFFN_ERR_INVALID_ARG;
  if (dtype != SFFN_F32 && dtype != SFFN_BF16) return SFFN_ERR_INVALID_ARG;
  if (act < SFFN_ACT_RELU || act > SFFN_ACT_RSPLUS) return SFFN_ERR_INVALID_ARG;
  if (D < 1 || H < 1) return SFFN_ERR_INVALID_ARG;
  if (D > kMaxD || H > kMaxH) return SFFN_ERR_UNSUPPORTED;  // beyond the built-in scratch: use a handle
  const bool bf16 = dtype == SFFN_BF16;
  const size_t esz = bf16 ? 2 : 4;
  if ((D * esz) % 16 || updown_max_tokens(bf16, D) == 0) return SFFN_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(W_g) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(y))
    return SFFN_ERR_UNSUPPORTED;
  int dev = 0;
  const int rc = setup_current_device(&dev);
  if (rc != SFFN_OK) return rc;
  unsigned char* s = g_scratch_ptr[dev];
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  int32_t* count = reinterpret_cast<int32_t*>(s + kOffCount);
  float* a = reinterpret_cast<float*>(s + kOffAct);
  uint8_t* flag = s + kOffFlag;
  int32_t* idx = reinterpret_cast<int32_t*>(s + kOffIdx);
  float* partial = reinterpret_cast<float*>(s + kOffPartial);

  // The array keeps the previous call's contents.  Everything a call reads it has written first
  // (a[0..H), flag[0..H), the list up to its new length, all kGrid partial rows); only the list
  // length is cleared explicitly so that a failed launch cannot leave a stale length behind.
  if (cudaMemsetAsync(count, 0, sizeof(int32_t), st) != cudaSuccess) return SFFN_ERR_CUDA;

  RowDotParams g{};
  g.W = W_g; g.R = H; g.K = D;
  g.vec = x; g.vec_stride = D;
  g.out = a; g.out_stride = H;
  g.b_g = b_g;
  g.x = x; g.x_stride = D;
  g.act = act;
  g.flag = flag; g.flag_or = 0;
  if (launch_rowdot(bf16, !bf16, 1, true, g, g_sm_count[dev], st) != cudaSuccess) return SFFN_ERR_CUDA;
  if (launch_compact(flag, H, idx, count, st) != cudaSuccess) return SFFN_ERR_CUDA;
  UpDownParams u{};
  u.W_up = W_up; u.W_down = W_down;
  u.x = x; u.x_stride = D;
  u.a = a; u.a_stride = H;
  u.idx = idx; u.count = count;
  u.H = H; u.D = D;
  u.partial = partial;
  u.act_up = SFFN_ACT_NONE;
  if (launch_updown(bf16, 1, u, kGrid, st) != cudaSuccess) return SFFN_ERR_CUDA;
  if (launch_reduce(partial, kGrid, 1, D, y, D, st) != cudaSuccess) return SFFN_ERR_CUDA;
  return SFFN_OK;
}
