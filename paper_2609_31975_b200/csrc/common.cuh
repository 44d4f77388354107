// Device helpers shared by the sparse-FFN kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sffn {

constexpr int kActRelu = 0;
constexpr int kActSqRelu = 1;
constexpr int kActRsPlus = 2;
constexpr int kActNone = 3;  // identity: internal stages that only need the raw products

// Activation of the gate (activation table of Sec. 3.1; squared RELU from the activation study).
// For all three, A(z) != 0 exactly when z > 0 in exact arithmetic; callers test z > 0.
// The R-S+ branch is kept out of line: `act` is the same for every thread, so the cheap activations then cost a
// compare and a max per element instead of a speculated exponential and division.
static __device__ __noinline__ float rsplus_of_nonnegative(float p) { return p / (1.f + __expf(-p)); }

__device__ __forceinline__ float activation(int act, float z) {
  if (act == kActNone) return z;
  const float p = fmaxf(z, 0.f);                 // 0 for z <= 0
  if (act == kActRelu) return p;
  if (act == kActSqRelu) return p * p;
  return rsplus_of_nonnegative(p);               // R-S+: z * sigmoid(z) on the non-negative side, 0 at 0
}

// Element traits: 16-byte vectors of the storage type, unpacked to fp32.
template <typename T>
struct Elem;

template <>
struct Elem<float> {
  static constexpr int kPerVec = 4;  // elements per 16 bytes
  __device__ __forceinline__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x);
    f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z);
    f[3] = __uint_as_float(v.w);
  }
  __device__ __forceinline__ static float to_float(float v) { return v; }
};

template <>
struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  // bf16 -> fp32 is a 16-bit shift: exact.
  __device__ __forceinline__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x << 16);
    f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16);
    f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16);
    f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16);
    f[7] = __uint_as_float(v.w & 0xffff0000u);
  }
  __device__ __forceinline__ static float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
};

// Streaming 16-byte load: weights are read once, so keep them out of L1.
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Programmatic dependent launch.  A kernel lets its successor in the stream start early
// (launch_dependents) and waits for its predecessor's completion and memory flush (wait) before it
// reads anything a predecessor may write and before its own first global write.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Host switch (diagnostics): false launches every kernel fully serialised.
inline bool& pdl_enabled() {
  static bool on = true;
  return on;
}

// Raises a kernel's dynamic shared-memory limit once per device (the attribute belongs to the device's copy of
// the kernel); `done` holds one bit per device ordinal.
template <typename K>
cudaError_t allow_dynamic_smem(K kernel, int bytes, unsigned long long& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) done |= bit;
  return e;
}

// Launch with the programmatic-stream-serialisation attribute: the kernel may begin while its
// predecessor in the stream is still running; its griddepcontrol.wait restores the ordering.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*k)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, k, args...);
}

}  // namespace sffn
