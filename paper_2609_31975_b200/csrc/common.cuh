// Device helpers shared by the sparse-FFN kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sffn {

// Debug builds (-DSFFN_DEBUG, `python -m paper_2609_31975_b200.build --debug`): an index that is about to address
// global memory through a list or a computed row number is checked first.  A violation puts SFFN_ERR_BOUNDS into the
// device status word and the number of the check into word 4 of the status block, and the caller skips or clamps the
// access; nothing traps.  In release builds the macro is the constant true and the checks compile away.
#ifdef SFFN_DEBUG
__device__ __forceinline__ bool in_bounds_or_record(bool ok, int32_t* status, int site) {
  if (!ok && status) {
    status[4] = site;
    atomicCAS(status, 0, 6 /* SFFN_ERR_BOUNDS */);
  }
  return ok;
}
#define SFFN_IN_BOUNDS(cond, status, site) ::sffn::in_bounds_or_record((cond), (status), (site))
#else
#define SFFN_IN_BOUNDS(cond, status, site) true
#endif

constexpr int kActRelu = 0;
constexpr int kActSqRelu = 1;
constexpr int kActRsPlus = 2;
constexpr int kActNone = 3;  // identity: internal stages that only need the raw products
constexpr int kActSilu = 4;  // z * sigmoid(z) on both sides: only ever A_3 on the up projection (it is not sparse)

// Activation of the gate (activation table of Sec. 3.1; squared RELU from the activation study).
// For all three, A(z) != 0 exactly when z > 0 in exact arithmetic; callers test z > 0.
// The R-S+ branch is kept out of line: `act` is the same for every thread, so the cheap activations then cost a
// compare and a max per element instead of a speculated exponential and division.
static __device__ __noinline__ float rsplus_of_nonnegative(float p) { return p / (1.f + __expf(-p)); }

__device__ __forceinline__ float activation(int act, float z) {
  if (act == kActNone) return z;
  if (act == kActSilu) return rsplus_of_nonnegative(z);  // the same expression on the whole axis (-0 for z -> -inf)
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

// Two fp32 operations in one instruction (sm_100 packed fp32): d = a * b + c and d = a + b, element-wise on pairs.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
  return d;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}

// int8 codes of weight-only quantisation (one fp32 scale per row, applied by the caller of unpack to the
// finished dot product or to the row's coefficient).  Tokens that meet such weights are bf16.
// code -> fp32 without an integer conversion: with the sign bit flipped the byte is u = code + 128 in 0..255;
// placed in the low mantissa byte of 2^23 it reads 2^23 + u exactly, and one subtraction of 2^23 + 128 leaves
// the code.
template <>
struct Elem<int8_t> {
  static constexpr int kPerVec = 16;
  // four codes of one 32-bit word as two pairs (codes 0, 1 and codes 2, 3)
  __device__ __forceinline__ static void unpack4(uint32_t w, float2& lo, float2& hi) {
    w ^= 0x80808080u;
    const float2 bias = make_float2(-8388736.f, -8388736.f);
    lo = add2(make_float2(__uint_as_float(__byte_perm(w, 0x4b000000u, 0x7650)),
                          __uint_as_float(__byte_perm(w, 0x4b000000u, 0x7651))), bias);
    hi = add2(make_float2(__uint_as_float(__byte_perm(w, 0x4b000000u, 0x7652)),
                          __uint_as_float(__byte_perm(w, 0x4b000000u, 0x7653))), bias);
  }
  __device__ __forceinline__ static void unpack4(uint32_t w, float* f) {
    float2 lo, hi;
    unpack4(w, lo, hi);
    f[0] = lo.x; f[1] = lo.y; f[2] = hi.x; f[3] = hi.y;
  }
  __device__ __forceinline__ static void unpack(const uint4& v, float* f) {
    unpack4(v.x, f);
    unpack4(v.y, f + 4);
    unpack4(v.z, f + 8);
    unpack4(v.w, f + 12);
  }
};

// 4-bit codes of weight-only quantisation: two's complement in [-8, 7], two per byte, the even column in the low
// nibble, one fp32 scale per row (applied by the caller, as for int8).  A tag type: rows are addressed in bytes.
// With the sign bits of all eight nibbles of a word flipped each nibble is u = code + 8 in 0..15; the even and the odd
// nibbles are separated into bytes, a byte goes into the low mantissa byte of 2^23 and one subtraction of 2^23 + 8
// leaves the code.
struct q4_t {};
template <>
struct Elem<q4_t> {
  static constexpr int kPerVec = 32;
  // eight codes of one 32-bit word, in column order
  __device__ __forceinline__ static void unpack8(uint32_t w, float* f) {
    w ^= 0x88888888u;
    const uint32_t even = w & 0x0f0f0f0fu, odd = (w >> 4) & 0x0f0f0f0fu;  // columns 0,2,4,6 and 1,3,5,7 as bytes
    const float2 bias = make_float2(-8388616.f, -8388616.f);
#pragma unroll
    for (int b = 0; b < 4; b += 2) {
      const float2 e = add2(make_float2(__uint_as_float(__byte_perm(even, 0x4b000000u, 0x7650 + b)),
                                        __uint_as_float(__byte_perm(even, 0x4b000000u, 0x7651 + b))), bias);
      const float2 o = add2(make_float2(__uint_as_float(__byte_perm(odd, 0x4b000000u, 0x7650 + b)),
                                        __uint_as_float(__byte_perm(odd, 0x4b000000u, 0x7651 + b))), bias);
      f[2 * b] = e.x; f[2 * b + 1] = o.x; f[2 * b + 2] = e.y; f[2 * b + 3] = o.y;
    }
  }
  __device__ __forceinline__ static void unpack(const uint4& v, float* f) {
    unpack8(v.x, f);
    unpack8(v.y, f + 8);
    unpack8(v.z, f + 16);
    unpack8(v.w, f + 24);
  }
};

// Packed fp32 pairs kept in 64-bit registers from unpacking to the final sum, so that no instruction is spent on moving
// halves in and out of pairs between the packed operations.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ unsigned long long fma2_b64(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2_b64(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float sum_halves(unsigned long long v) {
  float lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
  return lo + hi;
}
// Eight 4-bit codes of one word times eight entries of a vector given as four packed pairs (x0,x1) .. (x6,x7), added
// onto a packed running sum.
__device__ __forceinline__ unsigned long long dot8_q4(uint32_t w, const unsigned long long* xp, unsigned long long acc) {
  w ^= 0x88888888u;
  const uint32_t even = w & 0x0f0f0f0fu, odd = (w >> 4) & 0x0f0f0f0fu;
  const unsigned long long bias = pack2(-8388616.f, -8388616.f);
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const unsigned long long pr = pack2(__uint_as_float(__byte_perm(even, 0x4b000000u, 0x7650 + b)),
                                        __uint_as_float(__byte_perm(odd, 0x4b000000u, 0x7650 + b)));
    acc = fma2_b64(add2_b64(pr, bias), xp[b], acc);
  }
  return acc;
}

// Bytes of a row of n elements of storage type T (16 / kPerVec bytes per element: half a byte for 4-bit codes).
template <typename T>
__host__ __device__ constexpr size_t row_bytes_of(size_t n) { return n * 16 / Elem<T>::kPerVec; }

// Storage type of the tokens that go with weights of type T, and whether rows of T carry a scale.
template <typename T>
struct TokenOf { using type = T; static constexpr bool kScaled = false; };
template <>
struct TokenOf<int8_t> { using type = __nv_bfloat16; static constexpr bool kScaled = true; };
template <>
struct TokenOf<q4_t> { using type = __nv_bfloat16; static constexpr bool kScaled = true; };

// Weight storage kinds as the launchers take them (0 and 1 coincide with "is bf16" of older call sites).
constexpr int kWF32 = 0, kWBF16 = 1, kWQ8 = 2, kWQ4 = 3;
// elements per 16 bytes of a weight row
__host__ __device__ constexpr int weight_epv(int wkind) { return wkind == kWF32 ? 4 : wkind == kWBF16 ? 8 : wkind == kWQ8 ? 16 : 32; }

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
