// Fused sparse gated FFN for one token on B200 (sm_100a).
//
// One kernel per call: one persistent CTA per SM owns a share ("slab") of the H neurons and runs the whole
// of the paper's sparse execution scheme (Sec. 3.1) on it without leaving the SM:
//
//   gate producers two threads (two warps) stream the slab's gate rows (W_1, or U for the LoPA gate) into a
//                  shared-memory ring with bulk asynchronous copies (TMA, mbarrier complete_tx).
//                  They depend on nothing but free ring slots, so HBM stays busy from the first
//                  cycle of the CTA to the last gate row.
//   gate warps     each owns ring slots: z_j = row . vec + b_g[j] (+ fixed-matrix term),
//                  a_j = A(z_j), and publishes "fired" (z_j > 0) per neuron.
//   act producers  two warps walk the published results in ascending neuron order and queue the
//                  W_up / W_down rows of the neurons that fired into a second ring.
//   act warps      four warps (for the LoPA gate two groups of four on alternate rounds, and four gate warps)
//                  consume the second ring in order: u_j = W_up[j] . x (reduction over the group),
//                  h_j = a_j u_j, y_part += h_j W_down[j]; each thread keeps its own column slice of y_part in
//                  registers and writes it out once.
//
// The first CTAs to finish sum the per-CTA partials in CTA order (deterministic, no float atomics): every partial
// value is stored with the call's number in the same 64-bit word, so the summing CTAs need no counter or fence.
// Weights are fp32, bf16, int8 codes or packed 4-bit codes with one fp32 scale per row (bf16 token).
// For the LoPA gate (Eq. 3, Sec. 3.3) the rank-r stage v = V x is spread over the CTAs of the main
// kernel, exchanged through global memory as tagged values (bounded re-reads) and normalised (RMSNorm)
// into shared memory, with the U rows already sitting in the ring.
//
// Calls are chained with programmatic dependent launch: a kernel lets its successor start early
// and waits (griddepcontrol.wait) only before it touches anything a predecessor may write.  Weights
// are read before that wait -- they are parameters, not results -- so the next call's gate stream
// starts on an SM the moment the previous call's CTA leaves it.
// Every mbarrier / flag wait is bounded by a cycle budget; when it runs out the kernel records
// SFFN_ERR_TIMEOUT in the status word and every role winds down.
#include "fused_kernel.cuh"

#include "common.cuh"

namespace sffn {

namespace {

// Warp roles.  One thread can issue a bulk copy only every few hundred cycles, which caps a single
// producer near 4 TB/s over the whole GPU; two gate producers (alternate ring slots) and two act
// producers (W_up row / W_down row of the same slot) lift that above the HBM rate.
constexpr int kGateProducers = 2;                          // warps 0, 1
constexpr int kFirstActProducer = kGateProducers;          // warps 2, 3
constexpr int kActProducers = 2;
constexpr int kTokenLimbs = 2;      // int8 limbs of the token (quantised rows, standard gate)
constexpr int kFirstGateWarp = kFirstActProducer + kActProducers;
constexpr int kGateWarps = 8;
constexpr int kFirstActWarp = kFirstGateWarp + kGateWarps;
constexpr int kActWarps = 4;
constexpr int kThreads = 32 * (kFirstActWarp + kActWarps);  // 512
constexpr int kStageBase = 32 * kGateProducers;  // first thread that takes part in staging the token
constexpr int kStageThreads = kThreads - kStageBase;
constexpr int kMaxGrid = 256;
constexpr int kSmemBudget = 227 * 1024;

struct FusedParams {
  int D, H, K;  // K = length of a gate row: D (standard) or r (LoPA)
  const void* Wgate;  // [H, K]
  const void* W_up;
  const void* W_down;
  const void* x;
  const float* b_g;
  const int32_t* g_idx;
  const int8_t* g_sign;
  const float* gain;
  int use_rmsnorm;
  float eps;
  const void* V;      // LoPA: [r, D]
  unsigned long long* vtag;  // LoPA: [r] exchange buffer for v = V x, every value tagged with the call's number
  // Two arrival counters in the workspace, monotonic over calls.  Every call adds exactly gridDim.x to each and
  // calls on one workspace are serialised, so a CTA derives its call's first and last value from what its own
  // atomicAdd returned: nothing depends on a host-side count, and a captured launch can be replayed.
  unsigned long long* done_counter;  // CTAs that have written their partial of y
  float* y;                          // [D] result, written by the last CTAs to finish
  int act, dense;
  int act_up;        // activation on the up projection (double activation, Sec. 3.3); kActNone = Eq. 1
  const float* s_gate;  // int8 rows only: one scale per row of the gate matrix [H], of V [r], of W_up and W_down [H]
  const float* s_V;
  const float* s_up;
  const float* s_down;
  unsigned long long* partial;  // [grid][row] per-CTA partials of y, each value paired with the call's number
  uint32_t* epoch_word;         // number of calls completed on this workspace
  uint8_t* flag;
  int flag_or;       // 1 = flags are only set, never cleared (later tokens of a batch run token by token)
  int32_t* status;
  int rows_per_gate_slot, gate_slot_bytes, n_gate_slots, act_slot_bytes, n_act_slots, slab_max;
  int act_extra;     // LoPA: act slots inside the gate ring, used once the gate is done (0 = none)
  int act_groups;    // act groups: 1, LoPA 2, or 3 when the gate warps join as a group of their own after the gate
  int act_used;      // act slots the ring protocol cycles through: n_act_slots + act_extra, or fewer (see plan())
  int v_in_smem;     // LoPA: this CTA's rows of V are copied into the (idle) act ring at the start of the call
  int gate_workers;  // warps that take gate slots, slot s going to worker s % gate_workers: the gate warps, and for
                     // the LoPA gate also act warps (a ring slot that is reused always belongs to the same worker)
  int gate_warps;    // gate warps in use; n_gate_slots is a multiple of it, so a ring slot always
                     // belongs to the same warp and its phases are consumed strictly in order
  long long wait_cycles;  // budget of every wait below (about one second unless a test shortens it)
  int skip_arrival_cta;   // test hook: this CTA does not count itself as finished (-1: none)
  long long* trace;       // SFFN_TRACE builds: [grid][16] time stamps, or null
};

// Shared-memory carve-up, identical on host and device.
struct SmemLayout {
  int gate_ring, act_ring, sx, sn, aval, slot_a, red, ctl, bars, row_params, row_scales, slot_scales, gated_bars, gated_vals, xlimb, total;
  __host__ __device__ SmemLayout(int D, int K, bool lopa, int n_gate_slots, int gate_slot_bytes,
                                 int n_act_slots, int act_slot_bytes, int slab_max, bool scaled, int act_extra = 0,
                                 bool gated = false, bool limbs = false) {
    int off = 0;
    auto take = [&](int bytes) {
      int o = off;
      off = (off + bytes + 127) / 128 * 128;
      return o;
    };
    gate_ring = take(n_gate_slots * gate_slot_bytes);
    act_ring = take(n_act_slots * act_slot_bytes);
    sx = take(D * 4);
    sn = take(lopa ? K * 4 : 0);
    aval = take(slab_max * 4);
    slot_a = take((n_act_slots + act_extra) * 4);
    red = take(6 * (2 * 4 + 1) * 4);  // two buffers per act group (four warps each), up to three groups
    ctl = take(8 * 4);
    bars = take(2 * (n_gate_slots + n_act_slots + act_extra) * 8 + 8);  // + one for the CTA's rows of V (LoPA)
    row_params = take((lopa || scaled) ? (1 + (lopa ? 2 : 0) + (scaled ? 1 : 0)) * slab_max * 4 : 0);  // per-neuron gate parameters
    row_scales = take(scaled ? 2 * slab_max * 4 : 0);     // int8 rows: scales of the slab's W_up / W_down rows
    slot_scales = take(scaled ? 2 * (n_act_slots + act_extra) * 4 : 0);  // the same two for the row in each act slot
    // gated variant (W_down rows only where h != 0): the act ring is cut into single rows (2 per act slot), each with
    // up to three barriers and three values
    gated_bars = take(gated ? 3 * 2 * n_act_slots * 8 : 0);
    gated_vals = take(gated ? 3 * 2 * n_act_slots * 4 : 0);
    // quantised rows, standard gate: the token as two int8 limbs [2][D] for the integer dot products (after 128 spare
    // bytes), then one scale per 16 entries
    xlimb = take(limbs ? 128 + kTokenLimbs * D + D / 4 : 0);
    total = off;
  }
};

enum Ctl { kAbort = 0, kRank = 1, kGateDone = 2 };

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bulk asynchronous copy global -> shared, completion counted in bytes on an mbarrier.
// Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int threads) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// `site` says which wait gave up (diagnostics: word 3 of the status block holds site + 256 * CTA of the last one).
__device__ __forceinline__ void raise_timeout(volatile int* ctl, int32_t* status, int site) {
  ctl[kAbort] = 1;
  status[3] = site + 256 * (int)blockIdx.x;
  atomicExch(status, (int32_t)SFFN_ERR_TIMEOUT);
}

// After a wait has run out the CTA winds down.  Copies it has issued may still be in flight; they end within
// microseconds, so a thread that leaves an aborting CTA lets that time pass first: shared memory is only given back
// when nothing can write to it any more.
__device__ __forceinline__ void abort_grace(volatile int* ctl) {
  if (ctl[kAbort])
    for (int i = 0; i < 50; ++i) __nanosleep(1000);
}

// Bounded wait on an mbarrier phase.  try_wait parks the thread in hardware for a short,
// implementation-defined time, so waiting warps do not steal issue slots from working ones; the
// cycle budget is checked between attempts.  False when it ran out or the CTA is aborting.
template <bool kBackoff = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* ctl, int32_t* status,
                                          long long budget, int site) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      if (mbar_try(bar, parity)) return true;
      if (kBackoff) __nanosleep(100);  // a producer waiting for a free slot: keep out of the working warps' way
    }
    if (ctl[kAbort]) return false;
    if (clock64() - t0 > budget) {
      raise_timeout(ctl, status, site);
      return false;
    }
  }
}

// Position of element k of a vector inside its shared-memory copy.  For 8-element (bf16) and 16-element (int8)
// chunks the quarters of every chunk are stored in two / four planes so that a warp's float4 reads are conflict-free.
template <int EPV>
__device__ __forceinline__ int vec_pos(int k, int len) {
  if (EPV == 4) return k;
  const int c = k / EPV, q = k % EPV;
  return (q >> 2) * (len / (EPV / 4)) + 4 * c + (q & 3);
}

// Dot product of one 16-byte chunk of weights with the matching entries of the staged vector.
template <typename T>
__device__ __forceinline__ float chunk_dot(const uint4& w, const float* vec, int c, int nvec, float acc) {
  constexpr int EPV = Elem<T>::kPerVec;
  float f[EPV];
  Elem<T>::unpack(w, f);
  const float4 lo = reinterpret_cast<const float4*>(vec)[c];
  acc = fmaf(f[0], lo.x, acc);
  acc = fmaf(f[1], lo.y, acc);
  acc = fmaf(f[2], lo.z, acc);
  acc = fmaf(f[3], lo.w, acc);
#pragma unroll
  for (int q = 1; q < EPV / 4; ++q) {
    const float4 hi = reinterpret_cast<const float4*>(vec)[q * nvec + c];
    acc = fmaf(f[4 * q + 0], hi.x, acc);
    acc = fmaf(f[4 * q + 1], hi.y, acc);
    acc = fmaf(f[4 * q + 2], hi.z, acc);
    acc = fmaf(f[4 * q + 3], hi.w, acc);
  }
  return acc;
}

// Two int8 rows' chunks against the same entries of the staged vector (read once), packed fp32 arithmetic: the
// sums are kept as pairs (even / odd elements).
__device__ __forceinline__ void chunk_dot2_q8(const uint4& wa, const uint4& wb, const float* vec, int c, int nvec,
                                              float2& acc_a, float2& acc_b) {
  const uint32_t a[4] = {wa.x, wa.y, wa.z, wa.w}, b[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 v = reinterpret_cast<const float4*>(vec)[q * nvec + c];
    float2 lo, hi;
    Elem<int8_t>::unpack4(a[q], lo, hi);
    acc_a = fma2(lo, make_float2(v.x, v.y), acc_a);
    acc_a = fma2(hi, make_float2(v.z, v.w), acc_a);
    Elem<int8_t>::unpack4(b[q], lo, hi);
    acc_b = fma2(lo, make_float2(v.x, v.y), acc_b);
    acc_b = fma2(hi, make_float2(v.z, v.w), acc_b);
  }
}
// A small integer (|a| < 2^22) as fp32 without a conversion instruction: 1.5 x 2^23 + a is exact, and so is the
// subtraction.
__device__ __forceinline__ float small_int_as_float(int a) { return __int_as_float(0x4B400000 + a) - 12582912.f; }
// One int8 chunk against the staged vector, packed.
__device__ __forceinline__ float2 chunk_dot_q8(const uint4& w, const float* vec, int c, int nvec, float2 acc) {
  const uint32_t a[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 v = reinterpret_cast<const float4*>(vec)[q * nvec + c];
    float2 lo, hi;
    Elem<int8_t>::unpack4(a[q], lo, hi);
    acc = fma2(lo, make_float2(v.x, v.y), acc);
    acc = fma2(hi, make_float2(v.z, v.w), acc);
  }
  return acc;
}

// One value of a partial with the number of the call that wrote it: a naturally aligned 64-bit word is written and
// read as a whole, so a reader that finds the expected number has the value that belongs to it (no fence, no flag
// round trip between writer and reader).
__device__ __forceinline__ unsigned long long tagged(float v, uint32_t epoch) {
  return ((unsigned long long)epoch << 32) | (unsigned long long)__float_as_uint(v);
}
__device__ __forceinline__ void st_tagged2(unsigned long long* dst, unsigned long long a, unsigned long long b, uint64_t pol) {
  asm volatile("st.global.cg.L2::cache_hint.v2.b64 [%0], {%1, %2}, %3;" ::"l"(dst), "l"(a), "l"(b), "l"(pol) : "memory");
}
__device__ __forceinline__ void ld_tagged2(const unsigned long long* src, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.global.cg.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(src) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

#ifdef SFFN_TRACE
__device__ __forceinline__ long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return (long long)t;
}
#define SFFN_GSTAMP(slot)                                                    \
  do {                                                                       \
    if (p.trace) p.trace[(size_t)blockIdx.x * 16 + (slot)] = global_ns();    \
  } while (0)

#define SFFN_STAMP(slot)                                                          \
  do {                                                                            \
    if (p.trace) p.trace[(size_t)blockIdx.x * 16 + (slot)] = clock64() - t_entry; \
  } while (0)
#else
#define SFFN_GSTAMP(slot) do { } while (0)
#define SFFN_STAMP(slot) do { } while (0)
#endif

// GATED (double activation, standard gate, sparse route): the W_down row of a fired neuron is fetched only once
// h_j = a_j A_3(u_j) is known and is not zero (the "gated" sparsity site of the paper's table of sites).  The act ring
// is then two rings of single rows: the first act producer fills the "up" ring with W_up rows as before; the act
// warps dot two of them per round, publish the two h and release the rows at once; the second act producer follows
// the published h in order and copies the W_down rows that are needed into the "down" ring, which the act warps
// consume one round behind (whatever is left after the stop marker).  Rows are added in the same order as in the
// other variant and a skipped row would have added zeros, so y is bitwise the same.
template <typename T, int CPT, bool LOPA, bool GATED = false>
__global__ void __launch_bounds__(kThreads, 1) fused_ffn_kernel(const FusedParams p) {
  static_assert(!(GATED && LOPA), "the gated variant is built for the standard gate");
  // Warp roles: 2 gate producers, 2 act producers, then gate warps and act warps.  The standard gate needs its
  // eight gate warps to keep up with the stream; the LoPA gate is short (r elements per row), the call's time
  // is then set by the up/down rows, so eight of the twelve workers are act warps there.
  constexpr int kAW = LOPA ? 8 : 4;                         // act warps
  constexpr int kGW = kGateWarps + kActWarps - kAW;         // gate warps
  constexpr int kFAW = kFirstGateWarp + kGW;                // first act warp
  constexpr int kAT = 32 * kAW;                             // act threads
  // The act warps work in groups of four; a group takes whole rounds (two ring slots) by itself.  With the short LoPA
  // gate the act stage is what a call waits for, and one round is a chain of latencies (shared-memory loads, shuffles,
  // a barrier, loads again: 0.7 us for two rows however many warps share it), so two groups on alternate rounds double
  // the rows per microsecond; each keeps its own sums, added through shared memory at the end.
  constexpr int kGroups = LOPA ? 2 : 1;
  constexpr int kGAW = kAW / kGroups;                       // warps of a group
  constexpr int kGT = 32 * kGAW;                            // threads of a group
  static_assert(kGAW == 4, "the up projection's sum over a group's warps is written out for four");
  static_assert(kGW >= 2, "gate warps");

  extern __shared__ __align__(128) unsigned char smem[];
#ifdef SFFN_TRACE
  const long long t_entry = clock64();
#endif
  pdl_launch_dependents();
  if (threadIdx.x == 0) SFFN_GSTAMP(10);
  constexpr int EPV = Elem<T>::kPerVec;
  using X = typename TokenOf<T>::type;             // storage type of the token
  constexpr bool kScaled = TokenOf<T>::kScaled;    // int8 rows: every row comes with an fp32 scale
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  const int D = p.D, K = p.K;
  // Act slots: NAown in the act ring, plus (short LoPA gate) p.act_extra more that lie in the gate ring and come into
  // use once every gate row has been consumed -- from then on the rows of fired neurons are all that is left to
  // fetch, and how many of them are in flight sets how fast they come.
  const int NG = p.n_gate_slots, NAown = p.n_act_slots, NA = p.act_used;
  // int8 rows under a standard gate: dot products in integers (dp4a) against the token split into int8 limbs
  constexpr bool kLimbs = EPV == 16 && !LOPA;
  // int4 rows under a standard gate: the same, with every nibble used as the byte 16 x code (the nibble moved to the
  // upper half of a byte) and the limbs of even and odd columns stored apart, as the two masks of a word deliver them
  constexpr bool kLimbs4 = EPV == 32 && !LOPA;
  // Two limbs (dp4a is the scarce resource: 16-odd lanes per clock and SM; a third limb cost a third more gate time):
  // an error of 3e-5 of the chunk's largest |x| per entry, about 1e-4 of a typical |z| or |u|.
  constexpr int kGateLimbs = kTokenLimbs;
  constexpr int kUpLimbs = kTokenLimbs;
  const SmemLayout L(D, K, LOPA, NG, p.gate_slot_bytes, NAown, p.act_slot_bytes, p.slab_max, kScaled, p.act_extra, GATED, kLimbs || kLimbs4);

  unsigned char* gate_ring = smem + L.gate_ring;
  unsigned char* act_ring = smem + L.act_ring;
  auto act_slot = [&](int sl) -> unsigned char* {
    return sl < NAown ? act_ring + (size_t)sl * p.act_slot_bytes : gate_ring + (size_t)(sl - NAown) * p.act_slot_bytes;
  };
  float* sx = reinterpret_cast<float*>(smem + L.sx);
  float* sn = reinterpret_cast<float*>(smem + L.sn);
  // One word per neuron of the slab, written once by a gate warp and polled by the act producers:
  // all ones = gate not computed yet, 0x80000000 = not fired, otherwise the bits of a_j >= 0 (fired).
  // A single 32-bit store publishes value and state together, so no fence is needed on either side
  // (a fence in the producers would also wait for their bulk copies in flight).
  volatile uint32_t* row_state = reinterpret_cast<volatile uint32_t*>(smem + L.aval);
  float* slot_a = reinterpret_cast<float*>(smem + L.slot_a);  // per act slot: gate value, < 0 = stop
  // Per-neuron gate parameters of the slab, fetched before the dependency wait (parameters, like the weights), where
  // a neuron has several of them (LoPA: bias, fixed-matrix column and sign; int8 rows: bias and scale): the gate warps
  // then never wait for a global load between two ring slots.  The standard gate on fp32 / bf16 rows has the bias
  // alone: its gate warps load it per slot, before they wait for the slot's rows (measured 0.15 us faster per call
  // than the table at 4096 x 14336).
  constexpr bool kTables = LOPA || kScaled;
  float* row_bias = reinterpret_cast<float*>(smem + L.row_params);             // [slab_max] b_g
  float* row_sg = row_bias + p.slab_max;                                       // LoPA: sign of the fixed-matrix entry
  int* row_gi = reinterpret_cast<int*>(row_sg + p.slab_max);                   // LoPA: its column, -1 = none
  float* row_gscale = row_bias + (LOPA ? 3 : 1) * p.slab_max;                  // int8 rows: scale of the gate row
  float* row_su = reinterpret_cast<float*>(smem + L.row_scales);  // [slab_max] scale of the W_up row, then
  float* row_sd = row_su + p.slab_max;                            // [slab_max] of the W_down row (int8 only)
  float* slot_su = reinterpret_cast<float*>(smem + L.slot_scales);
  float* slot_sd = slot_su + NA;
  float* red = reinterpret_cast<float*>(smem + L.red);
  const float* xsc = reinterpret_cast<const float*>(smem + L.xlimb + 128 + kTokenLimbs * D);  // scale of the limbs of chunk c
  const uint4* xl = reinterpret_cast<const uint4*>(smem + L.xlimb + 128);  // limb l of chunk c: xl[l * nvecD + c]
  volatile int* ctl = reinterpret_cast<volatile int*>(smem + L.ctl);
  const uint32_t bars = smem_u32(smem + L.bars);
  const uint32_t full_gate = bars, empty_gate = bars + 8 * NG;
  const uint32_t full_act = bars + 16 * NG, empty_act = bars + 16 * NG + 8 * NA;
  const uint32_t v_bar = bars + 16 * (NG + NA);
  // Gated variant: NU rows of the act ring for W_up rows, ND for W_down rows (about a third: half of the fired neurons
  // need one, and it stays for one round trip only).
  const int NH = 2 * NAown, ND = NH / 3 < 2 ? 2 : NH / 3, NU = NH - ND;

  const uint32_t full_up = smem_u32(smem + L.gated_bars), empty_up = full_up + 8 * NU, h_ready = empty_up + 8 * NU;
  const uint32_t full_dn = h_ready + 8 * NU, empty_dn = full_dn + 8 * ND;
  float* up_a = reinterpret_cast<float*>(smem + L.gated_vals);       // [NU] gate value of the row, < 0 = stop marker
  volatile float* up_h = up_a + NU;                                  // [NU] h of the row, published by the act warps
  volatile float* dn_h = up_a + 2 * NU;                              // [ND] h of the row in a down slot

  const int nvecD = D / EPV, nvecK = K / EPV;
  const size_t row_bytes = row_bytes_of<T>(D);
  const size_t gate_row_bytes = row_bytes_of<T>(K);
  const int nr = p.rows_per_gate_slot;
  // Neurons are dealt to the CTAs in blocks of nr consecutive rows, round robin: CTA c owns the
  // blocks c, c + G, c + 2G, ...  One block = one gate ring slot.  Compared with one contiguous slab
  // per CTA this spreads neighbouring neurons, whose firing can be correlated (LoPA rows that share a
  // column of the fixed matrix), over different CTAs.  Local row l of this CTA is row l % nr of its
  // block l / nr; only the globally last block can be short, and it is the last block of its owner.
  const int n_blocks = (p.H + nr - 1) / nr;
  const int n_gslots = cta < n_blocks ? (n_blocks - cta + G - 1) / G : 0;
  const int slab_rows =
      n_gslots == 0 ? 0 : (n_gslots - 1) * nr + min(nr, p.H - (cta + (n_gslots - 1) * G) * nr);
  auto slot_first_neuron = [&](int s) { return (cta + s * G) * nr; };

  if (warp < kGateProducers) {
    // ======================= gate producers ===================================================
    // Warp 0 sets up the barriers; both producer warps then start streaming at once (alternate
    // ring slots): the weights do not depend on anything earlier in the stream.
    if (warp == 0 && lane == 0) {
      for (int s = 0; s < NG; ++s) {
        mbar_init(full_gate + 8 * s, 1);
        mbar_init(empty_gate + 8 * s, 1);
      }
      for (int s = 0; s < NA; ++s) {
        mbar_init(full_act + 8 * s, kActProducers);
        mbar_init(empty_act + 8 * s, kGAW);
      }
      if (GATED) {
        for (int s = 0; s < NU; ++s) {
          mbar_init(full_up + 8 * s, 1);
          mbar_init(empty_up + 8 * s, kGAW);
          mbar_init(h_ready + 8 * s, 1);
        }
        for (int s = 0; s < ND; ++s) {
          mbar_init(full_dn + 8 * s, 1);
          mbar_init(empty_dn + 8 * s, kGAW);
        }
      }
      mbar_init(v_bar, 1);
      for (int i = 0; i < 8; ++i) ctl[i] = 0;
      for (int i = 0; i < 6 * (2 * 4 + 1); ++i) red[i] = 0.f;
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    named_bar_sync(4, 32 * kGateProducers);  // barriers are initialised
    named_bar_arrive(3, kThreads);           // release the other warps (they block on barrier 3)
    if (LOPA && warp == 1 && lane == 0) {
      // This CTA's rows of V (consecutive rows: one copy) go into the act ring, which is idle until the gate vector
      // is complete; they are weights, so they travel while the CTA still waits for its predecessor.
      const int vlo = (int)((long long)K * cta / G), vhi = (int)((long long)K * (cta + 1) / G);
      if (vhi > vlo && p.v_in_smem) {
        mbar_expect_tx(v_bar, (uint32_t)((vhi - vlo) * row_bytes));
        bulk_g2s(smem_u32(act_ring), static_cast<const char*>(p.V) + (size_t)vlo * row_bytes,
                 (uint32_t)((vhi - vlo) * row_bytes), v_bar);
      } else {
        mbar_arrive(v_bar);
      }
    }
    if (lane == 0) {
      const char* Wg = static_cast<const char*>(p.Wgate);
      const uint32_t ring = smem_u32(gate_ring);
      for (int s = warp; s < n_gslots; s += kGateProducers) {
        const int slot = s % NG;
        if (!mbar_wait<true>(empty_gate + 8 * slot, ((s / NG) & 1) ^ 1, ctl, p.status, p.wait_cycles, 41)) break;
        const int j0 = slot_first_neuron(s);
        const uint32_t bytes = (uint32_t)(min(nr, p.H - j0) * gate_row_bytes);
        if (!SFFN_IN_BOUNDS(j0 >= 0 && j0 < p.H && (uint32_t)slot * p.gate_slot_bytes + bytes <= (uint32_t)NG * p.gate_slot_bytes,
                            p.status, 1))
          break;
        mbar_expect_tx(full_gate + 8 * slot, bytes);
        bulk_g2s(ring + (uint32_t)slot * p.gate_slot_bytes, Wg + (size_t)j0 * gate_row_bytes, bytes,
                 full_gate + 8 * slot);
      }
    }
    __syncwarp();
    abort_grace(ctl);
    return;
  }

  // The token itself may still be written by the predecessor, so it is not read before the wait -- but its lines can
  // be asked into L2 (a hint: whatever is written later lands in the same L2), which turns the staging loads right
  // after the wait into L2 hits when the token comes from HBM.
  if (warp == kGateProducers + 1) {
    const int lines = (int)(((size_t)D * sizeof(X) + 127) / 128);
    for (int i = lane; i < lines; i += 32)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(static_cast<const char*>(p.x) + (size_t)i * 128) : "memory");
  }

  // Per-neuron parameters of the slab go into shared memory now; for int8 rows also the scales of its W_up / W_down
  // rows, which the act producers hand to the act warps together with a fired row.
  float pre_bias[2] = {0.f, 0.f};  // standard gate, fp32 / bf16 rows: bias of a gate warp's first two slots
  if (!kTables && p.b_g && warp >= kFirstGateWarp && warp < kFAW && warp - kFirstGateWarp < p.gate_warps) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int sq = warp - kFirstGateWarp + q * p.gate_warps;
      if (sq < n_gslots && lane < nr && slot_first_neuron(sq) + lane < p.H) pre_bias[q] = p.b_g[slot_first_neuron(sq) + lane];
    }
  }
  for (int i = tid - kStageBase; kTables && i < slab_rows; i += kStageThreads) {
    const int j = slot_first_neuron(i / nr) + i % nr;
    row_bias[i] = p.b_g ? __ldg(p.b_g + j) : 0.f;
    if (LOPA) {
      row_gi[i] = p.g_idx ? __ldg(p.g_idx + j) : -1;
      row_sg[i] = (p.g_idx && p.g_sign && p.g_sign[j] < 0) ? -1.f : 1.f;
    }
    if (kScaled) {
      row_gscale[i] = __ldg(p.s_gate + j);
      row_su[i] = __ldg(p.s_up + j);
      row_sd[i] = __ldg(p.s_down + j);
    }
  }

  // ---- everyone else: wait for the predecessor in the stream, then stage the token ------------
  pdl_wait();
  if (tid == kStageBase) SFFN_GSTAMP(11);
  // this call's number: the tag of the partials and of the LoPA exchange values
  const uint32_t ep = (LOPA || warp >= kFirstGateWarp) ? __ldcg(p.epoch_word) + 1u : 0u;
  for (int i = tid - kStageBase; i < slab_rows; i += kStageThreads) row_state[i] = 0xffffffffu;
  constexpr int XEPV = Elem<X>::kPerVec;  // token elements per 16 bytes (the weights' EPV unless those are int8)
  // Quantised rows under a standard gate: the token is also split, 16 (int8) or 32 (int4) entries at a time -- the
  // entries one 16-byte chunk of a row meets -- into two int8 limbs and one scale per chunk:
  // x[k] = s_c (q0 + q1 / 128) up to 3e-5 of the chunk's largest |x| (s_c = that maximum / 127), which is two orders
  // below the step of the codes it is multiplied with.  A chunk's scale depends on its own entries only, so an
  // outlier costs the precision of its own chunk and no other.
  constexpr int kGroup = EPV / XEPV;  // threads that share a chunk of the token (2 or 4; 1 where not used)
  int8_t* planes = reinterpret_cast<int8_t*>(smem + L.xlimb + 128);
  float* xsc_w = reinterpret_cast<float*>(smem + L.xlimb + 128 + kTokenLimbs * D);
  for (int cx0 = warp * 32 - kStageBase; cx0 < D / XEPV; cx0 += kStageThreads) {  // warp-uniform trip count (shuffles)
    const int cx = cx0 + lane;
    const bool on = cx < D / XEPV;
    float f[XEPV];
    if (on) {
      Elem<X>::unpack(__ldg(reinterpret_cast<const uint4*>(p.x) + cx), f);
#pragma unroll
      for (int g4 = 0; g4 < XEPV / 4; ++g4) {
        const int k0 = cx * XEPV + 4 * g4;  // first of four consecutive elements: quarter (k0 % EPV) / 4 of chunk k0 / EPV
        reinterpret_cast<float4*>(sx)[((k0 % EPV) >> 2) * nvecD + k0 / EPV] =
            make_float4(f[4 * g4], f[4 * g4 + 1], f[4 * g4 + 2], f[4 * g4 + 3]);
      }
    } else {
#pragma unroll
      for (int e = 0; e < XEPV; ++e) f[e] = 0.f;
    }
    if constexpr (kLimbs || kLimbs4) {
      static_assert(!(kLimbs || kLimbs4) || XEPV == 8, "bf16 token: eight entries per 16 bytes");
      float mx = 0.f;
#pragma unroll
      for (int e = 0; e < XEPV; ++e) mx = fmaxf(mx, fabsf(f[e]));
#pragma unroll
      for (int d = 1; d < kGroup; d <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
      const float xs = mx > 0.f ? mx / 127.f : 1.f, inv = 1.f / xs;
      if (on && (cx & (kGroup - 1)) == 0) xsc_w[cx / kGroup] = xs;
      uint32_t q[kTokenLimbs][2];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float t = fminf(fmaxf(f[e] * inv, -127.f), 127.f);
#pragma unroll
        for (int l = 0; l < kTokenLimbs; ++l) {
          const float r = rintf(t);
          const uint32_t b = (uint32_t)(int)r & 0xffu;
          if ((e & 3) == 0) q[l][e >> 2] = b;
          else q[l][e >> 2] |= b << (8 * (e & 3));
          t = (t - r) * 128.f;
        }
      }
      if (on) {
#pragma unroll
        for (int l = 0; l < kTokenLimbs; ++l) {
          if (kLimbs4) {  // one word's worth of nibbles: even columns, then odd columns
            const uint32_t ev = __byte_perm(q[l][0], q[l][1], 0x6420), od = __byte_perm(q[l][0], q[l][1], 0x7531);
            *reinterpret_cast<uint2*>(planes + (size_t)l * D + cx * 8) = make_uint2(ev, od);
          } else {
            *reinterpret_cast<uint2*>(planes + (size_t)l * D + cx * 8) = make_uint2(q[l][0], q[l][1]);
          }
        }
      }
    }
  }
  if (LOPA) {
    // Rank-r stage of the LoPA gate, v = V x, spread over the grid: this CTA computes its share of the rows of V,
    // publishes them, and collects everybody's.  All CTAs of the call become resident without waiting for this one
    // (one CTA per SM, predecessors in the stream never wait on their successors), so the bounded wait below ends as
    // soon as the slowest CTA has started and published.  The stage sits on the call's critical path, so it is made of
    // as few dependent memory round trips as it can be: the CTA's rows of V are in shared memory by now, the warps
    // share them, the parts of a row are added in a fixed order, and the values are published with the call's number
    // in the same 64-bit word -- a reader that finds the number has the value, no counter and no fence in between.
    const int r = K;
    const int st = tid - kStageBase, sw = warp - kGateProducers;
    constexpr int kSW = kStageThreads / 32;
    const int vlo = (int)((long long)r * cta / G), vhi = (int)((long long)r * (cta + 1) / G);
    const int v_max = (r + G - 1) / G;                  // most rows of V a CTA has
    // where they do not fit beside the sums (wide rows, high rank) they are read from global memory instead
    const uint4* vsm = p.v_in_smem ? reinterpret_cast<const uint4*>(act_ring)
                                   : reinterpret_cast<const uint4*>(static_cast<const char*>(p.V) + (size_t)vlo * row_bytes);
    float* wss = reinterpret_cast<float*>(act_ring + (p.v_in_smem ? (size_t)v_max * row_bytes : 0));
    float* vpart = wss + 32;
    named_bar_sync(5, kStageThreads);  // the token is staged
    mbar_wait(v_bar, 0, ctl, p.status, p.wait_cycles, 50);
    // the warps share the CTA's rows: wpr warps per row (one when there are more rows than warps), each lane sums its
    // chunks in a register, one warp reduction per warp and row; the parts of a row are added in a fixed order
    const int nrows = vhi - vlo;
    const int wpr = nrows > 0 && nrows < kSW ? kSW / nrows : 1;
    for (int row = sw / wpr; row < nrows; row += kSW / wpr) {
      const int part = sw % wpr;
      float a = 0.f;
      for (int c = part * 32 + lane; c < nvecD; c += wpr * 32) a = chunk_dot<T>(vsm[(size_t)row * nvecD + c], sx, c, nvecD, a);
      a = warp_sum(a);
      if (lane == 0) vpart[row * wpr + part] = a;
    }
    named_bar_sync(5, kStageThreads);
    for (int k = vlo + st; k < vhi; k += kStageThreads) {
      float v = 0.f;
      for (int g = 0; g < wpr; ++g) v += vpart[(k - vlo) * wpr + g];
      if (kScaled) v *= __ldg(p.s_V + k);
      asm volatile("st.global.cg.b64 [%0], %1;" ::"l"(p.vtag + k), "l"(tagged(v, ep)) : "memory");
    }
    // collect: two values per thread and pass, both loads in flight; a value still carrying an older number is
    // read again (bounded)
    float ss = 0.f;
    const long long t0 = clock64();
    for (int k = st; k < r; k += 2 * kStageThreads) {
      const int k1 = k + kStageThreads;
      unsigned long long w0 = 0, w1 = 0;
      bool have0 = false, have1 = k1 >= r;
      for (;;) {
        if (!have0) asm volatile("ld.global.cg.b64 %0, [%1];" : "=l"(w0) : "l"(p.vtag + k) : "memory");
        if (!have1) asm volatile("ld.global.cg.b64 %0, [%1];" : "=l"(w1) : "l"(p.vtag + k1) : "memory");
        have0 = (uint32_t)(w0 >> 32) == ep;
        have1 = have1 || (uint32_t)(w1 >> 32) == ep;
        if ((have0 && have1) || ctl[kAbort]) break;
        if (clock64() - t0 > p.wait_cycles) { raise_timeout(ctl, p.status, 47); break; }
      }
      const float v0 = __uint_as_float((uint32_t)w0), v1 = k1 < r ? __uint_as_float((uint32_t)w1) : 0.f;
      ss = fmaf(v0, v0, ss);
      ss = fmaf(v1, v1, ss);
      sn[vec_pos<EPV>(k, r)] = v0;
      if (k1 < r) sn[vec_pos<EPV>(k1, r)] = v1;
    }
    // n = RMSNorm(v) (or v): the warps' sums of squares are added in a fixed order by everyone
    ss = warp_sum(ss);
    if (lane == 0) wss[sw] = ss;
    named_bar_sync(5, kStageThreads);
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < kSW; ++i) tot += wss[i];
    const float inv = p.use_rmsnorm ? rsqrtf(tot / (float)r + p.eps) : 1.f;
    for (int k = st; k < r; k += kStageThreads)
      sn[vec_pos<EPV>(k, r)] *= ((p.use_rmsnorm && p.gain) ? p.gain[k] : 1.f) * inv;
  }
  named_bar_sync(3, kThreads);
  if (tid == kStageBase) SFFN_STAMP(0);

  const float* gvec = LOPA ? sn : sx;  // the vector every gate row is dotted with

  // One ring slot of gate rows: dot every row with the gate vector, publish the results, give the slot back.  False
  // when the wait for the slot's rows ran out.
  const int gw = warp - kFirstGateWarp;
  auto gate_slot = [&](int s) -> bool {
    const int slot = s % NG;
    const int r0 = s * nr;
    const int j0 = slot_first_neuron(s);
    const int rows = min(nr, p.H - j0);
    float add = 0.f;  // bias + fixed-matrix term of the row this lane reports
    float scale = 1.f;  // int8 rows: scale of that row
    if (lane < rows) {
      if (kTables) add = row_bias[r0 + lane];
      else if (s == gw) add = pre_bias[0];
      else if (s == gw + p.gate_warps) add = pre_bias[1];
      else add = p.b_g ? p.b_g[j0 + lane] : 0.f;
      if (kScaled) scale = row_gscale[r0 + lane];
      if (LOPA) {
        const int gi = row_gi[r0 + lane];
        if (gi >= 0) add += row_sg[r0 + lane] * sx[vec_pos<EPV>(gi, D)];
      }
    }
    if (!mbar_wait(full_gate + 8 * slot, (s / NG) & 1, ctl, p.status, p.wait_cycles, 44)) return false;
    const unsigned char* base = gate_ring + (size_t)slot * p.gate_slot_bytes;
    float mine = 0.f;
    // Short gate rows (LoPA: r elements): a row is a few chunks per lane, and with one warp per scheduler the cost is
    // instruction latency, not throughput.  Eight rows are dotted side by side (eight independent chains, the vector
    // read once for all of them, every load requested before the first multiply) and reduced together: each
    // exchange halves the number of sums a lane carries, so eight rows cost 4 + 2 + 1 + 1 + 1 shuffles instead of 40.
    const int rows_short = (nvecK <= 128 && EPV < 32) ? rows : 0;
    int rr_short = 0;
    for (; rows_short - rr_short > 2; rr_short += 8) {  // one or two left-over rows are cheaper one by one (below)
      const int rr = rr_short;
      float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int c = lane; c < nvecK; c += 32) {
        uint4 w[8];
        float4 v[EPV / 4];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          w[i] = rr + i < rows ? reinterpret_cast<const uint4*>(base + (size_t)(rr + i) * gate_row_bytes)[c]
                               : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int q = 0; q < EPV / 4; ++q) v[q] = reinterpret_cast<const float4*>(gvec)[q * nvecK + c];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float f[EPV];
          Elem<T>::unpack(w[i], f);
#pragma unroll
          for (int q = 0; q < EPV / 4; ++q) {
            a[i] = fmaf(f[4 * q + 0], v[q].x, a[i]);
            a[i] = fmaf(f[4 * q + 1], v[q].y, a[i]);
            a[i] = fmaf(f[4 * q + 2], v[q].z, a[i]);
            a[i] = fmaf(f[4 * q + 3], v[q].w, a[i]);
          }
        }
      }
      // lanes with bit 4 set keep rows 4..7, the others rows 0..3; then bit 3 picks two of the four, bit 2 one of
      // the two; bits 1 and 0 are plain sums.  Afterwards lanes 4 k .. 4 k + 3 hold the dot product of row rr + k.
      float b4[4], b2[2];
      const bool up16 = lane & 16, up8 = lane & 8, up4 = lane & 4;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        b4[i] = (up16 ? a[4 + i] : a[i]) + __shfl_xor_sync(0xffffffffu, up16 ? a[i] : a[4 + i], 16);
#pragma unroll
      for (int i = 0; i < 2; ++i)
        b2[i] = (up8 ? b4[2 + i] : b4[i]) + __shfl_xor_sync(0xffffffffu, up8 ? b4[i] : b4[2 + i], 8);
      float z = (up4 ? b2[1] : b2[0]) + __shfl_xor_sync(0xffffffffu, up4 ? b2[0] : b2[1], 4);
      z += __shfl_xor_sync(0xffffffffu, z, 2);
      z += __shfl_xor_sync(0xffffffffu, z, 1);
      const float got = __shfl_sync(0xffffffffu, z, 4 * ((lane - rr) & 7));
      if (lane >= rr && lane < rr + 8) mine = got;
    }
    for (; rr_short < rows_short; ++rr_short) {
      const uint4* w = reinterpret_cast<const uint4*>(base + (size_t)rr_short * gate_row_bytes);
      float a0 = 0.f;
      for (int c = lane; c < nvecK; c += 32) a0 = chunk_dot<T>(w[c], gvec, c, nvecK, a0);
      const float z = warp_sum(a0);
      if (lane == rr_short) mine = z;
    }
    int rr_single = rows_short;
    if constexpr (kLimbs4) {
      // 4-bit rows, standard gate: integer dot products (dp4a) of the bytes 16 x code with the token's limbs; up to four
      // rows side by side share the reads of the limbs (96 bytes per 16-byte chunk of a row).
      // The integer sums of a chunk are exact and small; they are scaled by the chunk's limb scale and added in fp32.
      for (; rr_single < rows; rr_single += 4) {
        float facc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int c = lane; c < nvecK; c += 32) {
          uint4 xv[kGateLimbs][2];
#pragma unroll
          for (int l = 0; l < kGateLimbs; ++l) {
            xv[l][0] = xl[(l * nvecK + c) * 2];
            xv[l][1] = xl[(l * nvecK + c) * 2 + 1];
          }
          const float sc = xsc[c];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (rr_single + i < rows) {
              const uint4 w = reinterpret_cast<const uint4*>(base + (size_t)(rr_single + i) * gate_row_bytes)[c];
              const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
              int acc[kGateLimbs];
#pragma unroll
              for (int l = 0; l < kGateLimbs; ++l) acc[l] = 0;
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const int ev = (int)((ww[k] << 4) & 0xf0f0f0f0u), od = (int)(ww[k] & 0xf0f0f0f0u);
#pragma unroll
                for (int l = 0; l < kGateLimbs; ++l) {
                  const uint4 h = xv[l][k >> 1];
                  acc[l] = __dp4a(ev, (int)((k & 1) ? h.z : h.x), acc[l]);
                  acc[l] = __dp4a(od, (int)((k & 1) ? h.w : h.y), acc[l]);
                }
              }
              float v = small_int_as_float(acc[0]);
              if (kGateLimbs > 1) v = fmaf(small_int_as_float(acc[1]), 0.0078125f, v);
              facc[i] = fmaf(v, sc, facc[i]);
            }
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float z = warp_sum(facc[i]) * 0.0625f;
          if (lane == rr_single + i) mine = z;
        }
      }
    } else if constexpr (EPV == 32) {
      // 4-bit rows: the staged vector is eight times the bytes of a row.  Up to four rows are dotted side by side so
      // that every 128-byte read of it serves all of them; codes are unpacked in pairs and multiplied with packed FMAs.
      for (; rr_single < rows; rr_single += 4) {
        unsigned long long acc4[4] = {0ull, 0ull, 0ull, 0ull};  // (0.f, 0.f)
        for (int c = lane; c < nvecK; c += 32) {
          // plane q of the staged vector holds elements 4q .. 4q+3 of every chunk: two packed pairs per 16-byte read
          ulonglong2 xv[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) xv[q] = reinterpret_cast<const ulonglong2*>(gvec)[q * nvecK + c];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (rr_single + i < rows) {
              const uint4 w = reinterpret_cast<const uint4*>(base + (size_t)(rr_single + i) * gate_row_bytes)[c];
              const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {  // word k: elements 8k .. 8k+7 = planes 2k and 2k+1
                const unsigned long long xp[4] = {xv[2 * k].x, xv[2 * k].y, xv[2 * k + 1].x, xv[2 * k + 1].y};
                acc4[i] = dot8_q4(ww[k], xp, acc4[i]);
              }
            }
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float z = warp_sum(sum_halves(acc4[i]));
          if (lane == rr_single + i) mine = z;
        }
      }
    }
    if constexpr (kLimbs) {
      // int8 rows, standard gate: integer dot products against the token's three limbs (dp4a: four products per
      // instruction, no conversion), two rows side by side so that they share the reads of the limbs; exact int32
      // sums (at most 2^26 per row), recombined as s (A0 + A1 / 128 + A2 / 128^2).
      for (; rr_single < rows; rr_single += 2) {
        const bool two = rr_single + 1 < rows;
        const uint4* w0 = reinterpret_cast<const uint4*>(base + (size_t)rr_single * gate_row_bytes);
        const uint4* w1 = reinterpret_cast<const uint4*>(base + (size_t)(rr_single + (two ? 1 : 0)) * gate_row_bytes);
        float f0 = 0.f, f1 = 0.f;
        for (int c = lane; c < nvecK; c += 32) {
          const uint4 u0 = w0[c], u1 = w1[c];
          int a0[kGateLimbs], a1[kGateLimbs];
#pragma unroll
          for (int l = 0; l < kGateLimbs; ++l) {
            const uint4 xv = xl[l * nvecK + c];
            a0[l] = __dp4a((int)u0.x, (int)xv.x, 0); a0[l] = __dp4a((int)u0.y, (int)xv.y, a0[l]);
            a0[l] = __dp4a((int)u0.z, (int)xv.z, a0[l]); a0[l] = __dp4a((int)u0.w, (int)xv.w, a0[l]);
            a1[l] = __dp4a((int)u1.x, (int)xv.x, 0); a1[l] = __dp4a((int)u1.y, (int)xv.y, a1[l]);
            a1[l] = __dp4a((int)u1.z, (int)xv.z, a1[l]); a1[l] = __dp4a((int)u1.w, (int)xv.w, a1[l]);
          }
          const float sc = xsc[c];
          float v0 = small_int_as_float(a0[0]), v1 = small_int_as_float(a1[0]);
          if (kGateLimbs > 1) {
            v0 = fmaf(small_int_as_float(a0[1]), 0.0078125f, v0);
            v1 = fmaf(small_int_as_float(a1[1]), 0.0078125f, v1);
          }
          f0 = fmaf(v0, sc, f0);
          f1 = fmaf(v1, sc, f1);
        }
        const float z0 = warp_sum(f0), z1 = warp_sum(f1);
        if (lane == rr_single) mine = z0;
        if (two && lane == rr_single + 1) mine = z1;
      }
    } else if (EPV == 16) {
      // int8 rows: the staged vector is four times the bytes of a row, so two rows share every read of it
      for (; rr_single + 1 < rows; rr_single += 2) {
        const uint4* w0 = reinterpret_cast<const uint4*>(base + (size_t)rr_single * gate_row_bytes);
        const uint4* w1 = reinterpret_cast<const uint4*>(base + (size_t)(rr_single + 1) * gate_row_bytes);
        float2 a0 = make_float2(0.f, 0.f), a1 = a0, b0 = a0, b1 = a0;
        int c = lane;
        for (; c + 32 < nvecK; c += 64) {
          chunk_dot2_q8(w0[c], w1[c], gvec, c, nvecK, a0, b0);
          chunk_dot2_q8(w0[c + 32], w1[c + 32], gvec, c + 32, nvecK, a1, b1);
        }
        if (c < nvecK) chunk_dot2_q8(w0[c], w1[c], gvec, c, nvecK, a0, b0);
        const float z0 = warp_sum((a0.x + a0.y) + (a1.x + a1.y)), z1 = warp_sum((b0.x + b0.y) + (b1.x + b1.y));
        if (lane == rr_single) mine = z0;
        if (lane == rr_single + 1) mine = z1;
      }
    }
    for (int rr = rr_single; rr < rows; ++rr) {
      const uint4* w = reinterpret_cast<const uint4*>(base + (size_t)rr * gate_row_bytes);
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
      int c = lane;
      for (; c + 96 < nvecK; c += 128) {
        const uint4 w0 = w[c], w1 = w[c + 32], w2 = w[c + 64], w3 = w[c + 96];
        a0 = chunk_dot<T>(w0, gvec, c, nvecK, a0);
        a1 = chunk_dot<T>(w1, gvec, c + 32, nvecK, a1);
        a2 = chunk_dot<T>(w2, gvec, c + 64, nvecK, a2);
        a3 = chunk_dot<T>(w3, gvec, c + 96, nvecK, a3);
      }
      for (; c < nvecK; c += 32) a0 = chunk_dot<T>(w[c], gvec, c, nvecK, a0);
      const float z = warp_sum((a0 + a1) + (a2 + a3));
      if (lane == rr) mine = z;
    }
    if (lane < rows) {
      const float z = kScaled ? fmaf(mine, scale, add) : mine + add;
      const bool fired = z > 0.f;
      if (!p.dense && (fired || !p.flag_or) && SFFN_IN_BOUNDS(j0 + lane < p.H && r0 + lane < p.slab_max, p.status, 3))
        p.flag[j0 + lane] = fired ? 1 : 0;
      row_state[r0 + lane] = fired ? __float_as_uint(fmaxf(activation(p.act, z), 0.f)) : 0x80000000u;
    }
    __syncwarp();
    if (lane == 0) {
      mbar_arrive(empty_gate + 8 * slot);
      if (p.act_extra) atomicAdd(const_cast<int*>(ctl) + kGateDone, 1);  // this slot's rows have been read
    }
    return true;
  };

  if (warp < kFirstGateWarp) {
    // ======================= act producers: rows of fired neurons, ascending ===================
    // Both walk the published gate results in the same order; producer 0 copies the W_up row of a
    // fired neuron, producer 1 its W_down row, into the same ring slot.
    const int ap = warp - kFirstActProducer;
    const char* Wsrc = static_cast<const char*>(ap == 0 ? p.W_up : p.W_down);
    int slot = 0;
    uint32_t par = 1;
    bool ok = true;
    int n_seq = 0;  // ring slots handed out so far
    // ring that this loop fills: the act slots (both producers), or, gated variant, the W_up rows (first producer)
    const int NR = GATED ? NU : NA;
    const uint32_t pfull = GATED ? full_up : full_act, pempty = GATED ? empty_up : empty_act;
    float* pa = GATED ? up_a : slot_a;
#ifdef SFFN_TRACE
    int n_issued = 0;
#endif
    if (GATED && ap == 1) {
      // Gated variant, second producer: lane 0 follows the fired rows in order, waits for the h of each (published by
      // the act warps per W_up slot) and requests the W_down row into the next slot of the down ring if it is not zero.
      int us = 0, ds = 0;
      uint32_t upar = 0, dpar = 1;
      long long t_idle = 0;
      for (int base = 0; ok && base < slab_rows;) {
        const int row = base + lane;
        const uint32_t st = row < slab_rows ? row_state[row] : 0x80000000u;
        const unsigned done = __ballot_sync(0xffffffffu, st != 0xffffffffu);
        const int prefix = done == 0xffffffffu ? 32 : __ffs(~done) - 1;
        if (prefix == 0) {  // the next row's gate is not computed yet
          if (t_idle == 0) t_idle = clock64();
          __nanosleep(20);
          if (ctl[kAbort]) ok = false;
          else if (clock64() - t_idle > p.wait_cycles) { if (lane == 0) raise_timeout(ctl, p.status, 48); ok = false; }
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          continue;
        }
        t_idle = 0;
        unsigned fired = __ballot_sync(0xffffffffu, row < slab_rows && lane < prefix && st != 0x80000000u);
        if (lane == 0) {
          while (fired && ok) {
            const int r = base + __ffs(fired) - 1;
            fired &= fired - 1;
            ok = mbar_wait<true>(h_ready + 8 * us, upar, ctl, p.status, p.wait_cycles, 52);
            const float hv = ok ? up_h[us] : 0.f;
            if (++us == NU) { us = 0; upar ^= 1; }
            if (hv == 0.f) continue;  // the row would be multiplied by zero
            ok = mbar_wait<true>(empty_dn + 8 * ds, dpar, ctl, p.status, p.wait_cycles, 53);
            if (!ok) break;
            dn_h[ds] = hv;  // ordered before the act warps' read by the arrive below and the copy's completion
            size_t j = (size_t)(slot_first_neuron(r / nr) + r % nr);
            if (!SFFN_IN_BOUNDS(j < (size_t)p.H, p.status, 5)) j = 0;
            mbar_expect_tx(full_dn + 8 * ds, (uint32_t)row_bytes);
            bulk_g2s(smem_u32(act_ring) + (uint32_t)((NU + ds) * row_bytes), Wsrc + j * row_bytes, (uint32_t)row_bytes,
                     full_dn + 8 * ds);
            if (++ds == ND) { ds = 0; dpar ^= 1; }
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        base += prefix;
      }
    } else {
    // The whole warp classifies 32 rows per step (one shared-memory read + ballots); lane 0 issues
    // the copies of the fired ones in ascending order.  Only the leading run of finished rows is
    // consumed, so the order never depends on which gate warp was faster.
    long long t_idle = 0;
    for (int base = 0; ok && base < slab_rows;) {
      const int row = base + lane;
      const uint32_t st = row < slab_rows ? row_state[row] : 0x80000000u;
      const unsigned done = __ballot_sync(0xffffffffu, st != 0xffffffffu);
      const int prefix = done == 0xffffffffu ? 32 : __ffs(~done) - 1;
      if (prefix == 0) {  // the next row's gate is not computed yet
        if (t_idle == 0) t_idle = clock64();
        __nanosleep(20);
        if (ctl[kAbort]) ok = false;
        else if (clock64() - t_idle > p.wait_cycles) { if (lane == 0) raise_timeout(ctl, p.status, 48); ok = false; }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        continue;
      }
      t_idle = 0;
      const bool take = row < slab_rows && lane < prefix && (p.dense || st != 0x80000000u);
      unsigned fired = __ballot_sync(0xffffffffu, take);
      // Every lane issues the copy of its own row: up to NA rows go out per step, each into the ring slot of its
      // place among the fired rows (one lane issuing them one after the other manages a row every ~500 cycles, which
      // is what bounds a call with a short gate).
      while (fired && ok) {
        const int place = __popc(fired & ((1u << lane) - 1u));
        const int nb = min(__popc(fired), NR);
        const bool mine = ((fired >> lane) & 1u) != 0 && place < nb;
        bool good = true;
        if (mine) {
          int ms = slot + place;
          uint32_t mp = par;
          if (ms >= NR) { ms -= NR; mp ^= 1; }
          bool free_slot = mbar_wait<true>(pempty + 8 * ms, mp, ctl, p.status, p.wait_cycles, 42);
          if (!GATED && free_slot && ms >= NAown && n_seq + place < NA) {
            // first use of a slot inside the gate ring: not before the gate warps have read every gate row
            const long long t0 = clock64();
            while (ctl[kGateDone] < n_gslots) {
              if (ctl[kAbort]) { free_slot = false; break; }
              if (clock64() - t0 > p.wait_cycles) { raise_timeout(ctl, p.status, 51); free_slot = false; break; }
              __nanosleep(40);
            }
          }
          if (free_slot) {
            if (ap == 0) pa[ms] = st == 0x80000000u ? 0.f : __uint_as_float(st);
            if (kScaled && ap == 0) {
              slot_su[ms] = row_su[row];
              slot_sd[ms] = row_sd[row];
            }
            size_t j = (size_t)(slot_first_neuron(row / nr) + row % nr);
            if (!SFFN_IN_BOUNDS(j < (size_t)p.H && ms >= 0 && ms < NR, p.status, 2)) j = 0;
            mbar_expect_tx(pfull + 8 * ms, (uint32_t)row_bytes);
            const uint32_t dst = GATED ? smem_u32(act_ring) + (uint32_t)(ms * row_bytes)
                                       : smem_u32(act_slot(ms)) + (ap == 0 ? 0u : (uint32_t)row_bytes);
            bulk_g2s(dst, Wsrc + j * row_bytes, (uint32_t)row_bytes, pfull + 8 * ms);
          } else {
            good = false;
          }
        }
        ok = __all_sync(0xffffffffu, good);
        fired &= ~__ballot_sync(0xffffffffu, mine);
#ifdef SFFN_TRACE
        n_issued += nb;
#endif
        slot += nb;
        n_seq += nb;
        if (slot >= NR) { slot -= NR; par ^= 1; }
      }
      base += prefix;
    }
    // Stop markers (a negative gate value, the phase completed without data): every act group meets one in the first
    // slot of the round it would take next.
    if (lane == 0 && ap == 0) SFFN_STAMP(7);
    if (lane == 0) {
      const int per_round = NA >= 4 ? 2 : 1;
      const int n_end = p.act_groups == 1 || GATED ? n_seq + 1 : (n_seq / per_round + p.act_groups) * per_round;
      for (; ok && n_seq < n_end; ++n_seq) {
        if (mbar_wait<true>(pempty + 8 * slot, par, ctl, p.status, p.wait_cycles, 43)) {
          if (ap == 0) pa[slot] = -1.f;
          mbar_arrive(pfull + 8 * slot);
        } else {
          ok = false;
        }
        if (++slot == NR) { slot = 0; par ^= 1; }
      }
    }
    }  // not the gated variant's second producer
    if (ap == 0) {
      // This CTA's place in the order of finishing (the first R sum the partials), taken now so that the round trip
      // overlaps with the act warps' last rows; -1 under the test hook that makes a CTA go missing.
      if (lane == 0) {
        SFFN_STAMP(2);
#ifdef SFFN_TRACE
        if (p.trace) p.trace[(size_t)blockIdx.x * 16 + 1] = n_issued;
#endif
        int rank = -1;
        if (cta != p.skip_arrival_cta) {
          unsigned long long old;
          asm volatile("atom.add.relaxed.gpu.global.u64 %0, [%1], 1;" : "=l"(old) : "l"(p.done_counter) : "memory");
          rank = (int)(old - old / G * G);
        }
        ctl[kRank] = rank;
      }
      __syncwarp();
      asm volatile("bar.arrive 6, %0;" ::"r"(32 * (kGW + kAW) + 32) : "memory");
    }
    __syncwarp();
  } else {
    const bool gate_warp = warp < kFAW;
    if (gate_warp) {
      // ======================= gate warps ========================================================
      for (int s = gw; gw < p.gate_warps && s < n_gslots; s += p.gate_workers)
        if (!gate_slot(s)) break;
      if (lane == 0 && gw == (n_gslots - 1) % p.gate_workers) SFFN_STAMP(3);
    }
    // ======================= act warps =========================================================
    // (LoPA with three act groups: the four gate warps, done with the short gate, are the third group)
    const bool third = LOPA && gate_warp && p.act_groups == 3;
    if (!gate_warp || third) {
    const int at = gate_warp ? kAT + tid - 32 * kFirstGateWarp : tid - 32 * kFAW;
    const int aw = at >> 5;
    const int grp = aw / kGAW, gaw = aw % kGAW, gat = at % kGT;  // act group, warp and thread within it
    // Short gate (LoPA): the act warps have nothing to do until the first fired rows arrive, so they take gate slots
    // too -- with a dozen warps on it the whole gate is one or two slots per warp.
    if (LOPA && !gate_warp) {
      for (int s = p.gate_warps + aw; s < n_gslots; s += p.gate_workers)
        if (p.gate_warps + aw >= p.gate_workers || !gate_slot(s)) break;
      if (lane == 0 && p.gate_warps + aw == (n_gslots - 1) % p.gate_workers) SFFN_STAMP(3);
    }
    float acc[CPT][EPV];
#pragma unroll
    for (int i = 0; i < CPT; ++i)
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[i][e] = 0.f;
    // The entries of the token that this thread's chunks of a W_up row meet, in registers where they fit: the staged
    // fp32 token is twice the bytes of a bf16 row, and reading it from shared memory for every fired row made the
    // act warps' round (measured: 0.74 us for two rows at 4096 columns) a matter of shared-memory bandwidth.
    constexpr bool kXReg = CPT * EPV <= 32;
    float xr[kXReg ? CPT : 1][EPV];
    if (kXReg) {
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        const int c = gat + i * kGT;
#pragma unroll
        for (int q = 0; q < EPV / 4; ++q) {
          const float4 v = c < nvecD ? reinterpret_cast<const float4*>(sx)[q * nvecD + c] : make_float4(0.f, 0.f, 0.f, 0.f);
          xr[i][4 * q] = v.x; xr[i][4 * q + 1] = v.y; xr[i][4 * q + 2] = v.z; xr[i][4 * q + 3] = v.w;
        }
      }
    }

    // Two ring slots per round when the second one exists: both rows are dotted before the one
    // four-warp barrier, which halves the serial latency per fired row.  The stop marker always
    // arrives, so waiting for the second slot of a round cannot block for good.  A thread whose
    // wait ran out still joins the barrier and raises the group's stop flag, so the four warps
    // always leave the loop together.
    if constexpr (GATED) {
      // Two W_up rows per round; the W_down rows that the previous round asked for are added after this round's h
      // have been published, whatever is left after the stop marker.
      int us = 0, ds = 0;
      uint32_t upar = 0, dpar = 0;
      int pend = 0;         // W_down rows requested by the previous round
      bool failed = false;  // a wait ran out
      auto add_down = [&](int n) {
        for (int k = 0; k < n && !failed; ++k) {
          if (!mbar_wait(full_dn + 8 * ds, dpar, ctl, p.status, p.wait_cycles, 54)) { failed = true; break; }
          const float h = dn_h[ds];
          const uint4* wd = reinterpret_cast<const uint4*>(act_ring + (size_t)(NU + ds) * row_bytes);
#pragma unroll
          for (int i = 0; i < CPT; ++i) {
            const int c = gat + i * kGT;
            if (c < nvecD) {
              float f[EPV];
              Elem<T>::unpack(wd[c], f);
#pragma unroll
              for (int e = 0; e < EPV; e += 2) {
                const float2 t = fma2(make_float2(h, h), make_float2(f[e], f[e + 1]), make_float2(acc[i][e], acc[i][e + 1]));
                acc[i][e] = t.x;
                acc[i][e + 1] = t.y;
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_dn + 8 * ds);
          if (++ds == ND) { ds = 0; dpar ^= 1; }
        }
      };
      for (int round = 0;; ++round) {
        float* rp = red + (round & 1) * (2 * kGAW + 1);
        const int us1 = us + 1 == NU ? 0 : us + 1;
        const uint32_t upar1 = us + 1 == NU ? upar ^ 1 : upar;
        const bool got0 = mbar_wait(full_up + 8 * us, upar, ctl, p.status, p.wait_cycles, 45);
        const float a0 = got0 ? up_a[us] : -1.f;
        bool got1 = true;
        float a1 = -1.f;
        if (a0 >= 0.f) {
          got1 = mbar_wait(full_up + 8 * us1, upar1, ctl, p.status, p.wait_cycles, 46);
          a1 = got1 ? up_a[us1] : -1.f;
        }
        if (a0 >= 0.f) {
          const uint4* wu0 = reinterpret_cast<const uint4*>(act_ring + (size_t)us * row_bytes);
          const uint4* wu1 = reinterpret_cast<const uint4*>(act_ring + (size_t)us1 * row_bytes);
          float part0 = 0.f, part1 = 0.f;
          float2 pk0 = make_float2(0.f, 0.f), pk1 = pk0, pk0b = pk0, pk1b = pk0;
#pragma unroll
          for (int i = 0; i < CPT; ++i) {
            const int c = gat + i * kGT;
            if (c < nvecD) {
              if constexpr (kXReg && EPV != 16) {
                float f[EPV];
                Elem<T>::unpack(wu0[c], f);
#pragma unroll
                for (int e = 0; e < EPV; e += 4) {
                  pk0 = fma2(make_float2(f[e], f[e + 1]), make_float2(xr[i][e], xr[i][e + 1]), pk0);
                  pk0b = fma2(make_float2(f[e + 2], f[e + 3]), make_float2(xr[i][e + 2], xr[i][e + 3]), pk0b);
                }
                if (a1 >= 0.f) {
                  Elem<T>::unpack(wu1[c], f);
#pragma unroll
                  for (int e = 0; e < EPV; e += 4) {
                    pk1 = fma2(make_float2(f[e], f[e + 1]), make_float2(xr[i][e], xr[i][e + 1]), pk1);
                    pk1b = fma2(make_float2(f[e + 2], f[e + 3]), make_float2(xr[i][e + 2], xr[i][e + 3]), pk1b);
                  }
                }
              } else {
                part0 = chunk_dot<T>(wu0[c], sx, c, nvecD, part0);
                if (a1 >= 0.f) part1 = chunk_dot<T>(wu1[c], sx, c, nvecD, part1);
              }
            }
          }
          if constexpr (kXReg && EPV != 16) {
            part0 = (pk0.x + pk0.y) + (pk0b.x + pk0b.y);
            part1 = (pk1.x + pk1.y) + (pk1b.x + pk1b.y);
          }
          part0 = warp_sum(part0);
          part1 = warp_sum(part1);
          if (lane == 0) {
            rp[gaw] = part0;
            rp[kGAW + gaw] = part1;
          }
        }
        if (a0 < 0.f || !got1) rp[2 * kGAW] = 1.f;  // stop marker first in the round, or a failed wait
        named_bar_sync(2, kGT);
        const bool stop = rp[2 * kGAW] != 0.f;
        int asked = 0;
        if (!stop) {
          const float u0 = (rp[0] + rp[1]) + (rp[2] + rp[3]);
          const float u1 = (rp[kGAW] + rp[kGAW + 1]) + (rp[kGAW + 2] + rp[kGAW + 3]);
          const float h0 = a0 * activation(p.act_up, u0), h1 = a1 >= 0.f ? a1 * activation(p.act_up, u1) : 0.f;
          if (at == 0) {  // the arrive releases the store: the second producer reads up_h after its wait
            up_h[us] = h0;
            mbar_arrive(h_ready + 8 * us);
            if (a1 >= 0.f) {
              up_h[us1] = h1;
              mbar_arrive(h_ready + 8 * us1);
            }
          }
          __syncwarp();
          if (lane == 0) {  // the W_up rows have been read by every thread that passed the barrier
            mbar_arrive(empty_up + 8 * us);
            if (a1 >= 0.f) mbar_arrive(empty_up + 8 * us1);
          }
          asked = (h0 != 0.f ? 1 : 0) + (h1 != 0.f ? 1 : 0);
        }
        add_down(pend);
        pend = asked;
        if (stop || a1 < 0.f || failed) {
          add_down(pend);
          break;
        }
        us += 2;
        while (us >= NU) { us -= NU; upar ^= 1; }
      }
    } else {
    const bool pair = NA >= 4;  // with fewer slots, holding two at a time would stall the act producers
    const int stride = (pair ? 2 : 1) * p.act_groups;  // ring slots from one round of a group to its next
    int slot = (pair ? 2 : 1) * grp;
    uint32_t par = 0;
    while (slot >= NA) { slot -= NA; par ^= 1; }
    for (int round = 0;; ++round) {
      float* rp = red + (2 * grp + (round & 1)) * (2 * kGAW + 1);
      const int slot1 = slot + 1 == NA ? 0 : slot + 1;
      const uint32_t par1 = slot + 1 == NA ? par ^ 1 : par;
      const bool got0 = mbar_wait(full_act + 8 * slot, par, ctl, p.status, p.wait_cycles, 45);
      const float a0 = got0 ? slot_a[slot] : -1.f;
      bool got1 = true;
      float a1 = -1.f;
      if (pair && a0 >= 0.f) {
        got1 = mbar_wait(full_act + 8 * slot1, par1, ctl, p.status, p.wait_cycles, 46);
        a1 = got1 ? slot_a[slot1] : -1.f;
      }
      const unsigned char* s0 = act_slot(slot);
      const unsigned char* s1 = act_slot(slot1);
      float part0 = 0.f, part1 = 0.f;
      float2 pk0 = make_float2(0.f, 0.f), pk1 = pk0, pk0b = pk0, pk1b = pk0;  // packed partial sums
      int ia0[kTokenLimbs] = {0, 0}, ia1[kTokenLimbs] = {0, 0};                             // quantised rows, standard gate: a chunk's integer sums per limb
      if (a0 >= 0.f) {
        const uint4* wu0 = reinterpret_cast<const uint4*>(s0);
        const uint4* wu1 = reinterpret_cast<const uint4*>(s1);
#pragma unroll
        for (int i = 0; i < CPT; ++i) {
          const int c = gat + i * kGT;
          if (c < nvecD) {
            if constexpr (kLimbs4) {
              const uint4 u0 = wu0[c], u1 = wu1[c];
              const uint32_t w0[4] = {u0.x, u0.y, u0.z, u0.w}, w1[4] = {u1.x, u1.y, u1.z, u1.w};
#pragma unroll
              for (int l = 0; l < kUpLimbs; ++l) {
                const uint4 h0 = xl[(l * nvecD + c) * 2], h1 = xl[(l * nvecD + c) * 2 + 1];
                const uint32_t xe[4] = {h0.x, h0.z, h1.x, h1.z}, xo[4] = {h0.y, h0.w, h1.y, h1.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  ia0[l] = __dp4a((int)((w0[k] << 4) & 0xf0f0f0f0u), (int)xe[k], ia0[l]);
                  ia0[l] = __dp4a((int)(w0[k] & 0xf0f0f0f0u), (int)xo[k], ia0[l]);
                  if (a1 >= 0.f) {
                    ia1[l] = __dp4a((int)((w1[k] << 4) & 0xf0f0f0f0u), (int)xe[k], ia1[l]);
                    ia1[l] = __dp4a((int)(w1[k] & 0xf0f0f0f0u), (int)xo[k], ia1[l]);
                  }
                }
              }
              {  // the chunk's integer sums, scaled by its limb scale, join the fp32 sums
                const float sc = xsc[c];
                const float v0 = fmaf(small_int_as_float(ia0[1]), 0.0078125f, small_int_as_float(ia0[0]));
                const float v1 = fmaf(small_int_as_float(ia1[1]), 0.0078125f, small_int_as_float(ia1[0]));
                part0 = fmaf(v0, sc, part0);
                part1 = fmaf(v1, sc, part1);
                ia0[0] = ia0[1] = ia1[0] = ia1[1] = 0;
              }
            } else if constexpr (kLimbs) {
              const uint4 u0 = wu0[c], u1 = wu1[c];
#pragma unroll
              for (int l = 0; l < kUpLimbs; ++l) {
                const uint4 xv = xl[l * nvecD + c];
                ia0[l] = __dp4a((int)u0.x, (int)xv.x, ia0[l]); ia0[l] = __dp4a((int)u0.y, (int)xv.y, ia0[l]);
                ia0[l] = __dp4a((int)u0.z, (int)xv.z, ia0[l]); ia0[l] = __dp4a((int)u0.w, (int)xv.w, ia0[l]);
                if (a1 >= 0.f) {
                  ia1[l] = __dp4a((int)u1.x, (int)xv.x, ia1[l]); ia1[l] = __dp4a((int)u1.y, (int)xv.y, ia1[l]);
                  ia1[l] = __dp4a((int)u1.z, (int)xv.z, ia1[l]); ia1[l] = __dp4a((int)u1.w, (int)xv.w, ia1[l]);
                }
              }
              {  // the chunk's integer sums, scaled by its limb scale, join the fp32 sums
                const float sc = xsc[c];
                const float v0 = fmaf(small_int_as_float(ia0[1]), 0.0078125f, small_int_as_float(ia0[0]));
                const float v1 = fmaf(small_int_as_float(ia1[1]), 0.0078125f, small_int_as_float(ia1[0]));
                part0 = fmaf(v0, sc, part0);
                part1 = fmaf(v1, sc, part1);
                ia0[0] = ia0[1] = ia1[0] = ia1[1] = 0;
              }
            } else if constexpr (EPV == 16) {
              pk0 = chunk_dot_q8(wu0[c], sx, c, nvecD, pk0);
              if (a1 >= 0.f) pk1 = chunk_dot_q8(wu1[c], sx, c, nvecD, pk1);
            } else if constexpr (kXReg) {
              // packed FMAs on two pairs of running sums per row: half the instructions, chains a quarter as long
              float f[EPV];
              Elem<T>::unpack(wu0[c], f);
#pragma unroll
              for (int e = 0; e < EPV; e += 4) {
                pk0 = fma2(make_float2(f[e], f[e + 1]), make_float2(xr[i][e], xr[i][e + 1]), pk0);
                pk0b = fma2(make_float2(f[e + 2], f[e + 3]), make_float2(xr[i][e + 2], xr[i][e + 3]), pk0b);
              }
              if (a1 >= 0.f) {
                Elem<T>::unpack(wu1[c], f);
#pragma unroll
                for (int e = 0; e < EPV; e += 4) {
                  pk1 = fma2(make_float2(f[e], f[e + 1]), make_float2(xr[i][e], xr[i][e + 1]), pk1);
                  pk1b = fma2(make_float2(f[e + 2], f[e + 3]), make_float2(xr[i][e + 2], xr[i][e + 3]), pk1b);
                }
              }
            } else {
              part0 = chunk_dot<T>(wu0[c], sx, c, nvecD, part0);
              if (a1 >= 0.f) part1 = chunk_dot<T>(wu1[c], sx, c, nvecD, part1);
            }
          }
        }
        if constexpr (kLimbs || kLimbs4) {
          if (kLimbs4) {  // the bytes were 16 x code
            part0 *= 0.0625f;
            part1 *= 0.0625f;
          }
        } else if constexpr (EPV == 16) {
          part0 = pk0.x + pk0.y;
          part1 = pk1.x + pk1.y;
        } else if constexpr (kXReg) {
          part0 = (pk0.x + pk0.y) + (pk0b.x + pk0b.y);
          part1 = (pk1.x + pk1.y) + (pk1b.x + pk1b.y);
        }
        part0 = warp_sum(part0);
        part1 = warp_sum(part1);
        if (lane == 0) {
          rp[gaw] = part0;
          rp[kGAW + gaw] = part1;
        }
      }
      if (a0 < 0.f || !got1) rp[2 * kGAW] = 1.f;  // stop marker first in the round, or a failed wait
      named_bar_sync(2 + 6 * grp, kGT);
      if (rp[2 * kGAW] != 0.f) break;
      float u0 = (rp[0] + rp[1]) + (rp[2] + rp[3]);
      float u1 = (rp[kGAW] + rp[kGAW + 1]) + (rp[kGAW + 2] + rp[kGAW + 3]);
      if (kScaled) {  // int8 rows: u = s_up (codes . x); the W_down row's scale rides on h
        u0 *= slot_su[slot];
        u1 *= slot_su[slot1];
      }
      float h0 = a0 * activation(p.act_up, u0), h1 = a1 * activation(p.act_up, u1);
      if (kScaled) {
        h0 *= slot_sd[slot];
        h1 *= slot_sd[slot1];
      }
      const uint4* wd0 = reinterpret_cast<const uint4*>(s0 + row_bytes);
      const uint4* wd1 = reinterpret_cast<const uint4*>(s1 + row_bytes);
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        const int c = gat + i * kGT;
        if (c < nvecD) {
          float f[EPV];
          Elem<T>::unpack(wd0[c], f);
#pragma unroll
          for (int e = 0; e < EPV; e += 2) {
            const float2 t = fma2(make_float2(h0, h0), make_float2(f[e], f[e + 1]), make_float2(acc[i][e], acc[i][e + 1]));
            acc[i][e] = t.x;
            acc[i][e + 1] = t.y;
          }
          if (a1 >= 0.f) {
            Elem<T>::unpack(wd1[c], f);
#pragma unroll
            for (int e = 0; e < EPV; e += 2) {
              const float2 t = fma2(make_float2(h1, h1), make_float2(f[e], f[e + 1]), make_float2(acc[i][e], acc[i][e + 1]));
              acc[i][e] = t.x;
              acc[i][e + 1] = t.y;
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_act + 8 * slot);
      if (pair) {
        if (a1 < 0.f) break;  // the second slot was the stop marker
        if (lane == 0) mbar_arrive(empty_act + 8 * slot1);
      }
      slot += stride;
      while (slot >= NA) { slot -= NA; par ^= 1; }
    }
    }
    if (at == 0) SFFN_STAMP(4);
    if (kGroups == 2) {
      // the other groups' sums go to the first through the act ring, once every group has left it; added in group order
      float* xch = reinterpret_cast<float*>(act_ring);
      const int merge_threads = kGT * p.act_groups;
      named_bar_sync(9, merge_threads);
      if (grp > 0) {
#pragma unroll
        for (int i = 0; i < CPT; ++i)
#pragma unroll
          for (int e = 0; e < EPV; ++e) xch[(grp - 1) * (CPT * EPV * kGT) + (i * EPV + e) * kGT + gat] = acc[i][e];
      }
      named_bar_sync(9, merge_threads);
      if (grp == 0) {
        for (int og = 1; og < p.act_groups; ++og) {
#pragma unroll
          for (int i = 0; i < CPT; ++i)
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[i][e] += xch[(og - 1) * (CPT * EPV * kGT) + (i * EPV + e) * kGT + gat];
        }
      }
    }
    // This CTA's partial of y, every value tagged with the call's number.  Stored unit (two columns, 16 bytes)
    // (i * EPV / 2 + e) * kGT + gat holds columns EPV (gat + i kGT) + 2 e and the next one: a warp's store is 512
    // contiguous bytes; the summing threads undo the permutation when they write y.
    if (cta != p.skip_arrival_cta && grp == 0 && SFFN_IN_BOUNDS(cta < kMaxGrid, p.status, 4)) {
      const uint64_t keep = policy_evict_last();  // the partials are rewritten by every call: they should stay in L2
      unsigned long long* dst = p.partial + (size_t)cta * (CPT * EPV * kGT);
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        if (gat + i * kGT < nvecD) {
#pragma unroll
          for (int e = 0; e < EPV / 2; ++e)
            st_tagged2(dst + 2 * (size_t)((i * (EPV / 2) + e) * kGT + gat), tagged(acc[i][2 * e], ep),
                       tagged(acc[i][2 * e + 1], ep), keep);
        }
      }
    }
    if (at == 0) SFFN_STAMP(5);
    if (at == 0) SFFN_GSTAMP(12);
    }
  }

  // ---- y = sum over CTAs of their partials, by the first CTAs to finish ------------------------------------------
  // The first R CTAs of a call to finish stay and each sums one slice of the columns over all partials in a fixed order
  // (which CTA does a slice depends on timing, what it computes does not: y is bitwise the same on every run).  They
  // have time to spare until the slowest CTA is done and fetch the partials that are already there meanwhile.  A
  // summing CTA does not wait for a count or a flag: it reads the other CTAs' tagged values and re-reads those that
  // still carry an older call's number (bounded).  Thread (u, rg) takes two columns (one 16-byte unit) in the rows
  // rg, rg + RG, ...; the RG row groups are then added in order through shared memory.  The other CTAs leave at once
  // and their SMs take the next kernel of the stream.
  if (warp < kFirstGateWarp) {  // act producers (the gate producers left long ago)
    abort_grace(ctl);
    return;
  }
  constexpr int kTail = 32 * (kGW + kAW);
  constexpr int kRow = CPT * EPV * kGT;        // values of a stored partial
  constexpr int kUnits = kRow / 2;             // two columns each (a multiple of 32; those past D are never written)
  const int tt = tid - 32 * kFirstGateWarp;    // index among the tail threads
  // never more than half the grid stays, so that the waiting CTAs of two calls that overlap (two handles on two
  // streams) cannot hold every SM between them
  const int R = min(max(1, (G - 1) / 2), max(1, kUnits / 32));
  named_bar_sync(6, kTail + 32);  // + the act producer that took the rank
  const int rank = ctl[kRank];
  const int slice = rank >= 0 && rank < R ? rank : -1;
  if (rank == G - 1 && tt == 0 && !ctl[kAbort]) *p.epoch_word = ep;  // every CTA has its number: the next call tags with ep + 1
  if (slice < 0 || ctl[kAbort]) {
    abort_grace(ctl);
    return;
  }
  if (tt == 0) SFFN_GSTAMP(8);
  constexpr int kBatch = 13;
  const int32_t failed = __ldcg(p.status);  // in flight together with the partials, not after them
  float2* comb = reinterpret_cast<float2*>(gate_ring);  // the rings are idle by now
  const int U = (kUnits + R - 1) / R;
  const int UW = U <= 32 ? 32 : U <= 64 ? 64 : 128;
  const int RG = kTail / UW;
  const int u = tt % UW, rg = tt / UW;
  auto first_column = [&](int unit) {  // undoes the permutation of the stored units
    return EPV * ((unit % kGT) + (unit / ((EPV / 2) * kGT)) * kGT) + 2 * ((unit / kGT) % (EPV / 2));
  };
  bool ok = true;
  for (int u0 = 0; u0 < U; u0 += UW) {
    const int unit = slice * U + u0 + u;
    float2 sum = make_float2(0.f, 0.f);
    if (u0 + u < U && unit < kUnits && first_column(unit) < D) {
      const unsigned long long* src = p.partial + 2 * (size_t)unit;
      for (int g0 = rg; ok && g0 < G; g0 += RG * kBatch) {
        unsigned long long a[kBatch], b[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int g = g0 + k * RG;
          a[k] = b[k] = (unsigned long long)ep << 32;  // rows past the grid: zero, already "there"
          if (g < G) ld_tagged2(src + (size_t)g * kRow, a[k], b[k]);
        }
        long long t0 = 0;
        for (;;) {
          bool all = true;
#pragma unroll
          for (int k = 0; k < kBatch; ++k) {
            if ((uint32_t)(a[k] >> 32) != ep || (uint32_t)(b[k] >> 32) != ep) {
              all = false;
              ld_tagged2(src + (size_t)(g0 + k * RG) * kRow, a[k], b[k]);
            }
          }
          if (all) break;
          if (t0 == 0) t0 = clock64();
          if (ctl[kAbort]) { ok = false; break; }
          if (clock64() - t0 > p.wait_cycles) { raise_timeout(ctl, p.status, 49); ok = false; break; }
          __nanosleep(20);
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          sum.x += __uint_as_float((uint32_t)a[k]);
          sum.y += __uint_as_float((uint32_t)b[k]);
        }
      }
    }
    comb[rg * UW + u] = sum;
    named_bar_sync(7, kTail);
    if (tt < UW) {
      const int unit2 = slice * U + u0 + tt;
      const int col2 = first_column(unit2);
      if (u0 + tt < U && unit2 < kUnits && col2 < D) {
        float2 t = make_float2(0.f, 0.f);
        for (int r = 0; r < RG; ++r) {
          t.x += comb[r * UW + tt].x;
          t.y += comb[r * UW + tt].y;
        }
        if (!ctl[kAbort] && failed == 0) *reinterpret_cast<float2*>(p.y + col2) = t;
      }
    }
    named_bar_sync(7, kTail);
  }
  if (tt == 0) SFFN_GSTAMP(13);
  abort_grace(ctl);
}

// ---- host side --------------------------------------------------------------------------------
struct Geometry {
  int rows_per_gate_slot, gate_slot_bytes, n_gate_slots, act_slot_bytes, n_act_slots, slab_max, smem, cpt;
  int gate_warps, gate_workers;
  int act_extra;   // LoPA: act slots inside the gate ring (used once the gate is done)
  int act_used;    // act slots the ring cycles through (<= n_act_slots + act_extra)
  int act_groups;  // groups of four warps that take alternate rounds of the act ring (LoPA: 2 or 3)
  bool v_in_smem;  // LoPA: the CTA's rows of V are copied into the idle act ring ahead of the rank-r stage
  bool ok;
};

Geometry plan(int wkind, int D, int H, int K, bool lopa, int grid) {
  Geometry g{};
  const int epv = weight_epv(wkind);
  const bool scaled = wkind == kWQ8 || wkind == kWQ4;
  const int nvecD = D / epv;
  const int row_bytes = D * 16 / epv, gate_row_bytes = K * 16 / epv;
  if (D % epv || K % epv) return g;
  g.ok = false;
  const int act_threads = 128;                 // as in the kernel: the threads of one act group
  const int gate_warps_max = lopa ? 4 : 8;
  if (row_bytes % 16 || gate_row_bytes % 16 || nvecD > act_threads * 8) return g;
  g.cpt = nvecD <= act_threads ? 1 : nvecD <= 2 * act_threads ? 2 : nvecD <= 4 * act_threads ? 4 : 8;
  // at most 64 accumulators per act thread: the CUDA-core path takes wider rows of int8 / int4 codes
  if (scaled && g.cpt * epv > 64) return g;
  int nr = 8192 / gate_row_bytes;
  nr = nr < 1 ? 1 : nr > 32 ? 32 : nr;
  if (lopa) {
    // Short gate (LoPA): when the CTA's whole share of U fits in three slots per gate warp with a few more rows per
    // slot, take them: every row is then on its way before the token arrives and none waits for a slot to come free
    // (r = 512 at 14336 neurons: 11 slots of 9 rows instead of 13 of 8, whose last arrived 2 us into the gate phase).
    const int share = (H + grid - 1) / grid;
    for (int cand = nr; cand <= 32; ++cand) {
      const int slots = (share + cand - 1) / cand + 1;  // + 1: block-cyclic dealing can give one CTA an extra block
      if (slots <= 3 * gate_warps_max && slots * cand * gate_row_bytes <= 112 * 1024) {
        nr = cand;
        break;
      }
    }
  }
  g.rows_per_gate_slot = nr;
  g.gate_slot_bytes = (nr * gate_row_bytes + 127) / 128 * 128;
  g.act_slot_bytes = (2 * row_bytes + 127) / 128 * 128;
  g.slab_max = (((H + nr - 1) / nr + grid - 1) / grid) * nr;  // most rows one CTA can own
  const bool limbs = (wkind == kWQ8 || wkind == kWQ4) && !lopa;
  const SmemLayout fixed(D, K, lopa, 0, 0, 0, 0, g.slab_max, scaled, 0, false, limbs);
  // slack for what the layout sizes by slot count: gate values and scales per act slot (<= 2 x 128 B), barrier words
  // (<= 2 x (24 + 16) x 8 B)
  const int ring = kSmemBudget - fixed.total - 1024;
  if (ring <= 0) return g;
  // Gate ring first: two slots per gate warp hide the release -> refill latency; the act ring takes
  // what is left (at least two slots).
  int na = 2;
  int ng = (ring - na * g.act_slot_bytes) / g.gate_slot_bytes;
  if (ng < 2) return g;
  // An even number of gate warps (slots alternate between two producers).  Where memory allows only
  // one slot per warp (16 KB rows), eight warps with one slot each still beat four warps with two
  // (measured at 8192 x 28672: 104 us against 145 us per call).
  int gw = (ng < gate_warps_max ? ng : gate_warps_max) & ~1;
  if (gw < 2) gw = 2;
  g.gate_warps = gw;
  if (ng > 3 * gw) ng = 3 * gw;
  ng = ng / gw * gw;
  if (ng < gw) return g;
  // A short gate (LoPA: a CTA's whole share of U may fit in a few slots) needs no deeper ring than its
  // slot count; what that frees goes to the act ring.
  const int slots_of_cta = (g.slab_max + nr - 1) / nr;
  const int enough = (slots_of_cta + gw - 1) / gw * gw;
  if (ng > enough) ng = enough;
  na = (ring - ng * g.gate_slot_bytes) / g.act_slot_bytes;
  if (na > 16) na = 16;
  if (na < 2) return g;
  if (ng >= 3 * gw && na < 4) {  // rebalance: the act ring matters at low sparsity
    ng = 2 * gw;
    na = (ring - ng * g.gate_slot_bytes) / g.act_slot_bytes;
    if (na > 16) na = 16;
  }
  if (lopa && slots_of_cta > ng) {
    // The two act groups of the LoPA kernel use act slots in fours (twos below four, see further down); where the split
    // leaves slots over, a smaller gate ring may buy the next multiple (r = 1024 at 4096 columns: 8 + 8 instead of
    // 12 + 6 with two idle).
    auto usable = [](int a) { return a >= 4 ? a / 4 * 4 : a >= 2 ? 2 : 0; };
    int best_ng = ng, best = usable(na);
    for (int t = ng - gw; t >= gw; t -= gw) {
      int a = (ring - t * g.gate_slot_bytes) / g.act_slot_bytes;
      a = a > 16 ? 16 : a;
      if (usable(a) > best) { best = usable(a); best_ng = t; }
    }
    if (best_ng != ng) {
      ng = best_ng;
      na = (ring - ng * g.gate_slot_bytes) / g.act_slot_bytes;
      if (na > 16) na = 16;
    }
  }
  g.n_act_slots = na;
  g.n_gate_slots = ng;
  // the rank-r stage keeps the CTA's rows of V and one sum per 32-chunk segment of them in the (then idle) act ring
  g.v_in_smem = false;
  // the two act groups of the LoPA kernel add their sums through the act ring
  if (lopa && (size_t)na * g.act_slot_bytes < (size_t)g.cpt * epv * act_threads * 4) return g;
  // a short gate leaves the gate ring idle early: it then holds more act slots
  g.act_extra = 0;
  if (lopa && slots_of_cta <= ng) {
    g.act_extra = (int)((size_t)ng * g.gate_slot_bytes / g.act_slot_bytes);
    if (na + g.act_extra > 16) g.act_extra = 16 - na;
  }
  // Two act groups take alternate rounds.  A ring slot must always come back to the same group: a group that shared a
  // slot with the other one could arrive for its next row there while the other group's row in between has not landed,
  // and the barrier's parity cannot tell that phase from the one two back (seen as rare timeouts and a fault at
  // 8192 x 28672, three act slots).  So the slots in use are a multiple of what the two groups take per lap.
  g.act_used = na + g.act_extra;
  g.act_groups = lopa ? 2 : 1;
  if (lopa) {
    const int total = g.act_used;
    g.act_used = total >= 4 ? total / 4 * 4 : total >= 2 ? 2 : 0;
    if (g.act_used == 0) return g;
    // Three groups (the gate warps join once the short gate is done) where that costs no slots (six per lap) and the
    // merge of three sets of sums fits the act ring.
    if (slots_of_cta <= ng && total >= 6 && total / 6 * 6 >= g.act_used &&
        (size_t)na * g.act_slot_bytes >= (size_t)2 * g.cpt * epv * act_threads * 4) {
      g.act_groups = 3;
      g.act_used = total / 6 * 6;
    }
    g.act_extra = g.act_used > na ? g.act_used - na : 0;
  }
  if (lopa) {
    const size_t v_max = (size_t)(K + grid - 1) / grid, sums = (v_max * ((nvecD + 31) / 32) + 32) * 4;
    if (sums > (size_t)na * g.act_slot_bytes) return g;
    g.v_in_smem = v_max * row_bytes + sums <= (size_t)na * g.act_slot_bytes;
  }
  // Warps that take gate slots.  When the CTA's whole share of the gate rows sits in the ring at once (a short gate), the
  // act warps take slots too: they would idle until the first fired rows arrive.  A longer gate stays with the gate
  // warps (measured at r = 1024: act warps that are busy with gate slots drain the act ring too late).
  g.gate_workers = gw;
  if (lopa) {
    const int most = gw + 8;  // the eight act warps of the LoPA kernel
    if (slots_of_cta <= ng) g.gate_workers = slots_of_cta < gw ? gw : slots_of_cta > most ? most : slots_of_cta;
  }
  const SmemLayout full(D, K, lopa, ng, g.gate_slot_bytes, na, g.act_slot_bytes, g.slab_max, scaled, g.act_extra, false, limbs);
  g.smem = full.total;
  g.ok = g.smem <= kSmemBudget;
  return g;
}

int fused_grid(int sm_count, int H) {
  int grid = sm_count < kMaxGrid ? sm_count : kMaxGrid;
  return grid > H ? H : grid;
}

template <typename T, bool LOPA, bool GATED = false>
cudaError_t launch_main(const FusedParams& p, const Geometry& g, int grid, cudaStream_t s) {
  void (*k)(const FusedParams) = nullptr;
  constexpr int kMaxCpt = 64 / Elem<T>::kPerVec < 8 && TokenOf<T>::kScaled ? 64 / Elem<T>::kPerVec : 8;  // what plan() allows
  switch (g.cpt) {
    case 1: k = fused_ffn_kernel<T, 1, LOPA, GATED>; break;
    case 2: k = fused_ffn_kernel<T, 2, LOPA, GATED>; break;
    case 4: k = fused_ffn_kernel<T, (kMaxCpt >= 4 ? 4 : kMaxCpt), LOPA, GATED>; break;
    default: k = fused_ffn_kernel<T, kMaxCpt, LOPA, GATED>; break;
  }
  if (g.cpt > kMaxCpt) return cudaErrorInvalidValue;
  static unsigned long long configured[4] = {0, 0, 0, 0};  // per instantiation of this template, per row width
  const int slot = g.cpt == 1 ? 0 : g.cpt == 2 ? 1 : g.cpt == 4 ? 2 : 3;
  const cudaError_t e = allow_dynamic_smem(k, kSmemBudget, configured[slot]);
  if (e != cudaSuccess) return e;
  return launch_pdl(k, dim3(grid), dim3(kThreads), (size_t)g.smem, s, p);
}

}  // namespace

FusedTestKnobs& fused_test_knobs() {
  static FusedTestKnobs k;
  return k;
}

// Workspace of the single-token kernels: 256 bytes of counters, the fp32 partials [kMaxGrid][D] of this file's
// kernel, the LoPA exchange vector, then the tagged partials [kMaxGrid][D] x 8 bytes of the tensor-core kernel.
size_t fused_tagged_partials_offset(int D, int r_max) {
  const size_t plain = 256 + (size_t)kMaxGrid * D * 4 + (size_t)(r_max > 0 ? r_max : 1) * 4;
  return (plain + 255) / 256 * 256;
}
size_t fused_workspace_bytes(int D, int H, int r_max) {
  (void)H;
  // a row of tagged partials is padded to 4096, 8192 or 16384 values (whole chunks per act thread of either kernel)
  size_t row = 4096;
  while (row < (size_t)D) row *= 2;
  return fused_tagged_partials_offset(D, r_max) + (size_t)kMaxGrid * row * 8 + 256;
}

// Geometry of the fused kernel for a shape, as nine integers (for host-side checks): ok, rows per gate slot, gate
// slot bytes, gate slots, gate warps, act slot bytes, act slots, chunks per act thread, shared memory bytes.
void debug_fused_plan(int wkind, int D, int H, int K, bool lopa, int sm_count, int* out) {
  const Geometry g = plan(wkind, D, H, K, lopa, fused_grid(sm_count, H));
  const int v[9] = {g.ok ? 1 : 0, g.rows_per_gate_slot, g.gate_slot_bytes, g.n_gate_slots, g.gate_warps,
                    g.act_slot_bytes, g.n_act_slots, g.cpt, g.smem};
  for (int i = 0; i < 9; ++i) out[i] = v[i];
}

// Whether this call's gate goes to the tensor cores (see sffn_set_gate_engine).
static bool wants_tensor_gate(const FusedCall& c) {
  const int knob = fused_test_knobs().tensor_gate;
  if (knob >= 0) return knob != 0;
  if (c.engine == SFFN_GATE_ENGINE_AUTO) return c.dense;
  return c.engine == SFFN_GATE_ENGINE_TENSOR_CORE;
}

bool fused_supported(int wkind, int D, int H, int B, const sffn_gate* gate, int sm_count) {
  if (B != 1) return false;
  if (fused_test_knobs().tensor_gate != 0 && fused_tc_supported(wkind, D, H, B, gate, sm_count)) return true;
  const bool lopa = gate->kind == SFFN_GATE_LOPA;
  const int K = lopa ? gate->r : D;
  return plan(wkind, D, H, K, lopa, fused_grid(sm_count, H)).ok;
}

cudaError_t launch_fused(const FusedCall& c, cudaStream_t s, int* launched) {
  pdl_enabled() = fused_test_knobs().pdl;
  if (wants_tensor_gate(c) && fused_tc_supported(c.wkind, c.D, c.H, 1, c.gate, c.sm_count))
    return launch_fused_tc(c, s, launched);
  const bool lopa = c.gate->kind == SFFN_GATE_LOPA;
  const int K = lopa ? c.gate->r : c.D;
  const int grid = fused_grid(c.sm_count, c.H);
  Geometry g = plan(c.wkind, c.D, c.H, K, lopa, grid);
  if (!g.ok) return cudaErrorInvalidValue;
  // Double activation on the sparse route of a standard gate (bf16 / fp32 rows): W_down rows only where h != 0.
  bool gated = c.gated_skip && c.act_up != kActNone && !c.dense && !lopa &&
               (c.wkind == kWBF16 || c.wkind == kWF32) && g.n_act_slots >= 3 && g.act_extra == 0;
  if (gated) {
    const SmemLayout with(c.D, K, false, g.n_gate_slots, g.gate_slot_bytes, g.n_act_slots, g.act_slot_bytes, g.slab_max,
                          false, g.act_extra, true);
    if (with.total <= kSmemBudget) g.smem = with.total;
    else gated = false;
  }
  char* ws = static_cast<char*>(c.workspace);
  int n = 0;
  cudaError_t e;
  FusedParams p{};
  p.D = c.D; p.H = c.H; p.K = K;
  p.Wgate = lopa ? c.gate->U : c.gate->W_g;
  p.W_up = c.W_up; p.W_down = c.W_down; p.x = c.x; p.b_g = c.b_g;
  p.g_idx = lopa ? c.gate->g_idx : nullptr; p.g_sign = c.gate->g_sign;
  p.gain = c.gate->rms_gain; p.use_rmsnorm = c.gate->use_rmsnorm; p.eps = c.gate->rms_eps;
  p.V = c.gate->V;
  p.vtag = reinterpret_cast<unsigned long long*>(ws + 256);
  p.done_counter = reinterpret_cast<unsigned long long*>(ws) + 1;
  p.y = c.y;
  p.partial = reinterpret_cast<unsigned long long*>(ws + fused_tagged_partials_offset(c.D, c.r_max));
  p.epoch_word = reinterpret_cast<uint32_t*>(ws + 16);
  p.act = c.act; p.dense = c.dense ? 1 : 0;
  p.act_up = c.act_up;
  p.s_gate = c.s_gate; p.s_V = c.s_V; p.s_up = c.s_up; p.s_down = c.s_down;
  p.flag = c.flag; p.flag_or = c.flag_or ? 1 : 0; p.status = c.status;
  p.rows_per_gate_slot = g.rows_per_gate_slot; p.gate_slot_bytes = g.gate_slot_bytes;
  p.n_gate_slots = g.n_gate_slots; p.act_slot_bytes = g.act_slot_bytes; p.n_act_slots = g.n_act_slots;
  p.slab_max = g.slab_max;
  p.gate_warps = g.gate_warps; p.gate_workers = g.gate_workers; p.v_in_smem = g.v_in_smem ? 1 : 0; p.act_extra = g.act_extra; p.act_used = g.act_used; p.act_groups = g.act_groups;
  p.wait_cycles = fused_test_knobs().wait_cycles;
  p.skip_arrival_cta = fused_test_knobs().skip_arrival_cta;
  p.trace = fused_test_knobs().trace;
  if (c.wkind == kWQ8)
    e = lopa ? launch_main<int8_t, true>(p, g, grid, s) : launch_main<int8_t, false>(p, g, grid, s);
  else if (c.wkind == kWQ4)
    e = lopa ? launch_main<q4_t, true>(p, g, grid, s) : launch_main<q4_t, false>(p, g, grid, s);
  else if (c.wkind == kWBF16)
    e = lopa ? launch_main<__nv_bfloat16, true>(p, g, grid, s)
             : gated ? launch_main<__nv_bfloat16, false, true>(p, g, grid, s) : launch_main<__nv_bfloat16, false>(p, g, grid, s);
  else
    e = lopa ? launch_main<float, true>(p, g, grid, s)
             : gated ? launch_main<float, false, true>(p, g, grid, s) : launch_main<float, false>(p, g, grid, s);
  if (e != cudaSuccess) return e;
  ++n;
  if (launched) *launched = n;
  return cudaSuccess;
}

}  // namespace sffn
