// Fused sparse gated FFN for one bf16 token with the gate on the tensor cores (B200, sm_100a).
//
// Same scheme as fused_kernel.cu -- one persistent CTA per SM owns a share of the H neurons and runs the paper's
// sparse execution (Sec. 3.1: gate in full, then only the rows of W_3 / W_2 of fired neurons) on it without
// leaving the SM -- but the gate pre-activation z = W_1 x + b_g (Eq. 1) is computed by tcgen05.mma instead of by
// eight CUDA-core warps.  A single token is not a GEMM, so the row is folded: a gate row of D elements is read as
// 16 "segments" (K block kb of 64 elements belongs to segment kb mod 16), eight neurons x 16 segments fill the 128
// rows of an M = 128 tile, and the token is laid out the same way as the 16 columns of the B operand.  One MMA
// pass multiplies every segment of a row with every segment of the token; the diagonal (segment s of the row
// with segment s of the token) summed over s is the dot product.  15/16 of the tensor work is thrown away, which
// costs nothing: the tensor pipe is otherwise idle and the kernel is bound by HBM.  What it buys:
//   * a ring slot is held for the few hundred cycles of its four MMAs instead of the microsecond a warp needs to
//     dot an 8 KB row, so nearly the whole ring is in flight and the gate stream runs closer to the HBM rate;
//   * the eight gate warps are gone; eight act warps consume the rows of fired neurons instead of four.
//
//   gate producers two threads bring tiles of 8 neurons x 16 K blocks (16 KB) into a shared-memory ring with
//                  tensor-map TMA copies (3-D view {64 elements, K block, neuron} of W_1, 128-byte swizzle).
//   MMA issuers    two threads, alternate ring slots, an accumulator each (16 TMEM columns, double-buffered over
//                  tiles); four tcgen05.mma (M = 128, N = 16, K = 16) per slot, commit to the slot's "free" barrier.
//   epilogue warps four warps read the accumulators (tcgen05.ld), pick the diagonal, sum the 16 segments with
//                  shuffles, add the bias, apply A and publish one word per neuron ("fired with value a_j").
//   act producers  two warps walk the published words in ascending neuron order and queue the W_up / W_down rows of
//                  fired neurons into a second ring (bulk copies).
//   act warps      eight warps: u_j = W_up[j] . x (token slice in registers), h_j = a_j A_3(u_j),
//                  y_part += h_j W_down[j]; column slices of y_part in registers, written once.
// The last CTAs to finish sum the per-CTA partials in CTA order (deterministic, no float atomics).
// Calls are chained with programmatic dependent launch; weights are read before griddepcontrol.wait.
// Every wait is bounded by a cycle budget; on expiry SFFN_ERR_TIMEOUT is recorded, every role winds down and the
// TMEM columns are released before the CTA exits.
#include "fused_kernel.cuh"

#include <cuda.h>

#include <algorithm>

#include "common.cuh"

namespace sffn {

namespace {

constexpr int kGateProducers = 2;  // warps 0, 1
constexpr int kFirstActProducer = 2;
constexpr int kActProducers = 2;   // warps 2, 3
constexpr int kFirstEpi = 4;
constexpr int kEpiWarps = 4;       // warps 4..7: TMEM lane quarter = warp mod 4
constexpr int kFirstIssuer = 8;
constexpr int kIssuers = 2;        // warps 8, 9
constexpr int kFirstAct = 10;
constexpr int kActWarps = 8;       // warps 10..17
constexpr int kThreads = 32 * (kFirstAct + kActWarps);  // 576
constexpr int kAT = 32 * kActWarps;
constexpr int kTail = 32 * (kEpiWarps + kActWarps);  // threads that take part in the cross-CTA sum
constexpr int kStageThreads = 32 * (kFirstAct - kFirstActProducer);  // warps 2..9 build the B operand
constexpr int kTileRows = 8;       // neurons per gate tile
constexpr int kSegs = 16;          // K blocks per ring slot = columns of the MMA
constexpr int kStageBytes = kTileRows * kSegs * 128;  // 16 KB
constexpr int kXbBytes = kSegs * 128;                 // token K blocks of one slot position
constexpr int kMaxParked = 16;     // most gate stages parked in the act ring at the start of a call
constexpr int kTmemCols = 64;      // 2 tiles in flight x 2 issuers x 16 columns
constexpr int kMaxGrid = 256;
constexpr int kSmemBudget = 227 * 1024;

struct TcParams {
  int D, H;
  const void* W_up;
  const void* W_down;
  const void* x;
  const float* b_g;
  unsigned long long* done_counter;  // CTAs that have finished their rows, monotonic over calls
  uint32_t* epoch_word;              // number of calls completed on this workspace
  float* y;
  unsigned long long* partial;       // [grid][D] per-CTA partials of y, each value paired with the call's number
  uint8_t* flag;
  int32_t* status;
  int act, dense, act_up;
  int S, NA, act_slot_bytes, slab_max, kst, nacc;
  int E;         // gate stages that are prefetched into the (still idle) last E act slots at the start of a call
  int R;         // CTAs that stay to sum the partials (the last R to finish)
  int nf;        // full tiles of every CTA (tile t of CTA c is tile c + t * grid of the matrix)
  int rem_base;  // rows from here on are dealt in contiguous runs of <= 8 (each CTA's last, short tile)
  int rem;
  int l2_hints;           // bit 0: weights evict-first, bit 1: partials evict-last
  long long wait_cycles;  // budget of every wait (about one second unless a test shortens it)
  int skip_arrival_cta;   // test hook: this CTA does not count itself as finished (-1: none)
  long long* trace;       // SFFN_TRACE builds: [grid][16] time stamps, or null
};

struct TcLayout {
  int gate_ring, xb, act_ring, row_state, slot_a, red, ctl, bars, tmem_slot, total;
  __host__ __device__ TcLayout(int S, int NA, int act_slot_bytes, int slab_max, int kst) {
    int off = 0;
    auto take = [&](int bytes, int align) {
      off = (off + align - 1) / align * align;
      const int o = off;
      off += bytes;
      return o;
    };
    gate_ring = take(S * kStageBytes, 1024);
    xb = take(kst * kXbBytes, 1024);
    act_ring = take(NA * act_slot_bytes, 1024);
    row_state = take(slab_max * 4, 128);
    slot_a = take(NA * 4, 16);
    red = take(2 * (2 * kActWarps + 1) * 4, 16);
    ctl = take(8 * 4, 16);
    bars = take((2 * S + 3 * NA + kMaxParked + 4) * 8, 8);
    tmem_slot = take(8, 8);
    total = off + 1024;  // slack for aligning the dynamic shared memory to 1024 bytes
  }
};

enum Ctl { kAbort = 0, kRank = 1 };

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
// L2 policies: weights are read once per call (evict first); the per-CTA partials are rewritten by every call and
// should stay in L2 instead of being written back behind the weight stream (evict last).
__device__ __forceinline__ uint64_t policy_evict_first(bool on) {
  uint64_t pol;
  if (on) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t policy_evict_last(bool on) {
  uint64_t pol;
  if (on) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
  (void)pol;
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
// Tiled tensor-map copy of one box at (element 0, K block c1, neuron c2); parts of the box outside the tensor read
// as zero and still count towards the barrier's bytes.
__device__ __forceinline__ void tma_tile_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar,
                                            uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
  (void)pol;
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// K-major operand, 128-byte swizzle: rows 128 bytes apart, groups of eight rows 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3fff);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// D fp32, A and B bf16, both K-major, M = 128, N = 16.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kSegs >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}

// `site` says which wait gave up (diagnostics: word 3 of the status block holds site + 256 * CTA of the last one).
__device__ __forceinline__ void raise_timeout(volatile int* ctl, int32_t* status, int site) {
  ctl[kAbort] = 1;
  status[3] = site + 256 * (int)blockIdx.x;
  atomicExch(status, (int32_t)SFFN_ERR_TIMEOUT);
}
// After a wait has run out the CTA winds down.  Copies and MMAs it has issued may still be in flight; they end within
// microseconds, so a thread that leaves an aborting CTA lets that time pass first: shared memory and TMEM are
// only given back when nothing can write to them any more.
__device__ __forceinline__ void abort_grace(volatile int* ctl) {
  if (ctl[kAbort])
    for (int i = 0; i < 50; ++i) __nanosleep(1000);
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* ctl, int32_t* status,
                                          long long budget, int site) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try(bar, parity)) return true;
    if (ctl[kAbort]) return false;
    if (clock64() - t0 > budget) {
      raise_timeout(ctl, status, site);
      return false;
    }
  }
}

#ifdef SFFN_TRACE
__device__ __forceinline__ long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return (long long)t;
}
#define TC_STAMP(slot)                                                                   \
  do {                                                                                   \
    if (p.trace) p.trace[(size_t)blockIdx.x * 16 + (slot)] = global_ns();                \
  } while (0)
#else
#define TC_STAMP(slot) do { } while (0)
#endif

// Where the gate stages of a CTA's sequence live, walked by one thread with a fixed stride (the loops of the
// producer and issuer threads are single-thread latency chains: no division per stage).  Stage it < S: gate ring
// slot it; S <= it < S + E: parked in the act ring; later: gate ring slot (it - E) mod S, phase ((it - E) / S) & 1.
struct StageCursor {
  int S, E, step, it, slot;
  uint32_t phase;
  __device__ __forceinline__ void start(int S_, int E_, int first, int step_) {
    S = S_; E = E_; step = step_; it = first; slot = first; phase = 0;
    if (first >= S + E) { slot = (first - E) % S; phase = ((first - E) / S) & 1; }
  }
  __device__ __forceinline__ bool parked() const { return it >= S && it < S + E; }
  __device__ __forceinline__ bool in_ring_again() const { return it >= S + E; }
  __device__ __forceinline__ void next() {
    const bool was_ring = it >= S + E;
    it += step;
    if (it < S) { slot = it; }
    else if (it < S + E) { }
    else if (!was_ring) { slot = (it - E) % S; phase = ((it - E) / S) & 1; }
    else { slot += step; if (slot >= S) { slot -= S; phase ^= 1; } }
  }
};

template <int CPT>
__global__ void __launch_bounds__(kThreads, 1) fused_tc_kernel(const TcParams p, const __grid_constant__ CUtensorMap map8,
                                                               const __grid_constant__ CUtensorMap map1) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  if (tid == 0) TC_STAMP(10);
  const int D = p.D;
  const int S = p.S, NA = p.NA, kst = p.kst, nacc = p.nacc;
  const TcLayout L(S, NA, p.act_slot_bytes, p.slab_max, kst);
  unsigned char* act_ring = smem + L.act_ring;
  unsigned char* xb = smem + L.xb;
  volatile uint32_t* row_state = reinterpret_cast<volatile uint32_t*>(smem + L.row_state);
  float* slot_a = reinterpret_cast<float*>(smem + L.slot_a);
  float* red = reinterpret_cast<float*>(smem + L.red);
  volatile int* ctl = reinterpret_cast<volatile int*>(smem + L.ctl);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L.tmem_slot);
  const uint32_t gate_ring = smem_u32(smem + L.gate_ring);
  const uint32_t bars = smem_u32(smem + L.bars);
  const uint32_t full_gate = bars, empty_gate = bars + 8 * S;
  const uint32_t full_act = bars + 16 * S, empty_act = full_act + 8 * NA;
  const uint32_t extra_full = empty_act + 8 * NA, extra_done = extra_full + 8 * kMaxParked;
  const uint32_t acc_full = extra_done + 8 * NA, acc_empty = acc_full + 16;

  const int nvecD = D / 8;
  const size_t row_bytes = (size_t)D * 2;
  // This CTA's neurons: nf full tiles dealt round robin over the CTAs, then a contiguous run of the left-over rows.
  const int nf = p.nf;
  const int rem_lo = p.rem_base + (int)((long long)p.rem * cta / G);
  const int rc = p.rem_base + (int)((long long)p.rem * (cta + 1) / G) - rem_lo;
  const int n_tiles = nf + (rc > 0 ? 1 : 0);
  const int slab_rows = nf * kTileRows + rc;
  auto neuron_of = [&](int l) {
    const int t = l >> 3;
    return t < nf ? (cta + t * G) * kTileRows + (l & 7) : rem_lo + (l - nf * kTileRows);
  };
  // Where gate stage `it` of this CTA's sequence lives.  The first S stages fill the gate ring; the next E go into the
  // last act slots, which no fired row can need yet (no gate result exists before the token has arrived): the CTA
  // starts while its predecessor in the stream still runs, and everything it can fetch before the token is there
  // shortens the call.  From then on the gate ring is used round robin.
  const int m_per_slot = p.act_slot_bytes / kStageBytes;  // gate stages per act slot (p.E > 0 only if it divides)
  // stages parked by this CTA: no more than it has beyond the gate ring, whole act slots, an even number
  int E = min(p.E, max(0, n_tiles * kst - S));
  if (E > 0) {
    E = E / m_per_slot * m_per_slot;
    if (E & 1) E -= m_per_slot;
  }
  const int extra_slots = E > 0 ? E / m_per_slot : 0;      // act slots that start out holding gate stages
  const uint32_t extra_base = smem_u32(act_ring) + (uint32_t)(NA - extra_slots) * p.act_slot_bytes;
  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_gate + 8 * s, 1);
      mbar_init(empty_gate + 8 * s, 1);
    }
    for (int s = 0; s < NA; ++s) {
      mbar_init(full_act + 8 * s, kActProducers);
      mbar_init(empty_act + 8 * s, kActWarps);
      mbar_init(extra_done + 8 * s, m_per_slot > 0 ? m_per_slot : 1);
    }
    for (int s = 0; s < kMaxParked; ++s) mbar_init(extra_full + 8 * s, 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full + 8 * b, nacc);
      mbar_init(acc_empty + 8 * b, kEpiWarps);
    }
    for (int i = 0; i < 8; ++i) ctl[i] = 0;
    for (int i = 0; i < 2 * (2 * kActWarps + 1); ++i) red[i] = 0.f;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map8) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map1) : "memory");
  }
  if (warp == kFirstEpi) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp < kGateProducers) {
    // ======================= gate producers (alternate stages) ======================================
    // The weights depend on nothing earlier in the stream: the rings fill while the predecessor still runs.
    if (lane == 0) {
      const uint64_t once = policy_evict_first(p.l2_hints & 1);
      const int total = n_tiles * kst;
      StageCursor c;
      c.start(S, E, warp, kGateProducers);
      int t = warp / kst, st = warp - t * kst;
      for (; c.it < total; c.next()) {
        uint32_t dst, bar;
        if (c.parked()) {
          dst = extra_base + (uint32_t)(c.it - S) * kStageBytes;
          bar = extra_full + 8 * (c.it - S);
        } else {
          if (c.in_ring_again() && !mbar_wait(empty_gate + 8 * c.slot, c.phase ^ 1, ctl, p.status, p.wait_cycles, 2)) break;
          dst = gate_ring + (uint32_t)c.slot * kStageBytes;
          bar = full_gate + 8 * c.slot;
        }
        if (t < nf) {
          mbar_expect_tx(bar, kStageBytes);
          tma_tile_3d(dst, &map8, 0, st * kSegs, (cta + t * G) * kTileRows, bar, once);
        } else {
          mbar_expect_tx(bar, (uint32_t)rc * (kSegs * 128));
          for (int i = 0; i < rc; ++i)
            tma_tile_3d(dst + (uint32_t)i * (kSegs * 128), &map1, 0, st * kSegs, rem_lo + i, bar, once);
        }
        st += kGateProducers;
        while (st >= kst) { st -= kst; ++t; }
      }
      if (warp == 0) TC_STAMP(1);
    }
    __syncwarp();
    abort_grace(ctl);
    return;
  }

  // The token may still be written by the predecessor; its lines can be asked into L2 meanwhile (a hint).
  if (warp == kFirstActProducer) {
    const int lines = (int)((row_bytes + 127) / 128);
    for (int i = lane; i < lines; i += 32)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(static_cast<const char*>(p.x) + (size_t)i * 128) : "memory");
  }

  pdl_wait();
  if (tid == 32 * kFirstActProducer) TC_STAMP(11);

  const int at = tid - 32 * kFirstAct;  // act threads: 0 .. kAT - 1
  float2 xr[CPT][4];                    // act threads: this thread's slice of the token
  uint32_t ep = 0;                      // this call's number (epilogue and act warps: they write and sum the partials)
  uint64_t keep = 0;                    // act threads: L2 policy of the partial stores (made early: it takes a while)
  if (warp >= kFirstAct) {
    ep = __ldcg(p.epoch_word) + 1u;
    keep = policy_evict_last(p.l2_hints & 2);
#pragma unroll
    for (int i = 0; i < CPT; ++i) {
      const int c = at + i * kAT;
      float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (c < nvecD) Elem<__nv_bfloat16>::unpack(__ldcg(reinterpret_cast<const uint4*>(p.x) + c), f);
#pragma unroll
      for (int q = 0; q < 4; ++q) xr[i][q] = make_float2(f[2 * q], f[2 * q + 1]);
    }
  } else {
    // Token as the B operand: K block kb is row kb mod 16 of slot position kb / 16, 128 bytes, swizzled like the
    // weight tiles (16-byte chunk index xor row mod 8).  K blocks past the row's end are zero.
    if (warp >= kFirstEpi && warp < kFirstIssuer) ep = __ldcg(p.epoch_word) + 1u;
    const int st_tid = tid - 32 * kFirstActProducer;
    for (int i = st_tid; i < slab_rows; i += kStageThreads) row_state[i] = 0xffffffffu;
    const int chunks = kst * kSegs * 8;
    for (int cx = st_tid; cx < chunks; cx += kStageThreads) {
      const uint4 v = cx < nvecD ? __ldcg(reinterpret_cast<const uint4*>(p.x) + cx) : make_uint4(0u, 0u, 0u, 0u);
      const int kb = cx >> 3, ch = cx & 7, st = kb >> 4, s = kb & 15;
      *reinterpret_cast<uint4*>(xb + st * kXbBytes + s * 128 + ((ch ^ (s & 7)) << 4)) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    named_bar_sync(1, kStageThreads);
    if (tid == 32 * kFirstActProducer) TC_STAMP(0);
  }

  if (warp < kFirstEpi) {
    // ======================= act producers: rows of fired neurons, ascending ========================
    const int ap = warp - kFirstActProducer;
    const uint64_t once = policy_evict_first(p.l2_hints & 1);
    const char* Wsrc = static_cast<const char*>(ap == 0 ? p.W_up : p.W_down);
    const uint32_t ring = smem_u32(act_ring) + (ap == 0 ? 0u : (uint32_t)row_bytes);
    int slot = 0, used = 0;
    uint32_t par = 1;
    bool ok = true;
    long long t_idle = 0;
    for (int base = 0; ok && base < slab_rows;) {
      const int row = base + lane;
      const uint32_t st = row < slab_rows ? row_state[row] : 0x80000000u;
      const unsigned done = __ballot_sync(0xffffffffu, st != 0xffffffffu);
      const int prefix = done == 0xffffffffu ? 32 : __ffs(~done) - 1;
      if (prefix == 0) {  // the next neuron's gate is not computed yet
        if (t_idle == 0) t_idle = clock64();
        __nanosleep(20);
        if (ctl[kAbort]) ok = false;
        else if (clock64() - t_idle > p.wait_cycles) { if (lane == 0) raise_timeout(ctl, p.status, 20); ok = false; }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        continue;
      }
      t_idle = 0;
      const bool take = row < slab_rows && lane < prefix && (p.dense || st != 0x80000000u);
      unsigned fired = __ballot_sync(0xffffffffu, take);
      while (fired && ok) {
        const int l = __ffs(fired) - 1;
        fired &= fired - 1;
        const uint32_t sl = __shfl_sync(0xffffffffu, st, l);
        if (lane == 0) {
          bool free_now = mbar_wait(empty_act + 8 * slot, par, ctl, p.status, p.wait_cycles, 3);
          if (free_now && used < NA && slot >= NA - extra_slots)  // first use: the gate stages parked here must be gone
            free_now = mbar_wait(extra_done + 8 * (slot - (NA - extra_slots)), 0, ctl, p.status, p.wait_cycles, 4);
          if (free_now) {
            if (ap == 0) slot_a[slot] = sl == 0x80000000u ? 0.f : __uint_as_float(sl);
            size_t j = (size_t)neuron_of(base + l);
            if (!SFFN_IN_BOUNDS(j < (size_t)p.H, p.status, 20)) j = 0;
            mbar_expect_tx(full_act + 8 * slot, (uint32_t)row_bytes);
            bulk_g2s(ring + (uint32_t)slot * p.act_slot_bytes, Wsrc + j * row_bytes, (uint32_t)row_bytes,
                     full_act + 8 * slot, once);
          } else {
            ok = false;
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        ++used;
        if (++slot == NA) { slot = 0; par ^= 1; }
      }
      base += prefix;
    }
    if (lane == 0 && ok && mbar_wait(empty_act + 8 * slot, par, ctl, p.status, p.wait_cycles, 5)) {
      if (ap == 0) slot_a[slot] = -1.f;  // stop marker: a negative gate value
      mbar_arrive(full_act + 8 * slot);  // completes the phase without data
    }
    if (ap == 0) {
      // This CTA's place in the order of finishing (the last R sum the partials), taken now so that the round trip
      // overlaps with the act warps' last rows; -1 under the test hook that makes a CTA go missing.
      if (lane == 0) {
        TC_STAMP(2);
        int rank = -1;
        if (cta != p.skip_arrival_cta) {
          unsigned long long old;
          asm volatile("atom.add.relaxed.gpu.global.u64 %0, [%1], 1;" : "=l"(old) : "l"(p.done_counter) : "memory");
          rank = (int)(old - old / G * G);
        }
        ctl[kRank] = rank;
        TC_STAMP(7);
      }
      __syncwarp();
      asm volatile("bar.arrive 6, %0;" ::"r"(kTail + 32) : "memory");
    }
    abort_grace(ctl);
    return;
  }

  if (warp >= kFirstIssuer && warp < kFirstAct) {
    // ======================= MMA issuers ============================================================
    const int m = warp - kFirstIssuer;
    if (lane == 0 && m < nacc) {
      const int total = n_tiles * kst;
      const uint64_t bdesc0 = make_desc(smem_u32(xb));
      StageCursor c;
      c.start(S, E, m, nacc);
      int t = m / kst, st = m - t * kst;
      int t_cur = -1;
      uint32_t acc = 0, accumulate = 0;
      for (; c.it < total; c.next()) {
        if (t != t_cur) {  // first stage of this issuer in a new tile
          if (t_cur >= 0) umma_commit(acc_full + 8 * (t_cur & 1));
          t_cur = -1;
          if (!mbar_wait(acc_empty + 8 * (t & 1), ((t >> 1) & 1) ^ 1, ctl, p.status, p.wait_cycles, 6)) break;
          tc_fence_after();
          t_cur = t;
          acc = tmem_base + (uint32_t)(((t & 1) * kIssuers + m) * kSegs);
          accumulate = 0;
        }
        uint32_t addr, bar, done, par;
        if (c.parked()) {
          addr = extra_base + (uint32_t)(c.it - S) * kStageBytes;
          bar = extra_full + 8 * (c.it - S);
          done = extra_done + 8 * ((c.it - S) / m_per_slot);
          par = 0;
        } else {
          addr = gate_ring + (uint32_t)c.slot * kStageBytes;
          bar = full_gate + 8 * c.slot;
          done = empty_gate + 8 * c.slot;
          par = c.phase;
        }
        if (!mbar_wait(bar, par, ctl, p.status, p.wait_cycles, 7)) { t_cur = -1; break; }
        tc_fence_after();
        const uint64_t adesc = make_desc(addr);
        const uint64_t bdesc = bdesc0 + (uint64_t)(st * (kXbBytes >> 4));
        umma(acc, adesc, bdesc, accumulate);
#pragma unroll
        for (int k = 1; k < 4; ++k) umma(acc, adesc + 2 * k, bdesc + 2 * k, 1u);
        umma_commit(done);  // the stage's memory is free once these MMAs have read it
        accumulate = 1;
        st += nacc;
        while (st >= kst) { st -= kst; ++t; }
      }
      if (t_cur >= 0) umma_commit(acc_full + 8 * (t_cur & 1));
      if (m == 0) TC_STAMP(3);
    }
    __syncwarp();
    abort_grace(ctl);
    return;
  }

  const int tt = warp < kFirstIssuer ? tid - 32 * kFirstEpi : 32 * kEpiWarps + at;  // index among the tail threads
  if (warp < kFirstIssuer) {
    // ======================= epilogue warps =========================================================
    // TMEM lane 16 i + s holds neuron i of the tile against segment s of its row; column n is segment n of the token.
    const int q = warp & 3;
    const int i_loc = 2 * q + (lane >> 4), seg = lane & 15;
    bool ok = true;
    for (int t = 0; ok && t < n_tiles; ++t) {
      const int b = t & 1;
      const int rows = t < nf ? kTileRows : rc;
      const int l = t * kTileRows + i_loc;
      const int j = i_loc < rows ? neuron_of(l) : 0;
      const float bias = (seg == 0 && i_loc < rows && p.b_g) ? __ldg(p.b_g + j) : 0.f;
      int okw = 1;
      if (lane == 0) okw = mbar_wait(acc_full + 8 * b, (t >> 1) & 1, ctl, p.status, p.wait_cycles, 8) ? 1 : 0;
      okw = __shfl_sync(0xffffffffu, okw, 0);
      if (!okw) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * kIssuers * kSegs);
      uint32_t r0[16], r1[16];
      tmem_ld16(taddr, r0);
      if (nacc == 2) tmem_ld16(taddr + kSegs, r1);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + 8 * b);
      float v = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const float e = __uint_as_float(r0[c]) + (nacc == 2 ? __uint_as_float(r1[c]) : 0.f);
        v = seg == c ? e : v;
      }
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      v += __shfl_xor_sync(0xffffffffu, v, 8);
      if (seg == 0 && i_loc < rows) {
        const float z = v + bias;
        const bool fired = z > 0.f;
        if (!p.dense && SFFN_IN_BOUNDS(j >= 0 && j < p.H, p.status, 21)) p.flag[j] = fired ? 1 : 0;
        row_state[l] = fired ? __float_as_uint(fmaxf(activation(p.act, z), 0.f)) : 0x80000000u;
      }
    }
    if (warp == kFirstEpi && lane == 0) TC_STAMP(4);
    // the accumulators are idle once every epilogue warp has left its loop: release the TMEM columns
    abort_grace(ctl);
    tc_fence_before();
    named_bar_sync(7, 32 * kEpiWarps);
    if (warp == kFirstEpi) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
  } else {
    // ======================= act warps ==============================================================
    const int aw = warp - kFirstAct;
    float2 acc[CPT][4];
#pragma unroll
    for (int i = 0; i < CPT; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][e] = make_float2(0.f, 0.f);
    // Two ring slots per round when the second one exists (both rows are dotted before the one barrier of the
    // round).  The stop marker always arrives, so waiting for the second slot cannot block for good; a thread
    // whose wait ran out still joins the barrier and raises the group's stop flag.
    int slot = 0;
    uint32_t par = 0;
    const bool pair = NA >= 4;
    for (int round = 0;; ++round) {
      float* rp = red + (round & 1) * (2 * kActWarps + 1);
      const int slot1 = slot + 1 == NA ? 0 : slot + 1;
      const uint32_t par1 = slot + 1 == NA ? par ^ 1 : par;
      const bool got0 = mbar_wait(full_act + 8 * slot, par, ctl, p.status, p.wait_cycles, 9);
      const float a0 = got0 ? slot_a[slot] : -1.f;
      bool got1 = true;
      float a1 = -1.f;
      if (pair && a0 >= 0.f) {
        got1 = mbar_wait(full_act + 8 * slot1, par1, ctl, p.status, p.wait_cycles, 10);
        a1 = got1 ? slot_a[slot1] : -1.f;
      }
      const unsigned char* s0 = act_ring + (size_t)slot * p.act_slot_bytes;
      const unsigned char* s1 = act_ring + (size_t)slot1 * p.act_slot_bytes;
      if (a0 >= 0.f) {
        const uint4* wu0 = reinterpret_cast<const uint4*>(s0);
        const uint4* wu1 = reinterpret_cast<const uint4*>(s1);
        float2 pk0 = make_float2(0.f, 0.f), pk1 = pk0;
#pragma unroll
        for (int i = 0; i < CPT; ++i) {
          const int c = at + i * kAT;
          if (c < nvecD) {
            float f[8];
            Elem<__nv_bfloat16>::unpack(wu0[c], f);
#pragma unroll
            for (int e = 0; e < 4; ++e) pk0 = fma2(make_float2(f[2 * e], f[2 * e + 1]), xr[i][e], pk0);
            if (a1 >= 0.f) {
              Elem<__nv_bfloat16>::unpack(wu1[c], f);
#pragma unroll
              for (int e = 0; e < 4; ++e) pk1 = fma2(make_float2(f[2 * e], f[2 * e + 1]), xr[i][e], pk1);
            }
          }
        }
        const float part0 = warp_sum(pk0.x + pk0.y), part1 = warp_sum(pk1.x + pk1.y);
        if (lane == 0) {
          rp[aw] = part0;
          rp[kActWarps + aw] = part1;
        }
      }
      if (a0 < 0.f || !got1) rp[2 * kActWarps] = 1.f;  // stop marker first in the round, or a failed wait
      named_bar_sync(2, kAT);
      if (rp[2 * kActWarps] != 0.f) break;
      const float u0 = ((rp[0] + rp[1]) + (rp[2] + rp[3])) + ((rp[4] + rp[5]) + (rp[6] + rp[7]));
      const float u1 = ((rp[8] + rp[9]) + (rp[10] + rp[11])) + ((rp[12] + rp[13]) + (rp[14] + rp[15]));
      const float h0 = a0 * activation(p.act_up, u0), h1 = a1 * activation(p.act_up, u1);
      const uint4* wd0 = reinterpret_cast<const uint4*>(s0 + row_bytes);
      const uint4* wd1 = reinterpret_cast<const uint4*>(s1 + row_bytes);
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        const int c = at + i * kAT;
        if (c < nvecD) {
          float f[8];
          Elem<__nv_bfloat16>::unpack(wd0[c], f);
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[i][e] = fma2(make_float2(h0, h0), make_float2(f[2 * e], f[2 * e + 1]), acc[i][e]);
          if (a1 >= 0.f) {
            Elem<__nv_bfloat16>::unpack(wd1[c], f);
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][e] = fma2(make_float2(h1, h1), make_float2(f[2 * e], f[2 * e + 1]), acc[i][e]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_act + 8 * slot);
      if (!pair) {
        if (++slot == NA) { slot = 0; par ^= 1; }
        continue;
      }
      if (a1 < 0.f) break;  // the second slot was the stop marker
      if (lane == 0) mbar_arrive(empty_act + 8 * slot1);
      slot = slot1 + 1 == NA ? 0 : slot1 + 1;
      par = slot1 + 1 == NA ? par1 ^ 1 : par1;
    }
    if (at == 0) TC_STAMP(5);
    // This CTA's partial of y, every value tagged with the call's number.  Stored unit (two columns, 16 bytes)
    // (i * 4 + e) * kAT + at holds columns 8 (at + i kAT) + 2 e and the next one: a warp's store is 512 contiguous
    // bytes; the summing threads undo the permutation when they write y.
    if (cta != p.skip_arrival_cta) {
      unsigned long long* dst = p.partial + (size_t)cta * (CPT * 8 * kAT);
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        if (at + i * kAT < nvecD) {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            st_tagged2(dst + 2 * (size_t)((i * 4 + e) * kAT + at), tagged(acc[i][e].x, ep), tagged(acc[i][e].y, ep), keep);
        }
      }
    }
    if (at == 0) TC_STAMP(12);
  }

  // ---- y = sum over CTAs of their partials, by the last CTAs to finish (epilogue and act warps get here) --------
  // Which CTA sums a slice of the columns depends on timing, what it computes does not: y is bitwise repeatable.
  // A summing CTA does not wait for a count or a flag: it reads the other CTAs' tagged values and re-reads those
  // that still carry an older call's number (bounded).  Thread (u, rg) takes two columns (one 16-byte unit) in the
  // rows rg, rg + RG, ...; the RG row groups are then added in order through shared memory.
  const int units = CPT * 4 * kAT;  // stored units of a partial (a multiple of 32; those past D / 2 are never written)
  const int R = p.R;
  named_bar_sync(6, kTail + 32);  // + the act producer that took the rank
  // The first R CTAs to finish do the sum: they have time to spare until the slowest CTA is done, fetch the
  // partials that are already there meanwhile and only have the late ones left to fetch at the end.  Their SMs come
  // free last, so the next call starts with nothing prefetched there -- which costs little: the CTAs of a call
  // share the memory system's rate whatever their head start.
  const int rank = ctl[kRank];
  const int slice = rank >= 0 && rank < R ? rank : -1;
  if (rank == G - 1 && tt == 0 && !ctl[kAbort]) *p.epoch_word = ep;  // every CTA has its number: the next call tags with ep + 1
  if (slice < 0 || ctl[kAbort]) {
    abort_grace(ctl);
    return;
  }
  if (tt == 0) TC_STAMP(8);
  constexpr int kBatch = 13;
  const int32_t failed = __ldcg(p.status);  // in flight together with the partials, not after them
  float2* comb = reinterpret_cast<float2*>(smem + L.gate_ring);  // the rings are idle by now
  const int U = (units + R - 1) / R;
  const int UW = U <= 32 ? 32 : U <= 64 ? 64 : 128;
  const int RG = kTail / UW;
  const int u = tt % UW, rg = tt / UW;
  bool ok = true;
  for (int u0 = 0; u0 < U; u0 += UW) {
    const int unit = slice * U + u0 + u;
    float2 sum = make_float2(0.f, 0.f);
    const int col = 8 * ((unit % kAT) + (unit / (4 * kAT)) * kAT) + 2 * ((unit / kAT) & 3);  // first of its two columns
    if (u0 + u < U && unit < units && col < D) {
      const unsigned long long* src = p.partial + 2 * (size_t)unit;
      for (int g0 = rg; ok && g0 < G; g0 += RG * kBatch) {
        unsigned long long a[kBatch], b[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int g = g0 + k * RG;
          a[k] = b[k] = (unsigned long long)ep << 32;  // rows past the grid: zero, already "there"
          if (g < G) ld_tagged2(src + (size_t)g * (CPT * 8 * kAT), a[k], b[k]);
        }
        long long t0 = 0;
#ifdef SFFN_TRACE
        int tries = 0;
#endif
        for (;;) {
#ifdef SFFN_TRACE
          if (tt == 0 && g0 == rg && tries == 0 && p.trace) { asm volatile("" ::"l"(a[12]) : "memory"); TC_STAMP(9); }
          ++tries;
#endif
          bool all = true;
#pragma unroll
          for (int k = 0; k < kBatch; ++k) {
            if ((uint32_t)(a[k] >> 32) != ep || (uint32_t)(b[k] >> 32) != ep) {
              all = false;
              ld_tagged2(src + (size_t)(g0 + k * RG) * (CPT * 8 * kAT), a[k], b[k]);
            }
          }
          if (all) break;
          if (t0 == 0) t0 = clock64();
          if (ctl[kAbort]) { ok = false; break; }
          if (clock64() - t0 > p.wait_cycles) { raise_timeout(ctl, p.status, 21); ok = false; break; }
          __nanosleep(20);
        }
#ifdef SFFN_TRACE
        if (tt == 0 && g0 == rg && p.trace) { TC_STAMP(14); p.trace[(size_t)blockIdx.x * 16 + 15] = tries; }
#endif
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          sum.x += __uint_as_float((uint32_t)a[k]);
          sum.y += __uint_as_float((uint32_t)b[k]);
        }
      }
    }
    comb[rg * UW + u] = sum;
    named_bar_sync(5, kTail);
    if (tt < UW) {
      const int unit2 = slice * U + u0 + tt;
      const int col2 = 8 * ((unit2 % kAT) + (unit2 / (4 * kAT)) * kAT) + 2 * ((unit2 / kAT) & 3);
      if (u0 + tt < U && unit2 < units && col2 < D) {
        float2 t = make_float2(0.f, 0.f);
        for (int r = 0; r < RG; ++r) {
          t.x += comb[r * UW + tt].x;
          t.y += comb[r * UW + tt].y;
        }
        if (!ctl[kAbort] && failed == 0) *reinterpret_cast<float2*>(p.y + col2) = t;
      }
    }
    named_bar_sync(5, kTail);
  }
  abort_grace(ctl);
  if (tt == 0) TC_STAMP(13);
}

// ---- host side ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    cudaDriverEntryPointQueryResult q;
    void* ptr = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 matrix [H, D] seen as {64 elements, D / 64 K blocks, H neurons}; boxes of {64, 16, box_rows}.
bool make_gate_map(CUtensorMap* m, const void* base, int D, int H, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {64, (cuuint64_t)(D / 64), (cuuint64_t)H};
  const cuuint64_t strides[2] = {128, (cuuint64_t)D * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)kSegs, (cuuint32_t)box_rows};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The two tensor maps of a gate matrix, remembered per calling thread (encoding costs a few microseconds of host
// time, a decode loop comes back to the same few matrices).
struct MapEntry {
  const void* base;
  int D, H;
  alignas(64) CUtensorMap m8;
  alignas(64) CUtensorMap m1;
};
const MapEntry* gate_maps(const void* base, int D, int H) {
  constexpr int kEntries = 16;
  thread_local MapEntry cache[kEntries];
  thread_local int next = 0;
  for (int i = 0; i < kEntries; ++i)
    if (cache[i].base == base && cache[i].D == D && cache[i].H == H) return &cache[i];
  MapEntry* e = &cache[next];
  e->base = nullptr;
  if (!make_gate_map(&e->m8, base, D, H, kTileRows) || !make_gate_map(&e->m1, base, D, H, 1)) return nullptr;
  e->base = base; e->D = D; e->H = H;
  next = (next + 1) % kEntries;
  return e;
}

struct TcGeometry {
  int S, NA, E, act_slot_bytes, slab_max, kst, nacc, nf, rem_base, rem, cpt, smem, R;
  bool ok;
};

TcGeometry tc_plan(int D, int H, int grid) {
  TcGeometry g{};
  g.ok = false;
  if (D % 64 || D < 1024 || D > 8 * kAT * 8) return g;
  const int nvecD = D / 8;
  g.cpt = nvecD <= kAT ? 1 : nvecD <= 2 * kAT ? 2 : nvecD <= 4 * kAT ? 4 : 8;
  g.kst = (D / 64 + kSegs - 1) / kSegs;
  g.nacc = g.kst >= 2 ? 2 : 1;
  // CTAs that stay for the cross-CTA sum: one per 32 stored units of a partial, never more than half the grid (the
  // waiting CTAs of two calls that overlap must not hold every SM between them)
  const int units = g.cpt * 4 * kAT;
  g.R = std::min(std::max(1, (grid - 1) / 2), std::max(1, units / 32));
  g.nf = (H / kTileRows) / grid;
  g.rem_base = g.nf * grid * kTileRows;
  g.rem = H - g.rem_base;
  g.slab_max = g.nf * kTileRows + (g.rem + grid - 1) / grid;
  g.act_slot_bytes = (2 * D * 2 + 1023) / 1024 * 1024;
  // a slot that is nearly a whole number of gate stages is padded to it: it can then park gate stages at the start
  const int whole = (g.act_slot_bytes + kStageBytes - 1) / kStageBytes * kStageBytes;
  if (whole - g.act_slot_bytes <= g.act_slot_bytes / 8) g.act_slot_bytes = whole;
  const TcLayout fixed(0, 0, 0, g.slab_max, g.kst);
  const int ring = kSmemBudget - fixed.total - 1024;  // 1024: barrier words and gate values per slot
  // Gate slots first (an even number, each issuer and producer owns alternate ones), at least four act slots
  // where they fit so that the act warps can take two rows per round.
  int na = ring >= 6 * kStageBytes + 4 * g.act_slot_bytes ? 4 : 2;
  int s = (ring - na * g.act_slot_bytes) / kStageBytes & ~1;
  if (s > 12) s = 12;
  if (s < 2) return g;
  na = (ring - s * kStageBytes) / g.act_slot_bytes;
  if (na > 16) na = 16;
  if (na < 3 && s >= 6) {  // wide rows: a third act slot is worth two gate slots
    s -= 2;
    na = (ring - s * kStageBytes) / g.act_slot_bytes;
  }
  const FusedTestKnobs& knobs = fused_test_knobs();
  if (knobs.ring_S > 0 && knobs.ring_NA > 0) { s = knobs.ring_S & ~1; na = knobs.ring_NA; }
  if (s < 2 || na < 2) return g;
  g.S = s; g.NA = na;
  // gate stages parked in the last act slots at the start of a call: all but the first slot, an even number of stages
  g.E = 0;
  if (g.act_slot_bytes % kStageBytes == 0) {
    const int per = g.act_slot_bytes / kStageBytes;
    int e = (na - 1) * per;
    if (knobs.ring_E >= 0) e = knobs.ring_E < e ? knobs.ring_E : e;
    e = e / per * per;
    if (e > kMaxParked) e = kMaxParked / per * per;
    if (e & 1) e -= per;
    g.E = e < 0 ? 0 : e;
  }
  const TcLayout full(s, na, g.act_slot_bytes, g.slab_max, g.kst);
  g.smem = full.total;
  g.ok = g.smem <= kSmemBudget;
  return g;
}

int tc_grid(int sm_count, int H) {
  int grid = sm_count < kMaxGrid ? sm_count : kMaxGrid;
  return grid > H ? H : grid;
}

}  // namespace

bool fused_tc_supported(int wkind, int D, int H, int B, const sffn_gate* gate, int sm_count) {
  if (B != 1 || wkind != kWBF16 || gate->kind != SFFN_GATE_STANDARD) return false;
  return tc_plan(D, H, tc_grid(sm_count, H)).ok && encode_fn() != nullptr;
}

cudaError_t launch_fused_tc(const FusedCall& c, cudaStream_t s, int* launched) {
  const int grid = tc_grid(c.sm_count, c.H);
  const TcGeometry g = tc_plan(c.D, c.H, grid);
  if (!g.ok) return cudaErrorInvalidValue;
  const MapEntry* maps = gate_maps(c.gate->W_g, c.D, c.H);
  if (!maps) return cudaErrorNotSupported;
  char* ws = static_cast<char*>(c.workspace);
  TcParams p{};
  p.D = c.D; p.H = c.H;
  p.W_up = c.W_up; p.W_down = c.W_down; p.x = c.x; p.b_g = c.b_g;
  p.done_counter = reinterpret_cast<unsigned long long*>(ws) + 1;
  p.epoch_word = reinterpret_cast<uint32_t*>(ws + 16);
  p.y = c.y;
  p.partial = reinterpret_cast<unsigned long long*>(ws + fused_tagged_partials_offset(c.D, c.r_max));
  p.flag = c.flag; p.status = c.status;
  p.act = c.act; p.dense = c.dense ? 1 : 0; p.act_up = c.act_up;
  p.S = g.S; p.NA = g.NA; p.E = g.E;
  p.act_slot_bytes = g.act_slot_bytes; p.slab_max = g.slab_max; p.kst = g.kst; p.nacc = g.nacc;
  p.nf = g.nf; p.rem_base = g.rem_base; p.rem = g.rem; p.R = g.R;
  p.l2_hints = fused_test_knobs().l2_hints;
  p.wait_cycles = fused_test_knobs().wait_cycles;
  p.skip_arrival_cta = fused_test_knobs().skip_arrival_cta;
  p.trace = fused_test_knobs().trace;
  void (*k)(const TcParams, const CUtensorMap, const CUtensorMap) = nullptr;
  switch (g.cpt) {
    case 1: k = fused_tc_kernel<1>; break;
    case 2: k = fused_tc_kernel<2>; break;
    case 4: k = fused_tc_kernel<4>; break;
    default: k = fused_tc_kernel<8>; break;
  }
  static unsigned long long configured[4] = {0, 0, 0, 0};
  const int slot = g.cpt == 1 ? 0 : g.cpt == 2 ? 1 : g.cpt == 4 ? 2 : 3;
  cudaError_t e = allow_dynamic_smem(k, kSmemBudget, configured[slot]);
  if (e != cudaSuccess) return e;
  e = launch_pdl(k, dim3(grid), dim3(kThreads), (size_t)g.smem, s, p, maps->m8, maps->m1);
  if (e != cudaSuccess) return e;
  if (launched) *launched = 1;
  return cudaSuccess;
}

}  // namespace sffn
