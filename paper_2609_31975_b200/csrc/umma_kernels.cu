// Batched path on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM), bf16 storage.
//
//   umma_rows_kernel<GATE>  Z[H, B] = W[H, K] X[B, K]^T + bias (+ fixed-matrix term), activation, gate values,
//                           "any token fires" bit per neuron             (Eq. 1 gate / LoPA U and V stages, batched)
//   umma_rows_kernel<UP>    compacts those bits into the union list of fired neurons (Sec. 5.4), then over that
//                           list: Up = W_up[idx] X^T, Hm = a . A_3(Up), stored as bf16 HmT[b][u]
//   umma_down_kernel        partial[split][b][d] = sum over the split's list rows u of HmT[b][u] W_down[idx[u]][d]
//   rmsnorm_split_kernel    LoPA: n = RMSNorm(v) as bf16 high / low pairs (the B operand of the U stage)
//
// Rows kernels: one CTA owns a tile of up to 128 weight rows (TMEM lanes) x Npad token columns (Npad = columns
// rounded up to 16); tiles of up to 64 rows use M = 64:
//   warps 0-3  producers: TMA tensor-map copies bring the tile's weight rows and the Npad token rows of a stage's
//              64-wide K blocks into the 128-byte-swizzled K-major layout the tensor core reads (mbarrier
//              complete_tx).  Gate: one tiled copy of the tile's consecutive rows per block.  Union rows:
//              tile::gather4, each lane of the warp fetching four listed rows.
//   warps 8-11 one thread each issues tcgen05.mma (N=Npad, K=16, four per K block) for "its" ring slots into an
//              accumulator of its own and commits each stage's completion to the "slot free" mbarrier.  The serial
//              wait - issue - commit chain of one thread takes on the order of a thousand cycles per stage whatever
//              the MMA shape, so several issuers (four when the ring divides evenly among them, else two) are what
//              lets the copies run at memory speed; warp 8 allocates and frees the TMEM columns
//   warps 4-7  epilogue: tcgen05.ld the accumulator row of "their" neuron (all accumulators added), apply the
//              gate / scale epilogue; for wide batches all twelve warps share the epilogue of the CTA's last tile
// A tile has 128 rows when a CTA owns several tiles; a smaller problem is cut into one tile per SM.  The ring of
// stages (up to 12) is cut out of the dynamic shared memory on the device, once the tile height is known.
// Every kernel here is launched with programmatic dependent launch: set-up first, griddepcontrol.wait before the
// first dependent read or global write.
// Weight-only int8 / int4 rows (QB = 8 / 4): the copies bring the codes (and the token rows) into the ring slots;
// four more warps (the last four of the CTA, two pairs that alternate over the stages) expand the codes to bf16 --
// every code is an integer bf16 holds exactly -- in the swizzled layout, into a short ring of expanded blocks of
// its own (rows kernels) or the slot's block area (down kernel), and arrive on a "ready" barrier that the MMA
// issuers wait for instead of "full"; the row scales are applied to the accumulator rows in the epilogue (the
// down projection's are folded into Hm).  With the weights as the A operand the tensor core takes 32 bytes of
// bf16 per cycle and SM whatever the token count, i.e. 16 codes per cycle: quantised batches are bound by that
// rate, not by their bytes.
// Every wait is bounded by a cycle budget; on expiry the status word is set, all roles wind down and the TMEM
// columns are released before the CTA exits.
#include "umma_kernels.cuh"

#include <cuda.h>

#include "common.cuh"
#include "fused_kernel.cuh"
#include "sparse_ffn.h"

namespace sffn {

static_assert(kUmmaActIdentity == kActNone, "identity epilogue code");

namespace {

constexpr int kTileRows = 128;
constexpr int kAtomK = 64;                           // bf16 elements of one 128-byte swizzle row
constexpr int kAAtomBytes = kTileRows * 128;         // 16 KB: one [128 rows x 64 k] swizzled block
constexpr int kThreads = 320;                        // 4 producer warps, 4 epilogue warps, 2 MMA warps
constexpr int kThreadsRows = 384;                    // rows kernels: up to 4 MMA warps
constexpr int kProducerWarps = 4;
constexpr int kMaxStages = 16;                       // barrier slots; bf16 rows use up to 12
constexpr int kMaxStagesBf16 = 12;
constexpr int kExpandSlots = 4;                      // quantised rows: ring of expanded bf16 blocks
constexpr int kWalkMinTokens = 32;                   // batches from which the up kernel may walk every row
constexpr int kWalkAllPercent = 70;                  // union share of the rows from which "every row" is walked
constexpr int kMaxIssuers = 4;
constexpr int kExpandWarps = 4;                      // quantised rows: warps that expand the codes to bf16
constexpr int kScanChunks = 4;                       // in-kernel compaction: up to 4 * 384 mask words = 384 gate tiles
constexpr int kMaxOwnTiles = 8;                      // tiles of one CTA whose rows are kept in shared memory
constexpr int kHeaderBytes = 1024 + kMaxOwnTiles * kTileRows * 4;  // barriers + scratch, then the row lists

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          long long budget) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > budget) {
      *abort_flag = 1;
      atomicExch(status, (int32_t)SFFN_ERR_TIMEOUT);
      return false;
    }
  }
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 bytes apart, groups of
// eight rows 1024 bytes apart (stride byte offset), descriptor version 1 (Blackwell).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3fff);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset
  d |= (uint64_t)1 << 46;                            // version
  d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
  return d;
}
// The same for an MN-major operand (here: A[m][k] stored as rows k of 64 contiguous m, 128 bytes each):
// eight k rows form a 1024-byte swizzle atom; `k_group_bytes` apart lie successive groups of eight k rows
// (stride byte offset), `mn_atom_bytes` apart successive blocks of 64 m (leading byte offset).
__device__ __forceinline__ uint64_t make_desc_mn(uint32_t smem_addr, uint32_t mn_atom_bytes, uint32_t k_group_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3fff);
  d |= (uint64_t)((mn_atom_bytes >> 4) & 0x3fff) << 16;
  d |= (uint64_t)((k_group_bytes >> 4) & 0x3fff) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = m (64 or 128), N = n.
__device__ __forceinline__ uint32_t make_idesc(int n, int m = kTileRows) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same for int8 operands (D int32, A and B signed 8-bit, both K-major; one MMA covers K = 32).
__device__ __forceinline__ uint32_t make_idesc_i8(int n, int m = kTileRows) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8_raw(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
// Eight accumulator columns of this thread's TMEM lane, summed over the `nacc` (1, 2 or 4) accumulators
// that lie `stride` columns apart.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, int nacc, int stride, float* v) {
  uint32_t r0[8], r1[8], r2[8], r3[8];
  tmem_ld8_raw(taddr, r0);
  if (nacc >= 2) tmem_ld8_raw(taddr + stride, r1);
  if (nacc == 4) {
    tmem_ld8_raw(taddr + 2 * stride, r2);
    tmem_ld8_raw(taddr + 3 * stride, r3);
  }
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float a = __uint_as_float(r0[i]);
    if (nacc >= 2) a += __uint_as_float(r1[i]);
    if (nacc == 4) a += __uint_as_float(r2[i]) + __uint_as_float(r3[i]);
    v[i] = a;
  }
}

// The same for int32 accumulators (summed exactly).
__device__ __forceinline__ void tmem_ld8_int(uint32_t taddr, int nacc, int stride, int* v) {
  uint32_t r0[8], r1[8], r2[8], r3[8];
  tmem_ld8_raw(taddr, r0);
  if (nacc >= 2) tmem_ld8_raw(taddr + stride, r1);
  if (nacc == 4) {
    tmem_ld8_raw(taddr + 2 * stride, r2);
    tmem_ld8_raw(taddr + 3 * stride, r3);
  }
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int a = (int)r0[i];
    if (nacc >= 2) a += (int)r1[i];
    if (nacc == 4) a += (int)r2[i] + (int)r3[i];
    v[i] = a;
  }
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Tiled tensor-map copy: box {64 elements, rows} at (element c0, row c1); out-of-range rows read as zero.
__device__ __forceinline__ void tma_tile_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
// Gather copy: four rows r0..r3 (any order) x 64 elements starting at element c0 land as four
// consecutive 128-byte rows at dst (the map's box is {64, 1}).
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* map, int c0, int r0, int r1, int r2,
                                            int r3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, "
      "%4, %5, %6}], [%7];" ::"r"(dst),
      "l"(map), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
      : "memory");
}

// Expands a block of weight codes to bf16: `raw` holds [rows][64] codes (QB = 8: a byte each, +-127; QB = 4: two's-
// complement nibbles, even column in the low nibble), `dst` (1024-byte aligned) receives [rows][64] bf16 in the
// 128-byte-swizzled K-major layout (16-byte chunk c of row i at i * 128 + ((c ^ (i & 7)) * 16)).  Thread t of nthr
// takes the 16-code quarter t % 4 of rows t / 4, t / 4 + nthr / 4, ... (four of them in flight): a quarter warp reads two whole raw rows
// and writes chunks of two rows that share no bank.  A code c becomes the fp32 2^23 + (c + bias) by a byte
// permute, the bias and 2^23 are subtracted exactly, and the upper half of that fp32 is the bf16.
template <int QB>
__device__ __forceinline__ void expand_block(uint32_t raw, uint32_t dst, int rows, int t, int nthr) {
  constexpr int kRawRow = 8 * QB;  // bytes of 64 codes
  constexpr int kUnroll = 4;       // rows of one thread in flight
  const int c = t & 3, step = nthr >> 2;
  for (int row0 = t >> 2; row0 < rows; row0 += kUnroll * step) {
    uint32_t w[kUnroll][4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int row = row0 + u * step;
      const uint32_t src = raw + row * kRawRow + c * (kRawRow / 4);
      w[u][0] = w[u][1] = w[u][2] = w[u][3] = 0;
      if (row < rows) {
        if (QB == 8) {
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(w[u][0]), "=r"(w[u][1]), "=r"(w[u][2]), "=r"(w[u][3])
                       : "r"(src));
        } else {
          asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(w[u][0]), "=r"(w[u][1]) : "r"(src));
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int row = row0 + u * step;
      if (row >= rows) break;
      if (QB == 4) {
        const uint32_t a = w[u][0] ^ 0x88888888u, b = w[u][1] ^ 0x88888888u;
        // bytes of w[2i]: even columns of word i, of w[2i+1]: odd columns
        w[u][0] = a & 0x0f0f0f0fu; w[u][1] = (a >> 4) & 0x0f0f0f0fu;
        w[u][2] = b & 0x0f0f0f0fu; w[u][3] = (b >> 4) & 0x0f0f0f0fu;
      }
      uint32_t o[8];
      const float off = QB == 8 ? 8388736.f : 8388616.f;  // 2^23 + 128, 2^23 + 8
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        // o[i] = codes 2i, 2i+1 of the quarter
        uint32_t lo, hi;
        if (QB == 8) {
          const uint32_t v = w[u][i >> 1] ^ 0x80808080u;
          lo = __byte_perm(v, 0x4b000000u, (i & 1) ? 0x7442 : 0x7440);
          hi = __byte_perm(v, 0x4b000000u, (i & 1) ? 0x7443 : 0x7441);
        } else {
          const uint32_t sel = 0x7440 + (i & 3);
          lo = __byte_perm(w[u][(i >> 2) * 2], 0x4b000000u, sel);
          hi = __byte_perm(w[u][(i >> 2) * 2 + 1], 0x4b000000u, sel);
        }
        const float fl = __uint_as_float(lo) - off, fh = __uint_as_float(hi) - off;
        o[i] = __byte_perm(__float_as_uint(fl), __float_as_uint(fh), 0x7632);
      }
      const uint32_t drow = dst + row * 128;
      const int sw = row & 7;
      asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(drow + (((2 * c) ^ sw) << 4)), "r"(o[0]), "r"(o[1]),
                   "r"(o[2]), "r"(o[3])
                   : "memory");
      asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(drow + (((2 * c + 1) ^ sw) << 4)), "r"(o[4]), "r"(o[5]),
                   "r"(o[6]), "r"(o[7])
                   : "memory");
    }
  }
}
// The same for int4 codes on their way to the int8 MMA: `raw` holds [rows][128] nibbles (64 bytes a row), `dst`
// receives [rows][128] bytes, each 16 x its code (the nibble moved to the upper half of the byte: exact, and the factor
// goes into the row scale), in the same swizzled layout.  Thread t takes the 32 codes of quarter t % 4 of its rows: one
// 16-byte load, two 16-byte stores; per word of eight nibbles two masks and two byte permutes.
__device__ __forceinline__ void expand_block_q4_i8(uint32_t raw, uint32_t dst, int rows, int t, int nthr) {
  const int c = t & 3, step = nthr >> 2;
  for (int row = t >> 2; row < rows; row += step) {
    uint32_t w[4], o[8];
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(raw + row * 64 + c * 16));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t ev = (w[i] << 4) & 0xf0f0f0f0u, od = w[i] & 0xf0f0f0f0u;  // even / odd columns, times 16
      o[2 * i] = __byte_perm(ev, od, 0x5140);
      o[2 * i + 1] = __byte_perm(ev, od, 0x7362);
    }
    const uint32_t drow = dst + row * 128;
    const int sw = row & 7;
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(drow + (((2 * c) ^ sw) << 4)), "r"(o[0]), "r"(o[1]),
                 "r"(o[2]), "r"(o[3])
                 : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(drow + (((2 * c + 1) ^ sw) << 4)), "r"(o[4]), "r"(o[5]),
                 "r"(o[6]), "r"(o[7])
                 : "memory");
  }
}
// Makes this thread's shared-memory stores visible to the tensor core's reads.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Rows per tile: 128 when there is more than one tile per CTA, otherwise the row count spread over
// the whole grid (a multiple of 8, the swizzle period), so that every SM streams a share.
__host__ __device__ inline int tile_rows_for(int n_rows, int grid) {
  if (n_rows >= kTileRows * grid) return kTileRows;
  int t = ((n_rows + grid - 1) / grid + 7) & ~7;
  return t < 8 ? 8 : t > kTileRows ? kTileRows : t;
}

__host__ __device__ inline uint32_t tmem_cols_for(int cols) {
  return cols <= 32 ? 32 : cols <= 64 ? 64 : cols <= 128 ? 128 : cols <= 256 ? 256 : 512;
}

// Third tensor map of the up kernel that may walk every row (tiled boxes over all rows); empty otherwise, so
// that the other instantiations keep their two-map signature.
template <bool HAS>
struct WalkMap {
  CUtensorMap m;
  __device__ const CUtensorMap* get() const { return &m; }
};
template <>
struct WalkMap<false> {
  __device__ const CUtensorMap* get() const { return nullptr; }
};

enum RowsMode { kGate = 0, kUp = 1, kUpMayWalk = 2 };  // kUpMayWalk: wide batches, see walk_all below

template <int MODE, int QB>
__global__ void __launch_bounds__(kThreadsRows + ((QB == 8 || QB == 4 || QB == 2) ? 32 * kExpandWarps : 0), 1) umma_rows_kernel(const UmmaRowsParams p,
                                                                  const __grid_constant__ CUtensorMap map_w,
                                                                  const __grid_constant__ CUtensorMap map_x,
                                                                  const __grid_constant__ WalkMap<MODE == kUpMayWalk> map_t) {
  constexpr bool UP = MODE != kGate;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  // carve: stages first (1024-byte aligned), then barriers and control words
  const int npad = p.npad;
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // header: barriers (for the largest ring) and control words, scan scratch, this CTA's rows of the union
  // list; then the ring of stages, whose geometry is decided below once the tile height is known
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
  int* scan_wt = reinterpret_cast<int*>(smem + 512);   // [kScanChunks][warps]
  int* rows_sm = reinterpret_cast<int*>(smem + 1024);  // [kMaxOwnTiles][128]
  const uint32_t stage0 = smem_u32(smem) + kHeaderBytes;
  const uint32_t full = smem_u32(bars), empty = smem_u32(bars + kMaxStages);
  const uint32_t acc_full = smem_u32(bars + 2 * kMaxStages), acc_empty = smem_u32(bars + 2 * kMaxStages + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t ready = smem_u32(bars + 2 * kMaxStages + 4);  // quantised rows: slot t of the bf16 ring is written ...
  const uint32_t afree = ready + 8 * kExpandSlots;             // ... and has been read by its MMAs
  constexpr int kRawRow = QB == 2 ? 64 : 8 * QB;               // bytes of the codes of one K block (as copied)
  // QB = 1: int8 rows and the tokens as int8 limbs (four per token, see token_limbs_kernel) go straight into
  // kind::i8 MMAs with int32 accumulators: nothing to expand, a K block is 128 codes.  QB = 8 / 4: codes expanded
  // to bf16 by four more warps.
  // QB = 2: int4 rows expanded to int8 (16 x the code, a byte each) for the same kind::i8 MMAs.
  constexpr bool kNat = QB == 1 || QB == 2, kExp = QB == 8 || QB == 4 || QB == 2, kQ = QB != 0;
  constexpr int kAtomElems = kNat ? 128 : kAtomK;              // elements of one 128-byte swizzle row

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int kblocks = p.K / kAtomElems;

  // Set-up that needs nothing from earlier kernels runs while the predecessor in the stream finishes.
  pdl_launch_dependents();
  const int max_acc = npad > 128 ? 2 : kMaxIssuers;  // 512 TMEM columns: wide token blocks leave room for two accumulators
  const uint32_t tmem_cols = tmem_cols_for(max_acc * npad);
  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(full + 8 * s, 1);  // the producer's expect_tx arrive; the copies complete the bytes
      mbar_init(empty + 8 * s, 1);
    }
    if (kExp)
      for (int t = 0; t < kExpandSlots; ++t) {
        mbar_init(ready + 8 * t, kExpandWarps / 2);
        mbar_init(afree + 8 * t, 1);
      }
    mbar_init(acc_empty, 128);
    *abort_flag = 0;
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // The up kernel needs the gate's results from here on.  The gate kernel's tiles depend on nothing but its
  // own arguments, and its weights are parameters: its producers fill the ring before they wait (see below),
  // every other role of it waits just before its first dependent access.
  if (MODE != kGate) pdl_wait();

  // Union rows: either the list is given (idx, count), or every CTA compacts the gate's "fired" bit masks
  // itself.  The gate kernel leaves one 32-bit word per epilogue warp and tile (word 4 * tile + warp, bit =
  // lane = row rows_per_word * warp + lane of the tile, 32 rows per word for M = 128 tiles, 16 for M = 64); thread t takes word t of each chunk of `threads` words, a
  // warp scan plus the warp totals of all chunks give the list position of its first set bit.
  const bool own_list = UP && p.words_in != nullptr;
  uint32_t bits[kScanChunks];
  int first_pos[kScanChunks];
  int n_rows;
  const int nch = own_list ? (p.n_words + kThreadsRows - 1) / kThreadsRows : 0;
  if (own_list) {
#pragma unroll
    for (int k = 0; k < kScanChunks; ++k) {
      const int w = k * kThreadsRows + tid;
      bits[k] = (k < nch && tid < kThreadsRows && w < p.n_words) ? __ldcg(p.words_in + w) : 0u;
    }
#pragma unroll
    for (int k = 0; k < kScanChunks; ++k) {
      if (k < nch) {
        int incl = __popc(bits[k]);
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += t;
        }
        first_pos[k] = incl - __popc(bits[k]);
        if (lane == 31 && warp < kThreadsRows / 32) scan_wt[k * (kThreadsRows / 32) + warp] = incl;
      }
    }
    __syncthreads();
    int run = 0;
#pragma unroll
    for (int k = 0; k < kScanChunks; ++k) {
      if (k < nch) {
        int before = 0, total = 0;
        for (int w = 0; w < kThreadsRows / 32; ++w) {
          const int t = scan_wt[k * (kThreadsRows / 32) + w];
          before += w < warp ? t : 0;
          total += t;
        }
        first_pos[k] += run + before;
        run += total;
      }
    }
    n_rows = run;
  } else {
    n_rows = p.count ? *p.count : p.R;
  }
  // A union that covers most of the rows is cheaper to walk as "every row" with tiled copies (which stream about
  // 1.5x faster than gathered rows) than as a list: unfired rows have a = 0 for every token, so their h is 0.
  // The list and its length are still published; the down kernel is told through *walk_all to do the same.
  const int n_listed = n_rows;
  const bool walk_all = MODE == kUpMayWalk && own_list && p.walk_all &&
                        (long long)n_listed * 100 >= (long long)p.R * kWalkAllPercent;
  if (walk_all) n_rows = p.R;
  const int tile_rows = tile_rows_for(n_rows, gridDim.x);
  const int n_tiles = (n_rows + tile_rows - 1) / tile_rows;
  if (own_list && walk_all) {
    // publish the list only: word w is written out by CTA w mod grid
#pragma unroll
    for (int k = 0; k < kScanChunks; ++k) {
      const int w = k * kThreadsRows + tid;
      if (k < nch && bits[k] && w % (int)gridDim.x == (int)blockIdx.x) {
        const int j0 = (w >> 2) * p.gate_tile_rows + (w & 3) * p.gate_rows_per_word;
        uint32_t rest = bits[k];
        int li = first_pos[k];
        while (rest) {
          const int q = __ffs(rest) - 1;
          rest &= rest - 1;
          p.idx_out[li++] = j0 + q;
        }
      }
    }
    if (blockIdx.x == 0 && tid == 0) {
      *p.count_out = n_listed;
      *p.walk_all = 1;
    }
  } else if (own_list) {
    if (blockIdx.x == 0 && tid == 0 && p.walk_all) *p.walk_all = 0;
    // keep the rows of this CTA's tiles in shared memory and publish them (and the length) for the
    // down projection and the caller: every list position belongs to exactly one CTA's tile
#pragma unroll
    for (int k = 0; k < kScanChunks; ++k) {
      if (k < nch && bits[k]) {
        const int cnt = __popc(bits[k]);
        const int w = k * kThreadsRows + tid;
        const int j0 = (w >> 2) * p.gate_tile_rows + (w & 3) * p.gate_rows_per_word;  // row of bit 0
        int m = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++m) {
          const int lo = tile * tile_rows, hi = lo + tile_rows;
          if (first_pos[k] + cnt <= lo || first_pos[k] >= hi) continue;
          uint32_t rest = bits[k];
          int li = first_pos[k];
          while (rest) {
            const int q = __ffs(rest) - 1;
            rest &= rest - 1;
            if (li >= lo && li < hi) {
              rows_sm[m * kTileRows + li - lo] = j0 + q;
              p.idx_out[li] = j0 + q;
            }
            ++li;
          }
        }
      }
    }
    if (blockIdx.x == 0 && tid == 0) *p.count_out = n_rows;
  }
  // Stage geometry.  Tiles of up to 64 rows are multiplied with M = 64 (accumulator row i then sits in TMEM lane
  // 32 * (i / 16) + i % 16), taller ones with M = 128 (row i in lane i).  A stage holds `atoms` successive K
  // blocks of the tile -- short tiles take several, so that a stage stays near 16 KB and the bytes in flight do
  // not shrink with the tile -- followed by the token rows of the same K blocks.  Block a sits tile_rows * 128
  // bytes after block a - 1; its MMA reads M rows from its start, i.e. on into the following blocks and the
  // token rows of the same stage (rows that are ignored); the stage is sized so that it never reads past it.
  const bool m64 = tile_rows <= 64;
  const int mrows = m64 ? 64 : kTileRows;
  int atoms = kTileRows / tile_rows;
  const int atoms_cap = npad <= 16 ? 4 : npad <= 32 ? 2 : 1;  // at most 8 KB of token rows per stage
  atoms = atoms > atoms_cap ? atoms_cap : atoms;
  const int a_block_bytes = tile_rows * 128, b_block_bytes = npad * 128;
  // bytes of the bf16 weight blocks of a stage, including what the last block's MMA reads past its rows
  const int a_bytes = (max(atoms * a_block_bytes, (atoms - 1) * a_block_bytes + mrows * 128) + 1023) & ~1023;
  const int raw_block_bytes = tile_rows * kRawRow;
  // bf16 rows: a slot holds the weight blocks, then the token rows.  Quantised rows: the ring slots hold what the
  // copies bring (token rows, then the codes), and the expanded bf16 blocks have a short ring of their own (stage
  // `it` uses slot it mod 4 of it): the codes in flight, not the expanded blocks, are what has to cover the memory
  // latency.
  const int b_off = kExp ? 0 : atoms * a_block_bytes;           // token rows within a ring slot
  const int w_off = kExp ? atoms * b_block_bytes : 0;           // weights (as copied) within a ring slot
  int stage_bytes = kExp ? atoms * (b_block_bytes + raw_block_bytes) : max(atoms * (a_block_bytes + b_block_bytes), a_bytes);
  stage_bytes = (stage_bytes + 1023) & ~1023;
  const uint32_t ring0 = stage0 + (kExp ? kExpandSlots * a_bytes : 0);
  int S = (p.ring_bytes - (kExp ? kExpandSlots * a_bytes : 0)) / stage_bytes;
  S = S > (kExp ? kMaxStages : kMaxStagesBf16) ? (kExp ? kMaxStages : kMaxStagesBf16) : S;
  // four issuers when the ring divides evenly among them, otherwise two (slot mod issuers = owner)
  int issuers = (S >= 8 && S % 4 == 0) ? 4 : kExp && S >= 4 ? 4 : 2;
  S &= (kExp && S >= 4) ? ~3 : ~1;
  issuers = issuers > max_acc ? max_acc : issuers;
  const int kstages = (kblocks + atoms - 1) / atoms;
  // accumulator row that this thread's TMEM lane holds (-1: none); the same for every warp of a lane quarter
  const int row_thr = m64 ? (lane < 16 ? (warp & 3) * 16 + lane : -1) : (warp & 3) * 32 + lane;
  // The MMA issuers take the stages of their ring slots (slot mod issuers) into accumulators of their own
  // (npad TMEM columns each); the epilogue adds them.  A tile with at least as many stages as issuers
  // gives each issuer a stage; shorter tiles use fewer issuers.
  const int nacc = kstages >= issuers ? issuers : kstages >= 2 ? 2 : 1;
  if (tid == 0) {
    mbar_init(acc_full, nacc);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Epilogue of one tile for the token-column groups c0 = 8 * part, 8 * (part + nparts), ...: waits for the
  // tile's accumulators, then (gate) adds the fixed-matrix term and the bias, applies the activation and
  // stores the gate values, reporting whether any token fired; (union rows) scales by the gate values
  // and stores HmT.  Returns false if the wait was abandoned.
  const bool share_last = npad >= 32;  // four or more column groups: worth spreading over all warps
  // `shared`: all twelve warps take part.  Only the epilogue warps have followed the accumulator barrier through
  // every earlier tile (a warp that joins for the last tile could find it still in an earlier phase, which a parity
  // wait cannot tell from "complete"), so they wait for it and the others meet them at a named barrier.
  auto epilogue = [&](int tile, int tcount, int part, int nparts, bool shared, bool& fired) -> bool {
    const int row_in_tile = row_thr;
    const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const int B = p.B;
    const int li = tile * tile_rows + row_in_tile;
    const bool row_ok = row_in_tile >= 0 && row_in_tile < tile_rows && li < n_rows;
    int j = !row_ok ? 0 : (own_list && !walk_all) ? rows_sm[tcount * kTileRows + row_in_tile] : p.idx ? p.idx[li] : li;
    if (!SFFN_IN_BOUNDS(j >= 0 && j < p.R, p.status, 40)) j = 0;
    // everything that does not depend on the accumulator is fetched before the wait
    if (MODE == kGate) pdl_wait();  // before the first read of a buffer an earlier kernel may write, and the first store
    float bias = 0.f, sg = 1.f;
    const float sc = ((kQ && row_ok && p.w_scale) ? p.w_scale[j] : 1.f) * (QB == 2 ? 0.0625f : 1.f);  // scale of the weight row
    const float osc = (kQ && UP && row_ok && p.out_scale) ? p.out_scale[j] : 1.f;  // scale of the down row, folded into Hm
    int gi = -1;
    float pre[16];  // union rows: the gate values of this thread's first two column groups
    if (UP) {
#pragma unroll
      for (int g = 0; g < 2; ++g)
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int b = 8 * (part + g * nparts) + q;
          pre[8 * g + q] = (row_ok && b < B) ? p.a[(size_t)b * p.a_stride + j] : 0.f;
        }
    } else {
      bias = (row_ok && p.b_g) ? p.b_g[j] : 0.f;
      gi = (row_ok && p.g_idx) ? p.g_idx[j] : -1;
      sg = (row_ok && p.g_sign && p.g_sign[j] < 0) ? -1.f : 1.f;
    }
    int okw = 1;
    if (!shared || (warp >= 4 && warp < 8)) {
      if (lane == 0) okw = mbar_wait(acc_full, tcount & 1, abort_flag, p.status, p.wait_cycles) ? 1 : 0;
      okw = __shfl_sync(0xffffffffu, okw, 0);
    }
    if (shared) {
      tc_fence_before();
      named_bar_sync(3, kThreadsRows);  // reached by all twelve warps whatever happened before
      if (*abort_flag) okw = 0;
    }
    if (!okw) return false;
    tc_fence_after();
    if constexpr (kNat) {
      // int32 accumulators, four columns per token (its limbs, most significant first, 7 bits apart):
      // value = token scale * row scale * (i0 + i1 / 128 + i2 / 128^2 + i3 / 128^3)
      __nv_bfloat16* hm = static_cast<__nv_bfloat16*>(p.hmT) + li;
      float* arow = p.a_out + j;
      const __nv_bfloat16* xg = static_cast<const __nv_bfloat16*>(p.xtok) + (gi >= 0 ? gi : 0);
      for (int c0 = 8 * part; c0 < npad; c0 += 8 * nparts) {
        int iv[8];
        tmem_ld8_int(taddr + c0, nacc, npad, iv);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int b = c0 / 4 + q;
          if (row_ok && b < B) {
            const float val = p.tok_scale[b] * sc *
                              (((float)iv[4 * q] + (float)iv[4 * q + 1] * 0.0078125f) +
                               ((float)iv[4 * q + 2] * 6.103515625e-05f + (float)iv[4 * q + 3] * 4.76837158203125e-07f));
            if (UP) {
              const float av = p.a[(size_t)b * p.a_stride + j];
              hm[(size_t)b * p.hm_stride] = __float2bfloat16(av * activation(p.act_up, val) * osc);
            } else {
              float z = val + bias;
              if (gi >= 0) z += sg * __bfloat162float(xg[(size_t)b * p.xtok_stride]);
              fired |= z > 0.f;
              arow[(size_t)b * p.a_stride] = activation(p.act, z);
            }
          }
        }
      }
      return true;
    }
    if (UP) {
      __nv_bfloat16* hm = static_cast<__nv_bfloat16*>(p.hmT) + li;
      const float* arow = p.a + j;
      const int act_up = p.act_up;
      int g = 0;
      for (int c0 = 8 * part; c0 < npad; c0 += 8 * nparts, ++g) {
        float av[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
          av[q] = g == 0 ? pre[q] : g == 1 ? pre[8 + q] : (row_ok && c0 + q < B) ? arow[(size_t)(c0 + q) * p.a_stride] : 0.f;
        float v[8];
        tmem_ld8(taddr + c0, nacc, npad, v);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (row_ok && c0 + q < B)
            hm[(size_t)(c0 + q) * p.hm_stride] =
                __float2bfloat16(kQ ? av[q] * activation(act_up, v[q] * sc) * osc : av[q] * activation(act_up, v[q]));
      }
    } else {
      const int act = p.act;
      float* arow = p.a_out + j;
      const __nv_bfloat16* xg = static_cast<const __nv_bfloat16*>(p.xtok) + (gi >= 0 ? gi : 0);
      if (p.split_cols) {
        for (int c0 = 8 * part; c0 < npad; c0 += 8 * nparts) {
          float v[8];
          tmem_ld8(taddr + c0, nacc, npad, v);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int b = c0 / 2 + q;
            if (row_ok && b < B) {
              float z = kQ ? (v[2 * q] + v[2 * q + 1]) * sc + bias : v[2 * q] + v[2 * q + 1] + bias;
              if (gi >= 0) z += sg * __bfloat162float(xg[(size_t)b * p.xtok_stride]);
              fired |= z > 0.f;
              arow[(size_t)b * p.a_stride] = activation(act, z);
            }
          }
        }
      } else {
        for (int c0 = 8 * part; c0 < npad; c0 += 8 * nparts) {
          float v[8];
          tmem_ld8(taddr + c0, nacc, npad, v);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int b = c0 + q;
            if (row_ok && b < B) {
              float z = kQ ? v[q] * sc + bias : v[q] + bias;
              if (gi >= 0) z += sg * __bfloat162float(xg[(size_t)b * p.xtok_stride]);
              fired |= z > 0.f;
              arow[(size_t)b * p.a_stride] = activation(act, z);
            }
          }
        }
      }
    }
    return true;
  };

  if (warp < kProducerWarps) {
    // ======================= producers =========================================================
    // Stages are numbered it = 0, 1, ... over this CTA's (tile, K block) sequence and use ring slot
    // it mod S.  A slot always belongs to the same producer warp (slot mod 4) and the same MMA issuer
    // (slot mod 2, S is even): a waiter that owns its slot can never be two barrier phases behind it,
    // which a parity wait could not tell from "ready".  Lane 0 waits for the slot and announces the byte
    // count, then the copies go out: one tiled copy for the tile's consecutive rows (gate), or one
    // gather4 per lane for four listed rows each (union rows); the token block is one more tiled copy.
    const int my_tiles = (int)blockIdx.x < n_tiles ? (n_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total = my_tiles * kstages;
    // Stages [it0, it1) of this CTA's sequence; with_w / with_x say which of the two operands are copied.  A
    // stage is armed (slot waited for, byte count announced) together with its weight copy.
    auto produce = [&](int it0, int it1, bool with_w, bool with_x) -> bool {
      int s = it0 % S, ph = (it0 / S) & 1, kb = it0 % kstages, tl = it0 / kstages;
      int rows_of = -1;
      int r[4] = {0, 0, 0, 0};
      for (int it = it0; it < it1; ++it, ++s, ++kb) {
        if (s == S) { s = 0; ph ^= 1; }
        if (kb == kstages) { kb = 0; ++tl; }
        if ((s & (kProducerWarps - 1)) != warp) continue;
        const int tile = blockIdx.x + tl * gridDim.x;
        const int na = min(atoms, kblocks - kb * atoms);
        const uint32_t tx_bytes = kExp ? (uint32_t)(na * (tile_rows * kRawRow + npad * 128)) : (uint32_t)(na * (tile_rows + npad)) * 128;
        if (UP && !walk_all && tl != rows_of) {
          rows_of = tl;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int li = tile * tile_rows + lane * 4 + q;
            // rows beyond the list or the tile: row 0, ignored later
            r[q] = (li >= n_rows || lane * 4 + q >= tile_rows) ? 0
                   : own_list ? rows_sm[tl * kTileRows + lane * 4 + q] : p.idx ? p.idx[li] : li;
            if (!SFFN_IN_BOUNDS(r[q] >= 0 && r[q] < p.R, p.status, 41)) r[q] = 0;
          }
        }
        if (with_w) {
          int ok = 1;
          if (lane == 0) {
            ok = mbar_wait(empty + 8 * s, ph ^ 1, abort_flag, p.status, p.wait_cycles) ? 1 : 0;
            if (ok) mbar_expect_tx(full + 8 * s, tx_bytes);
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) return false;
        }
        const uint32_t abase = ring0 + s * stage_bytes;
        for (int a = 0; a < na; ++a) {
          const int k0 = (kb * atoms + a) * kAtomElems;
          // where the weight block lands, the byte column it starts at, and the bytes of one landed row
          const uint32_t wdst = abase + w_off + a * (kExp ? raw_block_bytes : a_block_bytes);
          const int wc0 = QB == 2 ? k0 / 2 : kExp ? k0 * QB / 8 : k0;
          const int wrow = kExp ? kRawRow : 128;
          if (with_w && !(MODE == kGate && blockIdx.x == 0 && it == p.drop_stage)) {  // test hook: a copy that never comes
            if (UP && !walk_all) {
              if (lane * 4 < tile_rows)
                tma_gather4(wdst + lane * 4 * wrow, &map_w, wc0, r[0], r[1], r[2], r[3], full + 8 * s);
            } else if (UP) {
              if (lane == 0) tma_tile_2d(wdst, map_t.get(), wc0, tile * tile_rows, full + 8 * s);
            } else if (lane == 0) {
              tma_tile_2d(wdst, &map_w, wc0, tile * tile_rows, full + 8 * s);
            }
          }
          if (with_x && lane == 0) tma_tile_2d(abase + b_off + a * b_block_bytes, &map_x, k0, 0, full + 8 * s);
        }
      }
      return true;
    };
    if (MODE == kGate) {
      // the first ring-full of weight tiles goes out while the predecessor in the stream still runs; the token
      // rows of those stages follow once it has finished
      const int ahead = total < S ? total : S;
      const bool ok = produce(0, ahead, true, false);
      pdl_wait();
      if (ok && produce(0, ahead, false, true)) produce(ahead, total, true, true);
    } else {
      produce(0, total, true, true);
    }
  } else if (kExp && warp >= kThreadsRows / 32) {
    // ======================= expanders (quantised rows): codes -> bf16 block of the slot ==========
    // Two pairs of warps; a pair takes the slots of its parity (S is even), in the producers' order, so it meets
    // every phase of its slots and cannot fall two phases behind; while one pair waits the other one converts.
    const int my_tiles = (int)blockIdx.x < n_tiles ? (n_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total = my_tiles * kstages;
    const int pair = (tid - kThreadsRows) / (16 * kExpandWarps);
    const int et = (tid - kThreadsRows) % (16 * kExpandWarps);
    int s = 0, ph = 0, kb = 0;
    for (int it = 0; it < total; ++it, ++s, ++kb) {
      if (s == S) { s = 0; ph ^= 1; }
      if (kb == kstages) kb = 0;
      if ((s & 1) != pair) continue;
      const int t = it % kExpandSlots;
      // the codes have landed, and the MMAs of the stage that used the bf16 slot before are done
      const bool ok = mbar_wait(full + 8 * s, ph, abort_flag, p.status, p.wait_cycles) &&
                      mbar_wait(afree + 8 * t, ((it / kExpandSlots) & 1) ^ 1, abort_flag, p.status, p.wait_cycles);
      if (!__all_sync(0xffffffffu, ok)) break;
      const uint32_t src = ring0 + s * stage_bytes + w_off, dst = stage0 + t * a_bytes;
      const int na = min(atoms, kblocks - kb * atoms);
      for (int a = 0; a < na; ++a)
        if (QB == 2) expand_block_q4_i8(src + a * raw_block_bytes, dst + a * a_block_bytes, tile_rows, et, 16 * kExpandWarps);
        else expand_block<(QB == 8 || QB == 4) ? QB : 8>(src + a * raw_block_bytes, dst + a * a_block_bytes, tile_rows, et, 16 * kExpandWarps);
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(ready + 8 * t);
    }
  } else if (warp >= 8) {
    // ======================= MMA issuers =======================================================
    const int m = warp - 8;
    if (lane == 0 && m < nacc) {
      const uint32_t idesc = kNat ? make_idesc_i8(npad, mrows) : make_idesc(npad, mrows);
      const uint32_t acc = tmem_base + m * npad;
      int tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++tcount) {
        if (!mbar_wait(acc_empty, (tcount & 1) ^ 1, abort_flag, p.status, p.wait_cycles)) break;
        tc_fence_after();
        const int it0 = tcount * kstages;
        int s = it0 % S, ph = (it0 / S) & 1;
        for (int kb = 0; kb < kstages; ++kb, ++s) {
          if (s == S) { s = 0; ph ^= 1; }
          if ((s & (nacc - 1)) != m) continue;   // another issuer's slot
          const int t = (it0 + kb) % kExpandSlots;  // quantised rows: slot of the bf16 ring
          if (kExp ? !mbar_wait(ready + 8 * t, ((it0 + kb) / kExpandSlots) & 1, abort_flag, p.status, p.wait_cycles)
                 : !mbar_wait(full + 8 * s, ph, abort_flag, p.status, p.wait_cycles)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sbase = ring0 + s * stage_bytes;
          const uint32_t wbase = kExp ? stage0 + t * a_bytes : sbase;
          const int na = min(atoms, kblocks - kb * atoms);
          for (int a = 0; a < na; ++a) {
            const uint64_t adesc = make_desc(wbase + a * a_block_bytes);
            const uint64_t bdesc = make_desc(sbase + b_off + a * b_block_bytes);
            if (kNat) {
              umma_i8(acc, adesc, bdesc, idesc, (kb >= nacc || a > 0) ? 1u : 0u);
#pragma unroll
              for (int k = 1; k < 4; ++k) umma_i8(acc, adesc + 2 * k, bdesc + 2 * k, idesc, 1u);
            } else {
              umma(acc, adesc, bdesc, idesc, (kb >= nacc || a > 0) ? 1u : 0u);
#pragma unroll
              for (int k = 1; k < kAtomK / 16; ++k) umma(acc, adesc + 2 * k, bdesc + 2 * k, idesc, 1u);
            }
          }
          umma_commit(empty + 8 * s);   // slot free once these MMAs have read it
          if (kExp) umma_commit(afree + 8 * t);
        }
        if (ok) umma_commit(acc_full);  // this issuer's accumulator is complete
      }
    }
    __syncwarp();
  } else {
    // ======================= epilogue warps (wide batches: every tile but the CTA's last) =========
    if (UP && blockIdx.x == 0) {
      // the down projection walks the list in blocks of 64 rows: entries past its end must read as zero
      __nv_bfloat16* hm = static_cast<__nv_bfloat16*>(p.hmT);
      const int end = (n_rows + 63) & ~63;
      for (int li = n_rows + (warp - 4) * 32 + lane; li < end; li += 128)
        for (int b = 0; b < p.B; ++b) hm[(size_t)b * p.hm_stride + li] = __float2bfloat16(0.f);
    }
    int tcount = 0;
    for (int tile = blockIdx.x; tile + (share_last ? (int)gridDim.x : 0) < n_tiles; tile += gridDim.x, ++tcount) {
      bool fired = false;
      if (!epilogue(tile, tcount, 0, 1, false, fired)) break;
      const int row_in_tile = row_thr;
      const int li = tile * tile_rows + row_in_tile;
      const bool valid = row_in_tile >= 0 && row_in_tile < tile_rows && li < n_rows;
      if (!UP && p.flag && valid) p.flag[li] = fired ? 1 : 0;
      if (!UP && p.words_out) {
        const unsigned m = __ballot_sync(0xffffffffu, fired && valid);
        if (lane == 0) p.words_out[4 * tile + (warp & 3)] = m;
      }
      tc_fence_before();
      mbar_arrive(acc_empty);
    }
  }

  // ---- the CTA's last tile (wide batches): by now the producer and issuer warps have nothing left to do, so
  // all twelve warps share its epilogue.  A warp reads the TMEM lanes of its quarter (warp mod 4); the three warps of
  // a quarter take every third group of eight token columns.
  if (share_last && (int)blockIdx.x < n_tiles && warp < kThreadsRows / 32) {
    const int my_tiles = (n_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
    const int last_tile = blockIdx.x + (my_tiles - 1) * gridDim.x;
    const int part = warp >= 8 ? 2 : warp >= 4 ? 0 : 1;
    bool fired = false;
    const bool done = epilogue(last_tile, my_tiles - 1, part, 3, true, fired);
    if (!UP && (p.flag || p.words_out)) {
      uint8_t* fired_sm = reinterpret_cast<uint8_t*>(scan_wt);  // [3][128], the scan scratch is free here
      const int row_in_tile = row_thr;
      const int me = (warp & 3) * 32 + lane;  // this thread's entry: the same in all three parts
      fired_sm[part * kTileRows + me] = fired ? 1 : 0;
      named_bar_sync(2, kThreadsRows);  // reached by every thread of a CTA that owns a tile, whatever happened
      const int li = last_tile * tile_rows + row_in_tile;
      if (part == 0) {  // warps 4-7, all lanes
        const bool valid = done && row_in_tile >= 0 && row_in_tile < tile_rows && li < n_rows;
        const bool any = (fired_sm[me] | fired_sm[kTileRows + me] | fired_sm[2 * kTileRows + me]) != 0;
        if (p.flag && valid) p.flag[li] = any ? 1 : 0;
        if (p.words_out) {
          const unsigned m = __ballot_sync(0xffffffffu, any && valid);
          if (lane == 0) p.words_out[4 * last_tile + (warp & 3)] = m;
        }
      }
    }
  }

  // ---- teardown: everybody meets, then the allocating warp frees the TMEM columns ------------------
  // (after a wait that ran out, copies and MMAs may still be in flight: they end within microseconds, and shared
  // memory and TMEM are only given back after that)
  if (*abort_flag)
    for (int i = 0; i < 50; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Down projection over the union list (Sec. 5.4): partial[sp][b][d] = sum over the split's listed rows u of
// Hm[b][u] * W_down[idx[u]][d].  One CTA owns 128 output columns d (TMEM lanes) and one split of the list;
// the contraction runs over list rows, so the gathered W_down rows are the MN-major A operand (each
// gathered row delivers 64 contiguous d per swizzle row) and HmT[b][u] is the K-major B operand.
// Same pipeline as above: 4 producer warps (gather4 per lane: 2 column halves x 16 row quads = one 64-row
// stage), 2 MMA issuers with their own accumulators, 4 epilogue warps; two CTAs share an SM.
template <int QB>
__global__ void __launch_bounds__(kThreads + (QB ? 32 * kExpandWarps : 0), 2) umma_down_kernel(const UmmaDownParams p,
                                                                  const __grid_constant__ CUtensorMap map_wg,
                                                                  const __grid_constant__ CUtensorMap map_wt,
                                                                  const __grid_constant__ CUtensorMap map_hm) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int npad = p.npad;
  constexpr int kRawBytes = QB * kTileRows * kAtomK / 8;  // quantised rows: the codes of a stage's 64 rows x 128 columns
  const int raw_off = kAAtomBytes + npad * 128;
  const int stage_bytes = raw_off + kRawBytes;
  const int S = p.stages;
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)S * stage_bytes);
  const uint32_t stage0 = smem_u32(smem);
  const uint32_t full = smem_u32(bars), empty = smem_u32(bars + S);
  const uint32_t acc_full = smem_u32(bars + 2 * S);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t ready = smem_u32(bars + 2 * S + 4);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d_tiles = p.D / kTileRows;
  const int dt = blockIdx.x % d_tiles, sp = blockIdx.x / d_tiles;
  const int d0 = dt * kTileRows;

  pdl_launch_dependents();
  const uint32_t tmem_cols = tmem_cols_for(2 * npad);
  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full + 8 * s, 1);
      mbar_init(empty + 8 * s, 1);
      if (QB) mbar_init(ready + 8 * s, kExpandWarps / 2);
    }
    *abort_flag = 0;
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_wg) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_wt) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_hm) : "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  pdl_wait();

  // both words are fetched at once (one round trip), then combined
  const int listed = p.count ? __ldcg(p.count) : p.R;
  const int walk_word = p.walk_all ? __ldcg(p.walk_all) : 0;
  const bool walk_all = p.idx == nullptr || walk_word != 0;  // every row, not the list
  const int n_rows = walk_all ? p.R : listed;
  // the split's share of the list, in blocks of 64 rows
  const int total_blocks = (n_rows + kAtomK - 1) / kAtomK;
  const int per_split = (total_blocks + p.splits - 1) / p.splits;
  const int kb0 = sp * per_split;
  const int kblocks = min(total_blocks, kb0 + per_split) - kb0;  // <= 0: nothing to add, the partial is zero
  const int nacc = kblocks >= 2 ? 2 : 1;
  if (tid == 0) {
    mbar_init(acc_full, nacc);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp < kProducerWarps) {
    // ======================= producers (slot s belongs to warp s mod 4) =========================
    const uint32_t tx_bytes = (uint32_t)((QB ? kRawBytes : kAAtomBytes) + npad * 128);
    const int half = lane >> 4, quad = lane & 15;
    constexpr int kHalfBytes = QB ? kRawBytes / 2 : kAAtomBytes / 2;  // landed bytes of 64 rows x 64 columns
    constexpr int kColDiv = QB == 4 ? 2 : 1;                          // codes per byte
    int s = 0, ph = 0;
    for (int kb = 0; kb < kblocks; ++kb, ++s) {
      if (s == S) { s = 0; ph ^= 1; }
      if ((s & (kProducerWarps - 1)) != warp) continue;
      const int u0 = (kb0 + kb) * kAtomK;
      int r[4] = {0, 0, 0, 0};
      if (!walk_all) {
        // four list entries of this lane (the list buffer is readable past its length; entries there are
        // replaced by row 0, whose products vanish against the zeroed tail of HmT)
        const int u = u0 + quad * 4;
        const int4 v = *reinterpret_cast<const int4*>(p.idx + u);
        r[0] = u + 0 < n_rows ? v.x : 0;
        r[1] = u + 1 < n_rows ? v.y : 0;
        r[2] = u + 2 < n_rows ? v.z : 0;
        r[3] = u + 3 < n_rows ? v.w : 0;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (!SFFN_IN_BOUNDS(r[q] >= 0 && r[q] < p.R, p.status, 42)) r[q] = 0;
      }
      int ok = 1;
      if (lane == 0) {
        ok = mbar_wait(empty + 8 * s, ph ^ 1, abort_flag, p.status, p.wait_cycles) ? 1 : 0;
        if (ok) mbar_expect_tx(full + 8 * s, tx_bytes);
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const uint32_t abase = stage0 + s * stage_bytes;
      const uint32_t wdst = QB ? abase + raw_off : abase;
      if (!walk_all) {
        tma_gather4(wdst + half * kHalfBytes + quad * (kHalfBytes / 16), &map_wg, (d0 + half * kAtomK) / kColDiv, r[0], r[1],
                    r[2], r[3], full + 8 * s);
      } else if (lane < 2) {
        // every row: 64 consecutive rows per column half; rows past the matrix read as zero
        tma_tile_2d(wdst + lane * kHalfBytes, &map_wt, (d0 + lane * kAtomK) / kColDiv, u0, full + 8 * s);
      }
      if (lane == 0) tma_tile_2d(abase + kAAtomBytes, &map_hm, u0, 0, full + 8 * s);
    }
  } else if (QB && warp >= kThreads / 32) {
    // ======================= expanders (quantised rows): the stage's codes -> its two bf16 blocks =
    // two pairs of warps, each with the slots of its parity (S is even)
    const int pair = (tid - kThreads) / (16 * kExpandWarps);
    const int et = (tid - kThreads) % (16 * kExpandWarps);
    int s = 0, ph = 0;
    for (int kb = 0; kb < kblocks; ++kb, ++s) {
      if (s == S) { s = 0; ph ^= 1; }
      if ((s & 1) != pair) continue;
      const bool ok = mbar_wait(full + 8 * s, ph, abort_flag, p.status, p.wait_cycles);
      if (!__all_sync(0xffffffffu, ok)) break;
      const uint32_t sbase = stage0 + s * stage_bytes;
      expand_block<QB ? QB : 8>(sbase + raw_off, sbase, kAtomK, et, 16 * kExpandWarps);
      expand_block<QB ? QB : 8>(sbase + raw_off + kRawBytes / 2, sbase + kAAtomBytes / 2, kAtomK, et, 16 * kExpandWarps);
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(ready + 8 * s);
    }
  } else if (warp >= 8) {
    // ======================= MMA issuers (slot s belongs to issuer s mod 2) =====================
    const int m = warp - 8;
    if (lane == 0 && m < nacc) {
      const uint32_t idesc = make_idesc(npad) | (1u << 15);  // A is MN-major
      const uint32_t acc = tmem_base + m * npad;
      int s = 0, ph = 0;
      bool ok = true;
      for (int kb = 0; kb < kblocks; ++kb, ++s) {
        if (s == S) { s = 0; ph ^= 1; }
        if (nacc == 2 && (s & 1) != m) continue;
        if (!mbar_wait((QB ? ready : full) + 8 * s, ph, abort_flag, p.status, p.wait_cycles)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sbase = stage0 + s * stage_bytes;
        const uint64_t bdesc = make_desc(sbase + kAAtomBytes);
#pragma unroll
        for (int k = 0; k < kAtomK / 16; ++k)  // 16 list rows = two groups of eight swizzle rows
          umma(acc, make_desc_mn(sbase + k * 2048, 8192, 1024), bdesc + 2 * k, idesc, (kb >= nacc || k > 0) ? 1u : 0u);
        umma_commit(empty + 8 * s);
      }
      if (ok && kblocks > 0) umma_commit(acc_full);
    }
    __syncwarp();
  } else {
    // ======================= epilogue: lane = output column d, TMEM columns = tokens ============
    const int ew = warp - 4;
    const int d = d0 + ew * 32 + lane;
    const int B = p.B;
    float* out = p.partial + (size_t)sp * B * p.D + d;
    const uint32_t taddr = tmem_base + ((uint32_t)(ew * 32) << 16);
    if (kblocks <= 0) {
      for (int b = 0; b < B; ++b) out[(size_t)b * p.D] = 0.f;
    } else {
      int okw = 1;
      if (lane == 0) okw = mbar_wait(acc_full, 0, abort_flag, p.status, p.wait_cycles) ? 1 : 0;
      okw = __shfl_sync(0xffffffffu, okw, 0);
      if (okw) {
        tc_fence_after();
        for (int c0 = 0; c0 < npad; c0 += 8) {
          float v[8];
          tmem_ld8(taddr + c0, nacc, npad, v);
#pragma unroll
          for (int q = 0; q < 8; ++q)
            if (c0 + q < B) out[(size_t)(c0 + q) * p.D] = v[q];
        }
      }
    }
  }

  if (*abort_flag)
    for (int i = 0; i < 50; ++i) __nanosleep(1000);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// LoPA gate, batched: n = RMSNorm(v) (or v itself), written as bf16 pairs for the tensor cores: row 2b of
// x2 holds the high parts of token b's vector, row 2b+1 the low parts (v - bf16(v)), so that the gate's
// U n keeps close to fp32 accuracy.  One CTA per token.
__global__ void __launch_bounds__(256) rmsnorm_split_kernel(const float* v, int r, int v_stride, const float* gain,
                                                            float eps, int use_rms, __nv_bfloat16* x2) {
  __shared__ float red[8];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const float* vb = v + (size_t)b * v_stride;
  float inv = 1.f;
  if (use_rms) {
    float ss = 0.f;
    for (int k = threadIdx.x; k < r; k += blockDim.x) ss = fmaf(vb[k], vb[k], ss);
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    inv = rsqrtf(tot / (float)r + eps);
  }
  for (int k = threadIdx.x; k < r; k += blockDim.x) {
    const float n = use_rms ? (gain ? gain[k] : 1.f) * vb[k] * inv : vb[k];
    const __nv_bfloat16 hi = __float2bfloat16(n);
    x2[(size_t)(2 * b) * r + k] = hi;
    x2[(size_t)(2 * b + 1) * r + k] = __float2bfloat16(n - __bfloat162float(hi));
  }
}

// Tokens as int8 limbs for the kind::i8 MMAs: t[k] = scale * (q0 + q1 / 128 + q2 / 128^2 + q3 / 128^3) up to
// scale * 2^-22, with scale = max |t| / 127, |q0| <= 127 and the other limbs <= 64 in magnitude.  Row 4 b + l of
// `limbs` holds limb l of token b.  One CTA per token; `val(k)` yields the token's entries.
template <typename F>
__device__ __forceinline__ void write_limbs(F val, int K, int8_t* limbs, float* scale_out, float* red) {
  float m = 0.f;
  for (int k = threadIdx.x; k < K; k += blockDim.x) m = fmaxf(m, fabsf(val(k)));
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
  __syncthreads();  // `red` may still be read by the caller
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  float mx = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) mx = fmaxf(mx, red[w]);
  const float scale = mx > 0.f ? mx / 127.f : 1.f;
  if (threadIdx.x == 0) *scale_out = scale;
  const float inv = 1.f / scale;
  for (int k = threadIdx.x; k < K; k += blockDim.x) {
    float t = val(k) * inv;
    t = fminf(fmaxf(t, -127.f), 127.f);
#pragma unroll
    for (int l = 0; l < 4; ++l) {
      const float q = rintf(t);
      limbs[(size_t)l * K + k] = (int8_t)(int)q;
      t = (t - q) * 128.f;
    }
  }
}

__global__ void __launch_bounds__(256) token_limbs_kernel(const __nv_bfloat16* x, int K, int x_stride, int8_t* limbs,
                                                          float* scale) {
  __shared__ float red[8];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const __nv_bfloat16* xb = x + (size_t)b * x_stride;
  write_limbs([&](int k) { return __bfloat162float(xb[k]); }, K, limbs + (size_t)4 * b * K, scale + b, red);
}

// LoPA gate with int8 rows: n = RMSNorm(v) (or v itself) as limbs.  One CTA per token.
__global__ void __launch_bounds__(256) rmsnorm_limbs_kernel(const float* v, int r, int v_stride, const float* gain,
                                                            float eps, int use_rms, int8_t* limbs, float* scale) {
  __shared__ float red[8];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const float* vb = v + (size_t)b * v_stride;
  float inv = 1.f;
  if (use_rms) {
    float ss = 0.f;
    for (int k = threadIdx.x; k < r; k += blockDim.x) ss = fmaf(vb[k], vb[k], ss);
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    inv = rsqrtf(tot / (float)r + eps);
  }
  write_limbs([&](int k) { return use_rms ? (gain ? gain[k] : 1.f) * vb[k] * inv : vb[k]; }, r, limbs + (size_t)4 * b * r,
              scale + b, red);
}

}  // namespace


// Tiling of the gate GEMM over R rows (the up kernel needs it to read the gate's bit masks).
void umma_gate_tiling(int R, int sm_count, int* tile_rows, int* n_tiles) {
  const int grid = R < 8 * sm_count ? (R + 7) / 8 : sm_count;
  *tile_rows = tile_rows_for(R, grid);
  *n_tiles = (R + *tile_rows - 1) / *tile_rows;
}

bool umma_own_list_supported(int R, int sm_count) {
  int tr, nt;
  umma_gate_tiling(R, sm_count, &tr, &nt);
  return 4 * nt <= kScanChunks * kThreadsRows && R <= (long long)kMaxOwnTiles * kTileRows * sm_count;
}

bool umma_may_walk(int B) { return B >= kWalkMinTokens; }

bool umma_rows_supported(int K, int cols) { return K % kAtomK == 0 && K >= kAtomK && cols >= 1 && cols <= 128; }
// int8 rows multiplied as int8 (tokens as four int8 limbs each): K blocks of 128 codes, up to 64 tokens.
bool umma_rows_native_i8_supported(int K, int tokens) { return K % 128 == 0 && K >= 128 && tokens >= 1 && tokens <= 64; }

namespace {

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

// bf16 matrix [rows, K] with row pitch `pitch_elems`, read in boxes of 64 elements x box_rows rows, 128-byte swizzle.
bool make_map(CUtensorMap* m, const void* base, int K, int rows, size_t pitch_elems, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kAtomK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Rows of weight codes [rows, K] (qbits 8 or 4 per code, `pitch_bytes` apart), read in boxes of 64 codes x box_rows
// rows that land densely, without swizzle.
bool make_map_codes(CUtensorMap* m, const void* base, int K, int rows, size_t pitch_bytes, int box_rows, int qbits,
                    int box_codes = kAtomK) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)K * qbits / 8, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)(box_codes * qbits / 8), (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// int8 matrix [rows, K] (row pitch in bytes), read in boxes of 128 codes x box_rows rows, 128-byte swizzle: the operand
// layout of the kind::i8 MMAs.
bool make_map_i8(CUtensorMap* m, const void* base, int K, int rows, size_t pitch_bytes, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch_bytes};
  const cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_weight_map(CUtensorMap* m, const void* base, int K, int rows, int box_rows, int qbits) {
  return qbits == 1 ? make_map_i8(m, base, K, rows, (size_t)K, box_rows)
         : qbits == 2 ? make_map_codes(m, base, K, rows, (size_t)K / 2, box_rows, 4, 128)  // int4 rows, K blocks of 128 codes
         : qbits    ? make_map_codes(m, base, K, rows, (size_t)K * qbits / 8, box_rows, qbits)
                    : make_map(m, base, K, rows, (size_t)K, box_rows);
}

template <int MODE, typename Map>
cudaError_t launch_rows_mode(const UmmaRowsParams& p, int grid, size_t smem, cudaStream_t s, const CUtensorMap& map_w,
                             const CUtensorMap& map_x, const Map& map_t) {
  static unsigned long long configured[4] = {0, 0, 0, 0};
  cudaError_t e;
  if (p.qbits == 1) {
    auto k = umma_rows_kernel<MODE, 1>;
    if ((e = allow_dynamic_smem(k, 227 * 1024, configured[3])) != cudaSuccess) return e;
    return launch_pdl(k, dim3(grid), dim3(kThreadsRows), smem, s, p, map_w, map_x, map_t);
  }
  if (p.qbits == 2) {
    static unsigned long long configured2 = 0;
    auto k = umma_rows_kernel<MODE, 2>;
    if ((e = allow_dynamic_smem(k, 227 * 1024, configured2)) != cudaSuccess) return e;
    return launch_pdl(k, dim3(grid), dim3(kThreadsRows + 32 * kExpandWarps), smem, s, p, map_w, map_x, map_t);
  }
  if (p.qbits == 8) {
    auto k = umma_rows_kernel<MODE, 8>;
    if ((e = allow_dynamic_smem(k, 227 * 1024, configured[0])) != cudaSuccess) return e;
    return launch_pdl(k, dim3(grid), dim3(kThreadsRows + 32 * kExpandWarps), smem, s, p, map_w, map_x, map_t);
  }
  if (p.qbits == 4) {
    auto k = umma_rows_kernel<MODE, 4>;
    if ((e = allow_dynamic_smem(k, 227 * 1024, configured[1])) != cudaSuccess) return e;
    return launch_pdl(k, dim3(grid), dim3(kThreadsRows + 32 * kExpandWarps), smem, s, p, map_w, map_x, map_t);
  }
  auto k = umma_rows_kernel<MODE, 0>;
  if ((e = allow_dynamic_smem(k, 227 * 1024, configured[2])) != cudaSuccess) return e;
  return launch_pdl(k, dim3(grid), dim3(kThreadsRows), smem, s, p, map_w, map_x, map_t);
}

}  // namespace

cudaError_t launch_umma_rows(bool up, UmmaRowsParams p, int cols, int sm_count, cudaStream_t s) {
  p.npad = (cols + 15) / 16 * 16;
  p.wait_cycles = fused_test_knobs().wait_cycles;
  p.drop_stage = fused_test_knobs().drop_stage;
  const int grid = p.R < 8 * sm_count ? (p.R + 7) / 8 : sm_count;
  // all the dynamic shared memory a CTA can have; the kernel cuts its ring out of it once it knows its tiles
  const size_t smem = 226 * 1024;
  p.ring_bytes = (int)smem - 1024 - kHeaderBytes;
  alignas(64) CUtensorMap map_w, map_x;
  if (p.qbits != 0 && p.qbits != 8 && p.qbits != 4 && p.qbits != 1 && p.qbits != 2) return cudaErrorInvalidValue;
  const bool i8 = p.qbits == 1 || p.qbits == 2;  // kind::i8 MMAs: X holds the tokens' int8 limbs
  if (i8 && (p.K % 128 || p.npad > 256 || !p.tok_scale)) return cudaErrorInvalidValue;
  // weights: all R rows; boxes of one tile's rows for the gate, single-row boxes for the gather
  if (!make_weight_map(&map_w, p.W, p.K, p.R, up ? 1 : tile_rows_for(p.R, grid), p.qbits)) return cudaErrorNotSupported;
  // tokens: only the rows that exist; the box covers npad rows and the rest reads as zero
  if (i8 ? !make_map_i8(&map_x, p.X, p.K, p.ncols_valid, (size_t)p.x_stride, p.npad)
                   : !make_map(&map_x, p.X, p.K, p.ncols_valid, (size_t)p.x_stride, p.npad))
    return cudaErrorNotSupported;
  if (!up) return launch_rows_mode<kGate>(p, grid, smem, s, map_w, map_x, WalkMap<false>{});
  if (p.walk_all && umma_may_walk(p.B)) {
    // wide batches: the union may cover most rows; the kernel then walks every row with tiled boxes of the tile
    // height of R rows (decided on the device from the union's size, so it depends on this call's inputs only)
    WalkMap<true> map_t;
    if (!make_weight_map(&map_t.m, p.W, p.K, p.R, tile_rows_for(p.R, grid), p.qbits)) return cudaErrorNotSupported;
    return launch_rows_mode<kUpMayWalk>(p, grid, smem, s, map_w, map_x, map_t);
  }
  return launch_rows_mode<kUp>(p, grid, smem, s, map_w, map_x, WalkMap<false>{});
}

int umma_down_splits(int D, int sm_count, int max_splits) {
  const int d_tiles = D / kTileRows;
  int splits = 2 * sm_count / (d_tiles > 0 ? d_tiles : 1);  // two CTAs per SM
  return splits < 1 ? 1 : splits > max_splits ? max_splits : splits;
}

bool umma_down_supported(int D, int cols) { return D % kTileRows == 0 && cols >= 1 && cols <= 64; }

namespace {
template <int QB>
cudaError_t launch_down_q(const UmmaDownParams& p, int grid, size_t smem, cudaStream_t s, const CUtensorMap& map_wg,
                          const CUtensorMap& map_wt, const CUtensorMap& map_hm) {
  static unsigned long long configured = 0;
  const cudaError_t e = allow_dynamic_smem(umma_down_kernel<QB>, 113 * 1024, configured);
  if (e != cudaSuccess) return e;
  return launch_pdl(umma_down_kernel<QB>, dim3(grid), dim3(kThreads + (QB ? 32 * kExpandWarps : 0)), smem, s, p, map_wg,
                    map_wt, map_hm);
}
}  // namespace

cudaError_t launch_umma_down(UmmaDownParams p, cudaStream_t s) {
  if (p.qbits != 0 && p.qbits != 8 && p.qbits != 4) return cudaErrorInvalidValue;
  p.npad = (p.B + 15) / 16 * 16;
  p.wait_cycles = fused_test_knobs().wait_cycles;
  const int stage_bytes = kAAtomBytes + p.npad * 128 + p.qbits * kTileRows * kAtomK / 8;
  int stages = (111 * 1024 - 1024 - 1024) / stage_bytes;
  if (stages > 12) stages = 12;
  stages &= ~1;
  if (stages < 2) return cudaErrorInvalidValue;
  p.stages = stages;
  const size_t smem = 1024 + (size_t)stages * stage_bytes + (3 * stages + 4) * 8 + 64;
  const int grid = (p.D / kTileRows) * p.splits;
  alignas(64) CUtensorMap map_wg, map_wt, map_hm;
  // W_down [H, D]: inner dimension d; single-row boxes for the gather, 64-row boxes for the dense walk
  if (!make_weight_map(&map_wg, p.W_down, p.D, p.R, 1, p.qbits)) return cudaErrorNotSupported;
  if (!make_weight_map(&map_wt, p.W_down, p.D, p.R, kAtomK, p.qbits)) return cudaErrorNotSupported;
  // HmT [B][hm_stride]: inner dimension u; token rows past B read as zero
  if (!make_map(&map_hm, p.hmT, p.hm_stride, p.B, (size_t)p.hm_stride, p.npad)) return cudaErrorNotSupported;
  const int g = grid;
  return p.qbits == 8   ? launch_down_q<8>(p, g, smem, s, map_wg, map_wt, map_hm)
         : p.qbits == 4 ? launch_down_q<4>(p, g, smem, s, map_wg, map_wt, map_hm)
                        : launch_down_q<0>(p, g, smem, s, map_wg, map_wt, map_hm);
}

cudaError_t launch_token_limbs(const void* x, int B, int K, int x_stride, void* limbs, float* scale, cudaStream_t s) {
  return launch_pdl(token_limbs_kernel, dim3(B), dim3(256), 0, s, static_cast<const __nv_bfloat16*>(x), K, x_stride,
                    static_cast<int8_t*>(limbs), scale);
}

cudaError_t launch_rmsnorm_limbs(const float* v, int B, int r, int v_stride, const float* gain, float eps, bool use_rms,
                                 void* limbs, float* scale, cudaStream_t s) {
  return launch_pdl(rmsnorm_limbs_kernel, dim3(B), dim3(256), 0, s, v, r, v_stride, gain, eps, use_rms ? 1 : 0,
                    static_cast<int8_t*>(limbs), scale);
}

cudaError_t launch_rmsnorm_split(const float* v, int B, int r, int v_stride, const float* gain, float eps,
                                 bool use_rms, void* x2, cudaStream_t s) {
  return launch_pdl(rmsnorm_split_kernel, dim3(B), dim3(256), 0, s, v, r, v_stride, gain, eps, use_rms ? 1 : 0,
                    static_cast<__nv_bfloat16*>(x2));
}

}  // namespace sffn
