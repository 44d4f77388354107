// Host side of the C ABI declared in include/sparse_ffn.h: argument checks, workspace carving and
// kernel dispatch.  No device memory is allocated or freed here.
#include "sparse_ffn.h"

#include <cstdio>

#include <cuda_runtime.h>

#include <new>

#include "batched_kernels.cuh"
#include "cast_kernels.cuh"
#include "common.cuh"
#include "fused_kernel.cuh"
#include "general_kernels.cuh"
#include "umma_kernels.cuh"

namespace {

constexpr int kMaxUpDownGrid = 304;  // upper bound of the up/down grid (2 CTAs per SM on 148 SMs)
constexpr int kMaxChunk = 4;         // tokens per pass of the general kernels
constexpr int kMaxSplits = 16;       // union-row splits of the batched down projection
constexpr int kMaxMmaTokens = 64;    // tokens per pass of the batched tensor-core kernels

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
  size_t status, act, flag, idx, v, n, partial, xstage, ystage, fused, hmT, x2, union_flag, xlimb, nlimb, tscale, total;
  int hm_stride;
};

Layout make_layout(int D, int H, int r_max, int B_max, int dtype) {
  const size_t esz = dtype == SFFN_BF16 ? 2 : 4;
  Layout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  L.status = take(256);  // [0] device status, [1] length of idx, [2] batched path: every row was walked
  L.act = take((size_t)B_max * H * 4);
  L.flag = take((size_t)2 * H + 256);  // bytes [H], or the tcgen05 gate's bit masks (16 bytes per tile of >= 8 rows)
  L.idx = take(((size_t)H + 64) * 4);  // readable one 64-row block past the list
  L.v = take((size_t)B_max * (r_max > 0 ? r_max : 1) * 4);
  L.n = take((size_t)B_max * (r_max > 0 ? r_max : 1) * 4);
  const size_t part_general = (size_t)kMaxUpDownGrid * kMaxChunk * D * 4;
  const size_t part_batched = (size_t)kMaxSplits * (B_max < kMaxMmaTokens ? B_max : kMaxMmaTokens) * D * 4;
  L.partial = take(part_general > part_batched ? part_general : part_batched);
  L.xstage = take((size_t)B_max * D * esz);
  L.ystage = take((size_t)B_max * D * 4);
  L.fused = take(sffn::fused_workspace_bytes(D, H, r_max));
  L.hm_stride = (H + 63) / 64 * 64 + 64;
  L.hmT = take((size_t)(B_max < kMaxMmaTokens ? B_max : kMaxMmaTokens) * L.hm_stride * 2);
  L.x2 = take((size_t)2 * (B_max < kMaxMmaTokens ? B_max : kMaxMmaTokens) * (r_max > 0 ? r_max : 1) * 2);
  L.union_flag = take((size_t)H + 256);  // fired flags accumulated over the chunks of a batch of more than 64 tokens
  // int8 rows on the tensor cores: the tokens (and the LoPA vector) as four int8 limbs each, and their scales
  const size_t bt = B_max < kMaxMmaTokens ? B_max : kMaxMmaTokens;
  L.xlimb = take(B_max > 1 && dtype == SFFN_BF16 ? 4 * bt * D : 0);
  L.nlimb = take(B_max > 1 && dtype == SFFN_BF16 ? 4 * bt * (size_t)(r_max > 0 ? r_max : 1) : 0);
  L.tscale = take(2 * kMaxMmaTokens * 4);
  L.total = off;
  return L;
}

bool shape_ok(int D, int H, int r_max, int B_max, int dtype) {
  return D > 0 && H > 0 && r_max >= 0 && B_max > 0 && (dtype == SFFN_F32 || dtype == SFFN_BF16);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

struct sffn_handle {
  int D, H, r_max, B_max, dtype;
  char* ws;
  Layout L;
  int sm_count;
  int path;
  int act_up;  // activation on the up projection (double activation), SFFN_ACT_NONE = Eq. 1
  int gated_skip;  // single-token fused kernel: W_down rows only where h != 0 (see sffn_set_gated_skip)
  int gate_engine = SFFN_GATE_ENGINE_AUTO;
  long long launches;
  int list_state;  // 0: no sparse call yet, 1: idx/count hold the last call's list, 2: flags hold it
  template <typename T>
  T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

extern "C" {


const char* sffn_status_string(int s) {
  switch (s) {
    case SFFN_OK: return "ok";
    case SFFN_ERR_INVALID_ARG: return "invalid argument";
    case SFFN_ERR_UNSUPPORTED: return "unsupported shape, alignment or path";
    case SFFN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SFFN_ERR_CUDA: return "CUDA runtime error";
    case SFFN_ERR_TIMEOUT: return "device-side bounded wait ran out";
    case SFFN_ERR_BOUNDS: return "debug build: index outside its array";
    default: return "unknown status";
  }
}

int sffn_workspace_bytes(int D, int H, int r_max, int B_max, int dtype, size_t* bytes) {
  if (!bytes || !shape_ok(D, H, r_max, B_max, dtype)) return SFFN_ERR_INVALID_ARG;
  const size_t esz = dtype == SFFN_BF16 ? 2 : 4;
  if ((D * esz) % 16 || (r_max * esz) % 16) return SFFN_ERR_UNSUPPORTED;
  if (sffn::updown_max_tokens(dtype == SFFN_BF16, D) == 0) return SFFN_ERR_UNSUPPORTED;
  *bytes = make_layout(D, H, r_max, B_max, dtype).total;
  return SFFN_OK;
}

int sffn_create(sffn_handle** handle, int D, int H, int r_max, int B_max, int dtype, void* workspace,
                size_t workspace_bytes) {
  if (!handle) return SFFN_ERR_INVALID_ARG;
  *handle = nullptr;
  size_t need = 0;
  const int rc = sffn_workspace_bytes(D, H, r_max, B_max, dtype, &need);
  if (rc != SFFN_OK) return rc;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
    return SFFN_ERR_WORKSPACE;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return SFFN_ERR_CUDA;
  if (cudaMemset(workspace, 0, need) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return SFFN_ERR_CUDA;
  sffn_handle* h = new (std::nothrow) sffn_handle();
  if (!h) return SFFN_ERR_INVALID_ARG;
  h->D = D;
  h->H = H;
  h->r_max = r_max;
  h->B_max = B_max;
  h->dtype = dtype;
  h->ws = static_cast<char*>(workspace);
  h->L = make_layout(D, H, r_max, B_max, dtype);
  h->sm_count = sms;
  h->path = SFFN_PATH_AUTO;
  h->act_up = SFFN_ACT_NONE;
  h->gated_skip = 0;
  h->launches = 0;
  h->list_state = 0;
  *handle = h;
  return SFFN_OK;
}

int sffn_destroy(sffn_handle* h) {
  if (!h) return SFFN_ERR_INVALID_ARG;
  delete h;
  return SFFN_OK;
}

int sffn_set_gate_engine(sffn_handle* h, int engine) {
  if (!h || engine < SFFN_GATE_ENGINE_AUTO || engine > SFFN_GATE_ENGINE_TENSOR_CORE) return SFFN_ERR_INVALID_ARG;
  h->gate_engine = engine;
  return SFFN_OK;
}

int sffn_set_gated_skip(sffn_handle* h, int on) {
  if (!h) return SFFN_ERR_INVALID_ARG;
  h->gated_skip = on != 0;
  return SFFN_OK;
}

int sffn_set_up_activation(sffn_handle* h, int act_up) {
  if (!h || act_up < SFFN_ACT_RELU || act_up > SFFN_ACT_SILU) return SFFN_ERR_INVALID_ARG;
  h->act_up = act_up;
  return SFFN_OK;
}

int sffn_set_path(sffn_handle* h, int path) {
  if (!h || path < SFFN_PATH_AUTO || path > SFFN_PATH_MMA_SYNC) return SFFN_ERR_INVALID_ARG;
  h->path = path;
  return SFFN_OK;
}

// ---- test hooks (declared in the last section of sparse_ffn.h) ------------------------------------------------
void sffn_test_fused_plan(int wkind, int D, int H, int K, int lopa, int sm_count, int* out9) {
  sffn::debug_fused_plan(wkind, D, H, K, lopa != 0, sm_count, out9);  // wkind: 0 fp32, 1 bf16, 2 int8 rows
}
void sffn_test_umma_tiling(int R, int sm_count, int* tile_rows, int* n_tiles, int* own_list) {
  sffn::umma_gate_tiling(R, sm_count, tile_rows, n_tiles);
  *own_list = sffn::umma_own_list_supported(R, sm_count) ? 1 : 0;
}
int sffn_test_set_knob(int knob, long long value) {
  sffn::FusedTestKnobs& k = sffn::fused_test_knobs();
  switch (knob) {
    case SFFN_KNOB_PDL: k.pdl = value != 0; return SFFN_OK;
    case SFFN_KNOB_TENSOR_GATE: k.tensor_gate = value < 0 ? -1 : (value != 0); return SFFN_OK;
    case SFFN_KNOB_WAIT_CYCLES: k.wait_cycles = value > 0 ? value : (1LL << 31); return SFFN_OK;
    case SFFN_KNOB_SKIP_ARRIVAL_CTA: k.skip_arrival_cta = (int)value; return SFFN_OK;
    case SFFN_KNOB_RING_GATE_SLOTS: k.ring_S = (int)value; return SFFN_OK;
    case SFFN_KNOB_RING_ACT_SLOTS: k.ring_NA = (int)value; return SFFN_OK;
    case SFFN_KNOB_RING_PARKED_STAGES: k.ring_E = (int)value; return SFFN_OK;
    case SFFN_KNOB_L2_HINTS: k.l2_hints = (int)value; return SFFN_OK;
    case SFFN_KNOB_DROP_STAGE: k.drop_stage = (int)value; return SFFN_OK;
    case SFFN_KNOB_POISON_LIST:
#ifdef SFFN_DEBUG
      k.poison_list = value != 0;
      return SFFN_OK;
#else
      return value ? SFFN_ERR_UNSUPPORTED : SFFN_OK;
#endif
    case SFFN_KNOB_TRACE_BUFFER: k.trace = reinterpret_cast<long long*>(static_cast<uintptr_t>(value)); return SFFN_OK;
    default: return SFFN_ERR_INVALID_ARG;
  }
}

int sffn_launch_count(sffn_handle* h, long long* launches) {
  if (!h || !launches) return SFFN_ERR_INVALID_ARG;
  *launches = h->launches;
  return SFFN_OK;
}

}  // extern "C"

namespace {

int check_call(const sffn_handle* h, const void* x, int B, const sffn_gate* g, const void* W_up,
               const void* W_down, int act, const void* y, const sffn_q8_scales* q8, int qbits) {
  if (!h || !x || !g || !W_up || !W_down || !y) return SFFN_ERR_INVALID_ARG;
  if (B < 1 || B > h->B_max) return SFFN_ERR_INVALID_ARG;
  if (act < SFFN_ACT_RELU || act > SFFN_ACT_RSPLUS) return SFFN_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(y)) return SFFN_ERR_UNSUPPORTED;
  // elements of a weight row per 16 bytes
  const int epv = q8 ? (qbits == 4 ? 32 : 16) : h->dtype == SFFN_BF16 ? 8 : 4;
  if (q8) {
    if (h->dtype != SFFN_BF16) return SFFN_ERR_UNSUPPORTED;  // int8 / int4 weights meet bf16 tokens
    if (!q8->s_gate || !q8->s_up || !q8->s_down) return SFFN_ERR_INVALID_ARG;
    if (g->kind == SFFN_GATE_LOPA && !q8->s_V) return SFFN_ERR_INVALID_ARG;
    if (h->D % epv) return SFFN_ERR_UNSUPPORTED;
    if (sffn::updown_max_tokens(qbits == 4 ? sffn::kWQ4 : sffn::kWQ8, h->D) == 0) return SFFN_ERR_UNSUPPORTED;
    if (h->path == SFFN_PATH_MMA_SYNC) return SFFN_ERR_UNSUPPORTED;
  }
  if (g->kind == SFFN_GATE_STANDARD) {
    if (!g->W_g) return SFFN_ERR_INVALID_ARG;
    if (!aligned16(g->W_g)) return SFFN_ERR_UNSUPPORTED;
  } else if (g->kind == SFFN_GATE_LOPA) {
    if (!g->V || !g->U || g->r < 1 || g->r > h->r_max) return SFFN_ERR_INVALID_ARG;
    if (!aligned16(g->V) || !aligned16(g->U) || g->r % epv) return SFFN_ERR_UNSUPPORTED;
  } else {
    return SFFN_ERR_INVALID_ARG;
  }
  return SFFN_OK;
}

// The CUDA error behind the calling thread's last SFFN_ERR_CUDA (sffn_last_cuda_error).
thread_local cudaError_t g_last_cuda_error = cudaSuccess;
thread_local int g_last_cuda_line = 0;

#define SFFN_CUDA(expr)               \
  do {                                \
    const cudaError_t e_ = (expr);    \
    if (e_ != cudaSuccess) {          \
      g_last_cuda_error = e_;         \
      g_last_cuda_line = __LINE__;    \
      return SFFN_ERR_CUDA;           \
    }                                 \
  } while (0)

// Batched tensor-core path (bf16, B >= 2): gate GEMM -> compaction of the union -> up GEMM over the
// union rows -> down GEMM (split over D-slices and union chunks) -> fixed-order sum of the splits.
// Tokens are taken kMaxMmaTokens at a time; the union (and the list) is that of the whole batch.
int run_batched(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                const void* W_up, const void* W_down, int act, float* y, bool dense, bool umma,
                const sffn_q8_scales* q8, int qbits, cudaStream_t s) {
  using namespace sffn;
  const int D = h->D, H = h->H;
  if (q8 && !umma) return SFFN_ERR_UNSUPPORTED;  // rows of weight codes: tcgen05 kernels only
  const int wq = q8 ? qbits : 0;
  // int8 rows whose K blocks are whole (128 codes): multiplied as int8 against the tokens' int8 limbs, nothing to expand
  // (the down projection keeps the expansion: its B operand, Hm, has no scale known before the whole of it exists)
  // (int4 rows: the nibbles expanded to int8 on the way, for the same MMAs)
  const bool native = q8 && B <= kMaxMmaTokens && umma_rows_native_i8_supported(D, B) &&
                      umma_rows_native_i8_supported(g->kind == SFFN_GATE_LOPA ? g->r : D, B);
  const int wq_rows = native ? (qbits == 8 ? 1 : 2) : wq;
  void* xlimb = h->ws + h->L.xlimb;
  void* nlimb = h->ws + h->L.nlimb;
  float* xscale = h->at<float>(h->L.tscale);
  float* nscale = xscale + kMaxMmaTokens;
  if (native) {
    SFFN_CUDA(launch_token_limbs(x, B, D, D, xlimb, xscale, s));
    ++h->launches;
  }
  float* actbuf = h->at<float>(h->L.act);
  uint8_t* flag = h->at<uint8_t>(h->L.flag);
  int32_t* idx = h->at<int32_t>(h->L.idx);
  int32_t* count = h->at<int32_t>(h->L.status) + 1;
  const int rs = h->r_max > 0 ? h->r_max : 1;
  float* vbuf = h->at<float>(h->L.v);
  float* nbuf = h->at<float>(h->L.n);
  const char* xb = static_cast<const char*>(x);
  const bool lopa = g->kind == SFFN_GATE_LOPA;
  const int grid_rows = 2 * h->sm_count;

  if (lopa && umma) {  // v = V x on the tensor cores: the rows kernel with the identity as its epilogue
    for (int b0 = 0; b0 < B; b0 += kMaxMmaTokens) {
      const int nb = B - b0 < kMaxMmaTokens ? B - b0 : kMaxMmaTokens;
      UmmaRowsParams p{};
      p.W = g->V; p.R = g->r; p.K = D;
      p.qbits = wq_rows; p.w_scale = q8 ? q8->s_V : nullptr;
      p.X = xb + (size_t)b0 * D * 2; p.x_stride = D; p.ncols_valid = nb; p.B = nb;
      if (native) { p.X = xlimb; p.ncols_valid = 4 * nb; p.tok_scale = xscale; }
      p.act = kUmmaActIdentity; p.a_out = vbuf + (size_t)b0 * rs; p.a_stride = rs;
      p.status = h->at<int32_t>(h->L.status);
      SFFN_CUDA(launch_umma_rows(false, p, native ? 4 * nb : nb, h->sm_count, s));
      ++h->launches;
    }
  } else if (lopa) {  // v = V x on the CUDA-core row kernel (r rows only), then RMSNorm
    for (int b0 = 0; b0 < B;) {
      const int nb = B - b0 >= 4 ? 4 : B - b0 >= 2 ? 2 : 1;
      RowDotParams p{};
      p.W = g->V; p.R = g->r; p.K = D;
      p.vec = xb + (size_t)b0 * D * 2; p.vec_stride = D;
      p.out = vbuf + (size_t)b0 * rs; p.out_stride = rs;
      SFFN_CUDA(launch_rowdot(true, false, nb, false, p, h->sm_count, s));
      ++h->launches;
      b0 += nb;
    }
    if (g->use_rmsnorm) {
      SFFN_CUDA(launch_rmsnorm(vbuf, nbuf, g->rms_gain, g->r, rs, g->rms_eps, B, s));
      ++h->launches;
    }
  }
  // The tcgen05 gate kernel can leave its "fired" flags as bit masks, which the up kernel compacts itself
  // (and publishes list and length): no byte flags, no compaction launch.
  const bool own_list = umma && !dense && umma_own_list_supported(H, h->sm_count);
  uint32_t* words = reinterpret_cast<uint32_t*>(flag);  // the flag buffer holds either form
  int gate_tile_rows = 0, gate_tiles = 0;
  umma_gate_tiling(H, h->sm_count, &gate_tile_rows, &gate_tiles);
  for (int b0 = 0; b0 < B; b0 += kMaxMmaTokens) {
    const int nb = B - b0 < kMaxMmaTokens ? B - b0 : kMaxMmaTokens;
    void* x2 = h->ws + h->L.x2;
    const float* nsrc = (g->use_rmsnorm ? nbuf : vbuf) + (size_t)b0 * rs;
    const void* xtok = xb + (size_t)b0 * D * 2;
    if (b0 > 0 && !dense) return SFFN_ERR_UNSUPPORTED;  // flags of later chunks would need OR-ing
    if (umma) {
      UmmaRowsParams p{};
      p.R = H; p.B = nb; p.b_g = b_g; p.act = act; p.status = h->at<int32_t>(h->L.status);
      p.qbits = wq_rows; p.w_scale = q8 ? q8->s_gate : nullptr;
      p.xtok = xtok; p.xtok_stride = D;
      p.a_out = actbuf + (size_t)b0 * H; p.a_stride = H;
      p.flag = (dense || own_list) ? nullptr : flag;
      p.words_out = own_list ? words : nullptr;
      int cols = nb;
      if (lopa && native) {
        // RMSNorm (or none) and the split into int8 limbs in one launch
        SFFN_CUDA(launch_rmsnorm_limbs(vbuf + (size_t)b0 * rs, nb, g->r, rs, g->rms_gain, g->rms_eps,
                                       g->use_rmsnorm != 0, nlimb, nscale, s));
        ++h->launches;
        p.W = g->U; p.K = g->r; p.X = nlimb; p.x_stride = g->r; p.tok_scale = nscale;
        p.g_idx = g->g_idx; p.g_sign = g->g_sign;
        cols = 4 * nb;
      } else if (lopa) {
        // RMSNorm (or none) and the split into bf16 pairs in one launch
        SFFN_CUDA(launch_rmsnorm_split(vbuf + (size_t)b0 * rs, nb, g->r, rs, g->rms_gain, g->rms_eps,
                                       g->use_rmsnorm != 0, x2, s));
        ++h->launches;
        p.W = g->U; p.K = g->r; p.X = x2; p.x_stride = g->r; p.split_cols = 1;
        p.g_idx = g->g_idx; p.g_sign = g->g_sign;
        cols = 2 * nb;
      } else if (native) {
        p.W = g->W_g; p.K = D; p.X = xlimb; p.x_stride = D; p.tok_scale = xscale;
        cols = 4 * nb;
      } else {
        p.W = g->W_g; p.K = D; p.X = xtok; p.x_stride = D;
      }
      p.ncols_valid = cols;
      SFFN_CUDA(launch_umma_rows(false, p, cols, h->sm_count, s));
    } else {
      RowsMmaParams p{};
      p.status = h->at<int32_t>(h->L.status);
      p.R = H; p.B = nb; p.b_g = b_g; p.act = act;
      p.xtok = xtok; p.xtok_stride = D;
      p.a_out = actbuf + (size_t)b0 * H; p.a_stride = H;
      p.flag = dense ? nullptr : flag;
      int cols = nb;
      if (lopa) {
        SFFN_CUDA(launch_split_bf16(nsrc, nb, g->r, rs, x2, s));
        ++h->launches;
        p.W = g->U; p.K = g->r; p.X = x2; p.x_stride = g->r; p.split_cols = 1;
        p.g_idx = g->g_idx; p.g_sign = g->g_sign;
        cols = 2 * nb;
      } else {
        p.W = g->W_g; p.K = D; p.X = xtok; p.x_stride = D;
      }
      p.ncols_valid = cols;
      SFFN_CUDA(launch_rows_mma(false, p, cols, grid_rows, s));
    }
    ++h->launches;
  }
  if (!dense) {
    if (!own_list) {
      SFFN_CUDA(launch_compact(flag, H, idx, count, s));
      ++h->launches;
    }
    h->list_state = 1;
  }
  int splits = h->sm_count / (D / 256);
  splits = splits < 1 ? 1 : splits > kMaxSplits ? kMaxSplits : splits;
  float* partial = h->at<float>(h->L.partial);
  void* hmT = h->ws + h->L.hmT;
  for (int b0 = 0; b0 < B; b0 += kMaxMmaTokens) {
    const int nb = B - b0 < kMaxMmaTokens ? B - b0 : kMaxMmaTokens;
    const int32_t* lidx = dense ? nullptr : idx;
    const int32_t* lcount = dense ? nullptr : count;
    if (umma) {
      UmmaRowsParams p{};
      p.W = W_up; p.R = H; p.K = D;
      p.qbits = wq_rows; p.w_scale = q8 ? q8->s_up : nullptr; p.out_scale = q8 ? q8->s_down : nullptr;
      if (own_list) {
        p.words_in = words; p.n_words = 4 * gate_tiles; p.gate_tile_rows = gate_tile_rows;
        p.gate_rows_per_word = gate_tile_rows <= 64 ? 16 : 32;
        p.idx_out = idx; p.count_out = count; p.walk_all = umma_may_walk(nb) ? count + 1 : nullptr;
      } else {
        p.idx = lidx; p.count = lcount;
      }
      p.X = xb + (size_t)b0 * D * 2; p.x_stride = D; p.ncols_valid = nb; p.B = nb;
      if (native) { p.X = xlimb; p.ncols_valid = 4 * nb; p.tok_scale = xscale; }
      p.a = actbuf + (size_t)b0 * H; p.a_stride = H;
      p.hmT = hmT; p.hm_stride = h->L.hm_stride; p.status = h->at<int32_t>(h->L.status);
      p.act_up = h->act_up;
      SFFN_CUDA(launch_umma_rows(true, p, native ? 4 * nb : nb, h->sm_count, s));
    } else {
      RowsMmaParams p{};
      p.status = h->at<int32_t>(h->L.status);
      p.W = W_up; p.R = H; p.K = D; p.idx = lidx; p.count = lcount;
      p.X = xb + (size_t)b0 * D * 2; p.x_stride = D; p.ncols_valid = nb; p.B = nb;
      p.a = actbuf + (size_t)b0 * H; p.a_stride = H;
      p.hmT = hmT; p.hm_stride = h->L.hm_stride;
      p.act_up = h->act_up;
      SFFN_CUDA(launch_rows_mma(true, p, nb, grid_rows, s));
    }
    int nsplit = splits;
    if (q8 && !umma_down_supported(D, nb)) return SFFN_ERR_UNSUPPORTED;
    if (umma && umma_down_supported(D, nb)) {
      UmmaDownParams d{};
      d.W_down = W_down; d.R = H; d.D = D; d.qbits = wq;
      d.idx = lidx; d.count = lcount;
      d.hmT = hmT; d.hm_stride = h->L.hm_stride; d.B = nb;
      d.splits = nsplit = umma_down_splits(D, h->sm_count, kMaxSplits);
      d.walk_all = (own_list && umma_may_walk(nb)) ? count + 1 : nullptr;
      d.partial = partial; d.status = h->at<int32_t>(h->L.status);
      SFFN_CUDA(launch_umma_down(d, s));
    } else {
      DownMmaParams d{};
      d.status = h->at<int32_t>(h->L.status);
      d.W_down = W_down; d.R = H; d.D = D;
      d.idx = lidx; d.count = lcount;
      d.hmT = hmT; d.hm_stride = h->L.hm_stride; d.B = nb;
      d.partial = partial;
      SFFN_CUDA(launch_down_mma(d, splits, s));
    }
    SFFN_CUDA(launch_reduce(partial, nsplit, nb, D, y + (size_t)b0 * D, D, s));
    h->launches += 3;
  }
  return SFFN_OK;
}

// General path: gate (all tokens, chunks of <= 4) -> compaction -> up/down + reduce per chunk.
int run_general(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                const void* W_up, const void* W_down, int act, float* y, bool dense,
                const sffn_q8_scales* q8, int qbits, cudaStream_t s) {
  using namespace sffn;
  const bool bf16 = h->dtype == SFFN_BF16;
  const int wkind = q8 ? (qbits == 4 ? kWQ4 : kWQ8) : bf16 ? kWBF16 : kWF32;
  const size_t esz = bf16 ? 2 : 4;  // bytes of a token element
  const int D = h->D, H = h->H;
  float* actbuf = h->at<float>(h->L.act);
  uint8_t* flag = h->at<uint8_t>(h->L.flag);
  int32_t* idx = h->at<int32_t>(h->L.idx);
  int32_t* count = h->at<int32_t>(h->L.status) + 1;
  const int rs = h->r_max > 0 ? h->r_max : 1;
  float* vbuf = h->at<float>(h->L.v);
  float* nbuf = h->at<float>(h->L.n);
  const char* xb = static_cast<const char*>(x);

  const bool lopa = g->kind == SFFN_GATE_LOPA;
  if (lopa) {
    const int v_nb_max = (size_t)4 * D * 4 <= 227 * 1024 ? 4 : (size_t)2 * D * 4 <= 227 * 1024 ? 2 : 1;
    for (int b0 = 0; b0 < B;) {
      int nb = B - b0 >= 4 ? 4 : B - b0 >= 2 ? 2 : 1;
      nb = nb > v_nb_max ? v_nb_max : nb;
      RowDotParams p{};
      p.W = g->V; p.R = g->r; p.K = D;
      p.vec = xb + (size_t)b0 * D * esz; p.vec_stride = D;
      p.out = vbuf + (size_t)b0 * rs; p.out_stride = rs;
      p.row_scale = q8 ? q8->s_V : nullptr;
      SFFN_CUDA(launch_rowdot(wkind, !bf16, nb, false, p, h->sm_count, s));
      ++h->launches;
      b0 += nb;
    }
    if (g->use_rmsnorm) {
      SFFN_CUDA(launch_rmsnorm(vbuf, nbuf, g->rms_gain, g->r, rs, g->rms_eps, B, s));
      ++h->launches;
    }
  }
  const int gate_k = lopa ? g->r : D;
  // the gate kernel stages its tokens as fp32 in shared memory: nb * K * 4 bytes must fit (two tokens above 14.5k)
  const int gate_nb_max = (size_t)4 * gate_k * 4 <= 227 * 1024 ? 4 : (size_t)2 * gate_k * 4 <= 227 * 1024 ? 2 : 1;
  for (int b0 = 0; b0 < B;) {
    int nb = B - b0 >= 4 ? 4 : B - b0 >= 2 ? 2 : 1;
    nb = nb > gate_nb_max ? gate_nb_max : nb;
    RowDotParams p{};
    if (lopa) {
      p.W = g->U; p.R = H; p.K = g->r;
      p.vec = (g->use_rmsnorm ? nbuf : vbuf) + (size_t)b0 * rs; p.vec_stride = rs;
      p.g_idx = g->g_idx; p.g_sign = g->g_sign;
    } else {
      p.W = g->W_g; p.R = H; p.K = D;
      p.vec = xb + (size_t)b0 * D * esz; p.vec_stride = D;
    }
    p.out = actbuf + (size_t)b0 * H; p.out_stride = H;
    p.b_g = b_g;
    p.x = xb + (size_t)b0 * D * esz; p.x_stride = D;
    p.act = act;
    p.flag = dense ? nullptr : flag;
    p.flag_or = b0 > 0;
    p.row_scale = q8 ? q8->s_gate : nullptr;
    SFFN_CUDA(launch_rowdot(wkind, lopa || !bf16, nb, true, p, h->sm_count, s));
    ++h->launches;
    b0 += nb;
  }
  if (!dense) {
    SFFN_CUDA(launch_compact(flag, H, idx, count, s));
    ++h->launches;
    h->list_state = 1;
#ifdef SFFN_DEBUG
    if (sffn::fused_test_knobs().poison_list) SFFN_CUDA(cudaMemsetAsync(idx, 0x7f, 4, s));  // entry 0 := 2139062143
#endif
  }
  const int nbmax = updown_max_tokens(wkind, D);
  int grid = 2 * h->sm_count;
  if (grid > kMaxUpDownGrid) grid = kMaxUpDownGrid;
  float* partial = h->at<float>(h->L.partial);
  for (int b0 = 0; b0 < B;) {
    const int left = B - b0;
    const int nb = (left >= 4 && nbmax >= 4) ? 4 : left >= 2 ? 2 : 1;
    UpDownParams p{};
    p.status = h->at<int32_t>(h->L.status);
    p.W_up = W_up; p.W_down = W_down;
    p.x = xb + (size_t)b0 * D * esz; p.x_stride = D;
    p.a = actbuf + (size_t)b0 * H; p.a_stride = H;
    p.idx = dense ? nullptr : idx;
    p.count = dense ? nullptr : count;
    p.H = H; p.D = D;
    p.partial = partial;
    p.act_up = h->act_up;
    p.s_up = q8 ? q8->s_up : nullptr; p.s_down = q8 ? q8->s_down : nullptr;
    SFFN_CUDA(launch_updown(wkind, nb, p, grid, s));
    SFFN_CUDA(launch_reduce(partial, grid, nb, D, y + (size_t)b0 * D, D, s));
    h->launches += 2;
    b0 += nb;
  }
  return SFFN_OK;
}

int run(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g, const void* W_up,
        const void* W_down, int act, float* y, bool dense, void* stream, const sffn_q8_scales* q8 = nullptr,
        int qbits = 8) {
  const int rc = check_call(h, x, B, g, W_up, W_down, act, y, q8, qbits);
  if (rc != SFFN_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int wkind = q8 ? (qbits == 4 ? sffn::kWQ4 : sffn::kWQ8) : h->dtype == SFFN_BF16 ? sffn::kWBF16 : sffn::kWF32;
  const bool lopa_gate = g->kind == SFFN_GATE_LOPA;
  const int gate_k = lopa_gate ? g->r : h->D;
  const int chunk = B < kMaxMmaTokens ? B : kMaxMmaTokens;
  // a batch the tensor-core kernels can take (bf16 tokens; bf16, int8 or int4 rows; more than 64 tokens: in chunks of 64)
  const int gate_cols_chunk = lopa_gate ? 2 * chunk : chunk;
  // rows of weight codes: the tcgen05 kernels only (they expand the codes to bf16 on the way to the tensor cores)
  const bool q_tensor_ok = !q8 || (h->path != SFFN_PATH_MMA_SYNC && sffn::umma_rows_supported(gate_k, gate_cols_chunk) &&
                                   sffn::umma_rows_supported(h->D, chunk) && sffn::umma_down_supported(h->D, chunk) &&
                                   (!lopa_gate || sffn::umma_rows_supported(h->D, chunk)));
  const bool tensor_batch = h->dtype == SFFN_BF16 && B >= 2 && h->path != SFFN_PATH_GENERAL && q_tensor_ok &&
                            h->path != SFFN_PATH_FUSED && sffn::batched_mma_supported(h->D, gate_k, gate_cols_chunk);
  // Any other batch (fp32 operands, a row width the tensor-core kernels do not tile, SFFN_PATH_FUSED): the single-token
  // kernel once per token, where it serves the shape.  The CUDA-core batch kernels are slower than B single-token calls
  // (int8, 4096 x 14336, B = 16: 1.66 ms against 0.33 ms; bf16 rows of 4000 elements: 1.03 ms against 0.46 ms; fp32:
  // 0.86 against 0.77 ms).
  // The fired flags of the tokens are OR-ed: the list is the batch's union.
  if (B > 1 && !tensor_batch && h->path != SFFN_PATH_GENERAL && h->path != SFFN_PATH_MMA_SYNC &&
      sffn::fused_supported(wkind, h->D, h->H, 1, g, h->sm_count)) {
    const size_t tok_bytes = (size_t)h->D * ((q8 || h->dtype == SFFN_BF16) ? 2 : 4);
    for (int b = 0; b < B; ++b) {
      sffn::FusedCall c{};
      c.wkind = wkind;
      if (q8) { c.s_gate = q8->s_gate; c.s_V = q8->s_V; c.s_up = q8->s_up; c.s_down = q8->s_down; }
      c.D = h->D; c.H = h->H;
      c.x = static_cast<const char*>(x) + (size_t)b * tok_bytes;
      c.gate = g; c.b_g = b_g; c.W_up = W_up; c.W_down = W_down; c.act = act; c.act_up = h->act_up;
      c.gated_skip = h->gated_skip != 0;
      c.engine = h->gate_engine; c.y = y + (size_t)b * h->D;
      c.dense = dense; c.flag_or = b > 0;
      c.workspace = h->ws + h->L.fused;
      c.r_max = h->r_max;
      c.status = h->at<int32_t>(h->L.status);
      c.flag = h->at<uint8_t>(h->L.flag);
      c.sm_count = h->sm_count;
      int launched = 0;
      if (sffn::launch_fused(c, s, &launched) != cudaSuccess) return SFFN_ERR_CUDA;
      h->launches += launched;
    }
    if (!dense) h->list_state = 2;
    return SFFN_OK;
  }
  const bool fused_ok = sffn::fused_supported(wkind, h->D, h->H, B, g, h->sm_count);
  if (h->path == SFFN_PATH_FUSED && !fused_ok) return SFFN_ERR_UNSUPPORTED;
  if (fused_ok && h->path != SFFN_PATH_GENERAL) {
    sffn::FusedCall c{};
    c.wkind = wkind;
    if (q8) { c.s_gate = q8->s_gate; c.s_V = q8->s_V; c.s_up = q8->s_up; c.s_down = q8->s_down; }
    c.D = h->D; c.H = h->H;
    c.x = x; c.gate = g; c.b_g = b_g; c.W_up = W_up; c.W_down = W_down; c.act = act; c.act_up = h->act_up; c.engine = h->gate_engine; c.y = y;
    c.gated_skip = h->gated_skip != 0;
    c.dense = dense;
    c.workspace = h->ws + h->L.fused;
    c.r_max = h->r_max;
    c.status = h->at<int32_t>(h->L.status);
    c.flag = h->at<uint8_t>(h->L.flag);
    c.sm_count = h->sm_count;
    int launched = 0;
    if (sffn::launch_fused(c, s, &launched) != cudaSuccess) return SFFN_ERR_CUDA;
    h->launches += launched;
    if (!dense) h->list_state = 2;
    return SFFN_OK;
  }
  if (tensor_batch) {
    // chunks of at most 64 tokens; with more than one chunk the fired sets are accumulated into the batch's union
    uint8_t* uni = h->at<uint8_t>(h->L.union_flag);
    const bool parts = B > kMaxMmaTokens;
    if (parts && !dense) SFFN_CUDA(cudaMemsetAsync(uni, 0, h->H, s));
    for (int b0 = 0; b0 < B; b0 += kMaxMmaTokens) {
      const int nb = B - b0 < kMaxMmaTokens ? B - b0 : kMaxMmaTokens;
      const int cols = lopa_gate ? 2 * nb : nb;
      const bool umma_ok = sffn::umma_rows_supported(gate_k, cols) && sffn::umma_rows_supported(h->D, nb);
      const int rc2 = run_batched(h, static_cast<const char*>(x) + (size_t)b0 * h->D * 2, nb, g, b_g, W_up, W_down, act,
                                  y + (size_t)b0 * h->D, dense, umma_ok && h->path != SFFN_PATH_MMA_SYNC, q8, qbits, s);
      if (rc2 != SFFN_OK) return rc2;
      if (parts && !dense) {
        SFFN_CUDA(sffn::launch_mark_union(h->at<int32_t>(h->L.idx), h->at<int32_t>(h->L.status) + 1, h->H, uni, s));
        ++h->launches;
      }
    }
    if (parts && !dense) {
      SFFN_CUDA(cudaMemcpyAsync(h->at<uint8_t>(h->L.flag), uni, h->H, cudaMemcpyDeviceToDevice, s));
      h->list_state = 2;  // the list is compacted from the union's flags on request
    }
    return SFFN_OK;
  }
  if (h->path == SFFN_PATH_MMA_SYNC) return SFFN_ERR_UNSUPPORTED;
  return run_general(h, x, B, g, b_g, W_up, W_down, act, y, dense, q8, qbits, s);
}

// Device-side alias of a 16-byte aligned pointer into pinned, mapped host memory; null for anything else.
const void* mapped_device_pointer(const void* host) {
  if (!host || (reinterpret_cast<uintptr_t>(host) & 15u)) return nullptr;
  cudaPointerAttributes attr{};
  if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
    cudaGetLastError();  // unregistered memory reports an error on some drivers: not ours to keep
    return nullptr;
  }
  return attr.type == cudaMemoryTypeHost ? attr.devicePointer : nullptr;
}

}  // namespace

extern "C" {

const char* sffn_last_cuda_error(void) {
  static thread_local char text[96];
  snprintf(text, sizeof(text), "%s (api.cu:%d)", cudaGetErrorName(g_last_cuda_error), g_last_cuda_line);
  return g_last_cuda_error == cudaSuccess ? "cudaSuccess" : text;
}


int sparse_ffn_forward(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                       const void* W_up, const void* W_down, int act, float* y, void* stream) {
  return run(h, x, B, g, b_g, W_up, W_down, act, y, false, stream);
}

int dense_ffn_forward(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                      const void* W_up, const void* W_down, int act, float* y, void* stream) {
  return run(h, x, B, g, b_g, W_up, W_down, act, y, true, stream);
}

int sparse_ffn_forward_q8(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                          const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                          void* stream) {
  if (!scales) return SFFN_ERR_INVALID_ARG;
  return run(h, x, B, g, b_g, W_up, W_down, act, y, false, stream, scales);
}

int dense_ffn_forward_q8(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                         const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                         void* stream) {
  if (!scales) return SFFN_ERR_INVALID_ARG;
  return run(h, x, B, g, b_g, W_up, W_down, act, y, true, stream, scales);
}

int sparse_ffn_forward_q4(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                          const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                          void* stream) {
  if (!scales) return SFFN_ERR_INVALID_ARG;
  return run(h, x, B, g, b_g, W_up, W_down, act, y, false, stream, scales, 4);
}

int dense_ffn_forward_q4(sffn_handle* h, const void* x, int B, const sffn_gate* g, const float* b_g,
                         const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                         void* stream) {
  if (!scales) return SFFN_ERR_INVALID_ARG;
  return run(h, x, B, g, b_g, W_up, W_down, act, y, true, stream, scales, 4);
}

int sparse_ffn_forward_host(sffn_handle* h, const void* x_host, int B, const sffn_gate* g,
                            const float* b_g, const void* W_up, const void* W_down, int act,
                            float* y_host, void* stream) {
  if (!h || !x_host || !y_host || B < 1 || B > h->B_max) return SFFN_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t esz = h->dtype == SFFN_BF16 ? 2 : 4;
  float* ys = h->at<float>(h->L.ystage);
  const size_t xbytes = (size_t)B * h->D * esz, ybytes = (size_t)B * h->D * 4;
  // Pinned (mapped) host memory is read and written by the kernels themselves: a small copy kernel brings
  // the tokens in and the last kernel of the call stores y straight to the host, so the stream carries no
  // copy-engine operation between kernels.  Pageable memory takes the two asynchronous copies.
  void* xs = h->ws + h->L.xstage;
  const void* x_map = mapped_device_pointer(x_host);
  float* y_map = static_cast<float*>(const_cast<void*>(mapped_device_pointer(y_host)));
  if (x_map) {
    SFFN_CUDA(sffn::launch_copy16(x_map, xs, xbytes, s));
    ++h->launches;
  } else {
    SFFN_CUDA(cudaMemcpyAsync(xs, x_host, xbytes, cudaMemcpyHostToDevice, s));
  }
  const int rc = run(h, xs, B, g, b_g, W_up, W_down, act, y_map ? y_map : ys, false, stream);
  if (rc != SFFN_OK) return rc;
  if (!y_map) SFFN_CUDA(cudaMemcpyAsync(y_host, ys, ybytes, cudaMemcpyDeviceToHost, s));
  return SFFN_OK;
}

int sffn_residual_cast(const float* y, const void* resid, float alpha, void* out, int n, int dtype, void* stream) {
  if (!y || !resid || !out || n < 4 || n % 4 || (dtype != SFFN_F32 && dtype != SFFN_BF16)) return SFFN_ERR_INVALID_ARG;
  if (!aligned16(y) || !aligned16(resid) || !aligned16(out)) return SFFN_ERR_UNSUPPORTED;
  SFFN_CUDA(sffn::launch_residual_cast(dtype == SFFN_BF16, y, resid, alpha, out, n, static_cast<cudaStream_t>(stream)));
  return SFFN_OK;
}

int sffn_lopa_m_step(const float* W, const float* P, int H, int D, int32_t* g_idx, int8_t* g_sign, double* row_energy,
                     float* row_best, void* stream) {
  if (!W || !g_idx || !g_sign || H < 1 || D < 1) return SFFN_ERR_INVALID_ARG;
  SFFN_CUDA(sffn::launch_lopa_m_step(W, P, H, D, g_idx, g_sign, row_energy, row_best, static_cast<cudaStream_t>(stream)));
  return SFFN_OK;
}

int sffn_lopa_residual(const float* W, const int32_t* g_idx, const int8_t* g_sign, int H, int D, float* A, void* stream) {
  if (!W || !g_idx || !g_sign || !A || H < 1 || D < 1) return SFFN_ERR_INVALID_ARG;
  SFFN_CUDA(sffn::launch_lopa_residual(W, g_idx, g_sign, H, D, A, static_cast<cudaStream_t>(stream)));
  return SFFN_OK;
}

int sffn_last_active(sffn_handle* h, const int32_t** idx_dev, const int32_t** count_dev, void* stream) {
  if (!h || !idx_dev || !count_dev) return SFFN_ERR_INVALID_ARG;
  if (h->list_state == 0) return SFFN_ERR_INVALID_ARG;
  int32_t* idx = h->at<int32_t>(h->L.idx);
  int32_t* count = h->at<int32_t>(h->L.status) + 1;
  if (h->list_state == 2) {
    SFFN_CUDA(sffn::launch_compact(h->at<uint8_t>(h->L.flag), h->H, idx, count,
                                   static_cast<cudaStream_t>(stream)));
    ++h->launches;
    h->list_state = 1;
  }
  *idx_dev = idx;
  *count_dev = count;
  return SFFN_OK;
}

int sffn_reset(sffn_handle* h, void* stream) {
  if (!h) return SFFN_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  SFFN_CUDA(cudaMemsetAsync(h->ws + h->L.status, 0, 256, s));
  // the single-token kernels' arrival counters, call number and tagged partials
  SFFN_CUDA(cudaMemsetAsync(h->ws + h->L.fused, 0, sffn::fused_workspace_bytes(h->D, h->H, h->r_max), s));
  h->list_state = 0;
  return SFFN_OK;
}

int sffn_last_device_status(sffn_handle* h, int* status) {
  if (!h || !status) return SFFN_ERR_INVALID_ARG;
  int32_t word = 0;
  SFFN_CUDA(cudaDeviceSynchronize());
  SFFN_CUDA(cudaMemcpy(&word, h->ws + h->L.status, sizeof word, cudaMemcpyDeviceToHost));
  *status = word;
  return SFFN_OK;
}

}  // extern "C"
