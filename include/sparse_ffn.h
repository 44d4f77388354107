/*
 * sparse_ffn.h -- C ABI of the activation-sparse gated FFN library for NVIDIA B200 (sm_100a).
 *
 * The library evaluates, for B independent tokens x_b in R^D,
 *
 *     y_b = W_2 ( A(W_1 x_b + b_g)  .  (W_3 x_b) )                       (paper Eq. 1)
 *
 * by the sparse execution scheme of the paper's Sec. 3.1 ("FFN FLOP-ratio"): the gate W_1 x is always
 * computed in full; a neuron j whose activation A(.)_j is zero is known before W_3 and W_2 are
 * touched, so row j of W_3 and column j of W_2 are never read.  W_1 is either a full matrix
 * (standard gating) or the low-parameter gate of Sec. 3.3 (Eq. 3), W_1 = G + U V, evaluated as
 * G x + U RMSNorm(V x), with the RMSNorm optional (architecture casting, Sec. 3.4, has none).
 * For B > 1 the rows are read once for the union of the tokens' active sets (Sec. 5.4).
 *
 * Storage (all row-major, all DEVICE memory unless a name ends in _host):
 *     x       [B, D]   element type = the handle's dtype (fp32 or bf16)
 *     W_g     [H, D]   = W_1                       same dtype
 *     W_up    [H, D]   = W_3                       same dtype
 *     W_down  [H, D]   = W_2 transposed (row j is column j of W_2)   same dtype
 *     V [r, D], U [H, r]                           same dtype
 *     b_g [H], rms_gain [r]                        fp32
 *     g_idx [H] int32, g_sign [H] int8 (+1 / -1)
 *     y       [B, D]   fp32, overwritten
 * The gate bias b_g is not part of Eq. 1 (pass NULL for the paper's form); it is the knob the
 * synthetic workloads use to set the sparsity.
 *
 * Ownership: every buffer is owned by the caller and only read (y and the workspace are written).
 * The library never allocates or frees device memory: the caller allocates `workspace`
 * (sffn_workspace_bytes) and hands it to sffn_create.  Pointers must be 16-byte aligned and rows
 * must be a multiple of 16 bytes (D and r multiples of 8 for bf16, of 4 for fp32), otherwise
 * SFFN_ERR_UNSUPPORTED.
 *
 * Stream order: a call is ordered after everything queued before it on `stream` as far as x, the workspace
 * and y are concerned.  The weights and per-neuron gate parameters (W_g, W_up, W_down, V, U, b_g, g_idx,
 * g_sign, rms_gain) are treated as parameters: the kernels may start reading them while the work queued
 * just before the call is still running (that is how back-to-back calls overlap), so they must not be
 * written by device work queued immediately before a call on the same stream -- put a stream or event
 * synchronisation between an update of the weights and the next call.
 * A single-token call runs one CTA on every SM, and its CTAs wait for one another (LoPA: for the rank-r vector;
 * always: the first CTAs to finish stay and wait for the partial results of the rest, which they sum; every wait is bounded).
 * Calls of different handles are therefore meant to run one after another -- one stream, or streams ordered by
 * events.  Two standard-gate calls that overlap still complete; LoPA calls, or three and more calls at once, can
 * starve each other of SMs and end with SFFN_ERR_TIMEOUT in the device status instead of a result.
 *
 * Errors: every entry point returns an sffn_status.  The return value covers host-side validation
 * and launch errors only; calls are asynchronous on `stream`.  Conditions detected on the device
 * (a bounded wait that ran out) are recorded in a status word inside the workspace and read back
 * with sffn_last_device_status; the kernels never trap and never spin without a limit.
 * The same inputs give bitwise the same y and the same index list on every call.
 * Inputs are assumed finite (an Inf/NaN in a skipped row would make sparse and dense differ).
 */
#ifndef SPARSE_FFN_H_
#define SPARSE_FFN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SFFN_OK = 0,
  SFFN_ERR_INVALID_ARG = 1, /* null handle/pointer, B out of range, bad enum                    */
  SFFN_ERR_UNSUPPORTED = 2, /* misaligned pointer, row size not a multiple of 16 bytes, too big */
  SFFN_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small                       */
  SFFN_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch, copy)                        */
  SFFN_ERR_TIMEOUT = 5,     /* device status only: a bounded device-side wait gave up           */
  SFFN_ERR_BOUNDS = 6       /* device status only, debug builds (-DSFFN_DEBUG): an index that was about to address
                               global memory lay outside its array; the access was skipped or clamped */
} sffn_status;

/* Activation A of Eq. 1.  RELU and R-S+ follow the table of Sec. 3.1 (R-S+: 0 for z < 0,
 * z*sigmoid(z) for z >= 0); SQRELU = max(z,0)^2 is one of the activations of the paper's activation
 * study.  For all three A(z) != 0 exactly when z > 0, which is the test the library applies. */
typedef enum { SFFN_ACT_RELU = 0, SFFN_ACT_SQRELU = 1, SFFN_ACT_RSPLUS = 2, SFFN_ACT_NONE = 3, SFFN_ACT_SILU = 4 } sffn_act;

typedef enum { SFFN_F32 = 0, SFFN_BF16 = 1 } sffn_dtype;

typedef enum { SFFN_GATE_STANDARD = 0, SFFN_GATE_LOPA = 1 } sffn_gate_kind;

/* Which kernels serve a call.  AUTO picks the fused kernels for B = 1 when the shape allows it and the
 * tcgen05 tensor-core kernels for batches (B >= 2) of bf16 tokens with bf16, int8 or int4 rows (int8 rows are
 * multiplied as int8 against the tokens split into int8 limbs, or, like int4 rows, expanded to bf16 in shared
 * memory on their way to the tensor cores; more than 64 tokens run in chunks of 64, the list of fired neurons
 * being the union over all chunks).  A batch those kernels do not take (fp32
 * operands, a row width they do not tile) runs the fused kernel once per token with the fired flags OR-ed,
 * which is faster than the CUDA-core batch kernels; what is left goes to the general CUDA-core kernels.
 * The others force one family (SFFN_ERR_UNSUPPORTED if it cannot serve the call): GENERAL = CUDA-core
 * kernels for any batch, FUSED = single-token fused kernels (a batch: once per token), MMA_SYNC = batched kernels on the
 * warp-level mma.sync tensor-core path. */
typedef enum { SFFN_PATH_AUTO = 0, SFFN_PATH_GENERAL = 1, SFFN_PATH_FUSED = 2, SFFN_PATH_MMA_SYNC = 3 } sffn_path;

/* Gate description.  STANDARD uses W_g only.  LOPA (Eq. 3; "LoPA in practice", Sec. 3.3) uses
 *   z_j = g_sign[j] * x[g_idx[j]] + sum_k U[j,k] n_k + b_g[j],   n = RMSNorm(V x) or V x,
 *   RMSNorm(v)_k = rms_gain[k] * v_k / sqrt(mean_k v_k^2 + rms_eps).
 * g_idx NULL drops the fixed matrix G (plain low-rank gate); g_sign NULL means +1 everywhere;
 * rms_gain NULL means 1. */
typedef struct {
  int32_t kind;            /* sffn_gate_kind                                        */
  int32_t r;               /* LOPA: rank, 1 <= r <= r_max of the handle             */
  const void* W_g;         /* STANDARD: [H, D]                                      */
  const void* V;           /* LOPA: [r, D]                                          */
  const void* U;           /* LOPA: [H, r]                                          */
  const int32_t* g_idx;    /* LOPA: [H] column of the single nonzero of G, or NULL  */
  const int8_t* g_sign;    /* LOPA: [H] +1/-1, or NULL                              */
  const float* rms_gain;   /* LOPA: [r] or NULL                                     */
  int32_t use_rmsnorm;     /* LOPA: 1 = with RMSNorm (Sec. 3.3), 0 = without (Sec. 3.4) */
  float rms_eps;           /* LOPA: added to the mean square; the paper gives no value */
} sffn_gate;

typedef struct sffn_handle sffn_handle;

/* Bytes of device workspace a handle for these limits needs.  r_max may be 0 (no LoPA calls). */
int sffn_workspace_bytes(int D, int H, int r_max, int B_max, int dtype, size_t* bytes);

/* Creates a handle on the current device.  `workspace` is device memory of at least
 * sffn_workspace_bytes(...) bytes, 256-byte aligned, owned by the caller and kept alive (and not
 * shared with another handle) until sffn_destroy.  The call clears the workspace and returns when that is done.
 * Calls on one handle must be issued to one stream at a time. */
int sffn_create(sffn_handle** handle, int D, int H, int r_max, int B_max, int dtype,
                void* workspace, size_t workspace_bytes);

/* Frees host state only; the workspace stays the caller's. */
int sffn_destroy(sffn_handle* handle);

int sffn_set_path(sffn_handle* handle, int path /* sffn_path */);

/* Where a single-token call (B = 1, fused path) computes the gate.  Both engines give the result of Eq. 1 and stream
 * the same bytes; they differ in what the SMs' issue slots are spent on.  CUDA_CORE: fp32 FMAs on bf16 / fp32 / int8
 * rows, any gate.  TENSOR_CORE: tcgen05 MMAs, which leaves the issue slots to the up / down stage -- bf16 rows,
 * standard gate, D a multiple of 64 and at least 1024; a call it does not cover runs on the CUDA cores.  AUTO (the
 * default) takes the CUDA cores for sparse calls, where at the paper's sparsity levels (0.8 and up) the gate stream
 * alone sets the time, and the tensor cores for dense calls; a caller whose models fire more than about a fifth of
 * their neurons sets TENSOR_CORE. */
typedef enum { SFFN_GATE_ENGINE_AUTO = 0, SFFN_GATE_ENGINE_CUDA_CORE = 1, SFFN_GATE_ENGINE_TENSOR_CORE = 2 } sffn_gate_engine;
int sffn_set_gate_engine(sffn_handle* handle, int engine /* sffn_gate_engine */);

/* Double activation (Sec. 3.3, "Double activation"): with act_up = RELU / SQRELU / RSPLUS / SILU every later
 * call on the handle computes y = W_2 ( A(W_1 x + b_g) . A_3(W_3 x) ), A_3 = act_up, in the sparse and
 * in the dense entry points alike; SFFN_ACT_NONE (the default) is Eq. 1.  SILU (z * sigmoid(z), the table of
 * Sec. 3.1) is what a model cast per Sec. 3.3 keeps on the up branch: only the activation of W_1 is cast to a
 * sparse one.  It exists as A_3 only: the gate's `act` must be one of the three sparse activations.  A neuron whose product
 * A(.) A_3(.) is zero for every token of the call contributes nothing (the "s_gated" site of the
 * paper's sparsity-sites table): the CUDA-core path (SFFN_PATH_GENERAL) then does not read its row of
 * W_down; the tensor-core paths fetch the two rows of a fired neuron together and read it, and so does the
 * single-token fused kernel unless sffn_set_gated_skip asks otherwise.
 * SFFN_ACT_NONE and SFFN_ACT_SILU are not gate activations: `act` of the forward calls stays one of the first three. */
int sffn_set_up_activation(sffn_handle* handle, int act_up /* sffn_act */);

/* The "s_gated" site on the single-token fused kernel (sparsity-sites table; Sec. 3.3 "Double activation").  on = 1:
 * sparse calls with one token, a standard gate, bf16 or fp32 rows and an up activation set fetch the W_down row of a
 * fired neuron only once h_j = a_j A_3(u_j) is known and is not zero: a second, dependent fetch per kept row instead of
 * two rows fetched together.  y is bitwise the same either way; fewer bytes are read (about half of the W_down rows
 * with A_3 = RELU), but the last rows of a call pay two round trips to memory instead of one, and on a B200 the call
 * is not faster for it (0 to 1.5 us slower): the default is 0.  Every other kind of call ignores the setting. */
int sffn_set_gated_skip(sffn_handle* handle, int on);

/* Sparse execution of Eq. 1 (Sec. 3.1): gate in full, then only the active rows of W_up / W_down.
 * x [B,D] and all weights on the device; y [B,D] fp32 on the device, fully overwritten (zeros when
 * no neuron fires).  1 <= B <= B_max.  `stream` is a cudaStream_t (NULL = default stream). */
int sparse_ffn_forward(sffn_handle* handle, const void* x, int B, const sffn_gate* gate,
                       const float* b_g, const void* W_up, const void* W_down, int act, float* y,
                       void* stream);

/* Dense comparator: the same function with every one of the H rows of W_up / W_down read
 * (Eq. 1 as written).  Same arguments; defines the "x1" of every speedup. */
int dense_ffn_forward(sffn_handle* handle, const void* x, int B, const sffn_gate* gate,
                      const float* b_g, const void* W_up, const void* W_down, int act, float* y,
                      void* stream);

/* Weight-only int8 (the paper's appendix on quantisation-aware training: only the weights become int8, at inference
 * time; tokens and all arithmetic stay in floating point).  The paper does not fix the format; here every
 * weight matrix is stored as int8 codes, row-major, with one fp32 scale per row:
 *     W[j, k] = s[j] * q[j, k],   q in [-127, 127].
 * In these two calls the pointers W_up, W_down and, inside `gate`, W_g (STANDARD) or V and U (LOPA) address the
 * int8 codes ([H,D], [H,D], [H,D], [r,D], [H,r]); `scales` carries the row scales.  Tokens x are bf16: the handle
 * must have been created with SFFN_BF16.  Rows must be a multiple of 16 bytes (D and r multiples of 16).
 * Everything else (b_g, g_idx, g_sign, RMSNorm, act, y, the active list, double activation) is as in
 * sparse_ffn_forward / dense_ffn_forward.  One token runs in the fused kernel; under a standard gate its gate and up
 * dot products are integer ones (dp4a) against the token split, 16 entries at a time, into two int8 limbs and a
 * scale (x = s_c (q0 + q1/128) up to 3e-5 of the largest |x| among those 16 entries; int4: 32 entries, nibbles used
 * as the bytes 16 x code), all sums in fp32 beyond a chunk; LoPA gates use fp32 arithmetic throughout.  A batch runs
 * the tcgen05 batch kernels (D and r multiples of 64, D of 256; otherwise, or under SFFN_PATH_FUSED, the fused kernel once per token; the
 * list of fired neurons is the union over the tokens).  There the gate and up products of int8 rows are int8 x int8
 * with int32 accumulators, each token entering as four int8 limbs and a scale (x = s (q0 + q1/128 + q2/128^2 +
 * q3/128^3) up to 2^-22 max|x|; D and r multiples of 128; int4 rows take the same route, their nibbles expanded to
 * int8 in shared memory), and the down product and other widths expand the codes to bf16 in shared memory; row scales
 * are applied to the accumulator rows.  The CUDA-core kernels (fp32 arithmetic on the decoded codes) serve
 * SFFN_PATH_GENERAL (SFFN_PATH_MMA_SYNC: SFFN_ERR_UNSUPPORTED).  Converting a trained model to this format is
 * an offline step outside this library. */
typedef struct {
  const float* s_gate; /* [H]  row scales of W_g (STANDARD) or of U (LOPA) */
  const float* s_V;    /* [r]  row scales of V (LOPA only; may be NULL otherwise) */
  const float* s_up;   /* [H]  row scales of W_up */
  const float* s_down; /* [H]  row scales of W_down (row j = column j of W_2) */
} sffn_q8_scales;

int sparse_ffn_forward_q8(sffn_handle* handle, const void* x, int B, const sffn_gate* gate, const float* b_g,
                          const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                          void* stream);
int dense_ffn_forward_q8(sffn_handle* handle, const void* x, int B, const sffn_gate* gate, const float* b_g,
                         const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                         void* stream);

/* Weight-only int4 (the same appendix names int4 beside int8 and fixes no format either).  Here: two's-complement
 * codes in [-8, 7], two per byte with the even column in the low nibble, row-major, one fp32 scale per row:
 *     W[j, 2b] = s[j] * low_nibble(p[j, b]),   W[j, 2b + 1] = s[j] * high_nibble(p[j, b]).
 * The weight pointers address the packed bytes ([H, D/2], [r, D/2], [H, r/2]); `scales` as for int8.  Rows must be a
 * multiple of 16 bytes (D and r multiples of 32).  Otherwise exactly like the _q8 calls: bf16 tokens, fp32 arithmetic,
 * one token in the fused kernel (rows of up to 8192 codes there), a batch on the tcgen05 batch kernels, wider rows in
 * the CUDA-core kernels. */
int sparse_ffn_forward_q4(sffn_handle* handle, const void* x, int B, const sffn_gate* gate, const float* b_g,
                          const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                          void* stream);
int dense_ffn_forward_q4(sffn_handle* handle, const void* x, int B, const sffn_gate* gate, const float* b_g,
                         const void* W_up, const void* W_down, const sffn_q8_scales* scales, int act, float* y,
                         void* stream);

/* End-to-end variant of sparse_ffn_forward for callers whose activations live on the host:
 * x_host [B,D] (handle dtype) and y_host [B,D] fp32 are HOST pointers; weights stay on the device.
 * Brings x in, runs the sparse path, puts y out, all on `stream`; y_host is valid once the stream has
 * synchronised.  Pinned host memory (cudaHostAlloc / cudaHostRegister, 16-byte aligned) is accessed by
 * the kernels directly -- a small copy kernel reads x, the call's last kernel stores y -- so no
 * copy-engine operation sits between the kernels; any other host memory goes through cudaMemcpyAsync.
 * x_host must hold its final contents when the call is made: the library may read it before earlier work
 * on `stream` has finished (as a copy from pageable memory would). */
int sparse_ffn_forward_host(sffn_handle* handle, const void* x_host, int B, const sffn_gate* gate,
                            const float* b_g, const void* W_up, const void* W_down, int act,
                            float* y_host, void* stream);

/* Introspection for tests and benchmarks, valid after the stream of the last sparse call has
 * synchronised.  *idx_dev points at the ascending list of active neurons of that call (for B > 1:
 * of the union over the tokens) and *count_dev at its length; both live in the workspace.  The list
 * is materialised by this call (one small launch on `stream`) and is valid once it synchronises. */
int sffn_last_active(sffn_handle* handle, const int32_t** idx_dev, const int32_t** count_dev,
                     void* stream);

/* Reads the device status word (synchronises the device): SFFN_OK or SFFN_ERR_TIMEOUT.  The word is sticky: once a
 * bounded wait has run out, the single-token kernels' arrival counters are out of step and every later call on the
 * handle leaves y unwritten until sffn_reset. */
int sffn_last_device_status(sffn_handle* handle, int* status);

/* Puts a handle back into its initial state after SFFN_ERR_TIMEOUT: clears the status word and the arrival counters
 * (two small asynchronous memsets on `stream`, ordered like a call).  The handle's stream must hold no unfinished
 * call of this handle that could still time out.  Weights, settings and the workspace's other contents are kept. */
int sffn_reset(sffn_handle* handle, void* stream);

/* Number of kernels this handle has launched since creation (host-side counter). */
int sffn_launch_count(sffn_handle* handle, long long* launches);

/* Sparse FFN without a handle, a workspace or any allocation -- the paper has no counterpart; this
 * entry point exists for callers that cannot obtain device memory at call time: code that runs after
 * the application has given all of HBM to its own pool (so cudaMalloc fails, or is forbidden by the
 * host framework), or inside a latency-critical loop where the device-wide synchronisation that
 * cudaMalloc/cudaFree imply is not acceptable, and that own no buffer they could pass to sffn_create.
 *
 * Standard gate, one token (B = 1): y = W_down^T (A(W_g x + b_g) . (W_up x)), sparse execution as
 * in sparse_ffn_forward, computed by the general-path kernels.  x [D], W_g / W_up / W_down [H, D] in
 * `dtype` (sffn_dtype), b_g [H] fp32 or NULL, y [D] fp32: all DEVICE pointers owned by the caller,
 * 16-byte aligned, rows a multiple of 16 bytes.
 *
 * Scratch: the gate values, fired flags, index list and per-CTA partial sums live in one array that
 * is part of this library's device image (about 4.3 MB; every GPU that loads the library keeps it
 * until the process exits).  That fixes the limits D <= SFFN_STATIC_MAX_D and H <= SFFN_STATIC_MAX_H;
 * larger shapes return SFFN_ERR_UNSUPPORTED (use a handle with your own workspace instead).
 * The call makes no cudaMalloc / cudaFree and calls no allocating library routine.
 *
 * The first call on each device looks up the array's device address (one cudaGetSymbolAddress with
 * that device current) and remembers it; make that first call before any stream capture begins.
 * All calls on a device share the one array, which keeps the previous call's contents: a call
 * rewrites everything it later reads and clears the list length itself, so back-to-back calls on
 * one stream are independent -- but two calls that can overlap on the GPU (different streams, or
 * different host threads on different streams) race on it and must be serialised by the caller. */
#define SFFN_STATIC_MAX_D 8192
#define SFFN_STATIC_MAX_H 32768
int sparse_ffn_forward_static(const void* x, const void* W_g, const float* b_g, const void* W_up,
                              const void* W_down, int D, int H, int dtype, int act, float* y,
                              void* stream);

/* Name of the CUDA runtime error (cudaGetErrorName, with the library source line that saw it) behind the last SFFN_ERR_CUDA that a handle call
 * returned on the calling thread; "cudaSuccess" if there was none.  Diagnostics only. */
const char* sffn_last_cuda_error(void);

/* Glue for a layer loop (not a step of the paper's FFN): out[i] = dtype(resid[i] + alpha * y[i]) for the n
 * elements (a multiple of 4) of an fp32 FFN output y, e.g. the residual stream's update and its cast back to
 * the token dtype.  Device pointers, 16-byte aligned; out may alias resid.  The kernel takes part in the
 * programmatic dependent launch chain of the FFN kernels, so a loop FFN -> this -> FFN runs without the
 * full serialisation a foreign elementwise kernel would put between two calls. */
int sffn_residual_cast(const float* y, const void* resid, float alpha, void* out, int n, int dtype /* sffn_dtype */,
                       void* stream);

/* Offline conversion of a full gate matrix W [H,D] (fp32) into a LoPA gate M + U V (architecture casting, Sec. 3.4,
 * "LoPA approximation": minimise ||W - M - U V||_F^2 by alternating two exact half-steps, M first, from U = V = 0).
 * These two calls are the half-steps' element-wise parts; the truncated SVD of the UV-step and the product U V are
 * left to a library (the Python package drives the loop, `lopa_approximation`).  All pointers are DEVICE memory.
 *
 * sffn_lopa_m_step: R = W - P (P [H,D] = U V, or NULL for the first step).  For every row i: g_idx[i] = column of the
 *   largest |R_ij| (the first one on ties), g_sign[i] = sign of that entry (+1 for an exact zero), row_best[i] =
 *   |R_ij| there, row_energy[i] = sum_j R_ij^2 (either may be NULL).  The objective after the step is
 *   sum_i (row_energy[i] - 2 row_best[i] + 1); called with W := W - M it also yields the objective after a UV-step.
 * sffn_lopa_residual: A = W - M, M[i, g_idx[i]] = g_sign[i]: the matrix whose truncated SVD at rank r is the best U V. */
int sffn_lopa_m_step(const float* W, const float* P, int H, int D, int32_t* g_idx, int8_t* g_sign, double* row_energy,
                     float* row_best, void* stream);
int sffn_lopa_residual(const float* W, const int32_t* g_idx, const int8_t* g_sign, int H, int D, float* A, void* stream);

/* Static string for a status code. */
const char* sffn_status_string(int status);

/* ---- test hooks ----------------------------------------------------------------------------------------------
 * Not steps of the paper's method: they let the tests look at launch geometry without a GPU and exercise the
 * device-side failure handling without ever hanging or faulting a GPU.  Process-wide, not thread-safe.
 *
 * sffn_test_fused_plan: geometry of the single-token CUDA-core kernel for a shape, as nine integers: ok, rows per
 *   gate slot, gate slot bytes, gate slots, gate warps, act slot bytes, act slots, chunks per act thread, shared
 *   memory bytes (wkind: 0 fp32, 1 bf16, 2 int8 rows).  sffn_test_umma_tiling: tiling of the batched gate GEMM.
 * sffn_test_set_knob(knob, value):
 *   PDL                 programmatic dependent launch between calls (default 1)
 *   TENSOR_GATE         1 / 0: single-token calls take the tensor-core gate kernel wherever it applies / nowhere,
 *                       whatever sffn_set_gate_engine said; -1 (the default): the handle's engine decides
 *   WAIT_CYCLES         budget of every device-side wait in clock cycles (default 2^31, about a second; 0 restores it)
 *   SKIP_ARRIVAL_CTA    index of a CTA of the single-token kernels that neither reports itself finished nor hands in
 *                       its partial result, so that the CTAs which sum the partials see their (bounded) wait run out
 *                       and record SFFN_ERR_TIMEOUT (-1 = none, the default; use it with a small WAIT_CYCLES)
 *   DROP_STAGE          index of a stage of the batched gate kernel whose weight copy CTA 0 leaves out, so that the wait
 *                       for it runs out and the kernel winds down and releases its TMEM columns (-1 = none, the default)
 *   RING_GATE_SLOTS, RING_ACT_SLOTS, RING_PARKED_STAGES
 *                       tensor-core gate kernel: split of its shared-memory rings and the number of gate stages it
 *                       prefetches into idle act slots at the start of a call (0, 0, -1 = planned)
 *   L2_HINTS            tensor-core gate kernel: bit 0 = weights are fetched evict-first, bit 1 = the per-CTA partial
 *                       results are stored evict-last (default 2)
 *   POISON_LIST         debug builds (-DSFFN_DEBUG) only, SFFN_ERR_UNSUPPORTED otherwise: 1 = the CUDA-core path
 *                       overwrites the first entry of its list of fired neurons with a number far beyond H before
 *                       the up / down kernel reads it, so that the kernel's index check has something to find (it
 *                       records SFFN_ERR_BOUNDS and takes row 0 instead; the bad index is never used as an address)
 *   TRACE_BUFFER        device address of [grid][16] int64 time stamps, written only by libraries built with
 *                       -DSFFN_TRACE (0 = none) */
typedef enum {
  SFFN_KNOB_PDL = 0, SFFN_KNOB_TENSOR_GATE = 1, SFFN_KNOB_WAIT_CYCLES = 2, SFFN_KNOB_SKIP_ARRIVAL_CTA = 3,
  SFFN_KNOB_RING_GATE_SLOTS = 4, SFFN_KNOB_RING_ACT_SLOTS = 5, SFFN_KNOB_TRACE_BUFFER = 6,
  SFFN_KNOB_RING_PARKED_STAGES = 7, SFFN_KNOB_L2_HINTS = 8, SFFN_KNOB_DROP_STAGE = 9, SFFN_KNOB_POISON_LIST = 10
} sffn_test_knob;
void sffn_test_fused_plan(int wkind, int D, int H, int K, int lopa, int sm_count, int* out9);
void sffn_test_umma_tiling(int R, int sm_count, int* tile_rows, int* n_tiles, int* own_list);
int sffn_test_set_knob(int knob, long long value);

#ifdef __cplusplus
}
#endif
#endif /* SPARSE_FFN_H_ */
