// CPU oracle for the activation-sparse gated FFN.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain definition that the CUDA library is checked
// against.  It shares no code with the CUDA path, is never linked into it and
// must never be called from it: only the tests, the smoke check and the
// benchmark's CPU-baseline legs may load it.
//
// What it computes (paper Sec. 3.1, Eq. 1, with W_2 stored transposed):
//     z = W_1 x + b_g                       gate pre-activation
//     a = A(z)                              activation table of Sec. 3.1
//     u = W_3 x
//     y = W_2 (a . u)       i.e.  y[d] = sum_j a_j u_j W_down[j, d]
// and, for the low-parameter gate (Sec. 3.3, Eq. 3 and "LoPA in practice"):
//     z = G x + U RMSNorm(V x) + b_g        (RMSNorm optional: Sec. 3.4 drops it)
// Sparse execution (Sec. 3.1, "FFN FLOP-ratio"): a zero of the gate output is
// known before W_3 and W_2 are touched, so row j of W_3 and column j of W_2 are
// skipped when a_j = 0.  The skipped terms are exact zeros, hence both routes
// give the same y; the oracle implements both so that their agreement is a test.
//
// Every sum is accumulated in double, in ascending index order, with no
// blocking, fusion or reordering.  bf16 / fp32 inputs are decoded exactly.
//
// Parity pins: tests/test_oracle_*.py (hand-worked examples, activation table,
// brute-force active sets, dense == sparse, 0 % / 100 % sparsity, LoPA against
// the materialised G + UV, the H=12, D=6 picture of the fixed matrices).
// Unpinned: absolute values of y on the full-size synthetic configs (the paper
// prints no worked output); they rest on the pins above and on this code being
// size-generic.

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

enum DType { F32 = 0, BF16 = 1, F64 = 2 };
enum Act { RELU = 0, SQRELU = 1, RSPLUS = 2, SILU = 3 };

// Exact decode of one stored element to double.
inline double load(const void* p, int dtype, size_t i) {
  switch (dtype) {
    case F32:
      return static_cast<double>(static_cast<const float*>(p)[i]);
    case BF16: {
      uint32_t bits = static_cast<uint32_t>(static_cast<const uint16_t*>(p)[i]) << 16;
      float f;
      std::memcpy(&f, &bits, sizeof f);
      return static_cast<double>(f);
    }
    default:
      return static_cast<const double*>(p)[i];
  }
}

// Activation table of Sec. 3.1 (RELU, SILU, R-S+) plus squared RELU (Sec. 5, other activations).  SILU is not
// sparse; it only ever serves as A_3 on the up projection (Sec. 3.3, "Double activation": the activation of W_1
// alone is cast, the other one stays what the model was trained with).
inline double activation(int act, double z) {
  if (act == SILU) return z / (1.0 + std::exp(-z));  // z * sigmoid(z) on both sides
  if (!(z > 0.0)) return 0.0;  // z <= 0 (and -0) give exactly 0 for the three sparse activations
  switch (act) {
    case RELU:
      return z;
    case SQRELU:
      return z * z;
    default:  // R-S+: z * sigmoid(z) on the non-negative side
      return z / (1.0 + std::exp(-z));
  }
}

}  // namespace

extern "C" {

// a = A(z) for one value; exported so the activation table can be pinned directly.
double oracle_activation(int act, double z) { return activation(act, z); }

// Standard gate, Eq. 1:  z_j = b_g[j] + sum_d W_1[j,d] x[d].   b_g may be NULL (paper's form).
void oracle_gate_standard(const void* W1, int wdtype, const void* x, int xdtype, const float* b_g,
                          int H, int D, double* z) {
  for (int j = 0; j < H; ++j) {
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += load(W1, wdtype, (size_t)j * D + d) * load(x, xdtype, d);
    z[j] = acc + (b_g ? (double)b_g[j] : 0.0);
  }
}

// LoPA gate, Eq. 3 / "LoPA in practice":
//   v_k = sum_d V[k,d] x[d]
//   n_k = gamma_k v_k / sqrt(mean_k(v_k^2) + eps)      if use_rmsnorm, else n_k = v_k
//   z_j = b_g[j] + sign_j x[g_idx[j]] + sum_k U[j,k] n_k
// g_idx NULL drops the fixed matrix (W_1 = UV); g_sign NULL means +1; gamma NULL means 1.
// v_out / n_out (each [r]) may be NULL.
void oracle_gate_lopa(const void* V, const void* U, int wdtype, const int32_t* g_idx,
                      const int8_t* g_sign, const float* gamma, int use_rmsnorm, double eps, int r,
                      const void* x, int xdtype, const float* b_g, int H, int D, double* z,
                      double* v_out, double* n_out) {
  std::vector<double> v(r), n(r);
  for (int k = 0; k < r; ++k) {
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += load(V, wdtype, (size_t)k * D + d) * load(x, xdtype, d);
    v[k] = acc;
  }
  if (use_rmsnorm) {
    double ss = 0.0;
    for (int k = 0; k < r; ++k) ss += v[k] * v[k];
    const double rms = std::sqrt(ss / (double)r + eps);
    for (int k = 0; k < r; ++k) n[k] = (gamma ? (double)gamma[k] : 1.0) * v[k] / rms;
  } else {
    for (int k = 0; k < r; ++k) n[k] = v[k];
  }
  for (int j = 0; j < H; ++j) {
    double acc = 0.0;
    for (int k = 0; k < r; ++k) acc += load(U, wdtype, (size_t)j * r + k) * n[k];
    double fixed = 0.0;
    if (g_idx) fixed = (g_sign ? (double)g_sign[j] : 1.0) * load(x, xdtype, (size_t)g_idx[j]);
    z[j] = acc + fixed + (b_g ? (double)b_g[j] : 0.0);
  }
  if (v_out) std::memcpy(v_out, v.data(), sizeof(double) * r);
  if (n_out) std::memcpy(n_out, n.data(), sizeof(double) * r);
}

// Active set S = { j : A(z_j) != 0 } = { j : z_j > 0 }, ascending.  Returns |S|.
int oracle_active_set(const double* z, int H, int32_t* idx) {
  int n = 0;
  for (int j = 0; j < H; ++j)
    if (z[j] > 0.0) idx[n++] = j;
  return n;
}

// Up projection, scaling and down projection for one token, given z.
//   route 0 (dense):  every j in 0..H-1           (Eq. 1 as written)
//   route 1 (sparse): only j with z_j > 0         (Sec. 3.1 skipping rule)
// W_down is W_2 transposed, [H, D] row-major.  y is [D] double.  Returns rows of W_3 touched.
// Double activation (Sec. 3.3, "Double activation"): with act_up >= 0 the activation A_3 = act_up is
// applied to the output of W_3 as well, h_j = A(z_j) * A_3(u_j); act_up < 0 is Eq. 1 as written.
// *n_gated (may be NULL) counts the j with h_j != 0, the "s_gated" site of the sparsity-sites table:
// rows of W_2 whose contribution is not identically zero.
int oracle_updown(const double* z, int act, int act_up, const void* W3, const void* Wdown, int wdtype,
                  const void* x, int xdtype, int H, int D, int route, double* y, int* n_gated) {
  for (int d = 0; d < D; ++d) y[d] = 0.0;
  int touched = 0, gated = 0;
  for (int j = 0; j < H; ++j) {
    if (route == 1 && !(z[j] > 0.0)) continue;
    ++touched;
    const double a = activation(act, z[j]);
    double u = 0.0;
    for (int d = 0; d < D; ++d) u += load(W3, wdtype, (size_t)j * D + d) * load(x, xdtype, d);
    const double h = a * (act_up >= 0 ? activation(act_up, u) : u);
    gated += h != 0.0;
    for (int d = 0; d < D; ++d) y[d] += h * load(Wdown, wdtype, (size_t)j * D + d);
  }
  if (n_gated) *n_gated = gated;
  return touched;
}

// Whole FFN for a batch of B independent tokens (a batch is B separate FFNs; Sec. 5.4 only adds
// that rows must be loaded for the union of the tokens' active sets).
//   gate_kind 0: standard (W1 used);  1: LoPA (V, U, g_idx, g_sign, gamma, use_rmsnorm, eps, r used)
//   act_up < 0: Eq. 1; >= 0: double activation with A_3 = act_up (see oracle_updown);
//   x [B,D];  y [B,D] double;  z_out [B,H] double or NULL;  n_act_out, n_gated_out [B] or NULL;
//   union_mask [H] bytes or NULL (1 where any token fires).
// threads > 1 splits the tokens over OpenMP threads; the arithmetic per token is unchanged.
// Returns 0, or -1 on a bad argument.
int oracle_ffn_batch(int gate_kind, const void* W1, const void* V, const void* U,
                     const int32_t* g_idx, const int8_t* g_sign, const float* gamma,
                     int use_rmsnorm, double eps, int r, const float* b_g, const void* W3,
                     const void* Wdown, int wdtype, const void* x, int xdtype, int B, int H, int D,
                     int act, int act_up, int route, int threads, double* y, double* z_out,
                     int32_t* n_act_out, int32_t* n_gated_out, uint8_t* union_mask) {
  if (B < 0 || H <= 0 || D <= 0 || !W3 || !Wdown || !x || !y) return -1;
  if (gate_kind == 0 && !W1) return -1;
  if (gate_kind == 1 && (!V || !U || r <= 0)) return -1;
  if (act < RELU || act > RSPLUS || act_up > SILU) return -1;  // the gate's activation must be a sparse one
  if (union_mask) std::memset(union_mask, 0, (size_t)H);
  const size_t xstride = (size_t)D * (xdtype == F32 ? 4 : xdtype == BF16 ? 2 : 8);
  std::vector<int32_t> n_act(B > 0 ? B : 1), n_gated(B > 0 ? B : 1);
  std::vector<std::vector<uint8_t>> masks;
  if (union_mask) masks.assign(B, std::vector<uint8_t>());
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads > 1 ? threads : 1)
  for (int b = 0; b < B; ++b) {
    const void* xb = static_cast<const char*>(x) + (size_t)b * xstride;
    std::vector<double> z(H);
    if (gate_kind == 0)
      oracle_gate_standard(W1, wdtype, xb, xdtype, b_g, H, D, z.data());
    else
      oracle_gate_lopa(V, U, wdtype, g_idx, g_sign, gamma, use_rmsnorm, eps, r, xb, xdtype, b_g, H,
                       D, z.data(), nullptr, nullptr);
    int gated = 0;
    oracle_updown(z.data(), act, act_up, W3, Wdown, wdtype, xb, xdtype, H, D, route, y + (size_t)b * D, &gated);
    n_gated[b] = gated;
    int cnt = 0;
    for (int j = 0; j < H; ++j) cnt += z[j] > 0.0;
    n_act[b] = cnt;
    if (z_out) std::memcpy(z_out + (size_t)b * H, z.data(), sizeof(double) * H);
    if (union_mask) {
      masks[b].resize(H);
      for (int j = 0; j < H; ++j) masks[b][j] = z[j] > 0.0;
    }
  }
  for (int b = 0; b < B; ++b) {
    if (n_act_out) n_act_out[b] = n_act[b];
    if (n_gated_out) n_gated_out[b] = n_gated[b];
    if (union_mask)
      for (int j = 0; j < H; ++j) union_mask[j] |= masks[b][j];
  }
  return 0;
}

}  // extern "C"
