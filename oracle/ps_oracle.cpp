// CPU oracle for the ParallelSpec draft+verify path.  TEST INFRASTRUCTURE ONLY:
// it exists so that tests, the smoke check and the benchmark's cpu_baseline leg
// can compare the CUDA library against a plain restatement of the paper.  It is
// deliberately slow: fp64 arithmetic, no blocking, no fusion, no reordering,
// OpenMP over independent output rows only.  It shares no code with the CUDA
// path and must never be linked or imported by it.
//
// What each function follows:
//   pso_kv_append   Sec. 4.1 (masks of earlier groups are never visible, so only
//                   real positions persist) + Sec. 4.3 (fc over [embedding; feature])
//   pso_draft_step  Sec. 4.1 "Inference" (k [MASK] positions appended, k+1 rows
//                   decoded in one pass), Sec. 4.3 / Sec. 5.1 "Models" (one
//                   Transformer layer with the target layer's hyper-parameters,
//                   shared LM head), Algorithm 1 (the k+1 draft distributions)
//   pso_group_forward  Sec. 4.1 "Group-wise Parallel Training" (Fig. 3): the training layout of
//                   parallel groups with its attention mask and position indices, forward only
//   pso_verify      Eq. 1 and Algorithm 1 in its chain case (each node has one child)
//   pso_verify_tree Algorithm 1 in full: a token tree, children tried in turn, the
//                   target distribution replaced by its normalised residual after
//                   every rejection
//   pso_build_tree  Algorithm 1's drafting of the tree N and the appendix "Token Tree
//                   Verification": the candidates of a position are its highest-probability
//                   tokens; with a parallel drafter every node of one depth shares one row
//   pso_gumbel_sample  Algorithm 1's "sampling from the parallel draft model": one token per
//                   row drawn from softmax(logits/T) by the Gumbel-max rule with Philox uniforms
//   pso_philox4x32  Salmon et al., "Parallel random numbers: as easy as 1, 2, 3"
//                   (SC'11), Philox-4x32 with 10 rounds
//
// Pinned by tests/test_oracle_*.py: a library Llama decoder layer run unmasked
// over context + rows 0..j (draft layer, RoPE, norms, mask rule), the 4H^2+3HF
// parameter count of Sec. 5.1, Philox known-answer vectors, closed forms of
// Eq. 1 (acceptance probability = 1 - TV(p,q), emitted token ~ p), Monte-Carlo
// losslessness on a 16-token vocabulary, and the special cases p = q, disjoint
// supports and temperature 0.  The tree walk is pinned by its reduction to the chain
// routine on chain-shaped trees, by Monte-Carlo losslessness with several children per
// node drawn independently from q, and by the greedy longest-matching-path rule.
// Parity unpinned: the numeric logits of a *trained* drafter and the paper's
// acceptance lengths / speed-ups (they need weights and data the paper does not print).
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

struct Config {
  int dtype;  // 0 fp32, 1 bf16 (storage type of weights, hidden states and the KV cache)
  int hidden, n_heads, n_kv_heads, head_dim, ffn, vocab, k_masks;
  int max_batch, max_ctx;
  double rope_base, rms_eps;
  int has_fc_bias;
  int no_fc;  // embedding-only input (the Medusa integration of Sec. 4.3): x0 = the embedding half
};

struct Weights {
  const void *embed, *mask_embed, *mask_feat, *w_fc, *b_fc, *g_in;
  const void *w_q, *w_k, *w_v, *w_o, *g_post;
  const void *w_gate, *w_up, *w_down, *g_final, *w_lm;
};

// Optional taps: every intermediate tensor of one draft step, [k+1][width] doubles.
struct Taps {
  double *x_in, *x0, *xn, *q, *k_new, *v_new, *attn, *a, *an, *act, *hdn, *hn;
};

struct Ctx {
  Config c;
  Weights w;
  std::vector<int> len;               // committed real positions per slot
  std::vector<std::vector<double>> K; // [slot][max_ctx][n_kv_heads*head_dim], post-RoPE
  std::vector<std::vector<double>> V;
};

inline double widen(const void* p, size_t i, int dtype) {
  if (dtype == 0) return (double)((const float*)p)[i];
  uint32_t bits = (uint32_t)((const uint16_t*)p)[i] << 16;
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}

// Round to nearest-even bf16 and widen again: the value a bf16 cache slot holds.
inline double round_bf16(double x) {
  float f = (float)x;
  uint32_t b;
  std::memcpy(&b, &f, 4);
  if ((b & 0x7f800000u) == 0x7f800000u) return (double)f;  // inf / nan unchanged
  b += 0x7fffu + ((b >> 16) & 1u);
  b &= 0xffff0000u;
  std::memcpy(&f, &b, 4);
  return (double)f;
}

inline double store_round(double x, int dtype) {
  return dtype == 1 ? round_bf16(x) : (double)(float)x;
}

// y[n] = sum_k W[n][k] x[k] (+ bias[n]);  W is row-major [N][K] in the storage dtype.
void matvec(const void* W, const void* bias, int dtype, size_t N, size_t K, const double* x,
            double* y) {
#pragma omp parallel for schedule(static)
  for (long long n = 0; n < (long long)N; ++n) {
    double acc = 0.0;
    if (dtype == 0) {
      const float* w = (const float*)W + (size_t)n * K;
      for (size_t k = 0; k < K; ++k) acc += (double)w[k] * x[k];
    } else {
      for (size_t k = 0; k < K; ++k) acc += widen(W, (size_t)n * K + k, 1) * x[k];
    }
    if (bias) acc += widen(bias, (size_t)n, dtype);
    y[n] = acc;
  }
}

// RMSNorm: x * g / sqrt(mean(x^2) + eps)
void rmsnorm(const double* x, const void* g, int dtype, size_t H, double eps, double* y) {
  double ss = 0.0;
  for (size_t i = 0; i < H; ++i) ss += x[i] * x[i];
  double inv = 1.0 / std::sqrt(ss / (double)H + eps);
  for (size_t i = 0; i < H; ++i) y[i] = x[i] * inv * widen(g, i, dtype);
}

// Rotary embedding of one head vector at absolute position pos: the pair
// (v[i], v[i + d/2]) is rotated by the angle pos * base^(-2i/d).
void rope(double* v, int d, long long pos, double base) {
  int half = d / 2;
  for (int i = 0; i < half; ++i) {
    double theta = (double)pos * std::pow(base, -2.0 * (double)i / (double)d);
    double c = std::cos(theta), s = std::sin(theta);
    double a = v[i], b = v[i + half];
    v[i] = a * c - b * s;
    v[i + half] = b * c + a * s;
  }
}

// fc over [embedding ; feature] followed by the pre-attention norm.
void fuse_and_norm(const Ctx& C, const double* x_in, double* x0, double* xn) {
  const Config& c = C.c;
  if (c.no_fc)
    for (int i = 0; i < c.hidden; ++i) x0[i] = x_in[i];
  else
    matvec(C.w.w_fc, c.has_fc_bias ? C.w.b_fc : nullptr, c.dtype, c.hidden, 2 * (size_t)c.hidden,
           x_in, x0);
  rmsnorm(x0, C.w.g_in, c.dtype, c.hidden, c.rms_eps, xn);
}

void fill_real_input(const Ctx& C, int token, const void* hidden, size_t row, double* x_in) {
  const Config& c = C.c;
  size_t H = c.hidden;
  for (size_t i = 0; i < H; ++i) x_in[i] = widen(C.w.embed, (size_t)token * H + i, c.dtype);
  for (size_t i = 0; i < H; ++i) x_in[H + i] = widen(hidden, row * H + i, c.dtype);
}

void project_kv(const Ctx& C, const double* xn, long long pos, double* k_out, double* v_out) {
  const Config& c = C.c;
  size_t Hkv = (size_t)c.n_kv_heads * c.head_dim;
  matvec(C.w.w_k, nullptr, c.dtype, Hkv, c.hidden, xn, k_out);
  matvec(C.w.w_v, nullptr, c.dtype, Hkv, c.hidden, xn, v_out);
  for (int h = 0; h < c.n_kv_heads; ++h) rope(k_out + (size_t)h * c.head_dim, c.head_dim, pos, c.rope_base);
  for (size_t i = 0; i < Hkv; ++i) {
    k_out[i] = store_round(k_out[i], c.dtype);
    v_out[i] = store_round(v_out[i], c.dtype);
  }
}

// ---------------------------------------------------------------- Philox-4x32-10
inline void mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
  uint64_t p = (uint64_t)a * (uint64_t)b;
  hi = (uint32_t)(p >> 32);
  lo = (uint32_t)p;
}

void philox4x32_10(const uint32_t key_in[2], const uint32_t ctr_in[4], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo(M0, c0, hi0, lo0);
    mulhilo(M1, c2, hi1, lo1);
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0;
    k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

inline double u24(uint32_t w) { return (double)(w >> 8) * (1.0 / 16777216.0); }

// Softmax statistics of logits/T for one row: zmax = max z, S = sum exp(z - zmax).
struct RowStat { double zmax, S; bool nonfinite; };

RowStat row_stat(const float* row, int V, double T) {
  RowStat s{-std::numeric_limits<double>::infinity(), 0.0, false};
  for (int v = 0; v < V; ++v) {
    double z = (double)row[v] / T;
    if (std::isnan(z) || z == std::numeric_limits<double>::infinity()) s.nonfinite = true;
    if (z > s.zmax) s.zmax = z;
  }
  if (s.nonfinite || !(s.zmax > -std::numeric_limits<double>::infinity())) {
    s.nonfinite = true;
    return s;
  }
  for (int v = 0; v < V; ++v) s.S += std::exp((double)row[v] / T - s.zmax);
  return s;
}

inline double prob(const float* row, int v, double T, const RowStat& s) {
  return std::exp((double)row[v] / T - s.zmax) / s.S;
}

// Arg-max with ties to the lower id; a NaN entry counts as -inf.
int argmax_row(const float* row, int V) {
  int best = 0;
  double bv = std::isnan(row[0]) ? -std::numeric_limits<double>::infinity() : (double)row[0];
  for (int v = 1; v < V; ++v) {
    double x = std::isnan(row[v]) ? -std::numeric_limits<double>::infinity() : (double)row[v];
    if (x > bv) { best = v; bv = x; }
  }
  return best;
}

// Inverse-CDF draw from unnormalised non-negative weights w[0..V): the first v whose
// running sum exceeds u*W; if rounding leaves none, the last v with positive weight.
// *margin receives the distance of u*W to the nearest running-sum boundary, over W.
// nb (optional) receives the positive-weight tokens next to the pick in the running sum:
// nb[0] the one before it, nb[1] the one after it (-1 if there is none) -- the only other
// tokens a draw whose sampling point sits on a boundary may land on.
int inverse_cdf(const std::vector<double>& w, double W, double u, double* margin, int* nb = nullptr) {
  double target = u * W, run = 0.0, best = std::numeric_limits<double>::infinity();
  int pick = -1, last_pos = -1;
  for (size_t v = 0; v < w.size(); ++v) {
    if (w[v] > 0.0) last_pos = (int)v;
    run += w[v];
    if (w[v] > 0.0 || v + 1 == w.size()) {
      double d = std::fabs(run - target);
      if (d < best) best = d;
    }
    if (pick < 0 && run > target) pick = (int)v;
  }
  if (pick < 0) pick = last_pos;
  if (margin) *margin = (W > 0.0) ? best / W : 0.0;
  if (nb) {
    nb[0] = nb[1] = -1;
    for (int v = pick - 1; v >= 0 && nb[0] < 0; --v) if (w[v] > 0.0) nb[0] = v;
    for (size_t v = (size_t)(pick + 1); pick >= 0 && v < w.size() && nb[1] < 0; ++v) if (w[v] > 0.0) nb[1] = (int)v;
  }
  return pick;
}

}  // namespace

extern "C" {

// Threads the row loops use (for reporting next to timings).
int pso_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Sets the number of threads the row loops use from now on (timing on one core and on all).
void pso_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

void* pso_create(const Config* cfg, const Weights* w) {
  Ctx* C = new Ctx();
  C->c = *cfg;
  C->w = *w;
  C->len.assign(cfg->max_batch, 0);
  C->K.resize(cfg->max_batch);
  C->V.resize(cfg->max_batch);
  return C;
}

void pso_destroy(void* ctx) { delete (Ctx*)ctx; }

int pso_kv_len(void* ctx, int slot) { return ((Ctx*)ctx)->len[slot]; }

void pso_kv_reset(void* ctx, int slot) {
  Ctx* C = (Ctx*)ctx;
  C->len[slot] = 0;
}

static void ensure_slab(Ctx* C, int slot) {
  size_t n = (size_t)C->c.max_ctx * C->c.n_kv_heads * C->c.head_dim;
  if (C->K[slot].size() != n) {
    C->K[slot].assign(n, 0.0);
    C->V[slot].assign(n, 0.0);
  }
}

// Test helper: copy `len` cached rows ([len][n_kv_heads*head_dim], doubles) in or out.
int pso_kv_import(void* ctx, int slot, int len, const double* K, const double* V) {
  Ctx* C = (Ctx*)ctx;
  if (len > C->c.max_ctx) return -3;
  ensure_slab(C, slot);
  size_t n = (size_t)len * C->c.n_kv_heads * C->c.head_dim;
  for (size_t i = 0; i < n; ++i) {
    C->K[slot][i] = store_round(K[i], C->c.dtype);
    C->V[slot][i] = store_round(V[i], C->c.dtype);
  }
  C->len[slot] = len;
  return 0;
}

int pso_kv_export(void* ctx, int slot, double* K, double* V) {
  Ctx* C = (Ctx*)ctx;
  ensure_slab(C, slot);
  size_t n = (size_t)C->len[slot] * C->c.n_kv_heads * C->c.head_dim;
  std::memcpy(K, C->K[slot].data(), n * sizeof(double));
  std::memcpy(V, C->V[slot].data(), n * sizeof(double));
  return 0;
}

// Sec. 4.1 / 4.3: append n_new real (feature, token) pairs to the drafter's cache.
// Only real positions are ever cached; [MASK] rows of a draft step never are.
int pso_kv_append(void* ctx, int slot, int n_new, const void* hidden, const int* tokens) {
  Ctx* C = (Ctx*)ctx;
  const Config& c = C->c;
  if (C->len[slot] + n_new > c.max_ctx) return -3;
  ensure_slab(C, slot);
  size_t H = c.hidden, Hkv = (size_t)c.n_kv_heads * c.head_dim;
  std::vector<double> x_in(2 * H), x0(H), xn(H), kk(Hkv), vv(Hkv);
  for (int i = 0; i < n_new; ++i) {
    long long pos = C->len[slot] + i;
    fill_real_input(*C, tokens[i], hidden, (size_t)i, x_in.data());
    fuse_and_norm(*C, x_in.data(), x0.data(), xn.data());
    project_kv(*C, xn.data(), pos, kk.data(), vv.data());
    std::memcpy(&C->K[slot][(size_t)pos * Hkv], kk.data(), Hkv * sizeof(double));
    std::memcpy(&C->V[slot][(size_t)pos * Hkv], vv.data(), Hkv * sizeof(double));
  }
  C->len[slot] += n_new;
  return 0;
}

// Sec. 4.1 "Inference": one forward over the last real position plus k_use [MASK]
// positions.  Row 0 decodes x_t, row j decodes x_{t+j}.  Row j attends to the cached
// real positions and to new rows 0..j.  Does not change the committed cache length.
//   logits [k_use+1][V], feat [k_use+1][H] (the residual stream before the final norm)
int pso_draft_step(void* ctx, int slot, const void* hidden_last, int token_last, int k_use,
                   double* logits, double* feat, const Taps* taps) {
  Ctx* C = (Ctx*)ctx;
  const Config& c = C->c;
  if (k_use < 0 || k_use > c.k_masks) return -1;
  int R = k_use + 1, L = C->len[slot];
  if (L + R > c.max_ctx) return -3;
  ensure_slab(C, slot);
  size_t H = c.hidden, d = c.head_dim, Hq = (size_t)c.n_heads * d, Hkv = (size_t)c.n_kv_heads * d;
  size_t F = c.ffn, V = c.vocab;
  int group = c.n_heads / c.n_kv_heads;

  std::vector<double> x_in(R * 2 * H), x0(R * H), xn(R * H), q(R * Hq), kn(R * Hkv), vn(R * Hkv);
  std::vector<double> attn(R * Hq), a(R * H), an(R * H), gate(F), up(F), act(R * F), hdn(R * H),
      hn(R * H), tmp(H);

  for (int j = 0; j < R; ++j) {
    double* xi = &x_in[(size_t)j * 2 * H];
    if (j == 0) {
      fill_real_input(*C, token_last, hidden_last, 0, xi);
    } else {
      for (size_t i = 0; i < H; ++i) {
        xi[i] = widen(C->w.mask_embed, (size_t)(j - 1) * H + i, c.dtype);
        xi[H + i] = widen(C->w.mask_feat, (size_t)(j - 1) * H + i, c.dtype);
      }
    }
    fuse_and_norm(*C, xi, &x0[j * H], &xn[j * H]);
    matvec(C->w.w_q, nullptr, c.dtype, Hq, H, &xn[j * H], &q[j * Hq]);
    for (int h = 0; h < c.n_heads; ++h) rope(&q[j * Hq + h * d], (int)d, L + j, c.rope_base);
    project_kv(*C, &xn[j * H], L + j, &kn[j * Hkv], &vn[j * Hkv]);
  }

  // Attention under the parallel-draft mask.
  double scale = 1.0 / std::sqrt((double)d);
  for (int j = 0; j < R; ++j) {
    for (int h = 0; h < c.n_heads; ++h) {
      int hk = h / group;
      int n_keys = L + j + 1;
      std::vector<double> s(n_keys);
      const double* qv = &q[j * Hq + h * d];
      double smax = -std::numeric_limits<double>::infinity();
      for (int t = 0; t < n_keys; ++t) {
        const double* kv = (t < L) ? &C->K[slot][(size_t)t * Hkv + hk * d] : &kn[(size_t)(t - L) * Hkv + hk * d];
        double dot = 0.0;
        for (size_t i = 0; i < d; ++i) dot += qv[i] * kv[i];
        s[t] = dot * scale;
        if (s[t] > smax) smax = s[t];
      }
      double denom = 0.0;
      for (int t = 0; t < n_keys; ++t) { s[t] = std::exp(s[t] - smax); denom += s[t]; }
      double* o = &attn[j * Hq + h * d];
      for (size_t i = 0; i < d; ++i) o[i] = 0.0;
      for (int t = 0; t < n_keys; ++t) {
        const double* vv = (t < L) ? &C->V[slot][(size_t)t * Hkv + hk * d] : &vn[(size_t)(t - L) * Hkv + hk * d];
        double p = s[t] / denom;
        for (size_t i = 0; i < d; ++i) o[i] += p * vv[i];
      }
    }
  }

  for (int j = 0; j < R; ++j) {
    matvec(C->w.w_o, nullptr, c.dtype, H, Hq, &attn[j * Hq], tmp.data());
    for (size_t i = 0; i < H; ++i) a[j * H + i] = x0[j * H + i] + tmp[i];
    rmsnorm(&a[j * H], C->w.g_post, c.dtype, H, c.rms_eps, &an[j * H]);
    matvec(C->w.w_gate, nullptr, c.dtype, F, H, &an[j * H], gate.data());
    matvec(C->w.w_up, nullptr, c.dtype, F, H, &an[j * H], up.data());
    for (size_t i = 0; i < F; ++i) {
      double g = gate[i];
      act[j * F + i] = g / (1.0 + std::exp(-g)) * up[i];  // silu(gate) * up
    }
    matvec(C->w.w_down, nullptr, c.dtype, H, F, &act[j * F], tmp.data());
    for (size_t i = 0; i < H; ++i) hdn[j * H + i] = a[j * H + i] + tmp[i];
    rmsnorm(&hdn[j * H], C->w.g_final, c.dtype, H, c.rms_eps, &hn[j * H]);
    if (logits) matvec(C->w.w_lm, nullptr, c.dtype, V, H, &hn[j * H], &logits[(size_t)j * V]);
  }
  if (feat) std::memcpy(feat, hdn.data(), R * H * sizeof(double));
  if (taps) {
    auto cp = [](double* dst, const std::vector<double>& src) {
      if (dst) std::memcpy(dst, src.data(), src.size() * sizeof(double));
    };
    cp(taps->x_in, x_in); cp(taps->x0, x0); cp(taps->xn, xn); cp(taps->q, q);
    cp(taps->k_new, kn); cp(taps->v_new, vn); cp(taps->attn, attn); cp(taps->a, a);
    cp(taps->an, an); cp(taps->act, act); cp(taps->hdn, hdn); cp(taps->hn, hn);
  }
  return 0;
}

// Sec. 4.1 "Group-wise Parallel Training" (Fig. 3), forward only.  The source sequence is n
// parallel groups; group t is the real pair (tokens[t], hidden[t]) followed by the k [MASK]
// positions.  Row (t, j) has position index L + t + j (L = committed length of the slot: the
// cached prefix) and attends to the cached positions, to the REAL rows of the groups 0..t and
// to the [MASK] rows 1..j of its own group: never to a [MASK] row of another group.
//   logits [n][k+1][V], feat [n][k+1][H].  Leaves the cache as it was.
int pso_group_forward(void* ctx, int slot, int n, const void* hidden, const int* tokens, double* logits,
                      double* feat) {
  Ctx* C = (Ctx*)ctx;
  const Config& c = C->c;
  const int R = c.k_masks + 1, L = C->len[slot];
  if (n < 1 || L + n + c.k_masks > c.max_ctx) return -3;
  ensure_slab(C, slot);
  const size_t H = c.hidden, d = c.head_dim, Hq = (size_t)c.n_heads * d, Hkv = (size_t)c.n_kv_heads * d;
  const size_t F = c.ffn, V = c.vocab, M = (size_t)n * R;
  const int group = c.n_heads / c.n_kv_heads;
  std::vector<double> x_in(2 * H), x0(M * H), xn(H), q(M * Hq), kn(M * Hkv), vn(M * Hkv), attn(M * Hq);
  for (int t = 0; t < n; ++t) {
    for (int j = 0; j < R; ++j) {
      const size_t r = (size_t)t * R + j;
      if (j == 0) {
        fill_real_input(*C, tokens[t], hidden, (size_t)t, x_in.data());
      } else {
        for (size_t i = 0; i < H; ++i) {
          x_in[i] = widen(C->w.mask_embed, (size_t)(j - 1) * H + i, c.dtype);
          x_in[H + i] = widen(C->w.mask_feat, (size_t)(j - 1) * H + i, c.dtype);
        }
      }
      fuse_and_norm(*C, x_in.data(), &x0[r * H], xn.data());
      matvec(C->w.w_q, nullptr, c.dtype, Hq, H, xn.data(), &q[r * Hq]);
      for (int h = 0; h < c.n_heads; ++h) rope(&q[r * Hq + h * d], (int)d, L + t + j, c.rope_base);
      project_kv(*C, xn.data(), L + t + j, &kn[r * Hkv], &vn[r * Hkv]);
    }
  }
  const double scale = 1.0 / std::sqrt((double)d);
  for (int t = 0; t < n; ++t) {
    for (int j = 0; j < R; ++j) {
      const size_t r = (size_t)t * R + j;
      // the keys row (t, j) may see, as (source, index): cache rows, real rows, own [MASK] rows
      std::vector<const double*> K, Vv;
      for (int h = 0; h < c.n_heads; ++h) {
        const int hk = h / group;
        K.clear(); Vv.clear();
        for (int p = 0; p < L; ++p) {
          K.push_back(&C->K[slot][(size_t)p * Hkv + hk * d]);
          Vv.push_back(&C->V[slot][(size_t)p * Hkv + hk * d]);
        }
        for (int g = 0; g <= t; ++g) {
          K.push_back(&kn[((size_t)g * R) * Hkv + hk * d]);
          Vv.push_back(&vn[((size_t)g * R) * Hkv + hk * d]);
        }
        for (int jj = 1; jj <= j; ++jj) {
          K.push_back(&kn[((size_t)t * R + jj) * Hkv + hk * d]);
          Vv.push_back(&vn[((size_t)t * R + jj) * Hkv + hk * d]);
        }
        const double* qv = &q[r * Hq + h * d];
        std::vector<double> sc(K.size());
        double smax = -std::numeric_limits<double>::infinity();
        for (size_t u = 0; u < K.size(); ++u) {
          double dot = 0.0;
          for (size_t i = 0; i < d; ++i) dot += qv[i] * K[u][i];
          sc[u] = dot * scale;
          if (sc[u] > smax) smax = sc[u];
        }
        double denom = 0.0;
        for (size_t u = 0; u < K.size(); ++u) { sc[u] = std::exp(sc[u] - smax); denom += sc[u]; }
        double* o = &attn[r * Hq + h * d];
        for (size_t i = 0; i < d; ++i) o[i] = 0.0;
        for (size_t u = 0; u < K.size(); ++u) {
          const double pw = sc[u] / denom;
          for (size_t i = 0; i < d; ++i) o[i] += pw * Vv[u][i];
        }
      }
    }
  }
  std::vector<double> a(H), an(H), gate(F), up(F), act(F), hdn(H), hn(H), tmp(H);
  for (size_t r = 0; r < M; ++r) {
    matvec(C->w.w_o, nullptr, c.dtype, H, Hq, &attn[r * Hq], tmp.data());
    for (size_t i = 0; i < H; ++i) a[i] = x0[r * H + i] + tmp[i];
    rmsnorm(a.data(), C->w.g_post, c.dtype, H, c.rms_eps, an.data());
    matvec(C->w.w_gate, nullptr, c.dtype, F, H, an.data(), gate.data());
    matvec(C->w.w_up, nullptr, c.dtype, F, H, an.data(), up.data());
    for (size_t i = 0; i < F; ++i) act[i] = gate[i] / (1.0 + std::exp(-gate[i])) * up[i];
    matvec(C->w.w_down, nullptr, c.dtype, H, F, act.data(), tmp.data());
    for (size_t i = 0; i < H; ++i) hdn[i] = a[i] + tmp[i];
    if (feat) std::memcpy(feat + r * H, hdn.data(), H * sizeof(double));
    rmsnorm(hdn.data(), C->w.g_final, c.dtype, H, c.rms_eps, hn.data());
    if (logits) matvec(C->w.w_lm, nullptr, c.dtype, V, H, hn.data(), &logits[r * V]);
  }
  return 0;
}

// Row statistics the LM-head stage reports: max, log-sum-exp and the top_n entries
// (descending logit, ties to the lower id) of each of n_rows rows of V doubles.
void pso_row_stats(const double* logits, int n_rows, int V, int top_n, double* row_max,
                   double* row_lse, int* top_ids, double* top_logit) {
  for (int r = 0; r < n_rows; ++r) {
    const double* row = logits + (size_t)r * V;
    double m = row[0];
    for (int v = 1; v < V; ++v) if (row[v] > m) m = row[v];
    double s = 0.0;
    for (int v = 0; v < V; ++v) s += std::exp(row[v] - m);
    row_max[r] = m;
    row_lse[r] = m + std::log(s);
    std::vector<char> used(V, 0);
    for (int t = 0; t < top_n; ++t) {
      int best = -1;
      for (int v = 0; v < V; ++v)
        if (!used[v] && (best < 0 || row[v] > row[best])) best = v;
      used[best] = 1;
      top_ids[r * top_n + t] = best;
      top_logit[r * top_n + t] = row[best];
    }
  }
}

void pso_philox4x32(const uint32_t* key, const uint32_t* ctr, uint32_t* out) {
  philox4x32_10(key, ctr, out);
}

// The two uniforms of decision i of sequence b: key = seed, counter = (i, b, offset).
void pso_uniforms(uint64_t seed, uint64_t offset, int b, int i, double* r, double* u2) {
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t ctr[4] = {(uint32_t)i, (uint32_t)b, (uint32_t)offset, (uint32_t)(offset >> 32)};
  uint32_t o[4];
  philox4x32_10(key, ctr, o);
  *r = u24(o[0]);
  *u2 = u24(o[1]);
}

// Eq. 1 / Algorithm 1, chain case, for B independent sequences.
//   draft_tokens [B][n_draft]; draft_logits [B][n_draft][V] or NULL (q is then the
//   point mass on the drafted token); target_logits [B][n_target][V], n_target is
//   n_draft or n_draft+1.  temperature 0 = greedy.
// Outputs: accept_len[B]; out_tokens[B][n_draft+1] (-1 = unused); n_out[B];
//   margin_accept[B][n_draft] = |r - min(1,p/q)| at each examined position (inf if not
//   examined or T=0); margin_cdf[B] = distance of the sampling point to the nearest CDF
//   boundary, as a fraction of the total weight (inf if nothing was sampled);
//   nonfinite[B] = 1 if a NaN/+inf logit was met; neighbours[B][2] (optional) = the
//   positive-weight tokens before / after the sampled one in the running sum (-1: none).
int pso_verify(int B, int n_draft, int n_target, int V, const int* draft_tokens,
               const float* draft_logits, const float* target_logits, double temperature,
               uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
               double* margin_accept, double* margin_cdf, int* nonfinite, int* neighbours) {
  if (n_target != n_draft && n_target != n_draft + 1) return -1;
  const double INF = std::numeric_limits<double>::infinity();
#pragma omp parallel for schedule(dynamic, 64)
  for (int b = 0; b < B; ++b) {
    int* out = out_tokens + (size_t)b * (n_draft + 1);
    for (int i = 0; i <= n_draft; ++i) out[i] = -1;
    if (margin_accept) for (int i = 0; i < n_draft; ++i) margin_accept[(size_t)b * n_draft + i] = INF;
    if (margin_cdf) margin_cdf[b] = INF;
    int nbr[2] = {-1, -1};
    int bad = 0, a = 0, emitted = -1;
    bool stopped = false;
    for (int i = 0; i < n_draft && !stopped; ++i) {
      const float* t = target_logits + ((size_t)b * n_target + i) * V;
      const float* dl = draft_logits ? draft_logits + ((size_t)b * n_draft + i) * V : nullptr;
      int x = draft_tokens[(size_t)b * n_draft + i];
      if (temperature == 0.0) {
        int tstar = argmax_row(t, V);
        if (x == tstar) { out[a++] = x; continue; }
        emitted = tstar; stopped = true; break;
      }
      double r, u2;
      pso_uniforms(seed, offset, b, i, &r, &u2);
      RowStat st = row_stat(t, V, temperature);
      RowStat sd{0.0, 1.0, false};
      if (dl) sd = row_stat(dl, V, temperature);
      bool accept;
      if (st.nonfinite || sd.nonfinite) {
        bad = 1; accept = false;
      } else {
        double logp = (double)t[x] / temperature - st.zmax - std::log(st.S);
        double logq = dl ? (double)dl[x] / temperature - sd.zmax - std::log(sd.S) : 0.0;
        double diff = logp - logq;           // -inf - (-inf) = NaN -> reject
        double ratio = std::exp(diff < 0.0 ? diff : 0.0);
        if (std::isnan(diff)) { ratio = 0.0; }
        accept = r < ratio;
        if (margin_accept) margin_accept[(size_t)b * n_draft + i] = std::fabs(r - ratio);
      }
      if (accept) { out[a++] = x; continue; }
      // rejection: sample from norm(max(0, p - q))
      std::vector<double> w(V, 0.0);
      double W = 0.0;
      if (!st.nonfinite && !sd.nonfinite) {
        for (int v = 0; v < V; ++v) {
          double pv = prob(t, v, temperature, st);
          double qv = dl ? prob(dl, v, temperature, sd) : (v == x ? 1.0 : 0.0);
          double wv = pv - qv;
          w[v] = wv > 0.0 ? wv : 0.0;
          W += w[v];
        }
        if (!(W > 0.0)) {
          W = 0.0;
          for (int v = 0; v < V; ++v) { w[v] = prob(t, v, temperature, st); W += w[v]; }
        }
        double mg;
        emitted = inverse_cdf(w, W, u2, &mg, nbr);
        if (margin_cdf) margin_cdf[b] = mg;
      } else {
        emitted = argmax_row(t, V);  // defined fallback for poisoned rows
      }
      stopped = true;
    }
    if (!stopped && n_target == n_draft + 1) {
      const float* t = target_logits + ((size_t)b * n_target + n_draft) * V;
      if (temperature == 0.0) {
        emitted = argmax_row(t, V);
      } else {
        double r, u2;
        pso_uniforms(seed, offset, b, n_draft, &r, &u2);
        RowStat st = row_stat(t, V, temperature);
        if (st.nonfinite) { bad = 1; emitted = argmax_row(t, V); }
        else {
          std::vector<double> w(V);
          double W = 0.0;
          for (int v = 0; v < V; ++v) { w[v] = prob(t, v, temperature, st); W += w[v]; }
          double mg;
          emitted = inverse_cdf(w, W, u2, &mg, nbr);
          if (margin_cdf) margin_cdf[b] = mg;
        }
      }
    }
    accept_len[b] = a;
    int n = a;
    if (emitted >= 0) out[n++] = emitted;
    n_out[b] = n;
    if (nonfinite) nonfinite[b] = bad;
    if (neighbours) { neighbours[2 * b] = nbr[0]; neighbours[2 * b + 1] = nbr[1]; }
  }
  return 0;
}

// One token per row from softmax(logits[r] / T) by the Gumbel-max rule: the arg-max over v of
// logits[r][v] / T + G, G = -ln(-ln u), u = ((w >> 8) + 0.5) / 2^24 with w = word 0 of
// Philox-4x32-10, key = (seed_lo ^ 0x6D756247, seed_hi), counter = (v, row_id[r], offset).
// Ties go to the lower id.  margin[r] = best perturbed value minus the runner-up.
int pso_gumbel_sample(const double* logits, int n_rows, int V, double temperature, uint64_t seed,
                      uint64_t offset, const int* row_id, int* tokens, double* margin) {
  if (!(temperature > 0.0)) return -1;
  uint32_t key[2] = {(uint32_t)seed ^ 0x6D756247u, (uint32_t)(seed >> 32)};
  for (int r = 0; r < n_rows; ++r) {
    const double* row = logits + (size_t)r * V;
    double best = -std::numeric_limits<double>::infinity(), second = best;
    int arg = -1;
    for (int v = 0; v < V; ++v) {
      uint32_t ctr[4] = {(uint32_t)v, (uint32_t)row_id[r], (uint32_t)offset, (uint32_t)(offset >> 32)};
      uint32_t o[4];
      philox4x32_10(key, ctr, o);
      const double u = ((double)(o[0] >> 8) + 0.5) / 16777216.0;
      const double y = row[v] / temperature - std::log(-std::log(u));
      if (y > best) { second = best; best = y; arg = v; }
      else if (y > second) second = y;
    }
    tokens[r] = arg;
    if (margin) margin[r] = best - second;
  }
  return 0;
}

// The draft tree of Algorithm 1 for a static shape (appendix "Token Tree Verification": each
// position's candidates are its most probable tokens).  The parallel drafter yields one
// distribution per depth, so node i at depth t carries the rank[i]-th entry of that depth's
// top-n list; when sampled tokens are given, rank 0 carries the sampled token of the depth and a
// deeper rank whose entry is that very token carries entry 0 instead.
//   parent[n_nodes] (-1: child of the root), rank[n_nodes], top_ids [B][R][top_n] (R rows per
//   sequence), sampled [B][R] or NULL  ->  tokens [B][n_nodes].  Returns -1 for a bad tree.
int pso_build_tree(int B, int n_nodes, int R, int top_n, const int* parent, const int* rank, const int* top_ids,
                   const int* sampled, int* tokens) {
  std::vector<int> depth(n_nodes);
  for (int i = 0; i < n_nodes; ++i) {
    if (parent[i] >= i || parent[i] < -1) return -1;
    depth[i] = parent[i] < 0 ? 0 : depth[parent[i]] + 1;
    if (depth[i] >= R || rank[i] < 0 || rank[i] >= top_n) return -1;
  }
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < n_nodes; ++i) {
      const int* list = top_ids + ((size_t)b * R + depth[i]) * top_n;
      int tok = list[rank[i]];
      if (sampled) {
        const int sx = sampled[(size_t)b * R + depth[i]];
        if (rank[i] == 0) tok = sx;
        else if (tok == sx) tok = list[0];
      }
      tokens[(size_t)b * n_nodes + i] = tok;
    }
  return 0;
}

// Algorithm 1 in full, for B independent sequences that share one tree shape.
//   parent[n_nodes]: parent node of node i (< i), -1 for the children of the root.  The
//   children of a node are tried in increasing node id (the Select order).  A child of the
//   root has depth 0, a child of node i depth(i) + 1; all nodes of depth t were drafted
//   from the same distribution q_t = softmax(draft_logits[b][t] / T) (the parallel drafter
//   gives one distribution per depth).  tokens [B][n_nodes].  target_logits
//   [B][n_nodes+1][V]: row 0 is the target distribution after the prefix, row 1+i the one
//   after the path that ends in node i.  Decision row u (0 or 1+i) draws r for its j-th
//   child from the Philox counter (u + (j << 16), b, offset), word 0, and its final sample
//   from word 1 of the counter (u, b, offset): a chain-shaped tree then uses exactly the
//   uniforms of pso_verify.
// Outputs: accept_len[B] accepted nodes; path[B][max_depth] their ids (-1 unused);
//   out_tokens[B][max_depth+1] their tokens followed by the token sampled at the node where
//   the walk stopped (-1 unused); n_out[B] = accept_len + 1; margin_accept[B] = the smallest
//   |r - min(1, p/q)| over the tests made; margin_cdf[B], neighbours[B][2] (optional) as in
//   pso_verify; nonfinite[B].
int pso_verify_tree(int B, int n_nodes, int max_depth, int V, const int* parent, const int* tokens,
                    const float* draft_logits, const float* target_logits, double temperature,
                    uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
                    int* path, double* margin_accept, double* margin_cdf, int* nonfinite, int* neighbours) {
  const double INF = std::numeric_limits<double>::infinity();
  std::vector<int> depth(n_nodes);
  for (int i = 0; i < n_nodes; ++i) {
    if (parent[i] >= i || parent[i] < -1) return -1;
    depth[i] = parent[i] < 0 ? 0 : depth[parent[i]] + 1;
    if (depth[i] >= max_depth) return -1;
  }
  if (temperature != 0.0 && !draft_logits) return -1;
#pragma omp parallel for schedule(dynamic, 16)
  for (int b = 0; b < B; ++b) {
    int* out = out_tokens + (size_t)b * (max_depth + 1);
    int* pth = path + (size_t)b * max_depth;
    for (int i = 0; i <= max_depth; ++i) out[i] = -1;
    for (int i = 0; i < max_depth; ++i) pth[i] = -1;
    double m_acc = INF, m_cdf = INF;
    int nbr[2] = {-1, -1};
    int bad = 0, a = 0, emitted = -1;
    int u = 0;                                   // decision row: 0 = root, 1 + node id
    std::vector<double> p(V), q(V);
    for (;;) {
      const float* t = target_logits + ((size_t)b * (n_nodes + 1) + u) * V;
      std::vector<int> H;                        // children of u, in Select order
      for (int i = 0; i < n_nodes; ++i)
        if (parent[i] == u - 1) H.push_back(i);
      const int d = u == 0 ? 0 : depth[u - 1] + 1;   // depth of the children
      if (temperature == 0.0) {
        int tstar = argmax_row(t, V), next = -1;
        for (int c : H)
          if (tokens[(size_t)b * n_nodes + c] == tstar) { next = c; break; }
        if (next < 0) { emitted = tstar; break; }
        out[a] = tstar; pth[a] = next; ++a; u = next + 1;
        continue;
      }
      RowStat st = row_stat(t, V, temperature);
      if (st.nonfinite) { bad = 1; emitted = argmax_row(t, V); break; }
      for (int v = 0; v < V; ++v) p[v] = prob(t, v, temperature, st);
      std::vector<double> p0 = p;
      int next = -1;
      if (!H.empty()) {
        const float* dl = draft_logits + ((size_t)b * max_depth + d) * V;
        RowStat sd = row_stat(dl, V, temperature);
        if (sd.nonfinite) { bad = 1; emitted = argmax_row(t, V); break; }
        for (int v = 0; v < V; ++v) q[v] = prob(dl, v, temperature, sd);
        for (size_t j = 0; j < H.size(); ++j) {
          const int x = tokens[(size_t)b * n_nodes + H[j]];
          double r, unused;
          pso_uniforms(seed, offset, b, u + (int)(j << 16), &r, &unused);
          double ratio;
          if (x < 0 || x >= V) ratio = 0.0;
          else if (q[x] > 0.0) ratio = p[x] / q[x] < 1.0 ? p[x] / q[x] : 1.0;
          else ratio = p[x] > 0.0 ? 1.0 : 0.0;
          if (std::fabs(r - ratio) < m_acc) m_acc = std::fabs(r - ratio);
          if (r < ratio) { next = H[j]; break; }
          // rejected: p := norm((p - q)+)
          double W = 0.0;
          for (int v = 0; v < V; ++v) { p[v] = p[v] > q[v] ? p[v] - q[v] : 0.0; W += p[v]; }
          if (W > 0.0) for (int v = 0; v < V; ++v) p[v] /= W;
          else { p = p0; }   // nothing left of the residual: fall back to the node's own p
        }
      }
      if (next >= 0) {
        out[a] = tokens[(size_t)b * n_nodes + next]; pth[a] = next; ++a; u = next + 1;
        continue;
      }
      double r_unused, u2, W = 0.0;
      pso_uniforms(seed, offset, b, u, &r_unused, &u2);
      for (int v = 0; v < V; ++v) W += p[v];
      emitted = inverse_cdf(p, W, u2, &m_cdf, nbr);
      break;
    }
    accept_len[b] = a;
    out[a] = emitted;
    n_out[b] = a + 1;
    if (margin_accept) margin_accept[b] = m_acc;
    if (margin_cdf) margin_cdf[b] = m_cdf;
    if (nonfinite) nonfinite[b] = bad;
    if (neighbours) { neighbours[2 * b] = nbr[0]; neighbours[2 * b + 1] = nbr[1]; }
  }
  return 0;
}

}  // extern "C"
