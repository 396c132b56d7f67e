// Unfused kernels with fp32 activations.  They cover every dtype and shape the library
// accepts and are the path for fp32 models; the fused bf16 kernels replace them stage by
// stage where they apply.  One kernel per step of the layer:
//   gather -> fc -> RMSNorm -> q,k,v -> RoPE + cache write -> attention -> o (+residual)
//   -> RMSNorm -> gate, up -> silu*up -> down (+residual) -> RMSNorm -> LM head -> row stats
// (Sec. 4.1 "Inference", Sec. 4.3, Sec. 5.1 "Models".)
#include <cfloat>

#include "ps_internal.cuh"

namespace ps {
namespace {

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_as(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_as(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// 8 consecutive weights as floats; p is 16-byte (bf16) / 32-byte (fp32) aligned.
__device__ __forceinline__ void load8(const float* p, float (&w)[8]) {
  float4 a = __ldg(reinterpret_cast<const float4*>(p));
  float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&w)[8]) {
  uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    w[2 * i] = __uint_as_float(u[i] << 16);
    w[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// S0: rows of the fc input.  Row j = 0 of a sequence: [embed[token] ; hidden]; rows j >= 1:
// [mask_embed[j-1] ; mask_feat[j-1]].  With all_real every row is a real (token, hidden) pair.
template <typename WT>
__global__ void k_gather(SeqMap sm, int all_real, const WT* embed, const WT* mask_embed,
                         const WT* mask_feat, const WT* hidden, const int* tokens, int H, int V,
                         float* x_in) {
  int m = blockIdx.x;
  int b, j;
  seq_of_row(sm, m, b, j);
  const WT *e, *f;
  if (all_real || j == 0) {
    int src = all_real ? (m + sm.row_base) : b;
    int tok = tokens[src];
    tok = min(max(tok, 0), V - 1);
    e = embed + (size_t)tok * H;
    f = hidden + (size_t)src * H;
  } else {
    e = mask_embed + (size_t)(j - 1) * H;
    f = mask_feat + (size_t)(j - 1) * H;
  }
  float* out = x_in + (size_t)m * 2 * H;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    out[i] = to_f32(e[i]);
    out[H + i] = hidden ? to_f32(f[i]) : 0.f;   // embedding-only input: no feature half
  }
}

// Y[m][n] = sum_k X[m][k] W[n][k] (+ bias[n]) (+ res[m][n]).  One warp per output feature n,
// MC rows per pass.  K is a multiple of 8.
template <typename WT, int MC>
__global__ void __launch_bounds__(256) k_linear(const float* __restrict__ X, int ldx,
                                                const WT* __restrict__ W,
                                                const WT* __restrict__ bias,
                                                const float* __restrict__ res, int ldr,
                                                float* __restrict__ Y, int ldy, int M, int N,
                                                int K) {
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int n = blockIdx.x * 8 + warp;
  if (n >= N) return;
  int m0 = blockIdx.y * MC;
  float acc[MC];
#pragma unroll
  for (int i = 0; i < MC; ++i) acc[i] = 0.f;
  const WT* wrow = W + (size_t)n * K;
  for (int k = lane * 8; k < K; k += 256) {
    float w[8];
    load8(wrow + k, w);
#pragma unroll
    for (int i = 0; i < MC; ++i) {
      if (m0 + i < M) {
        const float4* xp = reinterpret_cast<const float4*>(X + (size_t)(m0 + i) * ldx + k);
        float4 a = xp[0], c = xp[1];
        acc[i] += w[0] * a.x + w[1] * a.y + w[2] * a.z + w[3] * a.w + w[4] * c.x + w[5] * c.y +
                  w[6] * c.z + w[7] * c.w;
      }
    }
  }
#pragma unroll
  for (int i = 0; i < MC; ++i) {
    float v = warp_sum(acc[i]);
    if (lane == 0 && m0 + i < M) {
      if (bias) v += to_f32(bias[n]);
      if (res) v += res[(size_t)(m0 + i) * ldr + n];
      Y[(size_t)(m0 + i) * ldy + n] = v;
    }
  }
}

// y = x * g / sqrt(mean(x^2) + eps), one block per row.
template <typename WT>
__global__ void k_rmsnorm(const float* x, const WT* g, int H, float eps, float* y) {
  __shared__ float red[32];
  const float* xr = x + (size_t)blockIdx.x * H;
  float ss = 0.f;
  for (int i = threadIdx.x; i < H; i += blockDim.x) ss += xr[i] * xr[i];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) red[0] = rsqrtf(v / (float)H + eps);
  }
  __syncthreads();
  float inv = red[0];
  float* yr = y + (size_t)blockIdx.x * H;
  for (int i = threadIdx.x; i < H; i += blockDim.x) yr[i] = xr[i] * inv * to_f32(g[i]);
}

// RoPE on q (in place) and on k; k and v are written to the cache slab at the row's absolute
// position.  One block per row.  kv_tmp row = [k (Hkv) ; v (Hkv)] fp32.  The pair
// (i, i + d/2) of a head is rotated by pos * base^(-2i/d); angles are formed in double.
// With `side` != nullptr the new k / v rows go to side[m][2 * Hkv] (k then v) instead of the
// cache: a draft step leaves the cache untouched, and several groups may share one slot.
template <typename WT>
__global__ void k_rope_store(SeqMap sm, float* q, const float* kv_tmp, WT* kcache, WT* vcache, WT* side,
                             int n_heads, int n_kv_heads, int d, int max_ctx, float rope_base) {
  extern __shared__ float cs[];  // cos[d/2], sin[d/2]
  int m = blockIdx.x;
  int b, j;
  seq_of_row(sm, m, b, j);
  int pos = sm.len[b] + j;
  int half = d >> 1;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    double inv = exp2(-2.0 * (double)i / (double)d * log2((double)rope_base));
    double s, c;
    sincos((double)pos * inv, &s, &c);
    cs[i] = (float)c;
    cs[half + i] = (float)s;
  }
  __syncthreads();
  int Hq = n_heads * d, Hkv = n_kv_heads * d;
  if (q) {
    float* qr = q + (size_t)m * Hq;
    for (int t = threadIdx.x; t < n_heads * half; t += blockDim.x) {
      int h = t / half, i = t - h * half;
      float x = qr[h * d + i], y = qr[h * d + i + half];
      qr[h * d + i] = x * cs[i] - y * cs[half + i];
      qr[h * d + i + half] = y * cs[i] + x * cs[half + i];
    }
  }
  const float* kr = kv_tmp + (size_t)m * 2 * Hkv;
  const float* vr = kr + Hkv;
  size_t slab = (size_t)sm.slot[b] * n_kv_heads;
  for (int t = threadIdx.x; t < n_kv_heads * half; t += blockDim.x) {
    int h = t / half, i = t - h * half;
    float x = kr[h * d + i], y = kr[h * d + i + half];
    WT *kd, *vd;
    if (side) {
      kd = side + (size_t)m * 2 * Hkv + h * d;
      vd = kd + Hkv;
    } else {
      const size_t base = ((slab + h) * max_ctx + pos) * d;
      kd = kcache + base;
      vd = vcache + base;
    }
    store_as(kd + i, x * cs[i] - y * cs[half + i]);
    store_as(kd + i + half, y * cs[i] + x * cs[half + i]);
    store_as(vd + i, vr[h * d + i]);
    store_as(vd + i + half, vr[h * d + i + half]);
  }
}

// Attention under the parallel-draft mask: row j of a sequence sees cache rows [0, len) and
// the new rows 0..j, which sit in side[m][2 * Hkv] (k then v).  One block (4 warps) per (head, b);
// warps take keys round-robin, each lane owns D/32 channels; online softmax per (warp, row).
template <typename WT, int D>
__global__ void __launch_bounds__(128) k_attention(SeqMap sm, const float* q, const WT* kcache,
                                                   const WT* vcache, const WT* side, int n_heads,
                                                   int n_kv_heads, int max_ctx, float* attn) {
  constexpr int C = D / 32;
  constexpr int RMAX = kMaxRowsPerSeq;
  __shared__ float s_m[4][RMAX], s_l[4][RMAX];
  __shared__ float s_o[4][RMAX][D];
  int h = blockIdx.x, b = blockIdx.y;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int R = sm.row_off[b + 1] - sm.row_off[b];
  int L = sm.len[b];
  int m0 = sm.row_off[b] - sm.row_base;
  int hk = h / (n_heads / n_kv_heads);
  int Hq = n_heads * D;
  const float scale = rsqrtf((float)D);
  float qv[RMAX][C];
#pragma unroll
  for (int j = 0; j < RMAX; ++j)
#pragma unroll
    for (int c = 0; c < C; ++c)
      qv[j][c] = (j < R) ? q[(size_t)(m0 + j) * Hq + h * D + lane + 32 * c] * scale : 0.f;
  float mx[RMAX], l[RMAX], o[RMAX][C];
#pragma unroll
  for (int j = 0; j < RMAX; ++j) {
    mx[j] = -FLT_MAX; l[j] = 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) o[j][c] = 0.f;
  }
  const WT* kb = kcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;
  const WT* vb = vcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;
  for (int t = warp; t < L + R; t += 4) {
    float kx[C], vx[C];
#pragma unroll
    const WT* kr = t < L ? kb + (size_t)t * D : side + (size_t)(m0 + t - L) * 2 * n_kv_heads * D + hk * D;
    const WT* vr = t < L ? vb + (size_t)t * D : kr + n_kv_heads * D;
#pragma unroll
    for (int c = 0; c < C; ++c) {
      kx[c] = to_f32(kr[lane + 32 * c]);
      vx[c] = to_f32(vr[lane + 32 * c]);
    }
    int jmin = t < L ? 0 : t - L;  // rows that may see key t
#pragma unroll
    for (int j = 0; j < RMAX; ++j) {
      if (j >= jmin && j < R) {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < C; ++c) s += qv[j][c] * kx[c];
        s = warp_sum(s);
        float mnew = fmaxf(mx[j], s);
        float corr = __expf(mx[j] - mnew), p = __expf(s - mnew);
        l[j] = l[j] * corr + p;
#pragma unroll
        for (int c = 0; c < C; ++c) o[j][c] = o[j][c] * corr + p * vx[c];
        mx[j] = mnew;
      }
    }
  }
#pragma unroll
  for (int j = 0; j < RMAX; ++j) {
    if (lane == 0) { s_m[warp][j] = mx[j]; s_l[warp][j] = l[j]; }
#pragma unroll
    for (int c = 0; c < C; ++c) s_o[warp][j][lane + 32 * c] = o[j][c];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < R * D; idx += blockDim.x) {
    int j = idx / D, i = idx - j * D;
    float M = fmaxf(fmaxf(s_m[0][j], s_m[1][j]), fmaxf(s_m[2][j], s_m[3][j]));
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      float f = __expf(s_m[w][j] - M);
      num += f * s_o[w][j][i];
      den += f * s_l[w][j];
    }
    attn[(size_t)(m0 + j) * Hq + h * D + i] = num / den;
  }
}

__global__ void k_silu_mul(const float* gate, const float* up, float* out, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    float g = gate[i];
    out[i] = g / (1.f + __expf(-g)) * up[i];
  }
}

// Per-row max, log-sum-exp and top-n (descending logit, ties to the lower id).  One block per
// row; top-n by n selection passes, each picking the best entry that ranks after the last pick.
__global__ void __launch_bounds__(256) k_row_stats(const float* logits, int V, int top_n,
                                                   int* top_ids, float* top_logit, float* row_max,
                                                   float* row_lse) {
  __shared__ float s_v[8];
  __shared__ int s_i[8];
  __shared__ float s_f[8];
  const float* row = logits + (size_t)blockIdx.x * V;
  const int nv4 = (reinterpret_cast<uintptr_t>(row) & 15) == 0 ? V / 4 : 0;   // float4 part of the row
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float prev_v = FLT_MAX;
  int prev_i = -1;
  float rmax = 0.f;
  int passes = top_n > 0 ? top_n : 1;
  for (int t = 0; t < passes; ++t) {
    float bv = -FLT_MAX;
    int bi = 0x7fffffff;
    auto consider = [&](float x, int v) {
      const bool after = (x < prev_v) || (x == prev_v && v > prev_i);   // ranks after the last pick
      if (after && (x > bv || (x == bv && v < bi))) { bv = x; bi = v; }
    };
#pragma unroll 4
    for (int i = threadIdx.x; i < nv4; i += blockDim.x) {   // 16-byte loads, several in flight
      const float4 x = __ldg(reinterpret_cast<const float4*>(row) + i);
      consider(x.x, 4 * i); consider(x.y, 4 * i + 1); consider(x.z, 4 * i + 2); consider(x.w, 4 * i + 3);
    }
    for (int v = 4 * nv4 + threadIdx.x; v < V; v += blockDim.x) consider(row[v], v);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { s_v[warp] = bv; s_i[warp] = bi; }
    __syncthreads();
    bv = s_v[0]; bi = s_i[0];
    for (int w = 1; w < 8; ++w)
      if (s_v[w] > bv || (s_v[w] == bv && s_i[w] < bi)) { bv = s_v[w]; bi = s_i[w]; }
    __syncthreads();
    if (t == 0) rmax = bv;
    if (top_n > 0 && threadIdx.x == 0) {
      top_ids[(size_t)blockIdx.x * top_n + t] = bi;
      top_logit[(size_t)blockIdx.x * top_n + t] = bv;
    }
    prev_v = bv; prev_i = bi;
  }
  float s = 0.f;
#pragma unroll 4
  for (int i = threadIdx.x; i < nv4; i += blockDim.x) {
    const float4 x = __ldg(reinterpret_cast<const float4*>(row) + i);
    s += (expf(x.x - rmax) + expf(x.y - rmax)) + (expf(x.z - rmax) + expf(x.w - rmax));
  }
  for (int v = 4 * nv4 + threadIdx.x; v < V; v += blockDim.x) s += expf(row[v] - rmax);
  s = warp_sum(s);
  if (lane == 0) s_f[warp] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += s_f[w];
    if (row_max) row_max[blockIdx.x] = rmax;
    if (row_lse) row_lse[blockIdx.x] = rmax + logf(tot);
  }
}

// Gumbel-max token of each row of stored logits (draft sampling on the paths that keep logits
// in memory).  One block per row.
__global__ void __launch_bounds__(256) k_gumbel_argmax(const float* logits, int V, int R, SampleArgs sa) {
  __shared__ float s_v[8];
  __shared__ int s_i[8];
  const int m = blockIdx.x, b = m / R, j = m - b * R;
  const uint32_t row_id = ((uint32_t)b + sa.b_base) | ((uint32_t)j << 8);
  const float* row = logits + (size_t)m * V;
  float bv = -FLT_MAX;
  int bi = 0x7fffffff;
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    const float y = row[v] * sa.inv_temp + gumbel_noise(sa, (uint32_t)v, row_id);
    if (y > bv || (y == bv && v < bi)) { bv = y; bi = v; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  if ((threadIdx.x & 31) == 0) { s_v[threadIdx.x >> 5] = bv; s_i[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w)
      if (s_v[w] > bv || (s_v[w] == bv && s_i[w] < bi)) { bv = s_v[w]; bi = s_i[w]; }
    sa.sampled[m] = bi;
  }
}

template <typename WT>
__global__ void k_kv_copy(WT* kcache, WT* vcache, WT* K, WT* V, int slot, int len, int n_kv_heads,
                          int d, int max_ctx, int to_cache) {
  size_t n = (size_t)len * n_kv_heads * d;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (size_t)gridDim.x * blockDim.x) {
    int c = i % d;
    size_t r = i / d;
    int h = r % n_kv_heads;
    size_t t = r / n_kv_heads;
    size_t ci = (((size_t)slot * n_kv_heads + h) * max_ctx + t) * d + c;
    if (to_cache) { kcache[ci] = K[i]; vcache[ci] = V[i]; }
    else { K[i] = kcache[ci]; V[i] = vcache[ci]; }
  }
}

template <typename WT>
ps_status linear(ps_ctx* c, const float* X, int ldx, const void* W, const void* bias,
                 const float* res, int ldr, float* Y, int ldy, int M, int N, int K,
                 cudaStream_t st) {
  constexpr int MC = 8;
  dim3 grid((N + 7) / 8, (M + MC - 1) / MC);
  k_linear<WT, MC><<<grid, 256, 0, st>>>(X, ldx, (const WT*)W, (const WT*)bias, res, ldr, Y, ldy,
                                         M, N, K);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_linear");
}

template <typename WT>
ps_status fc_norm_kv(ps_ctx* c, const SeqMap& sm, int rows, int all_real, const void* hidden,
                     const int* tokens, bool with_q, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  int H = g.hidden, Hq = g.n_heads * g.head_dim, Hkv = g.n_kv_heads * g.head_dim;
  prof_mark(c, st, "begin");
  k_gather<WT><<<rows, 256, 0, st>>>(sm, all_real, (const WT*)w.embed, (const WT*)w.mask_embed,
                                     (const WT*)w.mask_feat,
                                     (g.flags & PS_FLAG_NO_FC) ? nullptr : (const WT*)hidden, tokens, H, g.vocab,
                                     c->x_in);
  c->launches++;
  ps_status s;
  const void* bias = (g.flags & PS_FLAG_FC_BIAS) ? w.b_fc : nullptr;
  if (g.flags & PS_FLAG_NO_FC) {   // x0 = the embedding half of x_in
    cudaError_t e = cudaMemcpy2DAsync(c->x0, (size_t)H * 4, c->x_in, (size_t)2 * H * 4, (size_t)H * 4, rows,
                                      cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return cuda_check(c, e, "x0 copy");
  } else if ((s = linear<WT>(c, c->x_in, 2 * H, w.w_fc, bias, nullptr, 0, c->x0, H, rows, H, 2 * H, st))) {
    return s;
  }
  k_rmsnorm<WT><<<rows, 256, 0, st>>>(c->x0, (const WT*)w.g_in, H, g.rms_eps, c->xn);
  c->launches++;
  prof_mark(c, st, "fc_norm");
  if (with_q)
    if ((s = linear<WT>(c, c->xn, H, w.w_q, nullptr, nullptr, 0, c->q, Hq, rows, Hq, H, st))) return s;
  if ((s = linear<WT>(c, c->xn, H, w.w_k, nullptr, nullptr, 0, c->kv_tmp, 2 * Hkv, rows, Hkv, H, st))) return s;
  if ((s = linear<WT>(c, c->xn, H, w.w_v, nullptr, nullptr, 0, c->kv_tmp + Hkv, 2 * Hkv, rows, Hkv, H, st))) return s;
  k_rope_store<WT><<<rows, 128, g.head_dim * sizeof(float), st>>>(
      sm, with_q ? c->q : nullptr, c->kv_tmp, (WT*)c->kcache, (WT*)c->vcache,
      with_q ? (WT*)c->kv_side : nullptr,   // a draft step keeps its new rows out of the cache
      g.n_heads, g.n_kv_heads, g.head_dim, g.max_ctx, g.rope_base);
  c->launches++;
  prof_mark(c, st, "qkv_rope");
  return cuda_check(c, cudaGetLastError(), "fc_norm_kv");
}

template <typename WT>
ps_status draft_impl(ps_ctx* c, const SeqMap& sm, int B, const void* hidden_last,
                     const int* token_last, int top_n, int* top_ids, float* top_logit,
                     float* row_max, float* row_lse, float* logits_out, float* feat_out,
                     const SampleArgs* sa, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  int H = g.hidden, Hq = g.n_heads * g.head_dim, F = g.ffn, V = g.vocab;
  int M = B * (g.k_masks + 1);
  ps_status s;
  if ((s = fc_norm_kv<WT>(c, sm, M, 0, hidden_last, token_last, true, st))) return s;
  dim3 ag(g.n_heads, B);
  if (g.head_dim == 64)
    k_attention<WT, 64><<<ag, 128, 0, st>>>(sm, c->q, (const WT*)c->kcache, (const WT*)c->vcache,
                                            (const WT*)c->kv_side, g.n_heads, g.n_kv_heads, g.max_ctx, c->attn);
  else
    k_attention<WT, 128><<<ag, 128, 0, st>>>(sm, c->q, (const WT*)c->kcache, (const WT*)c->vcache,
                                             (const WT*)c->kv_side, g.n_heads, g.n_kv_heads, g.max_ctx, c->attn);
  c->launches++;
  prof_mark(c, st, "attention");
  if ((s = linear<WT>(c, c->attn, Hq, w.w_o, nullptr, c->x0, H, c->a, H, M, H, Hq, st))) return s;
  prof_mark(c, st, "o_proj");
  k_rmsnorm<WT><<<M, 256, 0, st>>>(c->a, (const WT*)w.g_post, H, g.rms_eps, c->an);
  c->launches++;
  if ((s = linear<WT>(c, c->an, H, w.w_gate, nullptr, nullptr, 0, c->gate, F, M, F, H, st))) return s;
  if ((s = linear<WT>(c, c->an, H, w.w_up, nullptr, nullptr, 0, c->up, F, M, F, H, st))) return s;
  size_t n = (size_t)M * F;
  k_silu_mul<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(c->gate, c->up, c->gate, n);
  c->launches++;
  float* hdn = feat_out ? feat_out : c->hdn;
  if ((s = linear<WT>(c, c->gate, F, w.w_down, nullptr, c->a, H, hdn, H, M, H, F, st))) return s;
  prof_mark(c, st, "ffn");
  k_rmsnorm<WT><<<M, 256, 0, st>>>(hdn, (const WT*)w.g_final, H, g.rms_eps, c->hn);
  c->launches++;
  float* logits = logits_out ? logits_out : c->logits;
  if ((s = linear<WT>(c, c->hn, H, w.w_lm, nullptr, nullptr, 0, logits, V, M, V, H, st))) return s;
  if ((s = launch_row_stats(c, logits, M, V, top_n, top_ids, top_logit, row_max, row_lse, st))) return s;
  if (sa && (s = launch_gumbel_argmax(c, logits, M, V, g.k_masks + 1, *sa, st))) return s;
  prof_mark(c, st, "lm_head");
  return cuda_check(c, cudaGetLastError(), "draft_step");
}

}  // namespace

ps_status plain_kv_append(ps_ctx* c, const SeqMap& sm, int rows, const void* hidden,
                          const int* tokens, cudaStream_t st) {
  return c->cfg.dtype == PS_DTYPE_F32
             ? fc_norm_kv<float>(c, sm, rows, 1, hidden, tokens, false, st)
             : fc_norm_kv<__nv_bfloat16>(c, sm, rows, 1, hidden, tokens, false, st);
}

ps_status plain_draft_step(ps_ctx* c, const SeqMap& sm, int B, const void* hidden_last,
                           const int* token_last, int top_n, int* top_ids, float* top_logit,
                           float* row_max, float* row_lse, float* logits_out, float* feat_out,
                           const SampleArgs* sa, cudaStream_t st) {
  return c->cfg.dtype == PS_DTYPE_F32
             ? draft_impl<float>(c, sm, B, hidden_last, token_last, top_n, top_ids, top_logit,
                                 row_max, row_lse, logits_out, feat_out, sa, st)
             : draft_impl<__nv_bfloat16>(c, sm, B, hidden_last, token_last, top_n, top_ids,
                                         top_logit, row_max, row_lse, logits_out, feat_out, sa, st);
}

ps_status launch_rope_store_kv(ps_ctx* c, const SeqMap& sm, int rows, cudaStream_t st) {
  const ps_config& g = c->cfg;
  if (g.dtype == PS_DTYPE_F32)
    k_rope_store<float><<<rows, 128, g.head_dim * sizeof(float), st>>>(
        sm, nullptr, c->kv_tmp, (float*)c->kcache, (float*)c->vcache, nullptr, g.n_heads, g.n_kv_heads,
        g.head_dim, g.max_ctx, g.rope_base);
  else
    k_rope_store<__nv_bfloat16><<<rows, 128, g.head_dim * sizeof(float), st>>>(
        sm, nullptr, c->kv_tmp, (__nv_bfloat16*)c->kcache, (__nv_bfloat16*)c->vcache, nullptr, g.n_heads,
        g.n_kv_heads, g.head_dim, g.max_ctx, g.rope_base);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_rope_store");
}

ps_status launch_row_stats(ps_ctx* c, const float* logits, int M, int V, int top_n, int* top_ids,
                           float* top_logit, float* row_max, float* row_lse, cudaStream_t st) {
  if (top_n <= 0 && !row_max && !row_lse) return PS_OK;
  k_row_stats<<<M, 256, 0, st>>>(logits, V, top_n, top_ids, top_logit, row_max, row_lse);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_row_stats");
}

ps_status launch_gumbel_argmax(ps_ctx* c, const float* logits, int M, int V, int R, const SampleArgs& sa,
                               cudaStream_t st) {
  k_gumbel_argmax<<<M, 256, 0, st>>>(logits, V, R, sa);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_gumbel_argmax");
}

ps_status launch_kv_copy(ps_ctx* c, int slot, int len, void* K, void* V, bool to_cache,
                         cudaStream_t st) {
  const ps_config& g = c->cfg;
  if (len == 0) return PS_OK;
  if (g.dtype == PS_DTYPE_F32)
    k_kv_copy<float><<<296, 256, 0, st>>>((float*)c->kcache, (float*)c->vcache, (float*)K,
                                          (float*)V, slot, len, g.n_kv_heads, g.head_dim,
                                          g.max_ctx, to_cache ? 1 : 0);
  else
    k_kv_copy<__nv_bfloat16><<<296, 256, 0, st>>>(
        (__nv_bfloat16*)c->kcache, (__nv_bfloat16*)c->vcache, (__nv_bfloat16*)K,
        (__nv_bfloat16*)V, slot, len, g.n_kv_heads, g.head_dim, g.max_ctx, to_cache ? 1 : 0);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_kv_copy");
}

}  // namespace ps
