// Fused bf16 draft step for small M = B*(k+1) <= 16 (Sec. 4.1 "Inference", Sec. 4.3):
// every projection is a launch of the weight-streaming GEMM (ws_gemm.cuh) with the neighbouring
// element-wise work folded into its prologue / epilogue:
//   fc        prologue = gather of [embedding ; feature] / [MASK] rows     epilogue = store x0
//   q|k|v     prologue = RMSNorm(x0)                                       epilogue = store
//   o         prologue = merge of the attention splits                     epilogue = + x0
//   gate|up   prologue = RMSNorm(a)                                        epilogue = silu(g)*u
//   down      prologue = copy                                              epilogue = + a
//   LM head   prologue = RMSNorm(hdn)   epilogue = logits, per-CTA softmax/top-n partials,
//                                                  merged by the last CTA to finish
// Activations travel between the launches in fp32 (L2-resident, a few hundred KB).
#include <algorithm>
#include <cfloat>

#include "ws_gemm.cuh"

namespace ps {
namespace {

using namespace ws;

enum Pro { PRO_GATHER = 0, PRO_NORM = 1, PRO_F32 = 2, PRO_ATTN = 3 };
enum Epi { EPI_STORE = 0, EPI_SWIGLU = 1, EPI_LMHEAD = 2 };

constexpr int kMaxM = 16;
constexpr int kTopMax = PS_MAX_TOP_N;

struct LmPart {  // softmax / top-n summary of one CTA's vocabulary range for one row
  float vmax, sumexp;
  float top_v[kTopMax];
  int top_i[kTopMax];
};

struct GemmArgs {
  RowSrc rs;
  int N, K, M;
  int pass_cols;   // k columns per pass (multiple of 64), chosen by the host
  int rows_cap;    // capacity (features per CTA, x2 when zipped) of the CTA accumulator
  // ---- prologue inputs
  const float* x_f32;  int ldx;        // PRO_NORM / PRO_F32: [M][ldx]
  const __nv_bfloat16* gain; float eps;
  const float* ssq_in; int ssq_n;      // PRO_NORM: [ssq_n][M] partial sums of squares of x_f32 rows
  const __nv_bfloat16 *embed, *mask_embed, *mask_feat, *hidden;   // PRO_GATHER
  const int* tokens; int H, V, R;
  // PRO_ATTN: partial attention results [M][n_heads][n_split] (m, l) and [..][D] o
  const float* att_ml; const float* att_o; int n_heads, n_split, D;
  // ---- epilogue outputs
  float* out; int ldo;                 // EPI_STORE / EPI_SWIGLU: [M][ldo]
  const __nv_bfloat16* bias;
  const float* res; int ldr;
  float* ssq_out;                      // EPI_STORE: [gridDim.x][M] partial sums of squares, or nullptr
  // EPI_LMHEAD
  float* logits_out;                   // [M][N] or nullptr
  LmPart* parts;                       // [gridDim.x][M]
  unsigned* ticket;
  int top_n; int* top_ids; float* top_logit; float* row_max; float* row_lse;
  int* status;
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- prologues: the activation operand, columns [k0, k1), as hi/lo bf16 planes in shared memory
// One 8-column vector of row m starting at column k.
template <int PRO>
__device__ __forceinline__ void fetch8(const GemmArgs& a, int m, int k, float (&x)[8], uint4& raw) {
  if (PRO == PRO_GATHER) {
    // row m = (b, j): j == 0 -> [embed[token_b] ; hidden_b], j >= 1 -> [mask_embed ; mask_feat][j-1]
    const int H = a.H, b = m / a.R, j = m - b * a.R;
    const int half = k >= H ? 1 : 0, kk = k - half * H;
    const __nv_bfloat16* src;
    if (j == 0) {
      int tok = min(max(a.tokens[b], 0), a.V - 1);
      src = half == 0 ? a.embed + (size_t)tok * H : a.hidden + (size_t)b * H;
    } else {
      src = (half == 0 ? a.mask_embed : a.mask_feat) + (size_t)(j - 1) * H;
    }
    raw = *reinterpret_cast<const uint4*>(src + kk);
  } else if (PRO == PRO_NORM || PRO == PRO_F32) {
    const float4* xp = reinterpret_cast<const float4*>(a.x_f32 + (size_t)m * a.ldx + k);
    float4 x0 = xp[0], x1 = xp[1];
    x[0] = x0.x; x[1] = x0.y; x[2] = x0.z; x[3] = x0.w;
    x[4] = x1.x; x[5] = x1.y; x[6] = x1.z; x[7] = x1.w;
    if (PRO == PRO_NORM) raw = *reinterpret_cast<const uint4*>(a.gain + k);
  } else {  // PRO_ATTN: merge the key splits of (row m, head h): o = sum_s w_s o_s / sum_s w_s l_s
    const int D = a.D, S = a.n_split, nh = a.n_heads;
    const int h = k / D, d0 = k - h * D;
    const float* ml = a.att_ml + ((size_t)m * nh + h) * S * 2;
    float mx = -FLT_MAX;
    for (int s = 0; s < S; ++s) mx = fmaxf(mx, ml[2 * s]);
    float den = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = 0.f;
    for (int s = 0; s < S; ++s) {
      float w = __expf(ml[2 * s] - mx);
      den += w * ml[2 * s + 1];
      const float4* op = reinterpret_cast<const float4*>(a.att_o + (((size_t)m * nh + h) * S + s) * D + d0);
      float4 o0 = op[0], o1 = op[1];
      x[0] += w * o0.x; x[1] += w * o0.y; x[2] += w * o0.z; x[3] += w * o0.w;
      x[4] += w * o1.x; x[5] += w * o1.y; x[6] += w * o1.z; x[7] += w * o1.w;
    }
    const float inv = 1.f / den;
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] *= inv;
  }
}

template <int PRO>
__device__ void load_acts(const GemmArgs& a, unsigned char* a_hi, unsigned char* a_lo, int apitch,
                          const float* row_scale, int k0, int k1, int tid) {
  constexpr int U = 4;   // vectors in flight per thread: all loads are issued before any store
  const int M = a.M, vecs = (k1 - k0) / 8, total = M * vecs;
  for (int base = tid; base < total; base += U * kConsumerThreads) {
    float x[U][8];
    uint4 raw[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int idx = base + u * kConsumerThreads;
      if (idx < total) {
        const int m = idx / vecs, v = idx - m * vecs;
        fetch8<PRO>(a, m, k0 + v * 8, x[u], raw[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int idx = base + u * kConsumerThreads;
      if (idx < total) {
        const int m = idx / vecs, v = idx - m * vecs;
        const size_t off = (size_t)m * apitch + (size_t)v * 16;
        if (PRO == PRO_GATHER) {
          *reinterpret_cast<uint4*>(a_hi + off) = raw[u];
          *reinterpret_cast<uint4*>(a_lo + off) = make_uint4(0, 0, 0, 0);   // inputs are exact bf16
        } else {
          if (PRO == PRO_NORM) {
            const __nv_bfloat162* gp = reinterpret_cast<const __nv_bfloat162*>(&raw[u]);
            const float s = row_scale[m];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float2 gf = __bfloat1622float2(gp[i]);
              x[u][2 * i] = x[u][2 * i] * s * gf.x;
              x[u][2 * i + 1] = x[u][2 * i + 1] * s * gf.y;
            }
          }
          store_split8(a_hi, a_lo, off, x[u]);
        }
      }
    }
  }
}

// Shared-memory layout (dynamic): [Smem][red: 2 x warps x 16 sub-tile rows x ms(M) floats]
// [row scales][CTA accumulator: M x rows_cap floats][act hi plane][act lo plane][ring]
__host__ __device__ constexpr int m_stride(int M) { return M <= 8 ? 8 : 16; }
__host__ __device__ constexpr int red_floats(int M) { return kConsumerWarps * 16 * m_stride(M); }

struct Layout {
  int off_red, off_scale, off_out, off_hi, off_lo, off_ring, n_slots, total;
};

__host__ __device__ inline Layout make_layout(int M, int pass_cols, int rows_cap, int smem_limit) {
  Layout L;
  int off = (int)((sizeof(Smem) + 127) & ~127u);
  L.off_red = off; off += 2 * red_floats(M) * 4;
  L.off_scale = off; off += 128;
  L.off_out = off; off += ((rows_cap * M * 4) + 127) & ~127;
  const int plane = ((M * act_pitch(pass_cols)) + 127) & ~127;
  L.off_hi = off; off += plane;
  L.off_lo = off; off += plane;
  L.off_ring = off;
  int n = (smem_limit - off) / kSlotBytes;
  L.n_slots = n > kMaxSlots ? kMaxSlots : n;
  L.total = off + (L.n_slots > 0 ? L.n_slots : 0) * kSlotBytes;
  return L;
}

// Smallest number of k passes whose activation planes leave room for kMinSlots ring slots.
// Passes are whole numbers of KC-column chunks so that every bulk copy but the last of a row
// is a full chunk.  Returns the columns per pass or 0 if nothing fits.
int choose_pass_cols(int M, int K, int rows_cap, int smem_limit) {
  const int n_chunks = (K + KC - 1) / KC;
  for (int n_pass = 1; n_pass <= n_chunks; ++n_pass) {
    int cols = (n_chunks + n_pass - 1) / n_pass * KC;
    if (make_layout(M, std::min(cols, K), rows_cap, smem_limit).n_slots >= kMinSlots) return cols;
    if (n_pass == n_chunks && make_layout(M, std::min(cols, K), rows_cap, smem_limit).n_slots >= 2) return cols;
  }
  return 0;
}

template <int PRO, int EPI, int NB>
__global__ void __launch_bounds__(kThreads, 1) k_ws_gemm(GemmArgs a, int smem_limit) {
  extern __shared__ __align__(128) unsigned char smem[];
  Smem& sm = *reinterpret_cast<Smem*>(smem);
  const int pass_cols = a.pass_cols;
  const Layout L = make_layout(a.M, min(pass_cols, a.K), a.rows_cap, smem_limit);
  float* red = reinterpret_cast<float*>(smem + L.off_red);
  float* row_scale = reinterpret_cast<float*>(smem + L.off_scale);
  float* cta_out = reinterpret_cast<float*>(smem + L.off_out);   // [m][rows_cap]
  unsigned char* a_hi = smem + L.off_hi;
  unsigned char* a_lo = smem + L.off_lo;
  unsigned char* ring = smem + L.off_ring;
  const int apitch = act_pitch(min(pass_cols, a.K));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rows_cap = a.rows_cap, rows_half = rows_cap >> 1;

  if (tid == 0) {
    for (int i = 0; i < L.n_slots; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.empty[i], kConsumerWarps);
    }
    sm.abort_flag = 0;
    sm.is_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  int n_begin, n_end;
  cta_range(a.N, blockIdx.x, gridDim.x, n_begin, n_end);
  const int cnt = n_end - n_begin;
  const int n_st = n_subtiles(a.rs, n_begin, n_end);

  if (warp == kConsumerWarps) {
    produce(a.rs, a.K, pass_cols, n_begin, n_end, ring, L.n_slots, sm, lane);
  } else {
    if (PRO == PRO_NORM) {
      // scale[m] = rsqrt(mean(x^2) + eps): the producing kernel left one partial sum of squares
      // per CTA and row; they are added in a fixed order
      for (int m = warp; m < a.M; m += kConsumerWarps) {
        float ss = 0.f;
        for (int c = lane; c < a.ssq_n; c += 32) ss += a.ssq_in[(size_t)c * a.M + m];
        ss = warp_sum(ss);
        if (lane == 0) row_scale[m] = rsqrtf(ss / (float)a.K + a.eps);
      }
      consumer_sync();
    }
    int it = 0, buf = 0;
    bool alive = true;   // after a wait expired the loops still run (barriers stay matched) but do no work
    for (int k0 = 0; k0 < a.K; k0 += pass_cols) {
      const int k1 = min(a.K, k0 + pass_cols);
      consumer_sync();   // everyone is done reading the previous pass's planes
      load_acts<PRO>(a, a_hi, a_lo, apitch, row_scale, k0, k1, tid);
      consumer_sync();
      for (int st = 0; st < n_st; ++st, buf ^= 1) {
        float part[NB][4];
        if (alive)
          alive = consume_tile<NB>(a_hi, a_lo, apitch, a.M, k1 - k0, ring, L.n_slots, sm, it, warp, lane,
                                   part);
        // partial sums of this warp's k-slice: red[buf][warp][row of the sub-tile (0..15)][m]
        constexpr int MS = 8 * NB, kRed = kConsumerWarps * 16 * MS;
        {
          const int g = lane >> 2, t = lane & 3;
          float* r = red + (size_t)buf * kRed + (size_t)warp * 16 * MS;
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            r[g * MS + 8 * nb + 2 * t] = part[nb][0];
            r[g * MS + 8 * nb + 2 * t + 1] = part[nb][1];
            r[(g + 8) * MS + 8 * nb + 2 * t] = part[nb][2];
            r[(g + 8) * MS + 8 * nb + 2 * t + 1] = part[nb][3];
          }
        }
        consumer_sync();
        // 16 sub-tile rows x MS threads add the warps' partials into the CTA accumulator
        const int i = tid / MS, m = tid % MS;
        const int feat = subtile_feature(a.rs, n_begin, st, (i >> 3) & 1, i & 7);
        if (i < 16 && m < a.M && feat < n_end) {
          const float* rb = red + (size_t)buf * kRed;
          float v = 0.f;
#pragma unroll
          for (int w = 0; w < kConsumerWarps; ++w) v += rb[((size_t)w * 16 + i) * MS + m];
          const int idx = ((a.rs.zip && i >= 8) ? rows_half : 0) + (feat - n_begin);
          float* dst = cta_out + (size_t)m * rows_cap + idx;
          *dst = (k0 == 0) ? v : *dst + v;
        }
      }
    }
    consumer_sync();
    const bool ok = !*(volatile int*)&sm.abort_flag;
    // ---- CTA-level epilogue over the accumulated features --------------------------------
    if (ok && EPI == EPI_STORE) {
      // warp per row m; also this CTA's share of the row's sum of squares for the next RMSNorm
      for (int m = warp; m < a.M; m += kConsumerWarps) {
        float ss = 0.f;
        for (int idx = lane; idx < cnt; idx += 32) {
          const int n = n_begin + idx;
          float v = cta_out[(size_t)m * rows_cap + idx];
          if (a.bias) v += __bfloat162float(a.bias[n]);
          if (a.res) v += a.res[(size_t)m * a.ldr + n];
          a.out[(size_t)m * a.ldo + n] = v;
          ss += v * v;
        }
        ss = warp_sum(ss);
        if (a.ssq_out && lane == 0) a.ssq_out[(size_t)blockIdx.x * a.M + m] = ss;
      }
    } else if (ok && EPI == EPI_SWIGLU) {
      for (int e = tid; e < a.M * cnt; e += kConsumerThreads) {
        const int m = e / cnt, idx = e - m * cnt, n = n_begin + idx;
        const float gv = cta_out[(size_t)m * rows_cap + idx];
        const float uv = cta_out[(size_t)m * rows_cap + rows_half + idx];
        a.out[(size_t)m * a.ldo + n] = gv / (1.f + __expf(-gv)) * uv;
      }
    } else if (ok && EPI == EPI_LMHEAD) {
      if (a.logits_out)
        for (int e = tid; e < a.M * cnt; e += kConsumerThreads) {
          const int m = e / cnt, idx = e - m * cnt;
          a.logits_out[(size_t)m * a.N + n_begin + idx] = cta_out[(size_t)m * rows_cap + idx];
        }
      // per-row summary of this CTA's vocabulary range: warp per row m
      for (int m = warp; m < a.M; m += kConsumerWarps) {
        const float* lg = cta_out + (size_t)m * rows_cap;
        float mx = -FLT_MAX;
        for (int i = lane; i < cnt; i += 32) mx = fmaxf(mx, lg[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
        for (int i = lane; i < cnt; i += 32) se += __expf(lg[i] - mx);
        se = warp_sum(se);
        LmPart* p = a.parts + (size_t)blockIdx.x * a.M + m;
        if (lane == 0) { p->vmax = mx; p->sumexp = se; }
        float pv = FLT_MAX; int pi = -1;
        for (int tn = 0; tn < a.top_n; ++tn) {
          float bv = -FLT_MAX; int bi = 0x7fffffff;
          for (int i = lane; i < cnt; i += 32) {
            float x = lg[i]; int id = n_begin + i;
            bool after = (x < pv) || (x == pv && id > pi);
            if (after && (x > bv || (x == bv && id < bi))) { bv = x; bi = id; }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          if (lane == 0) { p->top_v[tn] = bv; p->top_i[tn] = bi; }
          pv = bv; pi = bi;
        }
      }
    }
  }

  if (EPI == EPI_LMHEAD) {
    // the last CTA to finish merges the per-CTA summaries (no CTA waits for another)
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      unsigned tk = atomicAdd(a.ticket, 1u);
      sm.is_last = (tk == gridDim.x - 1);
    }
    __syncthreads();
    if (sm.is_last && warp < kConsumerWarps) {
      __threadfence();
      const int G = gridDim.x;
      for (int m = warp; m < a.M; m += kConsumerWarps) {
        const LmPart* P = a.parts + m;
        float mx = -FLT_MAX;
        for (int c = lane; c < G; c += 32) mx = fmaxf(mx, P[(size_t)c * a.M].vmax);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
        for (int c = lane; c < G; c += 32) se += P[(size_t)c * a.M].sumexp * __expf(P[(size_t)c * a.M].vmax - mx);
        se = warp_sum(se);
        if (lane == 0) {
          if (a.row_max) a.row_max[m] = mx;
          if (a.row_lse) a.row_lse[m] = mx + logf(se);
        }
        float pv = FLT_MAX; int pi = -1;
        for (int tn = 0; tn < a.top_n; ++tn) {
          float bv = -FLT_MAX; int bi = 0x7fffffff;
          for (int e = lane; e < G * a.top_n; e += 32) {
            int c = e / a.top_n, k = e - c * a.top_n;
            float x = P[(size_t)c * a.M].top_v[k]; int id = P[(size_t)c * a.M].top_i[k];
            if (id == 0x7fffffff) continue;
            bool after = (x < pv) || (x == pv && id > pi);
            if (after && (x > bv || (x == bv && id < bi))) { bv = x; bi = id; }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          if (lane == 0) { a.top_ids[(size_t)m * a.top_n + tn] = bi; a.top_logit[(size_t)m * a.top_n + tn] = bv; }
          pv = bv; pi = bi;
        }
      }
      if (tid == 0) *a.ticket = 0u;
    }
  }
  __syncthreads();
  if (sm.abort_flag) {
    // let copies that are still in flight land before the shared memory is given up
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    if (tid == 0) atomicOr(a.status, kStatTimeout);
  }
}

int rows_cap_for(int N, int n_cta, bool zip) {
  int per = (N + n_cta - 1) / n_cta + 1;
  per = (per + 3) & ~3;
  return zip ? 2 * per : per;
}

template <int PRO, int EPI>
ps_status launch_gemm(ps_ctx* c, GemmArgs& a, cudaStream_t st) {
  const int n_cta = c->n_sm;
  const int smem_limit = c->smem_optin;
  a.rows_cap = rows_cap_for(a.N, n_cta, a.rs.zip != 0);
  a.pass_cols = choose_pass_cols(a.M, a.K, a.rows_cap, smem_limit);
  if (a.pass_cols == 0) return fail(c, PS_ERR_UNSUPPORTED, "activation operand does not fit shared memory");
  Layout L = make_layout(a.M, std::min(a.pass_cols, a.K), a.rows_cap, smem_limit);
  a.status = c->dev_status;
  auto kern = a.M > 8 ? k_ws_gemm<PRO, EPI, 2> : k_ws_gemm<PRO, EPI, 1>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_limit);
  if (e != cudaSuccess) return cuda_check(c, e, "ws_gemm smem attribute");
  kern<<<n_cta, kThreads, L.total, st>>>(a, smem_limit);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_ws_gemm");
}

struct FusedScratch {
  float* qkv; float* att_ml; float* att_o; float* act; LmPart* parts; unsigned* ticket;
  float* ssq[3];   // partial sums of squares of x0, a and hdn rows: [kMaxSm][kMaxM] each
  size_t bytes;
};

// One carve-up for sizing (base == nullptr) and for use; always kMaxM rows and kMaxSm CTAs.
FusedScratch carve_fused(const ps_config& g, char* base) {
  const size_t Hq = (size_t)g.n_heads * g.head_dim, Hkv = (size_t)g.n_kv_heads * g.head_dim;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off += (bytes + 255) & ~(size_t)255;
    return base ? base + at : nullptr;
  };
  FusedScratch s;
  s.qkv = (float*)take((size_t)kMaxM * (Hq + 2 * Hkv) * 4);
  s.att_ml = (float*)take((size_t)kMaxM * g.n_heads * kAttnMaxSplit * 2 * 4);
  s.att_o = (float*)take((size_t)kMaxM * g.n_heads * kAttnMaxSplit * g.head_dim * 4);
  s.act = (float*)take((size_t)kMaxM * g.ffn * 4);
  s.parts = (LmPart*)take((size_t)kMaxSm * kMaxM * sizeof(LmPart));
  s.ticket = (unsigned*)take(256);
  for (int i = 0; i < 3; ++i) s.ssq[i] = (float*)take((size_t)kMaxSm * kMaxM * 4);
  s.bytes = off;
  return s;
}

}  // namespace

bool fused_supported(const ps_ctx* c, int M) {
  const ps_config& g = c->cfg;
  if (g.dtype != PS_DTYPE_BF16 || (g.flags & PS_FLAG_UNFUSED_KERNELS)) return false;
  if (M > kMaxM) return false;
  const int Hq = g.n_heads * g.head_dim;
  const int lim = c->smem_optin, n = c->n_sm;
  return choose_pass_cols(M, 2 * g.hidden, rows_cap_for(g.hidden, n, false), lim) &&
         choose_pass_cols(M, g.hidden, rows_cap_for(Hq + 2 * g.n_kv_heads * g.head_dim, n, false), lim) &&
         choose_pass_cols(M, Hq, rows_cap_for(g.hidden, n, false), lim) &&
         choose_pass_cols(M, g.hidden, rows_cap_for(g.ffn, n, true), lim) &&
         choose_pass_cols(M, g.ffn, rows_cap_for(g.hidden, n, false), lim) &&
         choose_pass_cols(M, g.hidden, rows_cap_for(g.vocab, n, false), lim);
}

size_t fused_scratch_bytes(const ps_config& g) { return carve_fused(g, nullptr).bytes; }

ps_status fused_debug_buffer(ps_ctx* c, const char* name, void** ptr, size_t* bytes) {
  const ps_config& g = c->cfg;
  FusedScratch f = carve_fused(g, (char*)c->fused_scratch);
  if (!std::strcmp(name, "qkv")) {
    *ptr = f.qkv;
    *bytes = (size_t)kMaxM * (g.n_heads + 2 * g.n_kv_heads) * g.head_dim * 4;
    return PS_OK;
  }
  if (!std::strcmp(name, "act")) { *ptr = f.act; *bytes = (size_t)kMaxM * g.ffn * 4; return PS_OK; }
  return PS_ERR_INVALID_ARG;
}

ps_status fused_draft_step(ps_ctx* c, const SeqMap& sm, int B, const void* hidden_last,
                           const int* token_last, int top_n, int* top_ids, float* top_logit,
                           float* row_max, float* row_lse, float* logits_out, float* feat_out,
                           cudaStream_t st) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  const int H = g.hidden, Hq = g.n_heads * g.head_dim, Hkv = g.n_kv_heads * g.head_dim, F = g.ffn,
            V = g.vocab, R = g.k_masks + 1, M = B * R, D = g.head_dim;
  typedef const __nv_bfloat16* BP;
  const FusedScratch f = carve_fused(g, (char*)c->fused_scratch);
  ps_status s;
  prof_mark(c, st, "begin");
  {  // S1 fc: x0 = W_fc [e ; f] (+ b)
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_fc; a.rs.rows[0] = H; a.rs.n_mats = 1;
    a.N = H; a.K = 2 * H; a.M = M;
    a.embed = (BP)w.embed; a.mask_embed = (BP)w.mask_embed; a.mask_feat = (BP)w.mask_feat;
    a.hidden = (BP)hidden_last; a.tokens = token_last; a.H = H; a.V = V; a.R = R;
    a.out = c->x0; a.ldo = H; a.bias = (g.flags & PS_FLAG_FC_BIAS) ? (BP)w.b_fc : nullptr;
    a.ssq_out = f.ssq[0];
    if ((s = launch_gemm<PRO_GATHER, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "fc_norm");
  {  // S2 q|k|v = W rms(x0)
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_q; a.rs.W[1] = (BP)w.w_k; a.rs.W[2] = (BP)w.w_v;
    a.rs.rows[0] = Hq; a.rs.rows[1] = Hkv; a.rs.rows[2] = Hkv; a.rs.n_mats = 3;
    a.N = Hq + 2 * Hkv; a.K = H; a.M = M;
    a.x_f32 = c->x0; a.ldx = H; a.gain = (BP)w.g_in; a.eps = g.rms_eps;
    a.ssq_in = f.ssq[0]; a.ssq_n = c->n_sm;
    a.out = f.qkv; a.ldo = Hq + 2 * Hkv;
    if ((s = launch_gemm<PRO_NORM, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "qkv_rope");
  int n_split = 1;
  if ((s = launch_attn_split(c, sm, B, f.qkv, f.att_ml, f.att_o, &n_split, st))) return s;
  prof_mark(c, st, "attention");
  {  // S4 a = x0 + W_o attn
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_o; a.rs.rows[0] = H; a.rs.n_mats = 1;
    a.N = H; a.K = Hq; a.M = M;
    a.att_ml = f.att_ml; a.att_o = f.att_o; a.n_heads = g.n_heads; a.n_split = n_split; a.D = D;
    a.out = c->a; a.ldo = H; a.res = c->x0; a.ldr = H;
    a.ssq_out = f.ssq[1];
    if ((s = launch_gemm<PRO_ATTN, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "o_proj");
  {  // S5a act = silu(W_g rms(a)) * (W_u rms(a))
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_gate; a.rs.W[1] = (BP)w.w_up; a.rs.rows[0] = F; a.rs.rows[1] = F;
    a.rs.n_mats = 2; a.rs.zip = 1;
    a.N = F; a.K = H; a.M = M;
    a.x_f32 = c->a; a.ldx = H; a.gain = (BP)w.g_post; a.eps = g.rms_eps;
    a.ssq_in = f.ssq[1]; a.ssq_n = c->n_sm;
    a.out = f.act; a.ldo = F;
    if ((s = launch_gemm<PRO_NORM, EPI_SWIGLU>(c, a, st))) return s;
  }
  float* hdn = feat_out ? feat_out : c->hdn;
  {  // S5b hdn = a + W_d act
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_down; a.rs.rows[0] = H; a.rs.n_mats = 1;
    a.N = H; a.K = F; a.M = M;
    a.x_f32 = f.act; a.ldx = F;
    a.out = hdn; a.ldo = H; a.res = c->a; a.ldr = H;
    a.ssq_out = f.ssq[2];
    if ((s = launch_gemm<PRO_F32, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "ffn");
  {  // S6 logits = W_lm rms(hdn), softmax statistics and top-n without a second pass over logits
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_lm; a.rs.rows[0] = V; a.rs.n_mats = 1;
    a.N = V; a.K = H; a.M = M;
    a.x_f32 = hdn; a.ldx = H; a.gain = (BP)w.g_final; a.eps = g.rms_eps;
    a.ssq_in = f.ssq[2]; a.ssq_n = c->n_sm;
    a.logits_out = logits_out; a.parts = f.parts; a.ticket = f.ticket;
    a.top_n = top_n; a.top_ids = top_ids; a.top_logit = top_logit; a.row_max = row_max; a.row_lse = row_lse;
    if ((s = launch_gemm<PRO_NORM, EPI_LMHEAD>(c, a, st))) return s;
  }
  prof_mark(c, st, "lm_head");
  return PS_OK;
}

}  // namespace ps
