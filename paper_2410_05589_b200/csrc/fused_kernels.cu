// Fused bf16 draft step for small M = B*(k+1) <= 16 (Sec. 4.1 "Inference", Sec. 4.3):
// every projection is a launch of the weight-streaming GEMM (ws_gemm.cuh) with the neighbouring
// element-wise work folded into its epilogue:
//   fc        input = [embedding ; feature] / [MASK] rows (gathered by bulk copies)
//             epilogue: x0 (+ bias), planes of x0 * g_in, partial sums of squares
//   q|k|v     input = planes of x0 * g_in       epilogue: * rms scale of x0
//   o         input = planes of the merged attention output (written by the attention kernel)
//             epilogue: a = x0 + ., planes of a * g_post, partial sums of squares
//   gate|up   input = planes of a * g_post      epilogue: * rms scale, silu(g)*u as planes
//   down      input = planes of silu(g)*u       epilogue: hdn = a + ., planes of hdn * g_final
//   LM head   input = planes of hdn * g_final   epilogue: * rms scale, logits, per-CTA
//             softmax/top-n summaries merged by the last CTA to finish
// "Planes" are the hi/lo bf16 split of an fp32 activation, kept in global memory ([M][width],
// L2 resident) so that the next launch fetches its operand with a few bulk copies instead of
// converting it with thread code.  RMSNorm's row scale is a scalar per row, so it is applied
// to the product: W (s x * g) = s (W (x * g)).
#include <algorithm>
#include <cfloat>

#include "ws_gemm.cuh"

namespace ps {
namespace {

using namespace ws;

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
  int pass_cols;   // k columns per pass (multiple of KC), chosen by the host
  int rows_cap;    // capacity (features per CTA, x2 when zipped) of the CTA accumulator
  // ---- activation operand: planes [M][ld_in] bf16 in global memory, or (gather) rows of
  // [embed[token] ; hidden] for the first row of a sequence and [mask_embed ; mask_feat] after it
  const __nv_bfloat16 *in_hi, *in_lo; int ld_in;
  const __nv_bfloat16 *embed, *mask_embed, *mask_feat, *hidden;
  const int* tokens; int H, V, R;
  // ---- RMSNorm row scale from [ssq_n][M] partial sums of squares (nullptr: no scaling)
  const float* ssq_in; int ssq_n; float eps;
  // ---- epilogue outputs
  float* out; int ldo;                 // fp32 [M][ldo] (optional for EPI_SWIGLU)
  const __nv_bfloat16* bias;
  const float* res; int ldr;
  float* ssq_out;                      // [gridDim.x][M] partial sums of squares of out, or nullptr
  __nv_bfloat16 *out_hi, *out_lo; int ld_plane;   // planes of out * gain_next, or nullptr
  const __nv_bfloat16* gain_next;                 // nullptr: no gain
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

// hi = bf16(x), lo = bf16(x - hi)
__device__ __forceinline__ void split_store(__nv_bfloat16* hi, __nv_bfloat16* lo, float x) {
  const __nv_bfloat16 h = __float2bfloat16_rn(x);
  *hi = h;
  *lo = __float2bfloat16_rn(x - __bfloat162float(h));
}

// Shared-memory layout (dynamic): [Smem][red: 2 x warps x 16 sub-tile rows x 8 NB floats]
// [row scales][CTA accumulator: M x rows_cap floats][act hi plane][act lo plane][ring]
struct Layout {
  int off_red, off_scale, off_out, off_hi, off_lo, off_ring, n_slots, total;
};

__host__ __device__ inline Layout make_layout(int M, int pass_cols, int rows_cap, int smem_limit) {
  Layout L;
  int off = (int)((sizeof(Smem) + 127) & ~127u);
  L.off_red = off; off += 2 * kConsumerWarps * 16 * (M <= 8 ? 8 : 16) * 4;
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

// Smallest number of k passes whose activation planes leave room for kMinSlots ring slots (at
// the largest pass count two slots are enough).  Passes are whole numbers of KC-column chunks
// so that every bulk copy but the last of a row is a full chunk.  Returns the columns per pass
// or 0 if nothing fits.
int choose_pass_cols(int M, int K, int rows_cap, int smem_limit) {
  const int n_chunks = (K + KC - 1) / KC;
  for (int n_pass = 1; n_pass <= n_chunks; ++n_pass) {
    const int cols = (n_chunks + n_pass - 1) / n_pass * KC;
    const int slots = make_layout(M, std::min(cols, K), rows_cap, smem_limit).n_slots;
    if (slots >= kMinSlots || (n_pass == n_chunks && slots >= 3)) return cols;
  }
  return 0;
}

// Plane loader (one warp): fetches the activation operand of every pass with bulk copies, one
// per row and plane.  Lanes 0..15 own the hi plane rows, lanes 16..31 the lo plane rows.
template <bool GATHER>
__device__ __forceinline__ void load_planes(const GemmArgs& a, unsigned char* a_hi, unsigned char* a_lo,
                                            int apitch, Smem& sm, int lane) {
  const int m = lane & 15, plane = lane >> 4;
  const bool active = m < a.M && !(GATHER && plane == 1);
  const __nv_bfloat16 *src_e = nullptr, *src_f = nullptr;   // gather: embedding half, feature half
  if (GATHER && active) {
    const int b = m / a.R, j = m - b * a.R;
    if (j == 0) {
      const int tok = min(max(a.tokens[b], 0), a.V - 1);
      src_e = a.embed + (size_t)tok * a.H;
      src_f = a.hidden + (size_t)b * a.H;
    } else {
      src_e = a.mask_embed + (size_t)(j - 1) * a.H;
      src_f = a.mask_feat + (size_t)(j - 1) * a.H;
    }
  }
  int pass = 0;
  for (int k0 = 0; k0 < a.K; k0 += a.pass_cols, ++pass) {
    const int k1 = min(a.K, k0 + a.pass_cols);
    int ok = 1;
    if (lane == 0) {
      if (pass > 0) ok = mbar_wait(&sm.planes_empty, (pass - 1) & 1, &sm.abort_flag) ? 1 : 0;
      if (ok) mbar_arrive_expect_tx(&sm.planes_full, (uint32_t)((GATHER ? 1 : 2) * a.M * (k1 - k0) * 2));
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) return;
    if (!active) continue;
    unsigned char* dst = (plane ? a_lo : a_hi) + (size_t)m * apitch;
    if (GATHER) {
      const int e0 = max(k0, 0), e1 = min(k1, a.H);           // part inside the embedding half
      if (e1 > e0) bulk_g2s(dst + (size_t)(e0 - k0) * 2, src_e + e0, (uint32_t)((e1 - e0) * 2), &sm.planes_full);
      const int f0 = max(k0, a.H), f1 = min(k1, 2 * a.H);     // part inside the feature half
      if (f1 > f0)
        bulk_g2s(dst + (size_t)(f0 - k0) * 2, src_f + (f0 - a.H), (uint32_t)((f1 - f0) * 2), &sm.planes_full);
    } else {
      const __nv_bfloat16* src = (plane ? a.in_lo : a.in_hi) + (size_t)m * a.ld_in + k0;
      bulk_g2s(dst, src, (uint32_t)((k1 - k0) * 2), &sm.planes_full);
    }
  }
}

template <bool GATHER, int EPI, int NB>
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
    mbar_init(&sm.planes_full, 1);
    mbar_init(&sm.planes_empty, 1);
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
  } else if (warp == kConsumerWarps + 1) {
    load_planes<GATHER>(a, a_hi, a_lo, apitch, sm, lane);
  } else {
    // scale[m] = rsqrt(mean(x^2) + eps): the producing kernel left one partial sum of squares per
    // CTA and row; they are added in a fixed order.  Needed only by the epilogue.
    for (int m = warp; m < a.M; m += kConsumerWarps) {
      float sc = 1.f;
      if (a.ssq_in) {
        float ss = 0.f;
        for (int c = lane; c < a.ssq_n; c += 32) ss += a.ssq_in[(size_t)c * a.M + m];
        ss = warp_sum(ss);
        sc = rsqrtf(ss / (float)a.K + a.eps);
      }
      if (lane == 0) row_scale[m] = sc;
    }
    int it = 0, buf = 0, pass = 0;
    bool alive = true;   // after a wait expired the loops still run (barriers stay matched) but do no work
    for (int k0 = 0; k0 < a.K; k0 += pass_cols, ++pass) {
      const int k1 = min(a.K, k0 + pass_cols);
      if (alive) alive = mbar_wait(&sm.planes_full, pass & 1, &sm.abort_flag);
      for (int st = 0; st < n_st; ++st, buf ^= 1) {
        float part[NB][4];
        if (alive)
          alive = consume_tile<NB, !GATHER>(a_hi, a_lo, apitch, a.M, k1 - k0, ring, L.n_slots, sm, it,
                                            warp, lane, part);
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
      consumer_sync();                              // every warp is done with this pass's planes
      if (tid == 0) mbar_arrive(&sm.planes_empty);
    }
    const bool ok = !*(volatile int*)&sm.abort_flag;
    // ---- CTA-level epilogue over the accumulated features --------------------------------
    if (ok && EPI == EPI_STORE) {
      // warp per row m; also this CTA's share of the row's sum of squares for the next RMSNorm
      for (int m = warp; m < a.M; m += kConsumerWarps) {
        const float sc = row_scale[m];
        float ss = 0.f;
        for (int idx = lane; idx < cnt; idx += 32) {
          const int n = n_begin + idx;
          float v = cta_out[(size_t)m * rows_cap + idx] * sc;
          if (a.bias) v += __bfloat162float(a.bias[n]);
          if (a.res) v += a.res[(size_t)m * a.ldr + n];
          a.out[(size_t)m * a.ldo + n] = v;
          ss += v * v;
          if (a.out_hi) {
            const float gv = a.gain_next ? v * __bfloat162float(a.gain_next[n]) : v;
            split_store(a.out_hi + (size_t)m * a.ld_plane + n, a.out_lo + (size_t)m * a.ld_plane + n, gv);
          }
        }
        ss = warp_sum(ss);
        if (a.ssq_out && lane == 0) a.ssq_out[(size_t)blockIdx.x * a.M + m] = ss;
      }
    } else if (ok && EPI == EPI_SWIGLU) {
      for (int e = tid; e < a.M * cnt; e += kConsumerThreads) {
        const int m = e / cnt, idx = e - m * cnt, n = n_begin + idx;
        const float sc = row_scale[m];
        const float gv = cta_out[(size_t)m * rows_cap + idx] * sc;
        const float uv = cta_out[(size_t)m * rows_cap + rows_half + idx] * sc;
        const float act = gv / (1.f + __expf(-gv)) * uv;
        if (a.out) a.out[(size_t)m * a.ldo + n] = act;
        split_store(a.out_hi + (size_t)m * a.ld_plane + n, a.out_lo + (size_t)m * a.ld_plane + n, act);
      }
    } else if (ok && EPI == EPI_LMHEAD) {
      for (int e = tid; e < a.M * cnt; e += kConsumerThreads) {
        const int m = e / cnt, idx = e - m * cnt;
        const float v = cta_out[(size_t)m * rows_cap + idx] * row_scale[m];
        cta_out[(size_t)m * rows_cap + idx] = v;
        if (a.logits_out) a.logits_out[(size_t)m * a.N + n_begin + idx] = v;
      }
    }
    if (EPI == EPI_LMHEAD) {
      consumer_sync();
      // per-row summary of this CTA's vocabulary range: warp per row m
      for (int m = warp; m < a.M && ok; m += kConsumerWarps) {
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

template <bool GATHER, int EPI>
ps_status launch_gemm(ps_ctx* c, GemmArgs& a, cudaStream_t st) {
  const int n_cta = c->n_sm;
  const int smem_limit = c->smem_optin;
  a.rows_cap = rows_cap_for(a.N, n_cta, a.rs.zip != 0);
  a.pass_cols = choose_pass_cols(a.M, a.K, a.rows_cap, smem_limit);
  if (a.pass_cols == 0) return fail(c, PS_ERR_UNSUPPORTED, "activation operand does not fit shared memory");
  Layout L = make_layout(a.M, std::min(a.pass_cols, a.K), a.rows_cap, smem_limit);
  a.status = c->dev_status;
  auto kern = a.M > 8 ? k_ws_gemm<GATHER, EPI, 2> : k_ws_gemm<GATHER, EPI, 1>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_limit);
  if (e != cudaSuccess) return cuda_check(c, e, "ws_gemm smem attribute");
  kern<<<n_cta, kThreads, L.total, st>>>(a, smem_limit);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_ws_gemm");
}

struct Planes { __nv_bfloat16 *hi, *lo; };

struct FusedScratch {
  float* qkv; float* att_ml; float* att_o; float* act; LmPart* parts; unsigned* ticket;
  unsigned* attn_tickets;   // [PS_MAX_BATCH][n_heads]
  float* ssq[3];            // partial sums of squares of x0, a and hdn rows: [kMaxSm][kMaxM] each
  Planes x0p, ap, hdnp, attnp, actp;
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
  auto planes = [&](size_t width) {
    Planes p;
    p.hi = (__nv_bfloat16*)take((size_t)kMaxM * width * 2);
    p.lo = (__nv_bfloat16*)take((size_t)kMaxM * width * 2);
    return p;
  };
  FusedScratch s;
  s.qkv = (float*)take((size_t)kMaxM * (Hq + 2 * Hkv) * 4);
  s.att_ml = (float*)take((size_t)kMaxM * g.n_heads * kAttnMaxSplit * 2 * 4);
  s.att_o = (float*)take((size_t)kMaxM * g.n_heads * kAttnMaxSplit * g.head_dim * 4);
  s.act = (float*)take((size_t)kMaxM * g.ffn * 4);
  s.parts = (LmPart*)take((size_t)kMaxSm * kMaxM * sizeof(LmPart));
  s.ticket = (unsigned*)take(256);
  s.attn_tickets = (unsigned*)take((size_t)PS_MAX_BATCH * g.n_heads * 4);
  for (int i = 0; i < 3; ++i) s.ssq[i] = (float*)take((size_t)kMaxSm * kMaxM * 4);
  s.x0p = planes(g.hidden); s.ap = planes(g.hidden); s.hdnp = planes(g.hidden);
  s.attnp = planes(Hq); s.actp = planes(g.ffn);
  s.bytes = off;
  return s;
}

}  // namespace

bool fused_supported(const ps_ctx* c, int M) {
  const ps_config& g = c->cfg;
  if (g.dtype != PS_DTYPE_BF16 || (g.flags & PS_FLAG_UNFUSED_KERNELS)) return false;
  if (M > kMaxM || (g.head_dim != 64 && g.head_dim != 128)) return false;
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
            V = g.vocab, R = g.k_masks + 1, M = B * R;
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
    a.out_hi = f.x0p.hi; a.out_lo = f.x0p.lo; a.ld_plane = H; a.gain_next = (BP)w.g_in;
    if ((s = launch_gemm<true, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "fc_norm");
  {  // S2 q|k|v = W rms(x0)
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_q; a.rs.W[1] = (BP)w.w_k; a.rs.W[2] = (BP)w.w_v;
    a.rs.rows[0] = Hq; a.rs.rows[1] = Hkv; a.rs.rows[2] = Hkv; a.rs.n_mats = 3;
    a.N = Hq + 2 * Hkv; a.K = H; a.M = M;
    a.in_hi = f.x0p.hi; a.in_lo = f.x0p.lo; a.ld_in = H;
    a.ssq_in = f.ssq[0]; a.ssq_n = c->n_sm; a.eps = g.rms_eps;
    a.out = f.qkv; a.ldo = Hq + 2 * Hkv;
    if ((s = launch_gemm<false, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "qkv_rope");
  if ((s = launch_attn_split(c, sm, B, f.qkv, f.att_ml, f.att_o, f.attn_tickets, f.attnp.hi, f.attnp.lo, st)))
    return s;
  prof_mark(c, st, "attention");
  {  // S4 a = x0 + W_o attn
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_o; a.rs.rows[0] = H; a.rs.n_mats = 1;
    a.N = H; a.K = Hq; a.M = M;
    a.in_hi = f.attnp.hi; a.in_lo = f.attnp.lo; a.ld_in = Hq;
    a.out = c->a; a.ldo = H; a.res = c->x0; a.ldr = H;
    a.ssq_out = f.ssq[1];
    a.out_hi = f.ap.hi; a.out_lo = f.ap.lo; a.ld_plane = H; a.gain_next = (BP)w.g_post;
    if ((s = launch_gemm<false, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "o_proj");
  {  // S5a act = silu(W_g rms(a)) * (W_u rms(a))
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_gate; a.rs.W[1] = (BP)w.w_up; a.rs.rows[0] = F; a.rs.rows[1] = F;
    a.rs.n_mats = 2; a.rs.zip = 1;
    a.N = F; a.K = H; a.M = M;
    a.in_hi = f.ap.hi; a.in_lo = f.ap.lo; a.ld_in = H;
    a.ssq_in = f.ssq[1]; a.ssq_n = c->n_sm; a.eps = g.rms_eps;
    a.out = f.act; a.ldo = F;
    a.out_hi = f.actp.hi; a.out_lo = f.actp.lo; a.ld_plane = F;
    if ((s = launch_gemm<false, EPI_SWIGLU>(c, a, st))) return s;
  }
  float* hdn = feat_out ? feat_out : c->hdn;
  {  // S5b hdn = a + W_d act
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_down; a.rs.rows[0] = H; a.rs.n_mats = 1;
    a.N = H; a.K = F; a.M = M;
    a.in_hi = f.actp.hi; a.in_lo = f.actp.lo; a.ld_in = F;
    a.out = hdn; a.ldo = H; a.res = c->a; a.ldr = H;
    a.ssq_out = f.ssq[2];
    a.out_hi = f.hdnp.hi; a.out_lo = f.hdnp.lo; a.ld_plane = H; a.gain_next = (BP)w.g_final;
    if ((s = launch_gemm<false, EPI_STORE>(c, a, st))) return s;
  }
  prof_mark(c, st, "ffn");
  {  // S6 logits = W_lm rms(hdn), softmax statistics and top-n without a second pass over logits
    GemmArgs a{};
    a.rs.W[0] = (BP)w.w_lm; a.rs.rows[0] = V; a.rs.n_mats = 1;
    a.N = V; a.K = H; a.M = M;
    a.in_hi = f.hdnp.hi; a.in_lo = f.hdnp.lo; a.ld_in = H;
    a.ssq_in = f.ssq[2]; a.ssq_n = c->n_sm; a.eps = g.rms_eps;
    a.logits_out = logits_out; a.parts = f.parts; a.ticket = f.ticket;
    a.top_n = top_n; a.top_ids = top_ids; a.top_logit = top_logit; a.row_max = row_max; a.row_lse = row_lse;
    if ((s = launch_gemm<false, EPI_LMHEAD>(c, a, st))) return s;
  }
  prof_mark(c, st, "lm_head");
  return PS_OK;
}

}  // namespace ps
