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

#include "umma_gemm.cuh"
#include "ws_gemm.cuh"

namespace ps {
namespace {

using namespace ws;

enum Epi { EPI_STORE = 0, EPI_SWIGLU = 1, EPI_LMHEAD = 2 };

constexpr int kMaxM = 16;
constexpr int kTopMax = PS_MAX_TOP_N;

struct __align__(16) LmPart {  // softmax / top-n summary of one vocabulary range for one row
  float vmax, sumexp;
  float v0; int i0;          // copy of top_v[0], top_i[0]: the first 16 bytes decide a top-1 merge
  float top_v[kTopMax];
  int top_i[kTopMax];
  float sv; int si;          // draft sampling: best perturbed logit of the range and its token
  int pad_[2];
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
  // tensor-core path
  __nv_bfloat16* xin;       // [kMaxM][2H] gathered fc input (exact bf16: one plane)
  float* partials;          // [kMaxSm][2][16][128] partial tiles of CTAs that share a tile
  unsigned* tile_tickets;   // one per tile of the widest stage, zero between launches
  unsigned* chain_ctr;      // chained stages: finished-tile and passed-CTA counts, zero between launches
  int n_part_rows;          // rows of `parts` and of each ssq array
  size_t bytes;
};

// One carve-up for sizing (base == nullptr) and for use; always the largest row and CTA counts.
FusedScratch carve_fused(const ps_config& g, char* base) {
  constexpr int kRows = umma::kMaxRows;   // rows the tensor-core path can take (the mma.sync kernels: kMaxM)
  const size_t Hq = (size_t)g.n_heads * g.head_dim, Hkv = (size_t)g.n_kv_heads * g.head_dim;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off += (bytes + 255) & ~(size_t)255;
    return base ? base + at : nullptr;
  };
  auto planes = [&](size_t width) {
    Planes p;
    p.hi = (__nv_bfloat16*)take((size_t)kRows * width * 2);
    p.lo = (__nv_bfloat16*)take((size_t)kRows * width * 2);
    return p;
  };
  FusedScratch s;
  s.qkv = (float*)take((size_t)kRows * (Hq + 2 * Hkv) * 4);
  // (rows x splits is bounded: the attention launcher takes fewer splits when there are more rows)
  s.att_ml = (float*)take((size_t)kMaxM * g.n_heads * kAttnMaxSplit * 2 * 4);
  s.att_o = (float*)take((size_t)kMaxM * g.n_heads * kAttnMaxSplit * g.head_dim * 4);
  s.act = (float*)take((size_t)kRows * g.ffn * 4);
  // per-CTA (mma.sync path) or per-tile (tensor-core path) summaries
  const int tiles_v = (g.vocab + 127) / 128, tiles_h = (g.hidden + 127) / 128;
  s.n_part_rows = std::max(kMaxSm, std::max(tiles_v, tiles_h));
  s.parts = (LmPart*)take((size_t)s.n_part_rows * kRows * sizeof(LmPart));
  s.ticket = (unsigned*)take(256);
  s.attn_tickets = (unsigned*)take((size_t)PS_MAX_BATCH * g.n_heads * 4);
  for (int i = 0; i < 3; ++i) s.ssq[i] = (float*)take((size_t)s.n_part_rows * kRows * 4);
  s.xin = (__nv_bfloat16*)take((size_t)kRows * 2 * g.hidden * 2);
  s.partials = (float*)take((size_t)kMaxSm * 2 * kRows * 128 * 4);
  const size_t max_tiles = std::max<size_t>({(size_t)tiles_v, (size_t)(g.ffn + 63) / 64,
                                             (Hq + 127) / 128 + 2 * ((Hkv + 127) / 128), (size_t)tiles_h});
  s.tile_tickets = (unsigned*)take(max_tiles * 4);
  s.chain_ctr = (unsigned*)take(256);
  s.x0p = planes(g.hidden); s.ap = planes(g.hidden); s.hdnp = planes(g.hidden);
  s.attnp = planes(Hq); s.actp = planes(g.ffn);
  s.bytes = off;
  return s;
}


// =============================================================================================
// Tensor-core path (tcgen05 + tiled TMA), see umma_gemm.cuh
// =============================================================================================
struct UArgs {
  int N, K, M;
  int Mp;                  // M padded to 16, 32, 48, 64, 96 or 128: rows of a plane box, half the MMA's N
  int n_tiles, KB;         // tiles of 128 weight rows (64 features when zipped), k-blocks of 64
  int split;               // blocks a tile's k range is dealt in, 1..KB (see cta_begin)
  int zip;                 // 1: a tile is 64 rows of matrix 0 (gate) over 64 rows of matrix 1 (up)
  int lo;                  // 0: the activation operand is exact bf16 (no lo plane)
  int n_mats;              // concatenated matrices (q|k|v): tiles never straddle two of them
  int mat_tiles[3], mat_rows[3], mat_off[3];
  const float* ssq_in; int ssq_n; float eps;
  float* out; int ldo;
  const __nv_bfloat16* bias;
  const float* res; int ldr;
  float* ssq_out;          // [n_tiles][M]
  __nv_bfloat16 *out_hi, *out_lo; int ld_plane;
  const __nv_bfloat16* gain_next;
  float* logits_out; LmPart* parts; unsigned* ticket;
  int top_n; int* top_ids; float* top_logit; float* row_max; float* row_lse;
  float* partials; unsigned* tile_tickets;
  int sample; SampleArgs sa; int R;   // draft sampling in the LM head (sample != 0), rows per sequence
  int* status;
};

// CTA that owns unit u when CTA c owns [U c / G, U (c+1) / G).
// (Unit counts are small enough for 32-bit arithmetic: the launcher checks U * (G + 1) < 2^31.)
__device__ __forceinline__ int unit_owner(int u, int U, int G) {
  return (int)(((unsigned)(u + 1) * (unsigned)G - 1u) / (unsigned)U);
}
__device__ __forceinline__ int unit_begin(int c, int U, int G) {
  return (int)((unsigned)U * (unsigned)c / (unsigned)G);
}
// Units are dealt in blocks: the KB k-blocks of a tile are cut into a.split contiguous blocks
// (block j of a tile starts at its k-block j KB / split) and CTA c owns blocks
// [S c / G, S (c+1) / G) of the S = n_tiles * split blocks.  split = KB deals single units
// (every CTA streams the same bytes: the choice for few activation rows, where streaming is
// all that counts); split = 1 deals whole tiles (no tile is shared, nothing to reduce: the
// choice once a tile's epilogue and reduction cost more than an uneven load).
__device__ __forceinline__ int block_first_unit(const UArgs& a, int x) {
  const int t = x / a.split, j = x - t * a.split;
  return t * a.KB + (j * a.KB) / a.split;
}
__device__ __forceinline__ int cta_begin(const UArgs& a, int c, int G) {
  return block_first_unit(a, unit_begin(c, a.n_tiles * a.split, G));
}
__device__ __forceinline__ int cta_of_unit(const UArgs& a, int u, int G) {
  const int t = u / a.KB, w = u - t * a.KB;
  return unit_owner(t * a.split + ((w + 1) * a.split - 1) / a.KB, a.n_tiles * a.split, G);
}

// The tiles a CTA's unit range [u0, u1) touches, in the order the CTA works through them.  A
// range that ends inside a tile starts with that tail: the tiles a CTA shares with its
// neighbours are then reduced while the rest of its range still streams, and the last thing it
// does is a tile of its own.
struct Segs {
  int u0, u1, KB, t0, n, tail_first;
  __device__ Segs(int u0_, int u1_, int KB_) : u0(u0_), u1(u1_), KB(KB_) {
    t0 = u0 / KB;
    n = u1 > u0 ? (u1 - 1) / KB - t0 + 1 : 0;
    tail_first = n > 1 && (u1 % KB) != 0;
  }
  // i-th segment in working order: units [b, e) of tile t
  __device__ void get(int i, int& t, int& b, int& e) const {
    const int k = tail_first ? (i == 0 ? n - 1 : i - 1) : i;
    t = t0 + k;
    b = max(u0, t * KB);
    e = min(u1, (t + 1) * KB);
  }
};

// Walks a CTA's units in working order: the running tile t, its k-block kb, and the tile's
// matrix and first row.
struct UnitWalk {
  int si, t, kb, kb_end, mat, row0;
  __device__ void enter(const Segs& s, const UArgs& a) {
    int b, e;
    s.get(si, t, b, e);
    kb = b - t * a.KB;
    kb_end = e - t * a.KB;
    mat = 0;
    row0 = t * 64;
    if (!a.zip) {
      int tl = t;
      while (mat + 1 < a.n_mats && tl >= a.mat_tiles[mat]) { tl -= a.mat_tiles[mat]; ++mat; }
      row0 = tl * umma::kTile;
    }
  }
  __device__ void start(const Segs& s, const UArgs& a) {
    si = 0;
    if (s.n > 0) enter(s, a);
  }
  __device__ void next(const Segs& s, const UArgs& a) {
    if (++kb == kb_end && ++si < s.n) enter(s, a);
  }
};

// Feature of accumulator row r of tile t; valid = false for rows past the end of a matrix.
__device__ __forceinline__ int tile_feature(const UArgs& a, int t, int r, bool& valid) {
  if (a.zip) {
    const int f = t * 64 + (r & 63);
    valid = f < a.N;
    return f;
  }
  int m = 0;
  while (m + 1 < a.n_mats && t >= a.mat_tiles[m]) {
    t -= a.mat_tiles[m];
    ++m;
  }
  const int local = t * umma::kTile + r;
  valid = local < a.mat_rows[m];
  return a.mat_off[m] + local;
}

// Epilogue of one finished tile for the activation rows [m0, m0 + mc), mc <= 16; called by the
// 128 epilogue threads after each has put its accumulator row r (= 32 * q + lane) of those
// rows into ctl.acc[(m - m0) * 128 + r].  A dry call executes the same instructions and writes
// nothing to global memory.  res_pre: the caller has put the rows' residual values into
// ctl.land[m * 128 + r] already (m0 = 0).  With UNR = 1
// the loops over m are rolled on purpose: for up to 16 rows this code runs once or twice per
// CTA, so what it costs is the fetch of its instructions, not their execution.  With more rows
// it runs once per 16 rows of every tile and its single warp per scheduler is bound by the
// latency of dependent instructions: UNR = 4 interleaves four rows.
template <int EPI, int UNR>
__device__ __forceinline__ void tile_epilogue(const UArgs& a, umma::Ctl& ctl, int t, int r, int q, int lane,
                                              int m0, int mc, bool dry, bool res_pre = false) {
  using namespace umma;
  const int et = r;
  bool valid;
  const int n = tile_feature(a, t, r, valid);
  const float* acc = ctl.acc + r;
  if (EPI == EPI_STORE) {
    const float bias = (a.bias && valid) ? __bfloat162float(a.bias[n]) : 0.f;
    const float gain = (a.gain_next && valid) ? __bfloat162float(a.gain_next[n]) : 1.f;
    // eight rows at a time, so that their residual loads are in flight together
#pragma unroll 1
    for (int mg = 0; mg < mc; mg += 8) {
      float rv[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        rv[j] = (a.res && valid && mg + j < mc)
                    ? (res_pre ? ctl.land[(mg + j) * 128 + r] : __ldcg(a.res + (size_t)(m0 + mg + j) * a.ldr + n))
                    : 0.f;
      float sq[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int m = mg + j;
        sq[j] = 0.f;
        if (m < mc) {   // uniform across the threads
          if (valid && !dry) {
            const float x = acc[m * 128] * ctl.scale[m0 + m] + bias + rv[j];
            a.out[(size_t)(m0 + m) * a.ldo + n] = x;
            sq[j] = x * x;
            if (a.out_hi)
              split_store(a.out_hi + (size_t)(m0 + m) * a.ld_plane + n, a.out_lo + (size_t)(m0 + m) * a.ld_plane + n, x * gain);
          }
        }
      }
      if (a.ssq_out) {   // the eight rows' warp sums side by side (same tree as warp_sum)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
          for (int j = 0; j < 8; ++j) sq[j] += __shfl_xor_sync(0xffffffffu, sq[j], o);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (lane == 0 && mg + j < mc) ctl.red[q][mg + j] = sq[j];
      }
    }
    if (a.ssq_out) {
      epi_sync();
      if (et < mc && !dry) a.ssq_out[(size_t)t * a.M + m0 + et] = (ctl.red[0][et] + ctl.red[1][et]) + (ctl.red[2][et] + ctl.red[3][et]);
      epi_sync();
    }
  } else if (EPI == EPI_SWIGLU) {
    if (r >= 64) {
#pragma unroll UNR
      for (int m = 0; m < mc; ++m) ctl.xch[m * 64 + (r - 64)] = acc[m * 128] * ctl.scale[m0 + m];
    }
    epi_sync();
    if (r < 64 && valid && !dry) {
#pragma unroll UNR
      for (int m = 0; m < mc; ++m) {
        const float gv = acc[m * 128] * ctl.scale[m0 + m], uv = ctl.xch[m * 64 + r];
        const float act = gv / (1.f + __expf(-gv)) * uv;
        if (a.out) a.out[(size_t)(m0 + m) * a.ldo + n] = act;
        split_store(a.out_hi + (size_t)(m0 + m) * a.ld_plane + n, a.out_lo + (size_t)(m0 + m) * a.ld_plane + n, act);
      }
    }
    epi_sync();
  } else {  // EPI_LMHEAD: logits, and the tile's softmax / top-n summary per row
#pragma unroll UNR
    for (int m = 0; m < mc; ++m) {
      const float x = acc[m * 128] * ctl.scale[m0 + m];
      if (valid && a.logits_out && !dry) a.logits_out[(size_t)(m0 + m) * a.N + n] = x;
      float mx = valid ? x : -FLT_MAX;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      if (lane == 0) ctl.red[q][m] = mx;
    }
    epi_sync();
#pragma unroll UNR
    for (int m = 0; m < mc; ++m) {
      const float bmax = fmaxf(fmaxf(ctl.red[0][m], ctl.red[1][m]), fmaxf(ctl.red[2][m], ctl.red[3][m]));
      const float s = warp_sum(valid ? __expf(acc[m * 128] * ctl.scale[m0 + m] - bmax) : 0.f);
      if (lane == 0) ctl.red2[q][m] = s;
    }
    epi_sync();
    if (et < mc && !dry) {
      LmPart* p = a.parts + (size_t)t * a.M + m0 + et;
      p->vmax = fmaxf(fmaxf(ctl.red[0][et], ctl.red[1][et]), fmaxf(ctl.red[2][et], ctl.red[3][et]));
      p->sumexp = (ctl.red2[0][et] + ctl.red2[1][et]) + (ctl.red2[2][et] + ctl.red2[3][et]);
    }
    // top-n per row: repeated block arg-max over the values after the previous pick
#pragma unroll 1
    for (int tn = 0; tn < a.top_n; ++tn) {
#pragma unroll UNR
      for (int m = 0; m < mc; ++m) {
        const float x = acc[m * 128] * ctl.scale[m0 + m];
        const float pv = tn ? ctl.prev_v[m] : FLT_MAX;
        const int pi = tn ? ctl.prev_i[m] : -1;
        const bool after = valid && ((x < pv) || (x == pv && n > pi));
        float bv = after ? x : -FLT_MAX;
        int bi = after ? n : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { ctl.cand_v[q][m] = bv; ctl.cand_i[q][m] = bi; }
      }
      epi_sync();
      if (et < mc) {
        float bv = ctl.cand_v[0][et]; int bi = ctl.cand_i[0][et];
#pragma unroll
        for (int w = 1; w < 4; ++w) {
          const float ov = ctl.cand_v[w][et]; const int oi = ctl.cand_i[w][et];
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        ctl.prev_v[et] = bv; ctl.prev_i[et] = bi;
        if (!dry) {
          LmPart* p = a.parts + (size_t)t * a.M + m0 + et;
          p->top_v[tn] = bv; p->top_i[tn] = bi;
          if (tn == 0) { p->v0 = bv; p->i0 = bi; }
        }
      }
      epi_sync();
    }
    if (a.sample) {   // Gumbel-max candidate of this vocabulary range per row
#pragma unroll UNR
      for (int m = 0; m < mc; ++m) {
        const int sb = (m0 + m) / a.R;
        const uint32_t row_id = ((uint32_t)sb + a.sa.b_base) | ((uint32_t)(m0 + m - sb * a.R) << 8);
        float bv = -FLT_MAX;
        int bi = 0x7fffffff;
        if (valid) {
          bv = acc[m * 128] * ctl.scale[m0 + m] * a.sa.inv_temp + gumbel_noise(a.sa, (uint32_t)n, row_id);
          bi = n;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { ctl.cand_v[q][m] = bv; ctl.cand_i[q][m] = bi; }
      }
      epi_sync();
      if (et < mc) {
        float bv = ctl.cand_v[0][et]; int bi = ctl.cand_i[0][et];
#pragma unroll
        for (int w = 1; w < 4; ++w) {
          const float ov = ctl.cand_v[w][et]; const int oi = ctl.cand_i[w][et];
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (!dry) {
          LmPart* p = a.parts + (size_t)t * a.M + m0 + et;
          p->sv = bv; p->si = bi;
        }
      }
    }
    epi_sync();   // red / red2 / cand are free again
  }
}

// Epilogue of 16 activation rows [m0, m0 + mc) of a tile for launches of more than 16 rows
// (EPI_STORE and EPI_SWIGLU): the thread of accumulator row r holds the rows' sums in v[] (no
// detour through shared memory) and their residual values in rv[] (loaded by the caller before the
// sums were ready).  With that many rows the epilogue runs eight times per tile and is what a
// launch costs beyond its weight stream, so the per-row work is kept free of cross-lane steps:
// the rows' sums of squares go through a [16][128] tile in shared memory (ctl.acc) and are added
// by 8 threads per row, instead of a shuffle reduction per row and warp.
template <int EPI>
__device__ __forceinline__ void big_chunk_epilogue(const UArgs& a, umma::Ctl& ctl, int n, bool valid, int pidx, int r,
                                                   int m0, int mc, const float (&v)[16], float bias, float gain,
                                                   const float (&rv)[16], bool dry) {
  using namespace umma;
  constexpr int kSqLd = 132;   // row pitch of the squares' tile: the 8 x 4 threads of a warp read different banks
  static_assert(16 * kSqLd <= 2 * kN * 128, "the squares' tile fits ctl.acc + ctl.land");
  if (EPI == EPI_STORE) {
    float sq[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      sq[j] = 0.f;
      if (j < mc && valid) {
        const float x = v[j] * ctl.scale[m0 + j] + bias + rv[j];
        sq[j] = x * x;
        if (!dry) {
          a.out[(size_t)(m0 + j) * a.ldo + n] = x;
          if (a.out_hi)
            split_store(a.out_hi + (size_t)(m0 + j) * a.ld_plane + n, a.out_lo + (size_t)(m0 + j) * a.ld_plane + n, x * gain);
        }
      }
    }
    if (a.ssq_out) {
#pragma unroll
      for (int j = 0; j < 16; ++j) ctl.acc[j * kSqLd + r] = sq[j];   // (runs on into ctl.land, unused here)
      epi_sync();
      const int row = r >> 3, part = r & 7;   // 8 threads per row, every 8th feature each
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < 16; ++i) sum += ctl.acc[row * kSqLd + i * 8 + part];
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      sum += __shfl_xor_sync(0xffffffffu, sum, 4);
      if (part == 0 && row < mc && !dry) a.ssq_out[(size_t)pidx * a.M + m0 + row] = sum;
      epi_sync();
    }
  } else {   // EPI_SWIGLU: rows 0..63 of the tile are gate features, rows 64..127 the same features of up
    if (r >= 64) {
#pragma unroll
      for (int j = 0; j < 16; ++j) ctl.xch[j * 64 + (r - 64)] = v[j] * ctl.scale[min(m0 + j, kMaxRows - 1)];
    }
    epi_sync();
    if (r < 64 && valid && !dry) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (j < mc) {
          const float gv = v[j] * ctl.scale[m0 + j], uv = ctl.xch[j * 64 + r];
          const float act = gv / (1.f + __expf(-gv)) * uv;
          if (a.out) a.out[(size_t)(m0 + j) * a.ldo + n] = act;
          split_store(a.out_hi + (size_t)(m0 + j) * a.ld_plane + n, a.out_lo + (size_t)(m0 + j) * a.ld_plane + n, act);
        }
      }
    }
    epi_sync();
  }
}

// Last step of an LM-head launch, called by all threads of every CTA after its tiles are done:
// the last CTA to finish merges the per-tile summaries (no CTA waits for another).  It runs
// once, after everything else, so what it costs is round trips to L2 and the fetch of its own
// instructions: the summaries of as many rows as fit come into the (idle) ring by asynchronous
// 16-byte copies in one round trip, then a warp per row reduces them in small rolled loops.
__device__ __forceinline__ void lm_merge(const UArgs& a, umma::Ctl& ctl, unsigned char* ring, int tid, int warp,
                                         int lane) {
  if (tid == 0) {
    __threadfence();
    const unsigned tk = atomicAdd(a.ticket, 1u);
    ctl.is_last = (tk == gridDim.x - 1);
    if (ctl.is_last) __threadfence();
  }
  __syncthreads();
  if (ctl.is_last && !ctl.abort_flag) {
    const int Gt = a.n_tiles;
    static_assert(offsetof(LmPart, sv) % 16 == 0, "the sample pair starts a 16-byte group");
    const int rows_pass = max(1, min(a.M, umma::kRingBytes / (Gt * 32)));
    float4* s_h = reinterpret_cast<float4*>(ring);   // [rows of a pass][Gt]: vmax, sumexp, v0, i0
    float4* s_s = s_h + rows_pass * Gt;              // [rows of a pass][Gt]: sv, si
    for (int m0 = 0; m0 < a.M; m0 += rows_pass) {
      const int nr = min(rows_pass, a.M - m0);
      for (int mr = 0; mr < nr; ++mr) {
        for (int c = tid; c < Gt; c += umma::kThreads) {
          const LmPart* e = a.parts + (size_t)c * a.M + m0 + mr;
          umma::cp_async_16(s_h + mr * Gt + c, e);
          if (a.sample) umma::cp_async_16(s_s + mr * Gt + c, &e->sv);
        }
      }
      umma::cp_async_wait_all();
      __syncthreads();
      for (int mr = warp; mr < nr; mr += umma::kThreads / 32) {
        const int m = m0 + mr;
        const float4* H = s_h + mr * Gt;
        float mx = -FLT_MAX;
        float bv0 = -FLT_MAX; int bi0 = 0x7fffffff;   // the row's arg-max: the tiles' best tokens decide it
        for (int c = lane; c < Gt; c += 32) {
          const float4 hd = H[c];
          mx = fmaxf(mx, hd.x);
          const int ti = __float_as_int(hd.w);
          if (a.top_n > 0 && (hd.z > bv0 || (hd.z == bv0 && ti < bi0))) { bv0 = hd.z; bi0 = ti; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float add = 0.f;
        for (int c = lane; c < Gt; c += 32) add += H[c].y * __expf(H[c].x - mx);
        const float se = warp_sum(add);
        if (lane == 0) {
          if (a.row_max) a.row_max[m] = mx;
          if (a.row_lse) a.row_lse[m] = mx + logf(se);
        }
        const LmPart* P = a.parts + m;
        float pv = FLT_MAX; int pi = -1;
        for (int tn = 0; tn < a.top_n; ++tn) {
          float bv = bv0; int bi = bi0;
          if (tn > 0) {   // deeper picks: a tile's list is sorted, any of its entries may be next
            bv = -FLT_MAX; bi = 0x7fffffff;
            for (int k = 0; k < a.top_n; ++k) {
              for (int c0 = 0; c0 < Gt; c0 += 256) {
                float xv[8]; int id[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const int c = c0 + lane + 32 * j;
                  xv[j] = c < Gt ? __ldcg(&P[(size_t)c * a.M].top_v[k]) : 0.f;
                  id[j] = c < Gt ? __ldcg(&P[(size_t)c * a.M].top_i[k]) : 0x7fffffff;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const bool after = id[j] != 0x7fffffff && ((xv[j] < pv) || (xv[j] == pv && id[j] > pi));
                  if (after && (xv[j] > bv || (xv[j] == bv && id[j] < bi))) { bv = xv[j]; bi = id[j]; }
                }
              }
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          if (lane == 0) { a.top_ids[(size_t)m * a.top_n + tn] = bi; a.top_logit[(size_t)m * a.top_n + tn] = bv; }
          pv = bv; pi = bi;
        }
        if (a.sample) {   // the row's sampled token: arg-max of the ranges' perturbed maxima
          const float4* S = s_s + mr * Gt;
          float bv = -FLT_MAX; int bi = 0x7fffffff;
          for (int c = lane; c < Gt; c += 32) {
            const float xv = S[c].x;
            const int id = __float_as_int(S[c].y);
            if (xv > bv || (xv == bv && id < bi)) { bv = xv; bi = id; }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          if (lane == 0) a.sa.sampled[m] = bi;
        }
      }
      __syncthreads();   // the next pass overwrites the ring
    }
  }
  if (ctl.is_last && tid == 0) *a.ticket = 0u;
  __syncthreads();
}

static_assert(umma::kMaxCtas >= kMaxSm, "contributor table covers every CTA of a launch");

template <int EPI, int MP>
__global__ void __launch_bounds__(umma::kThreads, 1)
k_umma_gemm(const __grid_constant__ CUtensorMap tA0, const __grid_constant__ CUtensorMap tA1,
            const __grid_constant__ CUtensorMap tA2, const __grid_constant__ CUtensorMap tBh,
            const __grid_constant__ CUtensorMap tBl, UArgs a) {
  using namespace umma;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;             // shared-space address of stage 0
  unsigned char* stages = smem_raw + (base - raw);
  Ctl& ctl = *reinterpret_cast<Ctl*>(stages + kStages * kStageBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(&ctl.full[i], 1); mbar_init(&ctl.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&ctl.acc_full[i], 1); mbar_init(&ctl.acc_empty[i], kEpiThreads); }
    ctl.abort_flag = 0; ctl.is_last = 0; ctl.tile_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_launch_dependents();
  }
  if (warp == 1) {   // tensor memory for two accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                 "r"(tmem_cols(MP))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = *(volatile uint32_t*)&ctl.tmem_base;

  const int G = gridDim.x, U = a.n_tiles * a.KB;
  // (up to 16 rows single units are dealt: split = KB, and the block arithmetic drops out)
  auto begin_of = [&](int c) { return MP <= 16 ? unit_begin(c, U, G) : cta_begin(a, c, G); };
  auto owner_of = [&](int u) { return MP <= 16 ? unit_owner(u, U, G) : cta_of_unit(a, u, G); };
  const int u0 = begin_of(blockIdx.x), u1 = begin_of(blockIdx.x + 1);
  const Segs segs(u0, u1, a.KB);
  volatile int* abort_flag = &ctl.abort_flag;
  constexpr int Mp = MP, sbytes = stage_bytes(Mp), nst = n_stages(Mp), ksplit = k_split(Mp), acols = acc_cols(Mp);
  constexpr int plane_bytes = Mp * kBK * 2;

  if (warp == 0) {
    if (lane == 0) {   // ---- TMA producer
      const uint32_t bytes = kABytes + plane_bytes * (a.lo ? 2 : 1);
      // The weights do not depend on the kernel before this one, its activations do: the
      // weight boxes of the first kStages units are requested first, then the thread waits for
      // that kernel and adds their activation boxes.
      const int n_units = u1 - u0, n_early = min(nst, n_units);
      UnitWalk w;
      auto load_a = [&](const UnitWalk& uw, int st_i) {
        const uint32_t dst = base + st_i * sbytes;
        const int x = uw.kb * kBK;
        mbar_arrive_expect_tx(&ctl.full[st_i], bytes);
        if (a.zip) {
          tma_load_2d(dst, &tA0, x, uw.row0, &ctl.full[st_i]);
          tma_load_2d(dst + kABytes / 2, &tA1, x, uw.row0, &ctl.full[st_i]);
        } else {
          tma_load_2d(dst, uw.mat == 0 ? &tA0 : (uw.mat == 1 ? &tA1 : &tA2), x, uw.row0, &ctl.full[st_i]);
        }
      };
      auto load_b = [&](const UnitWalk& uw, int st_i) {
        const uint32_t dst = base + st_i * sbytes + kABytes;
        const int x = uw.kb * kBK;
        tma_load_2d(dst, &tBh, x, 0, &ctl.full[st_i]);
        if (a.lo) tma_load_2d(dst + plane_bytes, &tBl, x, 0, &ctl.full[st_i]);
      };
      w.start(segs, a);
      for (int i = 0; i < n_early; ++i) { load_a(w, i); w.next(segs, a); }
      pdl_wait();
      w.start(segs, a);
      for (int i = 0; i < n_early; ++i) { load_b(w, i); w.next(segs, a); }
      int stage = 0;
      uint32_t parity = 0;   // second use of a stage: its first release
      for (int i = n_early; i < n_units; ++i) {
        if (!mbar_wait(&ctl.empty[stage], parity, abort_flag)) break;
        load_a(w, stage);
        load_b(w, stage);
        w.next(segs, a);
        if (++stage == nst) { stage = 0; parity ^= 1; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---- MMA issuer
      int stage = 0;
      uint32_t parity = 0;
      bool alive = true;
      const uint32_t id = a.lo ? idesc(2 * Mp) : idesc(Mp);   // hi and lo planes as one operand of N = 2 Mp
      for (int si = 0; si < segs.n && alive; ++si) {
        int t, b, e;
        segs.get(si, t, b, e);
        const int buf = si & 1;
        if (!mbar_wait(&ctl.acc_empty[buf], ((si >> 1) & 1) ^ 1, abort_flag)) break;
        fence_after_sync();
        const uint32_t d = tmem + buf * acols;
        uint32_t acc = 0;
        for (int j = b; j < e; ++j) {
          if (!mbar_wait(&ctl.full[stage], parity, abort_flag)) { alive = false; break; }
          fence_after_sync();
          const uint32_t sa = base + stage * sbytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {   // k step k goes to accumulator k % ksplit
            const int ai = k & (ksplit - 1);   // ksplit is 1, 2 or 4
            mma_f16(d + ai * 2 * Mp, smem_desc(sa + k * 32), smem_desc(sa + kABytes + k * 32), id,
                    (acc || k >= ksplit) ? 1u : 0u);
          }
          acc = 1;
          mma_commit(&ctl.empty[stage]);
          if (++stage == nst) { stage = 0; parity ^= 1; }
        }
        if (alive) mma_commit(&ctl.acc_full[buf]);
      }
    }
  } else {
    // ---- epilogue warps: accumulator row r = 32 q + lane
    const int q = warp & 3, r = 32 * q + lane, et = r;
    // Pass -1 is a rehearsal: the reduction and epilogue code below runs once per CTA or
    // twice, at the very end for most CTAs, and its first execution costs several microseconds
    // of instruction fetches.  The rehearsal takes them before the kernel ahead of this one has
    // finished: it sums this CTA's own (stale) partial slot, runs the epilogue dry, and what it
    // reads may be in flux because nothing of it is kept.
    for (int seg = segs.n > 0 ? -1 : 0; seg < segs.n; ++seg) {
      const bool dry = seg < 0;
      if (seg == 0) {
        pdl_wait();   // everything below reads or writes what the kernel before this one touches
        if (MP <= 16) {
          for (int m = warp - 2; m < a.M; m += 4) {   // RMSNorm row scales of the input
            float sc = 1.f;
            if (a.ssq_in) {
              float ss = 0.f;
              for (int c = lane; c < a.ssq_n; c += 32) ss += a.ssq_in[(size_t)c * a.M + m];
              ss = warp_sum(ss);
              sc = rsqrtf(ss / (float)a.K + a.eps);
            }
            if (lane == 0) ctl.scale[m] = sc;
          }
        } else if (et < a.M) {   // many rows: one thread per row, its loads independent of each other
          float sc = 1.f;
          if (a.ssq_in) {
            float ss = 0.f;
#pragma unroll 8
            for (int c = 0; c < a.ssq_n; ++c) ss += a.ssq_in[(size_t)c * a.M + et];
            sc = rsqrtf(ss / (float)a.K + a.eps);
          }
          ctl.scale[et] = sc;
        }
        epi_sync();
      }
      int t, sb, se;
      segs.get(dry ? 0 : seg, t, sb, se);
      const int t_begin = t * a.KB, t_end = t_begin + a.KB;
      const bool whole = !dry && se - sb == a.KB;
      const int buf = seg & 1;
      // all four warps take the same decision although each thread waits for itself
      if (!dry && epi_any(!mbar_wait(&ctl.acc_full[buf], (seg >> 1) & 1, abort_flag))) break;
      fence_after_sync();
      const uint32_t ta = tmem + ((uint32_t)(32 * q) << 16) + buf * acols;
      // sums of activation rows [m0, m0 + 16) for accumulator row r: the ksplit accumulators and
      // their hi / lo halves added up
      auto load_chunk = [&](int m0, float (&v)[16]) {
        tmem_ld16(ta + m0, v);
#pragma unroll
        for (int c = 1; c < 2 * ksplit; ++c) {   // accumulator c / 2, its hi (even) or lo (odd) half
          if (!a.lo && (c & 1)) continue;
          float vp[16];
          tmem_ld16(ta + (c >> 1) * 2 * Mp + (c & 1) * Mp + m0, vp);
#pragma unroll
          for (int m = 0; m < 16; ++m) v[m] += vp[m];
        }
      };
      const int slot = (t == segs.t0) ? 0 : 1;   // partial tiles: 0 = this CTA's first segment, 1 = its last
      float* P = a.partials + ((size_t)blockIdx.x * 2 + slot) * kMaxRows * 128;
      bool finish = whole || dry;   // this CTA runs the tile's epilogue
      int c_first = blockIdx.x, c_last = blockIdx.x;
      // (launches of more than 16 rows keep a partial as [accumulator row][activation row]: a
      // thread writes and reads its 16 rows of a chunk as four 16-byte vectors)
      constexpr bool kBig = MP > 16 && EPI != EPI_LMHEAD;
      if (!whole && !dry) {
        for (int m0 = 0; m0 < a.M; m0 += 16) {
          float v[16];
          load_chunk(m0, v);
          if (kBig) {
            float4* d4 = reinterpret_cast<float4*>(P + (size_t)r * kMaxRows + m0);
            d4[0] = make_float4(v[0], v[1], v[2], v[3]);
            d4[1] = make_float4(v[4], v[5], v[6], v[7]);
            d4[2] = make_float4(v[8], v[9], v[10], v[11]);
            d4[3] = make_float4(v[12], v[13], v[14], v[15]);
          } else {
#pragma unroll
            for (int m = 0; m < 16; ++m)
              if (m0 + m < a.M) P[(m0 + m) * 128 + r] = v[m];
          }
        }
        fence_before_sync();
        mbar_arrive(&ctl.acc_empty[buf]);
        epi_sync();
        c_first = owner_of(t_begin);
        c_last = owner_of(t_end - 1);
        if (et == 0) {
          // one thread publishes the block's partial (the barrier above ordered the other
          // threads' stores before this release) and, if it came last, acquires the others'
          int n_contrib = 0;   // CTAs between the owners of the tile's ends that hold any unit
          for (int c = c_first; c <= c_last; ++c) n_contrib += begin_of(c) < begin_of(c + 1);
          unsigned old;
          asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(&a.tile_tickets[t]) : "memory");
          const int last = old == (unsigned)(n_contrib - 1);
          if (last) a.tile_tickets[t] = 0u;
          ctl.tile_last = last;
        }
        epi_sync();
        finish = ctl.tile_last != 0;
        epi_sync();   // everyone has read the flag before a later segment rewrites it
      }
      if (finish && !whole) {   // where each contributor's partial lies (a CTA without units has none)
        for (int j = et; j <= c_last - c_first; j += kEpiThreads) {
          const int c = c_first + j, cb = begin_of(c);
          int off = -1;
          if (cb < begin_of(c + 1)) {
            const int sl = (c == c_first && cb / a.KB != t) ? 1 : 0;
            off = (c * 2 + sl) * kMaxRows * 128;
          }
          ctl.coff[j] = off;
        }
        epi_sync();
      }
      if (finish && kBig) {
        // many rows: the sums stay in registers from tensor memory (or from the partials, added in
        // CTA order with all of a contributor's vectors in flight together) to the stores
        bool valid;
        const int n = tile_feature(a, t, r, valid);
        const float bias = (EPI == EPI_STORE && a.bias && valid) ? __bfloat162float(a.bias[n]) : 0.f;
        const float gain = (EPI == EPI_STORE && a.gain_next && valid) ? __bfloat162float(a.gain_next[n]) : 1.f;
        const int nc = c_last - c_first + 1;
        const int m_end = dry ? min(a.M, 16) : a.M;   // the rehearsal takes one chunk
        for (int m0 = 0; m0 < m_end; m0 += 16) {
          const int mc = min(16, a.M - m0);
          float rv[16];
#pragma unroll
          for (int j = 0; j < 16; ++j)
            rv[j] = (EPI == EPI_STORE && a.res && valid && j < mc && !dry) ? __ldcg(a.res + (size_t)(m0 + j) * a.ldr + n) : 0.f;
          float v[16];
          if (whole) {
            load_chunk(m0, v);
            if (m0 + 16 >= a.M) {   // the accumulator is read: the MMA warp may reuse it
              fence_before_sync();
              mbar_arrive(&ctl.acc_empty[buf]);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0.f;
            const float* Pr = a.partials + (size_t)r * kMaxRows + m0;
#pragma unroll 1
            for (int j0 = 0; j0 < nc; j0 += 2) {   // two contributors' vectors in flight at a time
              const int o0 = ctl.coff[j0], o1 = j0 + 1 < nc ? ctl.coff[j0 + 1] : -1;
              float4 x0[4], x1[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                x0[i] = o0 >= 0 ? __ldcg(reinterpret_cast<const float4*>(Pr + o0) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                x1[i] = o1 >= 0 ? __ldcg(reinterpret_cast<const float4*>(Pr + o1) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
              }
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                v[4 * i] += x0[i].x; v[4 * i + 1] += x0[i].y; v[4 * i + 2] += x0[i].z; v[4 * i + 3] += x0[i].w;
              }
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                v[4 * i] += x1[i].x; v[4 * i + 1] += x1[i].y; v[4 * i + 2] += x1[i].z; v[4 * i + 3] += x1[i].w;
              }
            }
          }
          big_chunk_epilogue<EPI>(a, ctl, n, valid, t, r, m0, mc, v, bias, gain, rv, dry);
        }
      } else if (finish) {
        // 16 activation rows at a time: the tile's sums into ctl.acc (from tensor memory, or the
        // partials added in CTA order, which does not depend on who came last), then the epilogue
        const int m_end = dry ? min(a.M, 16) : a.M;   // the rehearsal takes one chunk
        for (int m0 = 0; m0 < m_end; m0 += 16) {
          const int mc = min(16, a.M - m0);
          if (whole) {
            float v[16];
            load_chunk(m0, v);
#pragma unroll
            for (int m = 0; m < 16; ++m) ctl.acc[m * 128 + r] = v[m];
            if (m0 + 16 >= a.M) {   // the accumulator is read: the MMA warp may reuse it
              fence_before_sync();
              mbar_arrive(&ctl.acc_empty[buf]);
            }
          } else {
            // (row, contributor) pairs in row-major order, kN at a time: a rolled loop sends
            // each pair's value on its way into shared memory (asynchronous copies, nothing
            // waits on a register), one wait, a rolled loop adds them up.  The values come from
            // L2 while the next launch's weight requests keep it busy, and the code runs once:
            // round trips and instruction fetches are what it costs.
            const int nc = c_last - c_first + 1, total = mc * nc;
            const float* Pr = a.partials + m0 * 128 + r;
            float* land = ctl.land + r;
            int m = 0, j = 0, mm = 0, jj = 0;
            float sum = 0.f;   // of row m so far, contributors in CTA order
#pragma unroll 1
            for (int i0 = 0; i0 < total; i0 += kN) {
              const int nb = min(kN, total - i0);
#pragma unroll 1
              for (int u = 0; u < nb; ++u) {
                const int o = ctl.coff[jj];
                if (o >= 0) cp_async_4(land + u * 128, Pr + o + mm * 128);
                else land[u * 128] = 0.f;
                if (++jj == nc) { jj = 0; ++mm; }
              }
              cp_async_wait_all();   // each thread reads back what it asked for itself
#pragma unroll 1
              for (int u = 0; u < nb; ++u) {
                sum += land[u * 128];
                if (++j == nc) {
                  ctl.acc[m * 128 + r] = sum;
                  sum = 0.f; j = 0; ++m;
                }
              }
            }
          }
          tile_epilogue<EPI, (MP > 16 ? 4 : 1)>(a, ctl, t, r, q, lane, m0, mc, dry);
        }
      }
    }
    fence_before_sync();
  }

  __syncthreads();
  if (EPI == EPI_LMHEAD) lm_merge(a, ctl, stages, tid, warp, lane);
  if (ctl.abort_flag) {
    // let copies and MMAs that are still in flight finish before shared and tensor memory go
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    if (tid == 0) atomicOr(a.status, kStatTimeout);
    __syncthreads();
  }
  if (warp == 1) {
    fence_after_sync();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols(MP)) : "memory");
  }
}

// ---- several GEMM stages in one launch (up to 16 activation rows) ---------------------------------
// Consecutive stages of the draft step (fc -> q|k|v, and o -> gate|up -> down -> LM head) run
// as one launch of one CTA per SM.  Between two launches the stream of weights stops: the ring
// drains, the blocks leave, the next launch's blocks arrive and start asking again.  Inside one
// launch the producer thread goes straight on to the next stage's weight boxes as ring slots
// come free, so the stream only stops when the ring is full of them and the stage's
// activations are not there yet.  A stage's activations are complete when all tiles of the
// stage before it have run their epilogue: every finisher adds one to a counter in global
// memory (release); the producer thread and one epilogue thread of every CTA wait for the count
// (acquire, bounded), and the last of them to see it complete zeroes it for the next launch.
// The CTAs wait for one another, so all must be resident at once: one CTA per SM, see the
// launch in run_stages; every wait is bounded.  The tail of a tile (partials out, count, sum of
// the partials, epilogue, release) is a chain of round trips to L2 and is what a stage costs
// beyond its stream.  The owner of a tile's last k-block is its finisher: the other
// contributors store their partial and count themselves in, one thread of the finisher waits
// for the count while its own sums stay in registers; partials are kept as 16-byte vectors per
// accumulator row so that the finisher has all contributors' values in flight at once, and
// what does not depend on the sums (who shares the tile, the residual rows) is fetched while
// the MMAs still run.
constexpr int kChainMax = 4, kChainMaps = 13;
struct ChainParams {
  int n;                                  // stages
  int epi[kChainMax];
  int map_a[kChainMax][3], map_bh[kChainMax], map_bl[kChainMax];   // indices into maps
  unsigned* done;                         // [kChainMax] tiles finished per stage, zero between launches
  unsigned* passed;                       // [kChainMax] CTAs that have seen the stage complete
  UArgs a[kChainMax];
  CUtensorMap maps[kChainMaps];
};
static_assert(sizeof(ChainParams) <= 4000, "kernel parameters");

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

template <int MP>
__global__ void __launch_bounds__(umma::kThreads, 1) k_umma_chain(const __grid_constant__ ChainParams p) {
  using namespace umma;
  static_assert(MP == 16, "chained stages take up to 16 rows");
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* stages = smem_raw + (base - raw);
  Ctl& ctl = *reinterpret_cast<Ctl*>(stages + kStages * kStageBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(&ctl.full[i], 1); mbar_init(&ctl.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&ctl.acc_full[i], 1); mbar_init(&ctl.acc_empty[i], kEpiThreads); }
    ctl.abort_flag = 0; ctl.is_last = 0; ctl.tile_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_launch_dependents();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                 "r"(tmem_cols(MP))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = *(volatile uint32_t*)&ctl.tmem_base;

  const int G = gridDim.x;
  volatile int* abort_flag = &ctl.abort_flag;
  constexpr int sbytes = stage_bytes(MP), nst = n_stages(MP), ksplit = k_split(MP), acols = acc_cols(MP);
  constexpr int plane_bytes = MP * kBK * 2;
  auto stage_segs = [&](const UArgs& a) {
    const int U = a.n_tiles * a.KB;
    return Segs(unit_begin(blockIdx.x, U, G), unit_begin(blockIdx.x + 1, U, G), a.KB);
  };

  if (warp == 0) {
    if (lane == 0) {   // ---- TMA producer
      // Ring position g counts this CTA's units over all stages: unit g goes to slot g % nst and
      // is the slot's use number g / nst.  Two cursors per stage: weight boxes are requested as
      // soon as a slot is free, activation boxes follow once the stage before is complete.
      int sa = 0;                    // ring position of the next weight request: slot and use number
      uint32_t ua = 0;
      bool alive = true;
      for (int s = 0; s < p.n && alive; ++s) {
        const UArgs& a = p.a[s];
        const Segs segs = stage_segs(a);
        const int n_units = segs.u1 - segs.u0;
        bool seen_done = false;   // this thread has seen the count of the stage before complete
        if (s == 0 && n_units <= 0) pdl_wait();
        const uint32_t bytes = kABytes + plane_bytes * (a.lo ? 2 : 1);
        const CUtensorMap *tA0 = &p.maps[p.map_a[s][0]], *tA1 = &p.maps[p.map_a[s][1]], *tA2 = &p.maps[p.map_a[s][2]];
        const CUtensorMap *tBh = &p.maps[p.map_bh[s]], *tBl = &p.maps[p.map_bl[s]];
        UnitWalk wa, wb;
        wa.start(segs, a);
        wb.start(segs, a);
        int ia = 0, ib = 0, sb = sa;   // (sb: slot of the next activation request)
        bool dep_ok = false;
        long long t0 = 0;
        while (ib < n_units) {
          bool moved = false;
          if (ia < n_units && (ua == 0 || mbar_peek(&ctl.empty[sa], (ua & 1) ^ 1))) {
            const uint32_t dst = base + sa * sbytes;
            const int x = wa.kb * kBK;
            mbar_arrive_expect_tx(&ctl.full[sa], bytes);
            if (a.zip) {
              tma_load_2d(dst, tA0, x, wa.row0, &ctl.full[sa]);
              tma_load_2d(dst + kABytes / 2, tA1, x, wa.row0, &ctl.full[sa]);
            } else {
              tma_load_2d(dst, wa.mat == 0 ? tA0 : (wa.mat == 1 ? tA1 : tA2), x, wa.row0, &ctl.full[sa]);
            }
            wa.next(segs, a);
            ++ia;
            if (++sa == nst) { sa = 0; ++ua; }
            moved = true;
          }
          if (dep_ok) {
            if (ib < ia) {
              const uint32_t dst = base + sb * sbytes + kABytes;
              const int x = wb.kb * kBK;
              tma_load_2d(dst, tBh, x, 0, &ctl.full[sb]);
              if (a.lo) tma_load_2d(dst + plane_bytes, tBl, x, 0, &ctl.full[sb]);
              wb.next(segs, a);
              ++ib;
              if (++sb == nst) sb = 0;
              moved = true;
            }
          } else if (s == 0) {
            if (!moved) {   // the first stage's weight requests fill the ring, then the kernel before this one
              pdl_wait();
              dep_ok = true;
              moved = true;
            }
          } else if (ld_acquire_u32(p.done + (s - 1)) >= (unsigned)p.a[s - 1].n_tiles) {
            fence_proxy_async();   // what other SMs wrote is read by the copy engine from here on
            dep_ok = true;
            seen_done = true;
            moved = true;
          }
          if (!moved) {
            if (dep_ok) {   // every request made, the ring is full: wait for the slot
              if (!mbar_wait(&ctl.empty[sa], (ua & 1) ^ 1, abort_flag)) { alive = false; break; }
            } else {
              if (t0 == 0) t0 = clock64();
              if (*abort_flag || clock64() - t0 > ws::kWaitCycles) { *abort_flag = 1; alive = false; break; }
            }
          }
        }
        // both this thread and the epilogue warps' poller check in on every count, also a CTA
        // without units: the last of the 2 G to do so zeroes it
        if (s > 0 && alive) {
          if (!seen_done) {
            const long long t1 = clock64();
            while (ld_acquire_u32(p.done + (s - 1)) < (unsigned)p.a[s - 1].n_tiles) {
              if (*abort_flag || clock64() - t1 > ws::kWaitCycles) { *abort_flag = 1; alive = false; break; }
            }
          }
          if (alive && atomicAdd(p.passed + (s - 1), 1u) == (unsigned)(2 * G - 1)) {
            p.done[s - 1] = 0u;
            p.passed[s - 1] = 0u;
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---- MMA issuer
      int stage = 0, segc = 0;
      uint32_t parity = 0;
      bool alive = true;
      for (int s = 0; s < p.n && alive; ++s) {
        const UArgs& a = p.a[s];
        const Segs segs = stage_segs(a);
        const uint32_t id = a.lo ? idesc(2 * MP) : idesc(MP);
        for (int si = 0; si < segs.n && alive; ++si, ++segc) {
          int t, b, e;
          segs.get(si, t, b, e);
          const int buf = segc & 1;
          if (!mbar_wait(&ctl.acc_empty[buf], ((segc >> 1) & 1) ^ 1, abort_flag)) { alive = false; break; }
          fence_after_sync();
          const uint32_t d = tmem + buf * acols;
          uint32_t acc = 0;
          for (int j = b; j < e; ++j) {
            if (!mbar_wait(&ctl.full[stage], parity, abort_flag)) { alive = false; break; }
            fence_after_sync();
            const uint32_t sa = base + stage * sbytes;
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k) {
              const int ai = k & (ksplit - 1);
              mma_f16(d + ai * 2 * MP, smem_desc(sa + k * 32), smem_desc(sa + kABytes + k * 32), id,
                      (acc || k >= ksplit) ? 1u : 0u);
            }
            acc = 1;
            mma_commit(&ctl.empty[stage]);
            if (++stage == nst) { stage = 0; parity ^= 1; }
          }
          if (alive) mma_commit(&ctl.acc_full[buf]);
        }
      }
    }
  } else {
    // ---- epilogue warps: accumulator row r = 32 q + lane
    const int q = warp & 3, r = 32 * q + lane, et = r;
    int segc = 0;
    bool alive = true;
    for (int s = 0; s < p.n && alive; ++s) {
      const UArgs& a = p.a[s];
      const Segs segs = stage_segs(a);
      const int epi = p.epi[s];
      // (pass -1 of the first stage: a rehearsal of the reduction and epilogue code, see k_umma_gemm;
      // rehearsing the later stages' kinds of epilogue as well was measured and changes nothing)
      for (int seg = (s == 0 && segs.n > 0) ? -1 : 0; seg <= segs.n && alive; ++seg) {
        const bool dry = seg < 0;
        if (seg == 0) {
          // the stage before this one is complete: its outputs, sums of squares and residuals may be read
          if (s == 0) {
            pdl_wait();
          } else {
            if (et == 0) {
              const unsigned want = (unsigned)p.a[s - 1].n_tiles;
              const long long t0 = clock64();
              bool ok = true;
              while (ld_acquire_u32(p.done + (s - 1)) < want) {
                if (*abort_flag || clock64() - t0 > ws::kWaitCycles) { *abort_flag = 1; ok = false; break; }
              }
              if (ok && atomicAdd(p.passed + (s - 1), 1u) == (unsigned)(2 * G - 1)) {
                p.done[s - 1] = 0u;
                p.passed[s - 1] = 0u;
              }
            }
            if (epi_any(*abort_flag != 0)) { alive = false; break; }
          }
          for (int m = warp - 2; m < a.M; m += 4) {   // RMSNorm row scales of the input
            float sc = 1.f;
            if (a.ssq_in) {
              float ss = 0.f;
              for (int c = lane; c < a.ssq_n; c += 32) ss += __ldcg(a.ssq_in + (size_t)c * a.M + m);
              ss = warp_sum(ss);
              sc = rsqrtf(ss / (float)a.K + a.eps);
            }
            if (lane == 0) ctl.scale[m] = sc;
          }
          epi_sync();
        }
        if (seg == segs.n) break;
        int t, sb, se;
        segs.get(dry ? 0 : seg, t, sb, se);
        const int t_begin = t * a.KB, t_end = t_begin + a.KB;
        const bool whole = !dry && se - sb == a.KB;
        const int buf = segc & 1, mc = a.M, nvec = (mc + 3) >> 2;
        const int slot = (t == segs.t0) ? 0 : 1;
        // (a partial is kept as [accumulator row][16 activation rows]: a thread writes and reads its
        // rows as 16-byte vectors)
        float* P = a.partials + ((size_t)blockIdx.x * 2 + slot) * kMaxRows * 128;
        const int U = a.n_tiles * a.KB;
        // ---- while the MMAs still run: who shares the tile and where their partials lie, and the
        // residual rows of a storing epilogue (into ctl.land, each thread its own feature)
        int c_first = blockIdx.x, c_last = blockIdx.x;
        if (!whole) {
          if (!dry) {
            c_first = unit_owner(t_begin, U, G);
            c_last = unit_owner(t_end - 1, U, G);
          }
          for (int j = et; j <= c_last - c_first; j += kEpiThreads) {
            const int c = c_first + j, cb = unit_begin(c, U, G);
            int off = -1;
            if (cb < unit_begin(c + 1, U, G)) {
              const int sl = (c == c_first && cb / a.KB != t) ? 1 : 0;
              off = (c * 2 + sl) * kMaxRows * 128;
            }
            ctl.coff[j] = off;
          }
        }
        const bool res_pre = epi == EPI_STORE && a.res != nullptr;
        if (res_pre) {
          bool valid;
          const int n = tile_feature(a, t, r, valid);
          float rvp[16];
#pragma unroll
          for (int m = 0; m < 16; ++m) rvp[m] = (valid && m < mc) ? __ldcg(a.res + (size_t)m * a.ldr + n) : 0.f;
#pragma unroll
          for (int m = 0; m < 16; ++m) ctl.land[m * 128 + r] = rvp[m];
        }
        if (!whole) epi_sync();   // the contributor table is complete
        if (!dry && epi_any(!mbar_wait(&ctl.acc_full[buf], (segc >> 1) & 1, abort_flag))) { alive = false; break; }
        fence_after_sync();
        const uint32_t ta = tmem + ((uint32_t)(32 * q) << 16) + buf * acols;
        float v[16];
#pragma unroll
        for (int m = 0; m < 16; ++m) v[m] = 0.f;
        if (!dry) {   // the tile's sums over this CTA's k-blocks: the accumulators and their hi / lo halves
          // (the ksplit accumulators, hi half then lo half each, are 2 ksplit MP consecutive columns:
          // two loads bring them all, one wait)
          static_assert(2 * ksplit * MP == 128, "accumulators of a tile span 128 columns");
          float w0[64], w1[64];
          tmem_ld64(ta, w0);
          tmem_ld64(ta + 64, w1);
          tmem_ld_wait();
          const bool lo = a.lo != 0;
#pragma unroll
          for (int m = 0; m < 16; ++m) {
            // same order of additions as one load per group: acc0.hi, acc0.lo, acc1.hi, ...
            float x = w0[m];
            if (lo) x += w0[16 + m];
            x += w0[32 + m];
            if (lo) x += w0[48 + m];
            x += w1[m];
            if (lo) x += w1[16 + m];
            x += w1[32 + m];
            if (lo) x += w1[48 + m];
            v[m] = x;
          }
          fence_before_sync();
          mbar_arrive(&ctl.acc_empty[buf]);   // the accumulator is read: the MMA warp may reuse it
        }
        bool finish = whole || dry;
        // The CTA that owns the tile's last k-block finishes the tile.  The others store their
        // partial and count themselves in (release); one thread of the finisher waits for the
        // count (acquire, bounded) while its own sums stay in registers.
        if (!whole && !dry) {
          if (blockIdx.x != c_last) {
            float4* d4 = reinterpret_cast<float4*>(P + r * 16);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (i < nvec) d4[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            epi_sync();   // (orders the other threads' stores before the release below)
            if (et == 0) {
              __threadfence();
              atomicAdd(&a.tile_tickets[t], 1u);
            }
          } else {
            if (et == 0) {
              unsigned n_other = 0;
              for (int j = 0; j < c_last - c_first; ++j) n_other += ctl.coff[j] >= 0;
              const long long t0 = clock64();
              while (ld_acquire_u32(&a.tile_tickets[t]) < n_other) {
                if (*abort_flag || clock64() - t0 > ws::kWaitCycles) { *abort_flag = 1; break; }
              }
              a.tile_tickets[t] = 0u;   // everyone has counted itself in
            }
            epi_sync();
            finish = true;
          }
        }
        if (finish) {
          if (!whole) {
            // the partials added in CTA order (the sum does not depend on who came last), all of
            // up to four contributors' vectors in flight together
            const int nc = dry ? 1 : c_last - c_first;   // (the rehearsal reads this CTA's own slot)
            const float* Pr = a.partials + r * 16;
            float own[16];
#pragma unroll
            for (int m = 0; m < 16; ++m) { own[m] = v[m]; v[m] = 0.f; }
            const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (mc <= 8) {
#pragma unroll 1
              for (int j0 = 0; j0 < nc; j0 += 4) {
                float4 x[4][2];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int o = j0 + j < nc ? ctl.coff[j0 + j] : -1;
#pragma unroll
                  for (int i = 0; i < 2; ++i)
                    x[j][i] = o >= 0 ? __ldcg(reinterpret_cast<const float4*>(Pr + o) + i) : zero4;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                  for (int i = 0; i < 2; ++i) {
                    v[4 * i] += x[j][i].x; v[4 * i + 1] += x[j][i].y; v[4 * i + 2] += x[j][i].z; v[4 * i + 3] += x[j][i].w;
                  }
              }
            } else {
#pragma unroll 1
              for (int j0 = 0; j0 < nc; j0 += 2) {
                float4 x[2][4];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                  const int o = j0 + j < nc ? ctl.coff[j0 + j] : -1;
#pragma unroll
                  for (int i = 0; i < 4; ++i)
                    x[j][i] = o >= 0 ? __ldcg(reinterpret_cast<const float4*>(Pr + o) + i) : zero4;
                }
#pragma unroll
                for (int j = 0; j < 2; ++j)
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    v[4 * i] += x[j][i].x; v[4 * i + 1] += x[j][i].y; v[4 * i + 2] += x[j][i].z; v[4 * i + 3] += x[j][i].w;
                  }
              }
            }
#pragma unroll
            for (int m = 0; m < 16; ++m) v[m] += own[m];   // the finisher is the last in CTA order
          }
#pragma unroll
          for (int m = 0; m < 16; ++m) ctl.acc[m * 128 + r] = v[m];
          if (epi == EPI_STORE) tile_epilogue<EPI_STORE, 1>(a, ctl, t, r, q, lane, 0, mc, dry, res_pre);
          else if (epi == EPI_SWIGLU) tile_epilogue<EPI_SWIGLU, 1>(a, ctl, t, r, q, lane, 0, mc, dry);
          else tile_epilogue<EPI_LMHEAD, 1>(a, ctl, t, r, q, lane, 0, mc, dry);
          if (!dry && s + 1 < p.n) {   // one more tile of this stage is complete
            fence_proxy_async();
            epi_sync();
            if (et == 0) {
              __threadfence();
              atomicAdd(p.done + s, 1u);
            }
          }
        }
        if (!dry) ++segc;
      }
    }
    fence_before_sync();
  }

  __syncthreads();
  if (p.epi[p.n - 1] == EPI_LMHEAD) lm_merge(p.a[p.n - 1], ctl, stages, tid, warp, lane);
  if (ctl.abort_flag) {
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    if (tid == 0) atomicOr(p.a[0].status, kStatTimeout);
    __syncthreads();
  }
  if (warp == 1) {
    fence_after_sync();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols(MP)) : "memory");
  }
}

// Rows of the fc input: [embedding(token) ; hidden] for a sequence's first row, the learned
// [MASK] embedding and feature rows after it (Sec. 4.1).  One block per row.
__global__ void k_gather_x(const __nv_bfloat16* __restrict__ embed, const __nv_bfloat16* __restrict__ mask_embed,
                           const __nv_bfloat16* __restrict__ mask_feat, const __nv_bfloat16* __restrict__ hidden,
                           const int* __restrict__ tokens, int H, int V, int R, __nv_bfloat16* __restrict__ xin) {
  pdl_launch_dependents();
  pdl_wait();
  const int m = blockIdx.x, b = m / R, j = m - b * R;
  const __nv_bfloat16 *e, *f;
  if (j == 0) {
    const int tok = min(max(tokens[b], 0), V - 1);
    e = embed + (size_t)tok * H;
    f = hidden + (size_t)b * H;
  } else {
    e = mask_embed + (size_t)(j - 1) * H;
    f = mask_feat + (size_t)(j - 1) * H;
  }
  uint4* dst = reinterpret_cast<uint4*>(xin + (size_t)m * 2 * H);
  const int nv = H / 8;
  for (int i = threadIdx.x; i < nv; i += blockDim.x) {
    dst[i] = reinterpret_cast<const uint4*>(e)[i];
    dst[nv + i] = reinterpret_cast<const uint4*>(f)[i];
  }
}

// Embedding-only input (PS_FLAG_NO_FC): x0 = embedding(token) for a sequence's first row, the
// learned [MASK] embeddings after it; also the planes of x0 * g_in and each row's sum of
// squares (one partial per row).  One block per row.
__global__ void __launch_bounds__(256) k_embed_x0(const __nv_bfloat16* __restrict__ embed,
                                                  const __nv_bfloat16* __restrict__ mask_embed,
                                                  const int* __restrict__ tokens, const __nv_bfloat16* __restrict__ g_in,
                                                  int H, int V, int R, float* __restrict__ x0,
                                                  __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                  float* __restrict__ ssq) {
  __shared__ float s_part[8];
  pdl_launch_dependents();
  pdl_wait();
  const int m = blockIdx.x, b = m / R, j = m - b * R;
  const __nv_bfloat16* e = j == 0 ? embed + (size_t)min(max(tokens[b], 0), V - 1) * H : mask_embed + (size_t)(j - 1) * H;
  float ss = 0.f;
  for (int n = threadIdx.x; n < H; n += blockDim.x) {
    const float x = __bfloat162float(e[n]);
    x0[(size_t)m * H + n] = x;
    split_store(hi + (size_t)m * H + n, lo + (size_t)m * H + n, x * __bfloat162float(g_in[n]));
    ss += x * x;
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += s_part[w];
    ssq[m] = tot;
  }
}

// The bounded wait of the GEMM kernels on a barrier that nothing ever completes: what a lost
// copy would look like to them.  The wait gives up after `limit` cycles, the kernel raises the
// status word as they do and returns normally.
__global__ void k_wait_expires(long long limit, int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(&bar, 0, &abort_flag, limit)) atomicOr(status, kStatTimeout);
  }
}

// ---- host side: tensor maps ---------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// bf16 matrix [rows][cols] row-major; boxes of box_rows x 64 columns, 128-byte swizzle, zeros
// outside the matrix.
bool make_map(CUtensorMap* m, const void* base, size_t rows, size_t cols, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)umma::kBK, (cuuint32_t)box_rows};
  cuuint32_t es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct PlaneMaps {   // one activation plane with boxes of every padded row count (umma::kRowPads)
  CUtensorMap m[umma::kNumRowPads];
};
struct UmmaMaps {
  CUtensorMap w_fc, w_q, w_k, w_v, w_o, w_gate, w_up, w_down, w_lm;
  PlaneMaps xin, x0_hi, x0_lo, attn_hi, attn_lo, a_hi, a_lo, act_hi, act_lo, hdn_hi, hdn_lo;
};

bool make_plane_maps(PlaneMaps* pm, const void* base, size_t cols) {
  for (int i = 0; i < umma::kNumRowPads; ++i)
    if (!make_map(&pm->m[i], base, umma::kMaxRows, cols, umma::kRowPads[i])) return false;
  return true;
}

UmmaMaps* build_maps(const ps_ctx* c, const FusedScratch& f) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  const size_t H = g.hidden, Hq = (size_t)g.n_heads * g.head_dim, Hkv = (size_t)g.n_kv_heads * g.head_dim,
               F = g.ffn, V = g.vocab;
  UmmaMaps* u = new UmmaMaps;
  // (an embedding-only drafter has no fc matrix: its map is never used, w_q stands in)
  const bool no_fc = (g.flags & PS_FLAG_NO_FC) != 0;
  bool ok = (no_fc ? make_map(&u->w_fc, w.w_q, Hq, H, 128) : make_map(&u->w_fc, w.w_fc, H, 2 * H, 128)) &&
            make_map(&u->w_q, w.w_q, Hq, H, 128) &&
            make_map(&u->w_k, w.w_k, Hkv, H, 128) && make_map(&u->w_v, w.w_v, Hkv, H, 128) &&
            make_map(&u->w_o, w.w_o, H, Hq, 128) && make_map(&u->w_gate, w.w_gate, F, H, 64) &&
            make_map(&u->w_up, w.w_up, F, H, 64) && make_map(&u->w_down, w.w_down, H, F, 128) &&
            make_map(&u->w_lm, w.w_lm, V, H, 128);
  ok = ok && make_plane_maps(&u->xin, f.xin, 2 * H) && make_plane_maps(&u->x0_hi, f.x0p.hi, H) &&
       make_plane_maps(&u->x0_lo, f.x0p.lo, H) && make_plane_maps(&u->attn_hi, f.attnp.hi, Hq) &&
       make_plane_maps(&u->attn_lo, f.attnp.lo, Hq) && make_plane_maps(&u->a_hi, f.ap.hi, H) &&
       make_plane_maps(&u->a_lo, f.ap.lo, H) && make_plane_maps(&u->act_hi, f.actp.hi, F) &&
       make_plane_maps(&u->act_lo, f.actp.lo, F) && make_plane_maps(&u->hdn_hi, f.hdnp.hi, H) &&
       make_plane_maps(&u->hdn_lo, f.hdnp.lo, H);
  if (!ok) {
    delete u;
    return nullptr;
  }
  return u;
}

// Blocks per tile (UArgs::split) for a launch of M rows on G CTAs.  Up to 16 rows single units
// are dealt (split = KB).  Beyond, a tile shared between CTAs costs more the more rows there
// are (its partial sums come back 16 rows x one contributor at a time), so a model of the
// slowest CTA picks the split.  Its constants are fitted on a B200 with 80 to 144 rows: 0.3 us
// per unit, 2 us of epilogue per 16 rows of a finished tile, 1 us per contributor and 16 rows
// of a shared tile plus 0.5 us per 16 rows to publish a partial.  (At these row counts a unit
// brings 32 KB of activation planes from L2 beside its 16 KB of weights, and the launches are
// bound by that traffic rather than by HBM: the split moves their time by a tenth at most.)
static int choose_split(int M, int Mp, int n_tiles, int KB, int G) {
  if (Mp <= 16) return KB;
  const double t_unit = 0.3, t_epi = 2.0, t_trip = 1.0, t_part = 0.5;   // microseconds
  const int chunks = (M + 15) / 16, finished = (n_tiles + G - 1) / G;
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= KB; s = (s < 16 ? s + 1 : (s < KB ? KB : KB + 1))) {
    const long long S = (long long)n_tiles * s;
    const int blocks = (int)((S + G - 1) / G), units = blocks * ((KB + s - 1) / s);
    // contributors of a shared tile: its blocks lie on ceil(s / blocks) CTAs, one more when unaligned
    const int contrib = std::min(s, (s + blocks - 1) / blocks + 1);
    const double cost = units * t_unit + finished * chunks * t_epi +
                        (s > 1 ? chunks * (contrib * t_trip + t_part) : 0.0);
    if (cost < best_cost) { best_cost = cost; best = s; }
  }
  return best;
}

// Geometry of one GEMM stage: padded rows, tiles, k-blocks, the split, the shared scratch.
// *mi = index of the padded row count in umma::kRowPads.
ps_status prep_uargs(ps_ctx* c, UArgs& a, const FusedScratch& f, int* mi) {
  *mi = 0;
  while (umma::kRowPads[*mi] < a.M) ++*mi;
  a.Mp = umma::kRowPads[*mi];
  a.KB = (a.K + umma::kBK - 1) / umma::kBK;
  if (a.zip) {
    a.n_tiles = (a.N + 63) / 64;
  } else {
    a.n_tiles = 0;
    int off = 0;
    for (int m = 0; m < a.n_mats; ++m) {
      a.mat_tiles[m] = (a.mat_rows[m] + umma::kTile - 1) / umma::kTile;
      a.mat_off[m] = off;
      off += a.mat_rows[m];
      a.n_tiles += a.mat_tiles[m];
    }
  }
  if ((long long)a.n_tiles * a.KB * (c->n_sm + 1) >= (1ll << 31)) return fail(c, PS_ERR_UNSUPPORTED, "too many GEMM units");
  a.split = choose_split(a.M, a.Mp, a.n_tiles, a.KB, c->n_sm);
  a.partials = f.partials; a.tile_tickets = f.tile_tickets; a.status = c->dev_status;
  return PS_OK;
}

template <int EPI>
ps_status launch_umma(ps_ctx* c, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& a2,
                      const PlaneMaps& ph, const PlaneMaps& pl, UArgs& a, const FusedScratch& f,
                      cudaStream_t st) {
  int mi;
  ps_status s = prep_uargs(c, a, f, &mi);
  if (s) return s;
  const CUtensorMap &bh = ph.m[mi], &bl = pl.m[mi];
  auto kern = mi == 0   ? k_umma_gemm<EPI, 16>
              : mi == 1 ? k_umma_gemm<EPI, 32>
              : mi == 2 ? k_umma_gemm<EPI, 48>
              : mi == 3 ? k_umma_gemm<EPI, 64>
              : mi == 4 ? k_umma_gemm<EPI, 96>
                        : k_umma_gemm<EPI, 128>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, umma::kSmemBytes);
  if (e != cudaSuccess) return cuda_check(c, e, "umma smem attribute");
  e = launch_after(kern, dim3(c->n_sm), dim3(umma::kThreads), umma::kSmemBytes, st, !c->prof, a0, a1, a2, bh, bl, a);
  c->launches++;
  return cuda_check(c, e, "k_umma_gemm");
}

// One stage of the draft step as the launchers take it.
struct StageDesc {
  int epi;
  const CUtensorMap *a0, *a1, *a2;
  const PlaneMaps *ph, *pl;
  UArgs a;
  const char* name;   // of the stage, for the stage timers
};

// Runs stages d[0..n): as one chained launch (up to 16 rows, `chain`; chain_id 0 or 1: which of a
// step's chains), else one launch each.
ps_status run_stages(ps_ctx* c, StageDesc* d, int n, bool chain, int chain_id, const FusedScratch& f,
                     cudaStream_t st) {
  ps_status s;
  if (!chain || n < 2) {
    for (int i = 0; i < n; ++i) {
      StageDesc& x = d[i];
      if (x.epi == EPI_STORE) s = launch_umma<EPI_STORE>(c, *x.a0, *x.a1, *x.a2, *x.ph, *x.pl, x.a, f, st);
      else if (x.epi == EPI_SWIGLU) s = launch_umma<EPI_SWIGLU>(c, *x.a0, *x.a1, *x.a2, *x.ph, *x.pl, x.a, f, st);
      else s = launch_umma<EPI_LMHEAD>(c, *x.a0, *x.a1, *x.a2, *x.ph, *x.pl, x.a, f, st);
      if (s) return s;
      if (x.name) prof_mark(c, st, x.name);
    }
    return PS_OK;
  }
  if (n > kChainMax) return fail(c, PS_ERR_INVALID_ARG, "too many chained stages");
  ChainParams p{};
  p.n = n;
  // (every chain of a step has counters of its own: a launch may start before the one two ahead of it has ended)
  p.done = f.chain_ctr + chain_id * 2 * kChainMax;
  p.passed = p.done + kChainMax;
  int nm = 0;
  for (int i = 0; i < n; ++i) {
    StageDesc& x = d[i];
    int mi;
    if ((s = prep_uargs(c, x.a, f, &mi))) return s;
    if (mi != 0) return fail(c, PS_ERR_INVALID_ARG, "chained stages take up to 16 rows");
    p.a[i] = x.a;
    p.epi[i] = x.epi;
    const CUtensorMap* am[3] = {x.a0, x.a1, x.a2};
    for (int j = 0; j < 3; ++j) {
      if (j > 0 && am[j] == am[j - 1]) { p.map_a[i][j] = p.map_a[i][j - 1]; continue; }
      if (nm >= kChainMaps) return fail(c, PS_ERR_INVALID_ARG, "too many tensor maps in a chain");
      p.map_a[i][j] = nm;
      p.maps[nm++] = *am[j];
    }
    if (nm + 2 > kChainMaps + (x.a.lo ? 0 : 1)) return fail(c, PS_ERR_INVALID_ARG, "too many tensor maps in a chain");
    p.map_bh[i] = nm;
    p.maps[nm++] = x.ph->m[0];
    p.map_bl[i] = p.map_bh[i];
    if (x.a.lo) { p.map_bl[i] = nm; p.maps[nm++] = x.pl->m[0]; }
  }
  auto kern = k_umma_chain<16>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, umma::kSmemBytes);
  if (e != cudaSuccess) return cuda_check(c, e, "chain smem attribute");
  // A dependent launch like the others.  Its CTAs wait for one another: the grid is one CTA per
  // SM, each filling its SM's shared memory, and a launch's dependents start only once all of
  // its CTAs have, so on a device that runs nothing else beside this stream all are resident; if
  // they are not (kernels of other streams holding SMs), the bounded waits expire into
  // PS_ERR_TIMEOUT.  (A cooperative launch guarantees residency but does not overlap with the
  // launch before it: measured 15 us slower per step.)
  e = launch_after(kern, dim3(c->n_sm), dim3(umma::kThreads), umma::kSmemBytes, st, !c->prof, p);
  c->launches++;
  return cuda_check(c, e, "k_umma_chain");
}

// ps_kv_append on the tensor-core GEMM: rows [sm.row_base, sm.row_base + rows) of the call's real
// (token, feature) pairs: gather, fc (+ the planes of its normalised output), k | v projection,
// then RoPE and the store into the cache rows (the kernel the plain path uses).
ps_status umma_kv_append(ps_ctx* c, const UmmaMaps& u, const SeqMap& sm, int rows, const void* hidden,
                         const int* tokens, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  const int H = g.hidden, Hkv = g.n_kv_heads * g.head_dim, V = g.vocab;
  typedef const __nv_bfloat16* BP;
  const FusedScratch f = carve_fused(g, (char*)c->fused_scratch);
  const int tiles_h = (H + umma::kTile - 1) / umma::kTile;
  ps_status s;
  prof_mark(c, st, "begin");
  // every row is a real position: with one row per "sequence" the gather takes row m's own pair
  cudaError_t ge = launch_after(k_gather_x, dim3(rows), dim3(256), 0, st, !c->prof, (BP)w.embed, (BP)w.mask_embed,
                                (BP)w.mask_feat, (BP)hidden + (size_t)sm.row_base * H, tokens + sm.row_base, H, V, 1,
                                f.xin);
  c->launches++;
  if (ge != cudaSuccess) return cuda_check(c, ge, "k_gather_x");
  // (up to 16 rows the two stages share a launch, like fc and q|k|v of a draft step)
  const bool chain = rows <= 16 && (!c->prof || c->prof_launches) && !(g.flags & PS_FLAG_STAGE_LAUNCHES);
  StageDesc d[2];
  {
    d[0] = StageDesc{EPI_STORE, &u.w_fc, &u.w_fc, &u.w_fc, &u.xin, &u.xin, UArgs{}, "fc_norm"};
    UArgs& a = d[0].a;
    a.N = H; a.K = 2 * H; a.M = rows; a.n_mats = 1; a.mat_rows[0] = H; a.lo = 0;
    a.out = c->x0; a.ldo = H; a.bias = (g.flags & PS_FLAG_FC_BIAS) ? (BP)w.b_fc : nullptr;
    a.ssq_out = f.ssq[0];
    a.out_hi = f.x0p.hi; a.out_lo = f.x0p.lo; a.ld_plane = H; a.gain_next = (BP)w.g_in;
  }
  {
    d[1] = StageDesc{EPI_STORE, &u.w_k, &u.w_v, &u.w_v, &u.x0_hi, &u.x0_lo, UArgs{}, nullptr};
    UArgs& a = d[1].a;
    a.N = 2 * Hkv; a.K = H; a.M = rows; a.n_mats = 2; a.mat_rows[0] = Hkv; a.mat_rows[1] = Hkv; a.lo = 1;
    a.ssq_in = f.ssq[0]; a.ssq_n = tiles_h; a.eps = g.rms_eps;
    a.out = c->kv_tmp; a.ldo = 2 * Hkv;
  }
  if ((s = run_stages(c, d, 2, chain, 0, f, st))) return s;
  if ((s = launch_rope_store_kv(c, sm, rows, st))) return s;
  prof_mark(c, st, "qkv_rope");
  return PS_OK;
}

ps_status umma_draft_step(ps_ctx* c, const UmmaMaps& u, const SeqMap& sm, int B, const void* hidden_last,
                          const int* token_last, int top_n, int* top_ids, float* top_logit, float* row_max,
                          float* row_lse, float* logits_out, float* feat_out, const SampleArgs* sa,
                          cudaStream_t st) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  const int H = g.hidden, Hq = g.n_heads * g.head_dim, Hkv = g.n_kv_heads * g.head_dim, F = g.ffn,
            V = g.vocab, R = g.k_masks + 1, M = B * R;
  typedef const __nv_bfloat16* BP;
  const FusedScratch f = carve_fused(g, (char*)c->fused_scratch);
  const int tiles_h = (H + umma::kTile - 1) / umma::kTile;
  // up to 16 rows the stages on either side of the attention run as one launch each (the stage
  // timers need a launch per stage)
  const bool chain = M <= 16 && (!c->prof || c->prof_launches) && !(g.flags & PS_FLAG_STAGE_LAUNCHES);
  ps_status s;
  prof_mark(c, st, "begin");
  const bool no_fc = (g.flags & PS_FLAG_NO_FC) != 0;
  StageDesc d[kChainMax];
  int n = 0;
  if (no_fc) {   // embedding-only input: x0 and its planes come straight from the embedding rows
    cudaError_t ee = launch_after(k_embed_x0, dim3(M), dim3(256), 0, st, !c->prof, (BP)w.embed, (BP)w.mask_embed,
                                  token_last, (BP)w.g_in, H, V, R, c->x0, f.x0p.hi, f.x0p.lo, f.ssq[0]);
    c->launches++;
    if (ee != cudaSuccess) return cuda_check(c, ee, "k_embed_x0");
    prof_mark(c, st, "fc_norm");
  } else {
    cudaError_t ge = launch_after(k_gather_x, dim3(M), dim3(256), 0, st, !c->prof, (BP)w.embed, (BP)w.mask_embed,
                                  (BP)w.mask_feat, (BP)hidden_last, token_last, H, V, R, f.xin);
    c->launches++;
    if (ge != cudaSuccess) return cuda_check(c, ge, "k_gather_x");
    // S1 fc: x0 = W_fc [e ; f] (+ b)
    StageDesc& x = d[n++];
    x = StageDesc{EPI_STORE, &u.w_fc, &u.w_fc, &u.w_fc, &u.xin, &u.xin, UArgs{}, "fc_norm"};
    UArgs& a = x.a;
    a.N = H; a.K = 2 * H; a.M = M; a.n_mats = 1; a.mat_rows[0] = H; a.lo = 0;
    a.out = c->x0; a.ldo = H; a.bias = (g.flags & PS_FLAG_FC_BIAS) ? (BP)w.b_fc : nullptr;
    a.ssq_out = f.ssq[0];
    a.out_hi = f.x0p.hi; a.out_lo = f.x0p.lo; a.ld_plane = H; a.gain_next = (BP)w.g_in;
  }
  {  // S2 q|k|v = W rms(x0)
    StageDesc& x = d[n++];
    x = StageDesc{EPI_STORE, &u.w_q, &u.w_k, &u.w_v, &u.x0_hi, &u.x0_lo, UArgs{}, "qkv_rope"};
    UArgs& a = x.a;
    a.N = Hq + 2 * Hkv; a.K = H; a.M = M; a.n_mats = 3;
    a.mat_rows[0] = Hq; a.mat_rows[1] = Hkv; a.mat_rows[2] = Hkv; a.lo = 1;
    a.ssq_in = f.ssq[0]; a.ssq_n = no_fc ? 1 : tiles_h; a.eps = g.rms_eps;
    a.out = f.qkv; a.ldo = Hq + 2 * Hkv;
  }
  if ((s = run_stages(c, d, n, chain, 0, f, st))) return s;
  if (chain && n > 1) prof_mark(c, st, "chain_fc_qkv");
  if ((s = launch_attn_split(c, sm, B, f.qkv, f.att_ml, f.att_o, f.attn_tickets, f.attnp.hi, f.attnp.lo, st)))
    return s;
  prof_mark(c, st, "attention");
  n = 0;
  {  // S4 a = x0 + W_o attn
    StageDesc& x = d[n++];
    x = StageDesc{EPI_STORE, &u.w_o, &u.w_o, &u.w_o, &u.attn_hi, &u.attn_lo, UArgs{}, "o_proj"};
    UArgs& a = x.a;
    a.N = H; a.K = Hq; a.M = M; a.n_mats = 1; a.mat_rows[0] = H; a.lo = 1;
    a.out = c->a; a.ldo = H; a.res = c->x0; a.ldr = H;
    a.ssq_out = f.ssq[1];
    a.out_hi = f.ap.hi; a.out_lo = f.ap.lo; a.ld_plane = H; a.gain_next = (BP)w.g_post;
  }
  {  // S5a act = silu(W_g rms(a)) * (W_u rms(a))
    StageDesc& x = d[n++];
    x = StageDesc{EPI_SWIGLU, &u.w_gate, &u.w_up, &u.w_up, &u.a_hi, &u.a_lo, UArgs{}, "ffn_gate_up"};
    UArgs& a = x.a;
    a.N = F; a.K = H; a.M = M; a.zip = 1; a.n_mats = 2; a.lo = 1;
    a.ssq_in = f.ssq[1]; a.ssq_n = tiles_h; a.eps = g.rms_eps;
    a.out = f.act; a.ldo = F;
    a.out_hi = f.actp.hi; a.out_lo = f.actp.lo; a.ld_plane = F;
  }
  float* hdn = feat_out ? feat_out : c->hdn;
  {  // S5b hdn = a + W_d act
    StageDesc& x = d[n++];
    x = StageDesc{EPI_STORE, &u.w_down, &u.w_down, &u.w_down, &u.act_hi, &u.act_lo, UArgs{}, "ffn_down"};
    UArgs& a = x.a;
    a.N = H; a.K = F; a.M = M; a.n_mats = 1; a.mat_rows[0] = H; a.lo = 1;
    a.out = hdn; a.ldo = H; a.res = c->a; a.ldr = H;
    a.ssq_out = f.ssq[2];
    a.out_hi = f.hdnp.hi; a.out_lo = f.hdnp.lo; a.ld_plane = H; a.gain_next = (BP)w.g_final;
  }
  const bool stats_pass = M > 32 && logits_out;
  {
    StageDesc& x = d[n++];
    x = StageDesc{stats_pass ? EPI_STORE : EPI_LMHEAD, &u.w_lm, &u.w_lm, &u.w_lm, &u.hdn_hi, &u.hdn_lo, UArgs{}, "lm_head"};
    UArgs& a = x.a;
    a.N = V; a.K = H; a.M = M; a.n_mats = 1; a.mat_rows[0] = V; a.lo = 1;
    a.ssq_in = f.ssq[2]; a.ssq_n = tiles_h; a.eps = g.rms_eps;
    if (stats_pass) {
      // S6 with many rows and the logits kept: the row statistics in the tile epilogue cost more
      // than the weights' streaming then (they are serial in the rows), so the GEMM only stores
      // the logits and one block per row reads them back from L2
      a.out = logits_out; a.ldo = V;
      x.name = nullptr;   // (timed together with the statistics pass below)
    } else {  // S6 logits = W_lm rms(hdn), softmax statistics and top-n without a second pass over logits
      a.logits_out = logits_out; a.parts = f.parts; a.ticket = f.ticket;
      a.top_n = top_n; a.top_ids = top_ids; a.top_logit = top_logit; a.row_max = row_max; a.row_lse = row_lse;
      a.R = R;
      if (sa) { a.sample = 1; a.sa = *sa; }
    }
  }
  if ((s = run_stages(c, d, n, chain, 1, f, st))) return s;
  if (chain) prof_mark(c, st, "chain_o_ffn_lm");
  if (stats_pass) {
    if ((s = launch_row_stats(c, logits_out, M, V, top_n, top_ids, top_logit, row_max, row_lse, st))) return s;
    if (sa && (s = launch_gumbel_argmax(c, logits_out, M, V, R, *sa, st))) return s;
    prof_mark(c, st, "lm_head");
  }
  return PS_OK;
}

}  // namespace

// Builds the tensor maps of the tensor-core path once; without them (an old driver, unaligned
// weights, too little shared memory) the mma.sync kernels serve.
static void ensure_maps(ps_ctx* c) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  if ((g.flags & PS_FLAG_MMA_SYNC_GEMM) || c->umma_tried) return;
  c->umma_tried = true;
  const bool aligned = ((((uintptr_t)w.w_fc | (uintptr_t)w.w_q | (uintptr_t)w.w_k | (uintptr_t)w.w_v |
                          (uintptr_t)w.w_o | (uintptr_t)w.w_gate | (uintptr_t)w.w_up | (uintptr_t)w.w_down |
                          (uintptr_t)w.w_lm | (uintptr_t)w.embed | (uintptr_t)w.mask_embed |
                          (uintptr_t)w.mask_feat) & 15u) == 0);
  if (aligned && c->smem_optin >= umma::kSmemBytes)
    c->umma_maps = build_maps(c, carve_fused(g, (char*)c->fused_scratch));
}

bool fused_supported(ps_ctx* c, int M) {
  const ps_config& g = c->cfg;
  if (g.dtype != PS_DTYPE_BF16 || (g.flags & PS_FLAG_UNFUSED_KERNELS)) return false;
  if (M > umma::kMaxRows || (g.head_dim != 64 && g.head_dim != 128)) return false;
  const int Hq = g.n_heads * g.head_dim;
  if (g.hidden % 8 || Hq % 8 || g.ffn % 8) return false;   // 16-byte operand rows
  if ((g.vocab + 127) / 128 > umma::kRingBytes / 32) return false;   // a row's tile summaries fit the ring (LM-head merge)
  ensure_maps(c);
  if (c->umma_maps) return true;
  if (M > kMaxM) return false;   // the mma.sync kernels take 16 rows
  const int lim = c->smem_optin, n = c->n_sm;
  return choose_pass_cols(M, 2 * g.hidden, rows_cap_for(g.hidden, n, false), lim) &&
         choose_pass_cols(M, g.hidden, rows_cap_for(Hq + 2 * g.n_kv_heads * g.head_dim, n, false), lim) &&
         choose_pass_cols(M, Hq, rows_cap_for(g.hidden, n, false), lim) &&
         choose_pass_cols(M, g.hidden, rows_cap_for(g.ffn, n, true), lim) &&
         choose_pass_cols(M, g.ffn, rows_cap_for(g.hidden, n, false), lim) &&
         choose_pass_cols(M, g.hidden, rows_cap_for(g.vocab, n, false), lim);
}

int fused_row_limit(ps_ctx* c) {
  if (fused_supported(c, umma::kMaxRows)) return umma::kMaxRows;
  return fused_supported(c, kMaxM) ? kMaxM : 0;
}

// Rows per pass ps_kv_append may hand to fused_kv_append (0: the plain kernels serve).
int fused_kv_rows(ps_ctx* c) {
  if (c->cfg.flags & PS_FLAG_NO_FC) return 0;
  return fused_supported(c, umma::kMaxRows) && c->umma_maps ? umma::kMaxRows : 0;
}

ps_status fused_kv_append(ps_ctx* c, const SeqMap& sm, int rows, const void* hidden, const int* tokens,
                          cudaStream_t st) {
  return umma_kv_append(c, *static_cast<const UmmaMaps*>(c->umma_maps), sm, rows, hidden, tokens, st);
}

size_t fused_scratch_bytes(const ps_config& g) { return carve_fused(g, nullptr).bytes; }

ps_status launch_wait_expires(ps_ctx* c, long long limit_cycles, cudaStream_t st) {
  k_wait_expires<<<1, 32, 0, st>>>(limit_cycles, c->dev_status);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_wait_expires");
}

void fused_release(ps_ctx* c) {
  delete static_cast<UmmaMaps*>(c->umma_maps);
  c->umma_maps = nullptr;
}

ps_status fused_debug_buffer(ps_ctx* c, const char* name, void** ptr, size_t* bytes) {
  const ps_config& g = c->cfg;
  FusedScratch f = carve_fused(g, (char*)c->fused_scratch);
  if (!std::strcmp(name, "qkv")) {
    *ptr = f.qkv;
    *bytes = (size_t)umma::kMaxRows * (g.n_heads + 2 * g.n_kv_heads) * g.head_dim * 4;
    return PS_OK;
  }
  if (!std::strcmp(name, "act")) { *ptr = f.act; *bytes = (size_t)umma::kMaxRows * g.ffn * 4; return PS_OK; }
  return PS_ERR_INVALID_ARG;
}

ps_status fused_draft_step(ps_ctx* c, const SeqMap& sm, int B, const void* hidden_last,
                           const int* token_last, int top_n, int* top_ids, float* top_logit,
                           float* row_max, float* row_lse, float* logits_out, float* feat_out,
                           const SampleArgs* sa, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const ps_weights& w = c->w;
  const int H = g.hidden, Hq = g.n_heads * g.head_dim, Hkv = g.n_kv_heads * g.head_dim, F = g.ffn,
            V = g.vocab, R = g.k_masks + 1, M = B * R;
  typedef const __nv_bfloat16* BP;
  const FusedScratch f = carve_fused(g, (char*)c->fused_scratch);
  if (sa && !c->umma_maps && !logits_out)
    return fail(c, PS_ERR_UNSUPPORTED, "draft sampling on the mma.sync kernels needs logits_out");
  if (c->umma_maps && !(g.flags & PS_FLAG_MMA_SYNC_GEMM))
    return umma_draft_step(c, *static_cast<const UmmaMaps*>(c->umma_maps), sm, B, hidden_last, token_last, top_n,
                           top_ids, top_logit, row_max, row_lse, logits_out, feat_out, sa, st);
  ps_status s;
  prof_mark(c, st, "begin");
  const bool no_fc = (g.flags & PS_FLAG_NO_FC) != 0;
  if (no_fc) {   // embedding-only input: x0 and its planes come straight from the embedding rows
    k_embed_x0<<<M, 256, 0, st>>>((BP)w.embed, (BP)w.mask_embed, token_last, (BP)w.g_in, H, V, R, c->x0,
                                  f.x0p.hi, f.x0p.lo, f.ssq[0]);
    c->launches++;
  } else {  // S1 fc: x0 = W_fc [e ; f] (+ b)
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
    a.ssq_in = f.ssq[0]; a.ssq_n = no_fc ? 1 : c->n_sm; a.eps = g.rms_eps;
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
  prof_mark(c, st, "ffn_gate_up");
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
  prof_mark(c, st, "ffn_down");
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
  if (sa && (s = launch_gumbel_argmax(c, logits_out, M, V, R, *sa, st))) return s;
  prof_mark(c, st, "lm_head");
  return PS_OK;
}

}  // namespace ps
