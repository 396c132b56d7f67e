// ps_verify: speculative-sampling acceptance for a drafted chain (Eq. 1; Algorithm 1 with one
// child per node).  One thread block per (position, sequence) evaluates its row pair
// speculatively: softmax statistics of the target and draft rows, the test r < min(1, p/q),
// and -- if the test fails or the row is the extra target row -- the token that would be
// emitted there (residual max(0, p-q) normalised, or p itself).  The last block of a sequence
// to finish walks the positions in order and writes accept_len / out_tokens / n_out.
// Nothing spins: blocks only take a ticket, the last arriver does the merge.
#include <cfloat>
#include <cstdio>
#include <mutex>

#include <cooperative_groups.h>

#include "ps_internal.cuh"

namespace ps {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kSeg = 128;  // elements per warp-wide segment of the inverse-CDF search

__global__ void k_philox_fill(uint32_t k0, uint32_t k1, const uint32_t* ctr, uint32_t* out, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t c[4] = {ctr[4 * i], ctr[4 * i + 1], ctr[4 * i + 2], ctr[4 * i + 3]};
  philox4x32_10(k0, k1, c);
  for (int j = 0; j < 4; ++j) out[4 * i + j] = c[j];
}

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

struct Scratch {
  float fmax[kWarps];
  int imax[kWarps];
  double dsum[kWarps];
  int flag[kWarps];
  float bc_f;
  int bc_i;
  double bc_d;
  int bc_flag;
};

// Max over a row with NaN treated as -inf, ties to the lower index; also reports whether the
// row holds a NaN or +inf (or nothing above -inf).  Result broadcast to all threads.
__device__ void row_argmax(const float* row, int V, Scratch& s, float& vmax, int& imax, int& bad) {
  float bv = -INFINITY;
  int bi = 0x7fffffff, bd = 0;
  for (int v = threadIdx.x; v < V; v += kThreads) {
    float x = row[v];
    if (x != x || x == INFINITY) bd = 1;
    if (x != x) x = -INFINITY;
    if (x > bv || (x == bv && v < bi)) { bv = x; bi = v; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    bd |= __shfl_xor_sync(0xffffffffu, bd, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) { s.fmax[warp] = bv; s.imax[warp] = bi; s.flag[warp] = bd; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kWarps; ++w) {
      if (s.fmax[w] > bv || (s.fmax[w] == bv && s.imax[w] < bi)) { bv = s.fmax[w]; bi = s.imax[w]; }
      bd |= s.flag[w];
    }
    if (bv == -INFINITY) bd = 1;  // an all -inf row has no distribution
    s.bc_f = bv; s.bc_i = bi; s.bc_flag = bd;
  }
  __syncthreads();
  vmax = s.bc_f; imax = s.bc_i; bad = s.bc_flag;
  __syncthreads();
}

// sum_v exp((row[v] - vmax) / T), accumulated in double, broadcast to all threads.
__device__ double row_sumexp(const float* row, int V, float vmax, double inv_t, Scratch& s) {
  double acc = 0.0;
  for (int v = threadIdx.x; v < V; v += kThreads)
    acc += (double)expf((float)(((double)row[v] - (double)vmax) * inv_t));
  acc = warp_sum_d(acc);
  if ((threadIdx.x & 31) == 0) s.dsum[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kWarps; ++w) t += s.dsum[w];
    s.bc_d = t;
  }
  __syncthreads();
  double r = s.bc_d;
  __syncthreads();
  return r;
}

// Weight of token v in the distribution to sample: max(0, p_v - q_v), or p_v when use_q == 0.
// q is softmax(drow/T) when drow != nullptr, else the point mass on x.
__device__ __forceinline__ float weight_of(int v, const float* trow, const float* drow, int x,
                                           int use_q, float tmax, float dmax, double inv_t,
                                           float inv_st, float inv_sd) {
  float p = expf((float)(((double)trow[v] - (double)tmax) * inv_t)) * inv_st;
  if (!use_q) return p;
  float q = drow ? expf((float)(((double)drow[v] - (double)dmax) * inv_t)) * inv_sd
                 : (v == x ? 1.f : 0.f);
  return fmaxf(p - q, 0.f);
}

// Inverse-CDF draw with uniform u from the weights above: the first v whose running sum
// exceeds u * total.  seg_sum: shared array of ceil(V / kSeg) doubles.  Returns the token to
// all threads; returns -1 if the total weight is not positive.
__device__ int sample_weights(const float* trow, const float* drow, int x, int use_q, int V,
                              float tmax, float dmax, double inv_t, double st, double sd,
                              double u, double* seg_sum, Scratch& s) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nseg = (V + kSeg - 1) / kSeg;
  const float inv_st = (float)(1.0 / st), inv_sd = (float)(1.0 / sd);
  constexpr int E = kSeg / 32;
  for (int g = warp; g < nseg; g += kWarps) {
    double a = 0.0;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      int v = g * kSeg + lane * E + e;
      if (v < V) a += (double)weight_of(v, trow, drow, x, use_q, tmax, dmax, inv_t, inv_st, inv_sd);
    }
    a = warp_sum_d(a);
    if (lane == 0) seg_sum[g] = a;
  }
  __syncthreads();
  if (warp == 0) {
    // lane owns segments [lane*c, lane*c + c)
    int c = (nseg + 31) / 32;
    int g_lo = min(nseg, lane * c), g_hi = min(nseg, lane * c + c);
    double mine = 0.0;
    for (int g = g_lo; g < g_hi; ++g) mine += seg_sum[g];
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      double t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    double total = __shfl_sync(0xffffffffu, incl, 31);
    double target = u * total;
    int token = -1;
    if (total > 0.0) {  // uniform across the warp
      // first lane whose inclusive sum exceeds the target, else the last lane with weight
      unsigned over = __ballot_sync(0xffffffffu, incl > target);
      unsigned pos = __ballot_sync(0xffffffffu, mine > 0.0);
      int src = over ? __ffs(over) - 1 : (pos ? 31 - __clz(pos) : 0);
      int gsel = -1;
      double gbase = 0.0;
      if (lane == src) {
        double run = incl - mine;
        int last_pos = -1;
        double last_base = 0.0;
        for (int g = g_lo; g < g_hi; ++g) {
          if (seg_sum[g] > 0.0) { last_pos = g; last_base = run; }
          if (run + seg_sum[g] > target) { gsel = g; gbase = run; break; }
          run += seg_sum[g];
        }
        if (gsel < 0) { gsel = last_pos; gbase = last_base; }
      }
      gsel = __shfl_sync(0xffffffffu, gsel, src);
      gbase = __shfl_sync(0xffffffffu, gbase, src);
      // inside the segment: lane owns E consecutive tokens
      float wv[E];
      double lsum = 0.0;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        int v = gsel * kSeg + lane * E + e;
        wv[e] = (gsel >= 0 && v < V) ? weight_of(v, trow, drow, x, use_q, tmax, dmax, inv_t, inv_st, inv_sd) : 0.f;
        lsum += (double)wv[e];
      }
      double linc = lsum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, linc, o);
        if (lane >= o) linc += t;
      }
      unsigned over2 = __ballot_sync(0xffffffffu, gbase + linc > target);
      unsigned pos2 = __ballot_sync(0xffffffffu, lsum > 0.0);
      int src2 = over2 ? __ffs(over2) - 1 : (pos2 ? 31 - __clz(pos2) : 0);
      int pick = -1;
      if (lane == src2 && gsel >= 0 && (over2 | pos2)) {
        double run2 = gbase + linc - lsum;
        int lastp = -1;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          if (wv[e] > 0.f) lastp = e;
          run2 += (double)wv[e];
          if (pick < 0 && run2 > target) pick = e;
        }
        if (pick < 0) pick = lastp;
        pick = pick < 0 ? -1 : gsel * kSeg + lane * E + pick;
      }
      token = __shfl_sync(0xffffffffu, pick, src2);
    }
    if (lane == 0) s.bc_i = token;
  }
  __syncthreads();
  int tok = s.bc_i;
  __syncthreads();
  return tok;
}

struct VerifyArgs {
  int B, n_draft, n_target, V;
  const int* draft_tokens;
  const float* draft_logits;
  const float* target_logits;
  float temperature;
  uint32_t key0, key1, off_lo, off_hi;
  int* accept_len;
  int* out_tokens;
  int* n_out;
  VerifyRec* rec;      // [B][PS_MAX_MASKS+2]
  unsigned* tickets;   // [B], zero on entry and on exit
  int* status;
};

// Called by one thread per (position, sequence): records the speculative outcome, takes a
// ticket, and -- as the last arriver of its sequence -- walks the positions in order and writes
// accept_len / out_tokens / n_out.
__device__ void finish_position(const VerifyArgs& a, int i, int b, int accept, int bad, int token) {
  VerifyRec* recw = a.rec + (size_t)b * (PS_MAX_MASKS + 2);
  recw[i].accept = accept | (bad << 1);
  recw[i].token = token;
  __threadfence();
  unsigned t = atomicAdd(&a.tickets[b], 1u);
  if (t != (unsigned)a.n_target - 1u) return;
  __threadfence();
  volatile VerifyRec* rec = recw;
  int* out = a.out_tokens + (size_t)b * (a.n_draft + 1);
  int acc = 0, any_bad = 0, emitted = -1;
  while (acc < a.n_draft) {
    int f = rec[acc].accept;
    any_bad |= (f >> 1) & 1;
    if (!(f & 1)) { emitted = rec[acc].token; break; }
    out[acc] = a.draft_tokens[(size_t)b * a.n_draft + acc];
    ++acc;
  }
  if (acc == a.n_draft && a.n_target == a.n_draft + 1) {
    any_bad |= (rec[acc].accept >> 1) & 1;
    emitted = rec[acc].token;
  }
  int n = acc;
  if (emitted >= 0) out[n++] = emitted;
  for (int j = n; j <= a.n_draft; ++j) out[j] = -1;
  a.accept_len[b] = acc;
  a.n_out[b] = n;
  if (any_bad) atomicOr(a.status, kStatNonfinite);
  a.tickets[b] = 0u;
}

__global__ void __launch_bounds__(kThreads) k_verify(VerifyArgs a) {
  extern __shared__ double seg_sum[];
  __shared__ Scratch s;
  const int i = blockIdx.x, b = blockIdx.y, V = a.V;
  const bool bonus = i >= a.n_draft;
  const float* trow = a.target_logits + ((size_t)b * a.n_target + i) * V;
  const float* drow = (!bonus && a.draft_logits) ? a.draft_logits + ((size_t)b * a.n_draft + i) * V
                                                 : nullptr;
  int x = bonus ? -1 : a.draft_tokens[(size_t)b * a.n_draft + i];
  int accept = 0, token = -1, bad = 0;

  float tmax; int targ, tbad;
  row_argmax(trow, V, s, tmax, targ, tbad);
  if (a.temperature == 0.f) {
    accept = (!bonus && x == targ) ? 1 : 0;
    token = targ;
  } else {
    double inv_t = 1.0 / (double)a.temperature;
    float dmax = 0.f; int darg, dbad = 0;
    if (drow) row_argmax(drow, V, s, dmax, darg, dbad);
    bad = tbad | dbad;
    if (bad) {
      token = targ;
    } else {
      double st = row_sumexp(trow, V, tmax, inv_t, s);
      double sd = drow ? row_sumexp(drow, V, dmax, inv_t, s) : 1.0;
      uint32_t c[4] = {(uint32_t)i, (uint32_t)b, a.off_lo, a.off_hi};
      philox4x32_10(a.key0, a.key1, c);
      double r = (double)(c[0] >> 8) * (1.0 / 16777216.0);
      double u2 = (double)(c[1] >> 8) * (1.0 / 16777216.0);
      if (!bonus) {
        bool in_range = x >= 0 && x < V;
        double logp = in_range ? ((double)trow[x] - (double)tmax) * inv_t - log(st) : -INFINITY;
        double logq = drow ? (in_range ? ((double)drow[x] - (double)dmax) * inv_t - log(sd) : -INFINITY)
                           : 0.0;
        double diff = logp - logq;
        double ratio = (diff != diff) ? 0.0 : exp(fmin(diff, 0.0));
        accept = r < ratio ? 1 : 0;
      }
      if (!accept) {  // uniform across the block: every thread computed the same decision
        token = sample_weights(trow, drow, x, bonus ? 0 : 1, V, tmax, dmax, inv_t, st, sd, u2,
                               seg_sum, s);
        if (token < 0)
          token = sample_weights(trow, drow, x, 0, V, tmax, dmax, inv_t, st, sd, u2, seg_sum, s);
        if (token < 0) token = targ;
      }
    }
  }

  if (threadIdx.x == 0) finish_position(a, i, b, accept, bad, token);
}

// ---- cluster variant ------------------------------------------------------------------------
// A cluster of kClu thread blocks shares one (position, sequence) row pair, so that a batch of
// one still spreads its few rows over dozens of SMs.  Thread g = rank * kCluThreads + tid owns
// the contiguous tokens [g * C, g * C + C) of both rows and keeps them in registers: the logits
// are read from memory once, with all 16-byte loads in flight together.  Row statistics are
// combined through distributed shared memory (each block publishes its partials, a cluster
// barrier, every block reads all of them in rank order, so all blocks hold identical values).
// The inverse-CDF draw descends block -> warp -> lane -> token over running sums.
constexpr int kClu = 8;
constexpr int kCluThreads = 512;
constexpr int kCluWarps = kCluThreads / 32;
constexpr int kCluV4 = 4;  // float4 per thread and row: up to kClu * kCluThreads * 16 tokens
constexpr int kCluMaxVocab = kClu * kCluThreads * 4 * kCluV4;        // with the portable cluster size
constexpr int kCluMaxVocab16 = 16 * kCluThreads * 4 * kCluV4;         // with 16 blocks (opt-in size)

struct CluPart {       // one per block, read by the whole cluster
  float tmax, dmax;
  int targ, bad;
  double st, sd;
  double wsum;         // weight held by this block
  int pick, lastp;     // token chosen inside this block / its last token with weight
};

struct CluScratch {
  float f[kCluWarps], f2[kCluWarps];
  int i[kCluWarps], flag[kCluWarps];
  double d[kCluWarps], d2[kCluWarps];
};

// (NCLU blocks per cluster: 8; 16 for vocabularies beyond 65536; 4 for batches of several waves.)
// (V4: 16-byte vectors a thread holds per row: 4, or 2 when the row fits in half as many -- the
// loops over a thread's tokens are unrolled, and this kernel runs its code once per launch, so
// what it is not asked to execute it should not have to fetch.)
template <int NCLU, int V4>
__device__ __forceinline__ void verify_cluster_body(const VerifyArgs& a) {
  namespace cg = cooperative_groups;
  cg::cluster_group cl = cg::this_cluster();
  __shared__ CluPart part;
  __shared__ CluScratch s;
  const int rank = (int)cl.block_rank();
  constexpr int nclu = NCLU;
  const int i = blockIdx.x / nclu, b = blockIdx.y, V = a.V;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool bonus = i >= a.n_draft;
  const float* trow = a.target_logits + ((size_t)b * a.n_target + i) * V;
  const bool greedy = a.temperature == 0.f;
  const float* drow = (!bonus && !greedy && a.draft_logits)
                          ? a.draft_logits + ((size_t)b * a.n_draft + i) * V : nullptr;
  const int nv4 = ((V + nclu * kCluThreads - 1) / (nclu * kCluThreads) + 3) / 4;
  const int C = nv4 * 4, v0 = (rank * kCluThreads + tid) * C;

  // The target rows are an input of the call; the draft rows and the draft tokens may be what the
  // kernel before this one in the stream (the draft step) wrote last.  Were this kernel launched
  // as its dependent, it would ask for the target row first and wait for that kernel only then.
  pdl_launch_dependents();
  float t[V4 * 4], d[V4 * 4];
#pragma unroll
  for (int k = 0; k < V4; ++k) {
    const int v = v0 + 4 * k;   // V % 4 == 0: a vector lies inside the row or outside it
    float4 tv = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (k < nv4 && v < V) tv = __ldcs(reinterpret_cast<const float4*>(trow + v));
    t[4 * k] = tv.x; t[4 * k + 1] = tv.y; t[4 * k + 2] = tv.z; t[4 * k + 3] = tv.w;
  }
  pdl_wait();
  const int x = bonus ? -1 : a.draft_tokens[(size_t)b * a.n_draft + i];
#pragma unroll
  for (int k = 0; k < V4; ++k) {
    const int v = v0 + 4 * k;
    float4 dv = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (drow && k < nv4 && v < V) dv = *reinterpret_cast<const float4*>(drow + v);
    d[4 * k] = dv.x; d[4 * k + 1] = dv.y; d[4 * k + 2] = dv.z; d[4 * k + 3] = dv.w;
  }

  // ---- maxima (NaN counts as -inf, ties to the lower id) and non-finite flags
  float tm = -INFINITY, dm = -INFINITY;
  int ti = 0x7fffffff, bad = 0;
#pragma unroll
  for (int e = 0; e < V4 * 4; ++e) {
    const int v = v0 + e;
    if (e < C && v < V) {
      float xt = t[e];
      if (xt != xt || xt == INFINITY) bad = 1;
      if (xt != xt) xt = -INFINITY;
      if (xt > tm || (xt == tm && v < ti)) { tm = xt; ti = v; }
      if (drow) {
        float xd = d[e];
        if (xd != xd || xd == INFINITY) bad = 1;
        if (xd != xd) xd = -INFINITY;
        dm = fmaxf(dm, xd);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, tm, o);
    const int oi = __shfl_xor_sync(0xffffffffu, ti, o);
    if (ov > tm || (ov == tm && oi < ti)) { tm = ov; ti = oi; }
    dm = fmaxf(dm, __shfl_xor_sync(0xffffffffu, dm, o));
    bad |= __shfl_xor_sync(0xffffffffu, bad, o);
  }
  if (lane == 0) { s.f[warp] = tm; s.i[warp] = ti; s.flag[warp] = bad; s.f2[warp] = dm; }
  __syncthreads();
  if (warp == 0) {   // the warps' values, one per lane, through a shuffle tree
    static_assert(kCluWarps == 16, "one lane per warp in the low half of warp 0");
    tm = -INFINITY; dm = -INFINITY; ti = 0x7fffffff; bad = 0;
    if (lane < kCluWarps) { tm = s.f[lane]; ti = s.i[lane]; bad = s.flag[lane]; dm = s.f2[lane]; }
#pragma unroll
    for (int o = kCluWarps / 2; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, tm, o);
      const int oi = __shfl_xor_sync(0xffffffffu, ti, o);
      if (ov > tm || (ov == tm && oi < ti)) { tm = ov; ti = oi; }
      dm = fmaxf(dm, __shfl_xor_sync(0xffffffffu, dm, o));
      bad |= __shfl_xor_sync(0xffffffffu, bad, o);
    }
    if (lane == 0) {
      part.tmax = tm; part.targ = ti; part.dmax = dm; part.bad = bad;
      part.pick = -1; part.lastp = -1; part.wsum = 0.0; part.st = 0.0; part.sd = 0.0;
    }
  }
  cl.sync();
  // lane r of every warp fetches block r's partial (one round trip through distributed shared
  // memory for the whole cluster instead of one per block), a shuffle tree combines them; every
  // warp of every block runs the same tree on the same values
  tm = -INFINITY; dm = -INFINITY; ti = 0x7fffffff; bad = 0;
  if (lane < nclu) {
    const CluPart* pr = cl.map_shared_rank(&part, lane);
    tm = pr->tmax; ti = pr->targ; dm = pr->dmax; bad = pr->bad;
  }
#pragma unroll
  for (int o = nclu / 2; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, tm, o);
    const int oi = __shfl_xor_sync(0xffffffffu, ti, o);
    if (ov > tm || (ov == tm && oi < ti)) { tm = ov; ti = oi; }
    dm = fmaxf(dm, __shfl_xor_sync(0xffffffffu, dm, o));
    bad |= __shfl_xor_sync(0xffffffffu, bad, o);
  }
  tm = __shfl_sync(0xffffffffu, tm, 0); ti = __shfl_sync(0xffffffffu, ti, 0);
  dm = __shfl_sync(0xffffffffu, dm, 0); bad = __shfl_sync(0xffffffffu, bad, 0);
  if (tm == -INFINITY || (drow && dm == -INFINITY)) bad = 1;  // a row without a distribution
  const float tmax = tm, dmax = dm;
  const int targ = ti;

  int accept = 0, token = -1;
  if (greedy) {
    accept = (!bonus && x == targ) ? 1 : 0;
    token = targ;
    bad = 0;
  } else if (bad) {
    token = targ;
  } else {
    // every block takes the same branches below: the values they depend on are identical
    const double inv_t = 1.0 / (double)a.temperature;
    double st = 0.0, sd = 0.0;
#pragma unroll
    for (int e = 0; e < V4 * 4; ++e) {
      const bool in = e < C && v0 + e < V;
      t[e] = in ? expf((float)(((double)t[e] - (double)tmax) * inv_t)) : 0.f;
      st += (double)t[e];
      if (drow) {
        d[e] = in ? expf((float)(((double)d[e] - (double)dmax) * inv_t)) : 0.f;
        sd += (double)d[e];
      }
    }
    st = warp_sum_d(st);
    sd = warp_sum_d(sd);
    if (lane == 0) { s.d[warp] = st; s.d2[warp] = sd; }
    __syncthreads();
    if (warp == 0) {
      double x1 = lane < kCluWarps ? s.d[lane] : 0.0, x2 = lane < kCluWarps ? s.d2[lane] : 0.0;
#pragma unroll
      for (int o = kCluWarps / 2; o > 0; o >>= 1) {
        x1 += __shfl_xor_sync(0xffffffffu, x1, o);
        x2 += __shfl_xor_sync(0xffffffffu, x2, o);
      }
      if (lane == 0) { part.st = x1; part.sd = x2; }
    }
    cl.sync();
    st = 0.0; sd = 0.0;
    if (lane < nclu) {
      const CluPart* pr = cl.map_shared_rank(&part, lane);
      st = pr->st; sd = pr->sd;
    }
#pragma unroll
    for (int o = nclu / 2; o > 0; o >>= 1) {
      st += __shfl_xor_sync(0xffffffffu, st, o);
      sd += __shfl_xor_sync(0xffffffffu, sd, o);
    }
    st = __shfl_sync(0xffffffffu, st, 0); sd = __shfl_sync(0xffffffffu, sd, 0);
    if (!drow) sd = 1.0;
    uint32_t c[4] = {(uint32_t)i, (uint32_t)b, a.off_lo, a.off_hi};
    philox4x32_10(a.key0, a.key1, c);
    const double r = (double)(c[0] >> 8) * (1.0 / 16777216.0);
    const double u2 = (double)(c[1] >> 8) * (1.0 / 16777216.0);
    if (!bonus) {
      const bool in_range = x >= 0 && x < V;
      const double logp = in_range ? ((double)trow[x] - (double)tmax) * inv_t - log(st) : -INFINITY;
      const double logq = drow ? (in_range ? ((double)drow[x] - (double)dmax) * inv_t - log(sd) : -INFINITY)
                               : 0.0;
      const double diff = logp - logq;
      const double ratio = (diff != diff) ? 0.0 : exp(fmin(diff, 0.0));
      accept = r < ratio ? 1 : 0;
    }
    if (!accept) {
      const float inv_st = (float)(1.0 / st), inv_sd = (float)(1.0 / sd);
      // attempt 0: residual max(0, p - q); attempt 1: p itself (extra row, or an empty residual)
      for (int attempt = bonus ? 1 : 0; attempt < 2 && token < 0; ++attempt) {
        float w[V4 * 4];
        double mine = 0.0;
        int lastp = -1;
#pragma unroll
        for (int e = 0; e < V4 * 4; ++e) {
          const float p = t[e] * inv_st;
          float wv = p;
          if (attempt == 0) {
            const float q = drow ? d[e] * inv_sd : ((v0 + e == x) ? 1.f : 0.f);
            wv = fmaxf(p - q, 0.f);
          }
          w[e] = (e < C && v0 + e < V) ? wv : 0.f;
          mine += (double)w[e];
          if (w[e] > 0.f) lastp = v0 + e;
        }
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += up;
        }
        lastp = __reduce_max_sync(0xffffffffu, lastp);
        __syncthreads();   // the scratch arrays are free again
        if (lane == 31) { s.d[warp] = incl; s.i[warp] = lastp; }
        __syncthreads();
        if (tid == 0) {
          double x1 = 0.0;
          int lp = -1;
          for (int k = 0; k < kCluWarps; ++k) { x1 += s.d[k]; lp = max(lp, s.i[k]); }
          part.wsum = x1; part.lastp = lp; part.pick = -1;
        }
        cl.sync();
        // level 1: the block whose running sum first exceeds the target (lane r holds block r's
        // weight; a shuffle scan gives every block's running sum)
        double bw = lane < nclu ? cl.map_shared_rank(&part, lane)->wsum : 0.0;
        double binc = bw;
#pragma unroll
        for (int o = 1; o < nclu; o <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, binc, o);
          if (lane >= o) binc += up;
        }
        const double total = __shfl_sync(0xffffffffu, binc, nclu - 1);
        int sel = -1;
        if (total > 0.0) {
          const double target = u2 * total;
          const unsigned over_b = __ballot_sync(0xffffffffu, lane < nclu && binc > target);
          double base = 0.0;
          if (over_b) {
            sel = __ffs(over_b) - 1;
            base = __shfl_sync(0xffffffffu, binc - bw, sel);
          }
          if (sel == rank) {
            // level 2: the warp, level 3: the lane, level 4: the token
            double t2 = target - base, wrun = 0.0, wbase = 0.0;
            int wsel = -1;
            for (int k = 0; k < kCluWarps; ++k) {
              const double nx = wrun + s.d[k];
              if (wsel < 0 && nx > t2) { wsel = k; wbase = wrun; }
              wrun = nx;
            }
            if (warp == wsel) {
              const double t3 = t2 - wbase;
              const unsigned over = __ballot_sync(0xffffffffu, incl > t3);
              if (over) {
                const int src = __ffs(over) - 1;
                double excl = __shfl_up_sync(0xffffffffu, incl, 1);
                if (lane == 0) excl = 0.0;
                if (lane == src) {
                  const double t4 = t3 - excl;
                  double run4 = 0.0;
                  int pick = -1, lp = -1;
#pragma unroll
                  for (int e = 0; e < V4 * 4; ++e) {
                    if (w[e] > 0.f) lp = e;
                    run4 += (double)w[e];
                    if (pick < 0 && run4 > t4) pick = e;
                  }
                  if (pick < 0) pick = lp;
                  if (pick >= 0) part.pick = v0 + pick;
                }
              }
            }
          }
        }
        cl.sync();
        if (total > 0.0) {
          // rounding may leave no token chosen on the way down: take the last one with weight
          token = sel >= 0 ? cl.map_shared_rank(&part, sel)->pick : -1;
          if (token < 0)
            for (int rr = 0; rr < nclu; ++rr) token = max(token, cl.map_shared_rank(&part, rr)->lastp);
        }
        cl.sync();   // all reads of this attempt's partials are done before they are rewritten
      }
      if (token < 0) token = targ;
    }
  }
  if (rank == 0 && tid == 0) finish_position(a, i, b, accept, bad, token);
  cl.sync();   // no block leaves while another may still read its shared memory
}


// The 8-block cluster is fixed at compile time; the 16-block one (an opt-in size) is a launch attribute.
__global__ void __cluster_dims__(kClu, 1, 1) __launch_bounds__(kCluThreads) k_verify_cluster(VerifyArgs a) {
  verify_cluster_body<kClu, kCluV4>(a);
}
// (rows of up to 32768 tokens: 8 tokens per thread)
__global__ void __cluster_dims__(kClu, 1, 1) __launch_bounds__(kCluThreads) k_verify_cluster_v2(VerifyArgs a) {
  verify_cluster_body<kClu, 2>(a);
}
__global__ void __launch_bounds__(kCluThreads) k_verify_cluster16(VerifyArgs a) {
  verify_cluster_body<16, kCluV4>(a);
}
// Four blocks per row pair: for batches whose 8-block clusters would not be resident at once
// (one block fills an SM), while a thread can still hold its share of a row (16 tokens).
constexpr int kCluSmall = 4;
constexpr int kCluSmallMaxVocab = kCluSmall * kCluThreads * 4 * kCluV4;
__global__ void __cluster_dims__(kCluSmall, 1, 1) __launch_bounds__(kCluThreads) k_verify_cluster4(VerifyArgs a) {
  verify_cluster_body<kCluSmall, kCluV4>(a);
}

// ---- token-tree verification (Algorithm 1 in full) -------------------------------------------
// One cluster per (decision row, sequence): row u = 0 is the root, u = 1 + i the node i.  The
// cluster holds the target row of u and the draft row of its children's depth in registers and
// tries the children in turn.  After j rejections the target distribution of Algorithm 1 is
// norm((p - c q)+) with c_0 = 0, c_{j+1} = c_j + Z(c_j), Z(c) = sum_v (p_v - c q_v)+ (the
// repeated "subtract q, clip, renormalise" in closed form), so a rejection costs one reduction
// over the cluster.  If no child is accepted (or u is a leaf) the cluster draws the token that
// would be emitted at u.  The last cluster of a sequence to finish walks the tree from the root
// along the accepted children.  Nothing spins.
struct TreeTopo {
  int n_nodes, max_depth;
  unsigned char depth[PS_MAX_TREE_NODES];
  unsigned char child_off[PS_MAX_TREE_NODES + 2];   // children of decision row u: child_idx[off[u] .. off[u+1])
  unsigned char child_idx[PS_MAX_TREE_NODES];
};

struct TreeArgs {
  int B, V;
  TreeTopo topo;
  const int* tokens;           // [B][n_nodes]
  const float* draft_logits;   // [B][max_depth][V]
  const float* target_logits;  // [B][n_nodes+1][V]
  float temperature;
  uint32_t key0, key1, off_lo, off_hi;
  int* accept_len; int* out_tokens; int* n_out; int* path;
  TreeRec* rec;                // [B][PS_MAX_TREE_NODES+1]
  unsigned* tickets;           // [B], zero on entry and on exit
  int* status;
};

// Sum over the cluster of one double per thread; every thread of every block gets the value.
__device__ double cluster_sum(cooperative_groups::cluster_group& cl, CluPart& part, CluScratch& s, double v,
                              int tid, int warp, int lane) {
  v = warp_sum_d(v);
  __syncthreads();
  if (lane == 0) s.d[warp] = v;
  __syncthreads();
  if (tid == 0) {
    double x1 = 0.0;
    for (int w = 0; w < kCluWarps; ++w) x1 += s.d[w];
    part.wsum = x1;
  }
  cl.sync();
  // lane r fetches block r's sum (one remote round trip), a shuffle tree adds them
  double tot = lane < (int)cl.num_blocks() ? cl.map_shared_rank(&part, lane)->wsum : 0.0;
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
  tot = __shfl_sync(0xffffffffu, tot, 0);
  cl.sync();   // every block has read the partials before they are rewritten
  return tot;
}

// Inverse-CDF draw by the cluster over per-thread weights w[] (thread owns tokens v0 + e): the
// first token whose running sum exceeds u * total, found block -> warp -> lane -> token.
// Returns the token to every thread of every block, -1 if the total weight is not positive.
__device__ int cluster_draw(cooperative_groups::cluster_group& cl, CluPart& part, CluScratch& s,
                            const float (&w)[kCluV4 * 4], int v0, double u, int rank, int tid, int warp,
                            int lane) {
  double mine = 0.0;
  int lastp = -1;
#pragma unroll
  for (int e = 0; e < kCluV4 * 4; ++e) {
    mine += (double)w[e];
    if (w[e] > 0.f) lastp = v0 + e;
  }
  double incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  lastp = __reduce_max_sync(0xffffffffu, lastp);
  __syncthreads();
  if (lane == 31) { s.d[warp] = incl; s.i[warp] = lastp; }
  __syncthreads();
  if (tid == 0) {
    double x1 = 0.0;
    int lp = -1;
    for (int k = 0; k < kCluWarps; ++k) { x1 += s.d[k]; lp = max(lp, s.i[k]); }
    part.wsum = x1; part.lastp = lp; part.pick = -1;
  }
  cl.sync();
  // lane r holds block r's weight; a shuffle scan gives every block's running sum
  const int nb = (int)cl.num_blocks();
  const double bw = lane < nb ? cl.map_shared_rank(&part, lane)->wsum : 0.0;
  double binc = bw;
#pragma unroll
  for (int o = 1; o < 16; o <<= 1) {
    const double up = __shfl_up_sync(0xffffffffu, binc, o);
    if (lane >= o) binc += up;
  }
  const double total = __shfl_sync(0xffffffffu, binc, nb - 1);
  int sel = -1, token = -1;
  if (total > 0.0) {
    const double target = u * total;
    const unsigned over_b = __ballot_sync(0xffffffffu, lane < nb && binc > target);
    double base = 0.0;
    if (over_b) {
      sel = __ffs(over_b) - 1;
      base = __shfl_sync(0xffffffffu, binc - bw, sel);
    }
    if (sel == rank) {
      double t2 = target - base, wrun = 0.0, wbase = 0.0;
      int wsel = -1;
      for (int k = 0; k < kCluWarps; ++k) {
        const double nx = wrun + s.d[k];
        if (wsel < 0 && nx > t2) { wsel = k; wbase = wrun; }
        wrun = nx;
      }
      if (warp == wsel) {
        const double t3 = t2 - wbase;
        const unsigned over = __ballot_sync(0xffffffffu, incl > t3);
        if (over) {
          const int src = __ffs(over) - 1;
          double excl = __shfl_up_sync(0xffffffffu, incl, 1);
          if (lane == 0) excl = 0.0;
          if (lane == src) {
            const double t4 = t3 - excl;
            double run4 = 0.0;
            int pick = -1, lp = -1;
#pragma unroll
            for (int e = 0; e < kCluV4 * 4; ++e) {
              if (w[e] > 0.f) lp = e;
              run4 += (double)w[e];
              if (pick < 0 && run4 > t4) pick = e;
            }
            if (pick < 0) pick = lp;
            if (pick >= 0) part.pick = v0 + pick;
          }
        }
      }
    }
  }
  cl.sync();
  if (total > 0.0) {
    // rounding may leave no token chosen on the way down: take the last one with weight
    token = sel >= 0 ? cl.map_shared_rank(&part, sel)->pick : -1;
    if (token < 0)
      for (int rr = 0; rr < (int)cl.num_blocks(); ++rr) token = max(token, cl.map_shared_rank(&part, rr)->lastp);
  }
  cl.sync();   // all reads of the partials are done before they are rewritten
  return token;
}

// (The cluster size is a launch attribute: 8 blocks per row, or fewer when a large tree would
// otherwise need a second wave of blocks.)
__global__ void __launch_bounds__(kCluThreads) k_verify_tree(TreeArgs a) {
  namespace cg = cooperative_groups;
  cg::cluster_group cl = cg::this_cluster();
  __shared__ CluPart part;
  __shared__ CluScratch s;
  const int rank = (int)cl.block_rank();
  const int nclu = (int)cl.num_blocks();
  const int u = blockIdx.x / nclu, b = blockIdx.y, V = a.V, n_nodes = a.topo.n_nodes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int kid0 = a.topo.child_off[u], n_kids = a.topo.child_off[u + 1] - kid0;
  const int dq = u == 0 ? 0 : a.topo.depth[u - 1] + 1;   // depth of the children of u
  const bool greedy = a.temperature == 0.f;
  const float* trow = a.target_logits + ((size_t)b * (n_nodes + 1) + u) * V;
  const float* drow = (!greedy && n_kids > 0) ? a.draft_logits + ((size_t)b * a.topo.max_depth + dq) * V : nullptr;
  const int* toks = a.tokens + (size_t)b * n_nodes;
  const int nv4 = ((V + nclu * kCluThreads - 1) / (nclu * kCluThreads) + 3) / 4;
  const int C = nv4 * 4, v0 = (rank * kCluThreads + tid) * C;

  float t[kCluV4 * 4], d[kCluV4 * 4];
#pragma unroll
  for (int k = 0; k < kCluV4; ++k) {
    const int v = v0 + 4 * k;   // V % 4 == 0: a vector lies inside the row or outside it
    float4 tv = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY), dv = tv;
    if (k < nv4 && v < V) {
      tv = *reinterpret_cast<const float4*>(trow + v);
      if (drow) dv = *reinterpret_cast<const float4*>(drow + v);
    }
    t[4 * k] = tv.x; t[4 * k + 1] = tv.y; t[4 * k + 2] = tv.z; t[4 * k + 3] = tv.w;
    d[4 * k] = dv.x; d[4 * k + 1] = dv.y; d[4 * k + 2] = dv.z; d[4 * k + 3] = dv.w;
  }
  // ---- maxima (NaN counts as -inf, ties to the lower id) and non-finite flags
  float tm = -INFINITY, dm = -INFINITY;
  int ti = 0x7fffffff, bad = 0;
#pragma unroll
  for (int e = 0; e < kCluV4 * 4; ++e) {
    const int v = v0 + e;
    if (e < C && v < V) {
      float xt = t[e];
      if (xt != xt || xt == INFINITY) bad = 1;
      if (xt != xt) xt = -INFINITY;
      if (xt > tm || (xt == tm && v < ti)) { tm = xt; ti = v; }
      if (drow) {
        float xd = d[e];
        if (xd != xd || xd == INFINITY) bad = 1;
        if (xd != xd) xd = -INFINITY;
        dm = fmaxf(dm, xd);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, tm, o);
    const int oi = __shfl_xor_sync(0xffffffffu, ti, o);
    if (ov > tm || (ov == tm && oi < ti)) { tm = ov; ti = oi; }
    dm = fmaxf(dm, __shfl_xor_sync(0xffffffffu, dm, o));
    bad |= __shfl_xor_sync(0xffffffffu, bad, o);
  }
  if (lane == 0) { s.f[warp] = tm; s.i[warp] = ti; s.flag[warp] = bad; s.f2[warp] = dm; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kCluWarps; ++w) {
      if (s.f[w] > tm || (s.f[w] == tm && s.i[w] < ti)) { tm = s.f[w]; ti = s.i[w]; }
      dm = fmaxf(dm, s.f2[w]);
      bad |= s.flag[w];
    }
    part.tmax = tm; part.targ = ti; part.dmax = dm; part.bad = bad;
    part.pick = -1; part.lastp = -1; part.wsum = 0.0; part.st = 0.0; part.sd = 0.0;
  }
  cl.sync();
  tm = -INFINITY; dm = -INFINITY; ti = 0x7fffffff; bad = 0;
  for (int r = 0; r < (int)cl.num_blocks(); ++r) {
    const CluPart* pr = cl.map_shared_rank(&part, r);
    const float ov = pr->tmax;
    const int oi = pr->targ;
    if (ov > tm || (ov == tm && oi < ti)) { tm = ov; ti = oi; }
    dm = fmaxf(dm, pr->dmax);
    bad |= pr->bad;
  }
  cl.sync();   // the partials are free again
  if (tm == -INFINITY || (drow && dm == -INFINITY)) bad = 1;  // a row without a distribution
  const float tmax = tm, dmax = dm;
  const int targ = ti;

  int next = -1, token = -1;
  if (greedy) {
    for (int j = 0; j < n_kids && next < 0; ++j)
      if (toks[a.topo.child_idx[kid0 + j]] == targ) next = a.topo.child_idx[kid0 + j];
    token = targ;
    bad = 0;
  } else if (bad) {
    token = targ;
  } else {
    // every block takes the same branches below: the values they depend on are identical
    const double inv_t = 1.0 / (double)a.temperature;
    double st = 0.0, sd = 0.0;
#pragma unroll
    for (int e = 0; e < kCluV4 * 4; ++e) {
      const bool in = e < C && v0 + e < V;
      t[e] = in ? expf((float)(((double)t[e] - (double)tmax) * inv_t)) : 0.f;
      st += (double)t[e];
      d[e] = (in && drow) ? expf((float)(((double)d[e] - (double)dmax) * inv_t)) : 0.f;
      sd += (double)d[e];
    }
    st = cluster_sum(cl, part, s, st, tid, warp, lane);
    sd = drow ? cluster_sum(cl, part, s, sd, tid, warp, lane) : 1.0;
    const float inv_st = (float)(1.0 / st), inv_sd = (float)(1.0 / sd);
    double c = 0.0, Zc = 1.0;   // the target distribution at u is now (p - c q)+ / Zc
    for (int j = 0; j < n_kids; ++j) {
      const int kid = a.topo.child_idx[kid0 + j];
      const int x = toks[kid];
      uint32_t ctr[4] = {(uint32_t)u + ((uint32_t)j << 16), (uint32_t)b, a.off_lo, a.off_hi};
      philox4x32_10(a.key0, a.key1, ctr);
      const double r = (double)(ctr[0] >> 8) * (1.0 / 16777216.0);
      const bool in_range = x >= 0 && x < V;
      const double logp = in_range ? ((double)trow[x] - (double)tmax) * inv_t - log(st) : -INFINITY;
      const double logq = in_range ? ((double)drow[x] - (double)dmax) * inv_t - log(sd) : -INFINITY;
      double ratio;
      if (c == 0.0) {
        const double diff = logp - logq;
        ratio = (diff != diff) ? 0.0 : exp(fmin(diff, 0.0));
      } else {
        const double px = exp(logp), qx = exp(logq);
        const double wx = fmax(px - c * qx, 0.0) / Zc;
        ratio = qx > 0.0 ? fmin(wx / qx, 1.0) : (wx > 0.0 ? 1.0 : 0.0);
      }
      if (r < ratio) { next = kid; break; }
      // rejected: the target distribution becomes norm((p - (c + Zc) q)+)
      const double c_new = c + Zc;
      const float cf = (float)c_new;
      double mine = 0.0;
#pragma unroll
      for (int e = 0; e < kCluV4 * 4; ++e) mine += (double)fmaxf(t[e] * inv_st - cf * (d[e] * inv_sd), 0.f);
      const double Z = cluster_sum(cl, part, s, mine, tid, warp, lane);
      if (Z > 0.0) { c = c_new; Zc = Z; } else { c = 0.0; Zc = 1.0; }   // nothing left: back to p
    }
    if (next < 0) {
      uint32_t ctr[4] = {(uint32_t)u, (uint32_t)b, a.off_lo, a.off_hi};
      philox4x32_10(a.key0, a.key1, ctr);
      const double u2 = (double)(ctr[1] >> 8) * (1.0 / 16777216.0);
      const float cf = (float)c;
      float w[kCluV4 * 4];
#pragma unroll
      for (int e = 0; e < kCluV4 * 4; ++e) w[e] = fmaxf(t[e] * inv_st - cf * (d[e] * inv_sd), 0.f);
      token = cluster_draw(cl, part, s, w, v0, u2, rank, tid, warp, lane);
      if (token < 0 && c != 0.0) {   // the residual vanished in fp32: draw from p
#pragma unroll
        for (int e = 0; e < kCluV4 * 4; ++e) w[e] = t[e] * inv_st;
        token = cluster_draw(cl, part, s, w, v0, u2, rank, tid, warp, lane);
      }
      if (token < 0) token = targ;
    }
  }
  if (rank == 0 && tid == 0) {
    TreeRec* rec = a.rec + (size_t)b * (PS_MAX_TREE_NODES + 1);
    rec[u].next = next; rec[u].token = token; rec[u].bad = bad;
    __threadfence();
    const unsigned tk = atomicAdd(&a.tickets[b], 1u);
    if (tk == (unsigned)n_nodes) {   // the last of the n_nodes + 1 decision rows
      __threadfence();
      volatile TreeRec* R = rec;
      int* out = a.out_tokens + (size_t)b * (a.topo.max_depth + 1);
      int* pth = a.path + (size_t)b * a.topo.max_depth;
      int uu = 0, len = 0, any_bad = 0;
      for (;;) {
        any_bad |= R[uu].bad;
        const int nx = R[uu].next;
        if (nx < 0 || len >= a.topo.max_depth) { out[len] = R[uu].token; break; }
        out[len] = toks[nx];
        pth[len] = nx;
        ++len;
        uu = nx + 1;
      }
      for (int j = len + 1; j <= a.topo.max_depth; ++j) out[j] = -1;
      for (int j = len; j < a.topo.max_depth; ++j) pth[j] = -1;
      a.accept_len[b] = len;
      a.n_out[b] = len + 1;
      if (any_bad) atomicOr(a.status, kStatNonfinite);
      a.tickets[b] = 0u;
    }
  }
  cl.sync();   // no block leaves while another may still read its shared memory
}

// Token tree from the top-n lists of a draft step (see ps_build_tree): one thread per node.
struct BuildArgs {
  int B, n_nodes, R, top_n;
  unsigned char depth[PS_MAX_TREE_NODES], rank[PS_MAX_TREE_NODES];
  const int* top_ids; const int* sampled; int* tokens;
};
__global__ void k_build_tree(BuildArgs a) {
  const int i = threadIdx.x, b = blockIdx.x;
  if (i >= a.n_nodes) return;
  const int t = a.depth[i], r = a.rank[i];
  const int* top = a.top_ids + ((size_t)b * a.R + t) * a.top_n;
  int tok = top[r];
  if (a.sampled) {
    const int sx = a.sampled[(size_t)b * a.R + t];
    if (r == 0) tok = sx;
    else if (tok == sx) tok = top[0];
  }
  a.tokens[(size_t)b * a.n_nodes + i] = tok;
}

}  // namespace

ps_status launch_build_tree(ps_ctx* c, int B, int n_nodes, const int* parent, const int* rank, const int* top_ids,
                            int top_n, const int* sampled_ids, int* tokens, cudaStream_t st) {
  BuildArgs a;
  a.B = B; a.n_nodes = n_nodes; a.R = c->cfg.k_masks + 1; a.top_n = top_n;
  a.top_ids = top_ids; a.sampled = sampled_ids; a.tokens = tokens;
  for (int i = 0; i < n_nodes; ++i) {
    if (parent[i] >= i || parent[i] < -1) return fail(c, PS_ERR_INVALID_ARG, "parent[i] must be -1 or a node before i");
    const int d = parent[i] < 0 ? 0 : a.depth[parent[i]] + 1;
    if (d >= a.R) return fail(c, PS_ERR_INVALID_ARG, "the tree is deeper than the k+1 rows of a draft step");
    if (rank[i] < 0 || rank[i] >= top_n) return fail(c, PS_ERR_INVALID_ARG, "rank[i] must be in [0, top_n)");
    for (int j = 0; j < i; ++j)
      if (parent[j] == parent[i] && rank[j] == rank[i])
        return fail(c, PS_ERR_INVALID_ARG, "two siblings of the same rank would carry the same token");
    a.depth[i] = (unsigned char)d;
    a.rank[i] = (unsigned char)rank[i];
  }
  k_build_tree<<<B, PS_MAX_TREE_NODES, 0, st>>>(a);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_build_tree");
}

// Launch with a cluster of nclu blocks along x (a launch attribute, not a compile-time one).
template <class Args>
cudaError_t launch_cluster(void (*kern)(Args), dim3 grid, int nclu, cudaStream_t st, const Args& a) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kCluThreads);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = nclu; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

// Whether the context's device can co-schedule nclu blocks of this kernel as one cluster (sizes
// above 8 are an opt-in of the kernel, a per-device function attribute).  Asked once per context
// and size; `cache` is the context's row for this kernel.
template <class Args>
bool cluster_size_ok(int* cache, void (*kern)(Args), int nclu) {
  if (nclu <= 8) return true;
  if (cache[nclu] == 0) {
    cache[nclu] = -1;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(nclu);
      cfg.blockDim = dim3(kCluThreads);
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = nclu; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      cfg.attrs = at;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n > 0) cache[nclu] = 1;
    }
    (void)cudaGetLastError();
  }
  return cache[nclu] > 0;
}

ps_status launch_verify(ps_ctx* c, int B, int n_draft, int n_target, const int* draft_tokens,
                        const float* draft_logits, const float* target_logits, float temperature,
                        uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens,
                        int* n_out, cudaStream_t st) {
  VerifyArgs a;
  a.B = B; a.n_draft = n_draft; a.n_target = n_target; a.V = c->cfg.vocab;
  a.draft_tokens = draft_tokens; a.draft_logits = draft_logits; a.target_logits = target_logits;
  a.temperature = temperature;
  a.key0 = (uint32_t)seed; a.key1 = (uint32_t)(seed >> 32);
  a.off_lo = (uint32_t)offset; a.off_hi = (uint32_t)(offset >> 32);
  a.accept_len = accept_len; a.out_tokens = out_tokens; a.n_out = n_out;
  a.rec = c->vrec; a.tickets = c->tickets; a.status = c->dev_status;
  const bool aligned = (((uintptr_t)target_logits | (uintptr_t)draft_logits) & 15u) == 0;
  const int nclu = a.V <= kCluMaxVocab ? kClu : 16;
  if (a.V % 4 == 0 && a.V <= kCluMaxVocab16 && aligned && (nclu == kClu || cluster_size_ok(c->cluster_ok[0], k_verify_cluster16, 16))) {
    prof_mark(c, st, "begin");
    cudaError_t e;
    // (plain launches: as dependents of the LM head these kernels start their loads earlier and
    // run 3 us shorter alone, but the step gets 3 us longer -- measured twice: clusters of 8
    // blocks that each fill an SM are slow to place while the LM head's CTAs drain)
    const bool pdl = false;
    if (nclu == kClu && a.V <= kCluSmallMaxVocab && n_target * B * kClu > c->n_sm) {   // half the waves
      e = launch_after(k_verify_cluster4, dim3(n_target * kCluSmall, B), dim3(kCluThreads), 0, st, pdl, a);
    } else if (nclu == kClu) {
      e = launch_after(a.V <= kClu * kCluThreads * 4 * 2 ? k_verify_cluster_v2 : k_verify_cluster,
                       dim3(n_target * kClu, B), dim3(kCluThreads), 0, st, pdl, a);
    } else {
      e = launch_cluster(k_verify_cluster16, dim3(n_target * 16, B), 16, st, a);
    }
    c->launches++;
    prof_mark(c, st, "verify");
    return cuda_check(c, e, "k_verify_cluster");
  }
  size_t smem = (size_t)((a.V + kSeg - 1) / kSeg) * sizeof(double);
  if (smem > 160 * 1024) return fail(c, PS_ERR_UNSUPPORTED, "vocab too large for ps_verify");
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k_verify, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_check(c, e, "verify smem");
  }
  prof_mark(c, st, "begin");
  k_verify<<<dim3(n_target, B), kThreads, smem, st>>>(a);
  c->launches++;
  prof_mark(c, st, "verify");
  return cuda_check(c, cudaGetLastError(), "k_verify");
}

ps_status launch_verify_tree(ps_ctx* c, int B, int n_nodes, const int* parent, const int* tokens,
                             const float* draft_logits, const float* target_logits, float temperature,
                             uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
                             int* path, int* max_depth_out, cudaStream_t st) {
  TreeArgs a;
  a.B = B; a.V = c->cfg.vocab;
  TreeTopo& tp = a.topo;
  tp.n_nodes = n_nodes;
  tp.max_depth = 0;
  for (int i = 0; i < n_nodes; ++i) {
    if (parent[i] >= i || parent[i] < -1) return fail(c, PS_ERR_INVALID_ARG, "parent[i] must be -1 or a node before i");
    tp.depth[i] = (unsigned char)(parent[i] < 0 ? 0 : tp.depth[parent[i]] + 1);
    tp.max_depth = std::max(tp.max_depth, (int)tp.depth[i] + 1);
  }
  int off = 0;
  for (int u = 0; u <= n_nodes; ++u) {   // children of decision row u in increasing node id
    tp.child_off[u] = (unsigned char)off;
    for (int i = 0; i < n_nodes; ++i)
      if (parent[i] == u - 1) tp.child_idx[off++] = (unsigned char)i;
  }
  tp.child_off[n_nodes + 1] = (unsigned char)off;
  if (max_depth_out) *max_depth_out = tp.max_depth;
  if (temperature != 0.f && !draft_logits) return fail(c, PS_ERR_INVALID_ARG, "draft_logits needed at temperature > 0");
  const bool aligned = (((uintptr_t)target_logits | (uintptr_t)draft_logits) & 15u) == 0;
  if (a.V % 4 || a.V > kCluMaxVocab16 || !aligned)
    return fail(c, PS_ERR_UNSUPPORTED, "ps_verify_tree needs vocab % 4 == 0, vocab <= 131072 and 16-byte aligned logits");
  a.tokens = tokens; a.draft_logits = draft_logits; a.target_logits = target_logits;
  a.temperature = temperature;
  a.key0 = (uint32_t)seed; a.key1 = (uint32_t)(seed >> 32);
  a.off_lo = (uint32_t)offset; a.off_hi = (uint32_t)(offset >> 32);
  a.accept_len = accept_len; a.out_tokens = out_tokens; a.n_out = n_out; a.path = path;
  a.rec = c->trec; a.tickets = c->tree_tickets; a.status = c->dev_status;
  prof_mark(c, st, "begin");
  // blocks per decision row: 8 (16 for vocabularies beyond 65536), fewer when the tree would
  // otherwise need a second wave of blocks and a thread can still hold its share of a row
  int nclu = a.V <= kCluMaxVocab ? kClu : 16;
  if (!cluster_size_ok(c->cluster_ok[1], k_verify_tree, nclu))
    return fail(c, PS_ERR_UNSUPPORTED, "this device cannot run the 16-block clusters a vocabulary beyond 65536 needs");
  while (nclu > 1 && (long)(n_nodes + 1) * B * nclu > c->n_sm && a.V <= (nclu / 2) * kCluThreads * 4 * kCluV4)
    nclu /= 2;
  cudaError_t e = launch_cluster(k_verify_tree, dim3((n_nodes + 1) * nclu, B), nclu, st, a);
  c->launches++;
  prof_mark(c, st, "verify_tree");
  return cuda_check(c, e, "k_verify_tree");
}

}  // namespace ps

extern "C" ps_status ps_philox_fill(const uint32_t key[2], const uint32_t* ctr, uint32_t* out, int n,
                                    void* stream) {
  if (!key || !ctr || !out || n < 0) return PS_ERR_INVALID_ARG;
  if (n == 0) return PS_OK;
  ps::k_philox_fill<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>(key[0], key[1], ctr, out, n);
  return cudaGetLastError() == cudaSuccess ? PS_OK : PS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------
// ps_verify_static: the same kernel with its scratch in a fixed device array of this library
// instead of a caller-allocated workspace, for callers that must not allocate.
namespace ps {
namespace {

struct StaticScratch {
  unsigned tickets[PS_STATIC_MAX_BATCH];                       // must be zero when a call starts
  VerifyRec rec[PS_STATIC_MAX_BATCH * (PS_MAX_MASKS + 2)];     // fully rewritten by every call
  int status_sink;                                             // takes the flag when the caller passes none
};

// About 18 KB, held by every GPU that loads the library until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the CURRENT device, looked up once per device.  The array's
// name is only a host-side handle here; a kernel must be given the address obtained below.
cudaError_t static_scratch_address(StaticScratch** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = p;
  }
  *out = (StaticScratch*)g_static_ptr[dev];
  return cudaSuccess;
}

ps_status static_fail(char* err, size_t cap, ps_status s, const char* text) {
  if (err && cap) std::snprintf(err, cap, "%s", text);
  return s;
}

}  // namespace
}  // namespace ps

extern "C" ps_status ps_verify_static(int vocab, int B, int n_draft, int n_target,
                                      const int* draft_tokens, const float* draft_logits,
                                      const float* target_logits, float temperature, uint64_t seed,
                                      uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
                                      int* nonfinite_flag, char* err, size_t err_cap, void* stream) {
  using namespace ps;
  if (err && err_cap) err[0] = 0;
  if (!draft_tokens || !target_logits || !accept_len || !out_tokens || !n_out)
    return static_fail(err, err_cap, PS_ERR_INVALID_ARG, "ps_verify_static: null pointer");
  if (B < 1 || n_draft < 1 || vocab < 1)
    return static_fail(err, err_cap, PS_ERR_INVALID_ARG, "ps_verify_static: sizes must be positive");
  if (B > PS_STATIC_MAX_BATCH)
    return static_fail(err, err_cap, PS_ERR_CAPACITY,
                       "ps_verify_static: B exceeds PS_STATIC_MAX_BATCH (the fixed scratch holds 128 sequences)");
  if (n_draft > PS_MAX_MASKS + 1)
    return static_fail(err, err_cap, PS_ERR_CAPACITY,
                       "ps_verify_static: n_draft exceeds PS_MAX_MASKS+1 (16 positions per sequence)");
  if (vocab > PS_STATIC_MAX_VOCAB)
    return static_fail(err, err_cap, PS_ERR_CAPACITY,
                       "ps_verify_static: vocab exceeds PS_STATIC_MAX_VOCAB (262144)");
  if (n_target != n_draft && n_target != n_draft + 1)
    return static_fail(err, err_cap, PS_ERR_INVALID_ARG,
                       "ps_verify_static: n_target must be n_draft or n_draft+1");
  if (!(temperature >= 0.f))
    return static_fail(err, err_cap, PS_ERR_INVALID_ARG, "ps_verify_static: temperature must be >= 0");
  StaticScratch* sc = nullptr;
  cudaError_t e = static_scratch_address(&sc);
  if (e != cudaSuccess) return static_fail(err, err_cap, PS_ERR_CUDA, cudaGetErrorString(e));
  cudaStream_t st = (cudaStream_t)stream;
  // The arrival counters keep whatever the previous call left; they must start at zero.
  e = cudaMemsetAsync(sc->tickets, 0, sizeof(sc->tickets), st);
  if (e != cudaSuccess) return static_fail(err, err_cap, PS_ERR_CUDA, cudaGetErrorString(e));
  VerifyArgs a;
  a.B = B; a.n_draft = n_draft; a.n_target = n_target; a.V = vocab;
  a.draft_tokens = draft_tokens; a.draft_logits = draft_logits; a.target_logits = target_logits;
  a.temperature = temperature;
  a.key0 = (uint32_t)seed; a.key1 = (uint32_t)(seed >> 32);
  a.off_lo = (uint32_t)offset; a.off_hi = (uint32_t)(offset >> 32);
  a.accept_len = accept_len; a.out_tokens = out_tokens; a.n_out = n_out;
  a.rec = sc->rec; a.tickets = sc->tickets;
  a.status = nonfinite_flag ? nonfinite_flag : &sc->status_sink;
  size_t smem = (size_t)((vocab + kSeg - 1) / kSeg) * sizeof(double);   // <= 16 KB at the vocab limit
  k_verify<<<dim3(n_target, B), kThreads, smem, st>>>(a);
  e = cudaGetLastError();
  if (e != cudaSuccess) return static_fail(err, err_cap, PS_ERR_CUDA, cudaGetErrorString(e));
  return PS_OK;
}
