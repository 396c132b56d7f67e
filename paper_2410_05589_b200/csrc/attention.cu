// Split-KV attention of the fused bf16 draft step (Sec. 4.1: the k+1 rows of a sequence see the
// cached real positions and the new rows up to themselves).
//
// Work item = (head, key split, sequence); 128 threads.  A block walks its key range in tiles
// of 128 keys: the K and V rows of a tile are staged in shared memory with coalesced 16-byte
// loads (bf16, padded rows), every thread scores ONE key against all R query rows in fp32,
// the tile's softmax is folded into running (max, sum) pairs, and every thread then owns one
// output channel for the P*V product.  q and the new k rows are rotated on the fly (RoPE, pair
// (i, i + D/2), angle pos * base^(-2i/D), the angle formed and reduced in double); cached keys
// are already rotated.  New k/v rows are rounded to bf16 as a cache row would be.
// Output: un-normalised partial (max, sum, o) per (row, head, split); the last split of a
// (sequence, head) to finish merges them into the hi/lo bf16 planes the o-projection reads.
#include <cfloat>

#include "ps_internal.cuh"

namespace ps {
namespace {

constexpr int kTile = 128;      // keys per tile = threads per block
constexpr int kPad = 8;         // bf16 elements of padding per staged row (16 bytes)

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// 16-byte asynchronous copy global -> shared (both addresses 16-byte aligned).
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)),
               "l"(src)
               : "memory");
}

template <int D>
__global__ void __launch_bounds__(kTile) k_attn_tile(SeqMap sm, const float* __restrict__ qkv, int ldq,
                                                     int Hq, int Hkv,
                                                     const __nv_bfloat16* __restrict__ kcache,
                                                     const __nv_bfloat16* __restrict__ vcache,
                                                     int n_heads, int n_kv_heads, int max_ctx,
                                                     const double* __restrict__ inv_freq, int n_split,
                                                     float* __restrict__ att_ml,
                                                     float* __restrict__ att_o, unsigned* tickets,
                                                     __nv_bfloat16* __restrict__ out_hi,
                                                     __nv_bfloat16* __restrict__ out_lo) {
  constexpr int RMAX = kMaxRowsPerSeq, P = D + kPad, HALF = D / 2;
  extern __shared__ __align__(16) unsigned char att_smem[];
  const int h = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int R = sm.row_off[b + 1] - sm.row_off[b], L = sm.len[b], m0 = sm.row_off[b] - sm.row_base;
  const int hk = h / (n_heads / n_kv_heads);
  // shared memory carve-up
  float* s_q = reinterpret_cast<float*>(att_smem);              // [R][D], scaled and rotated
  float* s_cs = s_q + R * D;                                    // [R][HALF] cos
  float* s_sn = s_cs + R * HALF;                                // [R][HALF] sin
  float* s_p = s_sn + R * HALF;                                 // [R][kTile] scores / probabilities
  float* s_corr = s_p + R * kTile;                              // [2][RMAX] tile max, tile sum
  __nv_bfloat16* s_k = reinterpret_cast<__nv_bfloat16*>(s_corr + 2 * RMAX);   // [kTile][P]
  __nv_bfloat16* s_v = s_k + kTile * P;                                   // [kTile][P]

  // rotation table of the R new positions
  for (int idx = tid; idx < R * HALF; idx += kTile) {
    const int j = idx / HALF, i = idx - j * HALF;
    double ang = (double)(L + j) * inv_freq[i];
    ang -= 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
    float sn, cs;
    sincosf((float)ang, &sn, &cs);
    s_cs[idx] = cs;
    s_sn[idx] = sn;
  }
  __syncthreads();
  const float scale = rsqrtf((float)D);
  for (int idx = tid; idx < R * HALF; idx += kTile) {
    const int j = idx / HALF, i = idx - j * HALF;
    const float* row = qkv + (size_t)(m0 + j) * ldq + h * D;
    const float q0 = row[i], q1 = row[i + HALF], c = s_cs[idx], s = s_sn[idx];
    s_q[j * D + i] = (q0 * c - q1 * s) * scale;
    s_q[j * D + i + HALF] = (q1 * c + q0 * s) * scale;
  }

  const int total = L + R;
  int per = (total + n_split - 1) / n_split;
  per = (per + kTile - 1) / kTile * kTile;               // whole tiles per split
  const int t_begin = min(total, split * per), t_end = min(total, t_begin + per);
  const __nv_bfloat16* kb = kcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;
  const __nv_bfloat16* vb = vcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;

  float run_m[RMAX], run_l[RMAX], o[RMAX];     // running max / sum (replicated), output channel tid
#pragma unroll
  for (int j = 0; j < RMAX; ++j) { run_m[j] = -FLT_MAX; run_l[j] = 0.f; o[j] = 0.f; }

  for (int t0 = t_begin; t0 < t_end; t0 += kTile) {
    const int nk = min(kTile, t_end - t0);
    __syncthreads();                             // previous tile fully consumed
    // ---- stage K and V rows [t0, t0+nk): cached rows by 16-byte loads, new rows from qkv
    constexpr int VPR = D / 8;                   // 16-byte vectors per row
    // (asynchronous copies: all of a thread's loads are in flight together)
    for (int idx = tid; idx < nk * VPR; idx += kTile) {
      const int r = idx / VPR, v = idx - r * VPR, t = t0 + r;
      if (t < L) {
        cp_async16(s_k + r * P + v * 8, kb + (size_t)t * D + v * 8);
        cp_async16(s_v + r * P + v * 8, vb + (size_t)t * D + v * 8);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (t0 + nk > L) {                           // the tile holds new rows: rotate k, round k and v
      const int first = max(L, t0);
      for (int idx = tid; idx < (t0 + nk - first) * HALF; idx += kTile) {
        const int jj = idx / HALF, i = idx - jj * HALF, j = first - L + jj, r = first - t0 + jj;
        const float* row = qkv + (size_t)(m0 + j) * ldq;
        const float k0 = row[Hq + hk * D + i], k1 = row[Hq + hk * D + i + HALF];
        const float c = s_cs[j * HALF + i], s = s_sn[j * HALF + i];
        s_k[r * P + i] = __float2bfloat16_rn(k0 * c - k1 * s);
        s_k[r * P + i + HALF] = __float2bfloat16_rn(k1 * c + k0 * s);
        s_v[r * P + i] = __float2bfloat16_rn(row[Hq + Hkv + hk * D + i]);
        s_v[r * P + i + HALF] = __float2bfloat16_rn(row[Hq + Hkv + hk * D + i + HALF]);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // ---- scores: thread tid <-> key t0 + tid, all rows
    {
      float sc[RMAX];
#pragma unroll
      for (int j = 0; j < RMAX; ++j) sc[j] = 0.f;
      if (tid < nk) {
        const __nv_bfloat16* krow = s_k + tid * P;
#pragma unroll 4
        for (int v = 0; v < VPR; ++v) {
          const uint4 kq = *reinterpret_cast<const uint4*>(krow + v * 8);
          const uint32_t w[4] = {kq.x, kq.y, kq.z, kq.w};
          float kf[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            kf[2 * i] = __uint_as_float(w[i] << 16);
            kf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
          }
#pragma unroll
          for (int j = 0; j < RMAX; ++j) {
            if (j < R) {
              const float4 qa = *reinterpret_cast<const float4*>(s_q + j * D + v * 8);
              const float4 qb = *reinterpret_cast<const float4*>(s_q + j * D + v * 8 + 4);
              sc[j] += kf[0] * qa.x + kf[1] * qa.y + kf[2] * qa.z + kf[3] * qa.w + kf[4] * qb.x +
                       kf[5] * qb.y + kf[6] * qb.z + kf[7] * qb.w;
            }
          }
        }
      }
      const int t = t0 + tid;
#pragma unroll
      for (int j = 0; j < RMAX; ++j)
        if (j < R) s_p[j * kTile + tid] = (tid < nk && (t < L || t - L <= j)) ? sc[j] : -FLT_MAX;
    }
    __syncthreads();
    // ---- tile softmax: warp w handles rows w, w+4, ...
    for (int j = warp; j < R; j += kTile / 32) {
      float* pr = s_p + j * kTile;
      float x[kTile / 32], mx = -FLT_MAX;
#pragma unroll
      for (int i = 0; i < kTile / 32; ++i) { x[i] = pr[lane + 32 * i]; mx = fmaxf(mx, x[i]); }
      mx = warp_max(mx);
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < kTile / 32; ++i) {
        const float p = x[i] > -FLT_MAX ? __expf(x[i] - mx) : 0.f;
        pr[lane + 32 * i] = p;
        sum += p;
      }
      sum = warp_sum(sum);
      if (lane == 0) { s_corr[j] = mx; s_corr[RMAX + j] = sum; }   // tile max and tile sum
    }
    __syncthreads();
    // ---- fold the tile into the running state; thread tid <-> output channel tid
    float f_old[RMAX], f_new[RMAX];
#pragma unroll
    for (int j = 0; j < RMAX; ++j) {
      if (j < R) {
        const float tm = s_corr[j], ts = s_corr[RMAX + j];
        const float mnew = fmaxf(run_m[j], tm);
        f_old[j] = __expf(run_m[j] - mnew);
        f_new[j] = tm > -FLT_MAX ? __expf(tm - mnew) : 0.f;
        run_l[j] = run_l[j] * f_old[j] + ts * f_new[j];
        run_m[j] = mnew;
      }
    }
    if (tid < D) {
      float acc[RMAX];
#pragma unroll
      for (int j = 0; j < RMAX; ++j) acc[j] = 0.f;
      for (int r = 0; r < nk; r += 4) {
        float vv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) vv[u] = r + u < nk ? __bfloat162float(s_v[(r + u) * P + tid]) : 0.f;
#pragma unroll
        for (int j = 0; j < RMAX; ++j) {
          if (j < R) {
            const float4 p4 = *reinterpret_cast<const float4*>(s_p + j * kTile + r);
            acc[j] += p4.x * vv[0] + p4.y * vv[1] + p4.z * vv[2] + p4.w * vv[3];
          }
        }
      }
#pragma unroll
      for (int j = 0; j < RMAX; ++j)
        if (j < R) o[j] = o[j] * f_old[j] + acc[j] * f_new[j];
    }
  }
  // ---- partial result of this split
#pragma unroll
  for (int j = 0; j < RMAX; ++j) {
    if (j < R) {
      const size_t rec = ((size_t)(m0 + j) * n_heads + h) * n_split + split;
      if (tid < D) att_o[rec * D + tid] = o[j];
      if (tid == 0) { att_ml[rec * 2] = run_m[j]; att_ml[rec * 2 + 1] = run_l[j]; }
    }
  }
  // ---- the last split of this (sequence, head) to finish merges all of them and writes the
  // attention output as hi/lo bf16 planes [row][n_heads * D] (no block waits for another)
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned tk = atomicAdd(&tickets[b * n_heads + h], 1u);
    s_last = (tk == (unsigned)n_split - 1u);
    if (s_last) tickets[b * n_heads + h] = 0u;
  }
  __syncthreads();
  if (s_last && tid < D) {
    __threadfence();
    for (int j = 0; j < R; ++j) {
      const size_t rec0 = ((size_t)(m0 + j) * n_heads + h) * n_split;
      const volatile float* ml = att_ml + rec0 * 2;
      float mx = -FLT_MAX;
      for (int s = 0; s < n_split; ++s) mx = fmaxf(mx, ml[2 * s]);
      float den = 0.f, num = 0.f;
      for (int s = 0; s < n_split; ++s) {
        const float w = __expf(ml[2 * s] - mx);
        den += w * ml[2 * s + 1];
        num += w * ((const volatile float*)att_o)[(rec0 + s) * D + tid];
      }
      const float x = num / den;
      const __nv_bfloat16 hi = __float2bfloat16_rn(x);
      const size_t at = (size_t)(m0 + j) * n_heads * D + h * D + tid;
      out_hi[at] = hi;
      out_lo[at] = __float2bfloat16_rn(x - __bfloat162float(hi));
    }
  }
}

// inv_freq[i] = base^(-2i/D) in double, once per context.
__global__ void k_inv_freq(double* inv_freq, int D, double rope_base) {
  int i = threadIdx.x;
  if (i < D / 2) inv_freq[i] = exp2(-2.0 * (double)i / (double)D * log2(rope_base));
}

size_t attn_smem_bytes(int R, int D) {
  return (size_t)(R * D + 2 * R * (D / 2) + R * kTile + 2 * kMaxRowsPerSeq) * sizeof(float) +
         (size_t)2 * kTile * (D + kPad) * sizeof(__nv_bfloat16);
}

}  // namespace

ps_status launch_rope_table(ps_ctx* c, cudaStream_t st) {
  k_inv_freq<<<1, 64, 0, st>>>(c->rope_inv_freq, c->cfg.head_dim, (double)c->cfg.rope_base);
  return cuda_check(c, cudaGetLastError(), "k_inv_freq");
}

// Chooses the number of key splits and launches the kernel.  qkv: float [M][Hq+2Hkv] before
// RoPE.  Partials: att_ml [M][n_heads][n_split][2], att_o [M][n_heads][n_split][D]; merged
// output planes out_hi / out_lo: bf16 [M][n_heads * D]; tickets: [B][n_heads], zero between calls.
ps_status launch_attn_split(ps_ctx* c, const SeqMap& sm, int B, const float* qkv, float* att_ml,
                            float* att_o, unsigned* tickets, __nv_bfloat16* out_hi,
                            __nv_bfloat16* out_lo, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const int R = g.k_masks + 1, D = g.head_dim, Hq = g.n_heads * D, Hkv = g.n_kv_heads * D;
  typedef const __nv_bfloat16* BP;
  int max_len = 0;
  for (int b = 0; b < B; ++b) max_len = std::max(max_len, sm.len[b] + R);
  // enough blocks for about three per SM, never less than one tile of keys per split
  int want = (3 * c->n_sm + B * g.n_heads - 1) / (B * g.n_heads);
  int n_split = std::max(1, std::min(std::min(want, kAttnMaxSplit), (max_len + kTile - 1) / kTile));
  dim3 grid(g.n_heads, n_split, B);
  const size_t bytes = attn_smem_bytes(R, D);
  cudaError_t e = D == 64 ? cudaFuncSetAttribute(k_attn_tile<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes)
                          : cudaFuncSetAttribute(k_attn_tile<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return cuda_check(c, e, "attention smem attribute");
  if (D == 64)
    k_attn_tile<64><<<grid, kTile, bytes, st>>>(sm, qkv, Hq + 2 * Hkv, Hq, Hkv, (BP)c->kcache, (BP)c->vcache,
                                                g.n_heads, g.n_kv_heads, g.max_ctx, c->rope_inv_freq, n_split,
                                                att_ml, att_o, tickets, out_hi, out_lo);
  else
    k_attn_tile<128><<<grid, kTile, bytes, st>>>(sm, qkv, Hq + 2 * Hkv, Hq, Hkv, (BP)c->kcache, (BP)c->vcache,
                                                 g.n_heads, g.n_kv_heads, g.max_ctx, c->rope_inv_freq, n_split,
                                                 att_ml, att_o, tickets, out_hi, out_lo);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_attn_tile");
}

}  // namespace ps
