// Split-KV attention of the fused bf16 draft step (Sec. 4.1: the k+1 rows of a sequence see the
// cached real positions and the new rows up to themselves).
//
// Work item = (head, key split, sequence); 256 threads.  A block walks its key range in tiles
// of up to 128 keys.  The K and V rows of a tile are staged in shared memory with 16-byte
// asynchronous copies (bf16, padded rows) while the block rotates q and the new k rows (RoPE,
// pair (i, i + D/2), angle pos * base^(-2i/D), the angle formed and reduced in double; cached
// keys are already rotated; new k/v rows are rounded to bf16 as a cache row would be).
// Both products run on the tensor cores with the long dimension on the 16-row side of
// mma.m16n8k16 and the few query rows on the 8-wide side:
//   S^T[key][row] = K[key][d] * Q^T[d][row]      (warp w: keys 16w .. 16w+15 of the tile)
//   O^T[d][row]   = V^T[d][key] * P^T[key][row]  (warp w: channels 16w .. 16w+15)
// q and the probabilities are fp32 values split into bf16 hi + lo planes (x = hi + lo to about
// 2^-17 relative), two MMAs per product, so the only bf16 roundings are those of the cache.
// Output: un-normalised partial (max, sum, o) per (row, head, split); the last split of a
// (sequence, head) to finish merges them into the hi/lo bf16 planes the o-projection reads.
#include <cfloat>

#include "ps_internal.cuh"

namespace ps {
namespace {

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kTileMax = 16 * kAttnWarps;   // keys per tile: one 16-key MMA tile per warp
constexpr int kPad = 8;                     // bf16 elements of padding per staged row (16 bytes)
constexpr int kPP = kTileMax + kPad;        // bf16 elements per row of the probability planes

// 16-byte asynchronous copy global -> shared (both addresses 16-byte aligned).
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)),
               "l"(src)
               : "memory");
}

// Four 8x8 bf16 matrices from shared memory; thread i gives the address of row i%8 of matrix
// i/8.  Plain: thread (g, t) receives elements [g][2t], [g][2t+1] of each; .trans: [2t][g],
// [2t+1][g].
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"((uint32_t)__cvta_generic_to_shared(row)));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const void* row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"((uint32_t)__cvta_generic_to_shared(row)));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// Shared-memory bytes of one block: K and V tiles, q planes, probability planes, rotation
// table, cross-warp exchange.
__host__ __device__ constexpr size_t attn_smem_bytes(int D, int NB, int tile) {
  return (size_t)2 * tile * (D + kPad) * 2 + (size_t)2 * 8 * NB * (D + kPad) * 2 +
         (size_t)2 * 8 * NB * kPP * 2 + (size_t)2 * 8 * NB * (D / 2) * 4 +
         (size_t)kAttnWarps * 8 * NB * 4;
}

// NB: query rows padded to 8 * NB (the 8-wide MMA side).  tile: keys per tile, a multiple of 16.
template <int D, int NB>
__global__ void __launch_bounds__(kAttnThreads, NB == 1 ? 3 : 2) k_attn_mma(
    SeqMap sm, const float* __restrict__ qkv, int ldq, int Hq, int Hkv,
    const __nv_bfloat16* __restrict__ kcache, const __nv_bfloat16* __restrict__ vcache, int n_heads,
    int n_kv_heads, int max_ctx, const double* __restrict__ inv_freq, int n_split, int tile,
    float* __restrict__ att_ml, float* __restrict__ att_o, unsigned* tickets,
    __nv_bfloat16* __restrict__ out_hi, __nv_bfloat16* __restrict__ out_lo) {
  constexpr int P = D + kPad, HALF = D / 2, RB = 8 * NB, VPR = D / 8;
  extern __shared__ __align__(16) unsigned char att_smem[];
  const int h = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int R = sm.row_off[b + 1] - sm.row_off[b], L = sm.len[b], m0 = sm.row_off[b] - sm.row_base;
  const int hk = h / (n_heads / n_kv_heads);
  __nv_bfloat16* s_k = reinterpret_cast<__nv_bfloat16*>(att_smem);     // [tile][P]
  __nv_bfloat16* s_v = s_k + tile * P;                                 // [tile][P]
  __nv_bfloat16* s_qh = s_v + tile * P;                                // [RB][P] scaled, rotated q
  __nv_bfloat16* s_ql = s_qh + RB * P;
  __nv_bfloat16* s_ph = s_ql + RB * P;                                 // [RB][kPP] probabilities
  __nv_bfloat16* s_pl = s_ph + RB * kPP;
  float* s_cs = reinterpret_cast<float*>(s_pl + RB * kPP);             // [RB][HALF] cos
  float* s_sn = s_cs + RB * HALF;                                      // [RB][HALF] sin
  float* s_red = s_sn + RB * HALF;                                     // [warps][RB]

  const int total = L + R;
  int per = (total + n_split - 1) / n_split;
  per = (per + tile - 1) / tile * tile;                  // whole tiles per split
  const int t_begin = min(total, split * per), t_end = min(total, t_begin + per);
  const __nv_bfloat16* kb = kcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;
  const __nv_bfloat16* vb = vcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;

  // cached rows [t0, t0+nk) of a tile -> shared memory, asynchronously
  auto stage = [&](int t0, int nk) {
    for (int idx = tid; idx < nk * VPR; idx += kAttnThreads) {
      const int r = idx / VPR, v = idx - r * VPR, tk = t0 + r;
      if (tk < L) {
        cp_async16(s_k + r * P + v * 8, kb + (size_t)tk * D + v * 8);
        cp_async16(s_v + r * P + v * 8, vb + (size_t)tk * D + v * 8);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  pdl_launch_dependents();
  if (t_begin < t_end) stage(t_begin, min(tile, t_end - t_begin));   // the cache is older than the launch before
  // rotation table of the R new positions (needs nothing of the kernel before this one)
  for (int idx = tid; idx < R * HALF; idx += kAttnThreads) {
    const int j = idx / HALF, i = idx - j * HALF;
    double ang = (double)(L + j) * inv_freq[i];
    ang -= 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
    float sn, cs;
    sincosf((float)ang, &sn, &cs);
    s_cs[idx] = cs;
    s_sn[idx] = sn;
  }
  pdl_wait();   // q, k and v of the new rows come from the kernel before this one

  // q: rotated, scaled, split into hi/lo planes
  __syncthreads();
  const float scale = rsqrtf((float)D);
  for (int idx = tid; idx < RB * HALF; idx += kAttnThreads) {
    const int j = idx / HALF, i = idx - j * HALF;
    float r0 = 0.f, r1 = 0.f;
    if (j < R) {
      const float* row = qkv + (size_t)(m0 + j) * ldq + h * D;
      const float q0 = row[i], q1 = row[i + HALF], c = s_cs[idx], s = s_sn[idx];
      r0 = (q0 * c - q1 * s) * scale;
      r1 = (q1 * c + q0 * s) * scale;
    }
    split_bf16(r0, s_qh[j * P + i], s_ql[j * P + i]);
    split_bf16(r1, s_qh[j * P + i + HALF], s_ql[j * P + i + HALF]);
  }

  // per-thread state.  A thread's score / output fragments cover rows 8*nb + 2t and + 1.
  float run_m[NB][2], run_l[NB][2];   // running max (identical in all threads), partial sum
  float o[NB][4];                     // O^T fragment: channels 16*warp + g (+8), rows 2t (+1)
  uint32_t qf[NB][D / 16][2][2];      // q fragments [k step][hi/lo][b0, b1]
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    run_m[nb][0] = run_m[nb][1] = -FLT_MAX;
    run_l[nb][0] = run_l[nb][1] = 0.f;
    o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
  }

  bool first = true;
  for (int t0 = t_begin; t0 < t_end; t0 += tile) {
    const int nk = min(tile, t_end - t0), nk16 = (nk + 15) >> 4;
    if (!first) {
      __syncthreads();                           // previous tile fully consumed
      stage(t0, nk);
    }
    if (t0 + nk > L) {                           // the tile holds new rows: rotate k, round k and v
      const int first_new = max(L, t0);
      for (int idx = tid; idx < (t0 + nk - first_new) * HALF; idx += kAttnThreads) {
        const int jj = idx / HALF, i = idx - jj * HALF, j = first_new - L + jj, r = first_new - t0 + jj;
        const float* row = qkv + (size_t)(m0 + j) * ldq;
        const float k0 = row[Hq + hk * D + i], k1 = row[Hq + hk * D + i + HALF];
        const float c = s_cs[j * HALF + i], s = s_sn[j * HALF + i];
        s_k[r * P + i] = __float2bfloat16_rn(k0 * c - k1 * s);
        s_k[r * P + i + HALF] = __float2bfloat16_rn(k1 * c + k0 * s);
        s_v[r * P + i] = __float2bfloat16_rn(row[Hq + Hkv + hk * D + i]);
        s_v[r * P + i + HALF] = __float2bfloat16_rn(row[Hq + Hkv + hk * D + i + HALF]);
      }
    }
    // rows past the end of a ragged last 16-key group: V must be finite (0 * NaN), K is masked
    for (int idx = tid; idx < (nk16 * 16 - nk) * VPR; idx += kAttnThreads) {
      const int r = nk + idx / VPR, v = idx % VPR;
      *reinterpret_cast<uint4*>(s_v + r * P + v * 8) = make_uint4(0u, 0u, 0u, 0u);
      *reinterpret_cast<uint4*>(s_k + r * P + v * 8) = make_uint4(0u, 0u, 0u, 0u);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    if (first) {
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const int at = (8 * nb + g) * P + 16 * ks + 2 * t;
          qf[nb][ks][0][0] = *reinterpret_cast<const uint32_t*>(s_qh + at);
          qf[nb][ks][0][1] = *reinterpret_cast<const uint32_t*>(s_qh + at + 8);
          qf[nb][ks][1][0] = *reinterpret_cast<const uint32_t*>(s_ql + at);
          qf[nb][ks][1][1] = *reinterpret_cast<const uint32_t*>(s_ql + at + 8);
        }
      first = false;
    }
    // ---- scores of keys 16*warp .. +15 (fragment: keys g, g+8; rows 2t, 2t+1 of each nb)
    float sc[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
    const bool qk_warp = warp < nk16;
    if (qk_warp) {
      const __nv_bfloat16* arow = s_k + (16 * warp + (lane & 7) + ((lane >> 3) & 1) * 8) * P + (lane >> 4) * 8;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t a[4];
        ldsm_x4(a, arow + 16 * ks);
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          mma16816(sc[nb], a, qf[nb][ks][0][0], qf[nb][ks][0][1]);
          mma16816(sc[nb], a, qf[nb][ks][1][0], qf[nb][ks][1][1]);
        }
      }
    }
    // mask, tile max per row
    float mx[NB][2];
    bool ok[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = t0 + 16 * warp + g + (e >> 1) * 8, row = 8 * nb + 2 * t + (e & 1);
        ok[nb][e] = qk_warp && key < t0 + nk && row < R && (key < L || key - L <= row);
      }
      mx[nb][0] = fmaxf(ok[nb][0] ? sc[nb][0] : -FLT_MAX, ok[nb][2] ? sc[nb][2] : -FLT_MAX);
      mx[nb][1] = fmaxf(ok[nb][1] ? sc[nb][1] : -FLT_MAX, ok[nb][3] ? sc[nb][3] : -FLT_MAX);
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        mx[nb][0] = fmaxf(mx[nb][0], __shfl_xor_sync(0xffffffffu, mx[nb][0], off));
        mx[nb][1] = fmaxf(mx[nb][1], __shfl_xor_sync(0xffffffffu, mx[nb][1], off));
      }
      if (g == 0) {
        s_red[warp * RB + 8 * nb + 2 * t] = mx[nb][0];
        s_red[warp * RB + 8 * nb + 2 * t + 1] = mx[nb][1];
      }
    }
    __syncthreads();
    float f_old[NB][2];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float m = run_m[nb][e];
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) m = fmaxf(m, s_red[w * RB + 8 * nb + 2 * t + e]);
        f_old[nb][e] = __expf(run_m[nb][e] - m);
        run_m[nb][e] = m;
      }
      float pv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) pv[e] = ok[nb][e] ? __expf(sc[nb][e] - run_m[nb][e & 1]) : 0.f;
      run_l[nb][0] = run_l[nb][0] * f_old[nb][0] + pv[0] + pv[2];
      run_l[nb][1] = run_l[nb][1] * f_old[nb][1] + pv[1] + pv[3];
      if (qk_warp) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int at = (8 * nb + 2 * t + (e & 1)) * kPP + 16 * warp + g + (e >> 1) * 8;
          split_bf16(pv[e], s_ph[at], s_pl[at]);
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) o[nb][e] *= f_old[nb][e & 1];
    }
    __syncthreads();
    // ---- O^T += V^T P^T for channels 16*warp .. +15
    if (warp < D / 16) {
      const __nv_bfloat16* vrow = s_v + ((lane & 7) + (lane >> 4) * 8) * P + 16 * warp + ((lane >> 3) & 1) * 8;
      for (int kk = 0; kk < nk16; ++kk) {
        uint32_t a[4];
        ldsm_x4_trans(a, vrow + 16 * kk * P);
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          const int at = (8 * nb + g) * kPP + 16 * kk + 2 * t;
          mma16816(o[nb], a, *reinterpret_cast<const uint32_t*>(s_ph + at),
                   *reinterpret_cast<const uint32_t*>(s_ph + at + 8));
          mma16816(o[nb], a, *reinterpret_cast<const uint32_t*>(s_pl + at),
                   *reinterpret_cast<const uint32_t*>(s_pl + at + 8));
        }
      }
    }
  }
  // ---- partial result of this split: row sums over the key lanes and warps, then the store
  __syncthreads();
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      float l = run_l[nb][e];
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
      if (g == 0) s_red[warp * RB + 8 * nb + 2 * t + e] = l;
    }
  }
  __syncthreads();
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int j = 8 * nb + 2 * t + e;
      if (j < R) {
        const size_t rec = ((size_t)(m0 + j) * n_heads + h) * n_split + split;
        if (warp < D / 16) {
          att_o[rec * D + 16 * warp + g] = o[nb][e];
          att_o[rec * D + 16 * warp + g + 8] = o[nb][2 + e];
        }
        if (warp == 0 && g == 0) {
          float l = 0.f;
#pragma unroll
          for (int w = 0; w < kAttnWarps; ++w) l += s_red[w * RB + j];
          att_ml[rec * 2] = run_m[nb][e];
          att_ml[rec * 2 + 1] = l;
        }
      }
    }
  }
  // ---- the last split of this (sequence, head) to finish merges all of them and writes the
  // attention output as hi/lo bf16 planes [row][n_heads * D] (no block waits for another)
  __shared__ int s_last;
  __syncthreads();
  if (tid == 0) {
    // one thread publishes the block's partial (the barrier ordered the other threads' stores
    // before this fence) and, if it came last, acquires the other blocks'
    __threadfence();
    const unsigned tk = atomicAdd(&tickets[b * n_heads + h], 1u);
    s_last = (tk == (unsigned)n_split - 1u);
    if (s_last) {
      tickets[b * n_heads + h] = 0u;
      __threadfence();
    }
  }
  __syncthreads();
  if (s_last) {
    // This code runs once per (sequence, head), after everything else: what it costs is round
    // trips to L2 and the fetch of its own instructions, so it is a few small rolled loops.
    // All splits' partial outputs of a row are one contiguous block: asynchronous 16-byte
    // copies bring the rows into the shared memory of the (finished) K / V tiles, as many rows
    // per pass as fit, in one round trip; the (max, sum) pairs go to the q planes' place.
    float* s_o = reinterpret_cast<float*>(att_smem);     // [rows of a pass][n_split][D]
    float2* s_ml = reinterpret_cast<float2*>(s_qh);      // [R][n_split]
    const int row_f = n_split * D;                        // floats per row
    const int rows_pass = max(1, (2 * tile * P * 2) / (row_f * 4));
    const float2* ml2 = reinterpret_cast<const float2*>(att_ml);
    for (int j0 = 0; j0 < R; j0 += rows_pass) {
      const int nr = min(rows_pass, R - j0), vec_row = row_f / 4;
      for (int idx = tid; idx < nr * vec_row; idx += kAttnThreads) {
        const int jr = idx / vec_row, off = (idx - jr * vec_row) * 4;
        cp_async16(s_o + jr * row_f + off, att_o + ((size_t)(m0 + j0 + jr) * n_heads + h) * row_f + off);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      if (j0 == 0) {   // (while the copies are on their way)
        for (int idx = tid; idx < R * n_split; idx += kAttnThreads) {
          const int j = idx / n_split, sp = idx - j * n_split;
          s_ml[idx] = __ldcg(ml2 + ((size_t)(m0 + j) * n_heads + h) * n_split + sp);
        }
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();
      for (int idx = tid; idx < nr * D; idx += kAttnThreads) {
        const int jr = idx / D, d = idx - jr * D, j = j0 + jr;
        const float2* ml = s_ml + j * n_split;
        float mxs = -FLT_MAX;
        for (int sp = 0; sp < n_split; ++sp) mxs = fmaxf(mxs, ml[sp].x);
        float den = 0.f, num = 0.f;
        for (int sp = 0; sp < n_split; ++sp) {
          const float w = __expf(ml[sp].x - mxs);
          den += w * ml[sp].y;
          num += w * s_o[jr * row_f + sp * D + d];
        }
        const float x = num / den;
        const size_t at = (size_t)(m0 + j) * n_heads * D + h * D + d;
        split_bf16(x, out_hi[at], out_lo[at]);
      }
      __syncthreads();
    }
  }
}

// inv_freq[i] = base^(-2i/D) in double, once per context.
__global__ void k_inv_freq(double* inv_freq, int D, double rope_base) {
  int i = threadIdx.x;
  if (i < D / 2) inv_freq[i] = exp2(-2.0 * (double)i / (double)D * log2(rope_base));
}

}  // namespace

ps_status launch_rope_table(ps_ctx* c, cudaStream_t st) {
  k_inv_freq<<<1, 64, 0, st>>>(c->rope_inv_freq, c->cfg.head_dim, (double)c->cfg.rope_base);
  return cuda_check(c, cudaGetLastError(), "k_inv_freq");
}

// Chooses tile size and number of key splits and launches the kernel.  qkv: float
// [M][Hq+2Hkv] before RoPE.  Partials: att_ml [M][n_heads][n_split][2], att_o
// [M][n_heads][n_split][D]; merged output planes out_hi / out_lo: bf16 [M][n_heads * D];
// tickets: [B][n_heads], zero between calls.
template <int D, int NB>
static ps_status launch_attn_t(ps_ctx* c, const SeqMap& sm, int B, int max_len, const float* qkv,
                               float* att_ml, float* att_o, unsigned* tickets, __nv_bfloat16* out_hi,
                               __nv_bfloat16* out_lo, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const int Hq = g.n_heads * D, Hkv = g.n_kv_heads * D;
  // the largest tile whose grid, one tile per block, is resident at once; else full tiles and
  // several of them per block
  auto kern = k_attn_mma<D, NB>;
  // resident blocks per SM by tile size, asked of this context's device once (0 = not yet)
  int* blocks_per_sm = c->attn_blocks_per_sm[(D == 128 ? 0 : 2) + (NB == 1 ? 0 : 1)];
  static_assert(kTileMax / 16 + 1 <= 16, "cache row covers every tile size");
  // the partial buffers hold 16 rows x kAttnMaxSplit splits: more rows, fewer splits
  const int M_rows = B * (g.k_masks + 1);
  const int max_split = std::max(1, std::min(kAttnMaxSplit, 16 * kAttnMaxSplit / std::max(M_rows, 1)));
  int tile = kTileMax, n_split = 0;
  for (int cand = kTileMax; cand >= 32; cand -= 16) {
    const int tiles = (max_len + cand - 1) / cand;
    if (tiles > max_split) break;
    int& bps = blocks_per_sm[cand / 16];
    if (bps == 0) {
      const size_t bytes = attn_smem_bytes(D, NB, cand);
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
      if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, kern, kAttnThreads, bytes);
      if (e != cudaSuccess) return cuda_check(c, e, "attention occupancy");
      if (bps <= 0) bps = -1;
    }
    if (bps > 0 && (long)tiles * B * g.n_heads <= (long)bps * c->n_sm) { tile = cand; n_split = tiles; break; }
  }
  if (n_split == 0) {
    const int want = (3 * c->n_sm + B * g.n_heads - 1) / (B * g.n_heads);
    n_split = std::max(1, std::min(std::min(want, max_split), (max_len + tile - 1) / tile));
  }
  const size_t bytes = attn_smem_bytes(D, NB, tile);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return cuda_check(c, e, "attention smem attribute");
  typedef const __nv_bfloat16* BP;
  e = launch_after(kern, dim3(g.n_heads, n_split, B), dim3(kAttnThreads), bytes, st, !c->prof, sm, qkv,
                   Hq + 2 * Hkv, Hq, Hkv, (BP)c->kcache, (BP)c->vcache, g.n_heads, g.n_kv_heads, g.max_ctx,
                   (const double*)c->rope_inv_freq, n_split, tile, att_ml, att_o, tickets, out_hi, out_lo);
  c->launches++;
  return cuda_check(c, e, "k_attn_mma");
}

ps_status launch_attn_split(ps_ctx* c, const SeqMap& sm, int B, const float* qkv, float* att_ml,
                            float* att_o, unsigned* tickets, __nv_bfloat16* out_hi,
                            __nv_bfloat16* out_lo, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const int R = g.k_masks + 1;
  int max_len = 0;
  for (int b = 0; b < B; ++b) max_len = std::max(max_len, sm.len[b] + R);
#define PS_ATTN(D_, NB_) \
  return launch_attn_t<D_, NB_>(c, sm, B, max_len, qkv, att_ml, att_o, tickets, out_hi, out_lo, st)
  if (g.head_dim == 128) { if (R <= 8) PS_ATTN(128, 1); else PS_ATTN(128, 2); }
  if (g.head_dim == 64) { if (R <= 8) PS_ATTN(64, 1); else PS_ATTN(64, 2); }
#undef PS_ATTN
  return fail(c, PS_ERR_UNSUPPORTED, "fused attention needs head_dim 64 or 128");
}

}  // namespace ps
