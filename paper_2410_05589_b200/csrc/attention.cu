// Split-KV attention of the fused bf16 draft step (Sec. 4.1: the k+1 rows of a sequence see the
// cached real positions and the new rows up to themselves).
#include <cfloat>

#include "ps_internal.cuh"

namespace ps {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- split-KV attention under the parallel-draft mask -----------------------------------------
// Work item = (sequence b, head h, split s of the key range).  Each of the 4 warps of a block
// takes keys round-robin; lanes own D/32 channels.  q and the new k rows are rotated in
// registers (RoPE, pair (i, i+D/2), angle pos*base^(-2i/D)); cached keys are already rotated.
// New k/v rows are rounded to bf16 as a cache row would be.  Output: un-normalised partial
// (max, sum, o) per (row, head, split), merged by the o-projection's prologue.
template <int D>
__global__ void __launch_bounds__(128) k_attn_split(SeqMap sm, const float* qkv, int ldq, int Hq,
                                                    int Hkv, const __nv_bfloat16* kcache,
                                                    const __nv_bfloat16* vcache, int n_heads,
                                                    int n_kv_heads, int max_ctx, float rope_base,
                                                    int n_split, float* att_ml, float* att_o) {
  constexpr int C = D / 32, RMAX = kMaxRowsPerSeq;
  extern __shared__ float att_smem[];
  const int Rs = sm.row_off[1] - sm.row_off[0];          // rows per sequence (same for all)
  float (*s_q)[D] = reinterpret_cast<float (*)[D]>(att_smem);
  float (*s_kn)[D] = s_q + Rs;
  float (*s_vn)[D] = s_kn + Rs;
  float* s_o = reinterpret_cast<float*>(s_vn + Rs);      // [4][Rs][D]
  float* s_m = s_o + 4 * Rs * D;                         // [4][Rs]
  float* s_l = s_m + 4 * Rs;                             // [4][Rs]
  const int h = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int R = sm.row_off[b + 1] - sm.row_off[b], L = sm.len[b], m0 = sm.row_off[b];
  const int hk = h / (n_heads / n_kv_heads);
  const float scale = rsqrtf((float)D);
  // rotate q rows and new k rows (position L + j); round new k, v to bf16
  for (int idx = threadIdx.x; idx < R * (D / 2); idx += blockDim.x) {
    int j = idx / (D / 2), i = idx - j * (D / 2);
    double inv = exp2(-2.0 * (double)i / (double)D * log2((double)rope_base));
    double sn, cs;
    sincos((double)(L + j) * inv, &sn, &cs);
    float c = (float)cs, s = (float)sn;
    const float* row = qkv + (size_t)(m0 + j) * ldq;
    float q0 = row[h * D + i], q1 = row[h * D + i + D / 2];
    s_q[j][i] = (q0 * c - q1 * s) * scale;
    s_q[j][i + D / 2] = (q1 * c + q0 * s) * scale;
    float k0 = row[Hq + hk * D + i], k1 = row[Hq + hk * D + i + D / 2];
    s_kn[j][i] = __bfloat162float(__float2bfloat16_rn(k0 * c - k1 * s));
    s_kn[j][i + D / 2] = __bfloat162float(__float2bfloat16_rn(k1 * c + k0 * s));
    s_vn[j][i] = __bfloat162float(__float2bfloat16_rn(row[Hq + Hkv + hk * D + i]));
    s_vn[j][i + D / 2] = __bfloat162float(__float2bfloat16_rn(row[Hq + Hkv + hk * D + i + D / 2]));
  }
  __syncthreads();
  float qv[RMAX][C], mx[RMAX], l[RMAX], o[RMAX][C];
#pragma unroll
  for (int j = 0; j < RMAX; ++j) {
    mx[j] = -FLT_MAX; l[j] = 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) { qv[j][c] = j < R ? s_q[j][lane + 32 * c] : 0.f; o[j][c] = 0.f; }
  }
  const int total = L + R;
  const int per = (total + n_split - 1) / n_split;
  const int t_begin = split * per, t_end = min(total, t_begin + per);
  const __nv_bfloat16* kb = kcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;
  const __nv_bfloat16* vb = vcache + ((size_t)sm.slot[b] * n_kv_heads + hk) * max_ctx * D;
  for (int t = t_begin + warp; t < t_end; t += 4) {
    float kx[C], vx[C];
    if (t < L) {
#pragma unroll
      for (int c = 0; c < C; ++c) {
        kx[c] = __bfloat162float(kb[(size_t)t * D + lane + 32 * c]);
        vx[c] = __bfloat162float(vb[(size_t)t * D + lane + 32 * c]);
      }
    } else {
#pragma unroll
      for (int c = 0; c < C; ++c) { kx[c] = s_kn[t - L][lane + 32 * c]; vx[c] = s_vn[t - L][lane + 32 * c]; }
    }
    const int jmin = t < L ? 0 : t - L;
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
    if (j < R) {
      if (lane == 0) { s_m[warp * Rs + j] = mx[j]; s_l[warp * Rs + j] = l[j]; }
#pragma unroll
      for (int c = 0; c < C; ++c) s_o[((size_t)warp * Rs + j) * D + lane + 32 * c] = o[j][c];
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < R * D; idx += blockDim.x) {
    int j = idx / D, i = idx - j * D;
    float M = fmaxf(fmaxf(s_m[j], s_m[Rs + j]), fmaxf(s_m[2 * Rs + j], s_m[3 * Rs + j]));
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      float f = __expf(s_m[w * Rs + j] - M);
      num += f * s_o[((size_t)w * Rs + j) * D + i];
      den += f * s_l[w * Rs + j];
    }
    size_t rec = ((size_t)(m0 + j) * n_heads + h) * n_split + split;
    att_o[rec * D + i] = num;
    if (i == 0) { att_ml[rec * 2] = M; att_ml[rec * 2 + 1] = den; }
  }
}


}  // namespace

// Chooses the number of key splits and launches the kernel.  qkv: float [M][Hq+2Hkv] before
// RoPE.  Partials: att_ml [M][n_heads][n_split][2], att_o [M][n_heads][n_split][D].
ps_status launch_attn_split(ps_ctx* c, const SeqMap& sm, int B, const float* qkv, float* att_ml,
                            float* att_o, int* n_split_out, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const int R = g.k_masks + 1, D = g.head_dim, Hq = g.n_heads * D, Hkv = g.n_kv_heads * D;
  typedef const __nv_bfloat16* BP;
  int max_len = 0;
  for (int b = 0; b < B; ++b) max_len = std::max(max_len, sm.len[b] + R);
  // about two waves of blocks over the GPU, at least 64 keys per split
  int want = (2 * c->n_sm + B * g.n_heads - 1) / (B * g.n_heads);
  int n_split = std::max(1, std::min(std::min(want, kAttnMaxSplit), (max_len + 63) / 64));
  *n_split_out = n_split;
  dim3 grid(g.n_heads, n_split, B);
  size_t bytes = (size_t)(3 * R * D + 4 * R * (D + 2)) * sizeof(float);
  if (bytes > 48 * 1024) {
    cudaError_t e = D == 64 ? cudaFuncSetAttribute(k_attn_split<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes)
                            : cudaFuncSetAttribute(k_attn_split<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return cuda_check(c, e, "attention smem attribute");
  }
  if (D == 64)
    k_attn_split<64><<<grid, 128, bytes, st>>>(sm, qkv, Hq + 2 * Hkv, Hq, Hkv, (BP)c->kcache, (BP)c->vcache,
                                               g.n_heads, g.n_kv_heads, g.max_ctx, g.rope_base, n_split,
                                               att_ml, att_o);
  else
    k_attn_split<128><<<grid, 128, bytes, st>>>(sm, qkv, Hq + 2 * Hkv, Hq, Hkv, (BP)c->kcache, (BP)c->vcache,
                                                g.n_heads, g.n_kv_heads, g.max_ctx, g.rope_base, n_split,
                                                att_ml, att_o);
  c->launches++;
  return cuda_check(c, cudaGetLastError(), "k_attn_split");
}

}  // namespace ps
