// Weight-streaming small-M GEMM for the bf16 drafter:  Y[m][n] = sum_k A[m][k] * W[n][k],
// M = B*(k+1) <= 16 rows, W row-major bf16 (read exactly once from HBM), fp32 arithmetic.
//
// One CTA per SM owns a contiguous range of output features n (balanced to one row).  A
// producer warp streams that range through a ring of shared-memory slots with bulk async
// copies (cp.async.bulk + mbarrier transaction counts), 8 weight rows x KC columns per slot,
// one 4 KB copy per row (small bulk copies pay a fixed cost each and starve the memory system).
// The consumer warps split each slot along k.  At these row counts the path is bound by HBM,
// not by arithmetic: with M = 5 each weight needs 5 multiply-adds, about 45% of the fp32 rate
// at full memory bandwidth, so the contraction runs on the fp32 pipes with packed
// fma.rn.f32x2 (two k positions per instruction) on activations kept in shared memory as
// fp32.  (Legacy mma.sync tiles were measured to cap this kernel near 4 TB/s on this part and
// would need split bf16 activations to keep fp32 accuracy.)
// When M*K is too large for shared memory the k range is processed in passes; partial sums of
// the CTA's features stay in shared memory between passes.
// Every wait is bounded: on expiry the kernel raises the device status word and returns.
#pragma once
#include <cuda_bf16.h>

#include <cstdint>

#include "ps_internal.cuh"

namespace ps {
namespace ws {

#ifndef PS_CONSUMER_WARPS
#define PS_CONSUMER_WARPS 8
#endif
constexpr int kConsumerWarps = PS_CONSUMER_WARPS;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + one producer warp
constexpr int KC = 2048;                         // k-columns per slot
constexpr int kSlotRows = 8;
constexpr int kWPitch = KC * 2 + 32;             // bytes; = 32 mod 128 -> conflict-free 16-byte reads
constexpr int kSlotBytes = kSlotRows * kWPitch;
constexpr int kMaxSlots = 12;
constexpr int kMinSlots = 3;
constexpr int kColsPerWarp = KC / kConsumerWarps;
constexpr int kStepsPerWarp = kColsPerWarp / 64;   // a warp covers 8 k-vectors of 8 columns per step
constexpr long long kWaitCycles = 2000000000LL;    // ~1 s: bound of every mbarrier wait

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the bound expired or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_test(bar, parity)) return true;
  long long t0 = clock64();
  int spins = 0;
  while (!mbar_test(bar, parity)) {
    if ((++spins & 255) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        return false;
      }
    }
  }
  return true;
}
// Bulk async copy global -> shared of `bytes` (multiple of 16, both addresses 16-byte aligned),
// completion counted on `bar`.  No multicast.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}
// ---- where the weight rows come from ---------------------------------------------------------
// Logical output features are either the concatenation of up to three matrices (q|k|v) or, with
// zip = 1, feature n is the PAIR (W[0] row n, W[1] row n) (gate, up).
struct RowSrc {
  const __nv_bfloat16* W[3];
  int rows[3];
  int n_mats;
  int zip;
};

// Sub-tiles hold 8 weight rows.  Plain / concatenated sources: sub-tile st covers features
// n_begin + 8 st + i.  Zipped sources: sub-tiles alternate between the two matrices, st = 2 grp
// + which covers rows n_begin + 8 grp + i of W[which].
__device__ __forceinline__ int n_subtiles(const RowSrc& rs, int n_begin, int n_end) {
  int groups = (n_end - n_begin + 7) >> 3;
  return rs.zip ? 2 * groups : groups;
}
// Feature index of slot row i of sub-tile st (may be >= n_end: then the row does not exist).
__device__ __forceinline__ int subtile_feature(const RowSrc& rs, int n_begin, int st, int i) {
  return n_begin + 8 * (rs.zip ? (st >> 1) : st) + i;
}
// Global address of that row, nullptr if it lies beyond n_end.
__device__ __forceinline__ const __nv_bfloat16* slot_row_ptr(const RowSrc& rs, int n_begin, int st,
                                                             int i, int n_end, int K) {
  int n = subtile_feature(rs, n_begin, st, i);
  if (n >= n_end) return nullptr;
  if (rs.zip) return rs.W[st & 1] + (size_t)n * K;
  int m = 0;
  while (m + 1 < rs.n_mats && n >= rs.rows[m]) {
    n -= rs.rows[m];
    ++m;
  }
  return rs.W[m] + (size_t)n * K;
}

struct Smem {
  uint64_t full[kMaxSlots];
  uint64_t empty[kMaxSlots];
  int abort_flag;
  int is_last;
};

// Activations of one pass live in two fp32 planes: element (m, k) sits in plane (k >> 2) & 1 at
// float index m * plane_pitch(cols) + (k >> 3) * 4 + (k & 3).  A lane that needs the eight
// activations k..k+7 of a row reads one float4 from each plane; the eight lanes of a warp that
// work on neighbouring k-vectors read 128 contiguous bytes.
__host__ __device__ inline int plane_pitch(int cols) { return cols / 2 + 4; }   // floats per row

// Features [n_begin, n_end) of CTA `cta` out of `n_cta`, balanced to one feature.
__host__ __device__ inline void cta_range(int N, int cta, int n_cta, int& n_begin, int& n_end) {
  n_begin = (int)(((long long)N * cta) / n_cta);
  n_end = (int)(((long long)N * (cta + 1)) / n_cta);
}

// Producer: streams every (pass, sub-tile, k-chunk) of the CTA's feature range through the ring.
// Runs in one warp; lane i < 8 issues the copy of slot row i.  pass_cols is a multiple of 8.
__device__ __forceinline__ void produce(const RowSrc& rs, int K, int pass_cols, int n_begin,
                                        int n_end, unsigned char* ring, int n_slots, Smem& sm,
                                        int lane) {
  const int n_st = n_subtiles(rs, n_begin, n_end);
  int it = 0;
  for (int k0 = 0; k0 < K; k0 += pass_cols) {
    const int k1 = min(K, k0 + pass_cols);
    for (int st = 0; st < n_st; ++st) {
      const __nv_bfloat16* src =
          lane < kSlotRows ? slot_row_ptr(rs, n_begin, st, lane, n_end, K) : nullptr;
      unsigned valid = __ballot_sync(0xffffffffu, src != nullptr);
      int n_valid = __popc(valid);
      for (int kc = k0; kc < k1; kc += KC, ++it) {
        int slot = it % n_slots;
        uint32_t parity = ((it / n_slots) & 1) ^ 1;   // a fresh barrier passes a wait on parity 1
        int cols = min(KC, k1 - kc);
        int ok = 1;
        if (lane == 0) {
          ok = mbar_wait(&sm.empty[slot], parity, &sm.abort_flag) ? 1 : 0;
          if (ok) mbar_arrive_expect_tx(&sm.full[slot], (uint32_t)(n_valid * cols * 2));
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) return;
        if (src)
          bulk_g2s(ring + (size_t)slot * kSlotBytes + lane * kWPitch, src + kc, (uint32_t)(cols * 2),
                   &sm.full[slot]);
      }
    }
  }
}

// Two bf16 values packed in a 32-bit word, widened to a float pair (exact).
__device__ __forceinline__ float2 widen2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

// Consumer: accumulates one sub-tile (8 weight rows) over the k range of the current pass
// (`cols_pass` columns).  Lane = 4 * kq + r works on weight rows r and r + 4 and, in step s of
// a chunk, on the k-vector (8 columns) number warp * 32 + s * 8 + kq.  On return lanes 0..3
// (kq == 0) hold in out[j][m] the warp's partial sum for slot row r + 4 j and activation row m.
// M (the number of activation rows) is a template parameter so that every loop unrolls and the
// loads of a step are all issued before its multiply-adds.
// `it` is the running chunk counter shared with the producer's schedule.  Returns false if a
// wait expired.
template <int M>
__device__ __forceinline__ bool consume_tile(const float* plane_a, const float* plane_b, int ppitch,
                                             int cols_pass, const unsigned char* ring, int n_slots,
                                             Smem& sm, int& it, int warp, int lane,
                                             float (&out)[2][M]) {
  constexpr int MT = M;
  const int r = lane & 3, kq = lane >> 2;
  float2 acc[2][M];
#pragma unroll
  for (int j = 0; j < 2; ++j)
#pragma unroll
    for (int m = 0; m < M; ++m) acc[j][m] = make_float2(0.f, 0.f);
  for (int c0 = 0; c0 < cols_pass; c0 += KC, ++it) {
    int slot = it % n_slots;
    uint32_t parity = (it / n_slots) & 1;
    if (!mbar_wait(&sm.full[slot], parity, &sm.abort_flag)) return false;
    const int cols = min(KC, cols_pass - c0);
    const unsigned char* w0 = ring + (size_t)slot * kSlotBytes + r * kWPitch;
    const unsigned char* w1 = w0 + 4 * kWPitch;
#pragma unroll
    for (int s = 0; s < kStepsPerWarp; ++s) {
      const int col = warp * kColsPerWarp + s * 64 + kq * 8;     // column inside the chunk
      if (col < cols) {
        const uint4 q0 = *reinterpret_cast<const uint4*>(w0 + col * 2);
        const uint4 q1 = *reinterpret_cast<const uint4*>(w1 + col * 2);
        const int v4 = ((c0 + col) >> 3) * 4;
        float4 xa[M], xb[M];
#pragma unroll
        for (int m = 0; m < M; ++m) {
          xa[m] = *reinterpret_cast<const float4*>(plane_a + (size_t)m * ppitch + v4);
          xb[m] = *reinterpret_cast<const float4*>(plane_b + (size_t)m * ppitch + v4);
        }
        const float2 wa[4] = {widen2(q0.x), widen2(q0.y), widen2(q0.z), widen2(q0.w)};
        const float2 wb[4] = {widen2(q1.x), widen2(q1.y), widen2(q1.z), widen2(q1.w)};
        // k pair outermost: 2 M independent accumulators between two uses of the same one
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
          for (int m = 0; m < M; ++m) {
            const float2 x = i == 0 ? make_float2(xa[m].x, xa[m].y)
                           : i == 1 ? make_float2(xa[m].z, xa[m].w)
                           : i == 2 ? make_float2(xb[m].x, xb[m].y)
                                    : make_float2(xb[m].z, xb[m].w);
            acc[0][m] = __ffma2_rn(wa[i], x, acc[0][m]);
            acc[1][m] = __ffma2_rn(wb[i], x, acc[1][m]);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[slot]);
  }
  // even + odd k positions, then the eight k-vector lanes of each row (lane bits 2..4)
#pragma unroll
  for (int j = 0; j < 2; ++j)
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      float v = acc[j][m].x + acc[j][m].y;
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      v += __shfl_xor_sync(0xffffffffu, v, 8);
      v += __shfl_xor_sync(0xffffffffu, v, 16);
      out[j][m] = v;
    }
  return true;
}

}  // namespace ws
}  // namespace ps
