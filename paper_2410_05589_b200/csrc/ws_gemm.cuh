// Weight-streaming small-M GEMM for the bf16 drafter:  Y[m][n] = sum_k A[m][k] * W[n][k],
// M = B*(k+1) <= 16 rows, W row-major bf16 (read exactly once from HBM), fp32 accumulation.
//
// One CTA per SM owns a contiguous range of output features n (balanced to one row).  A
// producer warp streams that range through a ring of shared-memory slots with bulk async
// copies (cp.async.bulk + mbarrier transaction counts), 8 weight rows x KC columns per slot,
// one 4 KB copy per row (measured: 1 KB copies cap the ring near 3 TB/s, 4 KB copies reach the
// copy bandwidth of the part).  Slots travel in pairs: 16 weight rows are the 16-row operand of
// mma.sync.m16n8k16 and the (at most 8, else 16) activation rows the 8-wide one, so a warp
// spends 8 instructions (4 shared loads, 4 MMAs) per 512 weights.  Measured alternatives on
// this part: activations on the 16-row side (half the weights per MMA) saturate the legacy
// tensor pipe near 4 TB/s; an fp32 FMA inner loop (fma.rn.f32x2) is issue bound near 3.4 TB/s.
//
// Activations stay fp32-accurate although the tensor cores take bf16: each activation x is
// held in shared memory as two bf16 planes, hi = bf16(x) and lo = bf16(x - hi), and every
// weight fragment is multiplied with both (x*w = hi*w + lo*w up to 2^-17).  When M*K is too
// large for shared memory the k range is processed in passes; partial sums of the CTA's
// features stay in shared memory between passes.
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
constexpr int kThreads = kConsumerThreads + 64;  // + the weight producer warp and the plane loader warp
constexpr int KC = 2048;                         // k-columns per slot
constexpr int kSlotRows = 8;
constexpr int kWPitch = KC * 2 + 64;             // bytes; = 64 mod 128 -> conflict-free 16-byte reads
constexpr int kSlotBytes = kSlotRows * kWPitch;
constexpr int kMaxSlots = 12;
constexpr int kMinSlots = 5;                     // a pair being consumed + three slots in flight
constexpr int kColsPerWarp = KC / kConsumerWarps;
constexpr int kStepsPerWarp = kColsPerWarp / 32;   // a warp covers 32 columns per step
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
// One look at the barrier without waiting.
__device__ __forceinline__ bool mbar_peek(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the bound (`limit` cycles) expired or another thread already
// gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit = kWaitCycles) {
  if (mbar_test(bar, parity)) return true;
  long long t0 = clock64();
  int spins = 0;
  while (!mbar_test(bar, parity)) {
    if ((++spins & 255) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) {
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
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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

// A sub-tile holds 16 weight rows in two slots of 8 ("halves").  Plain / concatenated sources:
// half h of sub-tile st covers features n_begin + 16 st + 8 h + i.  Zipped sources: half h
// covers rows n_begin + 8 st + i of W[h] (gate in half 0, up in half 1).
__device__ __forceinline__ int n_subtiles(const RowSrc& rs, int n_begin, int n_end) {
  return rs.zip ? (n_end - n_begin + 7) >> 3 : (n_end - n_begin + 15) >> 4;
}
// Feature index of row i (0..7) of half h of sub-tile st (may be >= n_end: no such row).
__device__ __forceinline__ int subtile_feature(const RowSrc& rs, int n_begin, int st, int h, int i) {
  return rs.zip ? n_begin + 8 * st + i : n_begin + 16 * st + 8 * h + i;
}
// Global address of that row, nullptr if it lies beyond n_end.
__device__ __forceinline__ const __nv_bfloat16* slot_row_ptr(const RowSrc& rs, int n_begin, int st,
                                                             int h, int i, int n_end, int K) {
  int n = subtile_feature(rs, n_begin, st, h, i);
  if (n >= n_end) return nullptr;
  if (rs.zip) return rs.W[h] + (size_t)n * K;
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
  uint64_t planes_full;    // the activation planes of the current pass have landed
  uint64_t planes_empty;   // every consumer is done with them
  int abort_flag;
  int is_last;
};

// Activation pitch in bytes of one bf16 plane of `cols` columns: = 64 mod 128 so that the 8
// threads of a quarter warp (two rows x four 16-byte columns) hit 32 distinct banks.
__host__ __device__ inline int act_pitch(int cols) {
  int raw = cols * 2;
  return raw + ((64 - (raw & 127)) + 128) % 128;
}

// Features [n_begin, n_end) of CTA `cta` out of `n_cta`, balanced to one feature.
__host__ __device__ inline void cta_range(int N, int cta, int n_cta, int& n_begin, int& n_end) {
  n_begin = (int)(((long long)N * cta) / n_cta);
  n_end = (int)(((long long)N * (cta + 1)) / n_cta);
}

// Producer: streams every (pass, sub-tile, k-chunk, half) of the CTA's feature range through the
// ring, the two halves of a chunk in adjacent slots.  Runs in one warp; lane i < 8 issues the
// copy of row i of a half.  A half without rows still takes its slot (zero bytes expected) so
// that producer and consumers count slots alike.  pass_cols is a multiple of KC.
__device__ __forceinline__ void produce(const RowSrc& rs, int K, int pass_cols, int n_begin,
                                        int n_end, unsigned char* ring, int n_slots, Smem& sm,
                                        int lane) {
  const int n_st = n_subtiles(rs, n_begin, n_end);
  int it = 0;
  for (int k0 = 0; k0 < K; k0 += pass_cols) {
    const int k1 = min(K, k0 + pass_cols);
    for (int st = 0; st < n_st; ++st) {
      const __nv_bfloat16* src[2];
      int n_valid[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        src[h] = lane < kSlotRows ? slot_row_ptr(rs, n_begin, st, h, lane, n_end, K) : nullptr;
        n_valid[h] = __popc(__ballot_sync(0xffffffffu, src[h] != nullptr));
      }
      for (int kc = k0; kc < k1; kc += KC) {
        const int cols = min(KC, k1 - kc);
#pragma unroll
        for (int h = 0; h < 2; ++h, ++it) {
          int slot = it % n_slots;
          uint32_t parity = ((it / n_slots) & 1) ^ 1;   // a fresh barrier passes a wait on parity 1
          int ok = 1;
          if (lane == 0) {
            ok = mbar_wait(&sm.empty[slot], parity, &sm.abort_flag) ? 1 : 0;
            if (ok) mbar_arrive_expect_tx(&sm.full[slot], (uint32_t)(n_valid[h] * cols * 2));
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) return;
          if (src[h])
            bulk_g2s(ring + (size_t)slot * kSlotBytes + lane * kWPitch, src[h] + kc,
                     (uint32_t)(cols * 2), &sm.full[slot]);
        }
      }
    }
  }
}

// Consumer: accumulates one 16-row sub-tile over the k range of the current pass (`cols_pass`
// columns).  Thread (g = lane / 4, t = lane % 4) of warp w loads, per step, 16 bytes of weight
// row g of each half and 16 bytes of activation row g of each plane at the same columns; the 8
// bf16 of a vector feed two MMAs (a permutation of k that both operands share).  NB = 1: up to
// 8 activation rows; NB = 2: up to 16 (a second 8-wide tile).  On return acc[nb][plane pair..]
// is folded into out[nb][4]: out[nb][0..1] = weight row g of half 0, activation rows
// 8 nb + 2t, 2t+1; out[nb][2..3] = the same for half 1.
// `it` is the running slot counter shared with the producer's schedule.  Returns false if a
// wait expired.
template <int NB, bool LO>
__device__ __forceinline__ bool consume_tile(const unsigned char* a_hi, const unsigned char* a_lo,
                                             int apitch, int M, int cols_pass,
                                             const unsigned char* ring, int n_slots, Smem& sm,
                                             int& it, int warp, int lane, float (&out)[NB][4]) {
  const int g = lane >> 2, t = lane & 3;
  // independent accumulators: (hi, lo) x (two k halves of a vector): no MMA waits for another
  float p[NB][4][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int k = 0; k < 4; ++k) p[nb][j][k] = 0.f;
  bool row_ok[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) row_ok[nb] = g + 8 * nb < M;
  for (int c0 = 0; c0 < cols_pass; c0 += KC, it += 2) {
    const int slot0 = it % n_slots, slot1 = (it + 1) % n_slots;
    if (!mbar_wait(&sm.full[slot0], (it / n_slots) & 1, &sm.abort_flag)) return false;
    if (!mbar_wait(&sm.full[slot1], ((it + 1) / n_slots) & 1, &sm.abort_flag)) return false;
    const int cols = min(KC, cols_pass - c0);
    const unsigned char* w0 = ring + (size_t)slot0 * kSlotBytes + g * kWPitch;
    const unsigned char* w1 = ring + (size_t)slot1 * kSlotBytes + g * kWPitch;
    const unsigned char* ah = a_hi + (size_t)g * apitch + (size_t)c0 * 2;
    const unsigned char* al = a_lo + (size_t)g * apitch + (size_t)c0 * 2;
#pragma unroll
    for (int s = 0; s < kStepsPerWarp; ++s) {
      const int col = warp * kColsPerWarp + s * 32 + t * 8;     // column inside the chunk
      if (warp * kColsPerWarp + s * 32 < cols) {                // warp-uniform
        const bool in = col < cols;
        const uint4 z = make_uint4(0, 0, 0, 0);
        const uint4 q0 = in ? *reinterpret_cast<const uint4*>(w0 + col * 2) : z;
        const uint4 q1 = in ? *reinterpret_cast<const uint4*>(w1 + col * 2) : z;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          const size_t ro = (size_t)8 * nb * apitch + (size_t)col * 2;
          const uint4 h = (in && row_ok[nb]) ? *reinterpret_cast<const uint4*>(ah + ro) : z;
          mma_bf16(p[nb][0], q0.x, q1.x, q0.y, q1.y, h.x, h.y);
          mma_bf16(p[nb][1], q0.z, q1.z, q0.w, q1.w, h.z, h.w);
          if (LO) {   // the lo plane is identically zero when the operand is exact bf16
            const uint4 l = (in && row_ok[nb]) ? *reinterpret_cast<const uint4*>(al + ro) : z;
            mma_bf16(p[nb][2], q0.x, q1.x, q0.y, q1.y, l.x, l.y);
            mma_bf16(p[nb][3], q0.z, q1.z, q0.w, q1.w, l.z, l.w);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) {
      mbar_arrive(&sm.empty[slot0]);
      mbar_arrive(&sm.empty[slot1]);
    }
  }
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int k = 0; k < 4; ++k) out[nb][k] = (p[nb][0][k] + p[nb][1][k]) + (p[nb][2][k] + p[nb][3][k]);
  return true;
}

}  // namespace ws
}  // namespace ps
