// Weight-streaming small-M GEMM for the bf16 drafter:  Y[m][n] = sum_k A[m][k] * W[n][k],
// M = B*(k+1) <= 16 rows, W row-major bf16 (read exactly once from HBM), fp32 accumulation.
//
// One CTA per SM owns a contiguous range of output features n (balanced to one row).  A
// producer warp streams that range through a ring of shared-memory slots with bulk async
// copies (cp.async.bulk + mbarrier transaction counts), 16 weight rows x KC columns per slot;
// eight consumer warps split each slot along k and feed the tensor cores with
// mma.sync.m16n8k16 (activation rows on the 16-wide axis, 8 weight rows per tile).
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

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + one producer warp
constexpr int KC = 512;                          // k-columns per slot
constexpr int kSlotRows = 16;
constexpr int kWPitch = KC * 2 + 64;             // bytes; = 64 mod 128 -> conflict-free 16-byte reads
constexpr int kSlotBytes = kSlotRows * kWPitch;
constexpr int kMaxSlots = 12;
constexpr int kMinSlots = 4;
constexpr int kColsPerWarp = KC / kConsumerWarps;  // 64
constexpr int kStepsPerWarp = kColsPerWarp / 32;   // 2
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
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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

// Global address of slot row i (0..15) of the sub-tile that starts at logical feature n0; nullptr
// if that row lies beyond n_end.  Sub-tiles hold 16 features (8 when zipped).
__device__ __forceinline__ const __nv_bfloat16* slot_row_ptr(const RowSrc& rs, int n0, int i,
                                                             int n_end, int K) {
  if (rs.zip) {
    int n = n0 + (i & 7);
    return n < n_end ? rs.W[i >> 3] + (size_t)n * K : nullptr;
  }
  int n = n0 + i;
  if (n >= n_end) return nullptr;
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

// Producer: streams every (pass, sub-tile, k-chunk) of the CTA's feature range through the ring.
// Runs in one warp; lane i < 16 issues the copy of slot row i.  pass_cols is a multiple of KC.
__device__ __forceinline__ void produce(const RowSrc& rs, int K, int pass_cols, int n_begin,
                                        int n_end, unsigned char* ring, int n_slots, Smem& sm,
                                        int lane) {
  const int feat_per_tile = rs.zip ? 8 : 16;
  int it = 0;
  for (int k0 = 0; k0 < K; k0 += pass_cols) {
    const int k1 = min(K, k0 + pass_cols);
    for (int n0 = n_begin; n0 < n_end; n0 += feat_per_tile) {
      const __nv_bfloat16* src = lane < kSlotRows ? slot_row_ptr(rs, n0, lane, n_end, K) : nullptr;
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

// Consumer: accumulates one sub-tile over the k range of the current pass (`cols_pass` columns)
// into acc[ntile][4].  a_hi / a_lo: bf16 planes [M][cols_pass] with pitch apitch.  `it` is the
// running chunk counter shared with the producer's schedule.  Returns false if a wait expired.
template <bool kUpperRows>
__device__ __forceinline__ bool consume_tile(const unsigned char* a_hi, const unsigned char* a_lo,
                                             int apitch, int M, int cols_pass,
                                             const unsigned char* ring, int n_slots, Smem& sm,
                                             int& it, int warp, int lane, float (&acc)[2][4]) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const bool row_lo = g < M, row_hi = kUpperRows && (g + 8 < M);
  for (int c0 = 0; c0 < cols_pass; c0 += KC, ++it) {
    int slot = it % n_slots;
    uint32_t parity = (it / n_slots) & 1;
    if (*(volatile int*)&sm.abort_flag) return false;
    if (!mbar_wait(&sm.full[slot], parity, &sm.abort_flag)) return false;
    const int cols = min(KC, cols_pass - c0);
    const unsigned char* wbase = ring + (size_t)slot * kSlotBytes;
#pragma unroll
    for (int s = 0; s < kStepsPerWarp; ++s) {
      int col = warp * kColsPerWarp + s * 32 + t * 8;     // column inside the chunk
      if (warp * kColsPerWarp + s * 32 < cols) {          // warp-uniform
        bool in = col < cols;
        const uint4 z = make_uint4(0, 0, 0, 0);
        uint4 b0 = in ? *reinterpret_cast<const uint4*>(wbase + g * kWPitch + col * 2) : z;
        uint4 b1 = in ? *reinterpret_cast<const uint4*>(wbase + (g + 8) * kWPitch + col * 2) : z;
        size_t aoff = (size_t)g * apitch + (size_t)(c0 + col) * 2;
        uint4 h0 = (in && row_lo) ? *reinterpret_cast<const uint4*>(a_hi + aoff) : z;
        uint4 l0 = (in && row_lo) ? *reinterpret_cast<const uint4*>(a_lo + aoff) : z;
        uint4 h1 = z, l1 = z;
        if (kUpperRows) {
          size_t aoff1 = aoff + (size_t)8 * apitch;
          h1 = (in && row_hi) ? *reinterpret_cast<const uint4*>(a_hi + aoff1) : z;
          l1 = (in && row_hi) ? *reinterpret_cast<const uint4*>(a_lo + aoff1) : z;
        }
        mma_bf16(acc[0], h0.x, h1.x, h0.y, h1.y, b0.x, b0.y);
        mma_bf16(acc[0], h0.z, h1.z, h0.w, h1.w, b0.z, b0.w);
        mma_bf16(acc[1], h0.x, h1.x, h0.y, h1.y, b1.x, b1.y);
        mma_bf16(acc[1], h0.z, h1.z, h0.w, h1.w, b1.z, b1.w);
        mma_bf16(acc[0], l0.x, l1.x, l0.y, l1.y, b0.x, b0.y);
        mma_bf16(acc[0], l0.z, l1.z, l0.w, l1.w, b0.z, b0.w);
        mma_bf16(acc[1], l0.x, l1.x, l0.y, l1.y, b1.x, b1.y);
        mma_bf16(acc[1], l0.z, l1.z, l0.w, l1.w, b1.z, b1.w);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[slot]);
  }
  return true;
}

// Splits fp32 values into the hi / lo bf16 planes, 8 consecutive columns at a time.
__device__ __forceinline__ void store_split8(unsigned char* a_hi, unsigned char* a_lo, size_t off,
                                             const float (&x)[8]) {
  uint32_t h[4], l[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 hh = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
    float2 hf = __bfloat1622float2(hh);
    __nv_bfloat162 ll = __floats2bfloat162_rn(x[2 * i] - hf.x, x[2 * i + 1] - hf.y);
    h[i] = *reinterpret_cast<uint32_t*>(&hh);
    l[i] = *reinterpret_cast<uint32_t*>(&ll);
  }
  *reinterpret_cast<uint4*>(a_hi + off) = make_uint4(h[0], h[1], h[2], h[3]);
  *reinterpret_cast<uint4*>(a_lo + off) = make_uint4(l[0], l[1], l[2], l[3]);
}

}  // namespace ws
}  // namespace ps
