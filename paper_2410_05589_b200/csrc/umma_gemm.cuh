// Weight-streaming small-M GEMM on the 5th-generation tensor cores:
//   Y[m][n] = sum_k A[m][k] * W[n][k],  M = B*(k+1) <= 128 rows, W row-major bf16, fp32 sums.
// (The description below is for up to 16 rows; with Mp = 32, 48, 64, 96 or 128 padded rows the planes
// form an N = 2 Mp operand, stages grow and get fewer, and fewer accumulators fit: see
// stage_bytes(), n_stages(), k_split() below.)
//
// The weights are the M side of tcgen05.mma (128 weight rows per instruction), the activation
// rows its N side: the 16 rows of the hi plane and the 16 rows of the lo plane sit one after the
// other in shared memory and form one N = 32 operand, so one instruction retires a 128 x 16
// weight block (4 KB) against both planes (measured: the cost of these small MMAs is per
// instruction, not per column).  The accumulator (128 lanes x 32 columns of fp32) lives in
// tensor memory.  MMAs that add into the same accumulator run one after the other at full
// latency, so the four k steps of a unit go to four accumulators of their own; the epilogue
// adds the four and their two halves.  Operands reach shared memory by tiled TMA loads (cp.async.bulk.tensor.2d) in the
// 128-byte-swizzled K-major layout the instruction reads: per stage one 128-row x 64-column
// box of weights (16 KB) and the matching 16 x 64 boxes of the activation planes.
//
// Work is cut into units of (128-row tile, 64-column k-block); CTA c of a one-CTA-per-SM grid
// takes the contiguous unit range [U c / G, U (c+1) / G) in tile-major order, so the load is
// balanced to one 16 KB unit whatever N and K are (with more than 16 rows the units are dealt
// in larger blocks, down to whole tiles: UArgs::split).  A tile whose k range is shared by several
// CTAs is reduced through fp32 partials in global memory: every contributor writes its partial
// and takes a ticket, the last one adds the partials in CTA order (the sum does not depend on
// who was last) and runs the tile's epilogue.  No CTA waits for another.
//
// Warp roles: warp 0 issues the TMA loads, warp 1 allocates tensor memory and issues the MMAs
// (one lane), warps 2..5 read accumulators back (tcgen05.ld) and run the epilogues; two
// accumulator buffers let a tile's epilogue overlap the next tile's MMAs.
//
// Activations stay fp32-accurate although the tensor cores take bf16: every activation x is
// given as two bf16 planes, hi = bf16(x) and lo = bf16(x - hi), and every weight block is
// multiplied with both (x*w = hi*w + lo*w up to 2^-17).
// Every wait is bounded: on expiry the kernel raises the device status word and returns.
#pragma once
#include <cuda.h>

#include "ws_gemm.cuh"

namespace ps {
namespace umma {

using ws::mbar_arrive;
using ws::mbar_arrive_expect_tx;
using ws::mbar_init;
using ws::mbar_peek;
using ws::mbar_wait;
using ws::smem_u32;

constexpr int kTile = 128;                        // weight rows per tile (MMA M)
constexpr int kBK = 64;                           // k columns per unit: one 128-byte swizzle span
constexpr int kN = 16;                            // activation rows per epilogue chunk
constexpr int kMaxRows = 128;                     // activation rows of a launch (padded to one of kRowPads)
constexpr int kABytes = kTile * kBK * 2;          // 16 KB
constexpr int kBBytes = kN * kBK * 2;             // 2 KB per plane at 16 rows
constexpr int kStageBytes = kABytes + 2 * kBBytes;
constexpr int kStages = 10;                       // at 16 rows; fewer, larger stages for more rows
constexpr int kRingBytes = kStages * kStageBytes;
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
// Geometry of a launch with Mp padded activation rows (one of kRowPads): the hi and lo planes
// form one MMA operand of N = 2 Mp columns; ksplit independent accumulators per tile (one per k
// step of a unit while tensor memory allows: MMAs into one accumulator serialise); two tiles'
// accumulators in tensor memory.
__host__ __device__ constexpr int stage_bytes(int Mp) { return kABytes + 2 * Mp * kBK * 2; }
__host__ __device__ constexpr int n_stages(int Mp) {
  return kRingBytes / stage_bytes(Mp) < kStages ? kRingBytes / stage_bytes(Mp) : kStages;
}
// (a power of two: 4 up to 32 rows, 2 up to 64, else 1)
__host__ __device__ constexpr int k_split(int Mp) { return Mp <= 32 ? kBK / 16 : (Mp <= 64 ? 2 : 1); }
__host__ __device__ constexpr int acc_cols(int Mp) { return k_split(Mp) * 2 * Mp; }
// columns to allocate: two tiles' accumulators, rounded up to a power of two (256 or 512)
__host__ __device__ constexpr int tmem_cols(int Mp) { return 2 * acc_cols(Mp) <= 256 ? 256 : 512; }
// padded row counts the kernel is compiled for
constexpr int kRowPads[] = {16, 32, 48, 64, 96, 128};
constexpr int kNumRowPads = 6;
// Instruction descriptor of kind::f16: fp32 accumulator, bf16 x bf16, both operands K-major,
// N / 8 in bits [17,23), M / 16 in bits [24,29).
constexpr uint32_t idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
}

// ---- PTX wrappers ---------------------------------------------------------------------------
// Shared-memory matrix descriptor, K-major, 128-byte swizzle: rows of 128 bytes, groups of 8
// rows 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Tiled load of one box at element coordinates (x = column, y = row); x * 2 bytes must be a
// multiple of 16.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc_,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc_), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// 16 consecutive accumulator columns of this thread's lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// 64 consecutive accumulator columns of this thread's lane in one instruction.
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float (&v)[64]) {
  uint32_t r[64];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 4-byte asynchronous copy global -> shared and the wait for this thread's copies.
__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
// 16-byte asynchronous copy global -> shared through L2 only (both addresses 16-byte aligned).
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

__device__ __forceinline__ void epi_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
}

// Barrier of the epilogue threads that also tells every one of them whether any passed true.
__device__ __forceinline__ bool epi_any(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred), "n"(kEpiThreads)
      : "memory");
  return r != 0;
}

// ---- control block behind the stages ----------------------------------------------------------
constexpr int kMaxCtas = 192;   // CTAs of one launch (one per SM)

struct Ctl {
  uint64_t full[kStages];     // a stage's boxes have landed
  uint64_t empty[kStages];    // the MMAs that read a stage have completed
  uint64_t acc_full[2];       // an accumulator holds a finished segment
  uint64_t acc_empty[2];      // the epilogue warps have read it back
  uint32_t tmem_base;
  int abort_flag;
  int is_last;
  int tile_last;
  float scale[kMaxRows];
  float red[4][kN];           // one value per epilogue warp and activation row
  float red2[4][kN];
  float cand_v[4][kN];        // top-n candidates per epilogue warp, and the row's previous pick
  int cand_i[4][kN];
  float prev_v[kN];
  int prev_i[kN];
  float xch[kN * 64];         // gate/up exchange: [m][feature of the tile]
  float acc[kN * 128];        // a chunk of a tile's sums, [m][accumulator row]: each thread reads back its own
  float land[kN * 128];       // partials of a shared tile on their way in: [pair of a batch][accumulator row]
  int coff[kMaxCtas];         // a shared tile's contributors: element offset of each one's partial, -1: none
};

constexpr int kSmemBytes = kStages * kStageBytes + (int)sizeof(Ctl) + 1024;   // + alignment slack

}  // namespace umma
}  // namespace ps
