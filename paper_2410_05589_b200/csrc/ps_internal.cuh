// Internal declarations shared by the translation units of the library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <string>
#include <vector>

#include "ps.h"

namespace ps {

constexpr int kMaxRowsPerSeq = PS_MAX_MASKS + 1;  // rows of one sequence in a draft step
constexpr int kAppendChunk = 256;                 // rows handled per pass of ps_kv_append
constexpr int kAttnMaxSplit = 32;                 // key-range splits of the fused attention
constexpr int kMaxSm = 192;                       // bound used to size per-CTA scratch
constexpr size_t kGuardBytes = 256;               // guard words behind every slice of the workspace
constexpr int kGuardFill = 0x5A;

// Which sequence each row of a launch belongs to.  Passed by value as a kernel parameter.
// Row m (0-based within the launch) belongs to the sequence b with
// row_off[b] <= m + row_base < row_off[b+1]; its index inside the sequence is
// j = m + row_base - row_off[b] and its absolute position is len[b] + j.
struct SeqMap {
  int B;
  int row_base;
  int slot[PS_MAX_BATCH];
  int len[PS_MAX_BATCH];
  int row_off[PS_MAX_BATCH + 1];
};

__device__ __forceinline__ void seq_of_row(const SeqMap& s, int m, int& b, int& j) {
  int g = m + s.row_base;
  int lo = 0, hi = s.B - 1;
  while (lo < hi) {  // last b with row_off[b] <= g (empty sequences are skipped by taking the last)
    int mid = (lo + hi + 1) >> 1;
    if (s.row_off[mid] <= g) lo = mid; else hi = mid - 1;
  }
  b = lo;
  j = g - s.row_off[lo];
}

// Programmatic dependent launch.  A kernel launched with `launch_after` (pdl = true) may start
// while the kernel before it in the stream still runs; it must call pdl_wait() before it reads
// or writes anything that kernel touches (a no-op for a plain launch), and calls
// pdl_launch_dependents() early so that its own successor may be scheduled behind it.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <class... KArgs, class... Args>
cudaError_t launch_after(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                         Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Philox-4x32 with 10 rounds (Salmon et al., SC'11): counter (c0..c3), key (k0, k1).
__device__ __forceinline__ void philox4x32_10(uint32_t k0, uint32_t k1, uint32_t (&c)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0 = __umulhi(0xD2511F53u, c[0]), lo0 = 0xD2511F53u * c[0];
    uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]), lo1 = 0xCD9E8D57u * c[2];
    uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
    c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
}

// Draft sampling (Algorithm 1: the tree is drafted by sampling from the parallel drafter): the
// token of a row is the arg-max over v of logit_v / T + G(v, row), G = -ln(-ln u) (the
// Gumbel-max rule), u = ((w >> 8) + 0.5) / 2^24 with w = word 0 of Philox, key = (seed_lo ^
// 0x6D756247, seed_hi), counter = (v, row_id, offset); row_id = b | j << 8.
struct SampleArgs {
  float inv_temp;
  uint32_t key0, key1, off_lo, off_hi;
  int* sampled;   // [B][k+1]
  uint32_t b_base;   // index, in the caller's batch, of the first sequence of this launch
};
__device__ __forceinline__ float gumbel_noise(const SampleArgs& sa, uint32_t v, uint32_t row_id) {
  uint32_t c[4] = {v, row_id, sa.off_lo, sa.off_hi};
  philox4x32_10(sa.key0, sa.key1, c);
  // e = -ln u in single precision without losing u's distance from 1 (u can sit within 2^-25
  // of it): below one half from u itself, above from 1 - u = (2^24 - w - 0.5) / 2^24, which like
  // w + 0.5 is exact in fp32 on its half of the range.
  const uint32_t w = c[0] >> 8;
  float e;
  if (w < (1u << 23)) e = -__logf(((float)w + 0.5f) * (1.0f / 16777216.0f));
  else e = -log1pf(-((float)(16777216u - w) - 0.5f) * (1.0f / 16777216.0f));
  return -__logf(e);
}

// Device status word values (bit flags).
constexpr int kStatNonfinite = 1;
constexpr int kStatTimeout = 2;

struct TreeRec {    // one per (sequence, decision row) of the token-tree verification
  int next;         // accepted child node, -1 if none
  int token;        // token to emit if the walk stops here
  int bad;          // a non-finite logit was met
};

struct VerifyRec {  // one per (sequence, position): result of the acceptance test
  int accept;       // bit 0: accepted; bit 1: a non-finite logit was met
  int token;        // token to emit if this position ends the chain
};

}  // namespace ps

struct ps_ctx {
  ps_config cfg;
  ps_weights w;
  int device;
  char* ws;
  size_t ws_bytes;
  int max_rows;    // rows the activation buffers hold
  // workspace slices
  void* kcache;    // [max_batch][n_kv_heads][max_ctx][head_dim] storage dtype, post-RoPE
  void* vcache;
  int* dev_status;
  unsigned* tickets;        // [max_batch] arrival counters of the verify kernel (zero between calls)
  ps::VerifyRec* vrec;      // [max_batch][PS_MAX_MASKS+2]
  ps::TreeRec* trec;        // [max_batch][PS_MAX_TREE_NODES+1]
  unsigned* tree_tickets;   // [max_batch], zero between calls
  float *x_in, *x0, *xn, *q, *kv_tmp, *attn, *a, *an, *gate, *up, *hdn, *hn, *logits;
  void* kv_side;            // [max_rows][2 * Hkv] storage dtype: k / v of a draft step's new rows (plain kernels)
  // staging for ps_round_host
  void* fused_scratch;      // buffers of the fused bf16 path (see fused_kernels.cu)
  void* umma_maps = nullptr;   // tensor maps of the tensor-core GEMMs, built on first use
  bool umma_tried = false;
  double* rope_inv_freq;    // [head_dim/2] base^(-2i/d), filled once at ps_init
  int n_sm;                 // multiprocessors of the context's device
  int smem_optin;           // opt-in shared memory per block
  // answers asked of this context's device once (0 = not asked yet)
  int cluster_ok[2][17] = {};     // [chain verify, tree verify][cluster size]: 1 yes, -1 no
  int attn_blocks_per_sm[4][16] = {};   // [kernel variant][tile size / 16]: resident blocks, -1 none
  cudaStream_t copy_stream = nullptr;   // ps_round_host: carries the target logits beside the draft step
  cudaEvent_t copy_done = nullptr;
  int* host_res = nullptr;              // ps_round_host: pinned host copy of the round's results
  void* st_hidden; int* st_tok; float* st_tlogits; float* st_dlogits; int* st_top; int* st_res;
  std::vector<int> len;     // committed positions per slot (host is the source of truth)
  std::vector<size_t> guards;   // offsets of the guard words in the workspace
  long long launches;
  std::string err;
  // optional stage timing (ps_profile): events recorded between stages
  bool prof = false;
  bool prof_launches = false;   // events per launch: chained stages stay chained (ps_profile(ctx, 2))
  std::vector<cudaEvent_t> prof_ev;
  std::vector<const char*> prof_name;   // name of the stage that ENDS at the event
  size_t prof_used = 0;
};

namespace ps {

ps_status fail(ps_ctx* c, ps_status s, const std::string& what);
ps_status cuda_check(ps_ctx* c, cudaError_t e, const char* what);
// Records a timing event that closes stage `name` (no-op unless profiling is on).
void prof_mark(ps_ctx* c, cudaStream_t st, const char* name);

// ---- unfused kernels with fp32 activations (all dtypes, all shapes) -----------------------
ps_status plain_kv_append(ps_ctx* c, const SeqMap& sm, int rows, const void* hidden,
                          const int* tokens, cudaStream_t st);
ps_status plain_draft_step(ps_ctx* c, const SeqMap& sm, int B, const void* hidden_last,
                           const int* token_last, int top_n, int* top_ids, float* top_logit,
                           float* row_max, float* row_lse, float* logits_out, float* feat_out,
                           const SampleArgs* sa, cudaStream_t st);
// One block per row of stored logits [M][V]: max, log-sum-exp and top-n of the row.
ps_status launch_row_stats(ps_ctx* c, const float* logits, int M, int V, int top_n, int* top_ids,
                           float* top_logit, float* row_max, float* row_lse, cudaStream_t st);
// One block per row of stored logits [M][V]: the Gumbel-max token of the row (R rows per sequence).
ps_status launch_gumbel_argmax(ps_ctx* c, const float* logits, int M, int V, int R, const SampleArgs& sa,
                               cudaStream_t st);
// ---- fused bf16 kernels for small M ---------------------------------------------------------
bool fused_supported(ps_ctx* c, int M);
int fused_kv_rows(ps_ctx* c);     // rows per pass of fused_kv_append (0: not available)
ps_status fused_kv_append(ps_ctx* c, const SeqMap& sm, int rows, const void* hidden, const int* tokens,
                          cudaStream_t st);
// RoPE on the k half of kv_tmp rows [0, rows) and the store of k and v into the cache rows.
ps_status launch_rope_store_kv(ps_ctx* c, const SeqMap& sm, int rows, cudaStream_t st);
int fused_row_limit(ps_ctx* c);   // most rows fused_supported() takes for this context (0: none)
size_t fused_scratch_bytes(const ps_config& g);
void fused_release(ps_ctx* c);   // frees what the fused path holds on the host
ps_status fused_debug_buffer(ps_ctx* c, const char* name, void** ptr, size_t* bytes);
ps_status launch_rope_table(ps_ctx* c, cudaStream_t st);
// Test kernel: a bounded barrier wait that runs out after `limit_cycles` and raises the status word.
ps_status launch_wait_expires(ps_ctx* c, long long limit_cycles, cudaStream_t st);
ps_status launch_attn_split(ps_ctx* c, const SeqMap& sm, int B, const float* qkv, float* att_ml,
                            float* att_o, unsigned* tickets, __nv_bfloat16* out_hi,
                            __nv_bfloat16* out_lo, cudaStream_t st);
ps_status fused_draft_step(ps_ctx* c, const SeqMap& sm, int B, const void* hidden_last,
                           const int* token_last, int top_n, int* top_ids, float* top_logit,
                           float* row_max, float* row_lse, float* logits_out, float* feat_out,
                           const SampleArgs* sa, cudaStream_t st);
ps_status launch_verify(ps_ctx* c, int B, int n_draft, int n_target, const int* draft_tokens,
                        const float* draft_logits, const float* target_logits, float temperature,
                        uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens,
                        int* n_out, cudaStream_t st);
ps_status launch_verify_tree(ps_ctx* c, int B, int n_nodes, const int* parent, const int* tokens,
                             const float* draft_logits, const float* target_logits, float temperature,
                             uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
                             int* path, int* max_depth_out, cudaStream_t st);
ps_status launch_build_tree(ps_ctx* c, int B, int n_nodes, const int* parent, const int* rank, const int* top_ids,
                            int top_n, const int* sampled_ids, int* tokens, cudaStream_t st);
ps_status launch_kv_copy(ps_ctx* c, int slot, int len, void* K, void* V, bool to_cache,
                         cudaStream_t st);
}  // namespace ps
