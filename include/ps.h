/* ps.h -- C ABI of the ParallelSpec draft+verify library for NVIDIA B200 (sm_100a).
 *
 * One context = one drafter (weights + per-sequence KV caches) on one GPU.
 * The drafter is the EAGLE-style parallel drafter of the paper: a fully connected
 * layer over [token embedding ; target feature] followed by ONE Llama-style
 * Transformer layer with the target layer's hyper-parameters, decoded by the target's
 * LM head (Sec. 4.3, Sec. 5.1 "Models").  One call of ps_draft_step evaluates the last
 * real position plus k appended [MASK] positions in a single pass and so yields k+1
 * next-token distributions (Sec. 4.1 "Inference"); ps_verify applies speculative-sampling
 * acceptance (Eq. 1; Algorithm 1 with one child per node) against target logits.
 *
 * Conventions
 *   - "device" pointers are CUDA global memory of the context's GPU, "host" pointers are
 *     ordinary process memory.  Every tensor is dense, row-major, innermost index last.
 *   - The library allocates no device memory.  Weights, inputs, outputs and the workspace
 *     are owned by the caller and must stay valid while the context uses them.
 *   - dtype 0: weights, hidden states and the KV cache are float; dtype 1: bf16
 *     (accumulation is fp32 in both).  Logits and statistics are always float.
 *   - Calls validate on the host, enqueue work on the given CUDA stream (a cudaStream_t
 *     passed as void*, NULL = default stream) and return without waiting.  Conditions found
 *     on the device (non-finite logits) set a device status word that ps_poll reads.
 *   - Every function returns a negative ps_status on error and never aborts; after an error
 *     outputs are unspecified but nothing outside the declared extents is written.
 */
#ifndef PS_H_
#define PS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ps_ctx ps_ctx; /* opaque, host memory owned by the library */

typedef enum {
  PS_OK = 0,
  PS_ERR_INVALID_ARG = -1, /* null pointer, size out of range, slot used twice in a batch */
  PS_ERR_UNSUPPORTED = -2, /* a shape the kernels do not cover (see ps_init) */
  PS_ERR_CAPACITY = -3,    /* a KV slab or the workspace is too small */
  PS_ERR_CUDA = -4,        /* a CUDA runtime call failed; ps_last_error has its text */
  PS_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired */
  PS_ERR_NONFINITE = -6    /* NaN or +inf met in logits given to ps_verify */
} ps_status;

enum { PS_DTYPE_F32 = 0, PS_DTYPE_BF16 = 1 };
enum {
  PS_FLAG_FC_BIAS = 1,          /* ps_weights.b_fc is used */
  PS_FLAG_UNFUSED_KERNELS = 2,  /* force the unfused fp32-activation kernels (debugging aid) */
  PS_FLAG_MMA_SYNC_GEMM = 4,    /* fused path: mma.sync GEMM kernels instead of the tcgen05 ones */
  PS_FLAG_STAGE_LAUNCHES = 16,  /* tensor-core path: one launch per GEMM stage also with up to 16 rows, where
                                   the stages on either side of the attention otherwise share a launch */
  PS_FLAG_NO_FC = 8             /* embedding-only input (the Medusa integration, Sec. 4.3): x0 is the token /
                                   [MASK] embedding, there is no fc layer and no target feature; w_fc,
                                   mask_feat and every `hidden` argument are ignored and may be NULL */
};
enum { PS_MAX_BATCH = 128, PS_MAX_MASKS = 15, PS_MAX_TOP_N = 8 };
enum { PS_MAX_TREE_NODES = 64 };  /* nodes of a token tree (ps_verify_tree) */
enum { PS_STATIC_MAX_BATCH = 128, PS_STATIC_MAX_VOCAB = 262144 }; /* limits of ps_verify_static */

typedef struct ps_config {
  int dtype;      /* PS_DTYPE_* */
  int hidden;     /* H, multiple of 8 */
  int n_heads;    /* query heads; n_heads * head_dim is the attention width */
  int n_kv_heads; /* divides n_heads */
  int head_dim;   /* 64 or 128 */
  int ffn;        /* SwiGLU inner width F, multiple of 8 */
  int vocab;      /* V */
  int k_masks;    /* number of [MASK] positions k (Sec. 4.1), 0..PS_MAX_MASKS */
  int max_batch;  /* number of sequence slots, 1..PS_MAX_BATCH */
  int max_ctx;    /* KV rows per slot, INCLUDING the k+1 uncommitted rows of a draft step */
  float rope_base;
  float rms_eps;
  int flags;      /* PS_FLAG_* */
} ps_config;

/* Device pointers, storage type given by ps_config.dtype, matrices row-major [out][in].
 * Sec. 4.3: embed and w_lm are the target's (frozen) embedding and LM head; mask_embed and
 * mask_feat are the k learned [MASK] inputs of the fc layer (embedding half, feature half). */
typedef struct ps_weights {
  const void* embed;      /* [V][H] */
  const void* mask_embed; /* [k][H] */
  const void* mask_feat;  /* [k][H] */
  const void* w_fc;       /* [H][2H], input order [embedding ; feature] */
  const void* b_fc;       /* [H] or NULL */
  const void* g_in;       /* [H] RMSNorm gain before attention */
  const void* w_q;        /* [n_heads*head_dim][H] */
  const void* w_k;        /* [n_kv_heads*head_dim][H] */
  const void* w_v;        /* [n_kv_heads*head_dim][H] */
  const void* w_o;        /* [H][n_heads*head_dim] */
  const void* g_post;     /* [H] RMSNorm gain before the FFN */
  const void* w_gate;     /* [F][H] */
  const void* w_up;       /* [F][H] */
  const void* w_down;     /* [H][F] */
  const void* g_final;    /* [H] RMSNorm gain before the LM head */
  const void* w_lm;       /* [V][H] */
} ps_weights;

/* Bytes of device workspace ps_init needs for this configuration (KV slabs for max_batch
 * slots, activation buffers, verify scratch).  Returns 0 if the configuration is invalid. */
size_t ps_workspace_bytes(const ps_config* cfg);

/* Creates a context.  `workspace` is device memory of at least ps_workspace_bytes(cfg) bytes,
 * 256-byte aligned; the library zero-initialises what it needs on `stream`.  All KV caches
 * start empty.  PS_ERR_UNSUPPORTED: head_dim not 64/128, hidden or ffn not a multiple of 8,
 * n_heads not a multiple of n_kv_heads.  The CUDA device current at this call is the
 * context's device. */
ps_status ps_init(ps_ctx** out, const ps_config* cfg, const ps_weights* weights, void* workspace,
                  size_t workspace_bytes, void* stream);

/* Appends real positions to the drafter's KV caches (Sec. 4.1: only real tokens persist; the
 * [MASK] rows of a draft step are never cached).  For sequence i of the call, rows
 * row_offset[i] .. row_offset[i]+n_new[i]-1 of `hidden` / `tokens` are its new (target
 * feature, token) pairs in order; they pass through the fc layer, the pre-attention norm and
 * the K/V projections (+RoPE at their absolute positions) and land at cache rows
 * [len, len+n_new), then len += n_new.
 *   B            number of sequences in this call (1..max_batch)
 *   seq_slot     host [B], distinct slots in [0, max_batch)
 *   n_new        host [B], >= 0
 *   row_offset   host [B+1], row_offset[0] = 0, row_offset[i+1] = row_offset[i] + n_new[i]
 *   hidden       device [total][H], config dtype
 *   tokens       device [total] int32 in [0, V)
 * PS_ERR_CAPACITY if len + n_new > max_ctx for a sequence (nothing is appended).
 * The same rows in the same calls give the same cache bits; grouping the rows into calls
 * differently may flip the last bit of single bf16 cache entries (the GEMM's summation order
 * depends on the number of rows of a launch). */
ps_status ps_kv_append(ps_ctx* ctx, int B, const int* seq_slot, const int* n_new,
                       const int* row_offset, const void* hidden, const int* tokens, void* stream);

/* One parallel draft step (Sec. 4.1 "Inference"; the k+1 distributions of Algorithm 1).
 * For each sequence: row 0 is the last real position (token_last, hidden_last), rows 1..k are
 * [MASK]_1..[MASK]_k; row j sits at position len+j, attends to the cached real positions and
 * to rows 0..j, and its logits are the drafter's distribution for the token j places after
 * the next one.  Neither the committed cache length nor the cache rows change (the new rows'
 * k / v live in a side buffer of the workspace).  Calling it twice gives identical outputs.
 * A batch of more than 128 rows B*(k+1) runs as several launches per stage, each over a group
 * of whole sequences; a sequence's outputs do not depend on which other sequences are in the
 * call beyond fp32 rounding (the GEMMs' summation order follows the rows of a launch).
 *   B            sequences (1..max_batch);  seq_slot host [B], distinct
 *   hidden_last  device [B][H], config dtype;  token_last device [B] int32
 *   top_n        0..PS_MAX_TOP_N entries per row (0: top_ids/top_logit unused)
 *   top_ids      device [B][k+1][top_n] int32, descending logit, ties to the lower id
 *   top_logit    device [B][k+1][top_n] float
 *   row_max      device [B][k+1] float, max logit of the row (or NULL)
 *   row_lse      device [B][k+1] float, log-sum-exp of the row (or NULL)
 *   logits_out   device [B][k+1][V] float, or NULL to keep logits out of memory
 *   feat_out     device [B][k+1][H] float, or NULL: the layer output before the final norm
 *                (the drafted feature of Sec. 4.3)
 * PS_ERR_CAPACITY if len + k + 1 > max_ctx. */
ps_status ps_draft_step(ps_ctx* ctx, int B, const int* seq_slot, const void* hidden_last,
                        const int* token_last, int top_n, int* top_ids, float* top_logit,
                        float* row_max, float* row_lse, float* logits_out, float* feat_out,
                        void* stream);

/* ps_draft_step that also draws one token per row from softmax(logits / temperature)
 * (Algorithm 1: the draft tree is built "by sampling from the parallel draft model"), inside
 * the LM-head kernel, without a second pass over the logits.  The draw is the Gumbel-max rule:
 * sampled = argmax_v (logit_v / T + G_v), G_v = -ln(-ln u_v), u_v = ((w >> 8) + 0.5) / 2^24
 * with w = word 0 of Philox-4x32-10, key = (seed_lo ^ 0x6D756247, seed_hi), counter =
 * (v, b | j << 8, offset) for row j of the b-th sequence of the call; ties go to the lower id.
 * Passing these tokens and logits_out to ps_verify with the same temperature makes a round
 * lossless end to end.  temperature > 0.
 *   sampled_ids  device [B][k+1] int32
 * Everything else as ps_draft_step.  On the mma.sync fall-back kernels (PS_FLAG_MMA_SYNC_GEMM)
 * logits_out must be given (PS_ERR_UNSUPPORTED otherwise). */
ps_status ps_draft_step_sampled(ps_ctx* ctx, int B, const int* seq_slot, const void* hidden_last,
                                const int* token_last, float temperature, uint64_t seed,
                                uint64_t offset, int* sampled_ids, int top_n, int* top_ids,
                                float* top_logit, float* row_max, float* row_lse, float* logits_out,
                                float* feat_out, void* stream);

/* Group-wise parallel training layout, forward only (Sec. 4.1 "Group-wise Parallel Training",
 * Fig. 3).  The n_groups real pairs (tokens[t], hidden[t]) that follow the slot's committed
 * context each head a parallel group of k+1 rows: the pair and the k [MASK] positions.  Row j
 * of group t has position index len + t + j and attends to the committed context, to the real
 * rows of the groups 0..t and to the [MASK] rows 1..j of its own group, never to a [MASK] row
 * of another group: every group sees what the inference draft step sees after t more real
 * tokens.  Outputs as ps_draft_step with n_groups in the place of B ([n_groups][k+1]...).
 * The slot's committed length is unchanged (cache rows beyond it are used as scratch).
 * PS_ERR_CAPACITY if len + n_groups + k > max_ctx. */
ps_status ps_group_forward(ps_ctx* ctx, int slot, int n_groups, const void* hidden,
                           const int* tokens, int top_n, int* top_ids, float* top_logit,
                           float* row_max, float* row_lse, float* logits_out, float* feat_out,
                           void* stream);

/* Lossless verification of a drafted chain (Eq. 1; Algorithm 1 with one child per node).
 * For position i = 0..n_draft-1 of sequence b, with p = softmax(target_logits[b][i]/T),
 * q = softmax(draft_logits[b][i]/T) and x = draft_tokens[b][i]: accept iff
 * r < min(1, p(x)/q(x)); at the first rejection emit one token drawn from
 * max(0, p-q) normalised and stop; if every draft is accepted and n_target = n_draft+1, emit
 * one token drawn from p of the extra row.  r and the sampling uniform are words 0 and 1 of
 * Philox-4x32-10 with key = seed and counter = (i, b, offset), mapped to [0,1) by their top
 * 24 bits.  temperature 0 is greedy: accept iff x is the arg-max of the target row (ties to
 * the lower id), emit the arg-max otherwise.
 *   draft_tokens  device [B][n_draft] int32
 *   draft_logits  device [B][n_draft][V] float, or NULL: q is the point mass on x
 *   target_logits device [B][n_target][V] float, n_target = n_draft or n_draft+1
 *   accept_len    device [B] int32: number of accepted drafts
 *   out_tokens    device [B][n_draft+1] int32: accepted drafts, then the emitted token, then -1
 *   n_out         device [B] int32: tokens written to out_tokens
 * 1 <= n_draft <= PS_MAX_MASKS+1.  NaN or +inf in a row that is examined: that position is
 * rejected, the arg-max over its non-NaN target logits is emitted and ps_poll reports
 * PS_ERR_NONFINITE. */
ps_status ps_verify(ps_ctx* ctx, int B, int n_draft, int n_target, const int* draft_tokens,
                    const float* draft_logits, const float* target_logits, float temperature,
                    uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
                    void* stream);

/* Lossless verification of a drafted token tree (Algorithm 1 in full; Sec. 3 "token tree
 * verification").  The tree shape is shared by the batch: parent[i] is the parent of node i
 * (a node before i) or -1 for a child of the root; the children of a node are tried in
 * increasing node id (the algorithm's Select order).  A child of the root has depth 0; every
 * node of depth t was drafted from q_t = softmax(draft_logits[b][t]/T), the parallel drafter's
 * distribution for position t.  Decision row u = 0 is the root, u = 1+i the node i;
 * p_u = softmax(target_logits[b][u]/T) is the target distribution after the path that ends
 * there.  At row u the children are tried in turn: accept x iff r < min(1, p(x)/q(x)) and move
 * to that child; otherwise p := max(0, p-q) normalised and the next child is tried.  When no
 * child is left (or u is a leaf) one token is drawn from the current p and the walk stops.
 * r of the j-th child of row u is word 0 of Philox-4x32-10 with key = seed and counter =
 * (u + (j << 16), b, offset); the final draw uses word 1 of the counter (u, b, offset), so a
 * chain-shaped tree reproduces ps_verify with n_target = n_draft + 1.  temperature 0 is
 * greedy: the walk follows the first child that carries the arg-max of the target row.
 *   parent        HOST [n_nodes] int32, 1 <= n_nodes <= PS_MAX_TREE_NODES
 *   tokens        device [B][n_nodes] int32
 *   draft_logits  device [B][D][V] float, D = 1 + the largest depth (may be NULL at T = 0)
 *   target_logits device [B][n_nodes+1][V] float
 *   accept_len    device [B] int32: accepted nodes
 *   out_tokens    device [B][D+1] int32: their tokens, then the drawn token, then -1
 *   n_out         device [B] int32 = accept_len + 1
 *   path          device [B][D] int32: the accepted nodes' ids, then -1
 * Needs vocab % 4 == 0, vocab <= 131072 and 16-byte aligned logits (PS_ERR_UNSUPPORTED
 * otherwise).  Non-finite logits in an examined row: the walk stops there with the arg-max of
 * that target row and ps_poll reports PS_ERR_NONFINITE. */
ps_status ps_verify_tree(ps_ctx* ctx, int B, int n_nodes, const int* parent, const int* tokens,
                         const float* draft_logits, const float* target_logits, float temperature,
                         uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens,
                         int* n_out, int* path, void* stream);

/* Drafts a token tree of a static shape from one parallel draft step (Algorithm 1, the lines
 * that build the tree before the target pass; appendix "Token Tree Verification": the
 * highest-probability tokens of every drafted position are the candidates, fewer of them the
 * deeper the position).  The parallel drafter gives ONE distribution per depth, whatever the
 * path, so node i of depth t = depth(i) takes the rank[i]-th most likely token of row t of the
 * draft step: tokens[b][i] = top_ids[b][t][rank[i]]; where sampled_ids is given, rank 0 takes
 * sampled_ids[b][t] instead (the token ps_draft_step_sampled drew for that row), and a rank
 * r > 0 whose top-n entry equals that sampled token takes entry 0 (so that siblings stay
 * distinct).  parent[] as in ps_verify_tree; the outputs feed ps_verify_tree unchanged, with the
 * first D rows of the draft step's logits as its draft_logits.
 *   parent, rank  HOST [n_nodes] int32; 0 <= rank[i] < top_n; siblings must differ in rank
 *   top_ids       device [B][k+1][top_n] int32 (ps_draft_step's output), top_n >= 1
 *   sampled_ids   device [B][k+1] int32 or NULL
 *   tokens        device [B][n_nodes] int32 (output)
 * PS_ERR_INVALID_ARG for a malformed tree, a depth beyond k, a rank beyond top_n or two siblings
 * of the same rank.  Nothing runs on the host but the validation. */
ps_status ps_build_tree(ps_ctx* ctx, int B, int n_nodes, const int* parent, const int* rank,
                        const int* top_ids, int top_n, const int* sampled_ids, int* tokens,
                        void* stream);

/* Host-buffer convenience for one draft+verify round: copies hidden_last / token_last /
 * target_logits from host memory, runs the draft step for all k+1 rows and ps_verify
 * (n_draft = n_target = k+1) on `stream`, copies accept_len / out_tokens / n_out back and waits
 * for the stream.  At temperature 0 the drafts are the rows' arg-max tokens and verify is greedy;
 * at temperature > 0 they are drawn from softmax(draft logits / temperature) by
 * ps_draft_step_sampled with the same seed and offset, and verify gets those draft logits as q:
 * the round then emits tokens that follow the target distribution (Eq. 1 holds for drafts drawn
 * from q, not for arg-max drafts with a full q).  All pointers except ctx are host memory; pinned
 * memory makes the copies asynchronous.  The target logits travel on a stream of the context's
 * own while the draft step runs, and the three results come back in one copy through a small
 * pinned host buffer of the context (stream and buffer are created by the first call).
 *   hidden_last [B][H] config dtype, token_last [B], target_logits [B][k+1][V] float,
 *   accept_len [B], out_tokens [B][k+2], n_out [B]. */
ps_status ps_round_host(ps_ctx* ctx, int B, const int* seq_slot, const void* hidden_last,
                        const int* token_last, const float* target_logits, float temperature,
                        uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens,
                        int* n_out, void* stream);

/* Committed cache length of a slot (host bookkeeping, no device access). */
ps_status ps_kv_len(ps_ctx* ctx, int slot, int* len);
/* Empties a slot's cache (host bookkeeping only; nothing is enqueued). */
ps_status ps_kv_reset(ps_ctx* ctx, int slot);

/* Test helpers: copy a slot's committed cache rows out of / into the slab.
 * K, V: device [len][n_kv_heads*head_dim] in config dtype (K as cached, i.e. after RoPE). */
ps_status ps_kv_export(ps_ctx* ctx, int slot, void* K, void* V, void* stream);
ps_status ps_kv_import(ps_ctx* ctx, int slot, int len, const void* K, const void* V, void* stream);

/* Waits for `stream`, then returns and clears the device status word: PS_OK,
 * PS_ERR_NONFINITE or PS_ERR_TIMEOUT. */
ps_status ps_poll(ps_ctx* ctx, void* stream);

/* Test helper: device address and size of one of the context's intermediate buffers after a
 * draft step: "x0" (fc output, float [M][H]), "a" (attention block output, float [M][H]),
 * "qkv" (float [M][Hq+2Hkv], before RoPE), "act" (float [M][F], silu(gate)*up).  The last two
 * exist only on the fused bf16 path.  PS_ERR_INVALID_ARG for an unknown name. */
ps_status ps_debug_buffer(ps_ctx* ctx, const char* name, void** ptr, size_t* bytes);

/* Test helper: every slice of the workspace (KV slabs, activation buffers, scratch) is followed by
 * 256 bytes of guard words written at ps_init.  This call waits for `stream`, reads them back and
 * counts the slices whose guard no longer holds its fill: a kernel that wrote past the end of one
 * of its buffers.  n_bad: host int. */
ps_status ps_debug_check_guards(ps_ctx* ctx, void* stream, int* n_bad);

/* Test helper for the error path of bounded device-side waits.  Every wait of the kernels on a
 * copy or on tensor-core work gives up after about a second, raises the device status word
 * and lets the kernel return, so that a lost completion is an error code, not a hung GPU.  This
 * call enqueues a one-thread kernel that waits, with a limit of `limit_cycles` clock cycles
 * (at most 4e9), on a barrier nothing completes; ps_poll then returns PS_ERR_TIMEOUT. */
ps_status ps_debug_wait_expires(ps_ctx* ctx, long long limit_cycles, void* stream);

/* Number of kernel launches the context has enqueued so far (host counter). */
long long ps_launch_count(ps_ctx* ctx);

/* Stage timing.  ps_profile(ctx, 1) makes every later call record a CUDA event after each
 * stage it enqueues (a few microseconds of overhead per stage; every GEMM stage gets a launch
 * of its own, as with PS_FLAG_STAGE_LAUNCHES); ps_profile(ctx, 2) records an event after each
 * launch instead and leaves chained stages chained: their intervals are named "chain_fc_qkv"
 * and "chain_o_ffn_lm"; ps_profile(ctx, 0) stops.
 * ps_profile_read waits for the recorded events and returns, per stage name, the summed time
 * and the number of intervals since profiling was switched on or last read.
 *   names     host [max_stages][32] chars;  total_ms, count: host [max_stages];  n_stages: host */
ps_status ps_profile(ps_ctx* ctx, int enable);
ps_status ps_profile_read(ps_ctx* ctx, int max_stages, char* names, float* total_ms, int* count,
                          int* n_stages);

/* Text of the last error of this context (host string owned by the context). */
const char* ps_last_error(ps_ctx* ctx);
void ps_destroy(ps_ctx* ctx);

/* Philox-4x32-10 (Salmon et al., SC'11) evaluated on the device for n counters:
 * out[i] = philox(key, ctr[i]).  key: host [2]; ctr, out: device [n][4] uint32.  Lets a caller
 * check that the device stream equals the published generator word for word. */
ps_status ps_philox_fill(const uint32_t key[2], const uint32_t* ctr, uint32_t* out, int n,
                         void* stream);

/* ps_verify without a context and without any allocation.  (The paper has no counterpart:
 * this entry point exists for the way the library is embedded, not for the method.)
 *
 * Who needs it: code that runs where device memory may no longer be requested -- an inference
 * server that has handed its whole memory budget to a pool at start-up and forbids later
 * cudaMalloc calls, a plugin inside someone else's allocator-controlled process, a region
 * where an allocation would synchronise the device and stall other streams.  Such callers
 * cannot create a ps_ctx (it needs a workspace) just to run the acceptance test.
 *
 * What it does: exactly what ps_verify does, with the same arguments plus the vocabulary size,
 * but the kernel's scratch (per-sequence arrival counters and per-position records, about
 * 18 KB) lives in a fixed array inside the library's device image.  Every GPU that loads the
 * library holds that array until the process exits.  The call itself performs no cudaMalloc,
 * cudaFree or other allocating routine; inputs and outputs are still the caller's.
 *
 * Limits (PS_ERR_CAPACITY with a message in `err` beyond them): B <= PS_STATIC_MAX_BATCH,
 * n_draft <= PS_MAX_MASKS+1, vocab <= PS_STATIC_MAX_VOCAB.
 *
 * Sharing: there is ONE array per GPU and every call uses it.  It keeps the previous call's
 * contents; the counters that must start at zero are cleared on `stream` before the kernel.
 * Two calls whose kernels may overlap on the same GPU (different streams, different threads)
 * race on it and give wrong results: serialise them.
 *
 * First call on a device: looks up the array's device address once (with that device current)
 * and caches it.  Make that first call outside any stream capture.
 *
 *   nonfinite_flag  device [1] int or NULL: bit 0 is OR-ed in when a NaN/+inf logit was met in
 *                   an examined row (the caller zeroes it beforehand)
 *   err             host buffer for an error text, or NULL;  err_cap its size in bytes
 * All other arguments as in ps_verify. */
ps_status ps_verify_static(int vocab, int B, int n_draft, int n_target, const int* draft_tokens,
                           const float* draft_logits, const float* target_logits,
                           float temperature, uint64_t seed, uint64_t offset, int* accept_len,
                           int* out_tokens, int* n_out, int* nonfinite_flag, char* err,
                           size_t err_cap, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PS_H_ */
