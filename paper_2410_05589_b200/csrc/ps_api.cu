// C ABI entry points: argument validation, workspace carve-up, host bookkeeping of the
// cache lengths and the choice of kernels.  See include/ps.h for the contract of each call.
#include <algorithm>
#include <cstring>

#include "ps_internal.cuh"

namespace ps {

ps_status fail(ps_ctx* c, ps_status s, const std::string& what) {
  if (c) c->err = what;
  return s;
}

ps_status cuda_check(ps_ctx* c, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return PS_OK;
  if (c) c->err = std::string(what) + ": " + cudaGetErrorString(e);
  return PS_ERR_CUDA;
}

void prof_mark(ps_ctx* c, cudaStream_t st, const char* name) {
  if (!c->prof) return;
  if (c->prof_used == c->prof_ev.size()) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    c->prof_ev.push_back(e);
    c->prof_name.push_back(name);
  }
  c->prof_name[c->prof_used] = name;
  cudaEventRecord(c->prof_ev[c->prof_used++], st);
}

namespace {

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

size_t elem_bytes(const ps_config& g) { return g.dtype == PS_DTYPE_F32 ? 4 : 2; }

ps_status check_config(const ps_config* g) {
  if (!g) return PS_ERR_INVALID_ARG;
  if (g->dtype != PS_DTYPE_F32 && g->dtype != PS_DTYPE_BF16) return PS_ERR_INVALID_ARG;
  if (g->hidden <= 0 || g->n_heads <= 0 || g->n_kv_heads <= 0 || g->ffn <= 0 || g->vocab <= 0)
    return PS_ERR_INVALID_ARG;
  if (g->k_masks < 0 || g->k_masks > PS_MAX_MASKS) return PS_ERR_INVALID_ARG;
  if (g->max_batch < 1 || g->max_batch > PS_MAX_BATCH) return PS_ERR_INVALID_ARG;
  if (g->max_ctx < g->k_masks + 1) return PS_ERR_INVALID_ARG;
  if (!(g->rope_base > 1.f) || !(g->rms_eps >= 0.f)) return PS_ERR_INVALID_ARG;
  if (g->head_dim != 64 && g->head_dim != 128) return PS_ERR_UNSUPPORTED;
  if (g->hidden % 8 || g->ffn % 8) return PS_ERR_UNSUPPORTED;
  if (g->n_heads % g->n_kv_heads) return PS_ERR_UNSUPPORTED;
  return PS_OK;
}

// Walks the workspace layout; with c == nullptr only the size is computed.
size_t carve(const ps_config& g, ps_ctx* c, char* base) {
  size_t off = 0;
  // every slice is followed by kGuardBytes of guard words (filled at ps_init, compared by
  // ps_debug_check_guards): a kernel that writes past the end of its buffer shows up there
  auto take = [&](size_t bytes) {
    size_t at = off;
    off = align_up(off + bytes);
    if (c) c->guards.push_back(off);
    off += kGuardBytes;
    return base ? base + at : nullptr;
  };
  const size_t H = g.hidden, Hq = (size_t)g.n_heads * g.head_dim,
               Hkv = (size_t)g.n_kv_heads * g.head_dim, F = g.ffn, V = g.vocab;
  const size_t R = g.k_masks + 1;
  const size_t Md = (size_t)g.max_batch * R;                      // rows of a draft step
  const size_t Mx = std::max<size_t>(Md, kAppendChunk);           // rows of fc / norm / kv
  const size_t kv = (size_t)g.max_batch * g.n_kv_heads * g.max_ctx * g.head_dim * elem_bytes(g);
  void* kc = take(kv);
  void* vc = take(kv);
  void* status = take(256);
  void* tickets = take(sizeof(unsigned) * PS_MAX_BATCH);
  void* vrec = take(sizeof(VerifyRec) * PS_MAX_BATCH * (PS_MAX_MASKS + 2));
  void* trec = take(sizeof(TreeRec) * PS_MAX_BATCH * (PS_MAX_TREE_NODES + 1));
  void* ttick = take(sizeof(unsigned) * PS_MAX_BATCH);
  void* x_in = take(Mx * 2 * H * 4);
  void* x0 = take(Mx * H * 4);
  void* xn = take(Mx * H * 4);
  void* q = take(Md * Hq * 4);
  void* kv_tmp = take(Mx * 2 * Hkv * 4);
  void* kv_side = take(Md * 2 * Hkv * elem_bytes(g));
  void* attn = take(Md * Hq * 4);
  void* a = take(Md * H * 4);
  void* an = take(Md * H * 4);
  void* gate = take(Md * F * 4);
  void* up = take(Md * F * 4);
  void* hdn = take(Md * H * 4);
  void* hn = take(Md * H * 4);
  void* logits = take(Md * V * 4);
  void* fused = take(fused_scratch_bytes(g));
  void* inv_freq = take(sizeof(double) * 64);
  void* st_hidden = take((size_t)g.max_batch * H * elem_bytes(g));
  void* st_tok = take((size_t)g.max_batch * 4);
  void* st_tlogits = take(Md * V * 4);
  void* st_dlogits = take(Md * V * 4);
  void* st_top = take(Md * 8);  // arg-max ids, then their logits
  void* st_res = take((size_t)g.max_batch * (R + 3) * 4);
  if (c) {
    c->kcache = kc; c->vcache = vc; c->dev_status = (int*)status; c->tickets = (unsigned*)tickets;
    c->vrec = (VerifyRec*)vrec;
    c->trec = (TreeRec*)trec; c->tree_tickets = (unsigned*)ttick;
    c->x_in = (float*)x_in; c->x0 = (float*)x0; c->xn = (float*)xn; c->q = (float*)q;
    c->kv_tmp = (float*)kv_tmp; c->kv_side = kv_side; c->attn = (float*)attn; c->a = (float*)a; c->an = (float*)an;
    c->gate = (float*)gate; c->up = (float*)up; c->hdn = (float*)hdn; c->hn = (float*)hn;
    c->logits = (float*)logits;
    c->fused_scratch = fused;
    c->rope_inv_freq = (double*)inv_freq;
    c->st_hidden = st_hidden; c->st_tok = (int*)st_tok; c->st_tlogits = (float*)st_tlogits;
    c->st_dlogits = (float*)st_dlogits; c->st_top = (int*)st_top; c->st_res = (int*)st_res;
    c->max_rows = (int)Md;
  }
  return off;
}

ps_status check_slots(ps_ctx* c, int B, const int* seq_slot) {
  if (B < 1 || B > c->cfg.max_batch || !seq_slot) return fail(c, PS_ERR_INVALID_ARG, "bad batch");
  bool seen[PS_MAX_BATCH] = {false};
  for (int b = 0; b < B; ++b) {
    int s = seq_slot[b];
    if (s < 0 || s >= c->cfg.max_batch || seen[s])
      return fail(c, PS_ERR_INVALID_ARG, "slot out of range or used twice");
    seen[s] = true;
  }
  return PS_OK;
}

}  // namespace
}  // namespace ps

using namespace ps;

extern "C" {

size_t ps_workspace_bytes(const ps_config* cfg) {
  if (check_config(cfg) != PS_OK) return 0;
  return carve(*cfg, nullptr, nullptr);
}

ps_status ps_init(ps_ctx** out, const ps_config* cfg, const ps_weights* w, void* workspace,
                  size_t workspace_bytes, void* stream) {
  if (!out || !w || !workspace) return PS_ERR_INVALID_ARG;
  ps_status s = check_config(cfg);
  if (s != PS_OK) return s;
  if (((uintptr_t)workspace & 255) != 0) return PS_ERR_INVALID_ARG;
  if (workspace_bytes < carve(*cfg, nullptr, nullptr)) return PS_ERR_CAPACITY;
  const bool no_fc = (cfg->flags & PS_FLAG_NO_FC) != 0;
  const void* need[] = {w->embed, no_fc ? w->embed : w->w_fc, w->g_in, w->w_q, w->w_k, w->w_v, w->w_o, w->g_post,
                        w->w_gate, w->w_up, w->w_down, w->g_final, w->w_lm};
  for (const void* p : need)
    if (!p) return PS_ERR_INVALID_ARG;
  if (cfg->k_masks > 0 && (!w->mask_embed || (!w->mask_feat && !no_fc))) return PS_ERR_INVALID_ARG;
  if (no_fc && (cfg->flags & PS_FLAG_FC_BIAS)) return PS_ERR_INVALID_ARG;
  if ((cfg->flags & PS_FLAG_FC_BIAS) && !w->b_fc) return PS_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return PS_ERR_CUDA;
  ps_ctx* c = new ps_ctx();
  c->cfg = *cfg;
  c->w = *w;
  c->device = dev;
  c->ws = (char*)workspace;
  c->ws_bytes = workspace_bytes;
  c->launches = 0;
  c->len.assign(cfg->max_batch, 0);
  carve(*cfg, c, c->ws);
  cudaStream_t st = (cudaStream_t)stream;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    delete c;
    return PS_ERR_CUDA;
  }
  c->n_sm = std::min(prop.multiProcessorCount, kMaxSm);
  c->smem_optin = (int)prop.sharedMemPerBlockOptin;
  cudaError_t e = cudaSuccess;
  for (size_t go : c->guards)
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + go, kGuardFill, kGuardBytes, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->dev_status, 0, 256, st);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(c->fused_scratch, 0, fused_scratch_bytes(*cfg), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->tickets, 0, sizeof(unsigned) * PS_MAX_BATCH, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->tree_tickets, 0, sizeof(unsigned) * PS_MAX_BATCH, st);
  if (e != cudaSuccess || launch_rope_table(c, st) != PS_OK) {
    delete c;
    return PS_ERR_CUDA;
  }
  *out = c;
  return PS_OK;
}

void ps_destroy(ps_ctx* c) {
  if (!c) return;
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  fused_release(c);
  if (c->copy_stream) {
    cudaEventDestroy(c->copy_done);
    cudaStreamDestroy(c->copy_stream);
  }
  if (c->host_res) cudaFreeHost(c->host_res);
  delete c;
}

ps_status ps_profile(ps_ctx* c, int enable) {
  if (!c) return PS_ERR_INVALID_ARG;
  c->prof = enable != 0;
  c->prof_launches = enable == 2;
  c->prof_used = 0;
  return PS_OK;
}

ps_status ps_profile_read(ps_ctx* c, int max_stages, char* names, float* total_ms, int* count,
                          int* n_stages) {
  if (!c || !names || !total_ms || !count || !n_stages || max_stages < 1) return PS_ERR_INVALID_ARG;
  int n = 0;
  for (size_t i = 1; i < c->prof_used; ++i) {
    const char* nm = c->prof_name[i];
    if (!std::strcmp(nm, "begin")) continue;   // an interval that ends at a "begin" mark is idle time
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(c->prof_ev[i]);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, c->prof_ev[i - 1], c->prof_ev[i]);
    if (e != cudaSuccess) return cuda_check(c, e, "ps_profile_read");
    int j = 0;
    while (j < n && std::strncmp(names + 32 * j, nm, 31)) ++j;
    if (j == n) {
      if (n == max_stages) continue;
      std::strncpy(names + 32 * n, nm, 31);
      names[32 * n + 31] = 0;
      total_ms[n] = 0.f;
      count[n] = 0;
      ++n;
    }
    total_ms[j] += ms;
    count[j] += 1;
  }
  *n_stages = n;
  c->prof_used = 0;
  return PS_OK;
}

const char* ps_last_error(ps_ctx* c) { return c ? c->err.c_str() : "null context"; }

long long ps_launch_count(ps_ctx* c) { return c ? c->launches : 0; }

ps_status ps_debug_buffer(ps_ctx* c, const char* name, void** ptr, size_t* bytes) {
  if (!c || !name || !ptr || !bytes) return PS_ERR_INVALID_ARG;
  const ps_config& g = c->cfg;
  const size_t Md = (size_t)g.max_batch * (g.k_masks + 1);
  if (!std::strcmp(name, "x0")) { *ptr = c->x0; *bytes = Md * g.hidden * 4; return PS_OK; }
  if (!std::strcmp(name, "a")) { *ptr = c->a; *bytes = Md * g.hidden * 4; return PS_OK; }
  return fused_debug_buffer(c, name, ptr, bytes);
}

ps_status ps_debug_check_guards(ps_ctx* c, void* stream, int* n_bad) {
  if (!c || !n_bad) return PS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  std::vector<unsigned char> host(c->guards.size() * kGuardBytes);
  cudaError_t e = cudaSuccess;
  for (size_t i = 0; i < c->guards.size() && e == cudaSuccess; ++i)
    e = cudaMemcpyAsync(host.data() + i * kGuardBytes, c->ws + c->guards[i], kGuardBytes, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_check(c, e, "ps_debug_check_guards");
  int bad = 0;
  for (size_t i = 0; i < c->guards.size(); ++i) {
    bool ok = true;
    for (size_t j = 0; j < kGuardBytes; ++j) ok = ok && host[i * kGuardBytes + j] == (unsigned char)kGuardFill;
    bad += !ok;
  }
  *n_bad = bad;
  return PS_OK;
}

ps_status ps_debug_wait_expires(ps_ctx* c, long long limit_cycles, void* stream) {
  if (!c || limit_cycles < 0 || limit_cycles > 4000000000LL) return PS_ERR_INVALID_ARG;
  return launch_wait_expires(c, limit_cycles, (cudaStream_t)stream);
}

ps_status ps_kv_len(ps_ctx* c, int slot, int* len) {
  if (!c || !len || slot < 0 || slot >= c->cfg.max_batch) return PS_ERR_INVALID_ARG;
  *len = c->len[slot];
  return PS_OK;
}

ps_status ps_kv_reset(ps_ctx* c, int slot) {
  if (!c || slot < 0 || slot >= c->cfg.max_batch) return PS_ERR_INVALID_ARG;
  c->len[slot] = 0;
  return PS_OK;
}

ps_status ps_kv_export(ps_ctx* c, int slot, void* K, void* V, void* stream) {
  if (!c || !K || !V || slot < 0 || slot >= c->cfg.max_batch) return PS_ERR_INVALID_ARG;
  return launch_kv_copy(c, slot, c->len[slot], K, V, false, (cudaStream_t)stream);
}

ps_status ps_kv_import(ps_ctx* c, int slot, int len, const void* K, const void* V, void* stream) {
  if (!c || slot < 0 || slot >= c->cfg.max_batch || len < 0) return PS_ERR_INVALID_ARG;
  if (len > 0 && (!K || !V)) return PS_ERR_INVALID_ARG;
  if (len > c->cfg.max_ctx) return fail(c, PS_ERR_CAPACITY, "import exceeds max_ctx");
  ps_status s = launch_kv_copy(c, slot, len, (void*)K, (void*)V, true, (cudaStream_t)stream);
  if (s == PS_OK) c->len[slot] = len;
  return s;
}

ps_status ps_poll(ps_ctx* c, void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, c->dev_status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->dev_status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_check(c, e, "ps_poll");
  if (word & kStatTimeout) return fail(c, PS_ERR_TIMEOUT, "a bounded device wait expired");
  if (word & kStatNonfinite) return fail(c, PS_ERR_NONFINITE, "non-finite logits in ps_verify");
  return PS_OK;
}

// k / v of `total` real rows (sm.row_off lays them out over the sequences) into the cache, in
// passes of as many rows as the kernels take: the tensor-core GEMM where it serves, else the
// plain kernels.
static ps_status append_rows(ps_ctx* c, SeqMap& sm, int total, const void* hidden, const int* tokens,
                             cudaStream_t st) {
  const int fused_rows = fused_kv_rows(c), chunk = fused_rows > 0 ? fused_rows : kAppendChunk;
  for (int r0 = 0; r0 < total; r0 += chunk) {
    sm.row_base = r0;
    const int rows = std::min(chunk, total - r0);
    const ps_status s = fused_rows > 0 ? fused_kv_append(c, sm, rows, hidden, tokens, st)
                                       : plain_kv_append(c, sm, rows, hidden, tokens, st);
    if (s != PS_OK) return s;
  }
  return PS_OK;
}

ps_status ps_kv_append(ps_ctx* c, int B, const int* seq_slot, const int* n_new,
                       const int* row_offset, const void* hidden, const int* tokens, void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  ps_status s = check_slots(c, B, seq_slot);
  if (s != PS_OK) return s;
  if (!n_new || !row_offset) return fail(c, PS_ERR_INVALID_ARG, "null n_new / row_offset");
  if (row_offset[0] != 0) return fail(c, PS_ERR_INVALID_ARG, "row_offset[0] must be 0");
  for (int b = 0; b < B; ++b) {
    if (n_new[b] < 0 || row_offset[b + 1] != row_offset[b] + n_new[b])
      return fail(c, PS_ERR_INVALID_ARG, "row_offset does not match n_new");
    if (c->len[seq_slot[b]] + n_new[b] > c->cfg.max_ctx)
      return fail(c, PS_ERR_CAPACITY, "append exceeds max_ctx");
  }
  int total = row_offset[B];
  if (total == 0) return PS_OK;
  if ((!hidden && !(c->cfg.flags & PS_FLAG_NO_FC)) || !tokens)
    return fail(c, PS_ERR_INVALID_ARG, "null hidden / tokens");
  SeqMap sm;
  std::memset(&sm, 0, sizeof(sm));
  sm.B = B;
  for (int b = 0; b < B; ++b) {
    sm.slot[b] = seq_slot[b];
    sm.len[b] = c->len[seq_slot[b]];
    sm.row_off[b] = row_offset[b];
  }
  sm.row_off[B] = total;
  if ((s = append_rows(c, sm, total, hidden, tokens, (cudaStream_t)stream)) != PS_OK) return s;
  for (int b = 0; b < B; ++b) c->len[seq_slot[b]] += n_new[b];
  return PS_OK;
}

// Runs the draft rows of the B sequences in `sm` (R rows each, outputs laid out [B][R][...]).
// The tensor-core path takes a bounded number of rows per launch, so a larger batch is cut into
// groups of whole sequences (sequences are independent; each group streams the weights once);
// shapes the fused kernels do not take run on the plain kernels in one piece.
static ps_status run_draft_rows(ps_ctx* c, const SeqMap& sm, int B, const void* hidden, const int* tokens,
                                int top_n, int* top_ids, float* top_logit, float* row_max, float* row_lse,
                                float* logits_out, float* feat_out, const SampleArgs* sa, cudaStream_t st) {
  const ps_config& g = c->cfg;
  const int R = g.k_masks + 1;
  if (fused_supported(c, B * R))
    return fused_draft_step(c, sm, B, hidden, tokens, top_n, top_ids, top_logit, row_max, row_lse,
                            logits_out, feat_out, sa, st);
  const int per_max = fused_row_limit(c) / R;
  if (per_max < 1)
    return plain_draft_step(c, sm, B, hidden, tokens, top_n, top_ids, top_logit, row_max, row_lse,
                            logits_out, feat_out, sa, st);
  // full groups first: a launch costs by its padded row count (16, 32, 64 or 128), so the
  // remainder is better off alone in a small launch than evened out over large ones
  const int per = per_max;
  const size_t eb = g.dtype == PS_DTYPE_F32 ? 4 : 2;
  for (int b0 = 0; b0 < B; b0 += per) {
    const int nb = std::min(per, B - b0);
    SeqMap sub;
    std::memset(&sub, 0, sizeof(sub));
    sub.B = nb;
    for (int b = 0; b < nb; ++b) { sub.slot[b] = sm.slot[b0 + b]; sub.len[b] = sm.len[b0 + b]; sub.row_off[b] = b * R; }
    sub.row_off[nb] = nb * R;
    const size_t r0 = (size_t)b0 * R;
    SampleArgs sub_sa;
    if (sa) { sub_sa = *sa; sub_sa.b_base = sa->b_base + (uint32_t)b0; sub_sa.sampled = sa->sampled + r0; }
    ps_status s = fused_draft_step(
        c, sub, nb, hidden ? (const char*)hidden + (size_t)b0 * g.hidden * eb : nullptr, tokens + b0, top_n,
        top_ids ? top_ids + r0 * top_n : nullptr, top_logit ? top_logit + r0 * top_n : nullptr,
        row_max ? row_max + r0 : nullptr, row_lse ? row_lse + r0 : nullptr,
        logits_out ? logits_out + r0 * g.vocab : nullptr, feat_out ? feat_out + r0 * g.hidden : nullptr,
        sa ? &sub_sa : nullptr, st);
    if (s != PS_OK) return s;
  }
  return PS_OK;
}

static ps_status draft_common(ps_ctx* c, int B, const int* seq_slot, const void* hidden_last,
                              const int* token_last, int top_n, int* top_ids, float* top_logit,
                              float* row_max, float* row_lse, float* logits_out, float* feat_out,
                              const SampleArgs* sa, void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  ps_status s = check_slots(c, B, seq_slot);
  if (s != PS_OK) return s;
  if ((!hidden_last && !(c->cfg.flags & PS_FLAG_NO_FC)) || !token_last)
    return fail(c, PS_ERR_INVALID_ARG, "null hidden / token");
  if (top_n < 0 || top_n > PS_MAX_TOP_N || top_n > c->cfg.vocab)
    return fail(c, PS_ERR_INVALID_ARG, "top_n out of range");
  if (top_n > 0 && (!top_ids || !top_logit)) return fail(c, PS_ERR_INVALID_ARG, "null top-n output");
  const int R = c->cfg.k_masks + 1;
  SeqMap sm;
  std::memset(&sm, 0, sizeof(sm));
  sm.B = B;
  for (int b = 0; b < B; ++b) {
    sm.slot[b] = seq_slot[b];
    sm.len[b] = c->len[seq_slot[b]];
    sm.row_off[b] = b * R;
    if (sm.len[b] + R > c->cfg.max_ctx) return fail(c, PS_ERR_CAPACITY, "no room for the draft rows");
  }
  sm.row_off[B] = B * R;
  return run_draft_rows(c, sm, B, hidden_last, token_last, top_n, top_ids, top_logit, row_max, row_lse,
                        logits_out, feat_out, sa, (cudaStream_t)stream);
}

ps_status ps_draft_step(ps_ctx* c, int B, const int* seq_slot, const void* hidden_last,
                        const int* token_last, int top_n, int* top_ids, float* top_logit,
                        float* row_max, float* row_lse, float* logits_out, float* feat_out,
                        void* stream) {
  return draft_common(c, B, seq_slot, hidden_last, token_last, top_n, top_ids, top_logit, row_max, row_lse,
                      logits_out, feat_out, nullptr, stream);
}

ps_status ps_draft_step_sampled(ps_ctx* c, int B, const int* seq_slot, const void* hidden_last,
                                const int* token_last, float temperature, uint64_t seed, uint64_t offset,
                                int* sampled_ids, int top_n, int* top_ids, float* top_logit,
                                float* row_max, float* row_lse, float* logits_out, float* feat_out,
                                void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  if (!sampled_ids) return fail(c, PS_ERR_INVALID_ARG, "null sampled_ids");
  if (!(temperature > 0.f)) return fail(c, PS_ERR_INVALID_ARG, "temperature must be > 0 (use the arg-max of ps_draft_step at 0)");
  SampleArgs sa;
  sa.inv_temp = 1.f / temperature;
  sa.key0 = (uint32_t)seed ^ 0x6D756247u; sa.key1 = (uint32_t)(seed >> 32);
  sa.off_lo = (uint32_t)offset; sa.off_hi = (uint32_t)(offset >> 32);
  sa.sampled = sampled_ids;
  sa.b_base = 0;
  return draft_common(c, B, seq_slot, hidden_last, token_last, top_n, top_ids, top_logit, row_max, row_lse,
                      logits_out, feat_out, &sa, stream);
}

ps_status ps_group_forward(ps_ctx* c, int slot, int n_groups, const void* hidden, const int* tokens,
                           int top_n, int* top_ids, float* top_logit, float* row_max, float* row_lse,
                           float* logits_out, float* feat_out, void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  const ps_config& g = c->cfg;
  if (slot < 0 || slot >= g.max_batch) return fail(c, PS_ERR_INVALID_ARG, "slot out of range");
  if (n_groups < 1) return fail(c, PS_ERR_INVALID_ARG, "n_groups must be positive");
  if ((!hidden && !(g.flags & PS_FLAG_NO_FC)) || !tokens) return fail(c, PS_ERR_INVALID_ARG, "null hidden / tokens");
  if (top_n < 0 || top_n > PS_MAX_TOP_N || top_n > g.vocab) return fail(c, PS_ERR_INVALID_ARG, "top_n out of range");
  if (top_n > 0 && (!top_ids || !top_logit)) return fail(c, PS_ERR_INVALID_ARG, "null top-n output");
  const int R = g.k_masks + 1, L0 = c->len[slot];
  if (L0 + n_groups + g.k_masks > g.max_ctx) return fail(c, PS_ERR_CAPACITY, "no room for the groups");
  cudaStream_t st = (cudaStream_t)stream;
  const size_t eb = g.dtype == PS_DTYPE_F32 ? 4 : 2;
  ps_status s;
  // 1. the real rows' k / v at cache rows [L0, L0 + n): beyond the committed length, so the
  //    context stays as it was
  SeqMap sm;
  std::memset(&sm, 0, sizeof(sm));
  sm.B = 1; sm.slot[0] = slot; sm.len[0] = L0; sm.row_off[0] = 0; sm.row_off[1] = n_groups;
  if ((s = append_rows(c, sm, n_groups, hidden, tokens, st)) != PS_OK) return s;
  // 2. the groups as a batch of draft steps on the same slot: group t sees cache rows
  //    [0, L0 + t), i.e. the prefix and the real rows before it, and its own k + 1 new rows
  const int chunk = std::min(g.max_batch, (int)PS_MAX_BATCH);
  for (int g0 = 0; g0 < n_groups; g0 += chunk) {
    const int B = std::min(chunk, n_groups - g0);
    std::memset(&sm, 0, sizeof(sm));
    sm.B = B;
    for (int b = 0; b < B; ++b) { sm.slot[b] = slot; sm.len[b] = L0 + g0 + b; sm.row_off[b] = b * R; }
    sm.row_off[B] = B * R;
    const size_t r0 = (size_t)g0 * R;
    const void* h = hidden ? (const char*)hidden + (size_t)g0 * g.hidden * eb : nullptr;
    int* ti = top_ids ? top_ids + r0 * top_n : nullptr;
    float* tl = top_logit ? top_logit + r0 * top_n : nullptr;
    float* rm = row_max ? row_max + r0 : nullptr;
    float* rl = row_lse ? row_lse + r0 : nullptr;
    float* lo = logits_out ? logits_out + r0 * g.vocab : nullptr;
    float* fo = feat_out ? feat_out + r0 * g.hidden : nullptr;
    s = run_draft_rows(c, sm, B, h, tokens + g0, top_n, ti, tl, rm, rl, lo, fo, nullptr, st);
    if (s != PS_OK) return s;
  }
  return PS_OK;
}

ps_status ps_verify(ps_ctx* c, int B, int n_draft, int n_target, const int* draft_tokens,
                    const float* draft_logits, const float* target_logits, float temperature,
                    uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
                    void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  if (B < 1 || B > PS_MAX_BATCH) return fail(c, PS_ERR_INVALID_ARG, "bad batch");
  if (n_draft < 1 || n_draft > PS_MAX_MASKS + 1) return fail(c, PS_ERR_INVALID_ARG, "bad n_draft");
  if (n_target != n_draft && n_target != n_draft + 1)
    return fail(c, PS_ERR_INVALID_ARG, "n_target must be n_draft or n_draft+1");
  if (!draft_tokens || !target_logits || !accept_len || !out_tokens || !n_out)
    return fail(c, PS_ERR_INVALID_ARG, "null pointer");
  if (!(temperature >= 0.f)) return fail(c, PS_ERR_INVALID_ARG, "temperature must be >= 0");
  return launch_verify(c, B, n_draft, n_target, draft_tokens, draft_logits, target_logits,
                       temperature, seed, offset, accept_len, out_tokens, n_out,
                       (cudaStream_t)stream);
}

ps_status ps_verify_tree(ps_ctx* c, int B, int n_nodes, const int* parent, const int* tokens,
                         const float* draft_logits, const float* target_logits, float temperature,
                         uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens, int* n_out,
                         int* path, void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  if (B < 1 || B > PS_MAX_BATCH) return fail(c, PS_ERR_INVALID_ARG, "bad batch");
  if (n_nodes < 1 || n_nodes > PS_MAX_TREE_NODES) return fail(c, PS_ERR_CAPACITY, "tree of 1..PS_MAX_TREE_NODES nodes");
  if (!parent || !tokens || !target_logits || !accept_len || !out_tokens || !n_out || !path)
    return fail(c, PS_ERR_INVALID_ARG, "null pointer");
  if (!(temperature >= 0.f)) return fail(c, PS_ERR_INVALID_ARG, "temperature must be >= 0");
  return launch_verify_tree(c, B, n_nodes, parent, tokens, draft_logits, target_logits, temperature, seed,
                            offset, accept_len, out_tokens, n_out, path, nullptr, (cudaStream_t)stream);
}

ps_status ps_build_tree(ps_ctx* c, int B, int n_nodes, const int* parent, const int* rank, const int* top_ids,
                        int top_n, const int* sampled_ids, int* tokens, void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  if (B < 1 || B > PS_MAX_BATCH) return fail(c, PS_ERR_INVALID_ARG, "bad batch");
  if (n_nodes < 1 || n_nodes > PS_MAX_TREE_NODES) return fail(c, PS_ERR_CAPACITY, "tree of 1..PS_MAX_TREE_NODES nodes");
  if (!parent || !rank || !top_ids || !tokens) return fail(c, PS_ERR_INVALID_ARG, "null pointer");
  if (top_n < 1 || top_n > PS_MAX_TOP_N) return fail(c, PS_ERR_INVALID_ARG, "top_n out of range");
  return launch_build_tree(c, B, n_nodes, parent, rank, top_ids, top_n, sampled_ids, tokens, (cudaStream_t)stream);
}

ps_status ps_round_host(ps_ctx* c, int B, const int* seq_slot, const void* hidden_last,
                        const int* token_last, const float* target_logits, float temperature,
                        uint64_t seed, uint64_t offset, int* accept_len, int* out_tokens,
                        int* n_out, void* stream) {
  if (!c) return PS_ERR_INVALID_ARG;
  ps_status s = check_slots(c, B, seq_slot);
  if (s != PS_OK) return s;
  if (!hidden_last || !token_last || !target_logits || !accept_len || !out_tokens || !n_out)
    return fail(c, PS_ERR_INVALID_ARG, "null pointer");
  if (!(temperature >= 0.f)) return fail(c, PS_ERR_INVALID_ARG, "temperature must be >= 0");
  cudaStream_t st = (cudaStream_t)stream;
  const ps_config& g = c->cfg;
  const int R = g.k_masks + 1;
  const size_t eb = g.dtype == PS_DTYPE_F32 ? 4 : 2;
  cudaError_t e;
  // The target logits are needed by the verify step only: they travel on a stream of their own
  // while the draft step runs (the staging buffer is free: every round ends synchronised).
  if (!c->copy_stream) {
    e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->copy_done, cudaEventDisableTiming);
    if (e == cudaSuccess)   // (pinned HOST memory for the results; no device memory is allocated)
      e = cudaMallocHost((void**)&c->host_res, (size_t)g.max_batch * (g.k_masks + 4) * sizeof(int));
    if (e != cudaSuccess) return cuda_check(c, e, "ps_round_host copy stream");
  }
  e = cudaMemcpyAsync(c->st_tlogits, target_logits, (size_t)B * R * g.vocab * 4, cudaMemcpyHostToDevice,
                      c->copy_stream);
  if (e == cudaSuccess) e = cudaEventRecord(c->copy_done, c->copy_stream);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(c->st_hidden, hidden_last, (size_t)B * g.hidden * eb, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(c->st_tok, token_last, (size_t)B * 4, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return cuda_check(c, e, "ps_round_host h2d");
  // Drafts.  At temperature 0 the chain of arg-max tokens (top_n = 1: top_ids is then exactly
  // [B][k+1]) meets a greedy verify.  Above 0 the acceptance rule keeps the target distribution
  // only for drafts DRAWN from the q it is given (Eq. 1), so the tokens are sampled from
  // softmax(draft logits / T) in the LM head with the round's seed and offset (the sampler's
  // Philox key differs from verify's, so its uniforms are independent of the acceptance tests).
  if (temperature > 0.f)
    s = ps_draft_step_sampled(c, B, seq_slot, c->st_hidden, c->st_tok, temperature, seed, offset, c->st_top, 0,
                              nullptr, nullptr, nullptr, nullptr, c->st_dlogits, nullptr, st);
  else
    s = ps_draft_step(c, B, seq_slot, c->st_hidden, c->st_tok, 1, c->st_top, (float*)(c->st_top + (size_t)c->max_rows),
                      nullptr, nullptr, c->st_dlogits, nullptr, st);
  if (s != PS_OK) return s;
  int* r_acc = c->st_res;
  int* r_n = c->st_res + B;
  int* r_out = c->st_res + 2 * B;
  e = cudaStreamWaitEvent(st, c->copy_done, 0);
  if (e != cudaSuccess) return cuda_check(c, e, "ps_round_host wait");
  s = ps_verify(c, B, R, R, c->st_top, c->st_dlogits, c->st_tlogits, temperature, seed, offset,
                r_acc, r_out, r_n, st);
  if (s != PS_OK) return s;
  // one copy back for the three results (they are adjacent in the staging slice), into pinned
  // host memory of the context, then plain host copies into the caller's arrays
  const size_t res_words = (size_t)B * (R + 3);
  e = cudaMemcpyAsync(c->host_res, c->st_res, res_words * 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e == cudaSuccess) {
    std::memcpy(accept_len, c->host_res, (size_t)B * 4);
    std::memcpy(n_out, c->host_res + B, (size_t)B * 4);
    std::memcpy(out_tokens, c->host_res + 2 * B, (size_t)B * (R + 1) * 4);
  }
  return cuda_check(c, e, "ps_round_host d2h");
}

}  // extern "C"
