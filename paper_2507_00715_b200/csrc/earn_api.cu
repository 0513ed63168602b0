// C-ABI entry points: host-side validation, workspace layout and kernel dispatch.
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>

#include "earn_common.cuh"

namespace earn {

static std::atomic<uint64_t> g_launches{0};
void note_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return kDefaultSms; }
  if (dev >= 0 && dev < 64 && cached[dev].load(std::memory_order_relaxed) > 0) return cached[dev].load(std::memory_order_relaxed);
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { (void)cudaGetLastError(); return kDefaultSms; }
  if (dev >= 0 && dev < 64) cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

// ---- what the previous call of this library on a stream launched, remembered per stream (a small table, oldest entry
// reused).  A decode kernel may fetch its shared segment before the programmatic-launch wait when the kernel ahead of it
// on the stream (a) cannot have written that segment and (b) itself waited for ITS predecessor before it let its
// successor start -- true of the decode, register-attention and re-parenting kernels, not of the kernels that write a
// cache (compaction, the register projection) or of anything this table has not seen.
enum CallKind { CALL_UNKNOWN = 0, CALL_WRITES_CACHE = 1, CALL_LEAVES_CACHE = 2 };
static std::mutex g_stream_mutex;
static struct { earn_stream_t stream; int kind; uint64_t age; bool used; } g_streams[32];
static uint64_t g_stream_clock = 0;

static void note_call(earn_stream_t stream, int kind) {
  std::lock_guard<std::mutex> lock(g_stream_mutex);
  int slot = 0;
  for (int i = 0; i < 32; ++i) {
    if (g_streams[i].used && g_streams[i].stream == stream) { slot = i; break; }
    if (!g_streams[i].used) { slot = i; break; }
    if (g_streams[i].age < g_streams[slot].age) slot = i;
  }
  g_streams[slot].stream = stream; g_streams[slot].kind = kind; g_streams[slot].age = ++g_stream_clock; g_streams[slot].used = true;
}
static int last_call(earn_stream_t stream) {
  std::lock_guard<std::mutex> lock(g_stream_mutex);
  for (int i = 0; i < 32; ++i)
    if (g_streams[i].used && g_streams[i].stream == stream) return g_streams[i].kind;
  return CALL_UNKNOWN;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static earn_status_t check_model(const earn_model_t* m) {
  if (m == nullptr) return EARN_ERR_INVALID_ARG;
  if (m->n_layers <= 0 || m->split_k < 0 || m->split_k > m->n_layers) return EARN_ERR_INVALID_ARG;
  if (m->n_q_heads <= 0 || m->n_kv_heads <= 0 || m->n_q_heads % m->n_kv_heads != 0) return EARN_ERR_INVALID_ARG;
  if (m->dtype != EARN_F32 && m->dtype != EARN_BF16) return EARN_ERR_INVALID_ARG;
  if (!(m->softmax_scale >= 0.f)) return EARN_ERR_INVALID_ARG;
  if (m->head_dim <= 0) return EARN_ERR_INVALID_ARG;
  if (m->head_dim != 64 && m->head_dim != 128) return EARN_ERR_UNSUPPORTED;
  if (m->n_q_heads > 65535) return EARN_ERR_UNSUPPORTED;
  return EARN_OK;
}

static earn_status_t check_batch(const earn_batch_t* b) {
  if (b == nullptr) return EARN_ERR_INVALID_ARG;
  if (b->batch < 0 || b->total_tokens < 0 || b->max_seqlen < 0) return EARN_ERR_INVALID_ARG;
  if (b->n_head_reg < 0 || b->n_tail_reg < 0) return EARN_ERR_INVALID_ARG;
  if (b->batch > 65535) return EARN_ERR_UNSUPPORTED;
  if (b->batch == 0) return b->total_tokens == 0 ? EARN_OK : EARN_ERR_INVALID_ARG;
  if (b->cu_seqlens == nullptr || b->cu_seqlens_host == nullptr) return EARN_ERR_INVALID_ARG;
  const int32_t* cu = b->cu_seqlens_host;
  if (cu[0] != 0 || cu[b->batch] != b->total_tokens) return EARN_ERR_INVALID_ARG;
  int mx = 0;
  for (int i = 0; i < b->batch; ++i) {
    int len = cu[i + 1] - cu[i];
    if (len < 0) return EARN_ERR_INVALID_ARG;
    if (len < b->n_head_reg + b->n_tail_reg) return EARN_ERR_INVALID_ARG;   // registers are rows of the sequence
    mx = len > mx ? len : mx;
  }
  if (mx > b->max_seqlen) return EARN_ERR_INVALID_ARG;
  return EARN_OK;
}

static float scale_of(const earn_model_t* m) {
  return m->softmax_scale > 0.f ? m->softmax_scale : 1.0f / sqrtf((float)m->head_dim);
}
static size_t elem_size(const earn_model_t* m) { return m->dtype == EARN_F32 ? 4 : 2; }

DecodePlan make_decode_plan(const earn_model_t& m, const earn_batch_t& b, int beams, int max_shared_len) {
  DecodePlan p{};
  p.rows = beams * (m.n_q_heads / m.n_kv_heads);
  p.row_tiles = (p.rows + kDecodeRows - 1) / kDecodeRows;
  p.rows_pad = p.row_tiles * kDecodeRows;
  if (max_shared_len <= 0 || b.batch == 0) { p.chunk = 64; p.n_splits = 0; return p; }
  // Split only while the unsplit CTAs would leave the GPU short of work.  Measured on B200 (8 sequences of 4096
  // tokens, 8 kv heads): filling 4 CTA slots per SM took 32 us per layer, 6 slots 35 us, 8 slots 40 us, 3 slots
  // 45 us -- every split adds a partial to write and fold; at the 7B shapes (512 unsplit CTAs) any split cost time.
  // CTAs per split: one per (sequence, kv head) and group of row tiles (up to four row tiles share a CTA)
  const long units = (long)b.batch * m.n_kv_heads * (p.row_tiles <= 2 ? 1 : (p.row_tiles + 3) / 4);
#ifndef EARN_DECODE_SLOTS_PER_SM
#define EARN_DECODE_SLOTS_PER_SM 4
#endif
  const long slots = (long)EARN_DECODE_SLOTS_PER_SM * sm_count();
  long splits = slots / units;
  // Fewer (sequence, kv head) pairs than SMs and at most 2048 shared positions under one row tile: eight warps of one
  // CTA deal the tiles among themselves and fold their partials in shared memory -- no partials in global memory, no
  // ticket, no second pass (measured at the 1.5B shapes, 64 pairs: 10.2 us per layer against 12.8 us with eight splits
  // at 512 tokens, 14.1 against 15.9 at 1024, 21.0 against 22.4 at 2048, level at 3072).
  if (p.row_tiles == 1 && m.head_dim == 128 && units < sm_count() && max_shared_len <= kDecodeUnsplitMaxLen) splits = 1;
  long max_splits = (max_shared_len + 63) / 64;
  if (splits > max_splits) splits = max_splits;
  if (splits < 1) splits = 1;
  p.chunk = (int)round_up((size_t)((max_shared_len + splits - 1) / splits), 64);
  p.n_splits = (max_shared_len + p.chunk - 1) / p.chunk;
  return p;
}

size_t decode_partial_floats(const earn_model_t& m, const earn_batch_t& b, const DecodePlan& p) {
  return (size_t)b.batch * m.n_kv_heads * p.n_splits * p.rows_pad * (size_t)(m.head_dim + 1);
}

// one int32 ticket per (sequence, kv head, row tile), after the status word
static size_t ticket_bytes(const earn_model_t& m, const earn_batch_t& b, const DecodePlan& p) {
  return round_up(sizeof(int32_t) * (size_t)b.batch * m.n_kv_heads * p.row_tiles, 256);
}

size_t prefill_plan_bytes(const earn_batch_t& b) {
  if (b.batch <= 0 || b.cu_seqlens_host == nullptr) return 0;
  return round_up(sizeof(int4) * (size_t)prefill_plan_entries(b, 128), 256);   // an upper bound for either block size
}

size_t workspace_head_bytes(const earn_model_t& m, const earn_batch_t& b, int beams) {
  return kStatusBytes + prefill_plan_bytes(b) + ticket_bytes(m, b, make_decode_plan(m, b, beams, b.max_seqlen));
}

static size_t workspace_need(const earn_model_t* m, const earn_batch_t* b, int beams) {
  DecodePlan full = make_decode_plan(*m, *b, beams, b->max_seqlen);
  DecodePlan reg = make_decode_plan(*m, *b, beams, b->n_head_reg + b->n_tail_reg);
  size_t f = decode_partial_floats(*m, *b, full), r = decode_partial_floats(*m, *b, reg);
  return workspace_head_bytes(*m, *b, beams) + round_up(sizeof(float) * (f > r ? f : r), 256) + 256;
}

static earn_status_t check_cache_shared(const earn_model_t* m, const earn_batch_t* b, const earn_cache_t* c) {
  const int R = b->n_head_reg + b->n_tail_reg;
  if (c == nullptr) return EARN_ERR_INVALID_ARG;
  if (R == 0) return EARN_OK;
  if (c->k_shared == nullptr || c->v_shared == nullptr || !aligned16(c->k_shared) || !aligned16(c->v_shared))
    return EARN_ERR_INVALID_ARG;
  const int need = (R + EARN_PAGE_TOKENS - 1) / EARN_PAGE_TOKENS;
  if (c->pages_per_seq < need) return EARN_ERR_INVALID_ARG;
  if (c->block_table == nullptr && (int64_t)c->n_pages < (int64_t)b->batch * c->pages_per_seq) return EARN_ERR_INVALID_ARG;
  if (c->n_pages <= 0) return EARN_ERR_INVALID_ARG;
  (void)m;
  return EARN_OK;
}

static KeySource paged_source(const earn_batch_t* b, const earn_cache_t* c) {
  KeySource s{};
  s.k = c->k_shared; s.v = c->v_shared;
  s.block_table = c->block_table; s.pages_per_seq = c->pages_per_seq; s.n_pages = c->n_pages;
  s.paged = 1; s.n_regs = b->n_head_reg + b->n_tail_reg;
  return s;
}

// Every host-side check of a decode call except the workspace's (shared by earn_decode_attn and
// earn_decode_attn_static, which must run them before it touches its scratch array).
earn_status_t validate_decode(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t step,
                              const void* q, const void* k_new, const void* v_new, const void* k_full,
                              const void* v_full, const earn_cache_t* cache, const void* o, bool* nothing_to_do) {
  *nothing_to_do = false;
  earn_status_t s = check_model(model);
  if (s != EARN_OK) return s;
  s = check_batch(batch);
  if (s != EARN_OK) return s;
  if (layer < 0 || layer >= model->n_layers || cache == nullptr) return EARN_ERR_INVALID_ARG;
  if (cache->beams < 1 || cache->max_new < 1 || step < 1 || step > cache->max_new) return EARN_ERR_INVALID_ARG;
  if ((int64_t)batch->batch * cache->beams > 65535) return EARN_ERR_UNSUPPORTED;
  if (cache->priv_block_table != nullptr &&
      (cache->n_priv_pages < 1 || cache->priv_pages_per_beam < (cache->max_new + EARN_PAGE_TOKENS - 1) / EARN_PAGE_TOKENS))
    return EARN_ERR_INVALID_ARG;
  if (batch->batch == 0) { *nothing_to_do = true; return EARN_OK; }
  if (layer < model->split_k) {
    if (!k_full || !v_full || !aligned16(k_full) || !aligned16(v_full)) return EARN_ERR_INVALID_ARG;
  } else {
    s = check_cache_shared(model, batch, cache);
    if (s != EARN_OK) return s;
  }
  if (!q || !k_new || !v_new || !o || !cache->k_priv || !cache->v_priv) return EARN_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(o) || !aligned16(cache->k_priv) ||
      !aligned16(cache->v_priv))
    return EARN_ERR_INVALID_ARG;
  return EARN_OK;
}

}  // namespace earn

using namespace earn;

extern "C" {

int32_t earn_version(void) { return 100; }

uint64_t earn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* earn_status_string(earn_status_t s) {
  switch (s) {
    case EARN_OK: return "ok";
    case EARN_ERR_INVALID_ARG: return "invalid argument";
    case EARN_ERR_UNSUPPORTED: return "unsupported configuration";
    case EARN_ERR_WORKSPACE: return "workspace missing or too small";
    case EARN_ERR_CUDA: return "CUDA error at launch";
    case EARN_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

size_t earn_workspace_bytes(const earn_model_t* model, const earn_batch_t* batch, int32_t beams) {
  if (check_model(model) != EARN_OK || check_batch(batch) != EARN_OK || beams < 1) return kStatusBytes;
  return workspace_need(model, batch, beams);
}

earn_status_t earn_workspace_init(void* workspace, size_t workspace_bytes, earn_stream_t stream) {
  if (workspace == nullptr || workspace_bytes < (size_t)kStatusBytes || !aligned16(workspace)) return EARN_ERR_WORKSPACE;
  // status word and split tickets start at zero (the partial buffers behind them need no value)
  note_call(stream, CALL_UNKNOWN);
  return cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_device_status(const void* workspace, earn_stream_t stream) {
  if (workspace == nullptr) return EARN_ERR_WORKSPACE;
  int32_t word = 0;
  if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
    return EARN_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return EARN_ERR_CUDA;
  return word == 0 ? EARN_OK : EARN_ERR_TIMEOUT;
}

earn_status_t earn_prefill_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, const void* q,
                                const void* k, const void* v, void* o, float* lse_or_null, void* workspace,
                                size_t workspace_bytes, earn_stream_t stream) {
  earn_status_t s = check_model(model);
  if (s != EARN_OK) return s;
  s = check_batch(batch);
  if (s != EARN_OK) return s;
  if (layer < 0 || layer >= model->split_k) return EARN_ERR_INVALID_ARG;
  if (batch->total_tokens == 0) return EARN_OK;
  if (!q || !k || !v || !o || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return EARN_ERR_INVALID_ARG;
  if (lse_or_null && !aligned16(lse_or_null)) return EARN_ERR_INVALID_ARG;
  if (workspace == nullptr || workspace_bytes < (size_t)kStatusBytes) return EARN_ERR_WORKSPACE;
  PrefillArgs a{};
  a.q = q; a.k = k; a.v = v; a.o = o; a.lse = lse_or_null;
  a.cu_seqlens = batch->cu_seqlens;
  a.batch = batch->batch; a.max_seqlen = batch->max_seqlen;
  a.Hq = model->n_q_heads; a.Hkv = model->n_kv_heads; a.D = model->head_dim; a.dtype = model->dtype;
  a.scale = scale_of(model);
  note_call(stream, CALL_UNKNOWN);
  if (prefill_tc_supported(a, batch->total_tokens)) {
    if (!aligned16(workspace) || workspace_bytes < kStatusBytes + prefill_plan_bytes(*batch)) return EARN_ERR_WORKSPACE;
    return launch_prefill_tc(a, batch->total_tokens,
                             prefill_plan_entries(*batch, prefill_rows_per_entry(model->n_q_heads, model->n_kv_heads)),
                             reinterpret_cast<char*>(workspace) + kStatusBytes, reinterpret_cast<int32_t*>(workspace),
                             (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
  }
  return launch_prefill_simt(a, (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_compact_kv(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, const void* k,
                              const void* v, const void* q_or_null, void* q_reg_or_null, const earn_cache_t* cache,
                              earn_stream_t stream) {
  earn_status_t s = check_model(model);
  if (s != EARN_OK) return s;
  s = check_batch(batch);
  if (s != EARN_OK) return s;
  if (layer < model->split_k || layer >= model->n_layers) return EARN_ERR_INVALID_ARG;
  s = check_cache_shared(model, batch, cache);
  if (s != EARN_OK) return s;
  const int R = batch->n_head_reg + batch->n_tail_reg;
  if (R == 0 || batch->batch == 0) return EARN_OK;
  if (!k || !v || !aligned16(k) || !aligned16(v)) return EARN_ERR_INVALID_ARG;
  if ((q_or_null == nullptr) != (q_reg_or_null == nullptr)) return EARN_ERR_INVALID_ARG;
  if (q_or_null && (!aligned16(q_or_null) || !aligned16(q_reg_or_null))) return EARN_ERR_INVALID_ARG;
  CompactArgs a{};
  a.k = k; a.v = v; a.q = q_or_null;
  a.k_shared = cache->k_shared; a.v_shared = cache->v_shared; a.q_reg = q_reg_or_null;
  a.cu_seqlens = batch->cu_seqlens; a.block_table = cache->block_table; a.reg_idx = cache->reg_idx;
  a.pages_per_seq = cache->pages_per_seq; a.n_pages = cache->n_pages; a.batch = batch->batch;
  a.r_head = batch->n_head_reg; a.r_tail = batch->n_tail_reg;
  a.kv_row_bytes = (int)(model->n_kv_heads * model->head_dim * elem_size(model));
  a.q_row_bytes = (int)(model->n_q_heads * model->head_dim * elem_size(model));
  note_call(stream, CALL_WRITES_CACHE);
  return launch_compact(a, (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_register_qkv(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                const earn_proj_t* proj, const void* x, const void* w_norm, const void* w_qkv,
                                void* x_norm_scratch, const earn_cache_t* cache, void* q_reg, void* workspace,
                                size_t workspace_bytes, earn_stream_t stream) {
  earn_status_t s = check_model(model);
  if (s != EARN_OK) return s;
  s = check_batch(batch);
  if (s != EARN_OK) return s;
  if (layer < model->split_k || layer >= model->n_layers || proj == nullptr) return EARN_ERR_INVALID_ARG;
  if (model->dtype != EARN_BF16 || model->head_dim != 128) return EARN_ERR_UNSUPPORTED;
  if (proj->d_model <= 0 || proj->d_model % 64 != 0 || proj->max_pos <= 0 || !(proj->rms_eps >= 0.f)) return EARN_ERR_INVALID_ARG;
  if (batch->max_seqlen > proj->max_pos) return EARN_ERR_INVALID_ARG;
  s = check_cache_shared(model, batch, cache);
  if (s != EARN_OK) return s;
  const int R = batch->n_head_reg + batch->n_tail_reg;
  if (R == 0 || batch->batch == 0) return EARN_OK;
  if ((int64_t)batch->batch * R > (int64_t)1 << 24) return EARN_ERR_UNSUPPORTED;
  if (!x || !w_norm || !w_qkv || !x_norm_scratch || !q_reg || !proj->rope_cos || !proj->rope_sin) return EARN_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(w_norm) || !aligned16(w_qkv) || !aligned16(x_norm_scratch) || !aligned16(q_reg) ||
      !aligned16(proj->rope_cos) || !aligned16(proj->rope_sin))
    return EARN_ERR_INVALID_ARG;
  if (workspace == nullptr || workspace_bytes < (size_t)kStatusBytes) return EARN_ERR_WORKSPACE;
  RegisterQkvArgs a{};
  a.x = x; a.w_norm = w_norm; a.w_qkv = w_qkv; a.x_norm = x_norm_scratch; a.q_reg = q_reg;
  a.cache = paged_source(batch, cache);
  a.cu_seqlens = batch->cu_seqlens; a.reg_idx = cache->reg_idx;
  a.rope_cos = proj->rope_cos; a.rope_sin = proj->rope_sin;
  a.status = reinterpret_cast<int32_t*>(workspace);
  a.batch = batch->batch; a.R = R; a.r_head = batch->n_head_reg; a.r_tail = batch->n_tail_reg;
  a.Hq = model->n_q_heads; a.Hkv = model->n_kv_heads; a.d_model = proj->d_model;
  a.x_is_compact = proj->x_is_compact != 0; a.max_pos = proj->max_pos; a.rms_eps = proj->rms_eps;
  note_call(stream, CALL_WRITES_CACHE);
  return launch_register_qkv(a, (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_register_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                 const void* q_reg, const earn_cache_t* cache, void* o_reg, void* workspace,
                                 size_t workspace_bytes, earn_stream_t stream) {
  earn_status_t s = check_model(model);
  if (s != EARN_OK) return s;
  s = check_batch(batch);
  if (s != EARN_OK) return s;
  if (layer < model->split_k || layer >= model->n_layers) return EARN_ERR_INVALID_ARG;
  s = check_cache_shared(model, batch, cache);
  if (s != EARN_OK) return s;
  const int R = batch->n_head_reg + batch->n_tail_reg;
  if (R == 0 || batch->batch == 0) return EARN_OK;
  if (!q_reg || !o_reg || !aligned16(q_reg) || !aligned16(o_reg)) return EARN_ERR_INVALID_ARG;
  if (workspace == nullptr || workspace_bytes < (size_t)kStatusBytes) return EARN_ERR_WORKSPACE;
  RegisterArgs a{};
  a.q_reg = q_reg; a.o_reg = o_reg;
  a.src = paged_source(batch, cache);
  a.batch = batch->batch; a.R = R;
  a.Hq = model->n_q_heads; a.Hkv = model->n_kv_heads; a.D = model->head_dim; a.dtype = model->dtype;
  a.scale = scale_of(model);
  const cudaError_t e = register_mma_supported(a) ? launch_register_mma(a, (cudaStream_t)stream)
                                                  : launch_register_simt(a, (cudaStream_t)stream);
  note_call(stream, e == cudaSuccess ? CALL_LEAVES_CACHE : CALL_UNKNOWN);
  return e == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_compact_register_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                         const void* q, const void* k, const void* v, const earn_cache_t* cache,
                                         void* o_reg, void* workspace, size_t workspace_bytes, earn_stream_t stream) {
  earn_status_t s = check_model(model);
  if (s != EARN_OK) return s;
  s = check_batch(batch);
  if (s != EARN_OK) return s;
  if (layer < model->split_k || layer >= model->n_layers) return EARN_ERR_INVALID_ARG;
  s = check_cache_shared(model, batch, cache);
  if (s != EARN_OK) return s;
  const int R = batch->n_head_reg + batch->n_tail_reg;
  if (R == 0 || batch->batch == 0) return EARN_OK;
  if (!q || !k || !v || !o_reg || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o_reg)) return EARN_ERR_INVALID_ARG;
  if (workspace == nullptr || workspace_bytes < (size_t)kStatusBytes) return EARN_ERR_WORKSPACE;
  RegisterArgs a{};
  a.q_reg = nullptr; a.o_reg = o_reg;
  a.src = paged_source(batch, cache);
  a.batch = batch->batch; a.R = R;
  a.Hq = model->n_q_heads; a.Hkv = model->n_kv_heads; a.D = model->head_dim; a.dtype = model->dtype;
  a.scale = scale_of(model);
  a.q_full = q; a.k_full = k; a.v_full = v; a.cu_seqlens = batch->cu_seqlens; a.reg_idx = cache->reg_idx;
  a.r_head = batch->n_head_reg; a.r_tail = batch->n_tail_reg;
  if (!register_mma_supported(a)) return EARN_ERR_UNSUPPORTED;
  note_call(stream, CALL_WRITES_CACHE);
  return launch_register_mma(a, (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_decode_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t step,
                               const void* q, const void* k_new, const void* v_new, const void* k_full_or_null,
                               const void* v_full_or_null, const earn_cache_t* cache, void* o, void* workspace,
                               size_t workspace_bytes, earn_stream_t stream) {
  bool nothing_to_do = false;
  earn_status_t s = validate_decode(model, batch, layer, step, q, k_new, v_new, k_full_or_null, v_full_or_null, cache, o,
                                    &nothing_to_do);
  if (s != EARN_OK || nothing_to_do) return s;
  const bool early = layer < model->split_k;
  if (workspace == nullptr || !aligned16(workspace) || workspace_bytes < workspace_need(model, batch, cache->beams))
    return EARN_ERR_WORKSPACE;

  DecodeArgs a{};
  a.q = q; a.k_new = k_new; a.v_new = v_new; a.o = o;
  if (early) {
    a.src.k = k_full_or_null; a.src.v = v_full_or_null; a.src.cu_seqlens = batch->cu_seqlens; a.src.paged = 0;
  } else {
    a.src = paged_source(batch, cache);
  }
  a.cu_seqlens = batch->cu_seqlens;
  a.k_priv = cache->k_priv; a.v_priv = cache->v_priv; a.lineage = cache->lineage;
  a.priv_table = cache->priv_block_table; a.priv_pages_per_beam = cache->priv_pages_per_beam; a.n_priv_pages = cache->n_priv_pages;
  a.plan = make_decode_plan(*model, *batch, cache->beams,
                            early ? batch->max_seqlen : batch->n_head_reg + batch->n_tail_reg);
  const size_t tickets_at = kStatusBytes + prefill_plan_bytes(*batch);
  a.tickets = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(workspace) + tickets_at);
  a.part_o = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) + tickets_at + ticket_bytes(*model, *batch, a.plan));
  a.part_lse = a.part_o + (size_t)batch->batch * model->n_kv_heads * a.plan.n_splits * a.plan.rows_pad * model->head_dim;
  a.batch = batch->batch; a.beams = cache->beams; a.max_new = cache->max_new; a.step = step;
  a.Hq = model->n_q_heads; a.Hkv = model->n_kv_heads; a.D = model->head_dim; a.dtype = model->dtype;
  a.scale = scale_of(model);
  // Prompt-cache layers of a ragged batch: hand the CTAs out longest sequence first.  The order table (one small
  // launch ahead of the decode kernel) lives in the workspace's prefill-plan area, which holds at least 16 bytes per
  // sequence and is rewritten by every prefill call before it is read.  Worth it when the prompts are long and uneven.
  // The shared segment may be fetched ahead of the stream-order wait when the call before this one on the stream
  // launched a kernel that leaves every cache as it found it (see note_call above).
  a.prefetch_shared = last_call(stream) == CALL_LEAVES_CACHE ? 1 : 0;
  a.order = nullptr;
  if (early && model->dtype == EARN_BF16 && batch->batch >= 2 && batch->batch <= 1024 && batch->max_seqlen >= 1024 &&
      prefill_plan_bytes(*batch) >= sizeof(int32_t) * (size_t)batch->batch) {   // (empty sequences have no plan entry)
    int mn = batch->max_seqlen;
    for (int i = 0; i < batch->batch; ++i) {
      const int len = batch->cu_seqlens_host[i + 1] - batch->cu_seqlens_host[i];
      mn = len < mn ? len : mn;
    }
    if ((int64_t)batch->max_seqlen * 4 > (int64_t)mn * 5) {   // longest more than 1.25 x shortest
      int32_t* order = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(workspace) + kStatusBytes);
      if (launch_decode_order(batch->cu_seqlens, batch->batch, order, (cudaStream_t)stream) != cudaSuccess) return EARN_ERR_CUDA;
      a.order = order;
    }
  }
  const cudaError_t e = model->dtype == EARN_BF16 ? launch_decode_mma(a, early ? batch->max_seqlen : batch->n_head_reg + batch->n_tail_reg, (cudaStream_t)stream)
                                                   : launch_decode_simt(a, (cudaStream_t)stream);
  note_call(stream, e == cudaSuccess ? CALL_LEAVES_CACHE : CALL_UNKNOWN);
  return e == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_beam_reparent(int32_t batch, int32_t beams, int32_t max_new, int32_t step, const int32_t* parent,
                                 const int32_t* lineage_in_or_null, int32_t* lineage_out, earn_stream_t stream) {
  if (batch < 0 || beams < 1 || max_new < 1 || step < 1 || step > max_new) return EARN_ERR_INVALID_ARG;
  if (batch == 0) return EARN_OK;
  if (parent == nullptr || lineage_out == nullptr || lineage_out == lineage_in_or_null) return EARN_ERR_INVALID_ARG;
  const bool ok = launch_beam_reparent(batch, beams, max_new, step, parent, lineage_in_or_null, lineage_out,
                                       (cudaStream_t)stream) == cudaSuccess;
  note_call(stream, ok ? CALL_LEAVES_CACHE : CALL_UNKNOWN);   // an ordinary launch that writes the lineage table only
  return ok ? EARN_OK : EARN_ERR_CUDA;
}

static size_t train_scratch_bytes(const earn_model_t* m, const earn_batch_t* b) {
  return round_up(sizeof(float) * (size_t)m->n_q_heads * (size_t)b->total_tokens, 256);   // one [Hq, total] fp32 array
}

size_t earn_train_workspace_bytes(const earn_model_t* model, const earn_batch_t* batch) {
  if (check_model(model) != EARN_OK || check_batch(batch) != EARN_OK) return kStatusBytes;
  // status block | plan of the forward (and, afterwards, of the backward) | delta | LSE in the log2 domain
  return kStatusBytes + prefill_plan_bytes(*batch) + 2 * train_scratch_bytes(model, batch) + 256;
}

// shared argument checks of the two training calls; fills the kernel arguments
static earn_status_t train_setup(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t n_target,
                                 const void* q, const void* k, const void* v, const void* o, const float* lse,
                                 void* workspace, size_t workspace_bytes, TrainArgs* a, bool* nothing_to_do) {
  *nothing_to_do = false;
  earn_status_t s = check_model(model);
  if (s != EARN_OK) return s;
  s = check_batch(batch);
  if (s != EARN_OK) return s;
  if (layer < 0 || layer >= model->n_layers || n_target < 0) return EARN_ERR_INVALID_ARG;
  const int P = batch->n_head_reg + batch->n_tail_reg + n_target;
  for (int i = 0; i < batch->batch; ++i)
    if (batch->cu_seqlens_host[i + 1] - batch->cu_seqlens_host[i] < P) return EARN_ERR_INVALID_ARG;
  const bool full = layer < model->split_k;
  if (batch->batch == 0 || (full ? batch->total_tokens == 0 : P == 0)) { *nothing_to_do = true; return EARN_OK; }
  if (!q || !k || !v || !o || !lse) return EARN_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse)) return EARN_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned16(workspace) || workspace_bytes < earn_train_workspace_bytes(model, batch))
    return EARN_ERR_WORKSPACE;
  *a = TrainArgs{};
  a->q = q; a->k = k; a->v = v; a->o = o; a->lse = const_cast<float*>(lse);
  a->batch = batch->batch; a->Hq = model->n_q_heads; a->Hkv = model->n_kv_heads; a->D = model->head_dim;
  a->dtype = model->dtype; a->scale = scale_of(model);
  if (full) {
    a->cu_seqlens = batch->cu_seqlens; a->total = batch->total_tokens; a->max_seqlen = batch->max_seqlen;
  } else {
    a->cu_seqlens = nullptr; a->uniform_len = P; a->total = batch->batch * P; a->max_seqlen = P;
  }
  char* ws = reinterpret_cast<char*>(workspace);
  a->status = reinterpret_cast<int32_t*>(ws);
  a->delta = reinterpret_cast<float*>(ws + kStatusBytes + prefill_plan_bytes(*batch));
  a->lse2 = reinterpret_cast<float*>(ws + kStatusBytes + prefill_plan_bytes(*batch) + train_scratch_bytes(model, batch));
  return EARN_OK;
}

earn_status_t earn_train_attn_fwd(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t n_target,
                                  const void* q, const void* k, const void* v, void* o, float* lse, void* workspace,
                                  size_t workspace_bytes, earn_stream_t stream) {
  TrainArgs a;
  bool nothing = false;
  earn_status_t s = train_setup(model, batch, layer, n_target, q, k, v, o, lse, workspace, workspace_bytes, &a, &nothing);
  if (s != EARN_OK || nothing) return s;
  a.out_o = o;
  note_call(stream, CALL_UNKNOWN);
  if (layer < model->split_k) {
    // ordinary causal attention: the prefill kernel, with the softmax denominators kept for the backward
    PrefillArgs p{};
    p.q = q; p.k = k; p.v = v; p.o = o; p.lse = lse; p.cu_seqlens = batch->cu_seqlens;
    p.batch = batch->batch; p.max_seqlen = batch->max_seqlen;
    p.Hq = a.Hq; p.Hkv = a.Hkv; p.D = a.D; p.dtype = a.dtype; p.scale = a.scale;
    if (prefill_tc_supported(p, batch->total_tokens))
      return launch_prefill_tc(p, batch->total_tokens,
                               prefill_plan_entries(*batch, prefill_rows_per_entry(model->n_q_heads, model->n_kv_heads)),
                               reinterpret_cast<char*>(workspace) + kStatusBytes, a.status,
                               (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
  }
  return launch_train_fwd_simt(a, (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

earn_status_t earn_train_attn_bwd(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t n_target,
                                  const void* q, const void* k, const void* v, const void* o, const float* lse,
                                  const void* d_o, void* dq, void* dk, void* dv, void* workspace, size_t workspace_bytes,
                                  earn_stream_t stream) {
  TrainArgs a;
  bool nothing = false;
  earn_status_t s = train_setup(model, batch, layer, n_target, q, k, v, o, lse, workspace, workspace_bytes, &a, &nothing);
  if (s != EARN_OK || nothing) return s;
  if (!d_o || !dq || !dk || !dv || !aligned16(d_o) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv))
    return EARN_ERR_INVALID_ARG;
  a.d_o = d_o; a.dq = dq; a.dk = dk; a.dv = dv;
  note_call(stream, CALL_UNKNOWN);
  if (layer < model->split_k && train_bwd_tc_supported(a))
    return launch_train_bwd_tc(a, *batch, reinterpret_cast<char*>(workspace) + kStatusBytes, (cudaStream_t)stream) == cudaSuccess
               ? EARN_OK : EARN_ERR_CUDA;
  return launch_train_bwd_simt(a, (cudaStream_t)stream) == cudaSuccess ? EARN_OK : EARN_ERR_CUDA;
}

size_t earn_beam_topk_workspace_bytes(int32_t batch, int32_t beams, int32_t vocab) {
  if (batch < 0 || beams < 1 || beams > 32 || vocab < 1 || !beam_topk_supported(beams, vocab)) return 256;
  return beam_topk_workspace(batch, beams, vocab);
}

earn_status_t earn_beam_topk(int32_t batch, int32_t beams, int32_t n_live, int32_t vocab, const float* logprobs,
                             const float* beam_scores_or_null, int32_t* parent, int32_t* token, float* new_scores,
                             void* workspace, size_t workspace_bytes, earn_stream_t stream) {
  if (batch < 0 || beams < 1 || beams > 32 || vocab < 1 || n_live < 1 || n_live > beams) return EARN_ERR_INVALID_ARG;
  if ((int64_t)n_live * vocab < beams) return EARN_ERR_INVALID_ARG;   // fewer continuations than beams to fill
  if (batch > 65535 || !beam_topk_supported(beams, vocab)) return EARN_ERR_UNSUPPORTED;
  if (batch == 0) return EARN_OK;
  if (!logprobs || !parent || !token || !new_scores || new_scores == beam_scores_or_null) return EARN_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(logprobs) | reinterpret_cast<uintptr_t>(parent) | reinterpret_cast<uintptr_t>(token) |
       reinterpret_cast<uintptr_t>(new_scores) | reinterpret_cast<uintptr_t>(beam_scores_or_null)) & 3u)
    return EARN_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned16(workspace) || workspace_bytes < beam_topk_workspace(batch, beams, vocab))
    return EARN_ERR_WORKSPACE;
  const bool ok = launch_beam_topk(batch, beams, n_live, vocab, logprobs, beam_scores_or_null, parent, token, new_scores,
                                   workspace, (cudaStream_t)stream) == cudaSuccess;
  note_call(stream, ok ? CALL_LEAVES_CACHE : CALL_UNKNOWN);   // ordinary launches that write the beam tables only
  return ok ? EARN_OK : EARN_ERR_CUDA;
}

}  // extern "C"
