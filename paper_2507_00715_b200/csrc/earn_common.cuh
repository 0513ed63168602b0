// Shared declarations of the CUDA side of the EARN attention library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "earn.h"

namespace earn {

constexpr int kStatusBytes = 256;   // head of the workspace: device status word (+ padding)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Where the keys/values a query may see before the generated tokens live ("shared segment").
struct KeySource {
  const void* k;
  const void* v;
  const int32_t* cu_seqlens;   // packed source: row (b, j) is row cu_seqlens[b] + j of [total, Hkv, D]
  const int32_t* block_table;  // paged source: [B, pages_per_seq] or null (identity)
  int pages_per_seq;
  int n_pages;                 // paged: pages allocated (page numbers are clamped to it)
  int paged;                   // 0: packed prompt K/V, 1: compact register cache in pages of 16 tokens
  int n_regs;                  // paged: rows per sequence (R)
};

__device__ __forceinline__ int64_t key_row(const KeySource& s, int b, int j) {
  if (s.paged) {
    int page = j / EARN_PAGE_TOKENS;
    int phys = s.block_table ? s.block_table[b * s.pages_per_seq + page] : b * s.pages_per_seq + page;
    phys = min(max(phys, 0), s.n_pages - 1);   // a corrupt table reads a wrong page, never outside the cache
    return (int64_t)phys * EARN_PAGE_TOKENS + (j % EARN_PAGE_TOKENS);
  }
  return (int64_t)s.cu_seqlens[b] + j;
}

// How split-KV decode divides the shared segment; the same numbers size the workspace.
struct DecodePlan {
  int rows;        // W * g query rows per (sequence, kv head)
  int row_tiles;   // tiles of kDecodeRows rows
  int rows_pad;    // row_tiles * kDecodeRows
  int chunk;       // keys per split (multiple of 64)
  int n_splits;    // ceil(max shared length / chunk); 0 when the shared segment is empty
};
constexpr int kDecodeRows = 16;
constexpr int kDecodeUnsplitMaxLen = 2048;   // shared positions a grid of less than one CTA per SM walks without split-KV
DecodePlan make_decode_plan(const earn_model_t& m, const earn_batch_t& b, int beams, int max_shared_len);
size_t decode_partial_floats(const earn_model_t& m, const earn_batch_t& b, const DecodePlan& p);

// Workspace layout: status block | prefill plan | split-decode tickets | split-decode partials.
size_t prefill_plan_bytes(const earn_batch_t& b);
// status block + plan + tickets: the part of the workspace that must read zero before the first call
size_t workspace_head_bytes(const earn_model_t& m, const earn_batch_t& b, int beams);

// host-side argument checks of a decode call (everything but the workspace); *nothing_to_do: valid call, empty batch
earn_status_t validate_decode(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t step,
                              const void* q, const void* k_new, const void* v_new, const void* k_full,
                              const void* v_full, const earn_cache_t* cache, const void* o, bool* nothing_to_do);

void note_launch(int n = 1);
// SMs of the current device (queried once per device); kDefaultSms when no device can be asked (host-only sizing calls)
constexpr int kDefaultSms = 148;
int sm_count();

// Opt a kernel in to `bytes` of dynamic shared memory and the largest carveout, once per device (the attribute
// calls are not free).
template <auto Kernel>
cudaError_t ensure_dynamic_smem(int bytes) {
  static std::atomic<uint64_t> done{0};   // one bit per device ordinal < 64
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 64 && ((done.load(std::memory_order_relaxed) >> dev) & 1)) return cudaSuccess;
  e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  // ask for the largest shared-memory carveout: left to itself the driver may size it for a single CTA
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(Kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess && dev < 64) done.fetch_or(1ull << dev, std::memory_order_relaxed);
  return e;
}

// ---- programmatic dependent launch: a kernel launched through launch_pdl may start (be scheduled, set up its
// shared memory and barriers) while the kernel before it on the stream is still running; it must call pdl_wait()
// before it touches global memory, which returns once that kernel has completed and its writes are visible.
// pdl_launch_dependents() lets the kernel after this one do the same.  Both are no-ops in an ordinary launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- launchers (one per .cu file); all return cudaGetLastError() of their launches ----
struct PrefillArgs {
  const void *q, *k, *v;
  void* o;
  float* lse;
  const int32_t* cu_seqlens;
  int batch, max_seqlen, Hq, Hkv, D, dtype;
  float scale;
};
cudaError_t launch_prefill_simt(const PrefillArgs& a, cudaStream_t st);
// tensor-core path (bf16, head_dim 128); status_word receives EARN_ERR_TIMEOUT if a bounded wait runs out
bool prefill_tc_supported(const PrefillArgs& a, int total_tokens);
int prefill_rows_per_entry(int n_q_heads, int n_kv_heads);   // query rows one plan entry covers: 128 or 256
int prefill_plan_entries(const earn_batch_t& b, int rows);   // (sequence, block of `rows` query rows) pairs of the batch
// One plan entry per (sequence, block of `rows` rows): {first global row, rows of the sequence from there, block index,
// sequence}, blocks with the highest index (the longest key range) first; at most 2048 blocks per sequence.
cudaError_t launch_tile_plan(const int32_t* cu_seqlens, int batch, int max_seqlen, int rows, int group_seqs, void* plan,
                             cudaStream_t st);
// plan: device scratch of 16 bytes per plan entry, filled by a planning kernel launched ahead of the main one
cudaError_t launch_prefill_tc(const PrefillArgs& a, int total_tokens, int plan_entries, void* plan, int32_t* status_word,
                              cudaStream_t st);

struct RegisterArgs {
  const void* q_reg;
  void* o_reg;
  KeySource src;
  int batch, R, Hq, Hkv, D, dtype;
  float scale;
  // fused with the compaction (bf16 tensor-core kernel only): when k_full is not null the register rows of q, k, v are
  // read straight from the packed prompt tensors (row cu_seqlens[b] + idx_b[m]); K and V are also written to the
  // cache pages `src` names and idx to reg_idx, so that the call leaves what earn_compact_kv leaves
  const void *q_full, *k_full, *v_full;
  const int32_t* cu_seqlens;
  int32_t* reg_idx;
  int r_head, r_tail;
};
cudaError_t launch_register_simt(const RegisterArgs& a, cudaStream_t st);
bool register_mma_supported(const RegisterArgs& a);                      // bf16 and R <= 128
cudaError_t launch_register_mma(const RegisterArgs& a, cudaStream_t st);

struct DecodeArgs {
  const void *q, *k_new, *v_new;
  void* o;
  KeySource src;
  const int32_t* cu_seqlens;   // device, for the shared length of a packed source
  void *k_priv, *v_priv;
  const int32_t* lineage;
  const int32_t* priv_table;   // page table of the private segment [B*W, priv_pages_per_beam], or null: flat slabs
  int priv_pages_per_beam, n_priv_pages;
  float* part_o;               // [B, Hkv, n_splits, rows_pad, D]
  float* part_lse;             // [B, Hkv, n_splits, rows_pad]  (log2 domain)
  int32_t* tickets;            // [B, Hkv, row_tiles], zero between launches: which split finished last
  DecodePlan plan;
  int batch, beams, max_new, step, Hq, Hkv, D, dtype;
  float scale;
  const int32_t* order;        // bf16 kernels: if not null, grid index z is a rank and order[z] the sequence (longest shared segment first)
  // bf16 kernels: the kernel just ahead of this one on the stream cannot have written the shared segment (nor the block
  // table, nor cu_seqlens), so its first tiles may be fetched before the programmatic-launch wait
  int prefetch_shared;
  // bf16 kernels: let the next kernel on the stream be scheduled as soon as this one starts (short key lists) instead of
  // after the key loop
  int trigger_early;
};
// Row of the private (generated-token) segment that holds token t of slab `slab` (the beam that generated it): row
// slab * max_new + t of the flat layout, or, behind a page table, slot t % 16 of page priv_table[slab][t / 16].
__device__ __forceinline__ int64_t priv_row(const DecodeArgs& a, int64_t slab, int t) {
  if (a.priv_table == nullptr) return slab * a.max_new + t;
  int page = a.priv_table[slab * a.priv_pages_per_beam + t / EARN_PAGE_TOKENS];
  page = min(max(page, 0), a.n_priv_pages - 1);   // a corrupt table reads or writes a wrong page, never outside the cache
  return (int64_t)page * EARN_PAGE_TOKENS + t % EARN_PAGE_TOKENS;
}
cudaError_t launch_decode_simt(const DecodeArgs& a, cudaStream_t st);   // fp32 debug path
// bf16: cp.async ring + mma.sync; max_shared_len = longest shared segment of the batch (picks the ring depth)
cudaError_t launch_decode_mma(const DecodeArgs& a, int max_shared_len, cudaStream_t st);
// bf16, one row tile and a list of at most 128 positions (64 at head_dim 64): the whole list in shared memory at once
bool decode_short_supported(const DecodeArgs& a, int max_shared_len);
cudaError_t launch_decode_short(const DecodeArgs& a, int max_shared_len, cudaStream_t st);
// bf16, several row tiles (beams x group size > 16): the row tiles of a CTA share one pass over the shared segment
cudaError_t launch_decode_rows(const DecodeArgs& a, cudaStream_t st);
// order[rank] = sequence, by decreasing prompt length (ties by index); batch <= 1024
cudaError_t launch_decode_order(const int32_t* cu_seqlens, int batch, int32_t* order, cudaStream_t st);

struct CompactArgs {
  const void *k, *v, *q;
  void *k_shared, *v_shared, *q_reg;
  const int32_t* cu_seqlens;
  const int32_t* block_table;
  int32_t* reg_idx;
  int pages_per_seq, n_pages, batch, r_head, r_tail, kv_row_bytes, q_row_bytes;
};
cudaError_t launch_compact(const CompactArgs& a, cudaStream_t st);

// register rows of a layer l >= k straight from the hidden states: gather, RMSNorm, QKV projection, rotary embedding
struct RegisterQkvArgs {
  const void *x, *w_norm, *w_qkv;
  void *x_norm, *q_reg;
  KeySource cache;             // paged compact cache the K and V rows are written to
  const int32_t* cu_seqlens;
  int32_t* reg_idx;
  const float *rope_cos, *rope_sin;
  int32_t* status;
  int batch, R, r_head, r_tail, Hq, Hkv, d_model, x_is_compact, max_pos;
  float rms_eps;
};
cudaError_t launch_register_qkv(const RegisterQkvArgs& a, cudaStream_t st);

cudaError_t launch_beam_reparent(int batch, int beams, int max_new, int step, const int32_t* parent,
                                 const int32_t* lineage_in, int32_t* lineage_out, cudaStream_t st);

// training-time attention (Section 3.2 "Training"): forward with LSE and backward, over packed sequences
// (cu_seqlens) or over the gathered participating rows of the layers after the split (uniform_len rows per sequence)
struct TrainArgs {
  const void *q, *k, *v;       // [rows, Hq, D], [rows, Hkv, D]
  const void* o;               // backward: the forward's output
  const void* d_o;             // backward: upstream gradient, shape of o
  void* out_o;                 // forward: output
  float* lse;                  // natural-log softmax denominators: [Hq, total] (packed) or [B, Hq, P] (uniform); forward writes, backward reads
  void *dq, *dk, *dv;          // backward outputs, shapes of q, k, v
  const int32_t* cu_seqlens;   // device [B+1], or null: sequence b is rows b * uniform_len .. + uniform_len
  int uniform_len;
  int batch, total, max_seqlen, Hq, Hkv, D, dtype;
  float scale;
  float* delta;                // scratch fp32 [Hq, total]: rowsum(dO o O) (tensor-core path)
  float* lse2;                 // scratch fp32 [Hq, total]: LSE in the log2 domain (tensor-core path)
  int32_t* status;
};
cudaError_t launch_train_fwd_simt(const TrainArgs& a, cudaStream_t st);
cudaError_t launch_train_bwd_simt(const TrainArgs& a, cudaStream_t st);
bool train_bwd_tc_supported(const TrainArgs& a);   // bf16, head_dim 128, packed sequences
cudaError_t launch_train_bwd_tc(const TrainArgs& a, const earn_batch_t& b, void* plan, cudaStream_t st);

// beam selection (top W of n_live * vocab continuations per sequence)
bool beam_topk_supported(int beams, int vocab);
size_t beam_topk_workspace(int batch, int beams, int vocab);
cudaError_t launch_beam_topk(int batch, int beams, int n_live, int vocab, const float* logprobs, const float* beam_scores,
                             int32_t* parent, int32_t* token, float* new_scores, void* workspace, cudaStream_t st);

// ---- element helpers ----
template <typename T> struct Elem;
template <> struct Elem<float> {
  static __device__ __forceinline__ void load4(const float* p, float (&x)[4]) {
    float4 t = *reinterpret_cast<const float4*>(p);
    x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
  }
  static __device__ __forceinline__ void store4(float* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
};
template <> struct Elem<__nv_bfloat16> {
  static __device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&x)[4]) {
    uint2 t = *reinterpret_cast<const uint2*>(p);
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&t.x);
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&t.y);
    x[0] = __low2float(a); x[1] = __high2float(a); x[2] = __low2float(b); x[3] = __high2float(b);
  }
  static __device__ __forceinline__ void store4(__nv_bfloat16* p, const float (&x)[4]) {
    __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(x[2], x[3]);
    uint2 t;
    t.x = *reinterpret_cast<uint32_t*>(&a);
    t.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = t;
  }
};

}  // namespace earn
