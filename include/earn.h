/*
 * earn.h — C ABI of the EARN attention hot path for NVIDIA B200 (sm_100a).
 *
 * EARN runs the first k decoder layers over every prompt token and the
 * remaining N-k layers over the register tokens (a few learnable tokens at the
 * head and tail of the prompt) plus the generated tokens only (Section 3.2,
 * "Inference").  This library is the attention part of that pipeline:
 *
 *   layers l <  k : earn_prefill_attn                       (prefill)   earn_decode_attn with k_full/v_full (decode)
 *   layers l >= k : earn_compact_kv -> earn_register_attn    (prefill)   earn_decode_attn over the compact cache (decode)
 *                   (or earn_register_qkv -> earn_register_attn when the caller hands over hidden states and W_qkv)
 *
 * Layers are 0-indexed: 0..k-1 are full layers, k..N-1 register layers.
 *
 * Conventions for every call
 *   - "device" pointers are CUDA device memory owned by the caller; "host" pointers are
 *     ordinary host memory.  Nothing is retained after a call returns except where stated.
 *   - tensors are dense, innermost dimension contiguous, base addresses 16-byte aligned.
 *   - dtype EARN_BF16: elements are bfloat16, arithmetic is fp32 (softmax, accumulation),
 *     outputs are rounded once to bfloat16.  EARN_F32: fp32 in and out (debug path).
 *   - `stream` is a cudaStream_t passed as an opaque pointer (NULL = legacy default stream).
 *     Calls only enqueue work on it; they do not synchronise and allocate no device memory
 *     (workspace comes from the caller), except earn_device_status which synchronises.
 *   - every argument check happens on the host before anything is launched; a call that
 *     returns a status other than EARN_OK has launched nothing, except EARN_ERR_CUDA, which
 *     reports a failed launch.  Nothing throws or exits.
 */
#ifndef EARN_H_
#define EARN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void* earn_stream_t;

typedef enum {
  EARN_OK = 0,
  EARN_ERR_INVALID_ARG = 1, /* null/misaligned pointer, bad shape, layer on the wrong side of k, R > L_b ... */
  EARN_ERR_UNSUPPORTED = 2, /* legal request this build has no kernel for (e.g. head_dim not in {64,128}) */
  EARN_ERR_WORKSPACE = 3,   /* workspace NULL or smaller than earn_workspace_bytes() */
  EARN_ERR_CUDA = 4,        /* the CUDA runtime reported an error at launch */
  EARN_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (read back by earn_device_status) */
} earn_status_t;

typedef enum { EARN_F32 = 0, EARN_BF16 = 1 } earn_dtype_t;

#define EARN_PAGE_TOKENS 16 /* tokens per page of the compact register cache */

/* Model shape.  Section 3.3 notation: N layers, split k, n_h heads, d_a per-head dimension. */
typedef struct {
  int32_t n_layers;    /* N  > 0 */
  int32_t split_k;     /* k, 0 <= k <= N; k = N is a vanilla model, k = 0 compacts at the first layer */
  int32_t n_q_heads;   /* Hq, multiple of n_kv_heads */
  int32_t n_kv_heads;  /* Hkv */
  int32_t head_dim;    /* D in {64, 128} */
  int32_t dtype;       /* earn_dtype_t */
  float softmax_scale; /* 0 => 1/sqrt(head_dim), the scale of Eq. 3 */
} earn_model_t;

/* One batch of prompts, packed back to back (no padding tokens exist).  Eq. 5: every sequence is
 * [prefix registers; prompt; suffix registers]; its length L_b counts the registers. */
typedef struct {
  int32_t batch;                  /* B >= 0 */
  int32_t total_tokens;           /* sum of L_b */
  int32_t max_seqlen;             /* max L_b */
  const int32_t* cu_seqlens;      /* device [B+1], exclusive prefix sum of L_b */
  const int32_t* cu_seqlens_host; /* host   [B+1], the same values (used for validation and scheduling) */
  int32_t n_head_reg;             /* r_h >= 0 prefix registers = the first r_h positions of every sequence */
  int32_t n_tail_reg;             /* r_t >= 0 suffix registers = the last r_t positions; r_h + r_t <= every L_b */
} earn_batch_t;

/* KV cache of ONE register layer (l >= k) plus the generated-token cache of any layer.
 * Shared segment: the R = r_h + r_t register rows of every sequence in pages of EARN_PAGE_TOKENS
 * tokens, written once by earn_compact_kv and read by all beams of the sequence.
 * Private segment: the tokens generated so far, one slab per beam. */
typedef struct {
  void* k_shared;             /* device [n_pages, 16, Hkv, D]; may be NULL for a layer < k */
  void* v_shared;             /* device, same shape */
  const int32_t* block_table; /* device [B, pages_per_seq] page numbers, or NULL: page p of sequence b is b*pages_per_seq+p */
  int32_t pages_per_seq;      /* >= ceil(R / 16) */
  int32_t n_pages;            /* pages allocated in k_shared / v_shared (bounds the block table) */
  void* k_priv;               /* device [B*beams, max_new, Hkv, D] generated keys; row (j, t) is written at step t+1 by beam j
                                 (with priv_block_table: device [n_priv_pages, 16, Hkv, D], see below) */
  void* v_priv;               /* device, same shape */
  const int32_t* lineage;     /* device [B*beams, max_new] or NULL (identity): lineage[j][t] = slab holding token t of the
                                 history of beam j, maintained by earn_beam_reparent */
  int32_t beams;              /* W >= 1 */
  int32_t max_new;            /* T: capacity of the private segment in tokens */
  int32_t* reg_idx;           /* device [B, R] or NULL: earn_compact_kv writes the gathered source positions here */
  /* Optional page table of the private segment (NULL: the flat slabs above).  With a table, token t generated by beam j
   * lives in slot t % 16 of page priv_block_table[j * priv_pages_per_beam + t / 16] of k_priv / v_priv, so a beam costs
   * pages as it grows (one per 16 generated tokens) instead of a max_new-row slab up front.  The caller allocates a
   * beam's next page before the decode step that writes into it. */
  const int32_t* priv_block_table; /* device [B*beams, priv_pages_per_beam] or NULL */
  int32_t priv_pages_per_beam;     /* >= ceil(max_new / 16) */
  int32_t n_priv_pages;            /* pages allocated in k_priv / v_priv (bounds the table) */
} earn_cache_t;

/* Bytes of caller-provided scratch that cover every call below for this model, batch and beam
 * width (0 is never returned; the first 256 bytes hold the device status word).  Host only. */
size_t earn_workspace_bytes(const earn_model_t* model, const earn_batch_t* batch, int32_t beams);

/* Zeroes the workspace: the device status word and the split-decode tickets must start at zero.  Call once
 * after allocating the workspace and before the first call that uses it (asynchronous on `stream`).  A
 * workspace is used by one stream at a time: calls that overlap on the GPU must not share one. */
earn_status_t earn_workspace_init(void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* Synchronises `stream` and returns the device status word of the workspace: EARN_OK, or
 * EARN_ERR_TIMEOUT if a bounded wait inside a kernel ran out since earn_workspace_init. */
earn_status_t earn_device_status(const void* workspace, earn_stream_t stream);

/* Failure-path self-test (the paper has no counterpart): launches one small kernel that waits, with the bounded
 * wait the tensor-core kernels use, on a barrier nothing will ever complete.  After `limit_cycles` SM clocks
 * (1 .. 2e9, i.e. at most about a second) the wait gives up, the kernel writes EARN_ERR_TIMEOUT to the workspace
 * status word and returns normally; earn_device_status() then reports it and earn_workspace_init() clears it.
 * The context stays usable.  Errors: limit out of range -> INVALID_ARG; workspace NULL / too small -> WORKSPACE. */
earn_status_t earn_selftest_wait_timeout(void* workspace, size_t workspace_bytes, int64_t limit_cycles,
                                         earn_stream_t stream);

/* Step 1 — full causal attention of a layer l < k over every prompt token
 * (Section 3.2 "Full Computation Process"; Eq. 3 with the causal mask of a decoder-only model):
 *   O[i,h] = sum_{j<=i} softmax_j( Q[i,h].K[j,h/g] * scale ) V[j,h/g]   within each sequence, g = Hq/Hkv.
 * q,o: device [total_tokens, Hq, D]; k,v: device [total_tokens, Hkv, D] (read in place later by decode).
 * lse_or_null: device fp32 [Hq, total_tokens], natural-log softmax denominators, or NULL.
 * Errors: layer outside [0,k) -> INVALID_ARG. */
earn_status_t earn_prefill_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                const void* q, const void* k, const void* v, void* o, float* lse_or_null,
                                void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* Step 2 — keep only the register rows at a layer l >= k
 * (Section 3.2 "Register-Focused Process": X = [prefix; Prompt; suffix] -> X' = [prefix; suffix]).
 * For sequence b the source positions are idx_b = (0..r_h-1, L_b-r_t..L_b-1); row m of the compact cache
 * is a bit copy of row idx_b[m] of k and v.  If q_or_null is given, the same rows of q go to
 * q_reg_or_null (device [B, R, Hq, D]), ready for earn_register_attn.  cache->reg_idx (if not NULL)
 * receives idx.  Errors: layer outside [k,N), R > some L_b, page table too small -> INVALID_ARG. */
earn_status_t earn_compact_kv(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                              const void* k, const void* v, const void* q_or_null, void* q_reg_or_null,
                              const earn_cache_t* cache, earn_stream_t stream);

/* Projection of a layer l >= k from the hidden states (the paper's own statement of the register-focused process). */
typedef struct {
  int32_t d_model;        /* hidden size; a multiple of 64 */
  int32_t max_pos;        /* rows of the rotary tables; every prompt position must be below it */
  float   rms_eps;        /* epsilon of the RMS normalisation */
  int32_t x_is_compact;   /* 0: x holds every prompt token, [total_tokens, d_model];
                             1: x holds the register rows only, [B*R, d_model] (layers after the first register layer) */
  const float* rope_cos;  /* device fp32 [max_pos, D/2]: cos(pos * theta^(-2i/D)) */
  const float* rope_sin;  /* device fp32 [max_pos, D/2] */
} earn_proj_t;

/* Steps 2+ fused with the projection — Section 3.2 "Register-Focused Process", Eq. 2 restricted to X' = [prefix; suffix]:
 *   X_n = RMSNorm(X'[b,m]) * w_norm;   [Q' K' V'] = X_n W_qkv^T;   Q', K' rotated by the ORIGINAL position idx_b[m]
 * (rotary pairs (i, i + D/2)).  K', V' go to row m of sequence b's compact cache pages, Q' to q_reg (device [B, R, Hq, D]),
 * idx to cache->reg_idx if it is not NULL: the state earn_compact_kv leaves, without K/V of the other prompt tokens ever
 * being computed.  bf16 only, head_dim 128.
 * x: device bf16 (see x_is_compact); w_norm: device bf16 [d_model]; w_qkv: device bf16 [(Hq+2Hkv)*D, d_model], rows in the
 * order Q heads, K heads, V heads; x_norm_scratch: device bf16 [B*R, d_model], caller-owned, overwritten.
 * Arithmetic: fp32 sum of squares, X_n rounded to bf16, fp32 tensor-core accumulation, fp32 rotation, one rounding to bf16.
 * Errors: layer outside [k,N), d_model % 64 != 0, a prompt longer than max_pos -> INVALID_ARG; fp32 model or
 * head_dim != 128 -> UNSUPPORTED; workspace NULL / too small -> WORKSPACE. */
earn_status_t earn_register_qkv(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                const earn_proj_t* proj, const void* x, const void* w_norm, const void* w_qkv,
                                void* x_norm_scratch, const earn_cache_t* cache, void* q_reg,
                                void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* Step 3 — attention of a layer l >= k during prefill: causal attention among the R register tokens of
 * each sequence in the order [prefix; suffix] (Section 3.2: in layers l >= k only register and generated tokens
 * attend, by the training rule and by the inference rule above).  q_reg, o_reg: device [B, R, Hq, D]. */
earn_status_t earn_register_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                 const void* q_reg, const earn_cache_t* cache, void* o_reg,
                                 void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* Steps 2 and 3 in one launch (an additional call; the two above stay as they are): for a layer l >= k, read the register
 * rows of q, k, v straight from the packed prompt tensors (Section 3.2, X -> X' = [prefix; suffix]), write the K and V rows
 * into the compact cache pages and idx into cache->reg_idx exactly as earn_compact_kv does (bit copies), and compute the
 * causal attention among the R register tokens as earn_register_attn does: o_reg, device [B, R, Hq, D].  No gathered copy
 * of the queries is made.  bf16 with R <= 128 only; anything else -> EARN_ERR_UNSUPPORTED (use the two calls). */
earn_status_t earn_compact_register_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                         const void* q, const void* k, const void* v, const earn_cache_t* cache,
                                         void* o_reg, void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* Step 4 — one decode step of one layer (Eq. 4: append K_t, V_t, then attend over K_{1:t}, self included).
 * step is 1-based; beam j = b*W + w.  k_new/v_new (device [B*W, Hkv, D]) are stored at row (j, step-1) of the
 * private segment; q, o: device [B*W, Hq, D].  Keys seen by beam j:
 *   layer >= k : the R compact register rows of sequence b, then the step generated tokens of its lineage;
 *   layer <  k : all L_b prompt rows of sequence b read in place from k_full/v_full (device, packed like
 *                earn_prefill_attn's k and v; required), then the generated tokens.
 * For a layer < k of a batch with long, uneven prompts (longest >= 1024 tokens and more than 1.25 times the shortest,
 * at most 1024 sequences) one small extra kernel runs first: it writes, into the plan area of the workspace, the order
 * in which the main kernel takes the sequences (longest first).
 * Errors: step outside [1, max_new], missing k_full for a layer < k -> INVALID_ARG. */
earn_status_t earn_decode_attn(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t step,
                               const void* q, const void* k_new, const void* v_new,
                               const void* k_full_or_null, const void* v_full_or_null,
                               const earn_cache_t* cache, void* o,
                               void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* earn_decode_attn for callers that cannot allocate device memory (the paper has no counterpart: this is a
 * deployment variant of step 4, same arithmetic, same arguments minus the workspace).
 * Meant for hosts that hand a plug-in its inputs and outputs and nothing else -- a serving framework that owns
 * the whole memory pool, a latency-critical loop that cannot take cudaMalloc's device-wide synchronisation or
 * its failure under memory pressure.  The scratch memory (status block, split tickets, split partials) lives
 * in a fixed array of EARN_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library
 * holds that much until the process exits.  The call allocates nothing and frees nothing.
 *   - A batch whose earn_workspace_bytes() exceeds EARN_STATIC_SCRATCH_BYTES is rejected with
 *     EARN_ERR_WORKSPACE before anything is launched; use earn_decode_attn with your own workspace instead.
 *   - The first call on each device looks up the array's device address (that device must be current, as for
 *     every call); make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; each call clears
 *     the part that must start at zero on `stream` before its kernel.  Two calls that overlap on the GPU (different
 *     streams without an ordering between them) race on the array: serialise them.
 *   - The array's status block is cleared by every call and the caller holds no pointer to it, so earn_device_status
 *     cannot be used with this entry point (the decode kernels have no bounded waits to report).
 *   - The argument checks of earn_decode_attn run first, on the host; a rejected call has touched nothing. */
#define EARN_STATIC_SCRATCH_BYTES (8u << 20)
earn_status_t earn_decode_attn_static(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t step,
                                      const void* q, const void* k_new, const void* v_new,
                                      const void* k_full_or_null, const void* v_full_or_null,
                                      const earn_cache_t* cache, void* o, earn_stream_t stream);

/* Beam search bookkeeping between decode steps (Appendix A.3 uses beam search; the cache sharing is this
 * library's design): before step `step` (>= 2), beam j continues the history of beam parent[j] (an index in
 * [0,W) within its own sequence).  No K/V moves: lineage_out[j][t] = lineage_in[b*W+parent[j]][t] for
 * t < step-1 and lineage_out[j][step-1] = j.  lineage_in NULL means the identity table.  One table serves
 * all layers of a step.  lineage_in and lineage_out must not alias.  All pointers device. */
earn_status_t earn_beam_reparent(int32_t batch, int32_t beams, int32_t max_new, int32_t step,
                                 const int32_t* parent, const int32_t* lineage_in_or_null,
                                 int32_t* lineage_out, earn_stream_t stream);

/* Training-time attention (Section 3.2 "Training"; the loss of Eq. 7 is taken on the target identifier Y).  A training
 * sample is the sequence [prefix registers; prompt; suffix registers; Y] with the n_target tokens of Y teacher-forced at
 * its end; `batch` describes those sequences (every L_b counts the targets, L_b >= r_h + r_t + n_target).  The paper
 * changes one thing against ordinary finetuning: who takes part in the attention of a layer.
 *   layer <  k : every token (ordinary causal attention, Eq. 3).  q, o, d_o, dq: device [total_tokens, Hq, D];
 *                k, v, dk, dv: device [total_tokens, Hkv, D]; lse: device fp32 [Hq, total_tokens].
 *   layer >= k : only register and target tokens, P = r_h + r_t + n_target per sequence, in the order [prefix; suffix;
 *                targets] (the suffix registers and the targets are the last r_t + n_target rows of a sequence).  The
 *                prompt rows were removed from the hidden state at layer k, so the tensors hold the participating rows
 *                only: q, o, d_o, dq: device [B, P, Hq, D]; k, v, dk, dv: device [B, P, Hkv, D]; lse: fp32 [B, Hq, P];
 *                causal attention among them.  Removed tokens have no output and receive no gradient in these layers.
 * Forward writes o and lse (natural-log softmax denominators; required: the backward reads them).  Backward takes the
 * forward's inputs and outputs and the upstream gradient d_o and writes
 *   dV = P^T dO,   dS = P o (dO V^T - rowsum(dO o O)),   dQ = dS K * scale,   dK = dS^T Q * scale,
 * the query heads of a group adding into the kv head they share.  fp32 arithmetic, one rounding to the model dtype.
 * workspace: at least earn_train_workspace_bytes(model, batch) bytes, zeroed once by earn_workspace_init.
 * Errors: layer outside [0, N), n_target < 0, a sequence shorter than r_h + r_t + n_target, NULL or misaligned tensors
 * -> INVALID_ARG; workspace NULL / too small -> WORKSPACE. */
size_t earn_train_workspace_bytes(const earn_model_t* model, const earn_batch_t* batch);
earn_status_t earn_train_attn_fwd(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t n_target,
                                  const void* q, const void* k, const void* v, void* o, float* lse,
                                  void* workspace, size_t workspace_bytes, earn_stream_t stream);
earn_status_t earn_train_attn_bwd(const earn_model_t* model, const earn_batch_t* batch, int32_t layer, int32_t n_target,
                                  const void* q, const void* k, const void* v, const void* o, const float* lse,
                                  const void* d_o, void* dq, void* dk, void* dv,
                                  void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* Beam selection between decode steps (Appendix A.3: identifiers are generated by beam search, beam size 20; the paper
 * gives the beam size only, the rule is that of ordinary beam search).  For every sequence, of the n_live * vocab
 * continuations (beam w < n_live, token v), scored beam_scores[b*W + w] + logprobs[b*W + w][v] in fp32, the W best
 * survive: higher score first, equal scores by increasing flat index w * vocab + v.  Slot i of the sequence receives the
 * i-th best: parent[b*W + i] = w (ready for earn_beam_reparent), token[b*W + i] = v, new_scores[b*W + i] = its score.
 * n_live = 1 at the first step (all beams hold the same history), W afterwards.  A decode step is then
 * earn_beam_topk -> earn_beam_reparent -> earn_decode_attn per layer, with no host round trip.
 * logprobs: device fp32 [B*W, vocab], no NaN (-inf marks a forbidden token); beam_scores: device fp32 [B*W] or NULL
 * (zeros); parent, token: device int32 [B*W]; new_scores: device fp32 [B*W], must not alias beam_scores.
 * workspace: device, at least earn_beam_topk_workspace_bytes(batch, beams, vocab) bytes, 16-byte aligned; no need to
 * initialise it.  Errors: beams outside [1, 32], n_live outside [1, beams], n_live * vocab < beams -> INVALID_ARG;
 * beams * vocab beyond 2^31 - 257 (flat candidate indices are 32-bit) -> UNSUPPORTED; workspace NULL / too small
 * -> WORKSPACE. */
size_t earn_beam_topk_workspace_bytes(int32_t batch, int32_t beams, int32_t vocab);
earn_status_t earn_beam_topk(int32_t batch, int32_t beams, int32_t n_live, int32_t vocab, const float* logprobs,
                             const float* beam_scores_or_null, int32_t* parent, int32_t* token, float* new_scores,
                             void* workspace, size_t workspace_bytes, earn_stream_t stream);

/* Number of kernels this library has launched in this process so far (host counter, all streams). */
uint64_t earn_launch_count(void);

const char* earn_status_string(earn_status_t status);
int32_t earn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* EARN_H_ */
