/*
 * ippd.h -- C ABI of the B200 (sm_100a) IPPD decode-attention library.
 *
 * Intra-Prompt Parallel Decoding packs the Q questions that share one context
 * into one prompt; at every decode step each still-unfinished question emits one
 * token.  The query of that token is rotated (RoPE) to its VIRTUAL position --
 * the position it would have had if its (context, question, answer-so-far)
 * triplet had been prompted alone -- and attends to the prompt's shared context
 * K/V plus its own private branch (its question tokens and its answer so far),
 * never to another question's tokens.
 *
 * Conventions
 *   - Every call returns IPPD_OK (0) or a negative IPPD_ERR_* code; nothing throws
 *     across the boundary.  ippd_last_error() gives a thread-local message.
 *   - "host" pointers are ordinary CPU memory read during the call.  "device"
 *     pointers are CUDA device memory owned by the CALLER (for example torch
 *     allocations); they must stay alive until the stream has drained.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Kernels are enqueued on it; no call blocks except ippd_bind_cache,
 *     ippd_poll_status, ippd_export_mask, ippd_decode_step_host,
 *     ippd_host_steps_wait and ippd_destroy_layout.
 *   - There is no CPU fallback: a call that needs the GPU fails with IPPD_ERR_CUDA
 *     when no device is usable.
 *   - B prompts; prompt b has a context of L_b tokens (instruction + context of
 *     the paper merged, Sec. 4.1) and Q_b questions; global question id k in
 *     [0, NQ); n_k question tokens; decode step s = 0,1,.. is the paper's t = s+1.
 */
#ifndef IPPD_H_
#define IPPD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define IPPD_OK 0
#define IPPD_ERR_INVALID_ARG (-1)
#define IPPD_ERR_OOM (-2)
#define IPPD_ERR_CAPACITY (-3)
#define IPPD_ERR_NOT_BOUND (-4)
#define IPPD_ERR_CUDA (-5)
#define IPPD_ERR_TIMEOUT (-6)

#define IPPD_BF16 0
#define IPPD_F32 1

/* tokens per K/V tile of the cache; branch_align must be a multiple of it */
#define IPPD_TILE_TOKENS 128

/* `kind` of ippd_append_kv */
#define IPPD_APPEND_CONTEXT 0
#define IPPD_APPEND_QUESTION 1
#define IPPD_APPEND_STEP 2
#define IPPD_APPEND_SHARED 3
#define IPPD_APPEND_HEADER 4

/* keys of ippd_set_option */
#define IPPD_OPT_KERNEL 1          /* 0 = auto, 1 = mma.sync path, 2 = tcgen05 path */
#define IPPD_OPT_LAYERS_PER_CALL 2 /* layer_count the caller will pass to ippd_decode_attention (sizes the split) */
#define IPPD_OPT_TILES_PER_SPLIT 3 /* 0 = auto; else force this many key tiles per split-KV unit */
#define IPPD_OPT_WAIT_LIMIT_US 4   /* bound of every device-side wait; default 2000000; 0 = never wait
                                      (a wait on a phase not yet complete fails at once: IPPD_ERR_TIMEOUT) */
#define IPPD_OPT_PROFILE 5         /* N > 0: bracket the attention, merge and STEP-append kernels of every N-th step
                                      (counted from this call: steps 0, N, 2N, ...) with CUDA events; 0: off */
#define IPPD_OPT_KV_DTYPE 6        /* element type of the cache: IPPD_KV_BF16 (default) or IPPD_KV_E4M3.  Only before
                                      ippd_bind_cache (ippd_cache_bytes follows it); tensor-core path only.
                                      IPPD_KV_E4M3, a bandwidth variant that is not part of the paper: the rotated
                                      key and the value are stored as e4m3 numbers (1-4-3 bits, bias 7, largest
                                      magnitude 448, round to nearest even, saturating; no scale factor), half the
                                      bytes per token.  Scores and outputs are those of exact attention over the
                                      stored numbers, to the same tolerance as the bf16 cache: inside the kernel the
                                      query rows and the probabilities enter the 8-bit tensor-core products as sums
                                      of two e4m3 terms.  All entry points work unchanged on such a cache. */
#define IPPD_KV_BF16 0
#define IPPD_KV_E4M3 1

typedef struct {
  int32_t n_layers;
  int32_t n_q_heads;   /* Hq */
  int32_t n_kv_heads;  /* Hkv; Hq % Hkv == 0 and G = Hq/Hkv in {1,2,4,8,16} */
  int32_t head_dim;    /* D in {64, 128} */
  double rope_theta;   /* RoPE base; angle of pair (i, i+D/2) at position p is p * theta^(-2i/D) */
  int32_t branch_align; /* branch capacity granularity in tokens; multiple of IPPD_TILE_TOKENS */
  int32_t out_dtype;   /* IPPD_BF16 or IPPD_F32 */
} ippd_geometry_t;

typedef struct ippd_layout ippd_layout_t; /* opaque, library-owned */

/* Host views of the integer tables; valid until ippd_destroy_layout. */
typedef struct {
  const int32_t* q_begin;      /* [B+1] exclusive prefix sum of Q_b */
  const int32_t* prompt_of;    /* [NQ] prompt of each question */
  const int32_t* q_len;        /* [NQ] */
  const int32_t* ctx_len;      /* [B] */
  const int64_t* branch_off;   /* [NQ+1] first cache slot (in tokens) of each branch */
  const int32_t* ctx_tile_off; /* [B+1] first context tile of each prompt */
  const int64_t* hdr_begin;    /* [B+1] first header token of each prompt in the hdr_* arrays */
  const int32_t* hdr_pos_virt; /* [n_header_tokens] virtual position id */
  const int32_t* hdr_ctx_id;   /* context id (1-based prompt id) */
  const int32_t* hdr_qtn_id;   /* question id (global, 1-based; 0 for context tokens) */
  int32_t n_prompts, n_questions;
  int64_t n_header_tokens;
  int64_t n_branch_slots;      /* = branch_off[NQ] */
  int64_t n_tiles;             /* shared + context + branch tiles of the whole cache, per layer and KV head */
  int32_t n_shared_tokens;     /* length of the instruction shared by all prompts (0 without one); the hdr_* arrays
                                  start with its tokens (context id 0), hdr_begin[0] = n_shared_tokens */
} ippd_tables_t;

/*
 * ippd_build_layout -- virtual position ids, context/question ids, per-question
 * branch offsets and the ragged prompt/question tables (paper Sec. 4.1: stacked
 * header and the virtual-position equations; App. A.1: absolute positions, read
 * as per-question branch offsets in the fixed question order).
 *   pos_virt(context token i of prompt b)      = i
 *   pos_virt(token j of question k, prompt b)  = L_b + j
 *   pos_virt(answer token fed at step s)       = L_b + n_k + s       (cache slot branch_off[k] + n_k + s)
 *   capacity(k) = round_up(n_k + max_new[k], branch_align)
 * All arguments are host arrays, read during the call: ctx_len[B] >= 0, q_count[B] >= 1,
 * q_len[sum Q] >= 1, max_new[sum Q] >= 1.  Host-only: no CUDA call is made.  *out is
 * owned by the library; free it with ippd_destroy_layout.  Errors: IPPD_ERR_INVALID_ARG
 * (bad geometry, NULL, a length out of range, a position >= INT32_MAX), IPPD_ERR_OOM.
 */
int ippd_build_layout(const ippd_geometry_t* geom, int32_t n_prompts, const int32_t* ctx_len,
                      const int32_t* q_count, const int32_t* q_len, const int32_t* max_new,
                      ippd_layout_t** out);

/*
 * ippd_build_layout_shared -- ippd_build_layout for a batch whose prompts all start with the same
 * instruction p of `shared_len` tokens (paper Sec. 4.1: stacked header [p, c_1, x_11, .., c_2, ..], p
 * carries context id 0 and is attended by every token; Sec. 4.4: the instruction's K/V is kept once
 * and reused by all stacked prompts of the batch).  Three levels of sharing: p by every question of
 * the batch, context c_b by the questions of prompt b, a branch by its own question only.
 *   pos_virt(token i of p)                     = i                      (cache tiles 0 .. ceil(shared_len/128)-1)
 *   pos_virt(context token i of prompt b)      = shared_len + i
 *   pos_virt(token j of question k, prompt b)  = shared_len + L_b + j
 *   pos_virt(answer token fed at step s)       = shared_len + L_b + n_k + s
 * p's K/V is appended once with ippd_append_kv(IPPD_APPEND_SHARED) and stored once; every row block's key
 * sequence starts with p's tiles (tensor-core path only).  shared_len = 0 is ippd_build_layout.
 */
int ippd_build_layout_shared(const ippd_geometry_t* geom, int32_t shared_len, int32_t n_prompts,
                             const int32_t* ctx_len, const int32_t* q_count, const int32_t* q_len,
                             const int32_t* max_new, ippd_layout_t** out);

/* Host views of the tables built above, for bit-exact comparison.  Host-only. */
int ippd_layout_tables(const ippd_layout_t* layout, ippd_tables_t* out);

/* Bytes and alignment of the K/V cache the caller must allocate on the device
 * (all layers; K and V; bf16, or one byte per element after IPPD_OPT_KV_DTYPE = IPPD_KV_E4M3).  Host-only. */
int ippd_cache_bytes(const ippd_layout_t* layout, size_t* bytes, size_t* align);

/*
 * ippd_bind_cache -- hand the caller-owned device cache to the layout, mirror the
 * integer tables to the device and build the fp32 RoPE cos/sin table (angles
 * evaluated in fp64).  The library allocates only its own small tables here.
 * The cache is zero-filled: from then on it must only be written through ippd_append_kv
 * with finite values, because key/value rows past the valid tokens of a 128-row tile are
 * still multiplied (by probability zero) and must therefore be finite.  Synchronises `stream`.
 * Errors: IPPD_ERR_INVALID_ARG (too small / misaligned), IPPD_ERR_CUDA, IPPD_ERR_OOM.
 */
int ippd_bind_cache(ippd_layout_t* layout, void* dev_cache, size_t bytes, void* stream);

/* Tuning knobs (see IPPD_OPT_*).  Host-only.  IPPD_ERR_INVALID_ARG on an unknown key or value. */
int ippd_set_option(ippd_layout_t* layout, int32_t key, int64_t value);

/*
 * ippd_begin_step -- declare which questions take part in the next decode step
 * (paper Sec. 4.2, last paragraph: one token per unfinished answer per step;
 * finished answers are no longer appended).  active_q[A]: strictly increasing
 * global question ids (host).  answer_idx[A]: the step index s of each (host);
 * the token fed is answer token y_{s+1} at virtual position L_b + n_k + s.
 * Builds the step's work list (row blocks, key tiles, packed branch pieces) on the
 * host and stages it in a pinned slot; nothing is enqueued here.  The first
 * ippd_append_kv(STEP) / ippd_decode_attention call that follows moves the
 * descriptor to the device on ITS stream (inside its own kernel where it can), and
 * every later call of the step, for any layer, reuses it.  `stream` is only
 * remembered as the stream ippd_poll_status waits on.  A == 0 is allowed (the step
 * is then empty).  The descriptor always fits its staging slot for any step the
 * layout admits (see ippd_step_descriptor_bytes).  Errors: IPPD_ERR_INVALID_ARG,
 * IPPD_ERR_CAPACITY (answer_idx >= max_new), IPPD_ERR_NOT_BOUND, IPPD_ERR_CUDA.
 */
int ippd_begin_step(ippd_layout_t* layout, const int32_t* active_q, const int32_t* answer_idx,
                    int32_t n_active, void* stream);

/* Host-only: the size in bytes of the descriptor ippd_begin_step would stage for this
 * step (*bytes) and the capacity of a staging slot of this layout (*capacity, a bound over
 * every admissible step).  Same argument checks as ippd_begin_step; needs no bound cache. */
int ippd_step_descriptor_bytes(const ippd_layout_t* layout, const int32_t* active_q,
                               const int32_t* answer_idx, int32_t n_active, size_t* bytes,
                               size_t* capacity);

/*
 * ippd_append_kv -- rotate raw keys to their virtual positions (RoPE, fp32 math on an
 * fp64-built table, result rounded to bf16) and store K and V into the cache
 * (paper Sec. 4.2, last paragraph: the token appended at each step carries its virtual position).
 *   kind SHARED  : ids ignored; tokens = the shared instruction's tokens (ippd_build_layout_shared), position i.
 *   kind HEADER  : ids ignored; tokens = the whole stacked header in the order of the hdr_* tables (the shared
 *                  instruction, then per prompt its context tokens and its questions' tokens), each at its
 *                  virtual position: the whole prefill stand-in in one call.
 *   kind CONTEXT : ids[n_ids] = prompt ids (host); tokens = all context tokens of those
 *                  prompts, in id order; token i of prompt b gets position shared_len + i.
 *   kind QUESTION: ids[n_ids] = global question ids (host); tokens = their question
 *                  tokens in id order; token j gets position L_b + j, slot j of the branch.
 *   kind STEP    : ids ignored; one token per question of the last ippd_begin_step, in
 *                  that order, at position L_b + n_k + s, slot n_k + s.
 * k_raw, v_raw: device bf16 [layer_count, tokens, Hkv, D], pre-RoPE.  Layers
 * layer_begin .. layer_begin+layer_count-1 are written.  Appending slot t of a branch
 * does not touch any other slot; re-running a step rewrites the same slots.
 * Errors: IPPD_ERR_INVALID_ARG, IPPD_ERR_NOT_BOUND, IPPD_ERR_CUDA.
 */
int ippd_append_kv(ippd_layout_t* layout, int32_t layer_begin, int32_t layer_count, int32_t kind,
                   const int32_t* ids, int32_t n_ids, const void* k_raw, const void* v_raw,
                   void* stream);

/* Bytes of device scratch ippd_decode_attention needs for `layer_count` layers with the
 * step declared last (an upper bound valid for ANY step of this layout when called before
 * the first ippd_begin_step).  Host-only. */
int ippd_workspace_bytes(const ippd_layout_t* layout, int32_t layer_count, size_t* bytes);

/*
 * ippd_decode_attention -- the per-step IPPD attention (paper Sec. 4.1 mask, Sec. 4.2
 * equivalence, Sec. 4.3 / App. A.2 reuse of the shared context across the M_j queries):
 * for every question of the last ippd_begin_step and every query head,
 *   out = softmax(q~ K~^T / sqrt(D)) V   over { context of its prompt } U { its own
 *   branch slots 0 .. n_k + s }            (the token appended for step s included),
 * with q~ = RoPE(q_raw, L_b + n_k + s).  The mask is realised structurally: context
 * tiles are streamed once per (prompt, KV head) for all its query rows, branch tiles
 * only for their own question, and the partial results are merged by log-sum-exp.
 * q_raw: device bf16 [layer_count, A, Hq, D] (pre-RoPE, A questions in begin_step
 * order).  out: device [layer_count, A, Hq, D] in geom.out_dtype.  workspace: device
 * scratch of at least ippd_workspace_bytes (256-byte aligned); contents undefined
 * afterwards.  Errors: IPPD_ERR_INVALID_ARG, IPPD_ERR_NOT_BOUND, IPPD_ERR_CUDA.
 * Device-side waits are bounded; a wait that runs out sets the device error word
 * (see ippd_poll_status) and the kernel returns.
 */
int ippd_decode_attention(ippd_layout_t* layout, int32_t layer_begin, int32_t layer_count,
                          const void* q_raw, void* out, void* workspace, size_t workspace_bytes,
                          void* stream);

/*
 * ippd_decode_step -- ippd_append_kv(STEP) and ippd_decode_attention in ONE launch (paper Sec. 4.2,
 * last paragraph: the step's tokens are appended with their virtual positions and attended to in
 * the same step).  k_raw, v_raw: device bf16 [layer_count, A, Hkv, D], pre-RoPE, the step's tokens in
 * begin_step order; the other arguments as for ippd_decode_attention.  Inside the attention kernel
 * one warp per CTA rotates the keys and writes K~ and V into their branch slots just ahead of the
 * CTA's own loads of those slots, so the cache ends up exactly as after ippd_append_kv(STEP) and the
 * outputs are those of ippd_decode_attention after it.  Re-running the call rewrites the same slots.
 * (With IPPD_OPT_KERNEL = 1 the call runs the append kernel and the attention kernel one after the
 * other.)  Errors as for the two calls it replaces.
 */
int ippd_decode_step(ippd_layout_t* layout, int32_t layer_begin, int32_t layer_count, const void* q_raw,
                     const void* k_raw, const void* v_raw, void* out, void* workspace,
                     size_t workspace_bytes, void* stream);

/*
 * ippd_prefill_attention -- the prefill of the stacked header under the IPPD mask (paper Sec. 4: the
 * stacked prompt is prefilled once; Sec. 4.1: header rows of the mask; App. A.2: dim(q) of the prefill
 * is the whole header).  Appends the header's K/V (as ippd_append_kv(HEADER)) and returns the
 * attention output of EVERY header token:
 *   instruction token i   sees instruction tokens 0..i;
 *   context token i of b  sees the instruction and context tokens 0..i of its own prompt;
 *   token j of question k sees the instruction, the context of its prompt and tokens 0..j of its question
 * -- each row is the row of its own standalone causal prompt (Sec. 4.2).  q_raw: device bf16
 * [layer_count, n_header_tokens, Hq, D]; k_raw, v_raw: [layer_count, n_header_tokens, Hkv, D] (pre-RoPE, header
 * order of the hdr_* tables); out: [layer_count, n_header_tokens, Hq, D] in geom.out_dtype.  The same
 * tensor-core kernel as the decode step runs it: 128-row blocks of consecutive header tokens stream
 * the key tiles up to their own position, the diagonal tiles under per-row windows; question tokens
 * see their question's prefix through packed branch pieces.  workspace as for ippd_decode_attention with
 * layer_count layers.  Invalidates the step declared by ippd_begin_step.  Tensor-core path only.  The
 * call allocates a device buffer for its work list (kept by the layout, reused by later calls).
 * Errors: IPPD_ERR_INVALID_ARG, IPPD_ERR_NOT_BOUND, IPPD_ERR_OOM, IPPD_ERR_CUDA.
 */
int ippd_prefill_attention(ippd_layout_t* layout, int32_t layer_begin, int32_t layer_count, const void* q_raw,
                           const void* k_raw, const void* v_raw, void* out, void* workspace,
                           size_t workspace_bytes, void* stream);

/*
 * ippd_decode_step_grouped -- ippd_decode_step for ALL layers of the step, `layers_per_call` layers per
 * launch, back to back on `stream`: q_raw [n_layers, A, Hq, D], k_raw / v_raw [n_layers, A, Hkv, D], out
 * [n_layers, A, Hq, D].  layers_per_call = 1 is the launch pattern of a model whose layer l+1 needs layer
 * l's output (without the model's own work between the launches); = n_layers is one ippd_decode_step.
 * The workspace must satisfy ippd_workspace_bytes(layers_per_call); set IPPD_OPT_LAYERS_PER_CALL to the
 * same value before ippd_begin_step.  Errors as ippd_decode_step.
 */
int ippd_decode_step_grouped(ippd_layout_t* layout, int32_t layers_per_call, const void* q_raw,
                             const void* k_raw, const void* v_raw, void* out, void* workspace,
                             size_t workspace_bytes, void* stream);

/*
 * ippd_decode_step_host -- one whole decode step from HOST buffers: copies q_raw, k_raw,
 * v_raw (host, pinned or pageable; shapes as above with layer_count = n_layers) into the
 * caller's device staging buffers, runs ippd_begin_step + ippd_decode_step over all layers,
 * copies `out` back to the host and waits for
 * the stream.  dev_stage must hold the three inputs and the output back to back
 * (ippd_step_stage_bytes).  Same errors as the calls it wraps.
 */
int ippd_decode_step_host(ippd_layout_t* layout, const int32_t* active_q, const int32_t* answer_idx,
                          int32_t n_active, const void* host_q_raw, const void* host_k_raw,
                          const void* host_v_raw, void* host_out, void* dev_stage, size_t dev_stage_bytes,
                          void* workspace, size_t workspace_bytes, void* stream);
int ippd_step_stage_bytes(const ippd_layout_t* layout, int32_t n_active, size_t* bytes);

/*
 * ippd_decode_step_host_async -- ippd_decode_step_host without the wait, so that consecutive
 * steps pipeline: the host-to-device copies of step n+1 and the device-to-host copy of step n-1
 * run on two copy streams owned by the layout while the kernels of step n run on `stream`
 * (events order the three; the K/V cache dependency between steps stays on `stream`).
 * dev_stage must hold TWO slots of ippd_step_stage_bytes (for the largest n_active used), 256-byte
 * aligned; calls alternate between them.  The host buffers of a call (pinned memory, or the copies
 * are not asynchronous) must stay valid and untouched until ippd_host_steps_wait returns; the
 * result of a call is in host_out only after that.  All calls of one pipeline use the same stream.
 * The first call creates the streams and events.  Same errors as ippd_decode_step_host.
 *
 * ippd_host_steps_wait -- blocks until every step enqueued so far, its copy-out included, is done.
 */
int ippd_decode_step_host_async(ippd_layout_t* layout, const int32_t* active_q, const int32_t* answer_idx,
                                int32_t n_active, const void* host_q_raw, const void* host_k_raw,
                                const void* host_v_raw, void* host_out, void* dev_stage,
                                size_t dev_stage_bytes, void* workspace, size_t workspace_bytes, void* stream);
int ippd_host_steps_wait(ippd_layout_t* layout, void* stream);

/*
 * ippd_export_mask -- test aid: the dense IPPD mask M_fin (paper Sec. 4.1 mask equations)
 * of ONE prompt's stacked sequence, written by a device kernel that evaluates the library's
 * visibility rule (context of the own prompt; own branch slots up to the own slot) on the
 * device tables.  It restates that rule; it does not replay the tiles and packed branch
 * pieces the attention kernels walk.  Sequence order: context tokens, question blocks,
 * then answer tokens step by step (for t = 0.. : every question of the prompt, in
 * order, with n_answer[k] > t).  n_answer[Q_b] (host) gives how many answer tokens each
 * question of the prompt has.  host_out: [n, n] bytes (1 = attend), row-major, n
 * returned in *n_tokens; pass host_out = NULL to query n only.  Blocks.
 */
int ippd_export_mask(ippd_layout_t* layout, int32_t prompt, const int32_t* n_answer,
                     uint8_t* host_out, int64_t* n_tokens);

/* Waits for the stream last used with this layout and returns the device error word
 * (0 = none; bit 0 = a bounded wait ran out: IPPD_ERR_TIMEOUT; bit 1 = an id or slot was out of
 * range: IPPD_ERR_INVALID_ARG; bit 2 = ippd_append_kv was handed a NaN or an infinity:
 * IPPD_ERR_INVALID_ARG -- the value was stored, and because a key/value row shares its 128-row
 * tile with other questions' rows, outputs of OTHER questions may be non-finite too).  The word is cleared once reported; the outputs of the launches
 * since the previous poll are then undefined, the cache and the layout stay usable. */
int ippd_poll_status(ippd_layout_t* layout, int32_t* device_error_word);

/*
 * ippd_profile_read -- with IPPD_OPT_PROFILE = N, the ippd_decode_attention and ippd_append_kv(STEP)
 * calls of every N-th step (the steps declared by ippd_begin_step are counted from the moment the
 * option is set; steps 0, N, 2N, ... are measured) record CUDA events on the caller's stream right
 * before and after each of their kernels.  Each pair of events costs a few microseconds of stream
 * time, so N > 1 keeps a timed loop close to its unmeasured speed.  This call
 * waits for them, returns the summed device time of each kernel kind (milliseconds) and the number of
 * attention launches measured since the last read, and clears the record.  Any output may be NULL.
 */
int ippd_profile_read(ippd_layout_t* layout, double* attention_ms, double* merge_ms, double* append_ms,
                      int64_t* n_attention_launches);

/*
 * ippd_decode_attention_static -- ippd_decode_attention for callers that cannot allocate.
 * (The paper has no counterpart: this entry point exists for the library's users only.)
 *
 * Some callers may not call cudaMalloc at the point where they run attention: code running
 * inside a memory-budgeted serving loop whose allocator has already handed out all of the
 * device memory, a plug-in that is forbidden to allocate after start-up, or a latency-critical
 * loop that must not risk the implicit device synchronisation of an allocation.  They cannot
 * provide the split-KV workspace either.  This variant therefore keeps the partial results
 * (O, m, l of every split-KV unit) in a fixed array that lives inside the library's device image:
 * IPPD_STATIC_SCRATCH_BYTES bytes on EVERY GPU that loads the library, held until the process
 * exits.  Inputs and outputs are still the caller's: q_raw and out as for ippd_decode_attention.
 *
 * - It allocates nothing: no cudaMalloc / cudaFree, no allocating library call, no event creation
 *   (IPPD_OPT_PROFILE is ignored here).
 * - The step declared by ippd_begin_step must need at most IPPD_STATIC_SCRATCH_BYTES of scratch
 *   for `layer_count` layers (rows x (D+2) floats per split-KV unit, KV head and layer); otherwise
 *   the call fails with IPPD_ERR_CAPACITY and a message giving both numbers -- pass fewer layers
 *   per call or raise IPPD_OPT_TILES_PER_SPLIT.
 * - The first call on a device looks up the device address of the array (once per device, with that
 *   device current).  Make that first call before any stream capture begins.  The device current at
 *   the call must be the one the cache was bound on (IPPD_ERR_INVALID_ARG otherwise).
 * - All calls, from every layout and stream of the process, share the one array, which keeps
 *   whatever the last call left in it.  Nothing in it has to start at zero: every value the merge
 *   reads is written earlier in the same call.  Two calls that overlap on the GPU (different
 *   streams, no ordering between them) race on it; order them.
 * Errors otherwise as ippd_decode_attention.
 */
#define IPPD_STATIC_SCRATCH_BYTES (64u << 20)
int ippd_decode_attention_static(ippd_layout_t* layout, int32_t layer_begin, int32_t layer_count,
                                 const void* q_raw, void* out, void* stream);

/*
 * ippd_read_probe -- measuring aid: enqueues a kernel that streams the key/value tiles of the step
 * declared last, for `layer_count` layers, through the same bulk-copy ring, slices and grid as the
 * tensor-core attention kernel and discards them (no tensor-core or softmax work, nothing written).
 * Timed with events by the caller, it gives the read bandwidth attainable with the attention
 * kernel's own access pattern.  Errors: IPPD_ERR_INVALID_ARG, IPPD_ERR_NOT_BOUND, IPPD_ERR_CUDA.
 */
int ippd_read_probe(ippd_layout_t* layout, int32_t layer_begin, int32_t layer_count, void* stream);

/* Host time (microseconds, summed) spent inside ippd_begin_step -- planning the step, packing the
 * branch tiles, staging the descriptor; waiting for a free staging slot while the device is behind
 * is not counted -- and the number of steps, since the last read.  Host-only. */
int ippd_host_time_read(ippd_layout_t* layout, double* begin_step_us, int64_t* n_steps);

/* Number of kernels this library has launched through this layout since it was built. */
int64_t ippd_launch_count(const ippd_layout_t* layout);

const char* ippd_last_error(void);
void ippd_destroy_layout(ippd_layout_t* layout);

#ifdef __cplusplus
}
#endif
#endif /* IPPD_H_ */
