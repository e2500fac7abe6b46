/*
 * alora.h — C ABI of the B200 (sm_100a) Activated-LoRA layer library.
 *
 * What the library computes, per decoder layer, for a ragged batch of NEW tokens that sit on top of
 * per-request KV caches already filled by the base model:
 *
 *   1. gated fused q/k/v projection (Eq. 2 + Eq. 5 of the aLoRA paper):
 *          y_t = W x_t + [p_t >= a_req] * s_k * B_k (A_k x_t)       per q / k / v block
 *      p_t is the token's 0-based position in its sequence, a_req the request's activation offset
 *      (the paper's t_invoke - 1), k the request's adapter (-1 = base model, no delta at all);
 *   2. KV append: the new k/v rows go to their slots of a paged cache; bytes that belong to earlier
 *      positions are never written (Prop. 2, proof step 4: only O(T_new) new cache entries);
 *   3. causal grouped-query softmax attention of the new queries over cached ++ new rows
 *      (Eq. 1, per-token form Eq. 3; a token attends keys 0..p_t, itself included).
 *
 * A decode step is the same with one new token per request (Prop. 1, second sentence); the
 * full-LoRA entry is Eq. 4 (the delta on every token), i.e. what a conventional LoRA must do when
 * it cannot reuse the base cache.
 *
 * Conventions
 *   - Every pointer named d_* is DEVICE memory on the context's device; h_* is HOST memory.
 *     All tensors are dense row-major, element type = the context's dtype (bf16 or fp32), index
 *     arrays int32.  Buffers are caller-owned and only borrowed for the duration of the call
 *     (of the enqueued work, for asynchronous calls) unless stated otherwise.
 *   - Shapes: H hidden; Hq, Hkv heads; hd head_dim; Nq = Hq*hd; Nkv = Hkv*hd; N = Nq + 2*Nkv.
 *     Fused rows are [ q heads | k heads | v heads ]; query head h reads KV head h / (Hq/Hkv).
 *     Weights are output-major: W[N][H] (y = W x), A[r][H], B[out][r].
 *   - Ragged batch: T new tokens of R requests, request r owns rows query_start_loc[r] ..
 *     query_start_loc[r+1]-1, whose positions must be consecutive and end at seq_lens[r]-1.
 *   - Paged cache of one layer: pool[num_pages][2][Hkv][page_size][hd] (K plane, then V plane).
 *     Position p of request r lives in page block_tables[r][p / page_size], row p % page_size.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work is enqueued and the
 *     call returns; nothing synchronises unless stated.  Most kernels are launched with programmatic
 *     stream serialization: their set-up may run under the tail of the preceding kernel of the stream,
 *     but they read and write the call's buffers only after everything enqueued earlier has completed.
 *   - Every call returns an alora_status.  Host-side argument errors are detected before anything
 *     is launched.  Device-side findings (page id out of range, inconsistent positions, a bounded
 *     wait that ran out) are recorded in a status word readable with alora_get_status after the
 *     stream has been synchronised; a kernel that finds one skips the offending access, it never
 *     traps.  There is no CPU fallback: without a CUDA device every compute call fails.
 */
#ifndef ALORA_H
#define ALORA_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct alora_ctx alora_ctx;

typedef enum alora_status {
    ALORA_OK = 0,
    ALORA_ERR_INVALID_ARG = 1,   /* null pointer, negative size, misaligned pointer, T > 0 with R == 0 */
    ALORA_ERR_UNSUPPORTED = 2,   /* shape or dtype the kernels are not built for               */
    ALORA_ERR_CAPACITY = 3,      /* T, R, rank or adapter id beyond what alora_create was told */
    ALORA_ERR_NO_WEIGHTS = 4,    /* layer weights never set (return value); or, as a device finding,
                                    a row whose gate is open names an adapter that was never
                                    registered on the layer: that row gets the base projection  */
    ALORA_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed (see alora_last_cuda_error) */
    ALORA_ERR_BAD_BATCH = 6,     /* batch metadata inconsistent (host validation or device check) */
    ALORA_ERR_PAGE_RANGE = 7,    /* a block-table entry is outside [0, num_pages)              */
    ALORA_ERR_TIMEOUT = 8,       /* a bounded in-kernel wait expired                            */
    ALORA_ERR_NO_DEVICE = 9      /* no usable CUDA device                                       */
} alora_status;

typedef enum alora_dtype { ALORA_DTYPE_BF16 = 0, ALORA_DTYPE_FP32 = 1 } alora_dtype;

/* Execution mode of a layer / stack call. */
typedef enum alora_mode {
    ALORA_MODE_ALORA = 0,      /* Eq. 5: delta on rows with p >= a_req                            */
    ALORA_MODE_FULL_LORA = 1,  /* Eq. 4: delta on every row of a request that has an adapter      */
    ALORA_MODE_BASE = 2        /* Eq. 2: adapters ignored                                         */
} alora_mode;

typedef struct alora_config {
    int32_t hidden;        /* H                                                                   */
    int32_t n_q_heads;     /* Hq                                                                  */
    int32_t n_kv_heads;    /* Hkv, must divide Hq                                                 */
    int32_t head_dim;      /* hd                                                                  */
    int32_t page_size;     /* tokens per KV page                                                  */
    int32_t n_layers;      /* layers addressable by the per-layer calls                           */
    int32_t intermediate;  /* MLP width (0 if the stack entry is not used)                        */
    int32_t max_adapters;  /* adapter ids are 0 .. max_adapters-1                                 */
    int32_t max_rank;      /* largest adapter rank (<= 64)                                        */
    int32_t dtype;         /* alora_dtype                                                         */
    int32_t device;        /* CUDA device ordinal                                                 */
    int32_t max_tokens;    /* largest T of any call; sizes the context's workspaces               */
    int32_t max_requests;  /* largest R of any call                                               */
    float rms_eps;         /* RMSNorm epsilon (stack entry)                                       */
    float rope_theta;      /* 0 (default): no positional rotation, as in the method's equations;
                              > 0: rotary embedding with this base, see below                      */
    float softmax_scale;   /* 0 => 1/sqrt(head_dim) (Eq. 1)                                       */
} alora_config;

/*
 * Rotary position embedding (an option; the paper's equations carry no positional encoding, the model families it
 * evaluates are rotary models).  With cfg->rope_theta > 0 the new query and key rows are rotated by their
 * positions after the projection (delta included) and before the keys are cached: within a head, column i pairs
 * with column i + head_dim/2 and the pair at position p turns by p * rope_theta^(-2i/head_dim).  Cached keys are
 * therefore post-rotation, in every mode alike; rows whose gate is closed still equal the base model's rows bit
 * for bit.  alora_project_qkv then hands out the rotated q and k rows (what alora_kv_append would cache and
 * alora_attend would read).  On the layer paths the rotation and the KV append are one kernel.
 * alora_project_qkv_static does not rotate.
 */

/*
 * Create a context on cfg->device.  Allocates the context-owned workspaces (per-token metadata,
 * tile and work lists, the rank-r intermediate t = A x, a [max_tokens][N] q/k/v staging buffer,
 * split-KV partial results, the status word) with cudaMalloc.  *out is set only on success.
 * alora_destroy frees everything the context owns; it does not touch caller buffers.
 */
alora_status alora_create(const alora_config *cfg, alora_ctx **out);
alora_status alora_destroy(alora_ctx *ctx);

/*
 * Base weights of one layer (Eq. 2).  d_wqkv[N][H] is required; d_wo[H][Nq], d_wgate_up[2*I][H]
 * (gate rows first, then up rows), d_wdown[H][I], d_norm_attn[H], d_norm_mlp[H] may be NULL when
 * only the attention-block entries are used.  Pointers are BORROWED: the caller keeps the memory
 * alive and unchanged while the context uses it.
 */
alora_status alora_set_layer_weights(alora_ctx *ctx, int layer, const void *d_wqkv, const void *d_wo,
                                     const void *d_wgate_up, const void *d_wdown,
                                     const void *d_norm_attn, const void *d_norm_mlp);

/*
 * Register (or replace) adapter `adapter_id` of `layer`: Delta_blk = scale * B_blk A_blk for
 * blk in {q, k, v} (Eq. 4 / Eq. 5).  d_Aq/d_Ak/d_Av are [rank][H], d_Bq is [Nq][rank], d_Bk and
 * d_Bv are [Nkv][rank].  The matrices are COPIED into context-owned, rank-padded storage on the
 * given stream; the caller's buffers may be released once that stream has passed this point.
 * 1 <= rank <= max_rank.
 */
alora_status alora_register_adapter(alora_ctx *ctx, int adapter_id, int layer, int rank, float scale,
                                    const void *d_Aq, const void *d_Bq, const void *d_Ak,
                                    const void *d_Bk, const void *d_Av, const void *d_Bv,
                                    void *stream);

/*
 * Extend adapter `adapter_id` of `layer` to the MLP block: gate, up and down projections each get
 * Delta = scale * B A under the SAME per-token gate as q/k/v (the paper adapts q, k and v and remarks,
 * in its background section and after Eq. 5, that MLP blocks can be adapted in the same manner).
 * d_Agate and d_Aup are [rank][H], d_Bgate and d_Bup are [I][rank], d_Adown is [rank][I],
 * d_Bdown is [H][rank]; I = intermediate size.  Only alora_forward_stack and alora_decode_stack run
 * the MLP block, so only they use these matrices: rows whose gate is open get the deltas, rows whose
 * gate is closed (and every row in ALORA_MODE_BASE) keep the bits of the base MLP.  The matrices are
 * COPIED on the given stream.  The first registration on a layer allocates that layer's slabs
 * (cudaMalloc; about 384 * max_adapters * (H + I) bytes per layer, plus once per context the shrink results
 * and their partial sums), so register before timing anything.
 * Errors: ALORA_ERR_NO_WEIGHTS when the adapter has no q/k/v part on this layer yet (its gate is the
 * q/k/v adapter's); ALORA_ERR_UNSUPPORTED for fp32 contexts, contexts without an MLP (intermediate = 0)
 * and sizes where H or I is not a multiple of 256; ALORA_ERR_CAPACITY for the id or rank.
 */
alora_status alora_register_mlp_adapter(alora_ctx *ctx, int adapter_id, int layer, int rank, float scale,
                                        const void *d_Agate, const void *d_Bgate, const void *d_Aup,
                                        const void *d_Bup, const void *d_Adown, const void *d_Bdown,
                                        void *stream);

/*
 * Host-side consistency check of batch metadata (all pointers HOST memory; launches nothing, needs
 * no device).  Verifies: query_start_loc non-decreasing from 0 to T; positions of each request
 * consecutive and ending at seq_lens[r]-1; adapter ids in [-1, max_adapters); activation offsets
 * >= 0; every block-table entry a request can touch inside [0, num_pages); no physical page used
 * by the writable range of two requests.  Returns ALORA_OK, ALORA_ERR_BAD_BATCH,
 * ALORA_ERR_PAGE_RANGE or ALORA_ERR_CAPACITY.  `cfg` supplies page_size, max_* limits.
 */
alora_status alora_validate_batch(const alora_config *cfg, const int32_t *h_positions,
                                  const int32_t *h_activation_offsets, const int32_t *h_adapter_ids,
                                  const int32_t *h_query_start_loc, const int32_t *h_seq_lens,
                                  const int32_t *h_block_tables, int max_blocks, int num_pages,
                                  int T, int R);

/*
 * Batch metadata step, exposed for exact comparison.  Fills (each output may be NULL):
 *   d_token_request[T]  request index of every token,
 *   d_row_adapter[T]    adapter id applied to the row: adapter_ids[r] if the gate of Eq. 5 is open
 *                       (mode ALORA: p >= a_req; FULL_LORA: always), else -1,
 *   d_slot_mapping[T]   token slot = page * page_size + p % page_size of the row's position.
 * The same kernels run inside every layer call.
 */
alora_status alora_batch_metadata(alora_ctx *ctx, int mode, const int32_t *d_positions,
                                  const int32_t *d_activation_offsets, const int32_t *d_adapter_ids,
                                  const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                                  const int32_t *d_block_tables, int max_blocks, int num_pages,
                                  int T, int R, int32_t *d_token_request, int32_t *d_row_adapter,
                                  int32_t *d_slot_mapping, void *stream);

/*
 * Step 1 alone: d_qkv[T][N] = gated fused projection of d_hidden[T][H] with layer `layer`'s
 * weights (Eq. 5; Eq. 4 for mode FULL_LORA; Eq. 2 for mode BASE or adapter id -1).  Rows whose
 * gate is closed go through exactly the arithmetic of a base-only call, so they are bit-identical
 * to it (Prop. 1).
 */
alora_status alora_project_qkv(alora_ctx *ctx, int layer, int mode, const void *d_hidden,
                               const int32_t *d_positions, const int32_t *d_activation_offsets,
                               const int32_t *d_adapter_ids, const int32_t *d_query_start_loc,
                               const int32_t *d_seq_lens, int T, int R, void *d_qkv, void *stream);

/*
 * Step 2 alone: copy the k and v parts of d_qkv[T][N] into d_paged_kv at each token's slot.
 * Writes exactly T*2*Nkv elements; no other byte of the pool changes.
 */
alora_status alora_kv_append(alora_ctx *ctx, const void *d_qkv, const int32_t *d_positions,
                             const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                             const int32_t *d_block_tables, int max_blocks, int num_pages, int T,
                             int R, void *d_paged_kv, void *stream);

/*
 * Step 3 alone: d_attn_out[T][Nq] = causal GQA attention of the q part of d_qkv[T][N] over
 * positions 0 .. p_t of each request, read from d_paged_kv through d_block_tables (the new rows
 * must already be appended).
 */
alora_status alora_attend(alora_ctx *ctx, const void *d_qkv, const int32_t *d_positions,
                          const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                          const void *d_paged_kv, const int32_t *d_block_tables, int max_blocks,
                          int num_pages, int T, int R, void *d_attn_out, void *stream);

/*
 * The activated prefill of a suffix on a reused base cache: steps 1-3 for one layer (Eq. 5, then
 * Prop. 2's proof steps 1-4).  d_paged_kv must already hold positions 0 .. p_first-1 of every
 * request; it is written only at the slots of the T new positions.  The q/k/v rows are staged in
 * a context-owned buffer.
 */
alora_status alora_prefill_layer(alora_ctx *ctx, int layer, const void *d_hidden,
                                 const int32_t *d_positions, const int32_t *d_activation_offsets,
                                 const int32_t *d_adapter_ids, const int32_t *d_query_start_loc,
                                 const int32_t *d_seq_lens, void *d_paged_kv,
                                 const int32_t *d_block_tables, int max_blocks, int num_pages, int T,
                                 int R, void *d_attn_out, void *stream);

/*
 * One decode step (Prop. 1, second sentence; Eq. 3): exactly one new token per request (T == R,
 * query_start_loc[r] == r), mixed base / adapter requests.  Same results as alora_prefill_layer on
 * the same arguments (a one-token request takes the same few-row attention kernel in every entry
 * point; this one additionally knows that no request is longer, and launches nothing else).
 */
alora_status alora_decode_step(alora_ctx *ctx, int layer, const void *d_hidden,
                               const int32_t *d_positions, const int32_t *d_activation_offsets,
                               const int32_t *d_adapter_ids, const int32_t *d_seq_lens,
                               void *d_paged_kv, const int32_t *d_block_tables, int max_blocks,
                               int num_pages, int R, void *d_attn_out, void *stream);

/*
 * The comparison path (Eq. 4): a conventional LoRA cannot reuse the base cache, so the caller
 * passes ALL prefix + suffix tokens as new tokens (positions from 0) with private pages, and the
 * delta is applied to every row of a request that has an adapter.  With adapter_ids = -1 this is
 * the base model's prefill, which is how a reusable base cache is produced.
 */
alora_status alora_full_lora_prefill_layer(alora_ctx *ctx, int layer, const void *d_hidden,
                                           const int32_t *d_positions, const int32_t *d_adapter_ids,
                                           const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                                           void *d_paged_kv, const int32_t *d_block_tables,
                                           int max_blocks, int num_pages, int T, int R,
                                           void *d_attn_out, void *stream);

/*
 * All n_layers decoder layers (pre-norm residual: h += o_proj(attn(norm(h))); h += down(silu(gate)
 * * up) of norm(h)), adapters on q/k/v only, MLP and o_proj with base weights.  d_paged_kv_layers
 * is a HOST array of n_layers device pointers (one pool per layer, same block tables).
 * d_hidden_in[T][H] -> d_hidden_out[T][H] (may alias).  `mode` selects Eq. 5 / Eq. 4 / Eq. 2.
 * A step whose shape the kernels do not serve (for the tensor-core path: hidden, Nq or intermediate not a
 * multiple of 8) or whose launch fails ends the call there with ALORA_ERR_UNSUPPORTED / ALORA_ERR_CUDA; the
 * steps before it have been enqueued and d_hidden_out then holds an unfinished residual stream.
 */
alora_status alora_forward_stack(alora_ctx *ctx, int mode, const void *d_hidden_in,
                                 const int32_t *d_positions, const int32_t *d_activation_offsets,
                                 const int32_t *d_adapter_ids, const int32_t *d_query_start_loc,
                                 const int32_t *d_seq_lens, void *const *h_paged_kv_layers,
                                 const int32_t *d_block_tables, int max_blocks, int num_pages, int T,
                                 int R, void *d_hidden_out, void *stream);

/*
 * Read and clear the device status word.  Synchronises `stream` first.  *device_status receives
 * ALORA_OK or the first device-side finding since the last call.
 */
alora_status alora_get_status(alora_ctx *ctx, void *stream, int32_t *device_status);

/* Static description of a status code; never NULL. */
const char *alora_status_string(int status);

/* Text of the last CUDA error seen by this context ("" if none); valid until the next call. */
const char *alora_last_cuda_error(const alora_ctx *ctx);

/* Number of kernels this context has launched so far (all entry points). */
int64_t alora_launch_count(const alora_ctx *ctx);

/*
 * Gated q/k/v projection (same result as alora_project_qkv in mode ALORA with one adapter) for
 * callers that cannot allocate device memory.  (The paper has no counterpart: this is an
 * integration aid.)  Typical callers: a plug-in running inside a serving engine that already owns
 * all device memory through its own pool, or a latency-critical loop that must avoid the implicit
 * synchronisation of cudaMalloc/cudaFree.  They cannot use alora_create, which allocates the
 * context's workspaces, so this call needs no context and takes everything as arguments:
 *   dtype, hidden (H), n_q (Nq), n_kv (Nkv)         layer shape, N = n_q + 2*n_kv
 *   d_hidden[T][H], d_wqkv[N][H]                    inputs, device memory, element type = dtype
 *   d_positions[T], d_query_start_loc[R+1], d_activation_offsets[R]   as for alora_project_qkv
 *   d_adapter_on[R]                                 non-zero = request uses the adapter; NULL = all do
 *   rank, scale, d_Aq/d_Ak/d_Av[rank][H], d_Bq[n_q][rank], d_Bk/d_Bv[n_kv][rank]   the adapter,
 *                                                   read in place (nothing is copied or repacked)
 *   d_qkv[T][N]                                     output
 * It calls no cudaMalloc, cudaFree or allocating library routine.  Its scratch (one int32 gate per
 * row and the fp32 intermediate s*A x) lives in a fixed array inside the library image of
 * ALORA_STATIC_MAX_TOKENS * (4 + 12 * ALORA_STATIC_MAX_RANK) bytes (about 3 MiB), which every GPU
 * that loads the library holds until the process exits.  T > ALORA_STATIC_MAX_TOKENS or
 * rank > ALORA_STATIC_MAX_RANK returns ALORA_ERR_CAPACITY and launches nothing.
 * The device that is current when the call is made is used.  The first call on a device looks up
 * the array's device address (a set-up step); make that first call before any stream capture.
 * All calls on a device share the array and it keeps the previous call's contents; each call
 * rewrites whatever it reads, so no clearing is needed, but calls that overlap on the same GPU
 * (different streams or host threads) race on it: serialise them.
 */
#define ALORA_STATIC_MAX_TOKENS 4096
#define ALORA_STATIC_MAX_RANK 64
alora_status alora_project_qkv_static(int dtype, int hidden, int n_q, int n_kv, const void *d_hidden,
                                      const void *d_wqkv, const int32_t *d_positions,
                                      const int32_t *d_query_start_loc, const int32_t *d_activation_offsets,
                                      const int32_t *d_adapter_on, int rank, float scale, const void *d_Aq,
                                      const void *d_Bq, const void *d_Ak, const void *d_Bk, const void *d_Av,
                                      const void *d_Bv, int T, int R, void *d_qkv, void *stream);

/*
 * One decode step through all n_layers decoder layers: alora_forward_stack for a batch of R requests with one new
 * token each (position d_positions[r] = d_seq_lens[r] - 1; Prop. 1, second sentence).  Rows before a request's
 * activation offset, and requests with adapter id -1, run on the base weights.  d_hidden_in / d_hidden_out are
 * [R][H]; the other arguments are those of alora_forward_stack and alora_decode_step.
 */
alora_status alora_decode_stack(alora_ctx *ctx, const void *d_hidden_in, const int32_t *d_positions,
                                const int32_t *d_activation_offsets, const int32_t *d_adapter_ids,
                                const int32_t *d_seq_lens, void *const *h_paged_kv_layers,
                                const int32_t *d_block_tables, int max_blocks, int num_pages, int R,
                                void *d_hidden_out, void *stream);

/*
 * Several adapters on one reused base-model cache (paper, section "Activated LoRA": N adapters invoked on the same
 * conversation share its cache; Prop. 2, the N-adapter clause).  Requests whose block tables begin with the same
 * physical pages read them through the same memory; no page is copied.  The attention of decode-sized requests
 * (at most 16 / G new tokens each) additionally GROUPS neighbouring requests of a batch that have at least 256
 * leading keys in common (whole pages before every member's first new position, up to 64 stacked score rows): the
 * shared keys are then read once for all members, each member's own keys beyond them separately, and the parts are
 * merged by their running maximum and sum.  The results are those of the ungrouped computation up to rounding.
 *
 * alora_prefix_groups reports the grouping of the last layer / attend call of this context: per request the index
 * of its group's first request (its own index when ungrouped) and the number of keys the group shares (0 when
 * ungrouped).  Device arrays of R int32 each; asynchronous on `stream`.  ALORA_ERR_UNSUPPORTED on an fp32 context.
 *
 * alora_cow_tail_pages is the copy-on-write step a caller needs when the reused length is not a multiple of the
 * page size: the page that holds the last reused positions would also receive a request's first new rows.  For
 * every request r with d_fresh_pages[r] >= 0 (a page id the caller took from its free list; -1: nothing to do) the
 * rows of the reused positions on that page are copied to the fresh page (both planes, all KV heads) and
 * d_block_tables[r] is redirected to it, in place.  Run it before the layer call; alora_validate_batch rejects a
 * batch in which two requests would still write the same page.  Findings (fresh page out of range, request
 * without new tokens) go to the status word.
 */
alora_status alora_prefix_groups(alora_ctx *ctx, int R, int32_t *d_group_first, int32_t *d_shared_keys, void *stream);
alora_status alora_cow_tail_pages(alora_ctx *ctx, const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                                  int32_t *d_block_tables, int max_blocks, int num_pages, int R,
                                  const int32_t *d_fresh_pages, void *d_paged_kv, void *stream);

/*
 * Self-test of the bounded waits (the paper has no counterpart).  Every wait inside the tensor-core kernels
 * (on a shared-memory barrier, on another block's ready counter) gives up after a cycle limit, records
 * ALORA_ERR_TIMEOUT in the status word and lets the kernel return through its normal exit.  This call runs that
 * give-up path on purpose and harmlessly: one block of one warp waits on a barrier that nobody arrives at, with
 * the given limit (1 .. 200 000 000 clock cycles, i.e. at most about 0.1 s), then returns.  Afterwards
 * alora_get_status reads ALORA_ERR_TIMEOUT (and clears it); the context remains usable.  Asynchronous on `stream`.
 */
alora_status alora_selftest_wait_timeout(alora_ctx *ctx, int64_t limit_cycles, void *stream);

/*
 * Several contexts, streams and processes may use one GPU at the same time: they share its SMs, and a launch of
 * this library never assumes that all of its blocks are running at once.  Where one work item of a launch needs
 * another's result (a projection item needs its row tile's shrink item), the needed items are handed out through
 * a counter to blocks that are running, and no block starts on a dependent item before every needed item has been
 * claimed (csrc/claim_order.h).  Every in-kernel wait is bounded (about a second): if one still runs out, the
 * kernel returns through its normal exit, ALORA_ERR_TIMEOUT is recorded in the status word, and the outputs of
 * that call are not valid; the context stays usable.
 *
 * alora_selftest_claim_order is a HOST-ONLY model of that item order (no device, no context): a launch of `grid`
 * blocks with n_shrink shrink items and n_row_tiles x n_col_tiles projection items runs on a GPU that keeps only
 * `resident_slots` blocks running at a time, blocks entering free slots highest index first
 * (high_blocks_first != 0) or lowest first.  *completed = 1 when every item completes, 0 when running blocks end
 * up waiting for items that no running block holds.  static_order != 0 models dealing ALL items by block index
 * instead (the order the counter replaced), for comparison.  ALORA_ERR_INVALID_ARG for sizes out of range.
 */
alora_status alora_selftest_claim_order(int grid, int n_shrink, int n_row_tiles, int n_col_tiles,
                                        int resident_slots, int high_blocks_first, int static_order,
                                        int *completed);

/*
 * Optional per-kernel timing (a measurement aid; the paper has no counterpart).  While enabled,
 * every kernel family launched by this context is bracketed by CUDA events on the launching stream.
 * alora_profile_enable(ctx, 1) clears what was accumulated and starts, (ctx, 0) stops.
 * alora_profile_read synchronises the device and adds up, per family, the elapsed milliseconds and
 * the number of bracketed launch groups; both arrays have ALORA_PROFILE_KINDS entries.
 * Families: 0 batch metadata, 1 rank-r shrink (t = A x) when it is a launch of its own, or the per-row
 * low-rank delta of small batches, 2 q/k/v projection (on the bf16 layer paths it also appends the new k / v rows
 * to the cache), 3 KV append as a launch of its own (alora_kv_append, fp32 layers), 4 attention on the tensor-core
 * kernel (with the merge of cut work items) and the fp32 kernel, 5 attention on the few-row split-KV kernel (decode
 * steps, shortest suffixes, prefix groups), 6 other dense projections (o_proj, MLP), 7 norm / activation
 * glue.
 */
#define ALORA_PROFILE_KINDS 8
alora_status alora_profile_enable(alora_ctx *ctx, int on);
alora_status alora_profile_read(alora_ctx *ctx, double *ms_by_kind, int64_t *groups_by_kind);

#ifdef __cplusplus
}
#endif
#endif /* ALORA_H */
