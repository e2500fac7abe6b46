// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "alora.h"

namespace alora {

constexpr int kRankPadMax = 64;  // adapters are stored padded to a multiple of 16 rows, <= 64
constexpr int kRowwiseMaxTokens = 1024;  // largest batch that may take the row-wise delta route of the projection
constexpr int kMlpChunk = 8192;   // tokens per MLP pass of the stack entry (bounds the gate/up buffer)

// Per (layer, adapter) record as the kernels see it.  A is [3][rpad_max][H] (q, k, v blocks, rows
// beyond the rank are zero), B is [N][rpad_max] (row n holds the B row of output column n, columns
// beyond the rank are zero).
struct AdapterDev {
    const void *A;
    const void *B;
    int32_t rank;   // 0 = not registered
    int32_t rpad;   // rank rounded up to 16
    float scale;
    int32_t pad_;
};

// One adapter's part on the MLP block of one layer (gate, up and down projections share rank and scale).
struct MlpAdapterDev {
    int32_t rpad;   // rank rounded up to 16; 0 = no MLP part registered
    float scale;
};

struct LayerWeights {
    const void *wqkv = nullptr, *wo = nullptr, *wgate_up = nullptr, *wdown = nullptr;
    const void *norm_attn = nullptr, *norm_mlp = nullptr;
};

// One row-tile of the projection: rows [row_start, row_start + row_count) of the batch, all with
// the same applied adapter (or -1).  A tile never spans two different applied adapters, so rows
// whose gate is closed run through tiles that execute the base-only instruction sequence.
struct ProjTile {
    int32_t row_start;
    int32_t row_count;
    int32_t adapter;  // applied adapter id, -1 = none
    int32_t pad_;
};

// One unit of attention work: query tokens [q_start, q_start + q_count) of request `req` (flat
// token indices), one KV head, keys [kv_start, kv_end) of the request's sequence.
struct AttnWork {
    int32_t req;
    int32_t q_start;
    int32_t q_count;
    int32_t kv_head;
    int32_t kv_start;
    int32_t kv_end;
    int32_t split;     // 128-key tiles of all earlier items of the work list
    int32_t n_splits;
};
constexpr int kAttnKeysPerTile = 128;   // keys per K/V tile of the tensor-core attention kernel
constexpr int kRowwiseAlwaysRows = 24;  // batches of at most this many rows always take the projection's row-wise route
constexpr int kAttnMinRunTiles = 8;     // shortest run of key tiles given to one block
constexpr int kAttnCutMinTiles = 128;   // items are cut into runs only when a block has at least this many tiles to do
constexpr int kAttnCutMinWaves = 3;     // ... and the items make at least this many full rounds over the blocks
constexpr int kAttnSpreadMinGain = 24; // fewer items than blocks: spread them only if the longest item is this many tiles longer than a block's run

// One unit of few-row (decode / short suffix) attention work: score rows of `q_count` tokens starting at
// flat token q_start (rows are (token, query head of the group) pairs, `mt` tiles of 16 rows), one KV
// head, keys [kv_start, kv_end) of the request.  The `n_splits` key ranges of the same rows are
// consecutive items; their partial results are merged afterwards.
struct AttnSplitWork {
    int32_t req, q_start, q_count, kv_head;
    int32_t kv_start, kv_end, pos0, mt;      // pos0 = position of the first token of the block
    int32_t split, n_splits, part_row0;        // part_row0 = first row of this item in the partial-result arrays
    int32_t pad_;   // 0: every token of the block sees keys up to its own position.  kSplitOwnKeys | n_members: the item
                    // covers the OWN keys of a prefix group's members (requests req .. req + n_members - 1), i.e. their
                    // keys from position pos0 (the shared length) on, as one sequence of 64-key stages, member after
                    // member; kv_start / kv_end count those stages (x 64); a stage's keys are seen by its member's
                    // tokens only, up to each token's own position
};
constexpr int32_t kSplitOwnKeys = 0x40000000;
constexpr int kSplitItemsPerSm = 16;   // target number of (row tile, key range) pairs per SM

// Few-row projection (batches of at most kFewRowMax rows): what its two kernels need to know about the batch's
// adapters, written by the batch-metadata step: the adapters that occur among the rows' applied adapters
// (ascending ids), per slot the padded rank and the scale, and per row the slot of its adapter.
constexpr int kFewRowMax = 128;
struct FewRowMeta {
    int32_t n_present;
    int32_t pad_[3];
    int32_t slot_of_row[kFewRowMax];  // -1: the row adds no delta
    int32_t id[kFewRowMax];           // adapter id of each slot
    int32_t rpad[kFewRowMax];         // its rank rounded up to 16
    float scale[kFewRowMax];
};

// Kernel families, for the optional per-kernel timing (alora_profile_*).
enum KernelKind { KK_METADATA = 0, KK_SHRINK, KK_PROJECT, KK_KV_APPEND, KK_ATTENTION, KK_ATTN_FEW_ROW, KK_LINEAR,
                  KK_GLUE, KK_COUNT };

struct ProfEvent {
    cudaEvent_t begin, end;
    int kind;
};

// Tensor maps of one layer that depend only on registered weights (bf16 tensor-core path).
struct TcLayerMaps {
    CUtensorMap wqkv[3];      // W_qkv [N][H], boxes of 128 / 256 / 64 rows
    CUtensorMap a_all;        // all adapters' A rows [max_adapters*192][H], box 192 rows
    CUtensorMap a_all16;      // the same rows in boxes of 16 (shrink chunks of the few-row projection)
    CUtensorMap b_all_bn[3];  // all adapters' B rows [max_adapters*N][64], boxes of 128 / 256 / 64 rows
    // for the 256 x 192 tiles of gemm_pair_tcgen05.cu: W in boxes of 192 rows; per q / k / v block the B rows of all
    // adapters as (rank column, row inside the block, adapter), boxes of 192 rows
    CUtensorMap wqkv192;
    CUtensorMap b_blk[3];
    bool pair_ok = false;
};

struct Dims {
    int H, Hq, Hkv, hd, G, Nq, Nkv, N, page, I, RP;  // RP = padded max rank
    float softmax_scale;
};

}  // namespace alora

namespace alora { struct BatchArgs; }

struct alora_ctx {
    alora_config cfg;
    alora::Dims d;
    size_t esize = 2;
    std::vector<alora::LayerWeights> layers;
    std::vector<alora::AdapterDev> h_adapters;  // [layer * max_adapters + id], mirrors d_adapters
    alora::AdapterDev *d_adapters = nullptr;
    std::vector<void *> adapter_storage;         // context-owned A/B buffers, same indexing, 2 per entry

    // bf16 tensor-core path: per-layer adapter storage shared by all adapters of the layer
    std::vector<void *> tc_a_all, tc_b_all;          // [layer] -> [max_adapters][3*64][H], [max_adapters][N][64]
    std::vector<alora::TcLayerMaps> tc_maps;         // [layer]
    std::vector<char> layer_has_adapter;             // [layer] any adapter registered
    // adapters on the MLP block (bf16), allocated when the first one is registered on a layer: the A rows of all
    // adapters as one weight matrix per projection pair, the B rows per adapter
    std::vector<void *> mlp_a_gu, mlp_b_gu;          // [layer] -> [max_adapters][2][RP][H], [max_adapters][2 I][RP]
    std::vector<void *> mlp_a_dn, mlp_b_dn;          // [layer] -> [max_adapters][RP][I] (rows padded to 128), [max_adapters][H][RP]
    std::vector<int> mlp_n_adapters;                 // [layer] highest registered MLP adapter id + 1
    std::vector<alora::MlpAdapterDev> h_mlp_adapters;   // [layer * max_adapters + id], mirrors d_mlp_adapters
    alora::MlpAdapterDev *d_mlp_adapters = nullptr;
    void *d_mlp_t = nullptr;                         // [min(max_tokens, kMlpChunk)][max_adapters * 2 * RP] shrink results
    float *d_mlp_part = nullptr;                     // K-slice partials of the shrink kernel
    size_t mlp_part_floats = 0;
    int32_t *d_mlp_done = nullptr;                   // per 64 x 64 tile of the shrink result: slices stored (zero between launches)
    int mlp_done_ints = 0;

    // per-call workspaces
    int32_t *d_token_req = nullptr, *d_row_adapter = nullptr, *d_slot = nullptr;
    alora::ProjTile *d_tiles = nullptr;
    int32_t *d_counts = nullptr;  // [0] projection row tiles, [1] attention work items, [2] row tiles with an adapter,
                                  // [3] few-row attention items, [4] next unclaimed few-row item,
                                  // [5] 1 = the projection takes the row-wise route for this batch,
                                  // [6] key tiles of the attention items that are cut into runs, [7] tiles per run,
                                  // [8] attention items taken whole (the first ones), [9] key tiles of those
    int32_t *d_seg_scratch = nullptr;  // [14*max_requests+5] per-request values and merged row runs of the current batch
    int32_t *d_shrink_tiles = nullptr; // [max_tiles] indices of the row tiles with an adapter
    int32_t *d_t_ready = nullptr;      // [max_tiles] per row tile: epilogue warps that have published t
    int32_t *d_iota = nullptr;         // 0..max_requests: query_start_loc of a decode batch
    int32_t max_tiles = 0;
    alora::AttnWork *d_attn_items = nullptr;  // tensor-core attention work list (bf16)
    int32_t *d_attn_off = nullptr;            // [max_requests+1] block offsets per request
    int32_t max_attn_items = 0, attn_q_block = 0;
    // long batches: the tensor-core attention kernel takes some items whole and cuts the key tiles of the rest into runs
    int32_t *d_attn_cta_start = nullptr;      // [n_sm] first item of each block's run
    float *d_attn_part_o = nullptr;           // [2 * n_sm][hd][256] unnormalised outputs of the parts of cut items
    float *d_attn_part_ml = nullptr;          // [2 * n_sm][2][256] their exponent references and row sums
    // few-row attention (requests with at most small_max_tokens new tokens): split-KV work list and partials
    alora::AttnSplitWork *d_split_items = nullptr;
    int32_t *d_req_scratch = nullptr;   // [5][max_requests] items per request, item offset, partial-row offset, prefix groups
    int32_t *d_prefix_groups = nullptr; // [2][max_requests] per request of the last batch: first request of its prefix
                                        // group, keys the group shares (0: ungrouped)
    float *d_part_o = nullptr, *d_part_ml = nullptr;
    int32_t *d_group_done = nullptr;    // [max_split_items] finished key ranges per group (first item's index)
    int32_t max_split_items = 0, max_split_rows = 0, small_max_tokens = 0;
    void *d_t = nullptr;          // [max_tokens][3][RP] rank-r intermediate
    float *d_row_delta = nullptr; // [min(max_tokens, kRowwiseMaxTokens)][N] fp32 delta rows (bf16 row-wise route)
    // few-row projection (batches of <= 128 rows): K-slice partial products and partial shrink results
    float *d_skinny_part = nullptr;   // [skinny_max_items][128][256] fp32
    float *d_skinny_t = nullptr;      // [slices of the q/k/v projection][128][skinny_p_cap][192] fp32
    void *d_skinny_meta = nullptr;    // FewRowMeta of the current batch
    const alora::BatchArgs *pending_attn_meta = nullptr;   // run_layer: attention lists still to be built for this batch
    int skinny_max_items = 0, skinny_p_cap = 0;
    void *d_qkv = nullptr;        // [max_tokens][N]
    void *d_act[4] = {nullptr, nullptr, nullptr, nullptr};  // stack activations
    double *d_rope_inv_freq = nullptr;   // [hd / 2] theta^(-2i/hd), only with a rotary base configured
    int32_t *d_status = nullptr;
    int32_t *h_status = nullptr;  // pinned

    bool profiling = false;
    std::vector<alora::ProfEvent> prof_events;  // event pairs recorded since profiling was enabled
    size_t prof_used = 0;
    int64_t launches = 0;
    std::string cuda_err;
    int sm_count = 148;
};

namespace alora {

// Records a CUDA failure in the context and maps it to ALORA_ERR_CUDA.
alora_status cuda_fail(alora_ctx *ctx, cudaError_t e, const char *what);

#define ALORA_CUDA(ctx, call)                                              \
    do {                                                                   \
        cudaError_t e__ = (call);                                          \
        if (e__ != cudaSuccess) return ::alora::cuda_fail(ctx, e__, #call); \
    } while (0)

// Brackets the launches of one kernel family with CUDA events while profiling is on.
// Kernel launch with the programmatic-stream-serialization attribute (`dependent`: the kernel calls
// tc::grid_dep_wait() before it touches anything its predecessor in the stream wrote or still reads).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                 bool dependent, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = dependent ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

struct ProfScope {
    alora_ctx *ctx;
    cudaStream_t s;
    cudaEvent_t end = nullptr;
    ProfScope(alora_ctx *c, int kind, cudaStream_t st) : ctx(c), s(st) {
        if (!c->profiling) return;
        if (c->prof_used == c->prof_events.size()) {
            ProfEvent e{nullptr, nullptr, kind};
            if (cudaEventCreate(&e.begin) != cudaSuccess || cudaEventCreate(&e.end) != cudaSuccess) return;
            c->prof_events.push_back(e);
        }
        ProfEvent &e = c->prof_events[c->prof_used++];
        e.kind = kind;
        cudaEventRecord(e.begin, st);
        end = e.end;
    }
    ~ProfScope() { if (end) cudaEventRecord(end, s); }
};

// ---- launchers implemented in the kernel files (each returns the number of kernels launched or <0) ----
struct BatchArgs {
    const int32_t *positions, *activation_offsets, *adapter_ids, *query_start_loc, *seq_lens, *block_tables;
    int max_blocks, num_pages, T, R, mode;
    int all_small;  // host-side knowledge that no request has more than small_max_tokens new tokens (decode)
    int layer = -1; // layer whose adapter table the gate is checked against (-1: no check)
    int few_row = 0; // the projection of this batch takes the few-row route: build FewRowMeta instead of row tiles
};

// phases: bit 0 = per-token arrays and the projection's lists, bit 1 = the attention work lists.  A launch of
// the attention lists alone is a programmatic dependent launch: it may run beside the projection kernel that
// precedes it in the stream.  `timed`: bracket it with profiling events of the metadata family.
constexpr int kMetaProjection = 1, kMetaAttention = 2;
int launch_metadata(alora_ctx *ctx, const BatchArgs &b, cudaStream_t s, int phases = kMetaProjection | kMetaAttention,
                    bool timed = true);
int launch_repack_adapter(alora_ctx *ctx, int rank, const void *Aq, const void *Bq, const void *Ak,
                          const void *Bk, const void *Av, const void *Bv, void *A_dst, void *B_dst,
                          cudaStream_t s);
int launch_project(alora_ctx *ctx, int layer, const void *hidden, int T, void *qkv, cudaStream_t s, void *kv_pool,
                   int num_pages, bool *kv_appended);
int launch_kv_append(alora_ctx *ctx, const void *qkv, int T, int num_pages, void *pool, cudaStream_t s);
int launch_cow_tail_pages(alora_ctx *ctx, const int32_t *qsl, const int32_t *seq_lens, int32_t *block_tables, int max_blocks,
                          int num_pages, int R, const int32_t *fresh_pages, void *pool, cudaStream_t s);
int launch_rope(alora_ctx *ctx, void *qkv, const int32_t *positions, int T, void *pool, int num_pages, cudaStream_t s);
int launch_attend(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                  cudaStream_t s);
int launch_linear(alora_ctx *ctx, const void *x, const void *W, int T, int K, int N, void *y,
                  const void *residual, cudaStream_t s);
int launch_rmsnorm(alora_ctx *ctx, const void *x, const void *w, int T, void *y, cudaStream_t s);
int launch_swiglu(alora_ctx *ctx, const void *gate_up, int T, void *y, cudaStream_t s);

// device-side status recording: first finding wins
__device__ __forceinline__ void report(int32_t *status, int code) { atomicCAS(status, 0, code); }

}  // namespace alora
