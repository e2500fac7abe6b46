// C ABI of the library: context management, argument checks, and the order in which the kernels
// of one layer are enqueued.  No arithmetic of the method lives here.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "alora_internal.h"

namespace alora {

alora_status cuda_fail(alora_ctx *ctx, cudaError_t e, const char *what) {
    if (ctx) ctx->cuda_err = std::string(what) + ": " + cudaGetErrorString(e);
    return ALORA_ERR_CUDA;
}

int launch_project_simt(alora_ctx *, int, const void *, int, void *, cudaStream_t);
int launch_linear_simt(alora_ctx *, const void *, const void *, int, int, int, void *, const void *, cudaStream_t);
int launch_attend_simt(alora_ctx *, const void *, const BatchArgs &, const void *, void *, cudaStream_t);

int launch_project_tc(alora_ctx *, int, const void *, int, void *, cudaStream_t, void *, int);
int launch_linear_tc(alora_ctx *, const void *, const void *, int, int, int, void *, const void *, cudaStream_t);
int launch_repack_mlp(const void *, const void *, const void *, const void *, int, int, int, int, int, void *, void *,
                      cudaStream_t);   // mlp_adapter.cu
int launch_mlp_expand(alora_ctx *, void *, int, int, const void *, int, const void *, int, int, int, const int32_t *,
                      const MlpAdapterDev *, int, cudaStream_t);
int launch_mlp_shrink(alora_ctx *, const void *, const void *, int, int, int, void *, float *, size_t, int32_t *, int,
                      cudaStream_t);
bool build_layer_maps(alora_ctx *ctx, int layer);
bool project_is_few_row(const alora_ctx *ctx, int layer, int T);   // gemm_tcgen05.cu
int launch_attend_tc(alora_ctx *, const void *, const BatchArgs &, const void *, void *, cudaStream_t);

// bf16 runs on the tensor cores; the fp32 data type (tiny exact-precision configurations) on CUDA cores.
// With a page pool given, the bf16 projection also writes the k / v columns of every row to the row's cache slot
// (the KV append fused into its epilogue) and sets *kv_appended.
int launch_project(alora_ctx *ctx, int layer, const void *hidden, int T, void *qkv, cudaStream_t s, void *kv_pool,
                   int num_pages, bool *kv_appended) {
    if (kv_appended) *kv_appended = false;
    if (ctx->cfg.dtype == ALORA_DTYPE_BF16) {
        const int n = launch_project_tc(ctx, layer, hidden, T, qkv, s, kv_pool, num_pages);
        if (kv_appended && n >= 0 && kv_pool != nullptr) *kv_appended = true;
        return n;
    }
    return launch_project_simt(ctx, layer, hidden, T, qkv, s);
}
int launch_linear(alora_ctx *ctx, const void *x, const void *W, int T, int K, int N, void *y,
                  const void *residual, cudaStream_t s) {
    if (ctx->cfg.dtype == ALORA_DTYPE_BF16) return launch_linear_tc(ctx, x, W, T, K, N, y, residual, s);
    return launch_linear_simt(ctx, x, W, T, K, N, y, residual, s);
}
int launch_attend(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                  cudaStream_t s) {
    if (ctx->cfg.dtype == ALORA_DTYPE_BF16) return launch_attend_tc(ctx, qkv, b, pool, out, s);
    return launch_attend_simt(ctx, qkv, b, pool, out, s);
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static alora_status check_batch_args(alora_ctx *ctx, int T, int R) {
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    if (T < 0 || R < 0) return ALORA_ERR_INVALID_ARG;
    if (T > 0 && R == 0) return ALORA_ERR_INVALID_ARG;   // tokens that belong to no request
    if (T > ctx->cfg.max_tokens || R > ctx->cfg.max_requests) return ALORA_ERR_CAPACITY;
    return ALORA_OK;
}

static alora_status finish(alora_ctx *ctx, int launched) {
    if (launched < 0) return ALORA_ERR_UNSUPPORTED;
    ctx->launches += launched;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "kernel launch");
    return ALORA_OK;
}

// Steps 1-3 of one layer, in the order of Prop. 2's proof.
static alora_status run_layer(alora_ctx *ctx, int layer, const void *hidden, const BatchArgs &b_in, void *pool,
                              void *attn_out, cudaStream_t s) {
    if (layer < 0 || layer >= ctx->cfg.n_layers) return ALORA_ERR_INVALID_ARG;
    if (!ctx->layers[layer].wqkv) return ALORA_ERR_NO_WEIGHTS;
    BatchArgs b = b_in;
    b.layer = layer;
    b.few_row = project_is_few_row(ctx, layer, b.T) ? 1 : 0;
    int n = 0, k;
    // The per-token arrays and the projection's lists first; the attention work lists are built beside the
    // projection (the few-row projection launches them between its two kernels, the other routes right after).
    if ((k = launch_metadata(ctx, b, s, kMetaProjection)) < 0) return ALORA_ERR_UNSUPPORTED; n += k;
    bool kv_appended = false;
    const bool rope = ctx->d_rope_inv_freq != nullptr;   // the rotation comes between projection and append
    ctx->pending_attn_meta = &b;
    k = launch_project(ctx, layer, hidden, b.T, ctx->d_qkv, s, rope ? nullptr : pool, b.num_pages, &kv_appended);
    const bool attn_meta_pending = ctx->pending_attn_meta != nullptr;
    ctx->pending_attn_meta = nullptr;
    if (k < 0) return ALORA_ERR_UNSUPPORTED;
    n += k;
    if (attn_meta_pending) {
        if ((k = launch_metadata(ctx, b, s, kMetaAttention)) < 0) return ALORA_ERR_UNSUPPORTED;
        n += k;
    }
    if (rope) {   // rotate the new q and k rows by their positions and append the rotated keys and the values
        if ((k = launch_rope(ctx, ctx->d_qkv, b.positions, b.T, pool, b.num_pages, s)) < 0) return ALORA_ERR_UNSUPPORTED;
        n += k;
    } else if (!kv_appended) {
        if ((k = launch_kv_append(ctx, ctx->d_qkv, b.T, b.num_pages, pool, s)) < 0) return ALORA_ERR_UNSUPPORTED;
        n += k;
    }
    if ((k = launch_attend(ctx, ctx->d_qkv, b, pool, attn_out, s)) < 0) return ALORA_ERR_UNSUPPORTED; n += k;
    return finish(ctx, n);
}

}  // namespace alora

using namespace alora;

extern "C" {

const char *alora_status_string(int status) {
    switch (status) {
        case ALORA_OK: return "ok";
        case ALORA_ERR_INVALID_ARG: return "invalid argument";
        case ALORA_ERR_UNSUPPORTED: return "unsupported shape or data type";
        case ALORA_ERR_CAPACITY: return "exceeds the capacity given to alora_create";
        case ALORA_ERR_NO_WEIGHTS: return "layer weights or adapter not set";
        case ALORA_ERR_CUDA: return "CUDA call failed";
        case ALORA_ERR_BAD_BATCH: return "inconsistent batch metadata";
        case ALORA_ERR_PAGE_RANGE: return "block-table entry outside the page pool";
        case ALORA_ERR_TIMEOUT: return "bounded in-kernel wait expired";
        case ALORA_ERR_NO_DEVICE: return "no usable CUDA device";
        default: return "unknown status";
    }
}

const char *alora_last_cuda_error(const alora_ctx *ctx) { return ctx ? ctx->cuda_err.c_str() : ""; }
int64_t alora_launch_count(const alora_ctx *ctx) { return ctx ? ctx->launches : 0; }

alora_status alora_create(const alora_config *cfg, alora_ctx **out) {
    if (!cfg || !out) return ALORA_ERR_INVALID_ARG;
    const alora_config &c = *cfg;
    if (c.hidden <= 0 || c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.head_dim <= 0 || c.page_size <= 0 ||
        c.n_layers <= 0 || c.max_adapters < 0 || c.max_rank < 0 || c.max_tokens <= 0 || c.max_requests <= 0 ||
        c.intermediate < 0)
        return ALORA_ERR_INVALID_ARG;
    if (c.n_q_heads % c.n_kv_heads != 0) return ALORA_ERR_INVALID_ARG;
    if (c.dtype != ALORA_DTYPE_BF16 && c.dtype != ALORA_DTYPE_FP32) return ALORA_ERR_UNSUPPORTED;
    if (c.rope_theta < 0.f || (c.rope_theta != 0.f && c.head_dim % 2 != 0)) return ALORA_ERR_INVALID_ARG;
    if (c.max_rank > kRankPadMax) return ALORA_ERR_UNSUPPORTED;
    if (c.head_dim != 32 && c.head_dim != 64 && c.head_dim != 128) return ALORA_ERR_UNSUPPORTED;
    if (c.n_q_heads / c.n_kv_heads > 8) return ALORA_ERR_UNSUPPORTED;
    const size_t es = c.dtype == ALORA_DTYPE_FP32 ? 4 : 2;
    if ((c.head_dim * es) % 16 != 0 || (c.hidden * es) % 16 != 0) return ALORA_ERR_UNSUPPORTED;

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0 || c.device < 0 || c.device >= ndev) {
        cudaGetLastError();
        return ALORA_ERR_NO_DEVICE;
    }
    alora_ctx *ctx = new (std::nothrow) alora_ctx();
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    ctx->cfg = c;
    ctx->esize = es;
    Dims &d = ctx->d;
    d.H = c.hidden; d.Hq = c.n_q_heads; d.Hkv = c.n_kv_heads; d.hd = c.head_dim; d.G = d.Hq / d.Hkv;
    d.Nq = d.Hq * d.hd; d.Nkv = d.Hkv * d.hd; d.N = d.Nq + 2 * d.Nkv; d.page = c.page_size; d.I = c.intermediate;
    // adapters are stored rank-padded: to 64 columns on the tensor-core path (one 128-byte swizzle row),
    // to the next multiple of 16 on the fp32 path
    d.RP = c.dtype == ALORA_DTYPE_BF16 ? 64 : std::max(16, (c.max_rank + 15) / 16 * 16);
    d.softmax_scale = c.softmax_scale != 0.f ? c.softmax_scale : 1.0f / sqrtf((float)d.hd);
    ctx->layers.resize(c.n_layers);
    const size_t n_ad = (size_t)c.n_layers * std::max(1, c.max_adapters);
    ctx->h_adapters.assign(n_ad, AdapterDev{nullptr, nullptr, 0, 0, 0.f, 0});
    ctx->adapter_storage.assign(2 * n_ad, nullptr);

    alora_status st = ALORA_OK;
    auto alloc = [&](void **p, size_t bytes) {
        if (st != ALORA_OK) return;
        cudaError_t e = cudaMalloc(p, std::max<size_t>(bytes, 16));
        if (e != cudaSuccess) st = cuda_fail(ctx, e, "cudaMalloc");
    };
    cudaError_t e = cudaSetDevice(c.device);
    if (e != cudaSuccess) { delete ctx; return ALORA_ERR_NO_DEVICE; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c.device) == cudaSuccess) ctx->sm_count = prop.multiProcessorCount;
    const size_t Tm = (size_t)c.max_tokens;
    ctx->max_tiles = (int)(Tm / 128 + 2 * (size_t)c.max_requests + 2);
    alloc((void **)&ctx->d_adapters, n_ad * sizeof(AdapterDev));
    alloc((void **)&ctx->d_token_req, Tm * 4);
    alloc((void **)&ctx->d_row_adapter, Tm * 4);
    alloc((void **)&ctx->d_slot, Tm * 4);
    alloc((void **)&ctx->d_tiles, (size_t)ctx->max_tiles * sizeof(ProjTile));
    alloc((void **)&ctx->d_counts, 16 * 4);
    alloc((void **)&ctx->d_seg_scratch, ((size_t)14 * c.max_requests + 5) * 4);
    alloc((void **)&ctx->d_shrink_tiles, (size_t)ctx->max_tiles * 4);
    alloc((void **)&ctx->d_t_ready, (size_t)ctx->max_tiles * 4);
    alloc(&ctx->d_t, Tm * 3 * d.RP * 4);
    alloc(&ctx->d_qkv, Tm * d.N * es);
    alloc((void **)&ctx->d_status, 4);
    if (c.rope_theta != 0.f) alloc((void **)&ctx->d_rope_inv_freq, (size_t)(c.head_dim / 2) * sizeof(double));
    alloc((void **)&ctx->d_iota, ((size_t)c.max_requests + 1) * 4);   // 0, 1, ..: query_start_loc of a decode batch
    ctx->layer_has_adapter.assign(c.n_layers, 0);
    if (c.dtype == ALORA_DTYPE_BF16 && 128 % d.G == 0) {
        // tensor-core attention: one work item per (request, KV head, block of 2 * 128/G tokens)
        ctx->attn_q_block = 2 * (128 / d.G);
        ctx->max_attn_items = (int)((Tm / ctx->attn_q_block + (size_t)c.max_requests) * d.Hkv);
        alloc((void **)&ctx->d_attn_items, (size_t)ctx->max_attn_items * sizeof(AttnWork));
        alloc((void **)&ctx->d_attn_off, ((size_t)c.max_requests + 1) * 4);
        alloc((void **)&ctx->d_attn_cta_start, (size_t)ctx->sm_count * 4);
        alloc((void **)&ctx->d_attn_part_o, (size_t)2 * ctx->sm_count * d.hd * 256 * 4);
        alloc((void **)&ctx->d_attn_part_ml, (size_t)2 * ctx->sm_count * 2 * 256 * 4);
        if (16 % d.G == 0 && (d.hd == 64 || d.hd == 128)) {
            // few-row attention, for requests whose new tokens make at most 16 score rows per KV head (decode steps,
            // suffixes of up to 16 / G tokens); longer ones go to the tensor-core kernel, which is the faster of
            // the two from 32 rows on (measured: 8- and 16-token suffixes of 64 requests on 4096 cached tokens
            // reach 0.71 / 0.72 of the HBM bandwidth there against 0.57 / 0.37 here).  At most kSplitItemsPerSm * n_sm
            // key ranges plus one per (request, KV head, row block); a range of mt row tiles owns 16 * mt rows of
            // the partial-result arrays
            ctx->small_max_tokens = std::max(1, 16 / d.G);
            const int blocks_per_req = std::max(1, (ctx->small_max_tokens * d.G + 63) / 64);
            // (twice: in a prefix group every member adds a stream of its own keys to the shared one)
            const int groups = 2 * c.max_requests * blocks_per_req * d.Hkv;
            ctx->max_split_items = kSplitItemsPerSm * ctx->sm_count + groups;
            ctx->max_split_rows = 16 * (kSplitItemsPerSm * ctx->sm_count + 4 * groups);
            alloc((void **)&ctx->d_split_items, (size_t)ctx->max_split_items * sizeof(AttnSplitWork));
            alloc((void **)&ctx->d_req_scratch, (size_t)5 * c.max_requests * 4);
            alloc((void **)&ctx->d_prefix_groups, (size_t)2 * c.max_requests * 4);
            alloc((void **)&ctx->d_part_o, (size_t)ctx->max_split_rows * d.hd * 4);
            alloc((void **)&ctx->d_part_ml, (size_t)ctx->max_split_rows * 2 * 4);
            alloc((void **)&ctx->d_group_done, (size_t)ctx->max_split_items * 4);
        }
    }
    if (c.dtype == ALORA_DTYPE_BF16) {
        {
            // few-row projection: one 128 x 256 fp32 partial per work item (at most one item per SM, or one per column
            // tile of the widest matrix), and the partial shrink results of the q/k/v projection's K slices
            const int widest = std::max(std::max(d.N, d.H), 2 * d.I);
            ctx->skinny_max_items = std::max(ctx->sm_count, (widest + 255) / 256);
            ctx->skinny_p_cap = std::min(std::max(c.max_adapters, 0), 128);
            const int n_tiles = (d.N + 255) / 256, kb = (d.H + 63) / 64;
            const int ksplit = std::max(1, std::min(kb, ctx->sm_count / std::max(n_tiles, 1)));
            alloc((void **)&ctx->d_skinny_part, (size_t)ctx->skinny_max_items * 128 * 256 * 4);
            alloc((void **)&ctx->d_skinny_t, (size_t)ksplit * 128 * std::max(ctx->skinny_p_cap, 1) * 192 * 4);
            alloc(&ctx->d_skinny_meta, sizeof(FewRowMeta));
        }
        alloc((void **)&ctx->d_row_delta, std::min<size_t>(Tm, kRowwiseMaxTokens) * d.N * 4);
        const size_t na = (size_t)std::max(1, c.max_adapters);
        ctx->tc_a_all.assign(c.n_layers, nullptr);
        ctx->tc_b_all.assign(c.n_layers, nullptr);
        ctx->tc_maps.resize(c.n_layers);
        for (int l = 0; l < c.n_layers && st == ALORA_OK; ++l) {
            const size_t bytesA = na * 3 * d.RP * d.H * es, bytesB = na * (size_t)d.N * d.RP * es;
            alloc(&ctx->tc_a_all[l], bytesA);
            alloc(&ctx->tc_b_all[l], bytesB);
            if (st == ALORA_OK) {
                cudaError_t e2 = cudaMemset(ctx->tc_a_all[l], 0, bytesA);
                if (e2 == cudaSuccess) e2 = cudaMemset(ctx->tc_b_all[l], 0, bytesB);
                if (e2 != cudaSuccess) st = cuda_fail(ctx, e2, "cudaMemset");
                else if (!build_layer_maps(ctx, l)) st = ALORA_ERR_UNSUPPORTED;
            }
        }
    }
    if (d.I > 0) {
        const size_t chunk = std::min<size_t>(Tm, kMlpChunk);
        alloc(&ctx->d_act[0], Tm * std::max(d.H, d.Nq) * es);  // normed input / attention output
        alloc(&ctx->d_act[1], Tm * std::max(d.H, d.Nq) * es);
        alloc(&ctx->d_act[2], chunk * 2 * d.I * es);            // gate_up of one token chunk
        alloc(&ctx->d_act[3], chunk * d.I * es);                // swiglu output of one token chunk
    }
    if (st == ALORA_OK) {
        e = cudaMallocHost((void **)&ctx->h_status, 4);
        if (e != cudaSuccess) st = cuda_fail(ctx, e, "cudaMallocHost");
    }
    if (st == ALORA_OK) {
        e = cudaMemset(ctx->d_status, 0, 4);
        if (e == cudaSuccess) e = cudaMemset(ctx->d_adapters, 0, n_ad * sizeof(AdapterDev));
        if (e == cudaSuccess) e = cudaMemset(ctx->d_counts, 0, 64);
        if (e == cudaSuccess && ctx->d_rope_inv_freq) {
            std::vector<double> f((size_t)c.head_dim / 2);
            for (size_t i = 0; i < f.size(); ++i) f[i] = pow((double)c.rope_theta, -2.0 * (double)i / (double)c.head_dim);
            e = cudaMemcpy(ctx->d_rope_inv_freq, f.data(), f.size() * sizeof(double), cudaMemcpyHostToDevice);
        }
        if (e == cudaSuccess) {
            std::vector<int32_t> iota((size_t)c.max_requests + 1);
            for (size_t i = 0; i < iota.size(); ++i) iota[i] = (int32_t)i;
            e = cudaMemcpy(ctx->d_iota, iota.data(), iota.size() * 4, cudaMemcpyHostToDevice);
        }
        if (e != cudaSuccess) st = cuda_fail(ctx, e, "cudaMemset");
    }
    if (st != ALORA_OK) { alora_destroy(ctx); return st; }
    *out = ctx;
    return ALORA_OK;
}

alora_status alora_destroy(alora_ctx *ctx) {
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    cudaSetDevice(ctx->cfg.device);
    for (void *p : ctx->adapter_storage) if (p) cudaFree(p);
    for (void *p : ctx->tc_a_all) if (p) cudaFree(p);
    for (void *p : ctx->tc_b_all) if (p) cudaFree(p);
    for (auto *v : {&ctx->mlp_a_gu, &ctx->mlp_b_gu, &ctx->mlp_a_dn, &ctx->mlp_b_dn})
        for (void *p : *v) if (p) cudaFree(p);
    if (ctx->d_mlp_adapters) cudaFree(ctx->d_mlp_adapters);
    if (ctx->d_mlp_t) cudaFree(ctx->d_mlp_t);
    if (ctx->d_mlp_part) cudaFree(ctx->d_mlp_part);
    if (ctx->d_mlp_done) cudaFree(ctx->d_mlp_done);
    void *ptrs[] = {ctx->d_adapters, ctx->d_token_req, ctx->d_row_adapter, ctx->d_slot, ctx->d_tiles, ctx->d_counts,
                    ctx->d_seg_scratch, ctx->d_shrink_tiles, ctx->d_t_ready, ctx->d_t, ctx->d_qkv, ctx->d_status, ctx->d_act[0], ctx->d_act[1],
                    ctx->d_act[2], ctx->d_act[3], ctx->d_iota, ctx->d_attn_items, ctx->d_attn_off, ctx->d_split_items,
                    ctx->d_req_scratch, ctx->d_part_o, ctx->d_part_ml, ctx->d_group_done, ctx->d_row_delta,
                    ctx->d_skinny_part, ctx->d_skinny_t, ctx->d_skinny_meta, ctx->d_rope_inv_freq, ctx->d_prefix_groups,
                    ctx->d_attn_cta_start, ctx->d_attn_part_o, ctx->d_attn_part_ml};
    for (void *p : ptrs) if (p) cudaFree(p);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    for (ProfEvent &e : ctx->prof_events) { if (e.begin) cudaEventDestroy(e.begin); if (e.end) cudaEventDestroy(e.end); }
    delete ctx;
    return ALORA_OK;
}

alora_status alora_set_layer_weights(alora_ctx *ctx, int layer, const void *d_wqkv, const void *d_wo,
                                     const void *d_wgate_up, const void *d_wdown, const void *d_norm_attn,
                                     const void *d_norm_mlp) {
    if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers || !d_wqkv) return ALORA_ERR_INVALID_ARG;
    const void *all[] = {d_wqkv, d_wo, d_wgate_up, d_wdown, d_norm_attn, d_norm_mlp};
    for (const void *p : all) if (p && !aligned16(p)) return ALORA_ERR_INVALID_ARG;
    LayerWeights &lw = ctx->layers[layer];
    lw.wqkv = d_wqkv; lw.wo = d_wo; lw.wgate_up = d_wgate_up; lw.wdown = d_wdown;
    lw.norm_attn = d_norm_attn; lw.norm_mlp = d_norm_mlp;
    if (ctx->cfg.dtype == ALORA_DTYPE_BF16) {
        ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
        if (!build_layer_maps(ctx, layer)) return ALORA_ERR_UNSUPPORTED;
    }
    return ALORA_OK;
}

alora_status alora_register_adapter(alora_ctx *ctx, int adapter_id, int layer, int rank, float scale,
                                    const void *d_Aq, const void *d_Bq, const void *d_Ak, const void *d_Bk,
                                    const void *d_Av, const void *d_Bv, void *stream) {
    if (!ctx || !d_Aq || !d_Bq || !d_Ak || !d_Bk || !d_Av || !d_Bv) return ALORA_ERR_INVALID_ARG;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return ALORA_ERR_INVALID_ARG;
    if (adapter_id < 0 || adapter_id >= ctx->cfg.max_adapters) return ALORA_ERR_CAPACITY;
    if (rank < 1 || rank > ctx->cfg.max_rank) return ALORA_ERR_CAPACITY;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    const Dims &d = ctx->d;
    const size_t idx = (size_t)layer * ctx->cfg.max_adapters + adapter_id;
    const size_t bytesA = (size_t)3 * d.RP * d.H * ctx->esize, bytesB = (size_t)d.N * d.RP * ctx->esize;
    void *A, *B;
    if (ctx->cfg.dtype == ALORA_DTYPE_BF16) {
        // one slab per layer holds every adapter's rows, so that one tensor map addresses them all
        A = (char *)ctx->tc_a_all[layer] + (size_t)adapter_id * bytesA;
        B = (char *)ctx->tc_b_all[layer] + (size_t)adapter_id * bytesB;
    } else {
        if (!ctx->adapter_storage[2 * idx]) {
            ALORA_CUDA(ctx, cudaMalloc(&ctx->adapter_storage[2 * idx], bytesA));
            ALORA_CUDA(ctx, cudaMalloc(&ctx->adapter_storage[2 * idx + 1], bytesB));
        }
        A = ctx->adapter_storage[2 * idx]; B = ctx->adapter_storage[2 * idx + 1];
    }
    ctx->layer_has_adapter[layer] = 1;
    int n = launch_repack_adapter(ctx, rank, d_Aq, d_Bq, d_Ak, d_Bk, d_Av, d_Bv, A, B, s);
    AdapterDev rec{A, B, rank, (rank + 15) / 16 * 16, scale, 0};
    ctx->h_adapters[idx] = rec;
    // the table entry is a kernel argument of later launches on this stream: order the update after
    // earlier work by copying on the same stream (source is context-owned host memory).
    ALORA_CUDA(ctx, cudaMemcpyAsync(ctx->d_adapters + idx, &ctx->h_adapters[idx], sizeof(AdapterDev),
                                    cudaMemcpyHostToDevice, s));
    return finish(ctx, n);
}

// Rows of the down projection's A slab: every adapter's RP rows, rounded up to whole 128-row GEMM tiles.
static size_t mlp_dn_rows(const alora_ctx *ctx) {
    return ((size_t)std::max(1, ctx->cfg.max_adapters) * ctx->d.RP + 127) / 128 * 128;
}

alora_status alora_register_mlp_adapter(alora_ctx *ctx, int adapter_id, int layer, int rank, float scale,
                                        const void *d_Agate, const void *d_Bgate, const void *d_Aup, const void *d_Bup,
                                        const void *d_Adown, const void *d_Bdown, void *stream) {
    if (!ctx || !d_Agate || !d_Bgate || !d_Aup || !d_Bup || !d_Adown || !d_Bdown) return ALORA_ERR_INVALID_ARG;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return ALORA_ERR_INVALID_ARG;
    if (adapter_id < 0 || adapter_id >= ctx->cfg.max_adapters) return ALORA_ERR_CAPACITY;
    if (rank < 1 || rank > ctx->cfg.max_rank) return ALORA_ERR_CAPACITY;
    const Dims &d = ctx->d;
    if (ctx->cfg.dtype != ALORA_DTYPE_BF16 || d.I <= 0 || d.I % 256 != 0 || d.H % 256 != 0) return ALORA_ERR_UNSUPPORTED;
    // the per-row gate of a batch is the q/k/v adapter's: the MLP part extends an adapter registered on this layer
    if (ctx->h_adapters[(size_t)layer * ctx->cfg.max_adapters + adapter_id].rank == 0) return ALORA_ERR_NO_WEIGHTS;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    const size_t na = (size_t)std::max(1, ctx->cfg.max_adapters), es = ctx->esize;
    const size_t a_gu = (size_t)2 * d.RP * d.H * es, b_gu = (size_t)2 * d.I * d.RP * es;
    const size_t a_dn = (size_t)d.RP * d.I * es, b_dn = (size_t)d.H * d.RP * es;
    if (ctx->mlp_a_gu.empty()) {
        ctx->mlp_a_gu.assign(ctx->cfg.n_layers, nullptr); ctx->mlp_b_gu.assign(ctx->cfg.n_layers, nullptr);
        ctx->mlp_a_dn.assign(ctx->cfg.n_layers, nullptr); ctx->mlp_b_dn.assign(ctx->cfg.n_layers, nullptr);
        ctx->mlp_n_adapters.assign(ctx->cfg.n_layers, 0);
        ctx->h_mlp_adapters.assign((size_t)ctx->cfg.n_layers * na, MlpAdapterDev{0, 0.f});
    }
    if (!ctx->d_mlp_adapters) {
        const size_t bytes = ctx->h_mlp_adapters.size() * sizeof(MlpAdapterDev);
        ALORA_CUDA(ctx, cudaMalloc((void **)&ctx->d_mlp_adapters, bytes));
        ALORA_CUDA(ctx, cudaMemsetAsync(ctx->d_mlp_adapters, 0, bytes, s));
    }
    if (!ctx->d_mlp_t) {
        const size_t rows = (size_t)std::min(std::max(ctx->cfg.max_tokens, 1), kMlpChunk);
        const size_t rows_pad = (rows + 63) / 64 * 64;
        ALORA_CUDA(ctx, cudaMalloc(&ctx->d_mlp_t, rows * na * 2 * d.RP * es));
        // K-slice partials of the shrink kernel: room for four slices of the widest result, at most 64 MB (the
        // kernel takes fewer slices when a batch's partials would not fit)
        ctx->mlp_part_floats = std::min<size_t>(4 * rows_pad * na * 2 * d.RP, (size_t)16 << 20);
        ALORA_CUDA(ctx, cudaMalloc((void **)&ctx->d_mlp_part, ctx->mlp_part_floats * 4));
        ctx->mlp_done_ints = (int)((rows_pad / 64) * ((na * 2 * d.RP + 63) / 64));
        ALORA_CUDA(ctx, cudaMalloc((void **)&ctx->d_mlp_done, (size_t)ctx->mlp_done_ints * 4));
        ALORA_CUDA(ctx, cudaMemsetAsync(ctx->d_mlp_done, 0, (size_t)ctx->mlp_done_ints * 4, s));
    }
    if (!ctx->mlp_a_gu[layer]) {
        struct { void **p; size_t bytes; } slabs[] = {{&ctx->mlp_a_gu[layer], na * a_gu}, {&ctx->mlp_b_gu[layer], na * b_gu},
                                                      {&ctx->mlp_a_dn[layer], mlp_dn_rows(ctx) * d.I * es},
                                                      {&ctx->mlp_b_dn[layer], na * b_dn}};
        for (auto &sl : slabs) {
            ALORA_CUDA(ctx, cudaMalloc(sl.p, sl.bytes));
            ALORA_CUDA(ctx, cudaMemsetAsync(*sl.p, 0, sl.bytes, s));
        }
    }
    int n = 0, k;
    k = launch_repack_mlp(d_Agate, d_Aup, d_Bgate, d_Bup, 2, rank, d.RP, d.H, d.I,
                          (char *)ctx->mlp_a_gu[layer] + (size_t)adapter_id * a_gu,
                          (char *)ctx->mlp_b_gu[layer] + (size_t)adapter_id * b_gu, s);
    if (k < 0) return cuda_fail(ctx, cudaGetLastError(), "repack_mlp_kernel");
    n += k;
    k = launch_repack_mlp(d_Adown, nullptr, d_Bdown, nullptr, 1, rank, d.RP, d.I, d.H,
                          (char *)ctx->mlp_a_dn[layer] + (size_t)adapter_id * a_dn,
                          (char *)ctx->mlp_b_dn[layer] + (size_t)adapter_id * b_dn, s);
    if (k < 0) return cuda_fail(ctx, cudaGetLastError(), "repack_mlp_kernel");
    n += k;
    const size_t idx = (size_t)layer * na + adapter_id;
    ctx->h_mlp_adapters[idx] = MlpAdapterDev{(rank + 15) / 16 * 16, scale};
    ctx->mlp_n_adapters[layer] = std::max(ctx->mlp_n_adapters[layer], adapter_id + 1);
    ALORA_CUDA(ctx, cudaMemcpyAsync(ctx->d_mlp_adapters + idx, &ctx->h_mlp_adapters[idx], sizeof(MlpAdapterDev),
                                    cudaMemcpyHostToDevice, s));
    return finish(ctx, n);
}

alora_status alora_validate_batch(const alora_config *cfg, const int32_t *pos, const int32_t *a_req,
                                  const int32_t *ids, const int32_t *qsl, const int32_t *seq_lens,
                                  const int32_t *bt, int max_blocks, int num_pages, int T, int R) {
    if (!cfg || !pos || !qsl || !seq_lens || T < 0 || R < 0) return ALORA_ERR_INVALID_ARG;
    if (T > cfg->max_tokens || R > cfg->max_requests) return ALORA_ERR_CAPACITY;
    if (qsl[0] != 0 || qsl[R] != T) return ALORA_ERR_BAD_BATCH;
    const int ps = cfg->page_size;
    std::vector<uint8_t> owned;  // pages that some request may write
    if (bt) owned.assign((size_t)std::max(num_pages, 0), 0);
    for (int r = 0; r < R; ++r) {
        const int n_new = qsl[r + 1] - qsl[r];
        if (n_new < 0) return ALORA_ERR_BAD_BATCH;
        if (seq_lens[r] < n_new) return ALORA_ERR_BAD_BATCH;
        const int p_first = seq_lens[r] - n_new;
        for (int i = 0; i < n_new; ++i)
            if (pos[qsl[r] + i] != p_first + i) return ALORA_ERR_BAD_BATCH;
        if (ids) {
            if (ids[r] < -1 || ids[r] >= cfg->max_adapters) return ALORA_ERR_BAD_BATCH;
            if (ids[r] >= 0 && (!a_req || a_req[r] < 0)) return ALORA_ERR_BAD_BATCH;
        }
        if (bt) {
            const int nblk = (seq_lens[r] + ps - 1) / ps;
            if (nblk > max_blocks) return ALORA_ERR_BAD_BATCH;
            for (int b = 0; b < nblk; ++b) {
                const int page = bt[(size_t)r * max_blocks + b];
                if (page < 0 || page >= num_pages) return ALORA_ERR_PAGE_RANGE;
            }
            // pages that hold new positions are written: they must not be written by anyone else
            if (n_new > 0)
                for (int b = p_first / ps; b < nblk; ++b) {
                    const int page = bt[(size_t)r * max_blocks + b];
                    if (owned[page]) return ALORA_ERR_BAD_BATCH;
                    owned[page] = 1;
                }
        }
    }
    return ALORA_OK;
}

#define ALORA_BATCH(mode_)                                                                               \
    BatchArgs b{d_positions, d_activation_offsets, d_adapter_ids, d_query_start_loc, d_seq_lens,         \
                d_block_tables, max_blocks, num_pages, T, R, (mode_), 0}

alora_status alora_batch_metadata(alora_ctx *ctx, int mode, const int32_t *d_positions,
                                  const int32_t *d_activation_offsets, const int32_t *d_adapter_ids,
                                  const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                                  const int32_t *d_block_tables, int max_blocks, int num_pages, int T, int R,
                                  int32_t *d_token_request, int32_t *d_row_adapter, int32_t *d_slot_mapping,
                                  void *stream) {
    alora_status st = check_batch_args(ctx, T, R);
    if (st != ALORA_OK) return st;
    if (!d_positions || !d_query_start_loc || !d_seq_lens) return ALORA_ERR_INVALID_ARG;
    if (mode < ALORA_MODE_ALORA || mode > ALORA_MODE_BASE) return ALORA_ERR_INVALID_ARG;
    if (mode == ALORA_MODE_ALORA && d_adapter_ids && !d_activation_offsets) return ALORA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    ALORA_BATCH(mode);
    int n = launch_metadata(ctx, b, s, kMetaProjection);
    if (n < 0) return ALORA_ERR_UNSUPPORTED;
    if (T > 0) {
        if (d_token_request) ALORA_CUDA(ctx, cudaMemcpyAsync(d_token_request, ctx->d_token_req, (size_t)T * 4, cudaMemcpyDeviceToDevice, s));
        if (d_row_adapter) ALORA_CUDA(ctx, cudaMemcpyAsync(d_row_adapter, ctx->d_row_adapter, (size_t)T * 4, cudaMemcpyDeviceToDevice, s));
        if (d_slot_mapping) ALORA_CUDA(ctx, cudaMemcpyAsync(d_slot_mapping, ctx->d_slot, (size_t)T * 4, cudaMemcpyDeviceToDevice, s));
    }
    return finish(ctx, n);
}

alora_status alora_project_qkv(alora_ctx *ctx, int layer, int mode, const void *d_hidden,
                               const int32_t *d_positions, const int32_t *d_activation_offsets,
                               const int32_t *d_adapter_ids, const int32_t *d_query_start_loc,
                               const int32_t *d_seq_lens, int T, int R, void *d_qkv, void *stream) {
    alora_status st = check_batch_args(ctx, T, R);
    if (st != ALORA_OK) return st;
    if (!d_hidden || !d_positions || !d_query_start_loc || !d_seq_lens || !d_qkv) return ALORA_ERR_INVALID_ARG;
    if (!aligned16(d_hidden) || !aligned16(d_qkv)) return ALORA_ERR_INVALID_ARG;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return ALORA_ERR_INVALID_ARG;
    if (mode < ALORA_MODE_ALORA || mode > ALORA_MODE_BASE) return ALORA_ERR_INVALID_ARG;
    if (mode == ALORA_MODE_ALORA && d_adapter_ids && !d_activation_offsets) return ALORA_ERR_INVALID_ARG;
    if (!ctx->layers[layer].wqkv) return ALORA_ERR_NO_WEIGHTS;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    const int32_t *d_block_tables = nullptr; const int max_blocks = 0, num_pages = 0;
    ALORA_BATCH(mode);
    b.layer = layer;
    b.few_row = project_is_few_row(ctx, layer, T) ? 1 : 0;
    int n = launch_metadata(ctx, b, s, kMetaProjection), k;
    if (n < 0) return ALORA_ERR_UNSUPPORTED;
    if ((k = launch_project(ctx, layer, d_hidden, T, d_qkv, s, nullptr, 0, nullptr)) < 0) return ALORA_ERR_UNSUPPORTED;
    if (ctx->d_rope_inv_freq != nullptr) {   // the rows handed out are the rotated ones, as they would be cached
        int k2 = launch_rope(ctx, d_qkv, d_positions, T, nullptr, 0, s);
        if (k2 < 0) return ALORA_ERR_UNSUPPORTED;
        k += k2;
    }
    return finish(ctx, n + k);
}

alora_status alora_kv_append(alora_ctx *ctx, const void *d_qkv, const int32_t *d_positions,
                             const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                             const int32_t *d_block_tables, int max_blocks, int num_pages, int T, int R,
                             void *d_paged_kv, void *stream) {
    alora_status st = check_batch_args(ctx, T, R);
    if (st != ALORA_OK) return st;
    if (!d_qkv || !d_positions || !d_query_start_loc || !d_seq_lens || !d_block_tables || !d_paged_kv)
        return ALORA_ERR_INVALID_ARG;
    if (!aligned16(d_qkv) || !aligned16(d_paged_kv) || max_blocks <= 0 || num_pages <= 0) return ALORA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    const int32_t *d_activation_offsets = nullptr, *d_adapter_ids = nullptr;
    ALORA_BATCH(ALORA_MODE_BASE);
    int n = launch_metadata(ctx, b, s, kMetaProjection), k;
    if (n < 0) return ALORA_ERR_UNSUPPORTED;
    if ((k = launch_kv_append(ctx, d_qkv, T, num_pages, d_paged_kv, s)) < 0) return ALORA_ERR_UNSUPPORTED;
    return finish(ctx, n + k);
}

alora_status alora_attend(alora_ctx *ctx, const void *d_qkv, const int32_t *d_positions,
                          const int32_t *d_query_start_loc, const int32_t *d_seq_lens, const void *d_paged_kv,
                          const int32_t *d_block_tables, int max_blocks, int num_pages, int T, int R,
                          void *d_attn_out, void *stream) {
    alora_status st = check_batch_args(ctx, T, R);
    if (st != ALORA_OK) return st;
    if (!d_qkv || !d_positions || !d_query_start_loc || !d_seq_lens || !d_block_tables || !d_paged_kv || !d_attn_out)
        return ALORA_ERR_INVALID_ARG;
    if (!aligned16(d_qkv) || !aligned16(d_paged_kv) || !aligned16(d_attn_out) || max_blocks <= 0 || num_pages <= 0)
        return ALORA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    const int32_t *d_activation_offsets = nullptr, *d_adapter_ids = nullptr;
    ALORA_BATCH(ALORA_MODE_BASE);
    int n = launch_metadata(ctx, b, s), k;
    if (n < 0) return ALORA_ERR_UNSUPPORTED;
    if ((k = launch_attend(ctx, d_qkv, b, d_paged_kv, d_attn_out, s)) < 0) return ALORA_ERR_UNSUPPORTED;
    return finish(ctx, n + k);
}

static alora_status layer_entry(alora_ctx *ctx, int layer, int mode, const void *d_hidden,
                                const int32_t *d_positions, const int32_t *d_activation_offsets,
                                const int32_t *d_adapter_ids, const int32_t *d_query_start_loc,
                                const int32_t *d_seq_lens, void *d_paged_kv, const int32_t *d_block_tables,
                                int max_blocks, int num_pages, int T, int R, void *d_attn_out, void *stream,
                                bool one_token_per_request = false) {
    alora_status st = check_batch_args(ctx, T, R);
    if (st != ALORA_OK) return st;
    if (!d_hidden || !d_positions || !d_query_start_loc || !d_seq_lens || !d_block_tables || !d_paged_kv || !d_attn_out)
        return ALORA_ERR_INVALID_ARG;
    if (mode == ALORA_MODE_ALORA && d_adapter_ids && !d_activation_offsets) return ALORA_ERR_INVALID_ARG;
    if (!aligned16(d_hidden) || !aligned16(d_paged_kv) || !aligned16(d_attn_out) || max_blocks <= 0 || num_pages <= 0)
        return ALORA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    ALORA_BATCH(mode);
    b.all_small = one_token_per_request ? 1 : 0;
    return run_layer(ctx, layer, d_hidden, b, d_paged_kv, d_attn_out, s);
}

alora_status alora_prefill_layer(alora_ctx *ctx, int layer, const void *d_hidden, const int32_t *d_positions,
                                 const int32_t *d_activation_offsets, const int32_t *d_adapter_ids,
                                 const int32_t *d_query_start_loc, const int32_t *d_seq_lens, void *d_paged_kv,
                                 const int32_t *d_block_tables, int max_blocks, int num_pages, int T, int R,
                                 void *d_attn_out, void *stream) {
    return layer_entry(ctx, layer, ALORA_MODE_ALORA, d_hidden, d_positions, d_activation_offsets, d_adapter_ids,
                       d_query_start_loc, d_seq_lens, d_paged_kv, d_block_tables, max_blocks, num_pages, T, R,
                       d_attn_out, stream);
}

alora_status alora_full_lora_prefill_layer(alora_ctx *ctx, int layer, const void *d_hidden,
                                           const int32_t *d_positions, const int32_t *d_adapter_ids,
                                           const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                                           void *d_paged_kv, const int32_t *d_block_tables, int max_blocks,
                                           int num_pages, int T, int R, void *d_attn_out, void *stream) {
    return layer_entry(ctx, layer, ALORA_MODE_FULL_LORA, d_hidden, d_positions, nullptr, d_adapter_ids,
                       d_query_start_loc, d_seq_lens, d_paged_kv, d_block_tables, max_blocks, num_pages, T, R,
                       d_attn_out, stream);
}

alora_status alora_decode_step(alora_ctx *ctx, int layer, const void *d_hidden, const int32_t *d_positions,
                               const int32_t *d_activation_offsets, const int32_t *d_adapter_ids,
                               const int32_t *d_seq_lens, void *d_paged_kv, const int32_t *d_block_tables,
                               int max_blocks, int num_pages, int R, void *d_attn_out, void *stream) {
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    if (R < 0) return ALORA_ERR_INVALID_ARG;
    if (R > ctx->cfg.max_requests || R > ctx->cfg.max_tokens) return ALORA_ERR_CAPACITY;
    // query_start_loc of a decode batch is 0, 1, ..., R: kept in the context since alora_create
    return layer_entry(ctx, layer, ALORA_MODE_ALORA, d_hidden, d_positions, d_activation_offsets, d_adapter_ids,
                       ctx->d_iota, d_seq_lens, d_paged_kv, d_block_tables, max_blocks, num_pages, R, R, d_attn_out,
                       stream, /*one_token_per_request=*/true);
}

alora_status alora_forward_stack(alora_ctx *ctx, int mode, const void *d_hidden_in, const int32_t *d_positions,
                                 const int32_t *d_activation_offsets, const int32_t *d_adapter_ids,
                                 const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                                 void *const *h_paged_kv_layers, const int32_t *d_block_tables, int max_blocks,
                                 int num_pages, int T, int R, void *d_hidden_out, void *stream) {
    alora_status st = check_batch_args(ctx, T, R);
    if (st != ALORA_OK) return st;
    if (!d_hidden_in || !d_hidden_out || !d_positions || !d_query_start_loc || !d_seq_lens || !d_block_tables ||
        !h_paged_kv_layers)
        return ALORA_ERR_INVALID_ARG;
    if (mode < ALORA_MODE_ALORA || mode > ALORA_MODE_BASE) return ALORA_ERR_INVALID_ARG;
    if (mode == ALORA_MODE_ALORA && d_adapter_ids && !d_activation_offsets) return ALORA_ERR_INVALID_ARG;
    if (ctx->d.I <= 0) return ALORA_ERR_UNSUPPORTED;
    for (int l = 0; l < ctx->cfg.n_layers; ++l) {
        const LayerWeights &lw = ctx->layers[l];
        if (!lw.wqkv || !lw.wo || !lw.wgate_up || !lw.wdown || !lw.norm_attn || !lw.norm_mlp) return ALORA_ERR_NO_WEIGHTS;
        if (!h_paged_kv_layers[l] || !aligned16(h_paged_kv_layers[l])) return ALORA_ERR_INVALID_ARG;
    }
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    const Dims &d = ctx->d;
    ALORA_BATCH(mode);
    // one token per request (the decode entry passes the context's own 0, 1, ..., R as query_start_loc): every request
    // is on the few-row attention list, the tensor-core attention kernel has nothing to do and is not launched
    b.all_small = (d_query_start_loc == ctx->d_iota && T == R) ? 1 : 0;
    if (d_hidden_out != d_hidden_in && T > 0)
        ALORA_CUDA(ctx, cudaMemcpyAsync(d_hidden_out, d_hidden_in, (size_t)T * d.H * ctx->esize, cudaMemcpyDeviceToDevice, s));
    char *h = (char *)d_hidden_out;  // residual stream, updated in place
    int n = 0, k;
    // a launcher that returns < 0 has launched nothing (unsupported shape, failed tensor map or launch): the call
    // stops there with the residual stream as the completed steps left it
#define ALORA_STEP(call)                                                          \
    do {                                                                          \
        if ((k = (call)) < 0) {                                                   \
            ctx->launches += n;                                                   \
            cudaError_t e__ = cudaGetLastError();                                 \
            return e__ != cudaSuccess ? cuda_fail(ctx, e__, #call) : ALORA_ERR_UNSUPPORTED; \
        }                                                                         \
        n += k;                                                                   \
    } while (0)
    for (int l = 0; l < ctx->cfg.n_layers; ++l) {
        const LayerWeights &lw = ctx->layers[l];
        ALORA_STEP(launch_rmsnorm(ctx, h, lw.norm_attn, T, ctx->d_act[0], s));
        st = run_layer(ctx, l, ctx->d_act[0], b, h_paged_kv_layers[l], ctx->d_act[1], s);
        if (st != ALORA_OK) return st;
        ALORA_STEP(launch_linear(ctx, ctx->d_act[1], lw.wo, T, d.Nq, d.H, h, h, s));           // h += o_proj(attn)
        ALORA_STEP(launch_rmsnorm(ctx, h, lw.norm_mlp, T, ctx->d_act[0], s));
        for (int t0 = 0; t0 < T; t0 += kMlpChunk) {                                        // MLP, token chunks
            const int tc = std::min(kMlpChunk, T - t0);
            const char *xm = (const char *)ctx->d_act[0] + (size_t)t0 * d.H * ctx->esize;
            char *hc = h + (size_t)t0 * d.H * ctx->esize;
            // adapters on the MLP block: shrink against all of the layer's A rows (one launch), then the expand
            // step adds each open-gate row's delta in place (the row's applied adapter comes from this layer's
            // batch metadata; base-model batches and closed gates have none)
            const int n_mlp = (mode != ALORA_MODE_BASE && !ctx->mlp_n_adapters.empty()) ? ctx->mlp_n_adapters[l] : 0;
            const MlpAdapterDev *mlp_tab = n_mlp ? ctx->d_mlp_adapters + (size_t)l * std::max(1, ctx->cfg.max_adapters) : nullptr;
            ALORA_STEP(launch_linear(ctx, xm, lw.wgate_up, tc, d.H, 2 * d.I, ctx->d_act[2], nullptr, s));
            if (n_mlp) {
                const int tw = n_mlp * 2 * d.RP;
                ALORA_STEP(launch_mlp_shrink(ctx, xm, ctx->mlp_a_gu[l], tc, d.H, tw, ctx->d_mlp_t, ctx->d_mlp_part,
                                             ctx->mlp_part_floats, ctx->d_mlp_done, ctx->mlp_done_ints, s));
                ALORA_STEP(launch_mlp_expand(ctx, ctx->d_act[2], 2 * d.I, tc, ctx->d_mlp_t, tw, ctx->mlp_b_gu[l], 2 * d.I,
                                             d.I, 2, ctx->d_row_adapter + t0, mlp_tab, n_mlp, s));
            }
            ALORA_STEP(launch_swiglu(ctx, ctx->d_act[2], tc, ctx->d_act[3], s));
            ALORA_STEP(launch_linear(ctx, ctx->d_act[3], lw.wdown, tc, d.I, d.H, hc, hc, s));  // h += down(...)
            if (n_mlp) {
                const int tw = n_mlp * d.RP;
                ALORA_STEP(launch_mlp_shrink(ctx, ctx->d_act[3], ctx->mlp_a_dn[l], tc, d.I, tw, ctx->d_mlp_t, ctx->d_mlp_part,
                                             ctx->mlp_part_floats, ctx->d_mlp_done, ctx->mlp_done_ints, s));
                ALORA_STEP(launch_mlp_expand(ctx, hc, d.H, tc, ctx->d_mlp_t, tw, ctx->mlp_b_dn[l], d.H, d.H, 1,
                                             ctx->d_row_adapter + t0, mlp_tab, n_mlp, s));
            }
        }
    }
#undef ALORA_STEP
    return finish(ctx, n);
}

alora_status alora_prefix_groups(alora_ctx *ctx, int R, int32_t *d_group_first, int32_t *d_shared_keys, void *stream) {
    if (!ctx || R < 0 || !d_group_first || !d_shared_keys) return ALORA_ERR_INVALID_ARG;
    if (R > ctx->cfg.max_requests) return ALORA_ERR_CAPACITY;
    if (!ctx->d_prefix_groups) return ALORA_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    if (R > 0) {
        ALORA_CUDA(ctx, cudaMemcpyAsync(d_group_first, ctx->d_prefix_groups, (size_t)R * 4, cudaMemcpyDeviceToDevice, s));
        ALORA_CUDA(ctx, cudaMemcpyAsync(d_shared_keys, ctx->d_prefix_groups + R, (size_t)R * 4, cudaMemcpyDeviceToDevice, s));
    }
    return ALORA_OK;
}

alora_status alora_cow_tail_pages(alora_ctx *ctx, const int32_t *d_query_start_loc, const int32_t *d_seq_lens,
                                  int32_t *d_block_tables, int max_blocks, int num_pages, int R,
                                  const int32_t *d_fresh_pages, void *d_paged_kv, void *stream) {
    if (!ctx || R < 0 || !d_query_start_loc || !d_seq_lens || !d_block_tables || !d_fresh_pages || !d_paged_kv)
        return ALORA_ERR_INVALID_ARG;
    if (R > ctx->cfg.max_requests) return ALORA_ERR_CAPACITY;
    if (max_blocks <= 0 || num_pages <= 0 || !aligned16(d_paged_kv)) return ALORA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    return finish(ctx, launch_cow_tail_pages(ctx, d_query_start_loc, d_seq_lens, d_block_tables, max_blocks, num_pages, R,
                                             d_fresh_pages, d_paged_kv, s));
}

alora_status alora_decode_stack(alora_ctx *ctx, const void *d_hidden_in, const int32_t *d_positions,
                                const int32_t *d_activation_offsets, const int32_t *d_adapter_ids,
                                const int32_t *d_seq_lens, void *const *h_paged_kv_layers, const int32_t *d_block_tables,
                                int max_blocks, int num_pages, int R, void *d_hidden_out, void *stream) {
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    if (R < 0) return ALORA_ERR_INVALID_ARG;
    if (R > ctx->cfg.max_requests || R > ctx->cfg.max_tokens) return ALORA_ERR_CAPACITY;
    // one new token per request: query_start_loc is 0, 1, ..., R (kept in the context)
    return alora_forward_stack(ctx, ALORA_MODE_ALORA, d_hidden_in, d_positions, d_activation_offsets, d_adapter_ids,
                               ctx->d_iota, d_seq_lens, h_paged_kv_layers, d_block_tables, max_blocks, num_pages, R, R,
                               d_hidden_out, stream);
}

alora_status alora_profile_enable(alora_ctx *ctx, int on) {
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    ALORA_CUDA(ctx, cudaDeviceSynchronize());
    ctx->profiling = on != 0;
    if (on) ctx->prof_used = 0;
    return ALORA_OK;
}

alora_status alora_profile_read(alora_ctx *ctx, double *ms_by_kind, int64_t *groups_by_kind) {
    if (!ctx || !ms_by_kind || !groups_by_kind) return ALORA_ERR_INVALID_ARG;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    ALORA_CUDA(ctx, cudaDeviceSynchronize());
    for (int k = 0; k < ALORA_PROFILE_KINDS; ++k) { ms_by_kind[k] = 0.0; groups_by_kind[k] = 0; }
    for (size_t i = 0; i < ctx->prof_used; ++i) {
        const ProfEvent &e = ctx->prof_events[i];
        float ms = 0.f;
        ALORA_CUDA(ctx, cudaEventElapsedTime(&ms, e.begin, e.end));
        if (e.kind >= 0 && e.kind < ALORA_PROFILE_KINDS) { ms_by_kind[e.kind] += ms; groups_by_kind[e.kind] += 1; }
    }
    return ALORA_OK;
}

alora_status alora_get_status(alora_ctx *ctx, void *stream, int32_t *device_status) {
    if (!ctx || !device_status) return ALORA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    ALORA_CUDA(ctx, cudaMemcpyAsync(ctx->h_status, ctx->d_status, 4, cudaMemcpyDeviceToHost, s));
    ALORA_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, 4, s));
    ALORA_CUDA(ctx, cudaStreamSynchronize(s));
    *device_status = *ctx->h_status;
    return ALORA_OK;
}

}  // extern "C"
