// Rank-r shrink t = s A_k x on the tensor cores (the inner product of the low-rank delta of Eq. 5),
// split along the hidden dimension over a thread-block cluster.
//
// The shrink has few output tiles (one 128 x 192 tile per row tile: 3 blocks q/k/v of 64 padded rank
// columns) but a long contraction (the hidden dimension), so each row tile is given to a cluster of
// kShrinkSplits blocks.  Block c of the cluster contracts hidden columns of its own K range with
// tcgen05.mma into tensor memory, copies its fp32 partial tile into its shared memory, and after a
// cluster barrier reduces a 24-column slice of the tile over all blocks' shared memory (distributed
// shared memory loads) in the fixed order 0, 1, ..., 7.  The order does not depend on timing, so the
// result is run-to-run deterministic.  Row tiles without an applied adapter are skipped by their
// whole cluster.
#include <algorithm>

#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

constexpr int kShrinkSplits = 8;        // blocks per cluster = K ranges per row tile
constexpr int kShrinkBM = 128;          // rows per tile
constexpr int kShrinkBN = 192;          // 3 blocks x 64 padded rank columns
constexpr int kShrinkBK = 64;
constexpr int kShrinkStages = 4;
constexpr int kShrinkThreads = 192;     // warp 0 TMA, warp 1 MMA, warps 2-5 epilogue / reduction
constexpr int kShrinkSlice = kShrinkBN / kShrinkSplits;  // 24 columns reduced by each block

struct ShrinkArgs {
    const ProjTile *tiles;
    const int32_t *n_row_tiles;
    const AdapterDev *adapters;
    __nv_bfloat16 *t;   // [tokens][192]
    int K;              // hidden
    int32_t *status;
};

struct ShrinkSmem {
    static constexpr int kABytes = kShrinkBM * kShrinkBK * 2;
    static constexpr int kBBytes = kShrinkBN * kShrinkBK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kRingBytes = kShrinkStages * kStageBytes;        // 160 KB; reused as the fp32 partial tile
    static constexpr int kPartialBytes = kShrinkBN * kShrinkBM * 4;       // [192 columns][128 rows] fp32
    static constexpr int kBarOffset = kRingBytes;
    static constexpr int kTotal = kBarOffset + 256 + 1024;
    static_assert(kPartialBytes <= kRingBytes, "partial tile must fit in the ring");
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_dsmem_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

__global__ void __cluster_dims__(kShrinkSplits, 1, 1) __launch_bounds__(kShrinkThreads, 1)
shrink_tcgen05_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmA,
                      const ShrinkArgs a) {
    using S = ShrinkSmem;
    // the whole cluster takes the same decision: blockIdx.y selects the row tile
    if ((int)blockIdx.y >= *a.n_row_tiles || a.n_row_tiles[5] != 0) return;  // [5]: batch takes the row-wise route
    const ProjTile tile = a.tiles[blockIdx.y];
    if (tile.adapter < 0) return;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + S::kBarOffset);
    const uint32_t bar0 = smem_base + S::kBarOffset;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kShrinkStages + s); };
    const uint32_t acc_bar = bar0 + 8u * (2 * kShrinkStages);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * kShrinkStages + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * kShrinkStages + 2);
    float *partial = reinterpret_cast<float *>(smem_al);  // [192][128], aliases the ring once the MMAs are done

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kTmemCols = 256;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kShrinkStages; ++s) { tc::mbar_init(full_bar(s), 1); tc::mbar_init(empty_bar(s), 1); }
        tc::mbar_init(acc_bar, 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32((const void *)tmem_slot), kTmemCols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // this block's K range, in 64-column blocks
    const uint32_t crank = cluster_ctarank();
    const int kb_all = (a.K + kShrinkBK - 1) / kShrinkBK;
    const int kb_per = (kb_all + kShrinkSplits - 1) / kShrinkSplits;
    const int kb0 = (int)crank * kb_per;
    const int nkb = max(0, min(kb_per, kb_all - kb0));

    if (warp == 0) {
        if (lane == 0) {
            tc::tma_prefetch_desc(&tmX); tc::tma_prefetch_desc(&tmA);
            bool ok = true;
            int kc = 0;
            for (; kc < nkb; ++kc) {
                const int s = kc % kShrinkStages;
                if (!tc::mbar_wait(empty_bar(s), ((kc / kShrinkStages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                const uint32_t sa = smem_base + s * S::kStageBytes, sb = sa + S::kABytes;
                tc::mbar_arrive_expect_tx(full_bar(s), S::kStageBytes);
                tc::tma_load_2d(sa, &tmX, full_bar(s), (kb0 + kc) * kShrinkBK, tile.row_start);
                tc::tma_load_2d(sb, &tmA, full_bar(s), (kb0 + kc) * kShrinkBK, tile.adapter * kShrinkBN);
            }
            if (!ok) {
                // copies already in flight must land before the shared memory is reused or released
                for (int i = max(0, kc - kShrinkStages); i < kc; ++i) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(full_bar(i % kShrinkStages), (i / kShrinkStages) & 1) &&
                           clock64() - t0 < tc::kWaitCycleLimit) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && nkb > 0) {
            constexpr uint32_t idesc = tc::idesc_bf16_f32(kShrinkBM, kShrinkBN);
            for (int kc = 0; kc < nkb; ++kc) {
                const int s = kc % kShrinkStages;
                if (!tc::mbar_wait(full_bar(s), (kc / kShrinkStages) & 1, abort_flag)) break;
                tc::tc_fence_after();
                const uint32_t sa = smem_base + s * S::kStageBytes, sb = sa + S::kABytes;
                const uint64_t da = tc::smem_desc_k_sw128(sa), db = tc::smem_desc_k_sw128(sb);
                for (int k = 0; k < kShrinkBK / 16; ++k)
                    tc::mma_bf16(tmem_base, da + 2 * k, db + 2 * k, idesc, (kc | k) != 0 ? 1u : 0u);
                tc::mma_commit(empty_bar(s));
            }
            tc::mma_commit(acc_bar);  // arrives once every MMA issued above has completed (also after a failed wait)
        }
    } else {
        // epilogue warps: this block's partial tile -> shared memory, column-major so that the 32 rows of
        // a warp are 32 consecutive words
        const int q = warp & 3;
        const int r = q * 32 + lane;
        bool have = nkb > 0;
        if (have) have = tc::mbar_wait(acc_bar, 0, abort_flag);
        tc::tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < kShrinkBN; c += 32) {
            uint32_t v[32];
            if (have) {
                tc::tmem_ld_32x32(tmem_base + c + ((uint32_t)(q * 32) << 16), v);
                tc::tmem_ld_wait();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
#pragma unroll
            for (int e = 0; e < 32; ++e) partial[(c + e) * kShrinkBM + r] = __uint_as_float(v[e]);
        }
        tc::tc_fence_before();
    }

    __syncthreads();
    cluster_sync_all();  // every block's partial tile is in its shared memory

    if (warp >= 2) {
        const int q = warp & 3;
        const int r = q * 32 + lane;
        const float scale = a.adapters[tile.adapter].scale;
        const int c0 = (int)crank * kShrinkSlice;
        float acc[kShrinkSlice];
#pragma unroll
        for (int j = 0; j < kShrinkSlice; ++j) acc[j] = 0.f;
#pragma unroll 1
        for (uint32_t src = 0; src < (uint32_t)kShrinkSplits; ++src) {  // fixed order: deterministic sum
#pragma unroll
            for (int j = 0; j < kShrinkSlice; ++j)
                acc[j] += ld_dsmem_f32(tc::smem_u32(partial + (c0 + j) * kShrinkBM + r), src);
        }
        if (r < tile.row_count) {
            __nv_bfloat16 *orow = a.t + (size_t)(tile.row_start + r) * kShrinkBN + c0;
#pragma unroll
            for (int j = 0; j < kShrinkSlice; j += 8) {
                uint4 o;
                o.x = tc::pack_bf16(acc[j] * scale, acc[j + 1] * scale);
                o.y = tc::pack_bf16(acc[j + 2] * scale, acc[j + 3] * scale);
                o.z = tc::pack_bf16(acc[j + 4] * scale, acc[j + 5] * scale);
                o.w = tc::pack_bf16(acc[j + 6] * scale, acc[j + 7] * scale);
                *reinterpret_cast<uint4 *>(orow + j) = o;
            }
        }
    }

    cluster_sync_all();  // no block may release its shared memory while another still reads it
    if (threadIdx.x == 0 && *abort_flag) report(a.status, ALORA_ERR_TIMEOUT);
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// t = s A x for the adapter row tiles of the current batch.  Returns false if the launch could not be set up.
bool launch_shrink_tc(alora_ctx *ctx, const CUtensorMap &tmX, const CUtensorMap &tmA, const AdapterDev *adapters,
                      int K, int max_row_tiles, cudaStream_t s) {
    static bool attr_set[64] = {};
    const int dev = ctx->cfg.device;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(shrink_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ShrinkSmem::kTotal) != cudaSuccess)
            return false;
        attr_set[dev] = true;
    }
    ShrinkArgs a{ctx->d_tiles, ctx->d_counts, adapters, (__nv_bfloat16 *)ctx->d_t, K, ctx->d_status};
    dim3 grid(kShrinkSplits, std::max(1, max_row_tiles));
    shrink_tcgen05_kernel<<<grid, kShrinkThreads, ShrinkSmem::kTotal, s>>>(tmX, tmA, a);
    return true;
}

}  // namespace alora
