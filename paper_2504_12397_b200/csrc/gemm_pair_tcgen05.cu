// Gated multi-adapter q/k/v projection (Eq. 2 / Eq. 5) for batches of many rows: 256 x 192 output tiles.
//
// Same computation and the same work list as gemm_tcgen05.cu's tile route (row tiles of up to 128 rows segmented by
// (adapter, gate); t = s A_k x from leading "shrink items" of the same launch; an adapter tile appends t B_k^T to its
// K loop; optional KV append in the epilogue), with another tile shape: a block owns TWO row tiles that share the
// W tile, 56 KB of operands per 64-wide K block for 8 x 96 tensor-pipe cycles instead of 48 KB for 4 x 128, i.e.
// 1.3 x the flops per operand byte (one SM cannot fill its shared memory fast enough for the 128 x 256 tile), and
// 192-wide column tiles so that 2048 rows x 6144 columns make 256 tiles: two rounds over 148 blocks at 86 %.
// The two row tiles accumulate in the two halves of tensor memory (not double-buffered; the next item's loads run
// under the epilogue and its MMAs start on a half as soon as that half has been drained).
//
// A 192-wide column tile can straddle the q | k | v boundaries of the fused row.  The expand step therefore takes
// one K block per (row tile, q/k/v block that the column tile touches): A = that block's 64 (padded-rank) columns
// of t, B = the adapter's B rows of that block through a 3-D tensor map (rank column, row inside the block,
// adapter) whose out-of-range rows read as zero, so the columns of the other block get no contribution.
//
//   warp 0   TMA producer (4 slots of 56 KB)      warp 1   MMA issuer (whole warp walks, elected lane issues)
//   warps 2-5 / 6-9  epilogue of the first / second row tile: tcgen05.ld one row per thread, bf16, 16-byte stores,
//              KV append, or t for shrink items
// All waits are bounded; on expiry ALORA_ERR_TIMEOUT is recorded and the block leaves normally.
#include <algorithm>

#include "alora_internal.h"
#include "tc_common.cuh"
#include "claim_order.h"

namespace alora {

namespace {
constexpr int kBNp = 192, kBKp = 64, kStagesP = 4, kThreadsP = 320;   // producer, issuer, 2 x 4 epilogue warps
constexpr int kTensorRP = 64;                      // the tensor path stores adapters padded to 64 rank columns
constexpr int kHalfAp = 128 * kBKp * 2;            // one row tile's x (or t) block: 16 KB
constexpr int kBBytesP = kBNp * kBKp * 2;          // 24 KB
constexpr int kStageBytesP = 2 * kHalfAp + kBBytesP;
constexpr int kBarOffP = kStagesP * kStageBytesP;
constexpr int kItemRingOffP = kBarOffP + 256;
constexpr int kSmemTotalP = kItemRingOffP + 128 + 1024;
constexpr int kShrinkColsP = 3 * kTensorRP;        // 192 columns of t = one column tile

struct PairArgs {
    const ProjTile *tiles;
    const int32_t *n_row_tiles;
    int N, K, Nq, Nkv;
    __nv_bfloat16 *out;
    int ldo;
    const AdapterDev *adapters;
    const int32_t *shrink_tiles;    // row-tile indices that have an adapter ...
    const int32_t *n_shrink_tiles;  // ... and their count
    int32_t *t_ready;               // [row tile] epilogue warps that have published their part of t
    __nv_bfloat16 *t_out;           // [tokens][192]
    // KV append fused into the epilogue (nullptr: off), as in gemm_tcgen05.cu
    __nv_bfloat16 *kv_pool;
    const int32_t *slot_map;
    int kv_hd_shift, kv_heads, kv_page_size, kv_num_pages;
    int32_t *item_counters;         // [2] next unclaimed work item of the launch, blocks that have finished
    int32_t *status;
};

__device__ __forceinline__ int ld_acquire_p(const int32_t *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void tma_load_3d_p(uint32_t smem_dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                              int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// One work item: a shrink item (row tile m[0] only) or two row tiles (m[1] = -1: none) x one column tile.
struct PairItem {
    ProjTile t[2];
    int m[2];
    int n0;
    bool shrink;
};
__device__ __forceinline__ PairItem decode_pair(const PairArgs &a, int item, int n_shrink, int n_m, int n_n) {
    PairItem g;
    g.t[1].row_start = 0; g.t[1].row_count = 0; g.t[1].adapter = -1; g.t[1].pad_ = 0;
    if (item < n_shrink) {
        g.m[0] = a.shrink_tiles[item];
        g.m[1] = -1;
        g.n0 = 0;
        g.shrink = true;
    } else {
        const int j = item - n_shrink;
        g.m[0] = 2 * (j / n_n);
        g.m[1] = g.m[0] + 1 < n_m ? g.m[0] + 1 : -1;
        g.n0 = (j % n_n) * kBNp;
        g.shrink = false;
    }
    g.t[0] = a.tiles[g.m[0]];
    if (g.m[1] >= 0) g.t[1] = a.tiles[g.m[1]];
    return g;
}
// first row of q/k/v block `blk` in the fused row, and one past its last
__device__ __forceinline__ int blk_start(const PairArgs &a, int blk) { return blk == 0 ? 0 : (blk == 1 ? a.Nq : a.Nq + a.Nkv); }
__device__ __forceinline__ int blk_end(const PairArgs &a, int blk) { return blk == 0 ? a.Nq : (blk == 1 ? a.Nq + a.Nkv : a.N); }
// does the column tile at n0 touch block blk?
__device__ __forceinline__ bool touches(const PairArgs &a, int n0, int blk) {
    return n0 < blk_end(a, blk) && n0 + kBNp > blk_start(a, blk);
}

__global__ void __launch_bounds__(kThreadsP, 1)
gemm_pair_tcgen05_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                         const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmS,
                         const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1,
                         const __grid_constant__ CUtensorMap tmB2, const PairArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + kBarOffP);
    // barrier words: full[4], empty[4], acc_full, acc_empty[2] (one per half), drain
    const uint32_t bar0 = smem_base + kBarOffP;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kStagesP + s); };
    const uint32_t accf_bar = bar0 + 8u * (2 * kStagesP);
    auto acce_bar = [&](int h) { return bar0 + 8u * (2 * kStagesP + 1 + h); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kStagesP + 3);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * kStagesP + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * kStagesP + 5);

    tc::ItemRing ring{smem_base + kItemRingOffP, reinterpret_cast<volatile int *>(smem_al + kItemRingOffP + 16 * tc::kItemSlots)};
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        ring.init(9);   // the issuing warp and the eight epilogue warps
        for (int s = 0; s < kStagesP; ++s) { tc::mbar_init(full_bar(s), 1); tc::mbar_init(empty_bar(s), 1); }
        tc::mbar_init(accf_bar, 1);
        tc::mbar_init(acce_bar(0), 4); tc::mbar_init(acce_bar(1), 4);
        tc::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32((const void *)tmem_slot), 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    tc::grid_dep_launch();
    tc::grid_dep_wait();   // the metadata step's lists, the activations: all written by earlier kernels of the stream

    const int n_m = *a.n_row_tiles;
    const int n_n = (a.N + kBNp - 1) / kBNp;
    const int n_shrink = *a.n_shrink_tiles;
    const int total = n_shrink + ((n_m + 1) / 2) * n_n;
    const int kb_main = (a.K + kBKp - 1) / kBKp;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------ TMA producer ------------------------------
            tc::tma_prefetch_desc(&tmX); tc::tma_prefetch_desc(&tmW);
            uint32_t kc = 0;        // ring slots filled so far
            bool ok = true;
            // Order of this block's items.  Shrink items (the head of the list) are claimed from a global counter by
            // the blocks (see below which), one at a time, until none is left; only then does the block walk its
            // projection items, which are dealt out by block index as if the shrink items sat at list positions
            // 0 .. n_shrink-1 (what the first blocks to start normally take).  A projection item that waits for its row
            // tile's t therefore waits for a shrink item that a RUNNING block has claimed, however few blocks are
            // resident; and in the usual case every block keeps the items (and the L2 neighbours) it always had.
            bool shrink_phase = n_shrink > 0;
            int stat = (int)blockIdx.x;
            if (shrink_phase && !claims_at_once((int)blockIdx.x, n_shrink)) {
                // The blocks with the lowest indices have a free place in their list and normally take the shrink items
                // within a microsecond.  The others look on for a short while (about 30 us) and join the claiming
                // only if the shrink items are still not all taken by then (blocks that have not been scheduled).
                const long long t0 = clock64();
                while (ld_acquire_p(a.item_counters) < n_shrink && clock64() - t0 < 60000) {}
                if (ld_acquire_p(a.item_counters) >= n_shrink) shrink_phase = false;
            }
            while (ok) {
                int item = -1;
                if (shrink_phase) {
                    item = atomicAdd(a.item_counters, 1);
                    if (item >= n_shrink) { shrink_phase = false; item = -1; }
                }
                if (!shrink_phase && item < 0) {
                    item = next_dealt_item(stat, n_shrink, total, (int)gridDim.x);
                }
                if (!ring.put(item, abort_flag)) { ok = false; break; }
                if (item < 0) break;
                const PairItem g = decode_pair(a, item, n_shrink, n_m, n_n);
                const bool two = g.m[1] >= 0;
                for (int kb = 0; kb < kb_main && ok; ++kb, ++kc) {
                    const int s = kc % kStagesP;
                    if (!tc::mbar_wait(empty_bar(s), ((kc / kStagesP) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t sa = smem_base + s * kStageBytesP, sb = sa + 2 * kHalfAp;
                    tc::mbar_arrive_expect_tx(full_bar(s), (two ? 2 : 1) * kHalfAp + kBBytesP);
                    tc::tma_load_2d(sa, &tmX, full_bar(s), kb * kBKp, g.t[0].row_start);
                    if (two) tc::tma_load_2d(sa + kHalfAp, &tmX, full_bar(s), kb * kBKp, g.t[1].row_start);
                    if (g.shrink) tc::tma_load_2d(sb, &tmS, full_bar(s), kb * kBKp, g.t[0].adapter * kShrinkColsP);
                    else tc::tma_load_2d(sb, &tmW, full_bar(s), kb * kBKp, g.n0);
                }
                if (g.shrink) continue;
                // expand: per row tile with an adapter, one K block per q/k/v block the column tile touches
                for (int h = 0; h < 2 && ok; ++h) {
                    if (g.m[h] < 0 || g.t[h].adapter < 0) continue;
                    // t of this row tile is written by a shrink item (earlier in the list, so claimed by a running
                    // block): wait until its four epilogue warps have published, then order the TMA read after it
                    const long long t0 = clock64();
                    while (ld_acquire_p(a.t_ready + g.m[h]) < 4) {
                        if (*abort_flag || clock64() - t0 > tc::kWaitCycleLimit) { *abort_flag = 1; ok = false; break; }
                    }
                    if (!ok) break;
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    for (int blk = 0; blk < 3 && ok; ++blk) {
                        if (!touches(a, g.n0, blk)) continue;
                        const int s = kc % kStagesP;
                        if (!tc::mbar_wait(empty_bar(s), ((kc / kStagesP) & 1) ^ 1, abort_flag)) { ok = false; break; }
                        const uint32_t sa = smem_base + s * kStageBytesP, sb = sa + 2 * kHalfAp;
                        tc::mbar_arrive_expect_tx(full_bar(s), kHalfAp + kBBytesP);
                        tc::tma_load_2d(sa + h * kHalfAp, &tmT, full_bar(s), blk * kTensorRP, g.t[h].row_start);
                        tma_load_3d_p(sb, blk == 0 ? &tmB0 : (blk == 1 ? &tmB1 : &tmB2), full_bar(s), 0,
                                      g.n0 - blk_start(a, blk), g.t[h].adapter);
                        ++kc;
                    }
                }
            }
            if (!ok) {
                // give copies already in flight time to land before the block's shared memory is released
                const uint32_t first = kc > (uint32_t)kStagesP ? kc - kStagesP : 0;
                for (uint32_t i = first; i < kc; ++i) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(full_bar(i % kStagesP), (i / kStagesP) & 1) &&
                           clock64() - t0 < tc::kWaitCycleLimit) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        const bool leader = tc::elect_one();
        auto wait_all = [&](uint32_t bar, uint32_t parity) {
            return __all_sync(0xffffffffu, tc::mbar_wait(bar, parity, abort_flag));
        };
        constexpr uint32_t idesc = tc::idesc_bf16_f32(128, kBNp);
        uint32_t kc = 0, it = 0;
        bool ok = true;
        for (;; ++it) {
            const int item = ring.take(abort_flag);
            if (item < 0) { ok = item == -1; break; }
            const PairItem g = decode_pair(a, item, n_shrink, n_m, n_n);
            const bool two = g.m[1] >= 0;
            for (int kb = 0; kb < kb_main && ok; ++kb, ++kc) {
                const int s = kc % kStagesP;
                if (!wait_all(full_bar(s), (kc / kStagesP) & 1)) { ok = false; break; }
                tc::tc_fence_after();
                const uint32_t sa = smem_base + s * kStageBytesP;
                const uint64_t db = tc::smem_desc_k_sw128(sa + 2 * kHalfAp);
                const uint64_t da0 = tc::smem_desc_k_sw128(sa), da1 = tc::smem_desc_k_sw128(sa + kHalfAp);
                // a half's accumulator must have been drained by the previous item's epilogue before its first MMA
                if (kb == 0 && !wait_all(acce_bar(0), (it & 1) ^ 1)) { ok = false; break; }
                if (leader) {
#pragma unroll
                    for (int k = 0; k < kBKp / 16; ++k)
                        tc::mma_bf16(tmem_base, da0 + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                }
                if (kb == 0 && !wait_all(acce_bar(1), (it & 1) ^ 1)) { ok = false; break; }
                if (leader) {
                    if (two) {
#pragma unroll
                        for (int k = 0; k < kBKp / 16; ++k)
                            tc::mma_bf16(tmem_base + 256, da1 + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    tc::mma_commit(empty_bar(s));  // slot reusable once these MMAs have read it
                }
            }
            if (!ok) break;
            if (!g.shrink) {
                for (int h = 0; h < 2 && ok; ++h) {
                    if (g.m[h] < 0 || g.t[h].adapter < 0) continue;
                    const int steps = a.adapters[g.t[h].adapter].rpad / 16;
                    for (int blk = 0; blk < 3 && ok; ++blk) {
                        if (!touches(a, g.n0, blk)) continue;
                        const int s = kc % kStagesP;
                        if (!wait_all(full_bar(s), (kc / kStagesP) & 1)) { ok = false; break; }
                        tc::tc_fence_after();
                        const uint32_t sa = smem_base + s * kStageBytesP;
                        const uint64_t db = tc::smem_desc_k_sw128(sa + 2 * kHalfAp);
                        const uint64_t da = tc::smem_desc_k_sw128(sa + h * kHalfAp);
                        if (leader) {
                            for (int k = 0; k < steps; ++k) tc::mma_bf16(tmem_base + h * 256, da + 2 * k, db + 2 * k, idesc, 1u);
                            tc::mma_commit(empty_bar(s));
                        }
                        ++kc;
                    }
                }
                if (!ok) break;
            }
            if (leader) tc::mma_commit(accf_bar);      // accumulators complete
        }
        if (!ok && leader) {
            tc::mma_commit(drain_bar);                 // wait (bounded) for tensor-core work still in flight
            const long long t0 = clock64();
            while (!tc::mbar_try_wait(drain_bar, 0) && clock64() - t0 < tc::kWaitCycleLimit) {}
        }
    } else {
        // ------------------------------ epilogue (warps 2..5: first row tile, warps 6..9: second) ------------------------------
        const int q = warp & 3;           // tensor-memory lane quarter this warp may read
        const int my_h = (warp - 2) >> 2; // the half of tensor memory (row tile of the pair) this warp drains
        uint32_t it = 0;
        bool ok = true;
        for (;; ++it) {
            const int item = ring.take(abort_flag);
            if (item < 0) break;
            const PairItem g = decode_pair(a, item, n_shrink, n_m, n_n);
            if (!tc::mbar_wait(accf_bar, it & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            const int r = q * 32 + lane;
            if (g.shrink && my_h == 1) {   // a shrink item has one row tile only
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(acce_bar(1));
                continue;
            }
            if (g.shrink) {
                // t = s A x of this row tile: 192 columns, scaled, rounded to bf16
                const ProjTile t = g.t[0];
                const bool row_ok = r < t.row_count;
                const float scale = a.adapters[t.adapter].scale;
                __nv_bfloat16 *trow = a.t_out + (size_t)(t.row_start + r) * kShrinkColsP;
#pragma unroll 1
                for (int c = 0; c < kShrinkColsP; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(tmem_base + c + ((uint32_t)(q * 32) << 16), v);
                    tc::tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 o;
                            o.x = tc::pack_bf16(__uint_as_float(v[8 * j]) * scale, __uint_as_float(v[8 * j + 1]) * scale);
                            o.y = tc::pack_bf16(__uint_as_float(v[8 * j + 2]) * scale, __uint_as_float(v[8 * j + 3]) * scale);
                            o.z = tc::pack_bf16(__uint_as_float(v[8 * j + 4]) * scale, __uint_as_float(v[8 * j + 5]) * scale);
                            o.w = tc::pack_bf16(__uint_as_float(v[8 * j + 6]) * scale, __uint_as_float(v[8 * j + 7]) * scale);
                            *reinterpret_cast<uint4 *>(trow + c + 8 * j) = o;
                        }
                    }
                }
                tc::tc_fence_before();
                // publish: the rows are read by other blocks through TMA (async proxy)
                asm volatile("fence.proxy.async.global;" ::: "memory");
                __threadfence();
                __syncwarp();
                if (lane == 0) {
                    atomicAdd(a.t_ready + g.m[0], 1);
                    tc::mbar_arrive(acce_bar(0));
                }
                continue;
            }
            {
                const int h = my_h;
                if (g.m[h] >= 0) {
                    const ProjTile t = g.t[h];
                    const bool row_ok = r < t.row_count;
                    __nv_bfloat16 *orow = a.out + (size_t)(t.row_start + r) * a.ldo + g.n0;
                    // fused KV append: where this row's k / v columns go in the page pool
                    int kv_page = -1, kv_row = 0;
                    if (a.kv_pool != nullptr && row_ok && g.n0 + kBNp > a.Nq) {
                        const int slot = a.slot_map[t.row_start + r];
                        if (slot >= 0) {
                            kv_page = slot / a.kv_page_size;
                            kv_row = slot % a.kv_page_size;
                            if (kv_page >= a.kv_num_pages) { report(a.status, ALORA_ERR_PAGE_RANGE); kv_page = -1; }
                        }
                    }
#pragma unroll 1
                    for (int c = 0; c < kBNp; c += 32) {
                        uint32_t v[32];
                        tc::tmem_ld_32x32(tmem_base + h * 256 + c + ((uint32_t)(q * 32) << 16), v);
                        tc::tmem_ld_wait();
                        if (row_ok) {
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (g.n0 + c + 8 * j >= a.N) break;
                                uint4 o;
                                o.x = tc::pack_bf16(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1]));
                                o.y = tc::pack_bf16(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
                                o.z = tc::pack_bf16(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
                                o.w = tc::pack_bf16(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
                                *reinterpret_cast<uint4 *>(orow + c + 8 * j) = o;
                                const int kcol = g.n0 + c + 8 * j - a.Nq;   // column inside [k | v]
                                if (kv_page >= 0 && kcol >= 0) {
                                    const int plane = kcol >= a.Nkv ? 1 : 0, c2 = kcol - plane * a.Nkv;
                                    const int head = c2 >> a.kv_hd_shift, dd = c2 & ((1 << a.kv_hd_shift) - 1);
                                    __nv_bfloat16 *dst = a.kv_pool +
                                        ((((size_t)kv_page * 2 + plane) * a.kv_heads + head) * a.kv_page_size + kv_row << a.kv_hd_shift) + dd;
                                    *reinterpret_cast<uint4 *>(dst) = o;
                                }
                            }
                        }
                    }
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(acce_bar(h));   // this half may be overwritten
            }
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(a.status, ALORA_ERR_TIMEOUT);
    if (threadIdx.x == 0) tc::item_counter_release(a.item_counters);
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, 512);
    }
}
}  // namespace

bool make_tensor_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t ld,
                          uint32_t box_rows);  // gemm_tcgen05.cu
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn tensor_map_encoder();  // gemm_tcgen05.cu

// The per-layer tensor maps of this kernel: W in boxes of 192 rows, and for each of the q / k / v blocks the B
// rows of all adapters as (rank column, row inside the block, adapter).
bool build_pair_maps(alora_ctx *ctx, int layer) {
    const Dims &d = ctx->d;
    TcLayerMaps &lm = ctx->tc_maps[layer];
    const LayerWeights &lw = ctx->layers[layer];
    bool ok = true;
    if (lw.wqkv) ok &= make_tensor_map_bf16(&lm.wqkv192, lw.wqkv, d.N, d.H, d.H, kBNp);
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    const size_t na = (size_t)std::max(1, ctx->cfg.max_adapters);
    const int starts[3] = {0, d.Nq, d.Nq + d.Nkv}, rows[3] = {d.Nq, d.Nkv, d.Nkv};
    for (int blk = 0; blk < 3; ++blk) {
        cuuint64_t dims[3] = {(cuuint64_t)kTensorRP, (cuuint64_t)rows[blk], (cuuint64_t)na};
        cuuint64_t strides[2] = {(cuuint64_t)kTensorRP * 2, (cuuint64_t)d.N * kTensorRP * 2};
        cuuint32_t box[3] = {(cuuint32_t)kTensorRP, (cuuint32_t)kBNp, 1};
        cuuint32_t es[3] = {1, 1, 1};
        void *base = (char *)ctx->tc_b_all[layer] + (size_t)starts[blk] * kTensorRP * 2;
        ok &= enc(&lm.b_blk[blk], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    return ok;
}

// Returns the kernels launched (1), 0 when the batch is better served by the 128-row kernel (nothing launched) or
// -1 on error.  Only for batches too large for the row-wise route (the decision must not depend on the mode, so
// that rows with a closed gate come out bit-identical to the base-only projection of the same batch).
int launch_project_pair_tc(alora_ctx *ctx, int layer, const void *hidden, int T, void *qkv, cudaStream_t s,
                           void *kv_pool, int num_pages) {
    const Dims &d = ctx->d;
    if (T <= kRowwiseMaxTokens || d.H % 8 != 0 || d.N % 8 != 0 || d.Nq % 8 != 0 || d.Nkv % 8 != 0) return 0;
    const int G = ctx->sm_count;
    const int n_n = (d.N + kBNp - 1) / kBNp, n_n256 = (d.N + 255) / 256;
    const int items = ((T + 255) / 256) * n_n, items128 = ((T + 127) / 128) * n_n256;
    const double eff = (double)items / ((double)((items + G - 1) / G) * G);
    const double eff128 = (double)items128 / ((double)((items128 + G - 1) / G) * G);
    if (eff * 1.25 < eff128) return 0;
    const TcLayerMaps &lm = ctx->tc_maps[layer];
    CUtensorMap tmX, tmT;
    if (!make_tensor_map_bf16(&tmX, hidden, T, d.H, d.H, 128)) return -1;
    if (!make_tensor_map_bf16(&tmT, ctx->d_t, ctx->cfg.max_tokens, 3 * kTensorRP, 3 * kTensorRP, 128)) return -1;
    static bool attr_set[64] = {};
    const int dev = ctx->cfg.device;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(gemm_pair_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotalP) !=
            cudaSuccess)
            return -1;
        attr_set[dev] = true;
    }
    PairArgs g{};
    g.tiles = ctx->d_tiles; g.n_row_tiles = ctx->d_counts; g.N = d.N; g.K = d.H; g.Nq = d.Nq; g.Nkv = d.Nkv;
    g.out = (__nv_bfloat16 *)qkv; g.ldo = d.N;
    g.adapters = ctx->d_adapters + (size_t)layer * ctx->cfg.max_adapters;
    g.shrink_tiles = ctx->d_shrink_tiles; g.n_shrink_tiles = ctx->d_counts + 2;
    g.t_ready = ctx->d_t_ready; g.t_out = (__nv_bfloat16 *)ctx->d_t;
    g.item_counters = ctx->d_counts + 10;
    if (kv_pool != nullptr) {
        int shift = 0;
        while ((1 << shift) < d.hd) ++shift;
        g.kv_pool = (__nv_bfloat16 *)kv_pool; g.slot_map = ctx->d_slot; g.kv_hd_shift = shift; g.kv_heads = d.Hkv;
        g.kv_page_size = d.page; g.kv_num_pages = num_pages;
    }
    g.status = ctx->d_status;
    const int max_row_tiles = std::min(std::min(ctx->max_tiles, T / 128 + 2 * ctx->cfg.max_requests + 2), T);
    const int max_items = max_row_tiles + ((max_row_tiles + 1) / 2) * n_n;
    const int grid = std::max(1, std::min(G, max_items));
    if (launch_kernel(gemm_pair_tcgen05_kernel, dim3(grid), dim3(kThreadsP), kSmemTotalP, s, true, tmX, lm.wqkv192, tmT,
                      lm.a_all, lm.b_blk[0], lm.b_blk[1], lm.b_blk[2], g) != cudaSuccess)
        return -1;
    return 1;
}

}  // namespace alora
