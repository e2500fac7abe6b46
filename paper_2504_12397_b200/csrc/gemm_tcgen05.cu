// bf16 dense contraction on the 5th-generation tensor cores: out[rows][N] = act[rows][K] . W[N][K]^T
// with the aLoRA delta fused in.
//
// One persistent block per SM, three roles:
//   warp 0 (one lane)  TMA producer: streams 128 x 64 activation tiles and BN x 64 weight tiles
//                      (128-byte swizzle) through a 4-deep shared-memory ring;
//   warp 1 (one lane)  MMA issuer: tcgen05.mma 128 x BN x 16 steps into one of two fp32 accumulators in
//                      tensor memory, releasing ring slots and publishing accumulators via
//                      tcgen05.commit;
//   warps 2-5          epilogue: tcgen05.ld the accumulator (one row per thread), optional residual
//                      add / scale, round to bf16, 16-byte row-predicated stores.  The second
//                      accumulator lets the next tile's main loop overlap this epilogue.
//
// Row tiles come from the batch-metadata step: all rows of a tile have the same applied adapter.
// For a tile with an adapter the main K loop (the base term W x of Eq. 5) is followed by one more
// K block whose operands are t = s A x (rows of the tile) and the adapter's B rows of this column
// tile, i.e. the delta s B (A x) is accumulated by the same tensor-core instruction stream.  Tiles
// without an adapter execute exactly the base-only sequence: that is what makes gated-off rows
// bit-identical to a base-only call (Prop. 1).
//
// Where t = s A x comes from.  With 256-wide column tiles the shrink is part of this kernel: the first
// work items of the launch are one "shrink item" per adapter row tile, whose B operand is the adapter's
// 192 A rows (q, k, v blocks, rank padded to 64) and whose epilogue writes t and then raises a per-tile
// ready counter in global memory.  A projection item of an adapter tile waits (bounded) for that
// counter before it loads t for its extra K block; since every block walks the item list in increasing
// order and shrink items come first, the block that owns a shrink item never waits before finishing it.
// With 128-wide column tiles the shrink runs as a separate cluster split-K kernel (shrink_tcgen05.cu).
// No split-K, no atomics in the arithmetic: results are run-to-run deterministic.
//
// Every wait is bounded (tc::mbar_wait); on expiry the block records ALORA_ERR_TIMEOUT, drains its
// outstanding copies and tensor-core work with bounded waits, frees its tensor memory and returns.
#include "alora_internal.h"
#include "tc_common.cuh"
#include "claim_order.h"

namespace alora {

constexpr int kBM = 128;      // rows per tile (UMMA M)
constexpr int kBK = 64;       // K elements per ring slot (one 128-byte swizzle row)
constexpr int kGemmThreads = 192;
constexpr int kTensorRP = 64; // the tensor path stores adapters padded to 64 rank columns

struct GemmArgs {
    // Bytes one copy of the activation tile brings (0: the full 128-row tile).  A batch of at most 64 rows uses a
    // 64-row box: the other half of the tile in shared memory is never filled, the accumulator rows it feeds are
    // never read, and the shared-memory fill of a stage, which bounds this shape, drops by a third.
    int a_tile_bytes;
    const ProjTile *tiles;        // nullptr: dense row tiles 0..ceil(M/128)-1, no adapters
    const int32_t *n_row_tiles;   // device count of `tiles` entries (when tiles != nullptr)
    int M, N, K;
    __nv_bfloat16 *out;
    int ldo;
    const __nv_bfloat16 *residual;  // optional, same layout as out, may alias it
    const AdapterDev *adapters;     // this layer's adapter table (expand), or nullptr
    int Nq, Nkv;                    // block boundaries of the fused output row (expand)
    int total_adapter_rows;         // rows per adapter in the B_all map (= N of the layer)
    const int32_t *shrink_tiles;    // fused shrink: row-tile indices that have an adapter ...
    const int32_t *n_shrink_tiles;  // ... and their count (nullptr: no shrink items in this launch)
    int32_t *t_ready;               // [row tile] epilogue warps that have published their part of t
    __nv_bfloat16 *t_out;           // [tokens][192]
    // Row-wise route (batches of few rows per tile): when *rowwise_flag is set by the metadata step the launch
    // ignores the tile list, walks dense row tiles without any adapter, and its epilogue adds row_delta[row][n]
    // (fp32, made by lora_delta_rows_kernel) to the rows whose row_adapter is >= 0.
    const int32_t *rowwise_flag;
    const float *row_delta;
    const int32_t *row_adapter;
    // KV append fused into the epilogue (nullptr: off): columns Nq .. N of row t also go to the paged cache,
    // pool[page][plane][head][row in page][:] with page * page_size + row = slot_map[t] (-1: token rejected, skipped)
    __nv_bfloat16 *kv_pool;
    const int32_t *slot_map;
    int kv_hd_shift, kv_heads, kv_page_size, kv_num_pages;
    int32_t *item_counters;         // [2] next unclaimed work item of the launch, blocks that have finished
    int32_t *status;
};

template <int BN>
struct GemmSmem {
    // ring depth: 4 slots of 32 .. 48 KB for the wide tiles; the 64-wide tile of the skinny (few rows, weight
    // streaming) case gets 8 slots of 24 KB so that enough bytes are in flight per SM
    static constexpr int kStages = BN <= 64 ? 8 : 4;
    static constexpr int kABytes = kBM * kBK * 2;
    static constexpr int kBBytes = BN * kBK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kBarOffset = kStages * kStageBytes;
    static constexpr int kItemRingOffset = kBarOffset + 256;
    static constexpr int kTotal = kItemRingOffset + 128 + 1024;  // barriers, item ring, slack for 1024-byte alignment
};

__device__ __forceinline__ ProjTile load_tile(const GemmArgs &a, int m, bool dense) {
    if (a.tiles && !dense) return a.tiles[m];
    ProjTile t;
    t.row_start = m * kBM;
    t.row_count = min(kBM, a.M - m * kBM);
    t.adapter = -1;
    t.pad_ = 0;
    return t;
}

constexpr int kShrinkCols = 3 * kTensorRP;  // 192 columns of t: q, k, v blocks of 64 padded rank columns

// Work item `item` of a launch: shrink items first (one per adapter row tile), then the projection's
// (row tile, column tile) pairs.
struct GemmItem {
    ProjTile t;
    int m;        // row-tile index
    int n0;       // first output column (projection items)
    bool shrink;
};
__device__ __forceinline__ GemmItem decode_item(const GemmArgs &a, int item, int n_shrink, int n_n, int BN, bool dense) {
    GemmItem g;
    if (item < n_shrink) {
        g.m = a.shrink_tiles[item];
        g.n0 = 0;
        g.shrink = true;
    } else {
        const int j = item - n_shrink;
        g.m = j / n_n;
        g.n0 = (j % n_n) * BN;
        g.shrink = false;
    }
    g.t = load_tile(a, g.m, dense);
    return g;
}

__device__ __forceinline__ int ld_acquire(const int32_t *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmL,
                    const __grid_constant__ CUtensorMap tmS, const GemmArgs a) {
    using S = GemmSmem<BN>;
    constexpr int kStages = S::kStages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + S::kBarOffset);
    // barrier words: full[kStages], empty[kStages], acc_full[2], acc_empty[2], drain
    const uint32_t bar0 = smem_base + S::kBarOffset;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
    auto accf_bar = [&](int i) { return bar0 + 8u * (2 * kStages + i); };
    auto acce_bar = [&](int i) { return bar0 + 8u * (2 * kStages + 2 + i); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kStages + 4);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * kStages + 5);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * kStages + 6);
    tc::ItemRing ring{smem_base + S::kItemRingOffset,
                      reinterpret_cast<volatile int *>(smem_al + S::kItemRingOffset + 16 * tc::kItemSlots)};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kTmemCols = (2 * BN <= 256) ? 256 : 512;

    if (threadIdx.x == 0) {
        ring.init(5);   // the issuing warp and the four epilogue warps
        for (int s = 0; s < kStages; ++s) { tc::mbar_init(full_bar(s), 1); tc::mbar_init(empty_bar(s), 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(accf_bar(i), 1); tc::mbar_init(acce_bar(i), 4); }
        tc::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32((const void *)tmem_slot), kTmemCols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    tc::grid_dep_launch();
    tc::grid_dep_wait();   // the metadata step's lists, the activations: all written by earlier kernels of the stream

    const bool dense = a.rowwise_flag != nullptr && *a.rowwise_flag != 0;
    const int n_m = (a.tiles && !dense) ? *a.n_row_tiles : (a.M + kBM - 1) / kBM;
    const int n_n = (a.N + BN - 1) / BN;
    const int n_shrink = (BN >= kShrinkCols && a.n_shrink_tiles && !dense) ? *a.n_shrink_tiles : 0;
    const int total = n_shrink + n_m * n_n;
    const int kb_main = (a.K + kBK - 1) / kBK;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------ TMA producer ------------------------------
            tc::tma_prefetch_desc(&tmA); tc::tma_prefetch_desc(&tmB);
            const uint32_t a_bytes = a.a_tile_bytes ? (uint32_t)a.a_tile_bytes : (uint32_t)S::kABytes;
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
                while (ld_acquire(a.item_counters) < n_shrink && clock64() - t0 < 60000) {}
                if (ld_acquire(a.item_counters) >= n_shrink) shrink_phase = false;
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
                const GemmItem g = decode_item(a, item, n_shrink, n_n, BN, dense);
                const ProjTile t = g.t;
                const int n0 = g.n0;
                const int extra = (!g.shrink && t.adapter >= 0) ? 1 : 0;
                for (int kb = 0; kb < kb_main + extra; ++kb, ++kc) {
                    const int s = kc % kStages;
                    if (!tc::mbar_wait(empty_bar(s), ((kc / kStages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t sa = smem_base + s * S::kStageBytes, sb = sa + S::kABytes;
                    if (g.shrink) {
                        tc::mbar_arrive_expect_tx(full_bar(s), a_bytes + kShrinkCols * kBK * 2);
                        tc::tma_load_2d(sa, &tmA, full_bar(s), kb * kBK, t.row_start);
                        tc::tma_load_2d(sb, &tmS, full_bar(s), kb * kBK, t.adapter * kShrinkCols);
                    } else if (kb < kb_main) {
                        tc::mbar_arrive_expect_tx(full_bar(s), a_bytes + S::kBBytes);
                        tc::tma_load_2d(sa, &tmA, full_bar(s), kb * kBK, t.row_start);
                        tc::tma_load_2d(sb, &tmB, full_bar(s), kb * kBK, n0);
                    } else {
                        if (n_shrink > 0) {
                            // t of this row tile is written by a shrink item, which comes earlier in the list and has
                            // therefore been claimed by a running block: wait until its four epilogue warps have
                            // published, then order the TMA read after their writes
                            const long long t0 = clock64();
                            while (ld_acquire(a.t_ready + g.m) < 4) {
                                if (*abort_flag || clock64() - t0 > tc::kWaitCycleLimit) { *abort_flag = 1; ok = false; break; }
                            }
                            if (!ok) break;
                            fence_proxy_async_global();
                        }
                        tc::mbar_arrive_expect_tx(full_bar(s), S::kStageBytes);
                        const int blk = n0 < a.Nq ? 0 : (n0 < a.Nq + a.Nkv ? 1 : 2);
                        tc::tma_load_2d(sa, &tmT, full_bar(s), blk * kTensorRP, t.row_start);
                        tc::tma_load_2d(sb, &tmL, full_bar(s), 0, t.adapter * a.total_adapter_rows + n0);
                    }
                }
            }
            if (!ok) {
                // give copies already in flight time to land before the block's shared memory is released
                const uint32_t first = kc > (uint32_t)kStages ? kc - kStages : 0;
                for (uint32_t i = first; i < kc; ++i) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(full_bar(i % kStages), (i / kStages) & 1) &&
                           clock64() - t0 < tc::kWaitCycleLimit) {}
                }
            }
        }
    } else if (warp == 1) {
        {
            // ------------------------------ MMA issuer ------------------------------
            // The whole warp walks the schedule (uniform control flow keeps descriptors and loop state in uniform
            // registers, which is what lets the issue rate reach the tensor pipe's); one elected lane issues the
            // tensor-core instructions and their commits.
            const bool leader = tc::elect_one();
            auto wait_all = [&](uint32_t bar, uint32_t parity) {
                return __all_sync(0xffffffffu, tc::mbar_wait(bar, parity, abort_flag));
            };
            constexpr uint32_t idesc_main = tc::idesc_bf16_f32(kBM, BN);
            constexpr uint32_t idesc_shrink = tc::idesc_bf16_f32(kBM, BN >= kShrinkCols ? kShrinkCols : BN);
            uint32_t kc = 0, it = 0;
            bool ok = true;
            while (ok) {
                const int item = ring.take(abort_flag);
                if (item < 0) { ok = item == -1; break; }
                const GemmItem g = decode_item(a, item, n_shrink, n_n, BN, dense);
                const ProjTile t = g.t;
                const int extra = (!g.shrink && t.adapter >= 0) ? 1 : 0;
                const int extra_steps = extra ? a.adapters[t.adapter].rpad / 16 : 0;
                const uint32_t idesc = g.shrink ? idesc_shrink : idesc_main;
                const uint32_t acc = it & 1;
                if (!wait_all(acce_bar(acc), ((it >> 1) & 1) ^ 1)) { ok = false; break; }
                tc::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < kb_main + extra; ++kb, ++kc) {
                    const int s = kc % kStages;
                    if (!wait_all(full_bar(s), (kc / kStages) & 1)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t sa = smem_base + s * S::kStageBytes, sb = sa + S::kABytes;
                    const uint64_t da = tc::smem_desc_k_sw128(sa), db = tc::smem_desc_k_sw128(sb);
                    if (leader) {
                        if (kb < kb_main) {
#pragma unroll
                            for (int k = 0; k < kBK / 16; ++k)
                                tc::mma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                        } else {
                            for (int k = 0; k < extra_steps; ++k) tc::mma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, 1u);
                        }
                        tc::mma_commit(empty_bar(s));  // slot reusable once these MMAs have read it
                    }
                }
                if (!ok) break;
                if (leader) tc::mma_commit(accf_bar(acc));      // accumulator complete
                ++it;
            }
            if (!ok && leader) {
                tc::mma_commit(drain_bar);          // wait (bounded) for tensor-core work still in flight
                const long long t0 = clock64();
                while (!tc::mbar_try_wait(drain_bar, 0) && clock64() - t0 < tc::kWaitCycleLimit) {}
            }
        }
    } else {
        // ------------------------------ epilogue (warps 2..5) ------------------------------
        const int q = warp & 3;  // tensor-memory lane quarter this warp may read
        uint32_t it = 0;
        bool ok = true;
        while (ok) {
            const int item = ring.take(abort_flag);
            if (item < 0) break;
            const GemmItem g = decode_item(a, item, n_shrink, n_n, BN, dense);
            const ProjTile t = g.t;
            const int n0 = g.n0;
            const uint32_t acc = it & 1;
            if (!tc::mbar_wait(accf_bar(acc), (it >> 1) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            const int r = q * 32 + lane;
            const bool row_ok = r < t.row_count;
            if (g.shrink) {
                // t = s A x of this row tile: 192 columns, scaled, rounded to bf16
                const float scale = a.adapters[t.adapter].scale;
                __nv_bfloat16 *trow = a.t_out + (size_t)(t.row_start + r) * kShrinkCols;
#pragma unroll 1
                for (int c = 0; c < kShrinkCols && c < BN; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(tmem_base + acc * BN + c + ((uint32_t)(q * 32) << 16), v);
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
                fence_proxy_async_global();
                __threadfence();
                __syncwarp();
                if (lane == 0) {
                    atomicAdd(a.t_ready + g.m, 1);
                    tc::mbar_arrive(acce_bar(acc));
                }
                ++it;
                continue;
            }
            __nv_bfloat16 *orow = a.out + (size_t)(t.row_start + r) * a.ldo + n0;
            const __nv_bfloat16 *rrow = a.residual ? a.residual + (size_t)(t.row_start + r) * a.ldo + n0 : nullptr;
            // row-wise delta: only rows with an applied adapter add anything (a gated-off row never sees "+ 0")
            const float *drow = (dense && row_ok && a.row_adapter[t.row_start + r] >= 0)
                                    ? a.row_delta + (size_t)(t.row_start + r) * a.N + n0 : nullptr;
            // fused KV append: where this row's k / v columns go in the page pool
            int kv_page = -1, kv_row = 0;
            if (a.kv_pool != nullptr && row_ok && n0 + BN > a.Nq) {
                const int slot = a.slot_map[t.row_start + r];
                if (slot >= 0) {
                    kv_page = slot / a.kv_page_size;
                    kv_row = slot % a.kv_page_size;
                    if (kv_page >= a.kv_num_pages) { report(a.status, ALORA_ERR_PAGE_RANGE); kv_page = -1; }
                }
            }
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t v[32];
                tc::tmem_ld_32x32(tmem_base + acc * BN + c + ((uint32_t)(q * 32) << 16), v);
                tc::tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (n0 + c + 8 * j >= a.N) break;
                        float f[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[8 * j + e]);
                        if (drow) {
                            const float4 d0 = *reinterpret_cast<const float4 *>(drow + c + 8 * j);
                            const float4 d1 = *reinterpret_cast<const float4 *>(drow + c + 8 * j + 4);
                            f[0] += d0.x; f[1] += d0.y; f[2] += d0.z; f[3] += d0.w;
                            f[4] += d1.x; f[5] += d1.y; f[6] += d1.z; f[7] += d1.w;
                        }
                        if (rrow) {
                            const uint4 rv = *reinterpret_cast<const uint4 *>(rrow + c + 8 * j);
                            const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 b2 = *reinterpret_cast<const __nv_bfloat162 *>(&rw[e]);
                                f[2 * e] += __low2float(b2);
                                f[2 * e + 1] += __high2float(b2);
                            }
                        }
                        uint4 o;
                        o.x = tc::pack_bf16(f[0], f[1]); o.y = tc::pack_bf16(f[2], f[3]);
                        o.z = tc::pack_bf16(f[4], f[5]); o.w = tc::pack_bf16(f[6], f[7]);
                        *reinterpret_cast<uint4 *>(orow + c + 8 * j) = o;
                        const int kc = n0 + c + 8 * j - a.Nq;   // column inside [k | v]
                        if (kv_page >= 0 && kc >= 0) {
                            const int plane = kc >= a.Nkv ? 1 : 0, c2 = kc - plane * a.Nkv;
                            const int head = c2 >> a.kv_hd_shift, dd = c2 & ((1 << a.kv_hd_shift) - 1);
                            __nv_bfloat16 *dst = a.kv_pool +
                                ((((size_t)kv_page * 2 + plane) * a.kv_heads + head) * a.kv_page_size + kv_row << a.kv_hd_shift) + dd;
                            *reinterpret_cast<uint4 *>(dst) = o;
                        }
                    }
                }
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(acce_bar(acc));  // accumulator may be overwritten
            ++it;
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(a.status, ALORA_ERR_TIMEOUT);
    if (threadIdx.x == 0) tc::item_counter_release(a.item_counters);
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- host side -------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// Row-major bf16 matrix [rows][cols] (row pitch ld elements) viewed in boxes of 64 columns x box_rows
// rows, 128-byte swizzle, out-of-range elements read as zero.
bool make_tensor_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t ld,
                          uint32_t box_rows) {
    EncodeTiledFn fn = tensor_map_encoder();
    if (!fn || !base || rows == 0 || cols == 0) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || (ld * 2) % 16 != 0 || box_rows == 0 || box_rows > 256) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
static bool launch_gemm_bn(alora_ctx *ctx, const CUtensorMap &tmA, const CUtensorMap &tmB, const CUtensorMap &tmT,
                           const CUtensorMap &tmL, const CUtensorMap &tmS, const GemmArgs &args, int max_items,
                           cudaStream_t s) {
    static bool attr_set[64] = {};  // one per instantiation
    const int dev = ctx->cfg.device;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(gemm_tcgen05_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 GemmSmem<BN>::kTotal) != cudaSuccess)
            return false;
        attr_set[dev] = true;
    }
    const int grid = std::max(1, std::min(ctx->sm_count, max_items));
    if (launch_kernel(gemm_tcgen05_kernel<BN>, dim3(grid), dim3(kGemmThreads), GemmSmem<BN>::kTotal, s, true, tmA, tmB, tmT, tmL,
                      tmS, args) != cudaSuccess)
        return false;
    return true;
}

int launch_lora_delta_rows(alora_ctx *ctx, int layer, const void *hidden, int T, cudaStream_t s);  // simt_kernels.cu
bool launch_shrink_tc(alora_ctx *ctx, const CUtensorMap &tmX, const CUtensorMap &tmA, const AdapterDev *adapters,
                      int K, int max_row_tiles, cudaStream_t s);  // shrink_tcgen05.cu

// Picks the column-tile width: 256 when the q/k/v block boundaries allow it, else 128; 64 for batches of at most
// 128 rows, where the kernel streams the weights once and more, narrower tiles put more SMs to work.
static int pick_bn(int N, int Nq, int Nkv, bool lora, int T) {
    if (T <= kBM && N >= 64 * 48 && Nq % 64 == 0 && Nkv % 64 == 0) return 64;
    if (lora) {
        if (Nq % 256 == 0 && Nkv % 256 == 0) return 256;
        if (Nq % 128 == 0 && Nkv % 128 == 0) return 128;
        return 0;
    }
    return (N % 256 == 0 || N > 1024) ? 256 : 128;
}

// q/k/v projection of one layer on the tensor cores: shrink (t = s A x on adapter tiles), then the
// base GEMM with the expand step fused.  Returns kernels launched, or -1 when the shape is unsupported.
int launch_project_pair_tc(alora_ctx *ctx, int layer, const void *hidden, int T, void *qkv, cudaStream_t s,
                           void *kv_pool, int num_pages);  // gemm_pair_tcgen05.cu

bool skinny_route(const alora_ctx *ctx, int T, int N, int K, bool lora, int Nq, int Nkv);   // gemm_skinny_tcgen05.cu
int launch_skinny_tc(alora_ctx *ctx, const void *x, const CUtensorMap &tmW, const CUtensorMap *tmA16,
                     const AdapterDev *adapters, const void *b_all, int T, int K, int N, int Nq, int Nkv, void *out,
                     const void *residual, void *kv_pool, int num_pages, cudaStream_t s);

// Whether the q/k/v projection of a batch of T rows on this layer takes the few-row route (the batch-metadata step
// then prepares that route's adapter facts instead of row tiles).
bool project_is_few_row(const alora_ctx *ctx, int layer, int T) {
    if (ctx->cfg.dtype != ALORA_DTYPE_BF16 || layer < 0 || layer >= ctx->cfg.n_layers) return false;
    const Dims &d = ctx->d;
    return skinny_route(ctx, T, d.N, d.H, ctx->layer_has_adapter[layer] != 0, d.Nq, d.Nkv);
}

int launch_project_tc(alora_ctx *ctx, int layer, const void *hidden, int T, void *qkv, cudaStream_t s, void *kv_pool,
                      int num_pages) {
    if (T == 0) return 0;
    const Dims &d = ctx->d;
    const bool have_adapters = ctx->layer_has_adapter[layer];
    if (skinny_route(ctx, T, d.N, d.H, have_adapters, d.Nq, d.Nkv)) {   // at most 128 rows: weight-streaming route
        ProfScope prof(ctx, KK_PROJECT, s);
        const TcLayerMaps &lm = ctx->tc_maps[layer];
        const AdapterDev *ads = ctx->d_adapters + (size_t)layer * ctx->cfg.max_adapters;
        return launch_skinny_tc(ctx, hidden, lm.wqkv[1], have_adapters ? &lm.a_all16 : nullptr,
                                have_adapters ? ads : nullptr, ctx->tc_b_all[layer], T, d.H, d.N, d.Nq, d.Nkv, qkv, nullptr,
                                kv_pool, num_pages, s);
    }
    if (ctx->tc_maps[layer].pair_ok) {   // many rows: two row tiles per block, 192-wide column tiles
        ProfScope prof(ctx, KK_PROJECT, s);
        const int r = launch_project_pair_tc(ctx, layer, hidden, T, qkv, s, kv_pool, num_pages);
        if (r != 0) return r;
    }
    const int BN = pick_bn(d.N, d.Nq, d.Nkv, true, T);
    if (BN == 0 || d.H % 8 != 0) return -1;
    CUtensorMap tmX, tmTt, tmX64;
    if (!make_tensor_map_bf16(&tmX, hidden, T, d.H, d.H, kBM)) return -1;
    const bool half_box = T <= kBM / 2;   // see GemmArgs::a_tile_bytes
    if (half_box && !make_tensor_map_bf16(&tmX64, hidden, T, d.H, d.H, kBM / 2)) return -1;
    if (!make_tensor_map_bf16(&tmTt, ctx->d_t, ctx->cfg.max_tokens, 3 * kTensorRP, 3 * kTensorRP, kBM)) return -1;
    const TcLayerMaps &lm = ctx->tc_maps[layer];
    const AdapterDev *ads = ctx->d_adapters + (size_t)layer * ctx->cfg.max_adapters;
    // every row tile holds at least one row; a request contributes at most two partial tiles
    const int max_row_tiles = std::min(std::min(ctx->max_tiles, T / kBM + 2 * ctx->cfg.max_requests + 2), T);
    int n = 0;
    // Batches whose row tiles would hold only a few rows each may be switched to the row-wise route by the
    // metadata step (a device-side decision): the delta rows are prepared here, and both kernels read the flag.
    const bool may_rowwise = have_adapters && T <= kRowwiseMaxTokens && ctx->d_row_delta != nullptr;
    if (may_rowwise) {
        ProfScope prof(ctx, KK_SHRINK, s);
        n += launch_lora_delta_rows(ctx, layer, hidden, T, s);
    }
    const bool fuse_shrink = have_adapters && BN == 256;
    // (a batch of at most kRowwiseAlwaysRows rows always takes the row-wise route when it has adapter rows: no shrink
    // launch; otherwise the shrink kernel looks at the flag itself)
    if (have_adapters && !fuse_shrink && !(may_rowwise && T <= kRowwiseAlwaysRows)) {
        ProfScope prof(ctx, KK_SHRINK, s);
        if (!launch_shrink_tc(ctx, tmX, lm.a_all, ads, d.H, max_row_tiles, s)) return -1;
        ++n;
    }
    {
        ProfScope prof(ctx, KK_PROJECT, s);
        GemmArgs g{};
        g.a_tile_bytes = half_box ? (kBM / 2) * kBK * 2 : 0;
        const CUtensorMap &tmXg = half_box ? tmX64 : tmX;
        g.tiles = ctx->d_tiles; g.n_row_tiles = ctx->d_counts; g.M = T; g.N = d.N; g.K = d.H;
        g.out = (__nv_bfloat16 *)qkv; g.ldo = d.N; g.residual = nullptr; g.adapters = ads;
        g.Nq = d.Nq; g.Nkv = d.Nkv; g.total_adapter_rows = d.N; g.status = ctx->d_status;
        g.item_counters = ctx->d_counts + 10;
        if (may_rowwise) {
            g.rowwise_flag = ctx->d_counts + 5; g.row_delta = ctx->d_row_delta; g.row_adapter = ctx->d_row_adapter;
        }
        if (kv_pool != nullptr) {
            int shift = 0;
            while ((1 << shift) < d.hd) ++shift;
            g.kv_pool = (__nv_bfloat16 *)kv_pool; g.slot_map = ctx->d_slot; g.kv_hd_shift = shift; g.kv_heads = d.Hkv;
            g.kv_page_size = d.page; g.kv_num_pages = num_pages;
        }
        if (fuse_shrink) {
            g.shrink_tiles = ctx->d_shrink_tiles; g.n_shrink_tiles = ctx->d_counts + 2;
            g.t_ready = ctx->d_t_ready; g.t_out = (__nv_bfloat16 *)ctx->d_t;
        }
        const int items = max_row_tiles * ((d.N + BN - 1) / BN + (fuse_shrink ? 1 : 0));
        const bool ok = BN == 256
                            ? launch_gemm_bn<256>(ctx, tmXg, lm.wqkv[1], tmTt, lm.b_all_bn[1], lm.a_all, g, items, s)
                            : BN == 128
                                  ? launch_gemm_bn<128>(ctx, tmXg, lm.wqkv[0], tmTt, lm.b_all_bn[0], lm.a_all, g, items, s)
                                  : launch_gemm_bn<64>(ctx, tmXg, lm.wqkv[2], tmTt, lm.b_all_bn[2], lm.a_all, g, items, s);
        if (!ok) return -1;
        ++n;
    }
    return n;
}

int launch_linear256_tc(alora_ctx *ctx, const void *x, const void *W, int T, int K, int N, void *y,
                        const void *residual, cudaStream_t s);  // gemm256_tcgen05.cu
bool build_pair_maps(alora_ctx *ctx, int layer);                 // gemm_pair_tcgen05.cu

// Plain dense projection y = x W^T (+ residual) for o_proj and the MLP matrices.
int launch_linear_tc(alora_ctx *ctx, const void *x, const void *W, int T, int K, int N, void *y,
                     const void *residual, cudaStream_t s) {
    if (T == 0) return 0;
    if (K % 8 != 0 || N % 8 != 0) return -1;
    ProfScope prof(ctx, KK_LINEAR, s);
    if (skinny_route(ctx, T, N, K, false, N, 0)) {
        CUtensorMap tmW256;
        if (!make_tensor_map_bf16(&tmW256, W, N, K, K, 256)) return -1;
        return launch_skinny_tc(ctx, x, tmW256, nullptr, nullptr, nullptr, T, K, N, N, 0, y, residual, nullptr, 0, s);
    }
    {
        const int r = launch_linear256_tc(ctx, x, W, T, K, N, y, residual, s);   // many rows: 256 x 256 tiles
        if (r != 0) return r;
    }
    const int BN = pick_bn(N, N, 0, false, T);
    CUtensorMap tmX, tmW;
    const bool half_box = T <= kBM / 2;   // see GemmArgs::a_tile_bytes
    if (!make_tensor_map_bf16(&tmX, x, T, K, K, half_box ? kBM / 2 : kBM)) return -1;
    if (!make_tensor_map_bf16(&tmW, W, N, K, K, BN)) return -1;
    GemmArgs g{};
    g.a_tile_bytes = half_box ? (kBM / 2) * kBK * 2 : 0;
    g.tiles = nullptr; g.n_row_tiles = nullptr; g.M = T; g.N = N; g.K = K; g.out = (__nv_bfloat16 *)y; g.ldo = N;
    g.residual = (const __nv_bfloat16 *)residual; g.adapters = nullptr; g.Nq = N; g.Nkv = 0;
    g.total_adapter_rows = 0; g.status = ctx->d_status; g.item_counters = ctx->d_counts + 10;
    const int items = ((T + kBM - 1) / kBM) * ((N + BN - 1) / BN);
    const bool ok = BN == 256 ? launch_gemm_bn<256>(ctx, tmX, tmW, tmX, tmW, tmW, g, items, s)
                    : BN == 128 ? launch_gemm_bn<128>(ctx, tmX, tmW, tmX, tmW, tmW, g, items, s)
                                : launch_gemm_bn<64>(ctx, tmX, tmW, tmX, tmW, tmW, g, items, s);
    return ok ? 1 : -1;
}

// Tensor maps that depend only on registered weights; (re)built when weights or adapters are set.
bool build_layer_maps(alora_ctx *ctx, int layer) {
    const Dims &d = ctx->d;
    TcLayerMaps &lm = ctx->tc_maps[layer];
    const LayerWeights &lw = ctx->layers[layer];
    bool ok = true;
    if (lw.wqkv) {
        ok &= make_tensor_map_bf16(&lm.wqkv[0], lw.wqkv, d.N, d.H, d.H, 128);
        ok &= make_tensor_map_bf16(&lm.wqkv[1], lw.wqkv, d.N, d.H, d.H, 256);
        ok &= make_tensor_map_bf16(&lm.wqkv[2], lw.wqkv, d.N, d.H, d.H, 64);
    }
    const size_t na = (size_t)std::max(1, ctx->cfg.max_adapters);
    ok &= make_tensor_map_bf16(&lm.a_all, ctx->tc_a_all[layer], na * 3 * kTensorRP, d.H, d.H, 3 * kTensorRP);
    ok &= make_tensor_map_bf16(&lm.a_all16, ctx->tc_a_all[layer], na * 3 * kTensorRP, d.H, d.H, 16);
    ok &= make_tensor_map_bf16(&lm.b_all_bn[0], ctx->tc_b_all[layer], na * d.N, kTensorRP, kTensorRP, 128);
    ok &= make_tensor_map_bf16(&lm.b_all_bn[1], ctx->tc_b_all[layer], na * d.N, kTensorRP, kTensorRP, 256);
    ok &= make_tensor_map_bf16(&lm.b_all_bn[2], ctx->tc_b_all[layer], na * d.N, kTensorRP, kTensorRP, 64);
    lm.pair_ok = lw.wqkv != nullptr && build_pair_maps(ctx, layer);   // optional: the 128-row kernel serves every shape
    return ok;
}

}  // namespace alora
