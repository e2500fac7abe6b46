// Paged causal GQA attention for FEW query rows per KV head (Eq. 1 / Eq. 3): decode steps and short
// suffixes, where each K/V byte is used for only G x (a handful of tokens) score rows and the kernel
// is bound by reading the cache from HBM, not by arithmetic.
//
// Work item = (request, KV head, block of up to 64 score rows, key range).  Long contexts are cut
// into key ranges (split-KV) so that a batch of a few requests still fills every SM; the block that
// finishes the last range of a block of rows merges the ranges by their running maximum and sum.
// One persistent block per SM; items are claimed from a global counter, so a block that drew short
// items simply takes more of them:
//   warp 8      producer: walks the item list, looks up the pages of the next 64 keys in the block
//               table and fetches their K and V rows with TMA (one 4-D box per page: both planes and
//               both 64-wide halves of the head dim, 128-byte swizzle) into a 6-deep shared-memory ring; it runs ahead across
//               item boundaries, so the HBM stream never drains between items;
//   warps 0-7   consumers: 16 score rows each (rows are (token, query head of the group) pairs).
//               Scores with mma.sync m16n8k16 (Q fragments in registers, K fragments by ldmatrix),
//               online softmax in registers with quad shuffles for the row maximum and sum,
//               P V with V fragments by ldmatrix.trans.  The 16-key sub-blocks of the ring are dealt
//               round-robin to the 8 / 4 / 2 warps that share a row tile (16 / 32 / 64 rows in the item);
//               their partial results are combined through shared memory at the end of the item.
//               Two warps per scheduler hide each other's dependent chains (score, softmax, P V).
// Masking is by select (a masked score becomes -inf whatever bits the cache holds), and V rows of keys
// at or beyond the end of the item's key range are cleared in shared memory before use.
// All waits are bounded; on expiry ALORA_ERR_TIMEOUT is recorded and the block leaves normally.
#include <algorithm>

#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

constexpr int kSkConsumerWarps = 8;
constexpr int kSkThreads = (kSkConsumerWarps + 1) * 32;
constexpr int kSkStageKeys = 64;
constexpr int kSkStages = 6;
constexpr int kSkItemSlots = 4;

struct SplitArgs {
    const AttnSplitWork *items;
    const int32_t *n_items;
    const int32_t *block_tables;
    const int32_t *qsl, *seq_lens;   // per request: first new token (flat), sequence length (prefix groups' own keys)
    int max_blocks, num_pages;
    int Hkv, G, page_size, box_rows;
    int N, Nq;
    float scale_log2;
    const __nv_bfloat16 *qkv;   // [T][N], query part first
    __nv_bfloat16 *out;         // [T][Nq]
    float *part_o;              // [partial row][HD], unnormalised, relative to the row's maximum in the item
    float *part_ml;             // [partial row][2]: maximum (scaled, log2 units), sum
    int32_t *work_counter;      // next unclaimed item (cleared by the metadata step)
    int32_t *group_done;        // [item] per group (indexed by its first item): key ranges finished so far
    int32_t *status;
};

template <int HD>
struct SkSmem {
    static constexpr int kPlaneBytes = kSkStageKeys * HD * 2;    // K or V of one stage
    static constexpr int kStageBytes = 2 * kPlaneBytes;
    static constexpr int kOStride = HD + 4;                       // floats
    static constexpr int kOOff = kSkStages * kStageBytes;
    static constexpr int kOBytes = 4 * 16 * kOStride * 4;
    static constexpr int kMlOff = kOOff + kOBytes;
    static constexpr int kMlBytes = 4 * 16 * 2 * 4;
    static constexpr int kBarOff = kMlOff + kMlBytes;
    static constexpr int kTotal = kBarOff + 256 + 1024;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
// D (16x8 fp32) += A (16x16 bf16, row-major) * B (16x8 bf16, column-major)
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void tma_load_4d(uint32_t smem_dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// Barrier over the 256 consumer threads that also returns the OR of `pred` over all of them, so that
// every consumer takes the same decision.
__device__ __forceinline__ bool consumer_barrier_or(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"((uint32_t)pred) : "memory");
    return r != 0;
}

// Stage `v` of the own keys of a prefix group's members (requests f .. f + n - 1, own keys from position `shared` on,
// member after member in 64-key stages): which member, and the stage's first key position.
__device__ __forceinline__ void own_key_stage(const int32_t *seq_lens, int f, int n, int shared, int v, int &member, int &kbase) {
    int acc = 0;
    member = f + n - 1; kbase = shared;
    for (int m = f; m < f + n; ++m) {
        const int nst = (seq_lens[m] - shared + kSkStageKeys - 1) / kSkStageKeys;
        if (v < acc + nst) { member = m; kbase = shared + (v - acc) * kSkStageKeys; return; }
        acc += nst;
    }
}

// Merge of the key ranges of one block of rows: out = sum_s O_s 2^(m_s - M) / sum_s l_s 2^(m_s - M).
// `w` is the group's first range; called by 128 threads (threadIdx.x 0..127).
template <int HD>
__device__ __forceinline__ void merge_group(const AttnSplitWork w, const float *part_o, const float *part_ml, int G,
                                            int Nq, __nv_bfloat16 *out) {
    constexpr int kCols = HD / 8;
    const int t = threadIdx.x, r = t >> 3, c0 = (t & 7) * kCols;
    const int rows = 16 * w.mt;  // partial rows per key range of this group
    for (int mt = 0; mt < w.mt; ++mt) {
        const int rg = mt * 16 + r;
        const int tok = rg / G;
        if (tok >= w.q_count) continue;
        float M = -INFINITY;
        for (int s = 0; s < w.n_splits; ++s) M = fmaxf(M, __ldcg(part_ml + ((size_t)w.part_row0 + (size_t)s * rows + rg) * 2));
        float L = 0.f, acc[kCols];
#pragma unroll
        for (int c = 0; c < kCols; ++c) acc[c] = 0.f;
        for (int s = 0; s < w.n_splits; ++s) {
            const float *ml = part_ml + ((size_t)w.part_row0 + (size_t)s * rows + rg) * 2;
            const float wgt = ex2(__ldcg(ml) - M);
            L += __ldcg(ml + 1) * wgt;
            const float *src = part_o + ((size_t)w.part_row0 + (size_t)s * rows + rg) * HD + c0;
#pragma unroll
            for (int c = 0; c < kCols; c += 4) {
                const float4 v = __ldcg(reinterpret_cast<const float4 *>(src + c));
                acc[c] += v.x * wgt; acc[c + 1] += v.y * wgt; acc[c + 2] += v.z * wgt; acc[c + 3] += v.w * wgt;
            }
        }
        const float inv = 1.f / L;
        __nv_bfloat16 *dst = out + (size_t)(w.q_start + tok) * Nq + (size_t)(w.kv_head * G + rg % G) * HD + c0;
#pragma unroll
        for (int c = 0; c < kCols; c += 8) {
            uint4 u;
            u.x = tc::pack_bf16(acc[c] * inv, acc[c + 1] * inv); u.y = tc::pack_bf16(acc[c + 2] * inv, acc[c + 3] * inv);
            u.z = tc::pack_bf16(acc[c + 4] * inv, acc[c + 5] * inv); u.w = tc::pack_bf16(acc[c + 6] * inv, acc[c + 7] * inv);
            *reinterpret_cast<uint4 *>(dst + c) = u;
        }
    }
}

template <int HD>
__global__ void __launch_bounds__(kSkThreads, 1)
attn_splitkv_kernel(const __grid_constant__ CUtensorMap tmKV, const SplitArgs a) {
    using S = SkSmem<HD>;
    constexpr int kHalves = HD / 64;
    // A stage holds 64 keys as 64 / box_rows units; one unit is one TMA box:
    // [plane K, V][64-wide half of the head dim][box_rows keys][128 bytes], 128-byte swizzle inside each half block.
    const uint32_t half_bytes = (uint32_t)a.box_rows * 128u;
    const uint32_t plane_bytes = half_bytes * kHalves;
    const uint32_t unit_bytes = plane_bytes * 2u;
    const int box_shift = 31 - __clz(a.box_rows);
    constexpr int kKSteps = HD / 16;                 // k-steps of Q K^T
    constexpr int kNTiles = HD / 8;                  // 8-wide output column tiles of P V
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    const uint32_t bar0 = smem_base + S::kBarOff;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kSkStages + s); };
    // claimed item indices travel from the producer to the consumers through a small ring of their own
    auto item_full = [&](int s) { return bar0 + 8u * (2 * kSkStages + s); };
    auto item_empty = [&](int s) { return bar0 + 8u * (2 * kSkStages + kSkItemSlots + s); };
    volatile int *item_ring = reinterpret_cast<volatile int *>(smem_al + S::kBarOff + 8 * (2 * kSkStages + 2 * kSkItemSlots));
    volatile int *abort_flag = item_ring + kSkItemSlots;
    volatile int *merge_flag = item_ring + kSkItemSlots + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kSkStages; ++s) { tc::mbar_init(full_bar(s), 1); tc::mbar_init(empty_bar(s), kSkConsumerWarps); }
        for (int s = 0; s < kSkItemSlots; ++s) { tc::mbar_init(item_full(s), 1); tc::mbar_init(item_empty(s), kSkConsumerWarps); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    __syncthreads();
    tc::grid_dep_launch();
    tc::grid_dep_wait();   // work list, q/k/v rows and the cache rows of the new tokens come from earlier kernels
    const int n_items = *a.n_items;

    if (warp == kSkConsumerWarps) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) tc::tma_prefetch_desc(&tmKV);
        const int units_per_stage = kSkStageKeys / a.box_rows;
        uint32_t kt = 0, n_it = 0;
        bool ok = true;
        // items are handed out in list order to whichever block is free; the claim of the item after the current
        // one is issued before the current item's loads, so its latency is hidden behind them
        int it_next = 0;
        if (lane == 0) it_next = atomicAdd(a.work_counter, 1);
        while (ok) {
            int it = -1;
            if (lane == 0) {
                it = it_next < n_items ? it_next : -1;
                if (it >= 0) it_next = atomicAdd(a.work_counter, 1);
                const int slot = n_it % kSkItemSlots;
                ok = tc::mbar_wait(item_empty(slot), ((n_it / kSkItemSlots) & 1) ^ 1, abort_flag);
                if (ok) {
                    item_ring[slot] = it;
                    tc::mbar_arrive(item_full(slot));
                }
            }
            it = __shfl_sync(0xffffffffu, it, 0);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ++n_it;
            if (!ok || it < 0) break;
            const AttnSplitWork w = a.items[it];
            const int n_st = (w.kv_end - w.kv_start + kSkStageKeys - 1) / kSkStageKeys;
            // Window of the request's block-table row: lane l holds entry win0 + l (win0 a multiple of 32; 32 entries
            // cover a whole number of 64-key stages, and key ranges start at multiples of 64).  A table entry is a
            // dependent load from global memory that would otherwise sit in front of every stage's copies; the
            // following window is in flight while this one is used.
            if (w.pad_ & kSplitOwnKeys) {
                // the own keys of a prefix group's members: every stage has its own request (table row) and positions
                const int n_mem = w.pad_ & 0xffff;
                for (int j = 0; j < n_st && ok; ++j, ++kt) {
                    const int st = kt % kSkStages;
                    int member, kbase;
                    own_key_stage(a.seq_lens, w.req, n_mem, w.pos0, w.kv_start / kSkStageKeys + j, member, kbase);
                    const int kend = a.seq_lens[member];
                    const int units = min(units_per_stage, (kend - kbase + a.box_rows - 1) / a.box_rows);
                    int row = -1;
                    if (lane < units) {
                        const int key = kbase + lane * a.box_rows;
                        const int blk = key / a.page_size;
                        const int page = blk < a.max_blocks ? a.block_tables[(size_t)member * a.max_blocks + blk] : -1;
                        if (page < 0 || page >= a.num_pages) report(a.status, ALORA_ERR_PAGE_RANGE);
                        else row = (page * 2 * a.Hkv + w.kv_head) * a.page_size + key % a.page_size;
                    }
                    const unsigned valid = __ballot_sync(0xffffffffu, row >= 0);
                    if (lane == 0) {
                        ok = tc::mbar_wait_relaxed(empty_bar(st), ((kt / kSkStages) & 1) ^ 1, abort_flag);
                        if (ok) tc::mbar_arrive_expect_tx(full_bar(st), (uint32_t)__popc(valid) * unit_bytes);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (ok && row >= 0)
                        tma_load_4d(smem_base + st * S::kStageBytes + lane * unit_bytes, &tmKV, full_bar(st), 0, row, 0, 0);
                }
                continue;
            }
            const int32_t *bt_row = a.block_tables + (size_t)w.req * a.max_blocks;
            auto load_window = [&](int w0) { return w0 + lane < a.max_blocks ? bt_row[w0 + lane] : -1; };
            int win0 = (w.kv_start / a.page_size) & ~31;
            int win = load_window(win0), win_next = load_window(win0 + 32);
            for (int j = 0; j < n_st && ok; ++j, ++kt) {
                const int st = kt % kSkStages;
                const int kbase = w.kv_start + j * kSkStageKeys;
                if (kbase / a.page_size >= win0 + 32) {
                    win0 += 32;
                    win = win_next;
                    win_next = load_window(win0 + 32);
                }
                const int units = min(units_per_stage, (w.kv_end - kbase + a.box_rows - 1) / a.box_rows);
                const int page = __shfl_sync(0xffffffffu, win, ((kbase + lane * a.box_rows) / a.page_size - win0) & 31);
                int row = -1;
                if (lane < units) {
                    const int key = kbase + lane * a.box_rows;
                    if (page < 0 || page >= a.num_pages) report(a.status, ALORA_ERR_PAGE_RANGE);
                    else row = (page * 2 * a.Hkv + w.kv_head) * a.page_size + key % a.page_size;
                }
                const unsigned valid = __ballot_sync(0xffffffffu, row >= 0);
                if (lane == 0) {
                    ok = tc::mbar_wait_relaxed(empty_bar(st), ((kt / kSkStages) & 1) ^ 1, abort_flag);
                    if (ok) tc::mbar_arrive_expect_tx(full_bar(st), (uint32_t)__popc(valid) * unit_bytes);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (ok && row >= 0) {
                    // one box: both planes, both halves, box_rows keys of this page and KV head
                    tma_load_4d(smem_base + st * S::kStageBytes + lane * unit_bytes, &tmKV, full_bar(st), 0, row, 0, 0);
                }
            }
        }
        if (!ok && lane == 0) {
            // copies already in flight must land before the block's shared memory is released
            const uint32_t first = kt > (uint32_t)kSkStages ? kt - kSkStages : 0;
            for (uint32_t i = first; i < kt; ++i) {
                const long long t0 = clock64();
                while (!tc::mbar_try_wait(full_bar(i % kSkStages), (i / kSkStages) & 1) &&
                       clock64() - t0 < tc::kWaitCycleLimit) {}
            }
        }
    } else {
        // ------------------------------ consumers (warps 0..7) ------------------------------
        const int qr = lane >> 2, qc = lane & 3;          // fragment row (and +8), column pair
        float *o_s = reinterpret_cast<float *>(smem_al + S::kOOff);
        float *ml_s = reinterpret_cast<float *>(smem_al + S::kMlOff);
        uint32_t kt = 0, n_it = 0;
        bool ok = true;
        while (true) {
            const int slot = n_it % kSkItemSlots;
            const bool got = __all_sync(0xffffffffu, tc::mbar_wait(item_full(slot), (n_it / kSkItemSlots) & 1, abort_flag));
            const int it = got ? item_ring[slot] : -1;
            __syncwarp();
            if (lane == 0 && got) tc::mbar_arrive(item_empty(slot));
            ++n_it;
            if (consumer_barrier_or(!got)) break;     // a wait expired: all consumers leave together
            if (it < 0) break;                        // the producer found the list exhausted (same value in every warp)
            const AttnSplitWork w = a.items[it];
            const int mt_cnt = w.mt;                  // 1, 2 or 4 row tiles of 16
            const int my_mt = warp % mt_cnt;          // row tile of this warp
            const int kg = warp / mt_cnt;             // which share of the 16-key sub-blocks
            const int n_kg = kSkConsumerWarps / mt_cnt;   // 8, 4 or 2 key shares
            const int n_st = (w.kv_end - w.kv_start + kSkStageKeys - 1) / kSkStageKeys;

            // ---- this warp's 16 query rows as A fragments, straight from global memory (4 KB per warp and item):
            // registers 0 / 1 hold rows qr / qr + 8 at columns 16 ks + 2 qc, registers 2 / 3 the same rows 8 columns on
            uint32_t qa[kKSteps][4];
            {
                const int rg_lo = my_mt * 16 + qr, rg_hi = rg_lo + 8;
                const bool v_lo = rg_lo / a.G < w.q_count, v_hi = rg_hi / a.G < w.q_count;
                const uint32_t *q_lo = reinterpret_cast<const uint32_t *>(
                    a.qkv + (size_t)(w.q_start + (v_lo ? rg_lo / a.G : 0)) * a.N + (size_t)(w.kv_head * a.G + rg_lo % a.G) * HD);
                const uint32_t *q_hi = reinterpret_cast<const uint32_t *>(
                    a.qkv + (size_t)(w.q_start + (v_hi ? rg_hi / a.G : 0)) * a.N + (size_t)(w.kv_head * a.G + rg_hi % a.G) * HD);
#pragma unroll
                for (int ks = 0; ks < kKSteps; ++ks) {
                    qa[ks][0] = v_lo ? __ldg(q_lo + ks * 8 + qc) : 0u;
                    qa[ks][1] = v_hi ? __ldg(q_hi + ks * 8 + qc) : 0u;
                    qa[ks][2] = v_lo ? __ldg(q_lo + ks * 8 + 4 + qc) : 0u;
                    qa[ks][3] = v_hi ? __ldg(q_hi + ks * 8 + 4 + qc) : 0u;
                }
            }
            // causal limits of this thread's two rows (clamped to the item's key range)
            const int tok_lo = min((my_mt * 16 + qr) / a.G, w.q_count - 1);
            const int tok_hi = min((my_mt * 16 + qr + 8) / a.G, w.q_count - 1);
            const bool own_keys = (w.pad_ & kSplitOwnKeys) != 0;   // a prefix group's own keys: limits change per stage
            int lim_lo = min(w.pos0 + tok_lo, w.kv_end - 1);
            int lim_hi = min(w.pos0 + tok_hi, w.kv_end - 1);
            int kv_end_st = w.kv_end;

            float o[kNTiles][4];
#pragma unroll
            for (int n = 0; n < kNTiles; ++n) { o[n][0] = 0.f; o[n][1] = 0.f; o[n][2] = 0.f; o[n][3] = 0.f; }
            float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

            for (int j = 0; j < n_st && ok; ++j, ++kt) {
                const int st = kt % kSkStages;
                if (!__all_sync(0xffffffffu, tc::mbar_wait(full_bar(st), (kt / kSkStages) & 1, abort_flag))) { ok = false; break; }
                const uint32_t k_u32 = smem_base + st * S::kStageBytes;
                int kbase = w.kv_start + j * kSkStageKeys;
                if (own_keys) {
                    // this stage holds keys of one member: its tokens see them up to their own positions, the other
                    // rows of the stacked block see none of them
                    int member;
                    own_key_stage(a.seq_lens, w.req, w.pad_ & 0xffff, w.pos0, w.kv_start / kSkStageKeys + j, member, kbase);
                    kv_end_st = a.seq_lens[member];
                    const int t0 = a.qsl[member] - w.q_start, nn = a.qsl[member + 1] - a.qsl[member], p0 = kv_end_st - nn;
                    lim_lo = (tok_lo >= t0 && tok_lo < t0 + nn) ? p0 + tok_lo - t0 : -1;
                    lim_hi = (tok_hi >= t0 && tok_hi < t0 + nn) ? p0 + tok_hi - t0 : -1;
                }
#pragma unroll 1
                for (int sb = 0; sb < 4; ++sb) {
                    // 16-key sub-blocks are dealt round-robin over the key shares, across stages
                    if (((j * 4 + sb) & (n_kg - 1)) != kg) continue;
                    const int k0 = kbase + sb * 16;
                    if (k0 >= kv_end_st) break;
                    if (k0 + 16 > kv_end_st) {
                        // rows of keys beyond the range may hold anything: clear their V rows
                        uint8_t *v_gen = smem_al + st * S::kStageBytes + plane_bytes;
                        for (int i = lane; i < 16 * 8 * kHalves; i += 32) {
                            const int r = i / (8 * kHalves), c = i % (8 * kHalves);
                            const int key_l = sb * 16 + r;
                            if (k0 + r >= kv_end_st)
                                *reinterpret_cast<uint4 *>(v_gen + (key_l >> box_shift) * unit_bytes + (c / 8) * half_bytes +
                                                           (key_l & (a.box_rows - 1)) * 128 + (c % 8) * 16) = make_uint4(0, 0, 0, 0);
                        }
                        tc::fence_proxy_async();
                        __syncwarp();
                    }
                    // ---- scores of 16 rows x 16 keys
                    float s[2][4];
#pragma unroll
                    for (int n = 0; n < 2; ++n) { s[n][0] = 0.f; s[n][1] = 0.f; s[n][2] = 0.f; s[n][3] = 0.f; }
                    {
                        const int key_l = sb * 16 + (lane >> 4) * 8 + (lane & 7);
                        const uint32_t krow = k_u32 + (key_l >> box_shift) * unit_bytes + (key_l & (a.box_rows - 1)) * 128;
                        const int sw = key_l & 7;
#pragma unroll
                        for (int ks = 0; ks < kKSteps; ++ks) {
                            const int chunk = 2 * (ks & 3) + ((lane >> 3) & 1);
                            uint32_t b0, b1, b2, b3;
                            ldsm_x4(krow + (ks >> 2) * half_bytes + ((chunk ^ sw) << 4), b0, b1, b2, b3);
                            mma_16816(s[0], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                            mma_16816(s[1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
                        }
                    }
                    // ---- scale, causal mask, online softmax
                    const bool need_mask = k0 + 15 > min(lim_lo, lim_hi);
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float v = s[n][e] * a.scale_log2;
                            if (need_mask) {
                                const int key = k0 + n * 8 + 2 * qc + (e & 1);
                                if (key > (e < 2 ? lim_lo : lim_hi)) v = -INFINITY;
                            }
                            s[n][e] = v;
                        }
                    float mx_lo = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
                    float mx_hi = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
                    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
                    const float mu_lo = mn_lo == -INFINITY ? 0.f : mn_lo, mu_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
                    const float al_lo = ex2(m_lo - mu_lo), al_hi = ex2(m_hi - mu_hi);
                    m_lo = mn_lo; m_hi = mn_hi;
#pragma unroll
                    for (int n = 0; n < 2; ++n) {
                        s[n][0] = ex2(s[n][0] - mu_lo); s[n][1] = ex2(s[n][1] - mu_lo);
                        s[n][2] = ex2(s[n][2] - mu_hi); s[n][3] = ex2(s[n][3] - mu_hi);
                    }
                    l_lo = l_lo * al_lo + (s[0][0] + s[0][1] + s[1][0] + s[1][1]);
                    l_hi = l_hi * al_hi + (s[0][2] + s[0][3] + s[1][2] + s[1][3]);
                    if (al_lo != 1.f || al_hi != 1.f) {
#pragma unroll
                        for (int n = 0; n < kNTiles; ++n) { o[n][0] *= al_lo; o[n][1] *= al_lo; o[n][2] *= al_hi; o[n][3] *= al_hi; }
                    }
                    // ---- O += P V (P rounded to bf16, as the A operand of the second product)
                    const uint32_t pa0 = tc::pack_bf16(s[0][0], s[0][1]), pa1 = tc::pack_bf16(s[0][2], s[0][3]);
                    const uint32_t pa2 = tc::pack_bf16(s[1][0], s[1][1]), pa3 = tc::pack_bf16(s[1][2], s[1][3]);
                    {
                        const int key_l = sb * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
                        const uint32_t vrow = k_u32 + plane_bytes + (key_l >> box_shift) * unit_bytes +
                                              (key_l & (a.box_rows - 1)) * 128;
                        const int sw = key_l & 7;
#pragma unroll
                        for (int cp = 0; cp < kNTiles / 2; ++cp) {
                            const int c16 = 2 * cp + (lane >> 4);
                            uint32_t b0, b1, b2, b3;
                            ldsm_x4_trans(vrow + (c16 >> 3) * half_bytes + (((c16 & 7) ^ sw) << 4), b0, b1, b2, b3);
                            mma_16816(o[2 * cp], pa0, pa1, pa2, pa3, b0, b1);
                            mma_16816(o[2 * cp + 1], pa0, pa1, pa2, pa3, b2, b3);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(empty_bar(st));
            }
            // ---- combine the warps that share a row tile, then store the item's result
            l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
            l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
            // warps 4..7 hand their partial result to warps 0..3 (same row tile, same fragment layout) ...
            if (warp >= 4) {
                float *ow = o_s + (warp - 4) * 16 * S::kOStride;
#pragma unroll
                for (int n = 0; n < kNTiles; ++n) {
                    *reinterpret_cast<float2 *>(ow + qr * S::kOStride + n * 8 + 2 * qc) = make_float2(o[n][0], o[n][1]);
                    *reinterpret_cast<float2 *>(ow + (qr + 8) * S::kOStride + n * 8 + 2 * qc) = make_float2(o[n][2], o[n][3]);
                }
                if (qc == 0) {
                    ml_s[((warp - 4) * 16 + qr) * 2] = m_lo; ml_s[((warp - 4) * 16 + qr) * 2 + 1] = l_lo;
                    ml_s[((warp - 4) * 16 + qr + 8) * 2] = m_hi; ml_s[((warp - 4) * 16 + qr + 8) * 2 + 1] = l_hi;
                }
            }
            consumer_barrier();
            // ... which fold it into their own and publish the sum for the final combination
            if (warp < 4) {
                float *ow = o_s + warp * 16 * S::kOStride;
                const float m2_lo = ml_s[(warp * 16 + qr) * 2], l2_lo = ml_s[(warp * 16 + qr) * 2 + 1];
                const float m2_hi = ml_s[(warp * 16 + qr + 8) * 2], l2_hi = ml_s[(warp * 16 + qr + 8) * 2 + 1];
                const float M_lo = fmaxf(m_lo, m2_lo), M_hi = fmaxf(m_hi, m2_hi);
                const float mu_lo = M_lo == -INFINITY ? 0.f : M_lo, mu_hi = M_hi == -INFINITY ? 0.f : M_hi;
                const float a1_lo = ex2(m_lo - mu_lo), a2_lo = ex2(m2_lo - mu_lo);
                const float a1_hi = ex2(m_hi - mu_hi), a2_hi = ex2(m2_hi - mu_hi);
                __syncwarp();  // all lanes have read the row statistics before lane qc == 0 rewrites them
#pragma unroll
                for (int n = 0; n < kNTiles; ++n) {
                    float2 *p_lo = reinterpret_cast<float2 *>(ow + qr * S::kOStride + n * 8 + 2 * qc);
                    float2 *p_hi = reinterpret_cast<float2 *>(ow + (qr + 8) * S::kOStride + n * 8 + 2 * qc);
                    const float2 v_lo = *p_lo, v_hi = *p_hi;
                    *p_lo = make_float2(o[n][0] * a1_lo + v_lo.x * a2_lo, o[n][1] * a1_lo + v_lo.y * a2_lo);
                    *p_hi = make_float2(o[n][2] * a1_hi + v_hi.x * a2_hi, o[n][3] * a1_hi + v_hi.y * a2_hi);
                }
                if (qc == 0) {
                    ml_s[(warp * 16 + qr) * 2] = M_lo; ml_s[(warp * 16 + qr) * 2 + 1] = l_lo * a1_lo + l2_lo * a2_lo;
                    ml_s[(warp * 16 + qr + 8) * 2] = M_hi; ml_s[(warp * 16 + qr + 8) * 2 + 1] = l_hi * a1_hi + l2_hi * a2_hi;
                }
            }
            if (consumer_barrier_or(!ok)) break;  // a wait expired somewhere: all consumers leave together
            if (warp < 4) {
                const int n_src = 4 / mt_cnt;             // warps 0..3 that hold the same row tile
                constexpr int kCols = HD / 8;             // columns per thread: 8 threads cover a row
                const int t = threadIdx.x;                // 0..127
                const int r = t >> 3, c0 = (t & 7) * kCols;
                for (int mt = 0; mt < mt_cnt; ++mt) {
                    float M = -INFINITY;
                    for (int g = 0; g < n_src; ++g) M = fmaxf(M, ml_s[((mt + mt_cnt * g) * 16 + r) * 2]);
                    const float Mu = M == -INFINITY ? 0.f : M;
                    float L = 0.f, acc[kCols];
#pragma unroll
                    for (int c = 0; c < kCols; ++c) acc[c] = 0.f;
                    for (int g = 0; g < n_src; ++g) {
                        const int src = mt + mt_cnt * g;
                        const float wgt = ex2(ml_s[(src * 16 + r) * 2] - Mu);
                        L += ml_s[(src * 16 + r) * 2 + 1] * wgt;
                        const float *orow = o_s + (src * 16 + r) * S::kOStride + c0;
#pragma unroll
                        for (int c = 0; c < kCols; c += 4) {
                            const float4 v = *reinterpret_cast<const float4 *>(orow + c);
                            acc[c] += v.x * wgt; acc[c + 1] += v.y * wgt; acc[c + 2] += v.z * wgt; acc[c + 3] += v.w * wgt;
                        }
                    }
                    const int rg = mt * 16 + r;
                    const int tok = rg / a.G;
                    if (tok >= w.q_count) continue;
                    if (w.n_splits == 1) {
                        const float inv = 1.f / L;
                        __nv_bfloat16 *dst = a.out + (size_t)(w.q_start + tok) * a.Nq +
                                             (size_t)(w.kv_head * a.G + rg % a.G) * HD + c0;
#pragma unroll
                        for (int c = 0; c < kCols; c += 8) {
                            uint4 u;
                            u.x = tc::pack_bf16(acc[c] * inv, acc[c + 1] * inv); u.y = tc::pack_bf16(acc[c + 2] * inv, acc[c + 3] * inv);
                            u.z = tc::pack_bf16(acc[c + 4] * inv, acc[c + 5] * inv); u.w = tc::pack_bf16(acc[c + 6] * inv, acc[c + 7] * inv);
                            *reinterpret_cast<uint4 *>(dst + c) = u;
                        }
                    } else {
                        float *dst = a.part_o + ((size_t)w.part_row0 + rg) * HD + c0;
#pragma unroll
                        for (int c = 0; c < kCols; c += 4)
                            *reinterpret_cast<float4 *>(dst + c) = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
                        if ((t & 7) == 0) {
                            a.part_ml[((size_t)w.part_row0 + rg) * 2] = M;
                            a.part_ml[((size_t)w.part_row0 + rg) * 2 + 1] = L;
                        }
                    }
                }
            }
            if (w.n_splits > 1) {
                // the block that completes the last key range of a group merges the group (ranges in index order,
                // whichever block does it: the result does not depend on timing)
                __threadfence();
                consumer_barrier();
                if (threadIdx.x == 0) *merge_flag = atomicAdd(a.group_done + (it - w.split), 1) == w.n_splits - 1;
                consumer_barrier();
                if (*merge_flag && warp < 4) {
                    __threadfence();
                    merge_group<HD>(a.items[it - w.split], a.part_o, a.part_ml, a.G, a.Nq, a.out);
                }
            } else {
                consumer_barrier();  // the exchange buffers are rewritten by the next item
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(a.status, ALORA_ERR_TIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn tensor_map_encoder();  // gemm_tcgen05.cu

// Few-row attention over the context's split-KV work list.  Returns kernels launched or -1.
int launch_attend_splitkv(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                          cudaStream_t s) {
    const Dims &d = ctx->d;
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc || !ctx->d_split_items) return -1;
    const int box_rows = std::min(d.page, kSkStageKeys);
    CUtensorMap tmKV;
    {
        // the pool as (64 columns, cache rows, 64-wide halves of the head dim, K / V plane): one box fetches
        // box_rows keys of one page and KV head, both halves, both planes
        const cuuint64_t halves = (cuuint64_t)d.hd / 64;
        cuuint64_t dims[4] = {64, (cuuint64_t)b.num_pages * 2 * d.Hkv * d.page, halves, 2};
        cuuint64_t strides[3] = {(cuuint64_t)d.hd * 2, 128, (cuuint64_t)d.Hkv * d.page * d.hd * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)box_rows, (cuuint32_t)halves, 2};
        cuuint32_t es[4] = {1, 1, 1, 1};
        if (enc(&tmKV, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(pool), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -1;
    }
    SplitArgs a{};
    a.items = ctx->d_split_items; a.n_items = ctx->d_counts + 3; a.block_tables = b.block_tables;
    a.qsl = b.query_start_loc; a.seq_lens = b.seq_lens;
    a.max_blocks = b.max_blocks; a.num_pages = b.num_pages; a.Hkv = d.Hkv; a.G = d.G; a.page_size = d.page;
    a.box_rows = box_rows; a.N = d.N; a.Nq = d.Nq; a.scale_log2 = d.softmax_scale * 1.4426950408889634f;
    a.qkv = (const __nv_bfloat16 *)qkv; a.out = (__nv_bfloat16 *)out; a.part_o = ctx->d_part_o;
    a.part_ml = ctx->d_part_ml; a.work_counter = ctx->d_counts + 4; a.group_done = ctx->d_group_done;
    a.status = ctx->d_status;
    static bool attr_set[2][64] = {};
    const int dev = ctx->cfg.device, hi = d.hd == 128;
    if (dev >= 0 && dev < 64 && !attr_set[hi][dev]) {
        cudaError_t e = hi ? cudaFuncSetAttribute(attn_splitkv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  SkSmem<128>::kTotal)
                           : cudaFuncSetAttribute(attn_splitkv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  SkSmem<64>::kTotal);
        if (e != cudaSuccess) return -1;
        attr_set[hi][dev] = true;
    }
    const int grid = std::max(1, std::min(ctx->sm_count, ctx->max_split_items));
    {
        ProfScope prof(ctx, KK_ATTN_FEW_ROW, s);
        const cudaError_t e = hi ? launch_kernel(attn_splitkv_kernel<128>, dim3(grid), dim3(kSkThreads), SkSmem<128>::kTotal, s, true, tmKV, a)
                                 : launch_kernel(attn_splitkv_kernel<64>, dim3(grid), dim3(kSkThreads), SkSmem<64>::kTotal, s, true, tmKV, a);
        if (e != cudaSuccess) return -1;
    }
    return 1;
}

}  // namespace alora
