// Projection of a batch of at most 128 rows (decode steps, short invocation suffixes): out = x W^T with the
// aLoRA delta of Eq. 5 on the rows whose gate is open.  With so few rows the weights are read once and never
// reused: the step is bound by streaming W out of HBM, so the work is cut to put every SM on that stream.
//
// Kernel 1 (tensor cores, one work item per block): item = (256-column tile of W, slice of K).  The K dimension is
//   split over as many slices as it takes to give every SM an item; a block streams its [256 x K/slices] piece of W
//   and the matching columns of x through a TMA ring and accumulates a partial product in tensor memory
//   (tcgen05.mma 128 x 256 x 16), which its epilogue warps write out as fp32.
//   The rank-r shrink t = A x of every adapter present in the batch rides along: the adapters' A rows are dealt
//   out in chunks of 16 rows over the column tiles, and a block multiplies its chunks with the x columns it holds
//   anyway (tcgen05.mma 128 x 16 x 16 into spare tensor-memory columns).  x is never read a second time for the
//   shrink, and t costs no launch of its own.  Every row is multiplied with every present adapter's chunk; which
//   adapter a row really uses is decided in kernel 2.
// Kernel 2 (CUDA cores): per output element the K-slice partials are added in slice order; a row with an applied
//   adapter k adds s B_k t_k (t_k = the slice partials of ITS adapter's shrink, added in slice order, fp32); rows
//   without one add nothing, so they go through exactly the arithmetic of a base-only call (Prop. 1: gated-off rows
//   are bit-identical).  Optional residual add; bf16 store; the k / v columns also go to the row's cache slot.
// No atomics in the arithmetic, fixed summation orders: results are run-to-run deterministic.  The route is chosen
// by the row count alone, never by the mode or the adapters.
#include <algorithm>

#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

constexpr int kSkM = 128;            // rows of the accumulator (UMMA M); batches have at most this many rows
constexpr int kSkBN = 256;           // columns of W per work item
constexpr int kSkBK = 64;            // K elements per ring stage (one 128-byte swizzle row)
constexpr int kSkChunkRows = 16;     // adapter A rows per shrink chunk
constexpr int kSkChunksPerAdapter = 3 * kRankPadMax / kSkChunkRows;   // 192 stored A rows per adapter = 12 chunks
constexpr int kSkMaxChunks = 16;     // chunks per block: 16 x 16 spare tensor-memory columns
constexpr int kSkThreads = 192;
constexpr int kSkMaxStages = 8;
constexpr int kSkMaxPresent = kFewRowMax;   // a batch of <= 128 rows names at most 128 adapters
constexpr int kSkABytes = kSkM * kSkBK * 2, kSkWBytes = kSkBN * kSkBK * 2, kSkChunkBytes = kSkChunkRows * kSkBK * 2;

struct SkinnyArgs {
    int T, N, K;
    int n_tiles, ksplit;          // work items = n_tiles * ksplit, item = tile * ksplit + slice
    int x_box_bytes;              // bytes one copy of the x tile brings (a 64-row box for batches of <= 64 rows); the
                                  // stage reserves just that: the accumulator rows beyond the box are never read
    int stage_bytes, n_stages, chunk_cap;
    float *part;                  // [item][128][256] fp32 partial products (rows < T written)
    float *t_part;                // [slice][128][p_cap][192] fp32 partial shrink results
    int p_cap;                    // slots of present adapters in t_part
    const int32_t *row_adapter;   // [T] applied adapter per row, or nullptr (no adapters in this launch)
    const FewRowMeta *meta;       // the batch's adapter facts (from the batch-metadata step), nullptr without adapters
    int max_adapters;
    int32_t *status;
};

__global__ void __launch_bounds__(kSkThreads, 1)
gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                   const __grid_constant__ CUtensorMap tmA, const SkinnyArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int present_ids[kSkMaxPresent];
    __shared__ int present_n;
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    const int n_stages = a.n_stages;
    const uint32_t bar0 = smem_base + (uint32_t)(n_stages * a.stage_bytes);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + n_stages * a.stage_bytes);
    // barrier words: full[8], empty[8], acc_full, acc_empty, drain; then the tensor-memory address and the abort flag
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kSkMaxStages + s); };
    const uint32_t accf_bar = bar0 + 8u * (2 * kSkMaxStages), acce_bar = accf_bar + 8u, drain_bar = accf_bar + 16u;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * kSkMaxStages + 3);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * kSkMaxStages + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kTmemCols = 512;   // 256 accumulator columns + up to 16 x 16 shrink columns

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) { tc::mbar_init(full_bar(s), 1); tc::mbar_init(empty_bar(s), 1); }
        tc::mbar_init(accf_bar, 1); tc::mbar_init(acce_bar, 4); tc::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32((const void *)tmem_slot), kTmemCols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int total = a.n_tiles * a.ksplit;
    const int kb_total = (a.K + kSkBK - 1) / kSkBK;
    const int kb_base = kb_total / a.ksplit, kb_rem = kb_total % a.ksplit;
    const uint32_t x_bytes = (uint32_t)a.x_box_bytes;
    tc::grid_dep_launch();
    // The weights do not depend on anything earlier in the stream: the W tiles of the first ring round are requested
    // before the wait for the predecessor kernel, so that they stream in while it is still running.
    int w_ahead = 0;
    if (threadIdx.x == 0 && (int)blockIdx.x < total) {
        tc::tma_prefetch_desc(&tmW);
        const int tile = blockIdx.x / a.ksplit, sl = blockIdx.x % a.ksplit;
        const int kb0 = sl * kb_base + min(sl, kb_rem), nkb = kb_base + (sl < kb_rem ? 1 : 0);
        w_ahead = min(nkb, n_stages);
        for (int s = 0; s < w_ahead; ++s) {
            tc::mbar_expect_tx(full_bar(s), kSkWBytes);
            tc::tma_load_2d(smem_base + s * a.stage_bytes + x_bytes, &tmW, full_bar(s), (kb0 + s) * kSkBK, tile * kSkBN);
        }
    }
    tc::grid_dep_wait();   // x and the row -> adapter map are written by earlier kernels of the stream
    // the adapters present in the batch (one round trip; the list was made by the batch-metadata step)
    if (a.meta != nullptr) {
        if (threadIdx.x < kSkMaxPresent) present_ids[threadIdx.x] = a.meta->id[threadIdx.x];
        if (threadIdx.x == kSkThreads - 1) present_n = a.meta->n_present;
    } else if (threadIdx.x == 0) {
        present_n = 0;
    }
    __syncthreads();
    const int total_chunks = min(present_n, a.p_cap) * kSkChunksPerAdapter;
    // chunks of column tile j: j, j + n_tiles, j + 2 n_tiles, ...
    auto chunks_of = [&](int tile) {
        return total_chunks > tile ? min((total_chunks - tile + a.n_tiles - 1) / a.n_tiles, a.chunk_cap) : 0;
    };

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------ TMA producer ------------------------------
            tc::tma_prefetch_desc(&tmX);
            uint32_t kc = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < total && ok; item += gridDim.x) {
                const int tile = item / a.ksplit, sl = item % a.ksplit;
                const int kb0 = sl * kb_base + min(sl, kb_rem), nkb = kb_base + (sl < kb_rem ? 1 : 0);
                const int n_chunk = chunks_of(tile);
                for (int kb = kb0; kb < kb0 + nkb; ++kb, ++kc) {
                    const int s = kc % n_stages;
                    if (!tc::mbar_wait(empty_bar(s), ((kc / n_stages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t sx = smem_base + s * a.stage_bytes, sw = sx + x_bytes, sc = sw + kSkWBytes;
                    if ((int)kc < w_ahead) {   // this stage's W tile is already on its way
                        tc::mbar_arrive_expect_tx(full_bar(s), x_bytes + n_chunk * kSkChunkBytes);
                    } else {
                        tc::mbar_arrive_expect_tx(full_bar(s), x_bytes + kSkWBytes + n_chunk * kSkChunkBytes);
                        tc::tma_load_2d(sw, &tmW, full_bar(s), kb * kSkBK, tile * kSkBN);
                    }
                    tc::tma_load_2d(sx, &tmX, full_bar(s), kb * kSkBK, 0);
                    for (int i = 0; i < n_chunk; ++i) {
                        const int c = tile + i * a.n_tiles;
                        const int row = present_ids[c / kSkChunksPerAdapter] * (3 * kRankPadMax) +
                                        (c % kSkChunksPerAdapter) * kSkChunkRows;
                        tc::tma_load_2d(sc + i * kSkChunkBytes, &tmA, full_bar(s), kb * kSkBK, row);
                    }
                }
            }
            if (!ok) {
                // give copies already in flight time to land before the block's shared memory is released
                const uint32_t first = kc > (uint32_t)n_stages ? kc - n_stages : 0;
                for (uint32_t i = first; i < kc; ++i) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(full_bar(i % n_stages), (i / n_stages) & 1) &&
                           clock64() - t0 < tc::kWaitCycleLimit) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        // the whole warp walks the schedule (uniform control flow), one elected lane issues
        const bool leader = tc::elect_one();
        auto wait_all = [&](uint32_t bar, uint32_t parity) {
            return __all_sync(0xffffffffu, tc::mbar_wait(bar, parity, abort_flag));
        };
        constexpr uint32_t idesc_main = tc::idesc_bf16_f32(kSkM, kSkBN);
        constexpr uint32_t idesc_chunk = tc::idesc_bf16_f32(kSkM, kSkChunkRows);
        uint32_t kc = 0, it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total && ok; item += gridDim.x) {
            const int tile = item / a.ksplit, sl = item % a.ksplit;
            const int nkb = kb_base + (sl < kb_rem ? 1 : 0);
            const int n_chunk = chunks_of(tile);
            if (it > 0) {   // the epilogue must have read the previous item's accumulators
                if (!wait_all(acce_bar, (it - 1) & 1)) { ok = false; break; }
                tc::tc_fence_after();
            }
            for (int kb = 0; kb < nkb; ++kb, ++kc) {
                const int s = kc % n_stages;
                if (!wait_all(full_bar(s), (kc / n_stages) & 1)) { ok = false; break; }
                tc::tc_fence_after();
                const uint32_t sx = smem_base + s * a.stage_bytes, sw = sx + x_bytes, sc = sw + kSkWBytes;
                const uint64_t dx = tc::smem_desc_k_sw128(sx), dw = tc::smem_desc_k_sw128(sw);
                if (leader) {
#pragma unroll
                    for (int k = 0; k < kSkBK / 16; ++k)
                        tc::mma_bf16(tmem_base, dx + 2 * k, dw + 2 * k, idesc_main, (kb | k) != 0 ? 1u : 0u);
                    for (int i = 0; i < n_chunk; ++i) {
                        const uint64_t dc = tc::smem_desc_k_sw128(sc + i * kSkChunkBytes);
#pragma unroll
                        for (int k = 0; k < kSkBK / 16; ++k)
                            tc::mma_bf16(tmem_base + kSkBN + i * kSkChunkRows, dx + 2 * k, dc + 2 * k, idesc_chunk,
                                         (kb | k) != 0 ? 1u : 0u);
                    }
                    tc::mma_commit(empty_bar(s));
                }
            }
            if (!ok) break;
            if (leader) tc::mma_commit(accf_bar);
            ++it;
        }
        if (!ok && leader) {
            tc::mma_commit(drain_bar);
            const long long t0 = clock64();
            while (!tc::mbar_try_wait(drain_bar, 0) && clock64() - t0 < tc::kWaitCycleLimit) {}
        }
    } else {
        // ------------------------------ epilogue (warps 2..5) ------------------------------
        const int q = warp & 3;   // tensor-memory lane quarter this warp may read
        uint32_t it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total && ok; item += gridDim.x) {
            const int tile = item / a.ksplit, sl = item % a.ksplit;
            const int n_chunk = chunks_of(tile);
            if (!tc::mbar_wait(accf_bar, it & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            const int r = q * 32 + lane;
            if (q * 32 < a.T) {    // warp-uniform: quarters beyond the batch's rows hold nothing
                const bool row_ok = r < a.T;
                float *prow = a.part + ((size_t)item * kSkM + r) * kSkBN;
                const int n_cols = min(kSkBN, a.N - tile * kSkBN);
#pragma unroll 1
                for (int c = 0; c < n_cols; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(tmem_base + c + ((uint32_t)(q * 32) << 16), v);
                    tc::tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<uint4 *>(prow + c + 4 * j) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    }
                }
#pragma unroll 1
                for (int i0 = 0; i0 < n_chunk; i0 += 2) {   // two chunks of 16 columns per load
                    uint32_t v[32];
                    tc::tmem_ld_32x32(tmem_base + kSkBN + i0 * kSkChunkRows + ((uint32_t)(q * 32) << 16), v);
                    tc::tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (i0 + h >= n_chunk) break;
                            const int c = tile + (i0 + h) * a.n_tiles;
                            float *trow = a.t_part + (((size_t)sl * kSkM + r) * a.p_cap + c / kSkChunksPerAdapter) * (3 * kRankPadMax) +
                                          (c % kSkChunksPerAdapter) * kSkChunkRows;
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                *reinterpret_cast<uint4 *>(trow + 4 * j) =
                                    make_uint4(v[16 * h + 4 * j], v[16 * h + 4 * j + 1], v[16 * h + 4 * j + 2], v[16 * h + 4 * j + 3]);
                        }
                    }
                }
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(acce_bar);
            ++it;
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(a.status, ALORA_ERR_TIMEOUT);
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- kernel 2: add the slice partials, the delta of gated rows, the residual; store; append k / v ----
struct SkinnyFinArgs {
    int T, N, n_tiles, ksplit, p_cap;
    const float *part, *t_part;
    const FewRowMeta *meta;           // nullptr: no adapters in this launch
    const __nv_bfloat16 *b_all;       // the layer's B rows of all adapters, [adapter][N][64]
    int Nq, Nkv;
    const __nv_bfloat16 *residual;
    __nv_bfloat16 *out;
    int ldo;
    __nv_bfloat16 *kv_pool;
    const int32_t *slot_map;
    int kv_hd_shift, kv_heads, kv_page_size, kv_num_pages;
    int32_t *status;
};
constexpr int kFinCols = 64, kFinRows = 32, kFinThreads = 256;
constexpr int kFinAdGroup = 4;   // adapters whose B tile is staged in shared memory at a time
constexpr int kFinSliceGroup = 8;   // K slices whose loads are in flight together

__global__ void __launch_bounds__(kFinThreads, 2)
skinny_finish_kernel(const SkinnyFinArgs a) {
    __shared__ __align__(16) float t_s[kFinRows][kRankPadMax + 4];   // (+4: rows of a warp on different banks, float4 reads)
    __shared__ uint4 b_s[kFinAdGroup][kFinCols][kRankPadMax / 8];   // B rows of this column block; vector v of column c sits at v ^ (c / 8)
    __shared__ int slot_s[kFinRows], id_s[kSkMaxPresent], rpad_s[kSkMaxPresent];
    __shared__ float scale_s[kSkMaxPresent];
    __shared__ int n_present_s;
    tc::grid_dep_launch();
    tc::grid_dep_wait();
    const int row0 = blockIdx.y * kFinRows, colb = blockIdx.x * kFinCols;
    const int blk = colb < a.Nq ? 0 : (colb < a.Nq + a.Nkv ? 1 : 2);
    const int rr = threadIdx.x >> 3, row = row0 + rr, c0 = (threadIdx.x & 7) * 8, col = colb + c0;
    const bool mine = row < a.T && col < a.N;
    // ---- first round of loads, all independent: the batch's adapter facts, and the K-slice partials of this
    // thread's 8 outputs (added in slice order)
    if (a.meta != nullptr) {
        if (threadIdx.x < kFinRows) slot_s[threadIdx.x] = row0 + (int)threadIdx.x < a.T ? a.meta->slot_of_row[row0 + threadIdx.x] : -1;
        if (threadIdx.x < kSkMaxPresent) {
            id_s[threadIdx.x] = a.meta->id[threadIdx.x]; rpad_s[threadIdx.x] = a.meta->rpad[threadIdx.x];
            scale_s[threadIdx.x] = a.meta->scale[threadIdx.x];
        }
        if (threadIdx.x == kFinThreads - 1) n_present_s = a.meta->n_present;
    }
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = 0.f;
    if (mine) {
        const int tile = col / kSkBN, cin = col % kSkBN;
        const float *pp = a.part + (((size_t)tile * a.ksplit) * kSkM + row) * kSkBN + cin;
        const size_t sstride = (size_t)kSkM * kSkBN;
#pragma unroll 1
        for (int s0 = 0; s0 < a.ksplit; s0 += kFinSliceGroup) {
            float4 p[2 * kFinSliceGroup];
#pragma unroll
            for (int u = 0; u < kFinSliceGroup; ++u) {
                const int s = min(s0 + u, a.ksplit - 1);   // (a repeated slice is loaded but not added)
                p[2 * u] = *reinterpret_cast<const float4 *>(pp + s * sstride);
                p[2 * u + 1] = *reinterpret_cast<const float4 *>(pp + s * sstride + 4);
            }
#pragma unroll
            for (int u = 0; u < kFinSliceGroup; ++u) {
                if (s0 + u < a.ksplit) {
                    f[0] += p[2 * u].x; f[1] += p[2 * u].y; f[2] += p[2 * u].z; f[3] += p[2 * u].w;
                    f[4] += p[2 * u + 1].x; f[5] += p[2 * u + 1].y; f[6] += p[2 * u + 1].z; f[7] += p[2 * u + 1].w;
                }
            }
        }
    }
    int n_present = 0;
    if (a.meta != nullptr) {
        __syncthreads();
        n_present = n_present_s;
    }
    if (n_present > 0) {
        // ---- second round of loads: the B rows of a group of adapters, and (first group) t of this block's rows for
        // this column block: the slice partials of each row's own adapter, added in slice order.  The code is kept
        // small on purpose (one copy of each phase, short unrolled bodies): every warp runs it once, so its cost is
        // the instruction fetch.
        constexpr int kVec = kRankPadMax / 8, kPer = kFinAdGroup * kFinCols * kVec / kFinThreads;   // 8 vectors per thread
        const int my_slot = mine ? slot_s[rr] : -1;
#pragma unroll 1
        for (int g0 = 0; g0 < n_present; g0 += kFinAdGroup) {
            if (g0 > 0) __syncthreads();   // the previous group's B tile is no longer read
            uint4 bv[kPer];
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int idx = j * kFinThreads + threadIdx.x;
                const int g = idx / (kFinCols * kVec), c = (idx / kVec) % kFinCols, v = idx % kVec;
                bv[j] = make_uint4(0, 0, 0, 0);
                if (g0 + g < n_present && colb + c < a.N && v * 8 < rpad_s[g0 + g])
                    bv[j] = __ldg(reinterpret_cast<const uint4 *>(a.b_all + ((size_t)id_s[g0 + g] * a.N + colb + c) * kRankPadMax) + v);
            }
            if (g0 == 0) {
                constexpr int kRowsPerPass = kFinThreads / kRankPadMax;   // 4 rows per pass, a thread owns rank column r
                constexpr int kTRows = 8;   // rows of a thread whose loads are in flight together (all of them)
                const int r = threadIdx.x & (kRankPadMax - 1), rq = threadIdx.x / kRankPadMax;
                const size_t sstride = (size_t)kSkM * a.p_cap * (3 * kRankPadMax);
#pragma unroll 1
                for (int j0 = 0; j0 < kFinRows / kRowsPerPass; j0 += kTRows) {
                    const float *tp[kTRows];
                    float t[kTRows];
#pragma unroll
                    for (int j = 0; j < kTRows; ++j) {
                        const int rr2 = (j0 + j) * kRowsPerPass + rq, slot = slot_s[rr2];
                        tp[j] = (slot >= 0 && r < rpad_s[slot])
                                    ? a.t_part + ((size_t)(row0 + rr2) * a.p_cap + slot) * (3 * kRankPadMax) + blk * kRankPadMax + r
                                    : nullptr;
                        t[j] = 0.f;
                    }
#pragma unroll 1
                    for (int s0 = 0; s0 < a.ksplit; s0 += kFinSliceGroup) {
                        float v[kTRows][kFinSliceGroup];
#pragma unroll
                        for (int j = 0; j < kTRows; ++j)
#pragma unroll
                            for (int u = 0; u < kFinSliceGroup; ++u)
                                v[j][u] = (tp[j] && s0 + u < a.ksplit) ? tp[j][(s0 + u) * sstride] : 0.f;
#pragma unroll
                        for (int j = 0; j < kTRows; ++j)
#pragma unroll
                            for (int u = 0; u < kFinSliceGroup; ++u) t[j] += v[j][u];
                    }
#pragma unroll
                    for (int j = 0; j < kTRows; ++j) {
                        const int rr2 = (j0 + j) * kRowsPerPass + rq;
                        t_s[rr2][r] = tp[j] ? t[j] * scale_s[slot_s[rr2]] : 0.f;
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int idx = j * kFinThreads + threadIdx.x;
                const int g = idx / (kFinCols * kVec), c = (idx / kVec) % kFinCols, v = idx % kVec;
                b_s[g][c][v ^ ((c >> 3) & 7)] = bv[j];
            }
            __syncthreads();    // t_s (first pass) and the B tile are complete
            if (my_slot >= g0 && my_slot < g0 + kFinAdGroup) {
                // only rows with an applied adapter add anything (a gated-off row never sees "+ 0")
                const int g = my_slot - g0, rv = rpad_s[my_slot] / 8;
                float d[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) d[e] = 0.f;
#pragma unroll 1
                for (int v = 0; v < rv; ++v) {   // 8 rank columns per step, the 8 outputs as independent chains
                    const float4 t0 = *reinterpret_cast<const float4 *>(&t_s[rr][v * 8]);
                    const float4 t1 = *reinterpret_cast<const float4 *>(&t_s[rr][v * 8 + 4]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint4 b = b_s[g][c0 + e][v ^ (c0 >> 3)];
                        const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&b);
                        const float2 b0 = __bfloat1622float2(p[0]), b1 = __bfloat1622float2(p[1]);
                        const float2 b2 = __bfloat1622float2(p[2]), b3 = __bfloat1622float2(p[3]);
                        float acc = d[e];
                        acc = fmaf(b0.x, t0.x, acc); acc = fmaf(b0.y, t0.y, acc);
                        acc = fmaf(b1.x, t0.z, acc); acc = fmaf(b1.y, t0.w, acc);
                        acc = fmaf(b2.x, t1.x, acc); acc = fmaf(b2.y, t1.y, acc);
                        acc = fmaf(b3.x, t1.z, acc); acc = fmaf(b3.y, t1.w, acc);
                        d[e] = acc;
                    }
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] += d[e];
            }
        }
    }
    if (!mine) return;
    if (a.residual) {
        const uint4 rv4 = *reinterpret_cast<const uint4 *>(a.residual + (size_t)row * a.ldo + col);
        const uint32_t rw[4] = {rv4.x, rv4.y, rv4.z, rv4.w};
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
    *reinterpret_cast<uint4 *>(a.out + (size_t)row * a.ldo + col) = o;
    const int kc = col - a.Nq;   // column inside [k | v]
    if (a.kv_pool != nullptr && kc >= 0) {
        const int slot = a.slot_map[row];
        if (slot >= 0) {
            const int page = slot / a.kv_page_size, prow = slot % a.kv_page_size;
            if (page >= a.kv_num_pages) { report(a.status, ALORA_ERR_PAGE_RANGE); return; }
            const int plane = kc >= a.Nkv ? 1 : 0, c2 = kc - plane * a.Nkv;
            const int head = c2 >> a.kv_hd_shift, dd = c2 & ((1 << a.kv_hd_shift) - 1);
            __nv_bfloat16 *dst = a.kv_pool +
                ((((size_t)page * 2 + plane) * a.kv_heads + head) * a.kv_page_size + prow << a.kv_hd_shift) + dd;
            *reinterpret_cast<uint4 *>(dst) = o;
        }
    }
}

// ---- host side -------------------------------------------------------------------------------------
bool make_tensor_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t ld,
                          uint32_t box_rows);   // gemm_tcgen05.cu

// Whether a projection of T rows onto N columns takes this route: decided by the shapes alone (`lora`: the layer
// has adapters registered), so that a base-only call and an adapter call of the same batch shape take the same one.
static int skinny_p_cap(const alora_ctx *ctx, int T) {
    return std::min(std::min(ctx->cfg.max_adapters, T), ctx->skinny_p_cap);   // worst case: a different adapter per row
}
bool skinny_route(const alora_ctx *ctx, int T, int N, int K, bool lora, int Nq, int Nkv) {
    if (ctx->d_skinny_part == nullptr || T < 1 || T > kSkM || N % 8 != 0 || K % 8 != 0) return false;
    const int n_tiles = (N + kSkBN - 1) / kSkBN;
    if (n_tiles > ctx->skinny_max_items) return false;
    if (lora) {
        if (Nq % kFinCols != 0 || Nkv % kFinCols != 0 || ctx->cfg.max_adapters > 1024) return false;
        if (std::min(ctx->cfg.max_adapters, T) > ctx->skinny_p_cap) return false;
        if ((skinny_p_cap(ctx, T) * kSkChunksPerAdapter + n_tiles - 1) / n_tiles > kSkMaxChunks) return false;
    }
    return true;
}

// x[T][K] (T <= 128) times W[N][K]^T.  `lora`: the layer's adapter table, its B slab and its A-row tensor map (box of
// 16 rows), or nullptr for a plain dense projection.  Returns kernels launched, or -1.
int launch_skinny_tc(alora_ctx *ctx, const void *x, const CUtensorMap &tmW, const CUtensorMap *tmA16,
                     const AdapterDev *adapters, const void *b_all, int T, int K, int N, int Nq, int Nkv, void *out,
                     const void *residual, void *kv_pool, int num_pages, cudaStream_t s) {
    static bool attr_set[64] = {};
    const int dev = ctx->cfg.device;
    int extra_launches = 0;
    const int n_tiles = (N + kSkBN - 1) / kSkBN;
    const int kb_total = (K + kSkBK - 1) / kSkBK;
    const int ksplit = std::max(1, std::min(kb_total, ctx->sm_count / n_tiles));
    const bool lora = adapters != nullptr && tmA16 != nullptr;
    if (!skinny_route(ctx, T, N, K, lora, Nq, Nkv)) return -1;
    const int p_cap = lora ? skinny_p_cap(ctx, T) : 0;
    const int chunk_cap = lora ? (p_cap * kSkChunksPerAdapter + n_tiles - 1) / n_tiles : 0;
    CUtensorMap tmX;
    const bool half_box = T <= kSkM / 2;
    if (!make_tensor_map_bf16(&tmX, x, T, K, K, half_box ? kSkM / 2 : kSkM)) return -1;
    SkinnyArgs a{};
    a.T = T; a.N = N; a.K = K; a.n_tiles = n_tiles; a.ksplit = ksplit;
    a.x_box_bytes = half_box ? kSkABytes / 2 : kSkABytes;
    a.chunk_cap = chunk_cap;
    a.stage_bytes = a.x_box_bytes + kSkWBytes + chunk_cap * kSkChunkBytes;
    // shared memory of a block: 227 KB less 1 KB for the kernel's static part, less alignment slack and barriers
    constexpr int kDynSmemMax = 227 * 1024 - 1024;
    a.n_stages = std::min(kSkMaxStages, (kDynSmemMax - 1024 - 256) / a.stage_bytes);
    if (a.n_stages < 2) return -1;
    a.part = ctx->d_skinny_part; a.t_part = ctx->d_skinny_t; a.p_cap = p_cap;
    a.row_adapter = lora ? ctx->d_row_adapter : nullptr;
    a.meta = lora ? (const FewRowMeta *)ctx->d_skinny_meta : nullptr;
    a.max_adapters = ctx->cfg.max_adapters; a.status = ctx->d_status;
    const size_t smem = (size_t)a.n_stages * a.stage_bytes + 1024 + 256;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(gemm_skinny_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemMax) != cudaSuccess)
            return -1;
        attr_set[dev] = true;
    }
    const int grid = std::min(ctx->sm_count, n_tiles * ksplit);
    if (launch_kernel(gemm_skinny_kernel, dim3(grid), dim3(kSkThreads), smem, s, true, tmX, tmW, lora ? *tmA16 : tmW, a) !=
        cudaSuccess)
        return -1;
    if (ctx->pending_attn_meta != nullptr) {
        // the attention work lists of this batch are built now, beside the weight stream (a dependent launch that
        // reads nothing this kernel writes; its blocks wait for this kernel before they exit)
        const BatchArgs *bm = ctx->pending_attn_meta;
        ctx->pending_attn_meta = nullptr;
        if (launch_metadata(ctx, *bm, s, kMetaAttention, /*timed=*/false) < 0) return -1;
        ++extra_launches;
    }
    SkinnyFinArgs f{};
    f.T = T; f.N = N; f.n_tiles = n_tiles; f.ksplit = ksplit; f.p_cap = p_cap;
    f.part = ctx->d_skinny_part; f.t_part = ctx->d_skinny_t;
    f.meta = a.meta; f.b_all = (const __nv_bfloat16 *)b_all;
    f.Nq = Nq; f.Nkv = Nkv; f.residual = (const __nv_bfloat16 *)residual; f.out = (__nv_bfloat16 *)out; f.ldo = N;
    f.status = ctx->d_status;
    if (kv_pool != nullptr) {
        int shift = 0;
        while ((1 << shift) < ctx->d.hd) ++shift;
        f.kv_pool = (__nv_bfloat16 *)kv_pool; f.slot_map = ctx->d_slot; f.kv_hd_shift = shift; f.kv_heads = ctx->d.Hkv;
        f.kv_page_size = ctx->d.page; f.kv_num_pages = num_pages;
    }
    if (launch_kernel(skinny_finish_kernel, dim3((N + kFinCols - 1) / kFinCols, (T + kFinRows - 1) / kFinRows),
                      dim3(kFinThreads), 0, s, true, f) != cudaSuccess)
        return -1;
    return 2 + extra_launches;
}

}  // namespace alora
