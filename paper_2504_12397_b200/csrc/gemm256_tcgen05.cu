// Dense bf16 projection y = x W^T (+ residual) for large row counts: 256 x 256 output tiles per block.
//
// The 128 x 256 tile of gemm_tcgen05.cu needs 48 KB of operands per 64-wide K block for 4 x 128 cycles of
// tensor-pipe time, more than one SM can bring into shared memory in that time.  Here a block owns two
// 128-row halves that share the W tile: 64 KB per K block for 8 x 128 cycles, i.e. 1.5 x the flops per
// operand byte.  The two halves accumulate in the two halves of tensor memory (2 x 256 columns), so the
// accumulators are not double-buffered; the next tile's operand loads run under the epilogue, and its
// MMAs start on a half as soon as the epilogue has drained that half.  Used by the o_proj / MLP matrices
// of the layer stack (no adapter logic here).
//
//   warp 0   TMA producer: per K block x[256 rows][64] as two 128-row boxes and W[256 rows][64], 3 slots
//   warp 1   MMA issuer (the whole warp walks the schedule, an elected lane issues): per K block
//            4 x (128 x 256 x 16) for each half
//   warps 2-5  epilogue: tcgen05.ld one row per thread, optional residual, bf16, 16-byte stores
// All waits are bounded; on expiry ALORA_ERR_TIMEOUT is recorded and the block leaves normally.
#include <algorithm>

#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

namespace {
constexpr int kBM2 = 256, kBN2 = 256, kBK2 = 64, kStages2 = 3, kThreads2 = 192;
constexpr int kHalfA = 128 * kBK2 * 2;           // one 128-row half of the x tile
constexpr int kBBytes2 = kBN2 * kBK2 * 2;
constexpr int kStageBytes2 = 2 * kHalfA + kBBytes2;
constexpr int kBarOff2 = kStages2 * kStageBytes2;
constexpr int kSmemTotal2 = kBarOff2 + 256 + 1024;

struct Gemm256Args {
    int M, N, K;
    __nv_bfloat16 *out;
    const __nv_bfloat16 *residual;   // optional, same layout as out, may alias it
    int ldo;
    int32_t *status;
};

__global__ void __launch_bounds__(kThreads2, 1)
gemm256_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const Gemm256Args a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + kBarOff2);
    // barrier words: full[3], empty[3], acc_full, acc_empty[2] (one per half), drain
    const uint32_t bar0 = smem_base + kBarOff2;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kStages2 + s); };
    const uint32_t accf_bar = bar0 + 8u * (2 * kStages2);
    auto acce_bar = [&](int h) { return bar0 + 8u * (2 * kStages2 + 1 + h); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kStages2 + 3);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * kStages2 + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * kStages2 + 5);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages2; ++s) { tc::mbar_init(full_bar(s), 1); tc::mbar_init(empty_bar(s), 1); }
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
    tc::grid_dep_wait();   // x (and the residual) come from earlier kernels of the stream

    const int n_m = (a.M + kBM2 - 1) / kBM2, n_n = (a.N + kBN2 - 1) / kBN2;
    const int total = n_m * n_n;              // item = n * n_m + m: blocks running together share a W tile
    const int kb_n = (a.K + kBK2 - 1) / kBK2;

    if (warp == 0) {
        if (lane == 0) {
            tc::tma_prefetch_desc(&tmA); tc::tma_prefetch_desc(&tmB);
            uint32_t kc = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < total && ok; item += gridDim.x) {
                const int m0 = (item % n_m) * kBM2, n0 = (item / n_m) * kBN2;
                for (int kb = 0; kb < kb_n; ++kb, ++kc) {
                    const int s = kc % kStages2;
                    if (!tc::mbar_wait(empty_bar(s), ((kc / kStages2) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t sa = smem_base + s * kStageBytes2;
                    tc::mbar_arrive_expect_tx(full_bar(s), kStageBytes2);
                    tc::tma_load_2d(sa, &tmA, full_bar(s), kb * kBK2, m0);
                    tc::tma_load_2d(sa + kHalfA, &tmA, full_bar(s), kb * kBK2, m0 + 128);
                    tc::tma_load_2d(sa + 2 * kHalfA, &tmB, full_bar(s), kb * kBK2, n0);
                }
            }
            if (!ok) {
                // give copies already in flight time to land before the block's shared memory is released
                const uint32_t first = kc > (uint32_t)kStages2 ? kc - kStages2 : 0;
                for (uint32_t i = first; i < kc; ++i) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(full_bar(i % kStages2), (i / kStages2) & 1) &&
                           clock64() - t0 < tc::kWaitCycleLimit) {}
                }
            }
        }
    } else if (warp == 1) {
        const bool leader = tc::elect_one();
        auto wait_all = [&](uint32_t bar, uint32_t parity) {
            return __all_sync(0xffffffffu, tc::mbar_wait(bar, parity, abort_flag));
        };
        constexpr uint32_t idesc = tc::idesc_bf16_f32(128, kBN2);
        uint32_t kc = 0, it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total && ok; item += gridDim.x, ++it) {
            for (int kb = 0; kb < kb_n && ok; ++kb, ++kc) {
                const int s = kc % kStages2;
                if (!wait_all(full_bar(s), (kc / kStages2) & 1)) { ok = false; break; }
                const uint32_t sa = smem_base + s * kStageBytes2;
                const uint64_t db = tc::smem_desc_k_sw128(sa + 2 * kHalfA);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    // the half's accumulator must have been drained by the previous tile's epilogue
                    if (kb == 0 && !wait_all(acce_bar(h), (it & 1) ^ 1)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint64_t da = tc::smem_desc_k_sw128(sa + h * kHalfA);
                    if (leader) {
#pragma unroll
                        for (int k = 0; k < kBK2 / 16; ++k)
                            tc::mma_bf16(tmem_base + h * kBN2, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                }
                if (!ok) break;
                if (leader) tc::mma_commit(empty_bar(s));   // slot reusable once these MMAs have read it
            }
            if (!ok) break;
            if (leader) tc::mma_commit(accf_bar);           // both halves complete
        }
        if (!ok && leader) {
            tc::mma_commit(drain_bar);                      // wait (bounded) for tensor-core work still in flight
            const long long t0 = clock64();
            while (!tc::mbar_try_wait(drain_bar, 0) && clock64() - t0 < tc::kWaitCycleLimit) {}
        }
    } else {
        const int q = warp & 3;   // tensor-memory lane quarter this warp may read
        uint32_t it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total && ok; item += gridDim.x, ++it) {
            const int m0 = (item % n_m) * kBM2, n0 = (item / n_m) * kBN2;
            if (!tc::mbar_wait(accf_bar, it & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                const int row = m0 + h * 128 + q * 32 + lane;
                const bool row_ok = row < a.M;
                __nv_bfloat16 *orow = a.out + (size_t)row * a.ldo + n0;
                const __nv_bfloat16 *rrow = a.residual ? a.residual + (size_t)row * a.ldo + n0 : nullptr;
#pragma unroll 1
                for (int c = 0; c < kBN2; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(tmem_base + h * kBN2 + c + ((uint32_t)(q * 32) << 16), v);
                    tc::tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (n0 + c + 8 * j >= a.N) break;
                            float f[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[8 * j + e]);
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
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, 512);
    }
}
}  // namespace

bool make_tensor_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t ld,
                          uint32_t box_rows);  // gemm_tcgen05.cu

// Returns 1 (launched), 0 (shape better served by the 128-row kernel: not launched) or -1 (error).
int launch_linear256_tc(alora_ctx *ctx, const void *x, const void *W, int T, int K, int N, void *y,
                        const void *residual, cudaStream_t s) {
    const int tiles = ((T + kBM2 - 1) / kBM2) * ((N + kBN2 - 1) / kBN2);
    const int tiles128 = ((T + 127) / 128) * ((N + kBN2 - 1) / kBN2);
    const int G = ctx->sm_count;
    // share of the launch during which a block has a tile to work on, for this kernel and for the 128-row one
    const double eff = (double)tiles / ((double)((tiles + G - 1) / G) * G);
    const double eff128 = (double)tiles128 / ((double)((tiles128 + G - 1) / G) * G);
    // worth it when the rows fill the 256-row tiles and the coarser tiles do not idle the blocks too much
    if (T < 2 * kBM2 || T % 128 != 0 || K % 8 != 0 || N % 8 != 0 || eff * 1.3 < eff128) return 0;
    CUtensorMap tmX, tmW;
    if (!make_tensor_map_bf16(&tmX, x, T, K, K, 128)) return -1;
    if (!make_tensor_map_bf16(&tmW, W, N, K, K, kBN2)) return -1;
    static bool attr_set[64] = {};
    const int dev = ctx->cfg.device;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(gemm256_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotal2) !=
            cudaSuccess)
            return -1;
        attr_set[dev] = true;
    }
    Gemm256Args g{};
    g.M = T; g.N = N; g.K = K; g.out = (__nv_bfloat16 *)y; g.residual = (const __nv_bfloat16 *)residual; g.ldo = N;
    g.status = ctx->d_status;
    const int grid = std::max(1, std::min(ctx->sm_count, tiles));
    if (launch_kernel(gemm256_tcgen05_kernel, dim3(grid), dim3(kThreads2), kSmemTotal2, s, true, tmX, tmW, g) != cudaSuccess)
        return -1;
    return 1;
}

}  // namespace alora
