// Gated low-rank adapters on the MLP block's gate, up and down projections.  The paper adapts q, k and v and remarks
// that MLP blocks are adapted "by the corresponding equations": a row at or after its request's activation offset sees
// W + s B A, a row before it the base weight alone (the form of Eq. 5).  The dense product y = W x is the stack's
// ordinary GEMM; the low-rank part runs beside it in two steps:
//   shrink   t[row][k][blk][i] = sum_h A_k,blk[i][h] x[row][h]    for ALL registered adapters k of the layer at once:
//            one dense GEMM against the layer's slab of A rows (a few hundred output columns against the tens of
//            thousands of the base product), rounded to bf16 like every GEMM output;
//   expand   y[row][c] += s_k * sum_i t[row][k][blk(c)][i] B_k[c][i]    only on rows whose gate is open, k = the
//            row's applied adapter: mlp_expand_add_kernel below (mma.sync, fp32 accumulation, one pass over y).
// Rows whose gate is closed are neither read nor written by the expand step, so they keep the bits of the base MLP.
#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

// A rows of every adapter, rank-padded: dst[(k * nblk + blk) * RP + i][K] <- src_blk[i][K] (zero rows beyond the rank).
// B rows: dst[k][blk * width + c][RP] <- src_blk[c][rank] (zero columns beyond the rank).
__global__ void repack_mlp_kernel(const __nv_bfloat16 *__restrict__ a0, const __nv_bfloat16 *__restrict__ a1,
                                  const __nv_bfloat16 *__restrict__ b0, const __nv_bfloat16 *__restrict__ b1, int nblk,
                                  int rank, int RP, int K, int width, __nv_bfloat16 *__restrict__ A_dst,
                                  __nv_bfloat16 *__restrict__ B_dst) {
    const size_t nA = (size_t)nblk * RP * K, nB = (size_t)nblk * width * RP;
    const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < nA + nB; i += (size_t)gridDim.x * blockDim.x) {
        if (i < nA) {
            const int blk = (int)(i / ((size_t)RP * K));
            const int row = (int)((i / K) % RP);
            const int h = (int)(i % K);
            const __nv_bfloat16 *src = blk == 0 ? a0 : a1;
            A_dst[i] = row < rank ? src[(size_t)row * K + h] : zero;
        } else {
            const size_t j = i - nA;
            const int col = (int)(j / RP), c = (int)(j % RP);
            const int blk = col / width, n = col % width;
            const __nv_bfloat16 *src = blk == 0 ? b0 : b1;
            B_dst[j] = c < rank ? src[(size_t)n * rank + c] : zero;
        }
    }
}

int launch_repack_mlp(const void *a0, const void *a1, const void *b0, const void *b1, int nblk, int rank, int RP, int K,
                      int width, void *A_dst, void *B_dst, cudaStream_t s) {
    repack_mlp_kernel<<<256, 256, 0, s>>>((const __nv_bfloat16 *)a0, (const __nv_bfloat16 *)a1, (const __nv_bfloat16 *)b0,
                                         (const __nv_bfloat16 *)b1, nblk, rank, RP, K, width, (__nv_bfloat16 *)A_dst,
                                         (__nv_bfloat16 *)B_dst);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

constexpr int kMxRows = 64, kMxCols = 256, kMxThreads = 256;

struct MlpExpandArgs {
    __nv_bfloat16 *y;                  // [rows][ldy], updated in place on open-gate rows
    const __nv_bfloat16 *t;            // [rows][t_ld]: column (k * nblk + blk) * RP + i
    const __nv_bfloat16 *b;            // [adapters][ncols][RP]
    const int32_t *row_adapter;        // [rows] applied adapter of each row, -1 = none (gate closed or base model)
    const MlpAdapterDev *table;        // [adapters] padded rank and scale
    int rows, ldy, ncols, width, nblk, t_ld, RP, n_adapters;
};

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Block = 64 rows x 256 columns of y; warp w owns columns w * 32 .. w * 32 + 31 (four 8-wide tiles) of all 64 rows
// (four 16-row tiles).  The rows of a request are adjacent, so the applied adapter is constant along runs of rows: the
// block walks the runs of its 64 rows and, per run with an adapter, accumulates t (rows outside the run masked to
// zero) times that adapter's B rows.  Every row belongs to one run, so its accumulator holds its own adapter's
// product alone and the scale is applied per row at the end.
__global__ void __launch_bounds__(kMxThreads) mlp_expand_add_kernel(const MlpExpandArgs a) {
    tc::grid_dep_launch();
    tc::grid_dep_wait();
    __shared__ int s_ad[kMxRows];
    const int row0 = (int)blockIdx.x * kMxRows;
    const int warp = (int)threadIdx.x >> 5, lane = (int)threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int col0 = (int)blockIdx.y * kMxCols + warp * 32;
    if (threadIdx.x < kMxRows) {
        const int r = row0 + (int)threadIdx.x;
        int k = r < a.rows ? a.row_adapter[r] : -1;
        if (k >= a.n_adapters || (k >= 0 && a.table[k].rpad <= 0)) k = -1;   // no MLP part registered: base rows
        s_ad[threadIdx.x] = k;
    }
    __syncthreads();
    if (col0 >= a.ncols) return;
    const int blk = col0 / a.width;
    float acc[4][4][4];
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
    bool any = false;
    for (int ra = 0; ra < kMxRows;) {
        const int k = s_ad[ra];
        int rb = ra + 1;
        while (rb < kMxRows && s_ad[rb] == k) ++rb;
        if (k >= 0) {
            any = true;
            const int rpad = min(a.table[k].rpad, a.RP);
            const __nv_bfloat16 *tk = a.t + (size_t)(k * a.nblk + blk) * a.RP;
            const __nv_bfloat16 *bk = a.b + ((size_t)k * a.ncols + col0) * a.RP;
            for (int ks = 0; ks < rpad; ks += 16) {
                uint32_t bf[4][2];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    const bool in = col0 + nt * 8 + g < a.ncols;
                    const __nv_bfloat16 *p = bk + (size_t)(nt * 8 + g) * a.RP + ks + 2 * q;
                    bf[nt][0] = in ? *reinterpret_cast<const uint32_t *>(p) : 0u;
                    bf[nt][1] = in ? *reinterpret_cast<const uint32_t *>(p + 8) : 0u;
                }
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
                    if (rb <= mt * 16 || ra >= mt * 16 + 16) continue;   // the run has no row in this tile
                    const int lo = mt * 16 + g, hi = lo + 8;
                    const bool in_lo = lo >= ra && lo < rb, in_hi = hi >= ra && hi < rb;
                    const __nv_bfloat16 *plo = tk + (size_t)(row0 + lo) * a.t_ld + ks + 2 * q;
                    const __nv_bfloat16 *phi = tk + (size_t)(row0 + hi) * a.t_ld + ks + 2 * q;
                    uint32_t af[4];
                    af[0] = in_lo ? *reinterpret_cast<const uint32_t *>(plo) : 0u;
                    af[1] = in_hi ? *reinterpret_cast<const uint32_t *>(phi) : 0u;
                    af[2] = in_lo ? *reinterpret_cast<const uint32_t *>(plo + 8) : 0u;
                    af[3] = in_hi ? *reinterpret_cast<const uint32_t *>(phi + 8) : 0u;
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) mma_bf16_16816(acc[mt][nt], af, bf[nt][0], bf[nt][1]);
                }
            }
        }
        ra = rb;
    }
    if (!any) return;
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int lr = mt * 16 + g + half * 8;
            const int k = s_ad[lr];
            if (k < 0) continue;
            const float sc = a.table[k].scale;
            __nv_bfloat16 *yr = a.y + (size_t)(row0 + lr) * a.ldy + col0 + 2 * q;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                if (col0 + nt * 8 + 2 * q >= a.ncols) continue;
                __nv_bfloat162 *p = reinterpret_cast<__nv_bfloat162 *>(yr + nt * 8);
                const float2 v = __bfloat1622float2(*p);
                *p = __floats2bfloat162_rn(fmaf(sc, acc[mt][nt][half * 2], v.x), fmaf(sc, acc[mt][nt][half * 2 + 1], v.y));
            }
        }
    }
}

// y[rows][ldy] += the low-rank delta of the rows' applied adapters (see the head of this file).  `t` holds the shrink
// results of all adapters of the layer, `b` the layer's slab of B rows.  Returns kernels launched, or -1.
int launch_mlp_expand(alora_ctx *ctx, void *y, int ldy, int rows, const void *t, int t_ld, const void *b, int ncols,
                      int width, int nblk, const int32_t *row_adapter, const MlpAdapterDev *table, int n_adapters,
                      cudaStream_t s) {
    if (rows <= 0) return 0;
    if (ncols % 8 != 0 || width % 32 != 0 || ldy % 2 != 0 || t_ld % 2 != 0) return -1;
    MlpExpandArgs a{};
    a.y = (__nv_bfloat16 *)y; a.t = (const __nv_bfloat16 *)t; a.b = (const __nv_bfloat16 *)b;
    a.row_adapter = row_adapter; a.table = table;
    a.rows = rows; a.ldy = ldy; a.ncols = ncols; a.width = width; a.nblk = nblk; a.t_ld = t_ld; a.RP = ctx->d.RP;
    a.n_adapters = n_adapters;
    ProfScope prof(ctx, KK_LINEAR, s);
    const dim3 grid((rows + kMxRows - 1) / kMxRows, (ncols + kMxCols - 1) / kMxCols);
    if (launch_kernel(mlp_expand_add_kernel, grid, dim3(kMxThreads), 0, s, true, a) != cudaSuccess) return -1;
    return 1;
}

}  // namespace alora
