// Gated low-rank adapters on the MLP block's gate, up and down projections.  The paper adapts q, k and v and remarks
// that MLP blocks can be adapted in the same manner: a row at or after its request's activation offset sees
// W + s B A, a row before it the base weight alone (the form of Eq. 5).  The dense product y = W x is the stack's
// ordinary GEMM; the low-rank part runs beside it in two steps:
//   shrink   t[row][k][blk][i] = sum_h A_k,blk[i][h] x[row][h]    for ALL registered adapters k of the layer at once:
//            one launch against the layer's slab of A rows (a few hundred output columns against the tens of
//            thousands of the base product), rounded to bf16 like every GEMM output: mlp_shrink_kernel below;
//   expand   y[row][c] += s_k * sum_i t[row][k][blk(c)][i] B_k[c][i]    only on rows whose gate is open, k = the
//            row's applied adapter: mlp_expand_add_kernel below (mma.sync, fp32 accumulation, one pass over y).
// Rows whose gate is closed are neither read nor written by the expand step, so they keep the bits of the base MLP.
#include <algorithm>

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

constexpr int kMxRows = 64, kMxCols = 128, kMxThreads = 128;   // block tile of the expand step; one warp per 32 columns
constexpr int kMxRowsPerWarp = 32 / (kMxThreads / 32);            // rows of a 32-row pass that one warp updates
constexpr int kMxLanesPerRow = kMxCols / 8;                       // a lane updates a 16-byte piece (8 columns) of a row
constexpr int kMxRowsPerInst = 32 / kMxLanesPerRow;               // rows one warp instruction covers
constexpr int kMxUpdates = kMxRowsPerWarp / kMxRowsPerInst;       // update instructions per warp and pass
static_assert(kMxCols == 32 * (kMxThreads / 32) && 32 % kMxLanesPerRow == 0 && kMxRowsPerWarp % kMxRowsPerInst == 0, "tile shape");

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

// 16-byte asynchronous copy global -> shared; src_bytes (0 or 16) of the source are read, the rest is zero-filled
__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *gmem_src, int src_bytes) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gmem_src), "r"(src_bytes) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void *smem_row) {
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_row);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// ---------------------------------------------------------------------------------------------------------------
// Shrink: t[row][c] = sum_h x[row][h] A[c][h] for the A rows of all the layer's MLP adapters (c = (adapter, block, rank
// row), a few hundred at most) -- a product with very many rows, a long inner dimension and very few columns, which the
// tile kernels of the dense projections serve badly (one 128-column tile per 128 rows: 16 of 148 SMs busy on 2048
// rows).  Here a block takes 64 rows x 64 columns x one slice of K (mma.sync, fp32 accumulation, operands brought to
// shared memory by asynchronous copies, the next K chunk's in flight under the current chunk's arithmetic); K is cut into as
// many slices (at most 8) as it takes to give every SM about two blocks.  With more than one slice the blocks store fp32 partial tiles
// and count themselves per (row tile, column tile); the block that stores a tile's last slice adds the partials in
// slice order (fixed order: run-to-run identical) and writes bf16.
// ---------------------------------------------------------------------------------------------------------------
constexpr int kShRows = 64, kShCols = 64, kShChunk = 64, kShThreads = 128, kShLd = 72, kShMaxSplit = 8;

struct MlpShrinkArgs {
    const __nv_bfloat16 *x;     // [rows][K]
    const __nv_bfloat16 *a;     // [n_cols][K]: the layer's slab of A rows
    __nv_bfloat16 *t;           // [rows][n_cols]
    float *part;                // [ksplit][row tiles * 64][n_cols] fp32 (ksplit > 1)
    int32_t *done;              // [row tiles * column tiles] slices stored so far; the finishing block puts 0 back
    int rows, K, n_cols, ksplit;
};

__global__ void __launch_bounds__(kShThreads) mlp_shrink_kernel(const MlpShrinkArgs a) {
    tc::grid_dep_launch();
    tc::grid_dep_wait();
    __shared__ __align__(16) __nv_bfloat16 xs[2][kShRows * kShLd];
    __shared__ __align__(16) __nv_bfloat16 as[2][kShCols * kShLd];
    __shared__ int last_s;
    const int warp = (int)threadIdx.x >> 5, lane = (int)threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int col0 = (int)blockIdx.x * kShCols, row0 = (int)blockIdx.y * kShRows, ks = (int)blockIdx.z;
    const int n_chunks = (a.K + kShChunk - 1) / kShChunk;
    const int c_base = n_chunks / a.ksplit, c_rem = n_chunks % a.ksplit;
    const int c0 = ks * c_base + min(ks, c_rem), nc = c_base + (ks < c_rem ? 1 : 0);
    // a thread's four 16-byte pieces of each operand tile: piece p = threadIdx.x + 128 i -> row p / 8, vector p % 8.
    // The pieces go from global to shared memory by asynchronous copies (no trip through registers and no store
    // instruction: the kernel is bound by its shared-memory traffic); a piece outside K or past the last A row is
    // filled with zeros (zero source bytes), rows past the end repeat the last row and their results are dropped.
    auto issue = [&](int chunk, int buf) {
        const int k0 = chunk * kShChunk;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int p = (int)threadIdx.x + kShThreads * i, r = p >> 3, v = p & 7;
            const int k = k0 + v * 8;
            const bool kin = k < a.K;   // K is a multiple of 8: a vector is inside or outside as a whole
            const int xrow = min(row0 + r, a.rows - 1);
            const int acol = col0 + r;
            const bool ain = kin && acol < a.n_cols;
            const __nv_bfloat16 *sx = a.x + (size_t)xrow * a.K + (kin ? k : 0);
            const __nv_bfloat16 *sa = a.a + (ain ? (size_t)acol * a.K + k : 0);
            cp_async_16(&xs[buf][r * kShLd + v * 8], sx, kin ? 16 : 0);
            cp_async_16(&as[buf][r * kShLd + v * 8], sa, ain ? 16 : 0);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float acc[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
    if (nc > 0) issue(c0, 0);
    for (int c = 0; c < nc; ++c) {
        const int buf = c & 1;
        if (c + 1 < nc) {
            issue(c0 + c + 1, buf ^ 1);        // the next chunk's copies fly under this chunk's arithmetic
            asm volatile("cp.async.wait_group 1;" ::: "memory");   // all but the copies just issued have landed
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();                       // every thread's pieces of this chunk are in shared memory
#pragma unroll
        for (int kk = 0; kk < kShChunk; kk += 16) {
            uint32_t af[4];
            ldmatrix_x4(af, &xs[buf][(warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * kShLd + kk + (lane >> 4) * 8]);
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t bf[4];
                ldmatrix_x4(bf, &as[buf][(np * 16 + (lane & 7) + ((lane >> 4) & 1) * 8) * kShLd + kk + ((lane >> 3) & 1) * 8]);
                mma_bf16_16816(acc[2 * np], af, bf[0], bf[1]);
                mma_bf16_16816(acc[2 * np + 1], af, bf[2], bf[3]);
            }
        }
        __syncthreads();                       // this buffer may be overwritten by the copies of chunk c + 2
    }
    // this thread's accumulator elements: rows row0 + warp * 16 + g (+ 8), columns col0 + nt * 8 + 2 q (+ 1)
    const int r_lo = row0 + warp * 16 + g, r_hi = r_lo + 8;
    if (a.ksplit == 1) {
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const int col = col0 + nt * 8 + 2 * q;
            if (col >= a.n_cols) continue;
            if (r_lo < a.rows) *reinterpret_cast<__nv_bfloat162 *>(a.t + (size_t)r_lo * a.n_cols + col) = __floats2bfloat162_rn(acc[nt][0], acc[nt][1]);
            if (r_hi < a.rows) *reinterpret_cast<__nv_bfloat162 *>(a.t + (size_t)r_hi * a.n_cols + col) = __floats2bfloat162_rn(acc[nt][2], acc[nt][3]);
        }
        return;
    }
    const size_t rows_pad = (size_t)gridDim.y * kShRows;
    float *mine = a.part + (size_t)ks * rows_pad * a.n_cols;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        const int col = col0 + nt * 8 + 2 * q;
        if (col >= a.n_cols) continue;
        *reinterpret_cast<float2 *>(mine + (size_t)r_lo * a.n_cols + col) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2 *>(mine + (size_t)r_hi * a.n_cols + col) = make_float2(acc[nt][2], acc[nt][3]);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        int32_t *cnt = a.done + (size_t)blockIdx.y * gridDim.x + blockIdx.x;
        const int last = atomicAdd(cnt, 1) == a.ksplit - 1 ? 1 : 0;
        if (last) *cnt = 0;      // (nobody else counts on this tile any more in this launch)
        last_s = last;
    }
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    // 64 rows x 64 columns = 1024 float4; thread i takes float4 i, i + 128, ...: row = idx / 16, columns 4 (idx % 16) ..
    for (int idx = (int)threadIdx.x; idx < kShRows * (kShCols / 4); idx += kShThreads) {
        const int r = row0 + idx / (kShCols / 4), col = col0 + (idx % (kShCols / 4)) * 4;
        if (r >= a.rows || col >= a.n_cols) continue;     // n_cols is a multiple of 8
        // all slices' loads in flight together (one round trip to L2 per output vector, not one per slice), then
        // added in slice order
        float4 v[kShMaxSplit];
#pragma unroll
        for (int s2 = 0; s2 < kShMaxSplit; ++s2)
            if (s2 < a.ksplit)
                v[s2] = __ldcg(reinterpret_cast<const float4 *>(a.part + ((size_t)s2 * rows_pad + r) * a.n_cols + col));
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s2 = 0; s2 < kShMaxSplit; ++s2)
            if (s2 < a.ksplit) { sum.x += v[s2].x; sum.y += v[s2].y; sum.z += v[s2].z; sum.w += v[s2].w; }
        uint2 o;
        *reinterpret_cast<__nv_bfloat162 *>(&o.x) = __floats2bfloat162_rn(sum.x, sum.y);
        *reinterpret_cast<__nv_bfloat162 *>(&o.y) = __floats2bfloat162_rn(sum.z, sum.w);
        *reinterpret_cast<uint2 *>(a.t + (size_t)r * a.n_cols + col) = o;
    }
}

// t[rows][n_cols] = x[rows][K] A[n_cols][K]^T, bf16.  `part` holds part_floats floats, `done` one counter per 64 x 64
// tile (zero between launches).  Returns kernels launched, or -1.
int launch_mlp_shrink(alora_ctx *ctx, const void *x, const void *A, int rows, int K, int n_cols, void *t, float *part,
                      size_t part_floats, int32_t *done, int done_ints, cudaStream_t s) {
    if (rows <= 0) return 0;
    if (K % 8 != 0 || n_cols % 8 != 0 || n_cols <= 0) return -1;
    const int col_tiles = (n_cols + kShCols - 1) / kShCols, row_tiles = (rows + kShRows - 1) / kShRows;
    const int n_chunks = (K + kShChunk - 1) / kShChunk;
    // about two blocks per SM, at least two K chunks per block (more slices were slower: the kernel is bound by its
    // shared-memory traffic, and every slice adds a partial tile to store and to add up)
    int ksplit = (2 * ctx->sm_count + col_tiles * row_tiles - 1) / (col_tiles * row_tiles);
    ksplit = std::max(1, std::min(std::min(ksplit, kShMaxSplit), n_chunks / 2));
    while (ksplit > 1 && (size_t)ksplit * row_tiles * kShRows * n_cols > part_floats) --ksplit;
    if (col_tiles * row_tiles > done_ints) ksplit = 1;
    MlpShrinkArgs a{};
    a.x = (const __nv_bfloat16 *)x; a.a = (const __nv_bfloat16 *)A; a.t = (__nv_bfloat16 *)t; a.part = part; a.done = done;
    a.rows = rows; a.K = K; a.n_cols = n_cols; a.ksplit = ksplit;
    ProfScope prof(ctx, KK_LINEAR, s);
    if (launch_kernel(mlp_shrink_kernel, dim3(col_tiles, row_tiles, ksplit), dim3(kShThreads), 0, s, true, a) != cudaSuccess)
        return -1;
    return 1;
}

constexpr int kMxLd = 72;   // shared-memory row length of the t and B tiles in bf16: 64 + 8 (144 bytes: rows stay
                            // 16-byte aligned and eight consecutive rows fall into different banks for ldmatrix)
constexpr int kMxSB = kMxCols * kMxLd * 2, kMxST = kMxRows * kMxLd * 2;

// Block = 64 rows x 128 columns of y (all of one block of the projection: gate or up); warp w owns columns
// w * 32 .. w * 32 + 31 (four 8-wide tiles) of all 64 rows (four 16-row tiles).  The rows of a request are adjacent, so
// the applied adapter is constant along runs of rows: the block walks the runs of its 64 rows and, per run with an
// adapter, brings that adapter's 128 B rows and the run's t rows (rows outside the run as zeros) into shared memory
// with 16-byte loads, takes the fragments by ldmatrix and accumulates.  Every row belongs to one run, so its
// accumulator holds its own adapter's product alone and the scale is applied per row at the end.
__global__ void __launch_bounds__(kMxThreads, 4) mlp_expand_add_kernel(const MlpExpandArgs a) {
    tc::grid_dep_launch();
    tc::grid_dep_wait();
    __shared__ int s_ad[kMxRows];
    __shared__ unsigned s_starts[2];                    // bit i of word w: row 32 w + i starts a run
    __shared__ __align__(16) unsigned char s_raw[kMxSB + kMxST];
    __nv_bfloat16 *sB = reinterpret_cast<__nv_bfloat16 *>(s_raw);
    __nv_bfloat16 *sT = reinterpret_cast<__nv_bfloat16 *>(s_raw + kMxSB);
    // (column blocks are the fast grid dimension: the blocks that run together cover whole rows of y)
    const int row0 = (int)blockIdx.y * kMxRows, cbase = (int)blockIdx.x * kMxCols;
    const int warp = (int)threadIdx.x >> 5, lane = (int)threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int col0 = cbase + warp * 32;
    if (threadIdx.x < kMxRows) {
        // the row's applied adapter, or -1: gate closed, base model, past the last row, no MLP part registered
        auto applied = [&](int r) {
            const int k = r < a.rows ? a.row_adapter[r] : -1;
            return (k < 0 || k >= a.n_adapters || a.table[k].rpad <= 0) ? -1 : k;
        };
        const int r = row0 + (int)threadIdx.x;
        const int k = applied(r);
        s_ad[threadIdx.x] = k;
        const bool start = threadIdx.x == 0 || k != applied(r - 1);
        const unsigned starts = __ballot_sync(0xffffffffu, start);
        if (lane == 0) s_starts[warp] = starts;
    }
    __syncthreads();
    const unsigned long long run_starts = (unsigned long long)s_starts[0] | ((unsigned long long)s_starts[1] << 32);
    const bool warp_in = col0 < a.ncols;               // (warps past the last column still fill tiles and join barriers)
    const int blk = cbase / a.width;                   // the width is a multiple of the block's columns
    // The y values this thread will update are requested now: their trip to DRAM overlaps the tile fills and the
    // MMAs, and a block keeps its whole tile of reads in flight from its first microsecond on.
    // (a lane owns the 16-byte piece uc of row pass * 32 + warp * kMxRowsPerWarp + i * kMxRowsPerInst + ur)
    const int ur = lane / kMxLanesPerRow, uc = (lane % kMxLanesPerRow) * 8;
    const bool col_in = cbase + uc < a.ncols;          // ncols is a multiple of 8: a piece is inside or outside as a whole
    uint4 yv[2][kMxUpdates];
#pragma unroll
    for (int pass = 0; pass < 2; ++pass)
#pragma unroll
        for (int i = 0; i < kMxUpdates; ++i) {
            const int lr = pass * 32 + warp * kMxRowsPerWarp + i * kMxRowsPerInst + ur;
            yv[pass][i] = (s_ad[lr] >= 0 && col_in)
                              ? *reinterpret_cast<const uint4 *>(a.y + (size_t)(row0 + lr) * a.ldy + cbase + uc)
                              : make_uint4(0u, 0u, 0u, 0u);
        }
    float acc[4][4][4];
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
    bool any = false;
    for (int ra = 0; ra < kMxRows;) {                  // (block-uniform: every thread sees the same runs)
        const int k = s_ad[ra];
        const unsigned long long later = ra + 1 < kMxRows ? run_starts >> (ra + 1) : 0ull;
        const int rb = later ? ra + __ffsll((long long)later) : kMxRows;     // the next run's first row
        if (k >= 0) {
            const int rpad = min(a.table[k].rpad, a.RP);
            const int cpr = rpad >> 3;                 // 16-byte pieces per row
            if (any) __syncthreads();                  // the previous run's fragments have been taken
            any = true;
            const __nv_bfloat16 *tk = a.t + (size_t)(k * a.nblk + blk) * a.RP;
            const __nv_bfloat16 *bk = a.b + ((size_t)k * a.ncols + cbase) * a.RP;
            // (asynchronous copies; a piece outside the run or past the last column reads nothing and is zero-filled)
            for (int i = (int)threadIdx.x; i < kMxRows * cpr; i += kMxThreads) {
                const int r = i / cpr, c = i - r * cpr;
                const bool in = r >= ra && r < rb;
                cp_async_16(sT + r * kMxLd + c * 8, in ? tk + (size_t)(row0 + r) * a.t_ld + c * 8 : a.t, in ? 16 : 0);
            }
            for (int i = (int)threadIdx.x; i < kMxCols * cpr; i += kMxThreads) {
                const int n = i / cpr, c = i - n * cpr;
                const bool in = cbase + n < a.ncols;
                cp_async_16(sB + n * kMxLd + c * 8, in ? bk + (size_t)n * a.RP + c * 8 : a.b, in ? 16 : 0);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();
            if (warp_in) {
                for (int ks = 0; ks < rpad; ks += 16) {
                    // B fragments of two 8-column tiles per ldmatrix: rows = columns of y, 16 ranks wide
                    uint32_t bf[2][4];
#pragma unroll
                    for (int np = 0; np < 2; ++np)
                        ldmatrix_x4(bf[np], sB + (warp * 32 + np * 16 + (lane & 7) + ((lane >> 4) & 1) * 8) * kMxLd + ks +
                                                ((lane >> 3) & 1) * 8);
#pragma unroll
                    for (int mt = 0; mt < 4; ++mt) {
                        if (rb <= mt * 16 || ra >= mt * 16 + 16) continue;   // the run has no row in this tile
                        uint32_t af[4];
                        ldmatrix_x4(af, sT + (mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * kMxLd + ks + (lane >> 4) * 8);
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt)
                            mma_bf16_16816(acc[mt][nt], af, bf[nt >> 1][(nt & 1) * 2], bf[nt >> 1][(nt & 1) * 2 + 1]);
                    }
                }
            }
        }
        ra = rb;
    }
    // The deltas go through shared memory, 32 rows at a time, so that y is read and written in whole 256-byte row
    // segments (a lane's accumulator elements are 4-byte pieces of eight different rows: updating y straight from
    // the registers scatters 16-byte accesses over as many DRAM pages and ran 14x slower).  The staging rows reuse
    // the B tile's memory.
    static_assert(32 * (kMxCols + 8) * 4 <= kMxSB, "the delta rows fit into the B tile");
    float (*s_delta)[kMxCols + 8] = reinterpret_cast<float (*)[kMxCols + 8]>(s_raw);   // read as float4, written as float2
    if (!any) return;                                  // (block-uniform) no open-gate row in this tile
    __syncthreads();                                   // every warp has taken its last fragments
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
        if (pass) __syncthreads();
#pragma unroll
        for (int m2 = 0; m2 < 2; ++m2) {
            const int mt = pass * 2 + m2;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int lr = mt * 16 + g + half * 8;
                const int k = s_ad[lr];
                const float sc = k >= 0 ? a.table[k].scale : 0.f;
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
                    *reinterpret_cast<float2 *>(&s_delta[lr - pass * 32][warp * 32 + nt * 8 + 2 * q]) =
                        make_float2(sc * acc[mt][nt][half * 2], sc * acc[mt][nt][half * 2 + 1]);
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kMxUpdates; ++i) {
            const int lr = pass * 32 + warp * kMxRowsPerWarp + i * kMxRowsPerInst + ur;
            if (s_ad[lr] < 0 || !col_in) continue;             // closed gate: the row is neither read nor written
            // (lanes 4 .. 7 of every eight read their second half first: the eight 16-byte reads of a quarter warp then
            // fall into different banks)
            const int sw = (lane >> 2) & 1;
            const float4 da = *reinterpret_cast<const float4 *>(&s_delta[lr - pass * 32][uc + 4 * sw]);
            const float4 db = *reinterpret_cast<const float4 *>(&s_delta[lr - pass * 32][uc + 4 * (sw ^ 1)]);
            const float4 d0 = sw ? db : da, d1 = sw ? da : db;
            const uint4 raw = yv[pass][i];
            const float2 v0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.x));
            const float2 v1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.y));
            const float2 v2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.z));
            const float2 v3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.w));
            uint4 out;
            *reinterpret_cast<__nv_bfloat162 *>(&out.x) = __floats2bfloat162_rn(v0.x + d0.x, v0.y + d0.y);
            *reinterpret_cast<__nv_bfloat162 *>(&out.y) = __floats2bfloat162_rn(v1.x + d0.z, v1.y + d0.w);
            *reinterpret_cast<__nv_bfloat162 *>(&out.z) = __floats2bfloat162_rn(v2.x + d1.x, v2.y + d1.y);
            *reinterpret_cast<__nv_bfloat162 *>(&out.w) = __floats2bfloat162_rn(v3.x + d1.z, v3.y + d1.w);
            *reinterpret_cast<uint4 *>(a.y + (size_t)(row0 + lr) * a.ldy + cbase + uc) = out;
        }
    }
}

// y[rows][ldy] += the low-rank delta of the rows' applied adapters (see the head of this file).  `t` holds the shrink
// results of all adapters of the layer, `b` the layer's slab of B rows.  Returns kernels launched, or -1.
int launch_mlp_expand(alora_ctx *ctx, void *y, int ldy, int rows, const void *t, int t_ld, const void *b, int ncols,
                      int width, int nblk, const int32_t *row_adapter, const MlpAdapterDev *table, int n_adapters,
                      cudaStream_t s) {
    if (rows <= 0) return 0;
    if (ncols % 8 != 0 || width % kMxCols != 0 || ldy % 8 != 0 || t_ld % 8 != 0 || ((uintptr_t)y & 15) != 0) return -1;
    MlpExpandArgs a{};
    a.y = (__nv_bfloat16 *)y; a.t = (const __nv_bfloat16 *)t; a.b = (const __nv_bfloat16 *)b;
    a.row_adapter = row_adapter; a.table = table;
    a.rows = rows; a.ldy = ldy; a.ncols = ncols; a.width = width; a.nblk = nblk; a.t_ld = t_ld; a.RP = ctx->d.RP;
    a.n_adapters = n_adapters;
    ProfScope prof(ctx, KK_LINEAR, s);
    const dim3 grid((ncols + kMxCols - 1) / kMxCols, (rows + kMxRows - 1) / kMxRows);
    if (launch_kernel(mlp_expand_add_kernel, grid, dim3(kMxThreads), 0, s, true, a) != cudaSuccess) return -1;
    return 1;
}

}  // namespace alora
