// Paged causal GQA attention of suffix queries on the 5th-generation tensor cores (Eq. 1 / Eq. 3).
//
// One persistent block per SM works through (request, KV head, query block) items.  A query block
// is 2 x 128 score rows ("groups"): rows are (token, query head of the KV group) pairs, so the G
// query heads that share a KV head share every K/V tile brought on chip.  Keys come in tiles of 128
// and are consumed as two half tiles of 64.  Roles:
//   warps 8, 11 TMA producers.  Warp 8: the head-dim columns 64.. of the two 128-row query tiles (3-D boxes
//               d x head x token out of the fused q/k/v rows) and, per key tile, the K rows fetched through
//               the block table (one 3-D box per 8 / 16 / 64 cache rows, both 64-wide halves of the head
//               dim); warp 11: the V rows likewise.  Three-deep rings for K and for V;
//   warps 9, 10 MMA issuers of group 0 and 1 (the whole warp walks the schedule, an elected lane
//               issues): S_g = Q_g K^T of a half tile (fp32, tensor memory; head-dim columns 0..63 of
//               Q_g are the A operand from tensor memory, the rest from shared memory), issued as soon
//               as the group has taken the previous scores into registers, and P_g V with P_g read
//               from tensor memory and V consumed in place (MN-major);
//   warps 0-3, 4-7   softmax groups g = 0, 1, one thread per score row: they put their Q row's first
//               64 columns into tensor memory, keep a running exponent reference and sum (online
//               softmax; a thread owns its whole row, so the row reductions need no cross-lane
//               traffic), write P_g (bf16 pairs) to tensor memory; the output O_g accumulates in
//               tensor memory across tiles and is rescaled only when the reference moves: when a half
//               tile's probabilities sum to more than 2^14 (2^8 for a single one on masked tiles);
//               final normalisation and store.
// While one group does its exponentials the tensor pipe works for the other group and on the group's
// own next scores.  A block of at most 128 / G tokens (a short suffix) has score rows for one group only:
// both groups then hold the same rows, group g takes half g of every key tile, and the two partial results
// are merged out of tensor memory at the end of the item.
//
// Masking: key j is visible to a row at position p iff j <= p; masked probabilities are set to
// zero explicitly, and V rows of keys at or beyond the item's causal limit are cleared in shared
// memory before use, so stale cache bytes (whatever their bit pattern) cannot reach an output.
// All waits are bounded; on expiry ALORA_ERR_TIMEOUT is recorded and the block leaves normally.
#include <type_traits>
#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

constexpr int kAttnThreads = 384;   // 8 softmax warps, TMA producer for Q and K, two MMA issuers, TMA producer for V
constexpr int kKeysPerTile = 128;   // keys per K/V stage in shared memory
constexpr int kHalfKeys = 64;       // keys per score / probability tile in tensor memory
constexpr int kKvStages = 3;

struct AttnArgs {
    const AttnWork *items;
    const int32_t *n_items;
    const int32_t *block_tables;
    int max_blocks, num_pages;
    int Hkv, G, page_size;     // G * tokens_per_group == 128
    int box_rows;              // cache rows per TMA box: 8 (pages of 8), 16 (pages of 16 / 32) or 64 (larger pages)
    int N, Nq;                 // fused row width, query part width
    float scale_log2;          // softmax scale * log2(e)
    const __nv_bfloat16 *qkv;  // [T][N], query part first
    __nv_bfloat16 *out;        // [T][Nq]
    int32_t *status;
    // work split: items below n_whole are taken whole; the key tiles of the others are concatenated and cut into runs
    const int32_t *run_counts;  // [0] key tiles in the concatenation, [1] tiles per run, [2] n_whole, [3] tiles of the whole items
    const int32_t *cta_start;   // [blocks] item that holds the first tile of the block's run
    float *part_o;              // [2 * blocks][hd][256] unnormalised output of a part, column-major over the 256 rows
    float *part_ml;             // [2 * blocks][2][256] exponent reference and row sum of a part
};

// A block's work: whole items blockIdx, blockIdx + blocks, ... below n_whole, then the pieces of its run (tiles
// [blockIdx * len, +len) of the concatenated key tiles of the items from n_whole on).  One piece = tiles [t0, t1)
// of one item.  An item cut by run boundaries is worked on by n_parts consecutive blocks (this block holds part
// `part`, the first of them is block c_first); each writes its partial result to a slot and a merge kernel adds
// the parts up afterwards.
struct RunPiece {
    AttnWork w;
    int item, t0, t1, n_parts, part, c_first;
};
struct RunIter {
    int gt, gt_end, it, len, off, n_whole, whole;
    __device__ explicit RunIter(const AttnArgs &a) {
        const int total = a.run_counts[0];
        len = a.run_counts[1];
        n_whole = a.run_counts[2];
        off = a.run_counts[3];
        whole = (int)blockIdx.x;
        gt = min(total, (int)blockIdx.x * len);
        gt_end = min(total, gt + len);
        it = gt < gt_end ? a.cta_start[blockIdx.x] : 0;
    }
    __device__ bool next(const AttnArgs &a, RunPiece &p) {
        if (whole < n_whole) {
            p.item = whole;
            whole += (int)gridDim.x;
            p.w = a.items[p.item];
            p.t0 = 0;
            p.t1 = (p.w.kv_end + kKeysPerTile - 1) / kKeysPerTile;
            p.c_first = 0; p.n_parts = 1; p.part = 0;
            return true;
        }
        if (gt >= gt_end) return false;
        p.item = it;
        p.w = a.items[it];
        const int n_tiles = (p.w.kv_end + kKeysPerTile - 1) / kKeysPerTile;
        const int first = p.w.split - off;    // the item's first tile in the concatenation
        p.t0 = gt - first;
        p.t1 = min(n_tiles, gt_end - first);
        p.c_first = first / len;
        p.n_parts = (first + n_tiles - 1) / len - p.c_first + 1;
        p.part = (int)blockIdx.x - p.c_first;
        gt = first + p.t1;
        ++it;
        return true;
    }
};
// The same interface for batches whose items are all taken whole (what the host can tell in advance for short
// batches): items blockIdx, blockIdx + blocks, ...
struct WholeIter {
    int whole, n_items;
    __device__ explicit WholeIter(const AttnArgs &a) : whole((int)blockIdx.x), n_items(*a.n_items) {}
    __device__ bool next(const AttnArgs &a, RunPiece &p) {
        if (whole >= n_items) return false;
        p.item = whole;
        whole += (int)gridDim.x;
        p.w = a.items[p.item];
        p.t0 = 0;
        p.t1 = (p.w.kv_end + kKeysPerTile - 1) / kKeysPerTile;
        p.c_first = 0; p.n_parts = 1; p.part = 0;
        return true;
    }
};
// partial-result slot of part `part` of an item whose first part is held by block c_first: a block holds at
// most one part > 0 (the piece its run starts with) and at most one part 0 of a cut item (the piece it ends with)
__host__ __device__ __forceinline__ int part_slot(int c_first, int part) { return 2 * (c_first + part) + (part == 0 ? 1 : 0); }

template <int HD>
struct AttnSmem {
    static constexpr int kQBytes = 128 * (HD - 64) * 2;      // one query tile without its first 64 columns (those live in tensor memory)
    static constexpr int kKvBytes = kKeysPerTile * HD * 2;   // one K or V tile
    static constexpr int kQOff = 0;
    static constexpr int kKOff = 2 * kQBytes;
    static constexpr int kVOff = kKOff + kKvStages * kKvBytes;
    static constexpr int kBarOff = kVOff + kKvStages * kKvBytes;
    static constexpr int kTotal = kBarOff + 256 + 1024;
};

// V tile as the B operand of P V: N = head dim (contiguous in memory: "MN-major"), K = keys.
// Rows (keys) are 128 bytes apart, 8-key groups `sbo_bytes` apart (stride byte offset); the two
// 64-wide halves of the head dim are `half_bytes` apart (leading byte offset); 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t smem_addr, uint32_t half_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFF) | ((uint64_t)((half_bytes >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | (1ull << 46) | (2ull << 61);
}
// K-major tile (rows 128 bytes apart inside an 8-row group) whose 8-row groups are `sbo_bytes` apart.
__device__ __forceinline__ uint64_t smem_desc_k_sw128_sbo(uint32_t smem_addr, uint32_t sbo_bytes) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) |
           (1ull << 46) | (2ull << 61);
}

// kind::f16 instruction descriptor with B MN-major (bit 16).
__host__ __device__ constexpr uint32_t idesc_bf16_f32_bmn(int M, int N) { return tc::idesc_bf16_f32(M, N) | (1u << 16); }

// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_32x2(uint32_t taddr, uint32_t r0, uint32_t r1) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};" ::"r"(taddr), "r"(r0), "r"(r1) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x2(uint32_t taddr, uint32_t &r0, uint32_t &r1) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                            int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ uint32_t pack_cvt(float lo, float hi) {
    uint32_t r; asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo)); return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r; asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c)); return r;
}
__device__ __forceinline__ void fma2(float &d0, float &d1, float a0, float a1, float b, float c) {
    uint64_t d, A, B, C;
    asm("mov.b64 %0, {%1, %2};" : "=l"(A) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %1};" : "=l"(B) : "f"(b));
    asm("mov.b64 %0, {%1, %1};" : "=l"(C) : "f"(c));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(A), "l"(B), "l"(C));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(d));
}
__device__ __forceinline__ void add2(float &d0, float &d1, float a0, float a1) {
    uint64_t d, A, D;
    asm("mov.b64 %0, {%1, %2};" : "=l"(A) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(D) : "f"(d0), "f"(d1));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(D), "l"(A));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(d));
}
// 2^x for x <= 0 on the FMA pipe: x = n + f with n the nearest integer, a cubic for 2^f on [-0.5, 0.5] (relative
// error 7.5e-5, below the bf16 rounding of the probabilities), n added to the exponent field
__device__ __forceinline__ float exp2_poly(float x) {
    x = fmaxf(x, -125.f);
    const float magic = 12582912.f;
    const float xr = x + magic;
    const float f = x - (xr - magic);
    float p = fmaf(f, 0.05517113f, 0.24261114f);
    p = fmaf(p, f, 0.69326111f);
    p = fmaf(p, f, 0.99992807f);
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(xr) << 23));
}
// 4 x 4 transpose of 16-byte units across the 4 lanes of a quad (l = lane & 3): on entry u[0..3] are the units of
// this lane's own row; on return u[j] is unit l of the row held by quad lane j.  Every lane of the warp takes part.
__device__ __forceinline__ void quad_transpose(uint4 (&u)[4], int l) {
#pragma unroll
    for (int s = 2; s >= 1; s >>= 1) {
        const bool up = (l & s) != 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (i & s) continue;
            const uint4 send = up ? u[i] : u[i ^ s];
            uint4 recv;
            recv.x = __shfl_xor_sync(0xffffffffu, send.x, s); recv.y = __shfl_xor_sync(0xffffffffu, send.y, s);
            recv.z = __shfl_xor_sync(0xffffffffu, send.z, s); recv.w = __shfl_xor_sync(0xffffffffu, send.w, s);
            if (up) u[i] = recv; else u[i ^ s] = recv;
        }
    }
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int HD, bool kRuns>   // kRuns: items may be cut into runs (RunIter); else all items are whole (WholeIter)
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tcgen05_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV,
                    const AttnArgs a) {
    using S = AttnSmem<HD>;
    using Iter = typename std::conditional<kRuns, RunIter, WholeIter>::type;
    constexpr int kHalves = HD / 64;             // 64-wide column halves of the head dim
    constexpr int kHalfQ = 128 * 128;            // bytes of one 128-row x 64-col bf16 block
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    const uint32_t bar0 = smem_base + S::kBarOff;
    // barrier map (8 bytes each)
    const uint32_t q_full = bar0, q_free = bar0 + 8;
    auto k_full = [&](int s) { return bar0 + 16 + 8u * s; };
    auto k_free = [&](int s) { return bar0 + 16 + 8u * (kKvStages + s); };
    auto v_full = [&](int s) { return bar0 + 16 + 8u * (2 * kKvStages + s); };
    auto v_free = [&](int s) { return bar0 + 16 + 8u * (3 * kKvStages + s); };
    const uint32_t bar1 = bar0 + 16 + 8u * 4 * kKvStages;
    auto s_full = [&](int w) { return bar1 + 8u * w; };
    auto p_ready = [&](int w) { return bar1 + 16 + 8u * w; };
    auto pv_done = [&](int w) { return bar1 + 32 + 8u * w; };
    auto s_free = [&](int w) { return bar1 + 48 + 8u * w; };
    auto drain_bar = [&](int w) { return bar1 + 64 + 8u * w; };
    auto q_ready = [&](int w) { return bar1 + 80 + 8u * w; };
    // shared items (see below): both groups have their part of the result in tensor memory / have read the other's
    const uint32_t merge_bar = bar1 + 96, merge_done = bar1 + 104;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_al + S::kBarOff + 16 + 8 * 4 * kKvStages + 112);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_al + S::kBarOff + 16 + 8 * 4 * kKvStages + 120);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        tc::mbar_init(q_full, 1); tc::mbar_init(q_free, 2);   // *_free: one commit per group's MMA issuer
        for (int s = 0; s < kKvStages; ++s) {
            tc::mbar_init(k_full(s), 1); tc::mbar_init(k_free(s), 2);
            tc::mbar_init(v_full(s), 1); tc::mbar_init(v_free(s), 2);
        }
        for (int w = 0; w < 2; ++w) { tc::mbar_init(s_full(w), 1); tc::mbar_init(p_ready(w), 4); tc::mbar_init(pv_done(w), 1);
                                      tc::mbar_init(s_free(w), 4); tc::mbar_init(q_ready(w), 4); }
        tc::mbar_init(drain_bar(0), 1); tc::mbar_init(drain_bar(1), 1);
        tc::mbar_init(merge_bar, 8); tc::mbar_init(merge_done, 8);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 9) tc::tmem_alloc(tc::smem_u32((const void *)tmem_slot), 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    tc::grid_dep_launch();
    tc::grid_dep_wait();   // work list, q/k/v rows and the cache rows of the new tokens come from earlier kernels
    // tensor-memory columns of group g (base g*256): S_g 0..63, P_g 64..95, the first 64 head-dim columns of Q_g as
    // bf16 pairs 96..127, O_g 128..255
    // A work item with more than 128 / G tokens gives each group its own 128 score rows, and each group takes both
    // 64-key halves of every key tile.  A SHARED item (at most 128 / G tokens: a short suffix) has score rows for
    // one group only; both groups then hold the same rows, group g takes half g of every key tile, and the two
    // partial results (both in tensor memory) are merged when the item's last P V has completed.
    const int tok_per_group = 128 / a.G;
    // K/V stage layout.  One TMA box ("unit") brings box_rows cache rows of one page, both 64-wide halves of the
    // head dim: [half][box_rows][128 bytes], 128-byte swizzle inside each half block.  A stage holds the 128 / box_rows
    // units of a key tile one after the other.  The tensor cores want the 8-row groups of an operand at ONE stride, so
    // the 64 keys of a half tile are chosen as 8 groups at a fixed stride:
    //   box_rows 16: group hh of every unit (keys u*16 + hh*8 + 0..7: a permutation of the tile's keys, applied
    //                alike to the scores, the mask and the V rows), stride = unit size;
    //   box_rows  8: units 8*hh .. 8*hh+7 (natural key order), stride = unit size;
    //   box_rows 64: unit hh, its 8 groups (natural key order), stride = 1024 bytes.
    const uint32_t hstride = (uint32_t)a.box_rows * 128u;            // between the two halves of the head dim in a unit
    const uint32_t unit_bytes = hstride * kHalves;
    const int units_per_tile = kKeysPerTile / a.box_rows;
    const bool perm = a.box_rows == 16;
    const uint32_t sbo = a.box_rows == 64 ? 1024u : unit_bytes;
    const uint32_t half_off = a.box_rows == 16 ? 1024u : (a.box_rows == 8 ? 8u * unit_bytes : unit_bytes);

    if (warp == 8 || warp == 11) {
        // ------------------------------ TMA producers (whole warps): warp 8 for Q and K, warp 11 for V ------------------------------
        // One box per unit of a tile, each issued by the lane that holds its page.  A warp's copies of one tile are
        // issued one after the other (about 70 cycles each), and a block-table entry is a dependent load from global
        // memory (1000 cycles and more): so K and V have a warp each, and the table is read 32 entries at a time,
        // one window ahead.
        const int plane = warp == 8 ? 0 : 1;
        uint32_t n_item = 0, kt = 0;
        bool ok = true;
        Iter run(a);
        RunPiece pc;
        for (; ok && run.next(a, pc); ++n_item) {
            const AttnWork &w = pc.w;
            if (plane == 0) {
                if (lane == 0) {
                    ok = tc::mbar_wait_relaxed(q_free, (n_item & 1) ^ 1, abort_flag);
                    if (ok) {
                        if (kHalves > 1) {
                            tc::mbar_arrive_expect_tx(q_full, 2 * S::kQBytes);
                            for (int g = 0; g < 2; ++g)
                                for (int h = 1; h < kHalves; ++h)
                                    tma_load_3d(smem_base + S::kQOff + g * S::kQBytes + (h - 1) * kHalfQ, &tmQ, q_full, h * 64,
                                                w.kv_head * a.G, w.q_start + (w.q_count <= tok_per_group ? 0 : g * tok_per_group));
                        } else {
                            tc::mbar_arrive(q_full);   // nothing of Q goes through shared memory at this head dim
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
            }
            // Window of the request's block-table row: lane l holds entry win0 + l (win0 a multiple of 32; 32 entries
            // cover a whole number of key tiles), the following window is in flight while this one is used.
            const int32_t *bt_row = a.block_tables + (size_t)w.req * a.max_blocks;
            auto load_window = [&](int w0) { return w0 + lane < a.max_blocks ? bt_row[w0 + lane] : -1; };
            int win0 = (pc.t0 * kKeysPerTile / a.page_size) & ~31;
            int win = load_window(win0), win_next = load_window(win0 + 32);
            for (int j = pc.t0; j < pc.t1 && ok; ++j, ++kt) {
                const int kbase = j * kKeysPerTile;
                if (kbase / a.page_size >= win0 + 32) {
                    win0 += 32;
                    win = win_next;
                    win_next = load_window(win0 + 32);
                }
                const int st = kt % kKvStages;
                const uint32_t par = ((kt / kKvStages) & 1) ^ 1;
                // this lane's unit of the tile, if the tile has that many
                const int n_units = min(units_per_tile, (w.kv_end - kbase + a.box_rows - 1) / a.box_rows);
                const int page = __shfl_sync(0xffffffffu, win, ((kbase + lane * a.box_rows) / a.page_size - win0) & 31);
                int row = -1;
                if (lane < n_units) {
                    const int key = kbase + lane * a.box_rows;
                    if (page < 0 || page >= a.num_pages) report(a.status, ALORA_ERR_PAGE_RANGE);
                    else row = ((page * 2 + plane) * a.Hkv + w.kv_head) * a.page_size + key % a.page_size;
                }
                const unsigned valid = __ballot_sync(0xffffffffu, row >= 0);
                const uint32_t bytes = (uint32_t)__popc(valid) * unit_bytes;
                const uint32_t fullb = plane == 0 ? k_full(st) : v_full(st);
                const uint32_t freeb = plane == 0 ? k_free(st) : v_free(st);
                if (lane == 0) {
                    ok = tc::mbar_wait_relaxed(freeb, par, abort_flag);
                    if (ok) tc::mbar_arrive_expect_tx(fullb, bytes);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (ok && row >= 0)   // one box: both halves of the head dim
                    tma_load_3d(smem_base + (plane == 0 ? S::kKOff : S::kVOff) + st * S::kKvBytes + lane * unit_bytes,
                                &tmKV, fullb, 0, row, 0);
            }
        }
        (void)ok;
    } else if (warp == 9 || warp == 10) {
        // ------------------------------ MMA issuers: warp 9 for group 0, warp 10 for group 1 ------------------------------
        // Keys are processed in half tiles of 64.  S_g of the next half is issued as soon as group g has copied the
        // current scores into registers (s_free), so it runs underneath that group's softmax; P_g V of the current
        // half follows when the group has written P_g (p_ready).  Each group has its own issuing warp, so neither
        // group's chain ever waits behind a barrier of the other.  The whole warp walks the schedule (uniform
        // control flow keeps the descriptors in uniform registers); one elected lane issues the tensor-core
        // instructions and their commits.
        const int g = warp - 9;
        const bool leader = tc::elect_one();
        constexpr uint32_t idesc_s = tc::idesc_bf16_f32(128, kHalfKeys);
        constexpr uint32_t idesc_pv = idesc_bf16_f32_bmn(128, HD);
        uint32_t n_item = 0, kt = 0, nh = 0;   // nh: half tiles handled so far (phase counter of the group's barriers)
        bool ok = true;
        const uint32_t qa = smem_base + S::kQOff + g * S::kQBytes;
        const uint32_t s_tmem = tmem_base + g * 256, p_tmem = s_tmem + 64, q_tmem = s_tmem + 96, o_tmem = s_tmem + 128;
        // S_g = Q_g K^T for the 64 keys of half `hh` of the K tile in stage st
        auto issue_s = [&](int st, int hh) {
            const uint32_t ka = smem_base + S::kKOff + st * S::kKvBytes + hh * half_off;
            if (leader) {
                // head-dim columns 0..63: A = Q_g from tensor memory; the rest: A = Q_g from shared memory
                const uint64_t db0 = smem_desc_k_sw128_sbo(ka, sbo);
#pragma unroll
                for (int k = 0; k < 4; ++k) mma_bf16_ts(s_tmem, q_tmem + 8 * k, db0 + 2 * k, idesc_s, k != 0 ? 1u : 0u);
#pragma unroll
                for (int h = 1; h < kHalves; ++h) {
                    const uint64_t da = tc::smem_desc_k_sw128(qa + (h - 1) * kHalfQ), db = smem_desc_k_sw128_sbo(ka + h * hstride, sbo);
#pragma unroll
                    for (int k = 0; k < 4; ++k) tc::mma_bf16(s_tmem, da + 2 * k, db + 2 * k, idesc_s, 1u);
                }
                tc::mma_commit(s_full(g));
            }
        };
        auto wait_all = [&](uint32_t bar, uint32_t parity) {
            return __all_sync(0xffffffffu, tc::mbar_wait(bar, parity, abort_flag));
        };
        Iter run(a);
        RunPiece pc;
        for (; ok && run.next(a, pc); ++n_item) {
            const bool shared = pc.w.q_count <= tok_per_group;
            const int n_steps = (pc.t1 - pc.t0) << (shared ? 0 : 1);   // half tiles of this group in the piece
            if (!wait_all(q_full, n_item & 1)) { ok = false; break; }
            if (!wait_all(q_ready(g), n_item & 1)) { ok = false; break; }
            if (!wait_all(k_full(kt % kKvStages), (kt / kKvStages) & 1)) { ok = false; break; }
            tc::tc_fence_after();
            issue_s(kt % kKvStages, shared ? g : 0);
            // this group is done with a K tile once its last half of it has been issued, and with Q at the end
            if (leader && shared) tc::mma_commit(k_free(kt % kKvStages));
            if (leader && n_steps == 1) tc::mma_commit(q_free);
            for (int i = 0; i < n_steps && ok; ++i) {
                const int st = kt % kKvStages;          // stage of step i
                const int hh = shared ? g : (i & 1);    // its half of the tile
                const bool tile_end = shared || hh == 1;
                // ---- scores of step i + 1
                if (i + 1 < n_steps) {
                    const int st1 = tile_end ? (kt + 1) % kKvStages : st;
                    if (tile_end && !wait_all(k_full(st1), ((kt + 1) / kKvStages) & 1)) { ok = false; break; }
                    if (!wait_all(s_free(g), nh & 1)) { ok = false; break; }
                    tc::tc_fence_after();
                    const int hh1 = shared ? g : (hh ^ 1);
                    issue_s(st1, hh1);
                    if (leader && (shared || hh1 == 1)) tc::mma_commit(k_free(st1));
                    if (leader && i + 2 == n_steps) tc::mma_commit(q_free);
                }
                // ---- P V of step i
                if ((shared || hh == 0) && !wait_all(v_full(st), (kt / kKvStages) & 1)) { ok = false; break; }
                if (!wait_all(p_ready(g), nh & 1)) { ok = false; break; }
                ++nh;
                tc::tc_fence_after();
                if (leader) {
                    const uint32_t va = smem_base + S::kVOff + st * S::kKvBytes + hh * half_off;
#pragma unroll
                    for (int k = 0; k < kHalfKeys / 16; ++k)  // 16 keys per step (two 8-key groups): 8 packed columns of P
                        mma_bf16_ts(o_tmem, p_tmem + 8 * k, smem_desc_mn_sw128(va + 2 * k * sbo, hstride, sbo), idesc_pv,
                                    (i | k) != 0 ? 1u : 0u);
                    tc::mma_commit(pv_done(g));
                    if (tile_end) tc::mma_commit(v_free(st));
                }
                if (tile_end) ++kt;
            }
        }
        // tensor-core work still in flight must finish before tensor memory is released
        if (leader) {
            tc::mma_commit(drain_bar(g));
            const long long t0 = clock64();
            while (!tc::mbar_try_wait(drain_bar(g), 0) && clock64() - t0 < tc::kWaitCycleLimit) {}
        }
    } else if (warp < 8) {
        // ------------------------------ softmax groups (warps 0..7) ------------------------------
        // (warps q and 4 + q own the same quarter of the tensor-memory lanes, so a thread can read the other
        // group's accumulator rows of its own row index: that is how the two parts of a shared item are merged)
        const int g = warp >> 2;                 // group 0 / 1
        const int q = warp & 3;                  // tensor-memory lane quarter
        const int row = q * 32 + lane;           // score row of this thread inside the group's tile
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        const uint32_t s_addr = tmem_base + g * 256 + lane_off;          // scores of the current half tile (64 columns)
        const uint32_t p_addr = s_addr + 64;                              // probabilities, bf16 pairs (32 columns)
        const uint32_t q_addr = s_addr + 96;                              // first 64 head-dim columns of this Q row
        const uint32_t o_addr = s_addr + 128;
        const uint32_t o_other = tmem_base + (g ^ 1) * 256 + lane_off + 128;   // the other group's O, same rows
        const uint32_t ml_addr = s_addr + 64, ml_other = tmem_base + (g ^ 1) * 256 + lane_off + 64;
        uint32_t n_s = 0, kt = 0;   // n_s: half tiles of this group so far (phase counter of its barriers)
        uint32_t n_merge = 0;       // shared items so far (phase counter of the merge barriers)
        bool ok = true;
        Iter run(a);
        RunPiece pc, pc_next;
        // first token of this group's rows inside an item (a shared item: both groups hold the same rows)
        auto tok_base = [&](const AttnWork &w) { return w.q_count <= tok_per_group ? 0 : g * tok_per_group; };
        // the first 64 head-dim columns of this thread's row of Q of a piece: global memory -> registers
        uint32_t qv[32];
        auto load_q = [&](const AttnWork &w) {
            const int tok_local = tok_base(w) + row / a.G;
            const bool valid = tok_local < w.q_count;
            const uint4 *src = reinterpret_cast<const uint4 *>(
                a.qkv + (size_t)(w.q_start + (valid ? tok_local : 0)) * a.N + (size_t)(w.kv_head * a.G + row % a.G) * HD);
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                const uint4 u = valid ? __ldg(src + x) : make_uint4(0, 0, 0, 0);
                qv[4 * x] = u.x; qv[4 * x + 1] = u.y; qv[4 * x + 2] = u.z; qv[4 * x + 3] = u.w;
            }
        };
        // registers -> tensor memory, where they are the A operand of the first half of Q K^T (all earlier Q K^T of
        // this group have completed by then: the group has consumed their scores)
        auto publish_q = [&]() {
            tmem_st_32x32(q_addr, qv);
            tmem_st_wait();
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(q_ready(g));
        };
        bool have = run.next(a, pc);
        if (have) { load_q(pc.w); publish_q(); }
        while (ok && have) {
            const AttnWork &w = pc.w;
            const bool shared = w.q_count <= tok_per_group;
            // step i of the group works on half (i & step_sh) | half0 of tile t0 + (i >> step_sh)
            const int step_sh = shared ? 0 : 1, half0 = shared ? g : 0;
            const int n_half = (pc.t1 - pc.t0) << step_sh;   // half tiles of this group in the piece
            const int tok_local = tok_base(w) + row / a.G;
            // position of this row's token; rows past the end of the block behave like its last token
            const int pos = w.kv_end - w.q_count + min(tok_local, w.q_count - 1);
            // exponent reference (a running maximum that is only moved when it has drifted by more than
            // 2^8, so the accumulator in tensor memory rarely needs rescaling) and row sum
            float m_ref = -INFINITY, l_run = 0.f;
            for (int i = 0; i < n_half && ok; ++i, ++n_s) {
                const int tbase = (pc.t0 + (i >> step_sh)) * kKeysPerTile;   // first key of the tile; column e of half hh
                const int hh = (i & step_sh) | half0;        // is key tbase + (perm ? (e/8)*16 + hh*8 + e%8 : hh*64 + e)
                const bool tile_begin = hh == half0;         // this group's first half of the tile
                if (!tc::mbar_wait(s_full(g), n_s & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                uint32_t sv[kHalfKeys];
#pragma unroll
                for (int c = 0; c < kHalfKeys; c += 32)
                    tc::tmem_ld_32x32(s_addr + c, reinterpret_cast<uint32_t(&)[32]>(sv[c]));
                tc::tmem_ld_wait();
                // the scores are in registers: the next half tile's Q K^T may overwrite them, underneath this softmax
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(s_free(g));
                const bool masked = tbase + kKeysPerTile - 1 > pos;   // tile crosses this row's causal limit
                bool bump = false;     // the exponent reference moved: O_g and the row sum are rescaled by alpha
                float alpha = 1.f;
                float l0 = 0.f, l1 = 0.f;
                uint32_t pk[kHalfKeys / 2];   // probabilities (bf16 pairs); their row sum in fp32
                auto row_max = [&]() {
                    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
                    for (int e = 0; e < kHalfKeys; e += 4) {
                        m0 = max3(m0, __uint_as_float(sv[e]), __uint_as_float(sv[e + 1]));
                        m1 = max3(m1, __uint_as_float(sv[e + 2]), __uint_as_float(sv[e + 3]));
                    }
                    return fmaxf(m0, m1);
                };
                auto move_reference = [&](float m_tile) {
                    alpha = fast_exp2((m_ref - m_tile) * a.scale_log2);
                    m_ref = m_tile;
                    l_run *= alpha;
                    bump = true;
                };
                if (masked) {
                    float m_tile = -INFINITY;
                    const int k0 = tbase + (perm ? hh * 8 : hh * kHalfKeys);
#pragma unroll
                    for (int e = 0; e < kHalfKeys; ++e) {
                        const int key = k0 + (perm ? (e >> 3) * 16 + (e & 7) : e);
                        if (key > pos) sv[e] = 0xff800000u;  // -inf
                        m_tile = fmaxf(m_tile, __uint_as_float(sv[e]));
                    }
                    if ((m_tile - m_ref) * a.scale_log2 > 8.f) move_reference(m_tile);
                    // (a piece that starts at an item's last tile can hold rows that see none of its keys so far)
                    const float mb = m_ref == -INFINITY ? 0.f : m_ref * a.scale_log2;
#pragma unroll
                    for (int e = 0; e < kHalfKeys; e += 2) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sv[e]), a.scale_log2, -mb));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sv[e + 1]), a.scale_log2, -mb));
                        l0 += p0;
                        l1 += p1;
                        pk[e >> 1] = pack_cvt(p0, p1);
                    }
                } else {
                    // No pass over the scores for their maximum: the exponentials are taken against the current
                    // reference, and only if their sum says that one of them may have left the safe range
                    // (> 2^14; also catches inf / NaN) is the true maximum taken and the half tile redone.  The
                    // first half tile of an item has no reference yet and takes its maximum first.
                    auto exponentials = [&]() {
                        const float mb = m_ref * a.scale_log2;
                        l0 = 0.f; l1 = 0.f;
#pragma unroll
                        for (int e = 0; e < kHalfKeys; e += 2) {
                            float x0, x1, p0, p1;
                            x0 = fmaf(__uint_as_float(sv[e]), a.scale_log2, -mb);
                            x1 = fmaf(__uint_as_float(sv[e + 1]), a.scale_log2, -mb);
                            if ((e & 7) == 6) { p0 = exp2_poly(x0); p1 = exp2_poly(x1); }   // a quarter of them on the FMA pipe
                            else { p0 = fast_exp2(x0); p1 = fast_exp2(x1); }
                            add2(l0, l1, p0, p1);
                            pk[e >> 1] = pack_cvt(p0, p1);
                        }
                    };
                    if (m_ref == -INFINITY) move_reference(row_max());
                    exponentials();
                    if (!(l0 + l1 <= 16384.f)) {
                        move_reference(row_max());
                        exponentials();
                    }
                }
                l_run += l0 + l1;
                // P_g and O_g are still in use by the previous half tile's P V until it has completed
                if (i > 0) {
                    if (!tc::mbar_wait(pv_done(g), (n_s - 1) & 1, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
                    if (__any_sync(0xffffffffu, bump)) {
                        // O_g holds the earlier products relative to the old reference: scale the rows that moved
#pragma unroll 1
                        for (int c = 0; c < HD; c += 32) {
                            uint32_t v[32];
                            tc::tmem_ld_32x32(o_addr + c, v);
                            tc::tmem_ld_wait();
#pragma unroll
                            for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
                            tmem_st_32x32(o_addr + c, v);
                        }
                    }
                }
                tmem_st_32x16(p_addr, reinterpret_cast<uint32_t(&)[16]>(pk[0]));
                tmem_st_32x16(p_addr + 16, reinterpret_cast<uint32_t(&)[16]>(pk[16]));
                // V rows of keys at or beyond the item's causal limit are cleared before the tile's first P V uses them
                // (thread `row` of each group clears key tbase + row)
                if (tile_begin) kt += (i > 0);   // tile index of this half
                if (tile_begin && tbase + kKeysPerTile > w.kv_end) {
                    const int st = kt % kKvStages;
                    if (!tc::mbar_wait(v_full(st), (kt / kKvStages) & 1, abort_flag)) { ok = false; break; }
                    if (tbase + row >= w.kv_end) {
                        uint8_t *vrow = smem_al + S::kVOff + st * S::kKvBytes + (row / a.box_rows) * unit_bytes +
                                        (row % a.box_rows) * 128;
                        for (int h = 0; h < kHalves; ++h)
#pragma unroll
                            for (int x = 0; x < 8; ++x)
                                reinterpret_cast<uint4 *>(vrow + h * hstride)[x] = make_uint4(0, 0, 0, 0);
                    }
                    tc::fence_proxy_async();
                }
                tmem_st_wait();
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(p_ready(g));  // P_g (and O_g, if it was rescaled) ready for P V
            }
            ++kt;  // the item's last tile
            if (!ok) break;
            // the next item's rows of Q go to tensor memory underneath this item's last P V, so that its first
            // Q K^T runs underneath this item's output
            const bool have_next = run.next(a, pc_next);
            if (have_next) { load_q(pc_next.w); publish_q(); }
            // the item's last P V, normalisation, store
            if (!tc::mbar_wait(pv_done(g), (n_s - 1) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            // Output rows: 4 adjacent lanes hold 4 adjacent rows.  Their 16-byte units are transposed inside the quad
            // so that one store instruction writes 64 contiguous bytes of one row per quad (4x fewer memory lines
            // per instruction than lane = row).
            const int ql = lane & 3;
            __nv_bfloat16 *dst_quad[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = (row & ~3) + j;
                const int tl = tok_base(w) + r / a.G;
                dst_quad[j] = tl < w.q_count
                                  ? a.out + (size_t)(w.q_start + tl) * a.Nq + (size_t)(w.kv_head * a.G + r % a.G) * HD + ql * 8
                                  : nullptr;
            }
            auto store_chunk = [&](int c, const float (&o)[32]) {   // 32 output columns from column c on
                uint4 u[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    u[x].x = tc::pack_bf16(o[8 * x], o[8 * x + 1]); u[x].y = tc::pack_bf16(o[8 * x + 2], o[8 * x + 3]);
                    u[x].z = tc::pack_bf16(o[8 * x + 4], o[8 * x + 5]); u[x].w = tc::pack_bf16(o[8 * x + 6], o[8 * x + 7]);
                }
                quad_transpose(u, ql);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (dst_quad[j]) *reinterpret_cast<uint4 *>(dst_quad[j] + c) = u[j];
            };
            if (shared) {
                // Both groups hold a partial result for the same rows (over different halves of the key tiles).  Each
                // thread puts its exponent reference and row sum next to its O_g in tensor memory, then both groups
                // read both parts; group g normalises and stores half g of the head-dim columns.
                tmem_st_32x2(ml_addr, __float_as_uint(m_ref), __float_as_uint(l_run));
                tmem_st_wait();
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(merge_bar);
                if (!tc::mbar_wait(merge_bar, n_merge & 1, abort_flag)) { ok = false; break; }
                ++n_merge;
                tc::tc_fence_after();
                uint32_t mo, lo;
                tmem_ld_32x2(ml_other, mo, lo);
                tc::tmem_ld_wait();
                const float m_oth = __uint_as_float(mo), l_oth = __uint_as_float(lo);
                const float m_all = fmaxf(m_ref, m_oth);   // (finite: the row's own position is in one of the halves)
                const float w_own = m_ref == -INFINITY ? 0.f : fast_exp2((m_ref - m_all) * a.scale_log2);
                const float w_oth = m_oth == -INFINITY ? 0.f : fast_exp2((m_oth - m_all) * a.scale_log2);
                const float l_all = fmaf(l_run, w_own, l_oth * w_oth);
                const bool whole = !kRuns || pc.n_parts == 1;
                const float inv = whole ? 1.f / l_all : 1.f;
                // part of a cut item: the merged, unnormalised rows go to the part's slot as rows of group 0
                float *po = a.part_o, *pml = a.part_ml;
                if (kRuns && !whole) {
                    po += (size_t)part_slot(pc.c_first, pc.part) * HD * 256 + row;
                    pml += (size_t)part_slot(pc.c_first, pc.part) * 512 + row;
                }
#pragma unroll 1
                for (int c = g * (HD / 2); c < (g + 1) * (HD / 2); c += 32) {
                    uint32_t v[32], u[32];
                    tc::tmem_ld_32x32(o_addr + c, v);
                    tc::tmem_ld_32x32(o_other + c, u);
                    tc::tmem_ld_wait();
                    float o[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        o[e] = fmaf(__uint_as_float(v[e]), w_own, __uint_as_float(u[e]) * w_oth) * inv;
                    if (whole) {
                        store_chunk(c, o);
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) po[(size_t)(c + e) * 256] = o[e];
                    }
                }
                if (kRuns && !whole && g == 0) {
                    pml[0] = m_all;
                    pml[256] = l_all;
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(merge_done);
                // the reference and sum sit in two columns of P_g and O_g is overwritten by the next item's first
                // P V: the other group must have read both before this group goes on
                if (!tc::mbar_wait(merge_done, (n_merge - 1) & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
            } else if (!kRuns || pc.n_parts == 1) {
                const float inv = 1.f / l_run;
#pragma unroll 1
                for (int c = 0; c < HD; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(o_addr + c, v);
                    tc::tmem_ld_wait();
                    float o[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __uint_as_float(v[e]) * inv;
                    store_chunk(c, o);
                }
                tc::tc_fence_before();
            } else {
                // part of a cut item: unnormalised rows, exponent references and sums go to the part's slot
                const int grow = g * 128 + row;
                float *po = a.part_o + (size_t)part_slot(pc.c_first, pc.part) * HD * 256 + grow;
                float *pml = a.part_ml + (size_t)part_slot(pc.c_first, pc.part) * 512 + grow;
#pragma unroll 1
                for (int c = 0; c < HD; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(o_addr + c, v);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) po[(size_t)(c + e) * 256] = __uint_as_float(v[e]);
                }
                tc::tc_fence_before();
                pml[0] = m_ref;
                pml[256] = l_run;
            }
            pc = pc_next;
            have = have_next;
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(a.status, ALORA_ERR_TIMEOUT);
    if (warp == 9) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, 512);
    }
}


// Merge of the parts of the cut items.  Blocks (2 * (c - 1) + g, j), c = 1 .. runs - 1, j = 0 .. 3: if run boundary c
// falls strictly inside an item and is the first boundary inside it, the four blocks j merge the rows of group g of
// that item: O = sum_p 2^((m_p - m) scale) O_p / sum_p 2^((m_p - m) scale) l_p, m = max_p m_p, parts in order.
// Thread = (row, sixteenth of the head dim): block j holds quarter j of the columns.
template <int HD>
__global__ void __launch_bounds__(512) attn_merge_kernel(const AttnArgs a) {
    tc::grid_dep_launch();
    tc::grid_dep_wait();
    const int total = a.run_counts[0], len = a.run_counts[1], off = a.run_counts[3];
    const int c = (int)blockIdx.x / 2 + 1, g = (int)blockIdx.x & 1;
    if ((long long)c * len >= total) return;
    const int item = a.cta_start[c];
    const AttnWork w = a.items[item];
    const int first = w.split - off, n_tiles = (w.kv_end + kKeysPerTile - 1) / kKeysPerTile;
    const int c_first = first / len;
    const int n_parts = (first + n_tiles - 1) / len - c_first + 1;
    if (first == c * len || c != c_first + 1) return;   // boundary not inside the item / not its first boundary
    if (g == 1 && w.q_count <= 128 / a.G) return;       // no rows of the item in this group
    const int row = threadIdx.x & 127, grow = g * 128 + row;
    constexpr int kCols = HD / 16;
    const int col0 = ((int)blockIdx.y * 4 + (int)(threadIdx.x >> 7)) * kCols;
    const int tl = g * (128 / a.G) + row / a.G;
    if (tl >= w.q_count) return;
    const float *__restrict__ ml = a.part_ml + grow;
    const float *__restrict__ po = a.part_o + (size_t)col0 * 256 + grow;
    float m_all = -INFINITY;
#pragma unroll 4
    for (int p = 0; p < n_parts; ++p) m_all = fmaxf(m_all, ml[(size_t)part_slot(c_first, p) * 512]);
    float l_all = 0.f, acc[kCols];
#pragma unroll
    for (int e = 0; e < kCols; ++e) acc[e] = 0.f;
#pragma unroll 4
    for (int p = 0; p < n_parts; ++p) {
        const int slot = part_slot(c_first, p);
        const float m_p = ml[(size_t)slot * 512];
        const float wgt = m_p == -INFINITY ? 0.f : exp2f((m_p - m_all) * a.scale_log2);
        l_all = fmaf(ml[(size_t)slot * 512 + 256], wgt, l_all);
        const float *src = po + (size_t)slot * HD * 256;
#pragma unroll
        for (int e = 0; e < kCols; ++e) acc[e] = fmaf(src[(size_t)e * 256], wgt, acc[e]);
    }
    const float inv = 1.f / l_all;
    __nv_bfloat16 *dst = a.out + (size_t)(w.q_start + tl) * a.Nq + (size_t)(w.kv_head * a.G + row % a.G) * HD + col0;
    uint32_t u[kCols / 2];
#pragma unroll
    for (int x = 0; x < kCols / 2; ++x) u[x] = tc::pack_bf16(acc[2 * x] * inv, acc[2 * x + 1] * inv);
    if constexpr (kCols == 8) *reinterpret_cast<uint4 *>(dst) = make_uint4(u[0], u[1], u[2], u[3]);
    else *reinterpret_cast<uint2 *>(dst) = make_uint2(u[0], u[1]);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn tensor_map_encoder();  // gemm_tcgen05.cu

// Prefill attention on the tensor cores.  Returns kernels launched, or -1 when the shape is unsupported
// (head dim other than 64/128, group size not dividing 128, page size not a power of two in 8..128).
int launch_attend_splitkv(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                          cudaStream_t s);  // attn_splitkv.cu

static int launch_attend_long(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                              cudaStream_t s);

int launch_attend_tc(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                     cudaStream_t s) {
    if (b.T == 0) return 0;
    // Requests with few new tokens (decode, short suffixes) are on the few-row work list, the others on the
    // tensor-core kernel's; the two kernels write disjoint output rows.  The few-row kernel goes second: when its
    // list is empty (a prefill batch) its blocks come and go in the shadow of the first kernel's tail.
    int n = 0;
    if (!(b.all_small && ctx->max_split_items > 0)) {
        n = launch_attend_long(ctx, qkv, b, pool, out, s);
        if (n < 0) return -1;
    }
    if (ctx->max_split_items > 0) {
        const int n_small = launch_attend_splitkv(ctx, qkv, b, pool, out, s);
        if (n_small < 0) return -1;
        n += n_small;
    }
    return n;
}

static int launch_attend_long(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                              cudaStream_t s) {
    const int n_small = 0;
    const Dims &d = ctx->d;
    const bool page_ok = d.page >= 8 && d.page <= 128 && (d.page & (d.page - 1)) == 0;
    if ((d.hd != 64 && d.hd != 128) || 128 % d.G != 0 || !page_ok) return -1;
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return -1;
    CUtensorMap tmQ, tmKV;
    {
        cuuint64_t dims[3] = {(cuuint64_t)d.hd, (cuuint64_t)d.Hq, (cuuint64_t)b.T};
        cuuint64_t strides[2] = {(cuuint64_t)d.hd * 2, (cuuint64_t)d.N * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)d.G, (cuuint32_t)(128 / d.G)};
        cuuint32_t es[3] = {1, 1, 1};
        if (enc(&tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(qkv), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -1;
    }
    const int box_rows = d.page == 8 ? 8 : (d.page <= 32 ? 16 : 64);
    {
        // the pool as (64 columns, cache rows, 64-wide halves of the head dim): one box = box_rows rows, both halves
        const cuuint64_t halves = (cuuint64_t)d.hd / 64;
        cuuint64_t dims[3] = {64, (cuuint64_t)b.num_pages * 2 * d.Hkv * d.page, halves};
        cuuint64_t strides[2] = {(cuuint64_t)d.hd * 2, 128};
        cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)halves};
        cuuint32_t es[3] = {1, 1, 1};
        if (enc(&tmKV, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(pool), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -1;
    }
    AttnArgs a{};
    a.items = ctx->d_attn_items; a.n_items = ctx->d_counts + 1; a.block_tables = b.block_tables;
    a.max_blocks = b.max_blocks; a.num_pages = b.num_pages; a.Hkv = d.Hkv; a.G = d.G; a.page_size = d.page; a.box_rows = box_rows;
    a.N = d.N; a.Nq = d.Nq; a.qkv = (const __nv_bfloat16 *)qkv; a.scale_log2 = d.softmax_scale * 1.4426950408889634f;
    a.out = (__nv_bfloat16 *)out; a.status = ctx->d_status;
    a.run_counts = ctx->d_counts + 6; a.cta_start = ctx->d_attn_cta_start;
    a.part_o = ctx->d_attn_part_o; a.part_ml = ctx->d_attn_part_ml;
    const int max_items = (b.T / ctx->attn_q_block + b.R) * d.Hkv;
    ProfScope prof(ctx, KK_ATTENTION, s);
    static bool attr_set[2][64] = {};
    const int dev = ctx->cfg.device, hi = d.hd == 128;
    // Items are cut into runs (and need the merge kernel) only when the batch has at least kAttnCutMinTiles key tiles
    // per block and kAttnCutMinWaves items per block; upper bounds from what the host knows decide whether that
    // can be the case.
    // A batch that cannot have more items than there are SMs is cut too if its items can be long enough to give
    // every block a run of kAttnMinRunTiles key tiles (a few requests with long contexts); the work-list builder, which
    // knows the lengths, has the last word in both cases.
    const int n_sm = ctx->sm_count;
    const long long max_tiles = (long long)max_items * (((long long)b.max_blocks * d.page + kKeysPerTile - 1) / kKeysPerTile);
    const bool long_batch = max_tiles >= (long long)kAttnCutMinTiles * n_sm && max_items >= kAttnCutMinWaves * n_sm;
    // (not for a batch that looks like few-row work only, a handful of new tokens per request: an unused merge
    // launch would only lengthen its step; should a long request hide in such a batch it is taken whole)
    const bool few_items = max_items < n_sm && max_tiles >= (long long)kAttnMinRunTiles * n_sm &&
                           (long long)b.T > (long long)b.R * ctx->small_max_tokens;
    const bool runs = n_sm > 1 && (long_batch || few_items);
    const int grid = runs ? n_sm : std::max(1, std::min(n_sm, max_items));
    if (dev >= 0 && dev < 64 && !attr_set[hi][dev]) {
        cudaError_t e = hi ? cudaFuncSetAttribute(attn_tcgen05_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<128>::kTotal)
                           : cudaFuncSetAttribute(attn_tcgen05_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<64>::kTotal);
        if (e == cudaSuccess)
            e = hi ? cudaFuncSetAttribute(attn_tcgen05_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<128>::kTotal)
                   : cudaFuncSetAttribute(attn_tcgen05_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<64>::kTotal);
        if (e != cudaSuccess) return -1;
        attr_set[hi][dev] = true;
    }
    const dim3 g3(grid), b3(kAttnThreads);
    cudaError_t le;
    if (runs) le = hi ? launch_kernel(attn_tcgen05_kernel<128, true>, g3, b3, AttnSmem<128>::kTotal, s, true, tmQ, tmKV, a)
                      : launch_kernel(attn_tcgen05_kernel<64, true>, g3, b3, AttnSmem<64>::kTotal, s, true, tmQ, tmKV, a);
    else le = hi ? launch_kernel(attn_tcgen05_kernel<128, false>, g3, b3, AttnSmem<128>::kTotal, s, true, tmQ, tmKV, a)
                 : launch_kernel(attn_tcgen05_kernel<64, false>, g3, b3, AttnSmem<64>::kTotal, s, true, tmQ, tmKV, a);
    if (le != cudaSuccess) return -1;
    if (!runs) return 1 + n_small;
    const cudaError_t me = hi ? launch_kernel(attn_merge_kernel<128>, dim3(2 * (grid - 1), 4), dim3(512), 0, s, true, a)
                              : launch_kernel(attn_merge_kernel<64>, dim3(2 * (grid - 1), 4), dim3(512), 0, s, true, a);
    if (me != cudaSuccess) return -1;
    return 2 + n_small;
}

}  // namespace alora
