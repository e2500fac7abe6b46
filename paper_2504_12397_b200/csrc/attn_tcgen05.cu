// Paged causal GQA attention of suffix queries on the 5th-generation tensor cores (Eq. 1 / Eq. 3).
//
// One persistent block per SM works through (request, KV head, query block) items.  A query block
// is 2 x 128 score rows: rows are (token, query head of the KV group) pairs, so the G query heads
// that share a KV head share every K/V tile brought on chip.  Roles:
//   warp 8   TMA producer: the two 128 x hd query tiles of the item (3-D boxes d x head x token out
//            of the fused q/k/v rows) and, per 128-key tile, the K and V rows of up to 128/page
//            pages fetched through the block table (one 2-D box per page and 64-wide half of hd),
//            two-deep rings for K and for V;
//   warp 9   MMA issuer: S_w = Q_w K^T (fp32, tensor memory) for w = 0, 1, then PV_w = P_w V with P_w
//            read from tensor memory (it overwrites S_w in bf16) and V consumed in place (MN-major);
//   warps 0-3, 4-7   softmax groups w = 0, 1, one thread per score row: running maximum and sum
//            (online softmax; a thread owns its whole row, so the row reductions need no
//            cross-lane traffic), P_w written back to tensor memory; the output O_w accumulates in
//            tensor memory across tiles and is rescaled only when a row's maximum has moved by more
//            than 2^8 since the exponent reference was last set; final normalisation and store.
// While one group does its exponentials the tensor pipe works for the other group.
//
// Masking: key j is visible to a row at position p iff j <= p; masked probabilities are set to
// zero explicitly, and V rows of keys at or beyond the item's causal limit are cleared in shared
// memory before use, so stale cache bytes (whatever their bit pattern) cannot reach an output.
// All waits are bounded; on expiry ALORA_ERR_TIMEOUT is recorded and the block leaves normally.
#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

constexpr int kAttnThreads = 320;
constexpr int kKeysPerTile = 128;
constexpr int kKvStages = 2;

struct AttnArgs {
    const AttnWork *items;
    const int32_t *n_items;
    const int32_t *block_tables;
    int max_blocks, num_pages;
    int Hkv, G, page_size;     // G * tokens_per_group == 128
    int N, Nq;                 // fused row width, query part width
    float scale_log2;          // softmax scale * log2(e)
    __nv_bfloat16 *out;        // [T][Nq]
    int32_t *status;
};

template <int HD>
struct AttnSmem {
    static constexpr int kQBytes = 128 * HD * 2;             // one query tile (two 64-wide halves when HD = 128)
    static constexpr int kKvBytes = kKeysPerTile * HD * 2;   // one K or V tile
    static constexpr int kQOff = 0;
    static constexpr int kKOff = 2 * kQBytes;
    static constexpr int kVOff = kKOff + kKvStages * kKvBytes;
    static constexpr int kBarOff = kVOff + kKvStages * kKvBytes;
    static constexpr int kTotal = kBarOff + 256 + 1024;
};

// V tile as the B operand of P V: N = head dim (contiguous in memory: "MN-major"), K = keys.
// Rows (keys) are 128 bytes apart, 8-key groups 1024 bytes apart (stride byte offset); the two
// 64-wide halves of the head dim are `half_bytes` apart (leading byte offset); 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t smem_addr, uint32_t half_bytes) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFF) | ((uint64_t)((half_bytes >> 4) & 0x3FFF) << 16) | (64ull << 32) |
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
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                            int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tcgen05_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV,
                    const AttnArgs a) {
    using S = AttnSmem<HD>;
    constexpr int kHalves = HD / 64;             // 64-wide column halves of the head dim
    constexpr int kHalfQ = 128 * 128;            // bytes of one 128-row x 64-col bf16 block
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    const uint32_t bar0 = smem_base + S::kBarOff;
    // barrier map (8 bytes each)
    const uint32_t q_full = bar0, q_free = bar0 + 8;
    auto k_full = [&](int s) { return bar0 + 16 + 8u * s; };
    auto k_free = [&](int s) { return bar0 + 32 + 8u * s; };
    auto v_full = [&](int s) { return bar0 + 48 + 8u * s; };
    auto v_free = [&](int s) { return bar0 + 64 + 8u * s; };
    auto s_full = [&](int w) { return bar0 + 80 + 8u * w; };
    auto p_ready = [&](int w) { return bar0 + 96 + 8u * w; };
    auto pv_done = [&](int w) { return bar0 + 112 + 8u * w; };
    const uint32_t drain_bar = bar0 + 128;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem_al + S::kBarOff + 136);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_al + S::kBarOff + 144);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        tc::mbar_init(q_full, 1); tc::mbar_init(q_free, 1);
        for (int s = 0; s < kKvStages; ++s) {
            tc::mbar_init(k_full(s), 1); tc::mbar_init(k_free(s), 1);
            tc::mbar_init(v_full(s), 1); tc::mbar_init(v_free(s), 1);
        }
        for (int w = 0; w < 2; ++w) { tc::mbar_init(s_full(w), 1); tc::mbar_init(p_ready(w), 4); tc::mbar_init(pv_done(w), 1); }
        tc::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 9) tc::tmem_alloc(tc::smem_u32((const void *)tmem_slot), 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // tensor-memory columns: S_w / P_w at w*128, O_w at 256 + w*128
    const int n_items = *a.n_items;
    const int tok_per_group = 128 / a.G;
    const int pages_per_tile = kKeysPerTile / a.page_size;
    const uint32_t page_bytes = (uint32_t)a.page_size * 128u;  // one page's rows inside a 64-wide half

    if (warp == 8) {
        // ------------------------------ TMA producer (whole warp) ------------------------------
        uint32_t n_item = 0, kt = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++n_item) {
            const AttnWork w = a.items[it];
            if (lane == 0) {
                ok = tc::mbar_wait(q_free, (n_item & 1) ^ 1, abort_flag);
                if (ok) {
                    tc::mbar_arrive_expect_tx(q_full, 2 * S::kQBytes);
                    for (int g = 0; g < 2; ++g)
                        for (int h = 0; h < kHalves; ++h)
                            tma_load_3d(smem_base + S::kQOff + g * S::kQBytes + h * kHalfQ, &tmQ, q_full, h * 64,
                                        w.kv_head * a.G, w.q_start + g * tok_per_group);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            const int n_tiles = (w.kv_end + kKeysPerTile - 1) / kKeysPerTile;
            for (int j = 0; j < n_tiles && ok; ++j, ++kt) {
                const int st = kt % kKvStages;
                const uint32_t par = ((kt / kKvStages) & 1) ^ 1;
                const int kbase = j * kKeysPerTile;
                const int n_pages = min(pages_per_tile, (w.kv_end - kbase + a.page_size - 1) / a.page_size);
                // every lane looks up one page of the tile
                int page = -1;
                if (lane < n_pages) {
                    page = a.block_tables[(size_t)w.req * a.max_blocks + kbase / a.page_size + lane];
                    if (page < 0 || page >= a.num_pages) { report(a.status, ALORA_ERR_PAGE_RANGE); page = -1; }
                }
                const unsigned valid = __ballot_sync(0xffffffffu, page >= 0);
                const uint32_t bytes = (uint32_t)__popc(valid) * page_bytes * kHalves;
                for (int plane = 0; plane < 2 && ok; ++plane) {
                    const uint32_t fullb = plane == 0 ? k_full(st) : v_full(st);
                    const uint32_t freeb = plane == 0 ? k_free(st) : v_free(st);
                    if (lane == 0) {
                        ok = tc::mbar_wait(freeb, par, abort_flag);
                        if (ok) tc::mbar_arrive_expect_tx(fullb, bytes);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (ok && page >= 0) {
                        const uint32_t dst = smem_base + (plane == 0 ? S::kKOff : S::kVOff) + st * S::kKvBytes +
                                             lane * page_bytes;
                        const int row = ((page * 2 + plane) * a.Hkv + w.kv_head) * a.page_size;
                        for (int h = 0; h < kHalves; ++h)
                            tc::tma_load_2d(dst + h * kHalfQ, &tmKV, fullb, h * 64, row);
                    }
                }
            }
        }
        (void)ok;
    } else if (warp == 9) {
        if (lane == 0) {
            // ------------------------------ MMA issuer ------------------------------
            constexpr uint32_t idesc_s = tc::idesc_bf16_f32(128, kKeysPerTile);
            constexpr uint32_t idesc_pv = idesc_bf16_f32_bmn(128, HD);
            uint32_t n_item = 0, kt = 0, np[2] = {0, 0};
            bool ok = true;
            auto issue_s = [&](int w, int st) {
                const uint32_t qa = smem_base + S::kQOff + w * S::kQBytes;
                const uint32_t ka = smem_base + S::kKOff + st * S::kKvBytes;
                for (int h = 0; h < kHalves; ++h) {
                    const uint64_t da = tc::smem_desc_k_sw128(qa + h * kHalfQ), db = tc::smem_desc_k_sw128(ka + h * kHalfQ);
                    for (int k = 0; k < 4; ++k)
                        tc::mma_bf16(tmem_base + w * 128, da + 2 * k, db + 2 * k, idesc_s, (h | k) != 0 ? 1u : 0u);
                }
                tc::mma_commit(s_full(w));
            };
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++n_item) {
                const AttnWork w = a.items[it];
                const int n_tiles = (w.kv_end + kKeysPerTile - 1) / kKeysPerTile;
                if (!tc::mbar_wait(q_full, n_item & 1, abort_flag)) { ok = false; break; }
                if (!tc::mbar_wait(k_full(kt % kKvStages), (kt / kKvStages) & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                issue_s(0, kt % kKvStages);
                issue_s(1, kt % kKvStages);
                tc::mma_commit(k_free(kt % kKvStages));
                if (n_tiles == 1) tc::mma_commit(q_free);
                for (int j = 0; j < n_tiles && ok; ++j, ++kt) {
                    const int st = kt % kKvStages;
                    const bool more = j + 1 < n_tiles;
                    for (int g = 0; g < 2; ++g) {
                        if (!tc::mbar_wait(p_ready(g), np[g] & 1, abort_flag)) { ok = false; break; }
                        ++np[g];
                        if (g == 0 && !tc::mbar_wait(v_full(st), (kt / kKvStages) & 1, abort_flag)) { ok = false; break; }
                        tc::tc_fence_after();
                        const uint32_t va = smem_base + S::kVOff + st * S::kKvBytes;
                        for (int k = 0; k < kKeysPerTile / 16; ++k)  // 16 keys per step: 8 packed columns of P
                            mma_bf16_ts(tmem_base + 256 + g * 128, tmem_base + g * 128 + 8 * k,
                                        smem_desc_mn_sw128(va + k * 2048, kHalfQ), idesc_pv, (j | k) != 0 ? 1u : 0u);
                        tc::mma_commit(pv_done(g));
                        if (g == 1) tc::mma_commit(v_free(st));
                        if (more) {
                            const int st1 = (kt + 1) % kKvStages;
                            if (g == 0 && !tc::mbar_wait(k_full(st1), ((kt + 1) / kKvStages) & 1, abort_flag)) { ok = false; break; }
                            tc::tc_fence_after();
                            issue_s(g, st1);
                            if (g == 1) {
                                tc::mma_commit(k_free(st1));
                                if (j + 2 == n_tiles) tc::mma_commit(q_free);  // last S products of the item issued
                            }
                        }
                    }
                }
            }
            // tensor-core work still in flight must finish before tensor memory is released
            tc::mma_commit(drain_bar);
            const long long t0 = clock64();
            while (!tc::mbar_try_wait(drain_bar, 0) && clock64() - t0 < tc::kWaitCycleLimit) {}
        }
    } else {
        // ------------------------------ softmax groups (warps 0..7) ------------------------------
        const int g = warp >> 2;                 // group 0 / 1
        const int q = warp & 3;                  // tensor-memory lane quarter
        const int row = q * 32 + lane;           // score row of this thread inside the group's tile
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        const uint32_t s_addr = tmem_base + g * 128 + lane_off;
        const uint32_t o_addr = tmem_base + 256 + g * 128 + lane_off;
        uint32_t n_s = 0, kt = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const AttnWork w = a.items[it];
            const int n_tiles = (w.kv_end + kKeysPerTile - 1) / kKeysPerTile;
            const int tok_local = g * tok_per_group + row / a.G;
            const bool row_valid = tok_local < w.q_count;
            // position of this row's token; rows past the end of the block behave like its last token
            const int pos = w.kv_end - w.q_count + min(tok_local, w.q_count - 1);
            // exponent reference (a running maximum that is only moved when it has drifted by more than
            // 2^8, so the accumulator in tensor memory rarely needs rescaling) and row sum
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_tiles && ok; ++j, ++kt) {
                const int kbase = j * kKeysPerTile;
                if (!tc::mbar_wait(s_full(g), n_s & 1, abort_flag)) { ok = false; break; }
                ++n_s;
                tc::tc_fence_after();
                uint32_t sv[kKeysPerTile];
#pragma unroll
                for (int c = 0; c < kKeysPerTile; c += 32)
                    tc::tmem_ld_32x32(s_addr + c, reinterpret_cast<uint32_t(&)[32]>(sv[c]));
                tc::tmem_ld_wait();
                float m_tile = -INFINITY;
                if (kbase + kKeysPerTile - 1 > pos) {  // tile crosses this row's causal limit: mask
#pragma unroll
                    for (int e = 0; e < kKeysPerTile; ++e) {
                        if (kbase + e > pos) sv[e] = 0xff800000u;  // -inf
                        m_tile = fmaxf(m_tile, __uint_as_float(sv[e]));
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < kKeysPerTile; ++e) m_tile = fmaxf(m_tile, __uint_as_float(sv[e]));
                }
                const bool bump = (m_tile - m_ref) * a.scale_log2 > 8.f;  // always true on an item's first tile
                float alpha = 1.f;
                if (bump) {
                    alpha = fast_exp2((m_ref - m_tile) * a.scale_log2);
                    m_ref = m_tile;
                    l_run *= alpha;
                }
                if (j > 0 && __any_sync(0xffffffffu, bump)) {
                    // O_w holds the earlier tiles' products relative to the old reference: once the last P V
                    // has completed, scale the rows of this warp whose reference moved
                    if (!tc::mbar_wait(pv_done(g), n_s & 1, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
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
                // probabilities (bf16) over the score columns, row sum in fp32
                const float mb = m_ref * a.scale_log2;
                float l0 = 0.f, l1 = 0.f;
#pragma unroll
                for (int c = 0; c < kKeysPerTile; c += 32) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sv[c + e]), a.scale_log2, -mb));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sv[c + e + 1]), a.scale_log2, -mb));
                        l0 += p0;
                        l1 += p1;
                        pk[e >> 1] = tc::pack_bf16(p0, p1);
                    }
                    tmem_st_32x16(s_addr + (c >> 1), pk);
                }
                l_run += l0 + l1;
                // V rows of keys at or beyond the item's causal limit are cleared before P V uses them
                if (kbase + kKeysPerTile > w.kv_end) {
                    const int st = kt % kKvStages;
                    if (!tc::mbar_wait(v_full(st), (kt / kKvStages) & 1, abort_flag)) { ok = false; break; }
                    if (kbase + row >= w.kv_end) {
                        uint8_t *vrow = smem_al + S::kVOff + st * S::kKvBytes + row * 128;
                        for (int h = 0; h < kHalves; ++h)
#pragma unroll
                            for (int x = 0; x < 8; ++x)
                                reinterpret_cast<uint4 *>(vrow + h * kHalfQ)[x] = make_uint4(0, 0, 0, 0);
                    }
                    tc::fence_proxy_async();
                }
                tmem_st_wait();
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(p_ready(g));  // P_w (and O_w, if it was rescaled) ready for P V
            }
            if (!ok) break;
            // the item's last P V, normalisation, store
            if (!tc::mbar_wait(pv_done(g), (n_s - 1) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            float o[HD];
            {
                const float inv = 1.f / l_run;
#pragma unroll
                for (int c = 0; c < HD; c += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(o_addr + c, v);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[c + e] = __uint_as_float(v[e]) * inv;
                }
            }
            tc::tc_fence_before();
            if (row_valid) {
                const int token = w.q_start + tok_local;
                const int head = w.kv_head * a.G + row % a.G;
                uint4 *dst = reinterpret_cast<uint4 *>(a.out + (size_t)token * a.Nq + (size_t)head * HD);
#pragma unroll
                for (int x = 0; x < HD / 8; ++x) {
                    uint4 u;
                    u.x = tc::pack_bf16(o[8 * x], o[8 * x + 1]); u.y = tc::pack_bf16(o[8 * x + 2], o[8 * x + 3]);
                    u.z = tc::pack_bf16(o[8 * x + 4], o[8 * x + 5]); u.w = tc::pack_bf16(o[8 * x + 6], o[8 * x + 7]);
                    dst[x] = u;
                }
            }
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


typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn tensor_map_encoder();  // gemm_tcgen05.cu

// Prefill attention on the tensor cores.  Returns kernels launched, or -1 when the shape is unsupported
// (head dim other than 64/128, group size not dividing 128, page size not a power of two in 8..128).
int launch_attend_splitkv(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                          cudaStream_t s);  // attn_splitkv.cu

int launch_attend_tc(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                     cudaStream_t s) {
    if (b.T == 0) return 0;
    // requests with few new tokens (decode, short suffixes) are on the few-row work list
    int n_small = 0;
    if (ctx->max_split_items > 0) {
        n_small = launch_attend_splitkv(ctx, qkv, b, pool, out, s);
        if (n_small < 0) return -1;
        if (b.all_small) return n_small;
    }
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
    {
        cuuint64_t dims[2] = {(cuuint64_t)d.hd, (cuuint64_t)b.num_pages * 2 * d.Hkv * d.page};
        cuuint64_t strides[1] = {(cuuint64_t)d.hd * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)d.page};
        cuuint32_t es[2] = {1, 1};
        if (enc(&tmKV, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -1;
    }
    AttnArgs a{};
    a.items = ctx->d_attn_items; a.n_items = ctx->d_counts + 1; a.block_tables = b.block_tables;
    a.max_blocks = b.max_blocks; a.num_pages = b.num_pages; a.Hkv = d.Hkv; a.G = d.G; a.page_size = d.page;
    a.N = d.N; a.Nq = d.Nq; a.scale_log2 = d.softmax_scale * 1.4426950408889634f;
    a.out = (__nv_bfloat16 *)out; a.status = ctx->d_status;
    const int max_items = (b.T / ctx->attn_q_block + b.R) * d.Hkv;
    const int grid = std::max(1, std::min(ctx->sm_count, max_items));
    ProfScope prof(ctx, KK_ATTENTION, s);
    static bool attr_set[2][64] = {};
    const int dev = ctx->cfg.device, hi = d.hd == 128;
    if (dev >= 0 && dev < 64 && !attr_set[hi][dev]) {
        cudaError_t e = hi ? cudaFuncSetAttribute(attn_tcgen05_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  AttnSmem<128>::kTotal)
                           : cudaFuncSetAttribute(attn_tcgen05_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  AttnSmem<64>::kTotal);
        if (e != cudaSuccess) return -1;
        attr_set[hi][dev] = true;
    }
    if (hi) attn_tcgen05_kernel<128><<<grid, kAttnThreads, AttnSmem<128>::kTotal, s>>>(tmQ, tmKV, a);
    else attn_tcgen05_kernel<64><<<grid, kAttnThreads, AttnSmem<64>::kTotal, s>>>(tmQ, tmKV, a);
    return 1 + n_small;
}

}  // namespace alora
