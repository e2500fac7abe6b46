// The order in which the blocks of a projection launch take their work items.  The item list of a launch is
// [shrink items 0 .. n_shrink-1 | projection items]; a projection item of an adapter row tile waits for that tile's
// shrink item.  Two rules keep a running block from ever waiting for a block that has not been scheduled:
//   1. shrink items are CLAIMED, one at a time, from a counter (never dealt by block index): whoever holds one is
//      running.  Blocks whose index is below n_shrink claim at once (their list has a free place at its head); the
//      others look on for a short while and join the claiming only if shrink items are still unclaimed then;
//   2. a block starts on its projection items only after the counter has passed n_shrink, i.e. after every shrink
//      item has been claimed by a running block.  Projection items are dealt by block index as if the shrink items
//      occupied list positions 0 .. n_shrink-1, so that in the usual case every block keeps the items it always had.
// The two decisions below are shared by the kernels (gemm_tcgen05.cu, gemm_pair_tcgen05.cu) and by the host-side
// model that the tests run against small grids with few resident blocks (alora_selftest_claim_order).
#pragma once

#if defined(__CUDACC__)
#define ALORA_HD __host__ __device__ __forceinline__
#else
#define ALORA_HD inline
#endif

namespace alora {

// Whether block `block` claims shrink items as soon as it starts (rule 1).
ALORA_HD bool claims_at_once(int block, int n_shrink) { return block < n_shrink; }

// The next item dealt to a block by index, or -1 when its list is exhausted.  `stat` is the block's cursor, initially
// its block index; positions below n_shrink belong to the claimed shrink items and are skipped (rule 2).
ALORA_HD int next_dealt_item(int &stat, int n_shrink, int total, int grid) {
    while (stat < n_shrink) stat += grid;
    if (stat >= total) return -1;
    const int item = stat;
    stat += grid;
    return item;
}

}  // namespace alora
