// Synchronisation across GPUs when the job is sharded BY WORKER (the layout of the paper: the
// workers of Algorithm 3 live on different devices and every H steps exchange x and B^2).
//
// Each rank holds W_local replicas.  The synchronisation is split into three kernels around an
// exchange buffer S = [2][stride] per rank (sums of x, sums of B^2):
//   export   S <- adjacent-pair tree sum over the LOCAL replicas                 (local HBM only)
//   combine  for this rank's coordinate slice: total <- adjacent-pair tree over the ranks' S in
//            rank order, read with plain peer loads; the total is stored back into EVERY rank's
//            S (a reduce-scatter and an all-gather in one kernel, over NVLink peer memory)
//   import   x, B^2 of every local replica <- total / W_total; stale accumulator <- mean B^2
// With W_local a power of two, "local tree, then tree over ranks" is exactly the adjacent-pair
// tree over all W_total workers, so the result is bit-identical to the single-GPU kernels.
// The exchange moves 2N floats per rank whatever W_local is (Section 4.2: x and B^2).
// No kernel waits for another rank: the host orders the phases (stream sync + barrier).
//
// Export and import are instantiations of the sweep kernel (la_sweep with XCH = 1 / 2), alone or
// fused with the local step next to the synchronisation:
//   step + export   the local step that makes t' reach H.  Its results y_i, A_i^2 are about to be
//                   replaced by the means, so they are never stored: only their tree sums go to
//                   the exchange buffer (read 16 B, write ~0 B per worker*param).
//   import + step   the first step of the next period.  It starts from total / W_total read from
//                   the exchange buffer instead of from the replicas (read ~0 B, write 16 B).
// Together the synchronisation costs no HBM pass of its own; what crosses NVLink stays 2N floats.
// Only the combine kernel lives here.
#pragma once
#include "la_sweep.cuh"

namespace la {

constexpr int kMaxRanks = 16;

struct CombineParams {
  float* S[kMaxRanks];          // exchange buffers of all ranks; S[r] = sums of x, S[r] + stride = sums of B^2
  uint64_t stride;
  uint64_t slice_lo, slice_hi;  // this rank's coordinate slice (multiples of 64)
  uint32_t world;
};

template <int V>
__global__ void __launch_bounds__(LA_BLOCK) la_combine_sums(const CombineParams p) {
#ifdef LA_DEBUG
  dbg_begin(DebugRanges{});  // the ranks' buffers are not range-checked
#endif
  const uint64_t ngroups = (p.slice_hi - p.slice_lo) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += nthreads) {
    const uint64_t off = p.slice_lo + grp * V;
    PairTreeDyn<V> tree;
    for (uint32_t r = 0; r < p.world; ++r) {
      // Ordinary loads; for every rank but this one they cross NVLink.  The streaming
      // (evict-first) flavour fits: each line is fetched once and never read again here.
      const Vec<V> sx = ld_stream<V>(p.S[r] + off);
      const Vec<V> sb = ld_stream<V>(p.S[r] + p.stride + off);
      tree.push(r, sx, sb);
    }
    tree.finish(p.world);
    for (uint32_t r = 0; r < p.world; ++r) {
      st_stream<V>(p.S[r] + off, tree.x[0]);
      st_stream<V>(p.S[r] + p.stride + off, tree.b[0]);
    }
  }
}

}  // namespace la
