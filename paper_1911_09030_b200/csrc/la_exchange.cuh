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
#pragma once
#include "la_sweep.cuh"

namespace la {

constexpr int kMaxRanks = 16;

struct ExchangeParams {
  float* S[kMaxRanks];   // exchange buffers of all ranks; S[r] = sums of x, S[r] + stride = sums of B^2
  float* X;              // local replicas
  float* B2;
  float* Bs;
  uint64_t n, stride;
  uint64_t slice_lo, slice_hi;  // this rank's coordinate slice for `combine` (multiples of 64)
  uint32_t W, W_total, rank, world;
};

template <int W_, int V>
__global__ void __launch_bounds__(LA_BLOCK) la_export_sums(const ExchangeParams p) {
  constexpr int CH = (W_ > 0) ? (W_ < LA_CH ? W_ : LA_CH) : 4;
  constexpr int kOuterUnroll = (W_ > 0) ? kMaxWorkers : 1;
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;
  const uint64_t ngroups = (p.n + (uint64_t)(V - 1)) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t x_base = reinterpret_cast<uint64_t>(p.X);
  const uint64_t b_delta = reinterpret_cast<uint64_t>(p.B2) - x_base;
  const uint64_t stride_bytes = p.stride * sizeof(float);
  float* out = p.S[p.rank];
  for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += nthreads) {
    const uint64_t off = grp * V;
    uint64_t addr = x_base + off * sizeof(float);
    PairTree<V> tree;
#pragma unroll kOuterUnroll
    for (uint32_t i0 = 0; i0 < W; i0 += CH) {
      ReplicaChunk<V, CH> ch;
      load_chunk<V, CH>(ch, addr, b_delta, stride_bytes, W, i0);
#pragma unroll
      for (int k = 0; k < CH; ++k)
        if (i0 + k < W) tree.push(i0 + k, ch.x[k], ch.b[k]);
    }
    tree.finish();
    st_stream<V>(out + off, tree.x[0]);
    st_stream<V>(out + p.stride + off, tree.b[0]);
  }
}

template <int V>
__global__ void __launch_bounds__(LA_BLOCK) la_combine_sums(const ExchangeParams p) {
  const uint64_t ngroups = (p.slice_hi - p.slice_lo) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += nthreads) {
    const uint64_t off = p.slice_lo + grp * V;
    PairTree<V> tree;
    for (uint32_t r = 0; r < p.world; ++r) {
      // plain loads; for r != rank these are peer loads over NVLink.  Not the streaming
      // (evict-first) flavour: a peer's line is fetched once and not re-read.
      const Vec<V> sx = ld_stream<V>(p.S[r] + off);
      const Vec<V> sb = ld_stream<V>(p.S[r] + p.stride + off);
      tree.push(r, sx, sb);
    }
    tree.finish();
    for (uint32_t r = 0; r < p.world; ++r) {
      st_stream<V>(p.S[r] + off, tree.x[0]);
      st_stream<V>(p.S[r] + p.stride + off, tree.b[0]);
    }
  }
}

template <int V>
__global__ void __launch_bounds__(LA_BLOCK) la_import_means(const ExchangeParams p) {
  const uint64_t ngroups = (p.n + (uint64_t)(V - 1)) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t x_base = reinterpret_cast<uint64_t>(p.X);
  const uint64_t b_delta = reinterpret_cast<uint64_t>(p.B2) - x_base;
  const uint64_t stride_bytes = p.stride * sizeof(float);
  const float* in = p.S[p.rank];
  for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += nthreads) {
    const uint64_t off = grp * V;
    const Vec<V> xm = div_by_workers<0, V>(ld_stream<V>(in + off), p.W_total);
    const Vec<V> bm = div_by_workers<0, V>(ld_stream<V>(in + p.stride + off), p.W_total);
    st_stream<V>(p.Bs + off, bm);
    uint64_t addr = x_base + off * sizeof(float);
    for (uint32_t i = 0; i < p.W; ++i) store_replica<V>(addr, b_delta, stride_bytes, xm, bm);
  }
}

using ExchangeFn = void (*)(const ExchangeParams);
ExchangeFn lookup_export(int W);

}  // namespace la
