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
    typename TreeFor<W_, V>::type tree;
#pragma unroll kOuterUnroll
    for (uint32_t i0 = 0; i0 < W; i0 += CH) {
      ReplicaChunk<V, CH> ch;
      load_chunk<V, CH>(ch, addr, b_delta, stride_bytes, W, i0);
#pragma unroll
      for (int k = 0; k < CH; ++k)
        if (i0 + k < W) tree.push_in_chunk(i0 + k, k, i0 + CH <= W, ch.x[k], ch.b[k]);
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
    PairTreeDyn<V> tree;
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

// ---- the local steps next to a synchronisation, fused with the exchange -----------------------
// step_export: the local step that makes t' reach H.  Its results y_i, A_i^2 are about to be
// replaced by the means, so they are never stored: only their adjacent-pair tree sums go to the
// exchange buffer (read 16 B, write ~0 B per worker*param).
// import_step: the first step of the next period.  It starts from total / W_total read from the
// exchange buffer instead of from the replicas (read ~0 B, write 16 B per worker*param).
// Together the synchronisation costs no HBM pass of its own; what crosses NVLink stays 2N floats.
template <int W_, int V, int GM, bool BF16, int MINB>
__global__ void __launch_bounds__(LA_BLOCK, MINB) la_step_export(const SweepParams p, float* __restrict__ S) {
  constexpr bool kNeedsNoise = (GM == kGradNoise || GM == kGradNoiseScaled || GM == kGradQuadratic);
  constexpr bool kExternal = (GM == kGradExternalF32 || GM == kGradExternalBF16);
  constexpr uint64_t kGradElem = (GM == kGradExternalBF16) ? 2 : 4;
  constexpr int CH = (W_ > 0) ? (W_ < LA_CH ? W_ : LA_CH) : 4;
  constexpr int kOuterUnroll = (W_ > 0) ? kMaxWorkers : 1;
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;

  __shared__ uint64_t keys[kMaxWorkers];
  if (kNeedsNoise) {
    if (threadIdx.x < W) keys[threadIdx.x] = step_worker_key(p.seed, step_index(p), p.identical_workers ? 0u : p.worker_base + threadIdx.x);
    __syncthreads();
  }
  const float eps2 = __fmul_rn(p.eps, p.eps);
  const float q = __fmul_rn(__uint2float_rn(p.tp), eps2);
  float eta_t = p.eta;
  if (p.warm_up_steps != 0u) {
    const float ratio = __fdiv_rn(__ull2float_rn(step_index(p)), __uint2float_rn(p.warm_up_steps));
    eta_t = __fmul_rn(p.eta, fminf(1.0f, ratio));
  }

  const uint64_t ngroups = (p.n + (uint64_t)(V - 1)) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (grp >= ngroups) return;
  const uint64_t x_base = reinterpret_cast<uint64_t>(p.X);
  const uint64_t b_delta = reinterpret_cast<uint64_t>(p.B2) - x_base;
  const uint64_t stride_bytes = p.stride * sizeof(float);
  const uint64_t g_base = reinterpret_cast<uint64_t>(p.gext);
  const uint64_t g_row_bytes = p.n * kGradElem;

  ReplicaChunk<V, CH> nxt;
  GradChunk<V, kExternal ? CH : 1> gnxt;
  CoordInputs<V> in_next;
  load_coord<GM, true, true, V>(in_next, p, grp * V);
  uint64_t ld_addr = x_base + grp * (V * sizeof(float));
  uint64_t g_addr = g_base + grp * (V * kGradElem);
  load_chunk<V, CH>(nxt, ld_addr, b_delta, stride_bytes, W, 0u);
  if (kExternal) load_grads<GM, V, kExternal ? CH : 1>(gnxt, p, g_addr, g_row_bytes, W, 0u, grp * V);

  for (;;) {
    const uint64_t off = grp * V;
    const uint64_t next_grp = grp + nthreads;
    const bool has_next = next_grp < ngroups;
    const CoordInputs<V> in = in_next;
    const uint64_t ctr0 = kGoldenGamma * (((p.j_base + off) >> 1) + 1u);
    const Vec<V> r = step_size<V>(in.bs, q, eta_t);
    typename TreeFor<W_, V>::type tree;
#pragma unroll kOuterUnroll
    for (uint32_t i0 = 0; i0 < W; i0 += CH) {
      ReplicaChunk<V, CH> cur = nxt;
      GradChunk<V, kExternal ? CH : 1> gcur = gnxt;
      if (i0 + CH < W) {
        load_chunk<V, CH>(nxt, ld_addr, b_delta, stride_bytes, W, i0 + CH);
        if (kExternal) load_grads<GM, V, kExternal ? CH : 1>(gnxt, p, g_addr, g_row_bytes, W, i0 + CH, off);
      } else if (has_next) {
        load_coord<GM, true, true, V>(in_next, p, next_grp * V);
        ld_addr = x_base + next_grp * (V * sizeof(float));
        load_chunk<V, CH>(nxt, ld_addr, b_delta, stride_bytes, W, 0u);
        if (kExternal) {
          g_addr = g_base + next_grp * (V * kGradElem);
          load_grads<GM, V, kExternal ? CH : 1>(gnxt, p, g_addr, g_row_bytes, W, 0u, next_grp * V);
        }
      }
      asm volatile("" ::: "memory");
#pragma unroll
      for (int k = 0; k < CH; ++k)
        if (i0 + k < W) {
          const uint32_t i = i0 + k;
          const Vec<V> g = kExternal ? gcur.g[kExternal ? k : 0]
                                     : gradient<GM, BF16, V>(p, in, cur.x[k], kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
          apply<V>(r, g, cur.x[k], cur.b[k]);
          tree.push_in_chunk(i, k, i0 + CH <= W, cur.x[k], cur.b[k]);
        }
    }
    tree.finish();
    st_stream<V>(S + off, tree.x[0]);
    st_stream<V>(S + p.stride + off, tree.b[0]);
    if (!has_next) break;
    grp = next_grp;
  }
}

template <int W_, int V, int GM, bool BF16, int MINB>
__global__ void __launch_bounds__(LA_BLOCK, MINB) la_import_step(const SweepParams p, const float* __restrict__ S,
                                                                 uint32_t W_total) {
  constexpr bool kNeedsNoise = (GM == kGradNoise || GM == kGradNoiseScaled || GM == kGradQuadratic);
  constexpr int kOuterUnroll = (W_ > 0) ? kMaxWorkers : 1;
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;
  __shared__ uint64_t keys[kMaxWorkers];
  if (kNeedsNoise) {
    if (threadIdx.x < W) keys[threadIdx.x] = step_worker_key(p.seed, step_index(p), p.identical_workers ? 0u : p.worker_base + threadIdx.x);
    __syncthreads();
  }
  const float eps2 = __fmul_rn(p.eps, p.eps);
  const float q = __fmul_rn(__uint2float_rn(p.tp), eps2);  // p.tp == 1: first step of the period
  float eta_t = p.eta;
  if (p.warm_up_steps != 0u) {
    const float ratio = __fdiv_rn(__ull2float_rn(step_index(p)), __uint2float_rn(p.warm_up_steps));
    eta_t = __fmul_rn(p.eta, fminf(1.0f, ratio));
  }
  const uint64_t ngroups = (p.n + (uint64_t)(V - 1)) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t x_base = reinterpret_cast<uint64_t>(p.X);
  const uint64_t b_delta = reinterpret_cast<uint64_t>(p.B2) - x_base;
  const uint64_t stride_bytes = p.stride * sizeof(float);
  for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += nthreads) {
    const uint64_t off = grp * V;
    CoordInputs<V> in;
    load_coord<GM, true, false, V>(in, p, off);
    const Vec<V> xm = div_by_workers<0, V>(ld_stream<V>(S + off), W_total);
    const Vec<V> bm = div_by_workers<0, V>(ld_stream<V>(S + p.stride + off), W_total);
    st_stream<V>(p.Bs + off, bm);
    const Vec<V> r = step_size<V>(bm, q, eta_t);
    const uint64_t ctr0 = kGoldenGamma * (((p.j_base + off) >> 1) + 1u);
    uint64_t st_addr = x_base + off * sizeof(float);
#pragma unroll kOuterUnroll
    for (uint32_t i = 0; i < W; ++i) {
      Vec<V> xv = xm, bv = bm;
      const Vec<V> g = gradient<GM, BF16, V>(p, in, xv, kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
      apply<V>(r, g, xv, bv);
      store_replica<V>(st_addr, b_delta, stride_bytes, xv, bv);
    }
  }
}

using ExchangeFn = void (*)(const ExchangeParams);
using StepExportFn = void (*)(const SweepParams, float*);
using ImportStepFn = void (*)(const SweepParams, const float*, uint32_t);
StepExportFn lookup_step_export(int W, int gm, bool bf16);
ImportStepFn lookup_import_step(int W, int gm, bool bf16);
ExchangeFn lookup_export(int W);

}  // namespace la
