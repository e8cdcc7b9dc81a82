// Temporal blocking: up to kPeriodMax consecutive local iterations of Algorithm 3 in ONE pass.
//
// Between two synchronisations a worker's coordinate depends only on its own history (the
// gradient is evaluated at the worker's own x, the denominator B^2_{t-t'} + t' eps^2 is fixed at
// the last sync plus a known ramp), and the synthetic gradient lives in registers.  So a thread
// can load x and B^2 of a replica once, apply h steps back to back, and store once: HBM traffic
// per worker*param update falls from 16 + S/W bytes to (16 + S/W)/h, and the kernel becomes
// bound by instruction issue instead of HBM.  Every element sees exactly the operations of h
// separate local steps, in the same order, so the result is bit-identical.
// If the h steps close the period (POST), the synchronisation is applied before the store.
#pragma once
#include "la_sweep.cuh"

#ifndef LA_PERIOD_UNROLL
#define LA_PERIOD_UNROLL 2
#endif

namespace la {

constexpr int kPeriodMax = 8;  // steps per pass
constexpr int kPeriodUnroll = LA_PERIOD_UNROLL;

struct PeriodParams {
  SweepParams base;  // base.t = global step BEFORE the first of the h steps, base.tp = t' before it
  uint32_t h;        // 1..kPeriodMax
};

template <int W_, int V, int GM, bool BF16, bool POST, int MINB>
__global__ void __launch_bounds__(LA_BLOCK, MINB) la_period(const PeriodParams pp) {
  const SweepParams& p = pp.base;
  constexpr bool kNeedsNoise = (GM == kGradNoise || GM == kGradNoiseScaled || GM == kGradQuadratic);
  constexpr int CH = (W_ > 0) ? (W_ < LA_CH ? W_ : LA_CH) : 4;
  constexpr int kOuterUnroll = (W_ > 0) ? kMaxWorkers : 1;
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;
  const uint32_t h = pp.h;

  // stream keys of every (step, worker) of this pass, and the per-step scalars
  __shared__ uint64_t keys[kPeriodMax][kMaxWorkers];
  __shared__ float eta_s[kPeriodMax], q_s[kPeriodMax];
  __shared__ Vec<V> r_s[kPeriodMax][LA_BLOCK];
  if (kNeedsNoise) {
    for (uint32_t k = threadIdx.x; k < h * W; k += blockDim.x) {
      const uint32_t s = k / W, i = k - s * W;
      keys[s][i] = step_worker_key(p.seed, step_index(p) + 1u + s, p.identical_workers ? 0u : p.worker_base + i);
    }
  }
  if (threadIdx.x < h) {
    const uint32_t s = threadIdx.x;
    const float eps2 = __fmul_rn(p.eps, p.eps);
    q_s[s] = __fmul_rn(__uint2float_rn(p.tp + 1u + s), eps2);  // t' eps^2 of step s
    float e = p.eta;
    if (p.warm_up_steps != 0u) {
      const float ratio = __fdiv_rn(__ull2float_rn(step_index(p) + 1u + s), __uint2float_rn(p.warm_up_steps));
      e = __fmul_rn(p.eta, fminf(1.0f, ratio));
    }
    eta_s[s] = e;
  }
  __syncthreads();

  const uint64_t ngroups = (p.n + (uint64_t)(V - 1)) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (grp >= ngroups) return;
  const uint64_t x_base = reinterpret_cast<uint64_t>(p.X);
  const uint64_t b_delta = reinterpret_cast<uint64_t>(p.B2) - x_base;
  const uint64_t stride_bytes = p.stride * sizeof(float);

  ReplicaChunk<V, CH> nxt;
  CoordInputs<V> in_next;
  load_coord<GM, true, true, V>(in_next, p, grp * V);
  uint64_t ld_addr = x_base + grp * (V * sizeof(float));
  load_chunk<V, CH>(nxt, ld_addr, b_delta, stride_bytes, W, 0u);

  for (;;) {
    const uint64_t off = grp * V;
    const uint64_t next_grp = grp + nthreads;
    const bool has_next = next_grp < ngroups;
    const CoordInputs<V> in = in_next;
    const uint64_t ctr0 = kGoldenGamma * (((p.j_base + off) >> 1) + 1u);
    uint64_t st_addr = x_base + off * sizeof(float);

    // step sizes of the h steps: the stale accumulator is fixed, only t' eps^2 ramps.  They live
    // in this thread's own shared-memory column so that the loop over steps can stay rolled: with
    // it unrolled the kernel body (W x 8 copies of the gradient source) overflowed the
    // instruction cache and a fifth of the issue slots went to instruction-fetch stalls.
    for (uint32_t s = 0; s < h; ++s) r_s[s][threadIdx.x] = step_size<V>(in.bs, q_s[s], eta_s[s]);
    typename TreeFor<W_, V>::type tree;

#pragma unroll kOuterUnroll
    for (uint32_t i0 = 0; i0 < W; i0 += CH) {
      ReplicaChunk<V, CH> cur = nxt;
      if (i0 + CH < W) {
        load_chunk<V, CH>(nxt, ld_addr, b_delta, stride_bytes, W, i0 + CH);
      } else if (has_next) {
        load_coord<GM, true, true, V>(in_next, p, next_grp * V);
        ld_addr = x_base + next_grp * (V * sizeof(float));
        load_chunk<V, CH>(nxt, ld_addr, b_delta, stride_bytes, W, 0u);
      }
      asm volatile("" ::: "memory");
#pragma unroll
      for (int k = 0; k < CH; ++k)
        if (i0 + k < W) {
          const uint32_t i = i0 + k;
#pragma unroll kPeriodUnroll
          for (uint32_t s = 0; s < h; ++s) {
            const Vec<V> g = gradient<GM, BF16, V>(p, in, cur.x[k], kNeedsNoise ? keys[s][i] : 0ull, ctr0, i, off);
            apply<V>(r_s[s][threadIdx.x], g, cur.x[k], cur.b[k]);
          }
          if (POST) {
            tree.push_in_chunk(i, k, i0 + CH <= W, cur.x[k], cur.b[k]);
          } else {
            store_replica<V>(st_addr, b_delta, stride_bytes, cur.x[k], cur.b[k]);
          }
        }
    }
    if (POST) {
      tree.finish();
      const Vec<V> xm = div_by_workers<W_, V>(tree.x[0], W);
      const Vec<V> bm = div_by_workers<W_, V>(tree.b[0], W);
      st_stream<V>(p.Bs + off, bm);
#pragma unroll kOuterUnroll
      for (uint32_t i = 0; i < W; ++i) store_replica<V>(st_addr, b_delta, stride_bytes, xm, bm);
    }
    if (!has_next) break;
    grp = next_grp;
  }
}

using PeriodFn = void (*)(const PeriodParams);
struct PeriodKernel {
  PeriodFn fn;
  int vec;
};
PeriodKernel lookup_period(int W, int gm, bool bf16, bool post);

}  // namespace la
