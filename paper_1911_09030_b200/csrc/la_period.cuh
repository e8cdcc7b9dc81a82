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
#ifndef LA_PERIOD_BLOCK
#define LA_PERIOD_BLOCK LA_BLOCK
#endif
#ifndef LA_PERIOD_CH
#define LA_PERIOD_CH 8  // replicas whose gradient chains are interleaved
#endif

namespace la {

constexpr int kPeriodMax = 8;  // steps per pass
constexpr int kPeriodUnroll = LA_PERIOD_UNROLL;

struct PeriodParams {
  SweepParams base;  // base.t = global step BEFORE the first of the h steps, base.tp = t' before it
  uint32_t h;        // 1..kPeriodMax
};

template <int W_, int V, int GM, bool BF16, bool POST, int MINB>
__global__ void __launch_bounds__(LA_PERIOD_BLOCK, MINB) la_period(const PeriodParams pp) {
  const SweepParams& p = pp.base;
  constexpr bool kNeedsNoise = (GM == kGradNoise || GM == kGradNoiseScaled || GM == kGradQuadratic);
  // replicas per chunk: eight where W is a multiple of eight (not for the bf16 variants, which
  // would spill with eight chains in flight), four otherwise
  constexpr int kChunkMax = (W_ % 8 == 0 && !BF16) ? LA_PERIOD_CH : (LA_PERIOD_CH < 4 ? LA_PERIOD_CH : 4);
  constexpr int CH = (W_ > 0) ? (W_ < kChunkMax ? W_ : kChunkMax) : 4;
  constexpr int kOuterUnroll = (W_ > 0) ? kMaxWorkers : 1;
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;
  const uint32_t h = pp.h;

  // stream keys of every (step, worker) of this pass, and the per-step scalars
#ifdef LA_DEBUG
  dbg_begin(p.dbg);
#endif
  __shared__ uint64_t keys[kPeriodMax][kMaxWorkers];
  __shared__ float eta_s[kPeriodMax], q_s[kPeriodMax];
  __shared__ Vec<V> r_s[kPeriodMax][LA_PERIOD_BLOCK];
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
  const uint64_t x_base = reinterpret_cast<uint64_t>(p.X);
  const uint64_t b_delta = reinterpret_cast<uint64_t>(p.B2) - x_base;
  const uint64_t stride_bytes = p.stride * sizeof(float);

  // The kernel is bound by instruction issue, not by HBM (a sixth of the bandwidth is in use), so
  // unlike la_sweep it does not prefetch the next chunk while one is processed: the registers that
  // would hold loads in flight are worth more as room for interleaving the gradient chains, and
  // the other resident blocks cover the load latency.
  for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += nthreads) {
    const uint64_t off = grp * V;
    CoordInputs<V> in;
    load_coord<GM, true, true, V>(in, p, off);
    const uint64_t ctr0 = kGoldenGamma * (((p.j_base + off) >> 1) + 1u);
    uint64_t ld_addr = x_base + off * sizeof(float);
    uint64_t st_addr = ld_addr;

    // step sizes of the h steps: the stale accumulator is fixed, only t' eps^2 ramps.  They live
    // in this thread's own shared-memory column so that the loop over steps can stay rolled: with
    // it unrolled the kernel body (W x 8 copies of the gradient source) overflowed the
    // instruction cache and a fifth of the issue slots went to instruction-fetch stalls.
    for (uint32_t s = 0; s < h; ++s) r_s[s][threadIdx.x] = step_size<V>(in.bs, q_s[s], eta_s[s]);
    typename TreeFor<W_, V>::type tree;

#pragma unroll kOuterUnroll
    for (uint32_t i0 = 0; i0 < W; i0 += CH) {
      ReplicaChunk<V, CH> cur;
      load_chunk<V, CH>(cur, ld_addr, b_delta, stride_bytes, W, i0 LA_DBG_ARG(x_base + off * sizeof(float)));
      // steps outside, the chunk's replicas inside: CH independent gradient chains per iteration
#pragma unroll kPeriodUnroll
      for (uint32_t s = 0; s < h; ++s) {
        const Vec<V> r = r_s[s][threadIdx.x];
#pragma unroll
        for (int k = 0; k < CH; ++k)
          if (i0 + k < W) {
            const uint32_t i = i0 + k;
            const Vec<V> g = gradient<GM, BF16, V>(p, in, cur.x[k], kNeedsNoise ? keys[s][i] : 0ull, ctr0, i, off);
            apply<V>(r, g, cur.x[k], cur.b[k]);
          }
      }
#pragma unroll
      for (int k = 0; k < CH; ++k)
        if (i0 + k < W) {
          if (POST) {
            tree.push_in_chunk(i0 + k, k, i0 + CH <= W, cur.x[k], cur.b[k]);
          } else {
            store_replica<V>(st_addr, b_delta, stride_bytes, cur.x[k], cur.b[k]
                             LA_DBG_ARG(x_base + off * sizeof(float) + (uint64_t)(i0 + k) * stride_bytes));
          }
        }
    }
    if (POST) {
      tree.finish(W);
      const Vec<V> xm = div_by_workers<W_, V>(tree.x[0], W);
      const Vec<V> bm = div_by_workers<W_, V>(tree.b[0], W);
      st_stream<V>(p.Bs + off, bm);
#pragma unroll kOuterUnroll
      for (uint32_t i = 0; i < W; ++i)
        store_replica<V>(st_addr, b_delta, stride_bytes, xm, bm LA_DBG_ARG(x_base + off * sizeof(float) + (uint64_t)i * stride_bytes));
    }
  }
}

using PeriodFn = void (*)(const PeriodParams);
struct PeriodKernel {
  PeriodFn fn;
  int vec;
  int block;  // threads per block the kernel was compiled for
};
PeriodKernel lookup_period(int W, int gm, bool bf16, bool post);

}  // namespace la
