// The sweep kernel: Algorithm 3 (Local AdaAlter) for all W workers, one pass over HBM.
//
// Mapping.  Algorithm 3 is coordinate-wise (Hadamard operations and a per-coordinate mean
// over workers), so one thread owns a group of four consecutive coordinates FOR ALL W
// replicas: it reads the worker-independent data once (the stale accumulator, the problem
// arrays), forms the shared step size once, then walks the replicas.  The mean over workers
// is therefore a register reduction in a fixed order; no shuffles, shared memory or atomics.
//
// One template covers the four kernels of the path:
//   PRE   average the replicas that are read (a synchronisation BEFORE the step)
//   STEP  one local iteration: gradient, x update, B^2 accumulate
//   POST  average the replicas that are written (the synchronisation of Algorithm 3's
//         else-branch, applied to y and A^2 of this very step)
//   K1 = STEP            local step
//   K2 = PRE             stand-alone synchronisation
//   K3 = STEP+POST       step t'=H fused with its synchronisation
//   K4 = PRE+STEP        synchronisation fused into the first step of the next period
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "grad_source.cuh"

namespace la {

enum GradKind : int {
  kGradNoise = 0,        // g = xi
  kGradNoiseScaled = 1,  // g = s_j xi
  kGradQuadratic = 2,    // g = a_j (x - c_j) + sigma xi
  kGradConstant = 3,     // g = s_j (s == nullptr: 1)
  kGradExternalF32 = 4,  // g read from a [W][N] fp32 table
  kGradExternalBF16 = 5  // g read from a [W][N] bf16 table
};

struct SweepParams {
  float* X;        // [W][stride]
  float* B2;       // [W][stride]
  float* Bs;       // [stride]   accumulator as of the last synchronisation
  const float* a;  // [stride] or null
  const float* c;  // [stride] or null
  const float* s;  // [stride] or null
  const void* gext;    // external gradients, [W][N]
  uint64_t n;          // logical coordinates N
  uint64_t ngroups;    // ceil(N / 4)
  uint64_t stride;     // replica stride in floats (multiple of 64, >= 4*ngroups)
  uint64_t j_base;     // global index of coordinate 0 (multiple of 4)
  uint64_t seed;
  uint64_t t;          // 1-based global step index of the STEP part
  uint32_t W;
  uint32_t tp;         // t' of the STEP part (local steps since the last sync, incl. this one)
  uint32_t warm_up_steps;
  uint32_t identical_workers;
  float eta, eps, sigma;
};

constexpr int kMaxWorkers = 64;
constexpr int kTreeDepth = 7;  // log2(kMaxWorkers) + 1 partial sums

__device__ __forceinline__ float4 ld_stream(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st_stream(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

__device__ __forceinline__ float4 add4(float4 l, float4 r) {
  return make_float4(__fadd_rn(l.x, r.x), __fadd_rn(l.y, r.y), __fadd_rn(l.z, r.z), __fadd_rn(l.w, r.w));
}

// Mean over workers = adjacent-pair tree sum, then one division by (float)W.  For a power of
// two the division is replaced by the multiplication with the exact reciprocal, which rounds
// the same real number and therefore gives the same bits.
template <int W_>
__device__ __forceinline__ float4 div_by_workers(float4 v, uint32_t W) {
  if (W_ > 0 && (W_ & (W_ - 1)) == 0) {
    const float inv = 1.0f / (float)W_;
    return make_float4(__fmul_rn(v.x, inv), __fmul_rn(v.y, inv), __fmul_rn(v.z, inv), __fmul_rn(v.w, inv));
  }
  const float w = __uint2float_rn(W);
  return make_float4(__fdiv_rn(v.x, w), __fdiv_rn(v.y, w), __fdiv_rn(v.z, w), __fdiv_rn(v.w, w));
}

// Streaming form of the adjacent-pair tree: a stack of partial sums, one per level, merged
// like the carries of a binary counter.  After pushing worker i the two top entries are
// merged once for every trailing zero bit of (i+1); left operand = older entry.  With W known
// at compile time the loop unrolls and every stack index is a constant (registers only).
struct PairTree {
  float4 x[kTreeDepth], b[kTreeDepth];
  int sp = 0;
  __device__ __forceinline__ void push(uint32_t i, float4 vx, float4 vb) {
    x[sp] = vx;
    b[sp] = vb;
    ++sp;
    for (uint32_t cnt = i + 1u; (cnt & 1u) == 0u; cnt >>= 1) {
      --sp;
      x[sp - 1] = add4(x[sp - 1], x[sp]);
      b[sp - 1] = add4(b[sp - 1], b[sp]);
    }
  }
  __device__ __forceinline__ void finish() {
    while (sp > 1) {
      --sp;
      x[sp - 1] = add4(x[sp - 1], x[sp]);
      b[sp - 1] = add4(b[sp - 1], b[sp]);
    }
  }
};

// Worker-independent data of one coordinate group: the stale accumulator and the problem arrays.
struct CoordInputs {
  float4 bs, a, c, s;
};

template <int GM, bool STEP, bool LOAD_BS>
__device__ __forceinline__ void load_coord(CoordInputs& in, const SweepParams& p, uint64_t off) {
  if (LOAD_BS) in.bs = ld_stream(p.Bs + off);
  if (STEP) {
    if (GM == kGradQuadratic) {
      in.a = ld_stream(p.a + off);
      in.c = ld_stream(p.c + off);
    }
    if (GM == kGradNoiseScaled) in.s = ld_stream(p.s + off);
    if (GM == kGradConstant) in.s = p.s ? ld_stream(p.s + off) : make_float4(1.f, 1.f, 1.f, 1.f);
  }
}

// x and B^2 of CH consecutive replicas for one coordinate group.
template <int CH>
struct ReplicaChunk {
  float4 x[CH], b[CH];
};

template <int CH>
__device__ __forceinline__ void load_chunk(ReplicaChunk<CH>& ch, const SweepParams& p, uint32_t W, uint32_t i0,
                                           uint64_t off) {
#pragma unroll
  for (int k = 0; k < CH; ++k)
    if (i0 + k < W) {
      ch.x[k] = ld_stream(p.X + (uint64_t)(i0 + k) * p.stride + off);
      ch.b[k] = ld_stream(p.B2 + (uint64_t)(i0 + k) * p.stride + off);
    }
}

// r = eta_t / sqrt(B^2_{t-t'} + t' eps^2): the step size all workers share (Section 4.2).
__device__ __forceinline__ float4 step_size(float4 bs, float q, float eta_t) {
  float4 r;
  r.x = __fdiv_rn(eta_t, __fsqrt_rn(__fadd_rn(bs.x, q)));
  r.y = __fdiv_rn(eta_t, __fsqrt_rn(__fadd_rn(bs.y, q)));
  r.z = __fdiv_rn(eta_t, __fsqrt_rn(__fadd_rn(bs.z, q)));
  r.w = __fdiv_rn(eta_t, __fsqrt_rn(__fadd_rn(bs.w, q)));
  return r;
}

// Gradient of four coordinates for one worker.  `xv` is the worker's own iterate
// (Algorithm 3: G_{i,t} = grad f(x_{i,t-1}; z_{i,t})).
template <int GM, bool BF16>
__device__ __forceinline__ float4 gradient4(const SweepParams& p, const CoordInputs& in, float4 xv,
                                            uint64_t key, uint64_t ctr0, uint32_t worker, uint64_t off) {
  float4 g;
  if (GM == kGradConstant) {
    return in.s;
  } else if (GM == kGradExternalF32 || GM == kGradExternalBF16) {
    const uint64_t base = (uint64_t)worker * p.n + off;
    float v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v[k] = 0.0f;
      if (off + k < p.n) {
        if (GM == kGradExternalF32) {
          v[k] = __ldcs(reinterpret_cast<const float*>(p.gext) + base + k);
        } else {
          const unsigned short h = __ldcs(reinterpret_cast<const unsigned short*>(p.gext) + base + k);
          v[k] = __uint_as_float((uint32_t)h << 16);
        }
      }
    }
    return make_float4(v[0], v[1], v[2], v[3]);
  } else {
    float4 xi;
    normal_pair(key, ctr0, xi.x, xi.y);
    normal_pair(key, ctr0 + kGoldenGamma, xi.z, xi.w);
    if (GM == kGradNoise) {
      g = xi;
    } else if (GM == kGradNoiseScaled) {
      g = make_float4(__fmul_rn(in.s.x, xi.x), __fmul_rn(in.s.y, xi.y), __fmul_rn(in.s.z, xi.z),
                      __fmul_rn(in.s.w, xi.w));
    } else {  // quadratic
      g.x = __fmaf_rn(in.a.x, __fsub_rn(xv.x, in.c.x), __fmul_rn(p.sigma, xi.x));
      g.y = __fmaf_rn(in.a.y, __fsub_rn(xv.y, in.c.y), __fmul_rn(p.sigma, xi.y));
      g.z = __fmaf_rn(in.a.z, __fsub_rn(xv.z, in.c.z), __fmul_rn(p.sigma, xi.z));
      g.w = __fmaf_rn(in.a.w, __fsub_rn(xv.w, in.c.w), __fmul_rn(p.sigma, xi.w));
    }
    if (BF16) {
      g.x = round_through_bf16(g.x);
      g.y = round_through_bf16(g.y);
      g.z = round_through_bf16(g.z);
      g.w = round_through_bf16(g.w);
    }
  }
  return g;
}

// y = x - r g ; A^2 = B^2 + g g   (Algorithm 3), one fused multiply-add each.
__device__ __forceinline__ void apply4(float4 r, float4 g, float4& x, float4& b) {
  x.x = __fmaf_rn(-r.x, g.x, x.x);
  x.y = __fmaf_rn(-r.y, g.y, x.y);
  x.z = __fmaf_rn(-r.z, g.z, x.z);
  x.w = __fmaf_rn(-r.w, g.w, x.w);
  b.x = __fmaf_rn(g.x, g.x, b.x);
  b.y = __fmaf_rn(g.y, g.y, b.y);
  b.z = __fmaf_rn(g.z, g.z, b.z);
  b.w = __fmaf_rn(g.w, g.w, b.w);
}

#ifndef LA_BLOCK
#define LA_BLOCK 256
#endif
#ifndef LA_CH
#define LA_CH 4
#endif
constexpr int kBlockThreads = LA_BLOCK;

template <int W_, int GM, bool BF16, bool PRE, bool STEP, bool POST, int MINB>
__global__ void __launch_bounds__(LA_BLOCK, MINB) la_sweep(const SweepParams p) {
  static_assert(!(PRE && POST), "one synchronisation per pass");
  constexpr bool kNeedsNoise = STEP && (GM == kGradNoise || GM == kGradNoiseScaled || GM == kGradQuadratic);
  constexpr int CH = (W_ > 0) ? (W_ < LA_CH ? W_ : LA_CH) : 4;  // replicas loaded before any is consumed
  constexpr int kOuterUnroll = (W_ > 0) ? kMaxWorkers : 1;  // static W: unroll fully, so that the
                                                             // reduction stack is indexed by constants
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;

  __shared__ uint64_t keys[kMaxWorkers];
  if (kNeedsNoise) {
    if (threadIdx.x < W) keys[threadIdx.x] = step_worker_key(p.seed, p.t, p.identical_workers ? 0u : threadIdx.x);
    __syncthreads();
  }

  // per-step scalars (worker- and coordinate-independent)
  float q = 0.f, eta_t = 0.f;
  if (STEP) {
    const float eps2 = __fmul_rn(p.eps, p.eps);
    q = __fmul_rn(__uint2float_rn(p.tp), eps2);  // t' eps^2, the placeholder of Section 4.2
    eta_t = p.eta;
    if (p.warm_up_steps != 0u) {  // Section 6.2: eta_t = eta min(1, t / warm_up_steps)
      const float ratio = __fdiv_rn(__ull2float_rn(p.t), __uint2float_rn(p.warm_up_steps));
      eta_t = __fmul_rn(p.eta, fminf(1.0f, ratio));
    }
  }

  // Grid-stride loop over coordinate groups, software-pipelined: while the replicas of one
  // chunk are being consumed, the loads of the next chunk (or of the next group's first chunk
  // and worker-independent data) are already in flight.  The empty asm statements pin that
  // order against the compiler's scheduler.
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (grp >= p.ngroups) return;
  constexpr bool kLoadsBs = STEP && !PRE;

  ReplicaChunk<CH> nxt;
  CoordInputs in_next;
  load_coord<GM, STEP, kLoadsBs>(in_next, p, grp * 4u);
  load_chunk<CH>(nxt, p, W, 0u, grp * 4u);

  for (;;) {
    const uint64_t off = grp * 4u;
    const uint64_t next_grp = grp + nthreads;
    const bool has_next = next_grp < p.ngroups;
    const CoordInputs in = in_next;
    const uint64_t ctr0 = kGoldenGamma * (((p.j_base + off) >> 1) + 1u);

    float4 r;
    if (kLoadsBs) r = step_size(in.bs, q, eta_t);
    PairTree tree;

#pragma unroll kOuterUnroll
    for (uint32_t i0 = 0; i0 < W; i0 += CH) {
      ReplicaChunk<CH> cur = nxt;
      if (i0 + CH < W) {
        load_chunk<CH>(nxt, p, W, i0 + CH, off);
      } else if (has_next) {
        load_coord<GM, STEP, kLoadsBs>(in_next, p, next_grp * 4u);
        load_chunk<CH>(nxt, p, W, 0u, next_grp * 4u);
      }
      asm volatile("" ::: "memory");
#pragma unroll
      for (int k = 0; k < CH; ++k)
        if (i0 + k < W) {
          const uint32_t i = i0 + k;
          if (PRE) {
            tree.push(i, cur.x[k], cur.b[k]);
          } else {
            const float4 g = gradient4<GM, BF16>(p, in, cur.x[k], kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
            apply4(r, g, cur.x[k], cur.b[k]);
            if (POST) {
              tree.push(i, cur.x[k], cur.b[k]);
            } else {
              st_stream(p.X + (uint64_t)i * p.stride + off, cur.x[k]);
              st_stream(p.B2 + (uint64_t)i * p.stride + off, cur.b[k]);
            }
          }
        }
    }

    if (PRE || POST) {
      // synchronisation branch of Algorithm 3: means over workers; the mean accumulator is
      // also the new stale denominator
      tree.finish();
      const float4 xm = div_by_workers<W_>(tree.x[0], W);
      const float4 bm = div_by_workers<W_>(tree.b[0], W);
      st_stream(p.Bs + off, bm);
      if (PRE && STEP) {
        // first step of the next period: every replica starts from the mean, t' = 1
        r = step_size(bm, q, eta_t);
#pragma unroll kOuterUnroll
        for (uint32_t i = 0; i < W; ++i) {
          float4 xv = xm, bv = bm;
          const float4 g = gradient4<GM, BF16>(p, in, xv, kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
          apply4(r, g, xv, bv);
          st_stream(p.X + (uint64_t)i * p.stride + off, xv);
          st_stream(p.B2 + (uint64_t)i * p.stride + off, bv);
        }
      } else {
#pragma unroll kOuterUnroll
        for (uint32_t i = 0; i < W; ++i) {
          st_stream(p.X + (uint64_t)i * p.stride + off, xm);
          st_stream(p.B2 + (uint64_t)i * p.stride + off, bm);
        }
      }
    }
    if (!has_next) break;
    grp = next_grp;
  }
}

// Host-side launcher table entry.
using SweepFn = void (*)(const SweepParams);
SweepFn lookup_sweep(int W, int gm, bool bf16, bool pre, bool step, bool post);

}  // namespace la
