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
// and, when the workers are spread over several GPUs, the same passes cut at the exchange:
//   XCH = 1 (export)     the adjacent-pair tree SUMS over the local replicas go to the exchange
//                        buffer instead of the means going back to the replicas
//                        (PRE: export of the stored replicas; STEP+POST: of this step's y, A^2)
//   XCH = 2 (import)     the read side is the exchange buffer holding the totals over all ranks
//                        (one "replica" of sums); means = totals / W_total go to every local replica
//                        (PRE: plain import; PRE+STEP: import and the first step of the next period)
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include <type_traits>

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

// Checked build (compile with -DLA_DEBUG; a separate library, never the one that is timed).
// compute-sanitizer's job, done by the kernels themselves: every global access is tested against
// the byte ranges the pass may touch, and the running row pointers against the closed form
// base + (replica * stride + coordinate) * 4.  A violation is counted in a status word that the
// host reads at the next synchronising call; the offending access is skipped (loads give 0), so a
// wrong address is reported, never dereferenced.  Nothing traps or asserts.
struct DebugRanges {
  uint64_t lo[3], hi[3];       // state arena, caller's gradient table, exchange buffer (hi exclusive; 0,0 = absent)
  unsigned long long* status;  // device: [0] violations, [1] first offending address, [2] its kind | bytes << 8
};                             //         kind 1 = outside every range, 2 = not the row it should be
#ifdef LA_DEBUG
#define LA_DBG_ARG(...) , __VA_ARGS__
__device__ __forceinline__ DebugRanges& dbg_ranges() {
  __shared__ DebugRanges r;
  return r;
}
__device__ __forceinline__ void dbg_begin(const DebugRanges& from_params) {
  if (threadIdx.x == 0) dbg_ranges() = from_params;
  __syncthreads();
}
static __device__ __noinline__ void dbg_report(uint64_t addr, unsigned long long kind) {
  unsigned long long* st = dbg_ranges().status;
  if (atomicAdd(st, 1ull) == 0ull) {
    st[1] = addr;
    st[2] = kind;
  }
}
__device__ __forceinline__ bool dbg_access_ok(const void* ptr, uint32_t bytes) {
  const DebugRanges& r = dbg_ranges();
  if (r.status == nullptr) return true;  // unchecked launch (no context behind it)
  const uint64_t a = reinterpret_cast<uint64_t>(ptr);
  bool ok = false;
#pragma unroll
  for (int k = 0; k < 3; ++k) ok = ok || (a >= r.lo[k] && a + bytes <= r.hi[k]);
  if (!ok) dbg_report(a, 1ull | ((unsigned long long)bytes << 8));
  return ok;
}
__device__ __forceinline__ void dbg_expect_row(uint64_t addr, uint64_t expected) {
  if (dbg_ranges().status != nullptr && addr != expected) dbg_report(addr, 2ull);
}
#else
#define LA_DBG_ARG(...)
#endif

struct SweepParams {
#ifdef LA_DEBUG
  DebugRanges dbg;
#endif
  float* X;        // [W][stride]
  float* B2;       // [W][stride]
  float* Bs;       // [stride]   accumulator as of the last synchronisation
  const float* a;  // [stride] or null
  const float* c;  // [stride] or null
  const float* s;  // [stride] or null
  const void* gext;    // external gradients, [W][N]
  uint32_t gext_vec;   // 1: every row of gext is aligned for V-wide loads (N % V == 0, aligned base)
  uint64_t n;          // logical coordinates N
  uint64_t stride;     // replica stride in floats (multiple of 64, >= N rounded up to 4)
  uint64_t j_base;     // global index of coordinate 0 (multiple of 4)
  uint64_t seed;
  uint64_t t;          // 1-based global step index of the STEP part ...
  const uint64_t* t_dev;  // ... plus *t_dev when non-null: a device-resident step counter, so that a
                          // captured CUDA graph of one period can be replayed without new arguments
  uint32_t W;
  uint32_t tp;         // t' of the STEP part (local steps since the last sync, incl. this one)
  uint32_t warm_up_steps;
  uint32_t identical_workers;
  uint32_t worker_base;  // global index of local replica 0 (sharding by worker); keys use worker_base + i
  float eta, eps, sigma;
  float* xch;            // XCH kernels only: where the sums of x over the replicas go to / come from ...
  uint64_t xch_b_off;    // ... and, this many floats further, the sums of B^2 (an exchange buffer [2][stride]
                         // has them one stride apart; replica 0's own rows, W strides)
  uint32_t W_total;      // workers over all ranks; divisor of the imported totals
};

__device__ __forceinline__ uint64_t step_index(const SweepParams& p) {
  return p.t + (p.t_dev != nullptr ? *p.t_dev : 0ull);
}

constexpr int kMaxWorkers = 64;
constexpr int kTreeDepth = 7;  // log2(kMaxWorkers) + 1 partial sums

#ifndef LA_BLOCK
#define LA_BLOCK 256
#endif
#ifndef LA_CH
#define LA_CH 4
#endif
#ifndef LA_CH_V4
#define LA_CH_V4 1
#endif
#ifndef LA_CH_V4_STEP  // ... but two for the plain local step, whose stores would otherwise keep the next loads
#define LA_CH_V4_STEP (LA_CH_V4 < 2 ? 2 : LA_CH_V4)  // from being issued early (bf16 table, W = 4 / 8: 0.94 / 0.95 against 0.89)
#endif
#ifndef LA_WRITE_CH_V4
#define LA_WRITE_CH_V4 2  // table rows fetched ahead by a four-coordinate step that follows an average
                          // (bf16 table, one-copy step at W = 4 / 8 / 16: 1 row 0.92 / 0.94 / 0.95 of the copy
                          // bandwidth, 2 rows 0.94 / 0.95 / 0.95, 4 rows the same)
#endif
constexpr int kBlockThreads = LA_BLOCK;

// V consecutive coordinates held by one thread (V = 4: one 128-bit access, two Box-Muller
// pairs; V = 2: one 64-bit access, one pair).
template <int V>
struct Vec {
  float v[V];
};

// Row addresses are carried as running 64-bit byte addresses that advance by one replica stride
// per worker.  The advance is an opaque add so that the compiler keeps ONE running pointer
// instead of hoisting a separate loop-invariant row base per worker out of the grid-stride loop
// (2W 64-bit bases = up to 64 registers, which would halve the occupancy).
__device__ __forceinline__ void advance(uint64_t& addr, uint64_t bytes) {
  asm volatile("add.u64 %0, %0, %1;" : "+l"(addr) : "l"(bytes));
}
__device__ __forceinline__ const float* as_ptr(uint64_t addr) { return reinterpret_cast<const float*>(addr); }
__device__ __forceinline__ float* as_mut(uint64_t addr) { return reinterpret_cast<float*>(addr); }

template <int V>
__device__ __forceinline__ Vec<V> ld_stream(const float* p) {
  Vec<V> r;
#ifdef LA_DEBUG
  if (!dbg_access_ok(p, V * sizeof(float))) {
#pragma unroll
    for (int k = 0; k < V; ++k) r.v[k] = 0.0f;
    return r;
  }
#endif
  if (V == 4) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    r.v[0] = t.x; r.v[1] = t.y; r.v[V - 2] = t.z; r.v[V - 1] = t.w;
  } else {
    const float2 t = __ldcs(reinterpret_cast<const float2*>(p));
    r.v[0] = t.x; r.v[1] = t.y;
  }
  return r;
}

template <int V>
__device__ __forceinline__ void st_stream(float* p, const Vec<V>& a) {
#ifdef LA_DEBUG
  if (!dbg_access_ok(p, V * sizeof(float))) return;
#endif
  if (V == 4) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(a.v[0], a.v[1], a.v[V - 2], a.v[V - 1]));
  } else {
    __stcs(reinterpret_cast<float2*>(p), make_float2(a.v[0], a.v[1]));
  }
}

template <int V>
__device__ __forceinline__ Vec<V> splat(float f) {
  Vec<V> r;
#pragma unroll
  for (int k = 0; k < V; ++k) r.v[k] = f;
  return r;
}

template <int V>
__device__ __forceinline__ Vec<V> add(const Vec<V>& l, const Vec<V>& r) {
  Vec<V> o;
#pragma unroll
  for (int k = 0; k < V; ++k) o.v[k] = __fadd_rn(l.v[k], r.v[k]);
  return o;
}

// Mean over workers = adjacent-pair tree sum, then one division by (float)W.  For a power of
// two the division is replaced by the multiplication with the exact reciprocal, which rounds
// the same real number and therefore gives the same bits.
template <int W_, int V>
__device__ __forceinline__ Vec<V> div_by_workers(const Vec<V>& a, uint32_t W) {
  Vec<V> o;
  if (W_ > 0 && (W_ & (W_ - 1)) == 0) {
    const float inv = 1.0f / (float)W_;
#pragma unroll
    for (int k = 0; k < V; ++k) o.v[k] = __fmul_rn(a.v[k], inv);
  } else {
    const float w = __uint2float_rn(W);
#pragma unroll
    for (int k = 0; k < V; ++k) o.v[k] = __fdiv_rn(a.v[k], w);
  }
  return o;
}

// Streaming form of the adjacent-pair tree: a stack of partial sums, one per level, merged
// like the carries of a binary counter.  After pushing worker i the two top entries are
// merged once for every trailing zero bit of (i+1); left operand = older entry.  With W known
// at compile time the loop unrolls and every stack index is a constant (registers only).
// ACC = false drops the accumulator component (Local SGD averages x only; AdaGrad averages
// gradients).
template <int V, bool ACC = true>
struct PairTree {
  Vec<V> x[kTreeDepth], b[ACC ? kTreeDepth : 1];
  // Before worker i is pushed the stack holds one entry per set bit of i, so every position
  // follows from i alone (no running stack pointer to carry through the unrolled code): the new
  // entry goes to slot popcount(i) and is merged downwards once per trailing one bit of i.
  __device__ __forceinline__ void push(uint32_t i, const Vec<V>& vx, const Vec<V>& vb) {
    const int top = __popc(i);
    const int merges = __popc(i & ~(i + 1u));
    x[top] = vx;
    if (ACC) b[ACC ? top : 0] = vb;
#pragma unroll
    for (int m = 0; m < kTreeDepth - 1; ++m)
      if (m < merges) {
        x[top - 1 - m] = add(x[top - 1 - m], x[top - m]);
        if (ACC) b[ACC ? top - 1 - m : 0] = add(b[ACC ? top - 1 - m : 0], b[ACC ? top - m : 0]);
      }
  }
  // position k within a chunk of replicas is irrelevant here (see PairTreeDyn)
  __device__ __forceinline__ void push_in_chunk(uint32_t i, int, bool, const Vec<V>& vx, const Vec<V>& vb) {
    push(i, vx, vb);
  }
  // After n pushes: merge what is left, older entries on the left; the total ends in slot 0.
  __device__ __forceinline__ void finish(uint32_t n) {
    const int sp = __popc(n);
#pragma unroll
    for (int m = 0; m < kTreeDepth - 1; ++m)
      if (m < sp - 1) {
        x[sp - 2 - m] = add(x[sp - 2 - m], x[sp - 1 - m]);
        if (ACC) b[ACC ? sp - 2 - m : 0] = add(b[ACC ? sp - 2 - m : 0], b[ACC ? sp - 1 - m : 0]);
      }
  }
};

// The same tree when the number of workers is only known at run time.  One slot per level, like
// the digits of a binary counter: pushing worker number n walks up the levels, merging (older
// partial sum on the left) while bit L of n is set and parking the carry in the first clear
// level.  Every slot index is a compile-time constant (the run-time part is predication), so the
// partial sums stay in registers; a stack with a run-time top would live in local memory.
template <int V, bool ACC = true>
struct PairTreeDyn {
  Vec<V> x[kTreeDepth], b[ACC ? kTreeDepth : 1];
  uint32_t n = 0;
  __device__ __forceinline__ void push(uint32_t, const Vec<V>& vx, const Vec<V>& vb) {
    Vec<V> cx = vx, cb = vb;
    bool placed = false;
#pragma unroll
    for (int L = 0; L < kTreeDepth; ++L) {
      if (!placed) {
        if ((n >> L) & 1u) {
          cx = add(x[L], cx);
          if (ACC) cb = add(b[ACC ? L : 0], cb);
        } else {
          x[L] = cx;
          if (ACC) b[ACC ? L : 0] = cb;
          placed = true;
        }
      }
    }
    ++n;
  }
  // Push of a partial sum that already covers 2^LOG consecutive workers starting at a multiple
  // of 2^LOG: the walk up the levels simply starts at level LOG.
  template <int LOG>
  __device__ __forceinline__ void push_block(const Vec<V>& vx, const Vec<V>& vb) {
    Vec<V> cx = vx, cb = vb;
    bool placed = false;
#pragma unroll
    for (int L = LOG; L < kTreeDepth; ++L) {
      if (!placed) {
        if ((n >> L) & 1u) {
          cx = add(x[L], cx);
          if (ACC) cb = add(b[ACC ? L : 0], cb);
        } else {
          x[L] = cx;
          if (ACC) b[ACC ? L : 0] = cb;
          placed = true;
        }
      }
    }
    n += 1u << LOG;
  }
  // Replica i = i0 + k of a chunk of four that starts at a multiple of four.  When the chunk is
  // complete its members are first summed as (v0 + v1) + (v2 + v3) — the bottom two levels of
  // the same tree — with compile-time positions, and enter the counter as one block: a quarter
  // of the run-time level walks.
  __device__ __forceinline__ void push_in_chunk(uint32_t i, int k, bool chunk_complete, const Vec<V>& vx,
                                                const Vec<V>& vb) {
    if (!chunk_complete) {
      push(i, vx, vb);
    } else if (k == 0) {
      px0 = vx; pb0 = vb;
    } else if (k == 1) {
      px0 = add(px0, vx);
      if (ACC) pb0 = add(pb0, vb);
    } else if (k == 2) {
      px1 = vx; pb1 = vb;
    } else {
      px1 = add(px1, vx);
      if (ACC) pb1 = add(pb1, vb);
      push_block<2>(add(px0, px1), ACC ? add(pb0, pb1) : pb0);
    }
  }
  Vec<V> px0, px1, pb0, pb1;

  // Leaves the total in x[0], b[0]: the occupied levels are merged from the lowest up, each
  // higher (older) level on the left.
  __device__ __forceinline__ void finish(uint32_t) {
    Vec<V> ax = x[0], ab = b[0];
    bool have = false;
#pragma unroll
    for (int L = 0; L < kTreeDepth; ++L) {
      if ((n >> L) & 1u) {
        if (have) {
          ax = add(x[L], ax);
          if (ACC) ab = add(b[ACC ? L : 0], ab);
        } else {
          ax = x[L];
          if (ACC) ab = b[ACC ? L : 0];
          have = true;
        }
      }
    }
    x[0] = ax;
    if (ACC) b[0] = ab;
  }
};

// Static worker count: the stack form (constant indices after unrolling); otherwise the counter form.
template <int W_, int V, bool ACC = true>
struct TreeFor {
  using type = typename std::conditional<(W_ > 0), PairTree<V, ACC>, PairTreeDyn<V, ACC>>::type;
};

// Worker-independent data of one coordinate group: the stale accumulator and the problem arrays.
template <int V>
struct CoordInputs {
  Vec<V> bs, a, c, s;
};

template <int GM, bool STEP, bool LOAD_BS, int V>
__device__ __forceinline__ void load_coord(CoordInputs<V>& in, const SweepParams& p, uint64_t off) {
  if (LOAD_BS) in.bs = ld_stream<V>(p.Bs + off);
  if (STEP) {
    if (GM == kGradQuadratic) {
      in.a = ld_stream<V>(p.a + off);
      in.c = ld_stream<V>(p.c + off);
    }
    if (GM == kGradNoiseScaled) in.s = ld_stream<V>(p.s + off);
    if (GM == kGradConstant) in.s = p.s ? ld_stream<V>(p.s + off) : splat<V>(1.0f);
  }
}

// x and B^2 of CH consecutive replicas for one coordinate group.
template <int V, int CH>
struct ReplicaChunk {
  Vec<V> x[CH], b[CH];
};

// Loads replicas i0 .. i0+CH-1; `addr` is the address of x of replica i0 for this coordinate
// group and is left pointing at replica i0+CH.  B^2 of a replica sits `b_delta` bytes after x.
template <int V, int CH, bool ACC = true>
__device__ __forceinline__ void load_chunk(ReplicaChunk<V, CH>& ch, uint64_t& addr, uint64_t b_delta,
                                           uint64_t stride_bytes, uint32_t W, uint32_t i0
                                           LA_DBG_ARG(uint64_t row0_addr)) {  // checked build: address of replica 0
#pragma unroll
  for (int k = 0; k < CH; ++k)
    if (i0 + k < W) {
#ifdef LA_DEBUG
      dbg_expect_row(addr, row0_addr + (uint64_t)(i0 + k) * stride_bytes);
#endif
      ch.x[k] = ld_stream<V>(as_ptr(addr));
      if (ACC) ch.b[k] = ld_stream<V>(as_ptr(addr + b_delta));
      advance(addr, stride_bytes);
    }
}

// Stores x and B^2 of one replica at `addr` and advances to the next replica.
template <int V, bool ACC = true>
__device__ __forceinline__ void store_replica(uint64_t& addr, uint64_t b_delta, uint64_t stride_bytes,
                                              const Vec<V>& x, const Vec<V>& b
                                              LA_DBG_ARG(uint64_t expected_addr)) {
#ifdef LA_DEBUG
  dbg_expect_row(addr, expected_addr);
#endif
  st_stream<V>(as_mut(addr), x);
  if (ACC) st_stream<V>(as_mut(addr + b_delta), b);
  advance(addr, stride_bytes);
}

// Caller-supplied gradients of CH consecutive replicas for one coordinate group (fp32 or bf16
// table [W][N], worker-major), fetched together with the replicas so that they are in flight
// while the previous chunk is consumed.
template <int V, int CH>
struct GradChunk {
  Vec<V> g[CH];  // fp32 table: the values; bf16 table: the V/2 loaded words in slots 0 .. V/2-1, widened on use
};

// The gradient values of one row of a chunk.  A bf16 row stays in the packed form it was loaded in
// until it is used, so that no instruction between a load and its use waits for the data (and a
// chunk fetched ahead costs half the registers); widening bf16 -> fp32 is exact.
template <int GM, int V>
__device__ __forceinline__ Vec<V> unpack_grads(const Vec<V>& raw) {
  if (GM != kGradExternalBF16) return raw;
  Vec<V> g;
#pragma unroll
  for (int k = 0; k < V; k += 2) {
    const uint32_t w = __float_as_uint(raw.v[k / 2]);
    g.v[k] = __uint_as_float(w << 16);
    g.v[k + 1] = __uint_as_float(w & 0xFFFF0000u);
  }
  return g;
}

template <int GM, int V, int CH>
__device__ __forceinline__ void load_grads(GradChunk<V, CH>& gc, const SweepParams& p, uint64_t& g_addr,
                                           uint64_t row_bytes, uint32_t W, uint32_t i0, uint64_t off) {
  constexpr bool kF32 = (GM == kGradExternalF32);
  [[maybe_unused]] constexpr uint32_t kElem = kF32 ? 4u : 2u;
#pragma unroll
  for (int k = 0; k < CH; ++k)
    if (i0 + k < W) {
#ifdef LA_DEBUG
      dbg_expect_row(g_addr, reinterpret_cast<uint64_t>(p.gext) + (uint64_t)(i0 + k) * row_bytes + off * kElem);
#endif
      if (p.gext_vec) {
#ifdef LA_DEBUG
        if (!dbg_access_ok(reinterpret_cast<const void*>(g_addr), V * kElem)) {
          gc.g[k] = splat<V>(0.0f);
        } else
#endif
        if (kF32) {
          gc.g[k] = ld_stream<V>(as_ptr(g_addr));
        } else {
          // V bf16 values in one 32- or 64-bit load, kept packed (see unpack_grads)
          gc.g[k] = splat<V>(0.0f);
          if (V == 2) {
            gc.g[k].v[0] = __uint_as_float(__ldcs(reinterpret_cast<const uint32_t*>(g_addr)));
          } else {
            const uint2 w = __ldcs(reinterpret_cast<const uint2*>(g_addr));
            gc.g[k].v[0] = __uint_as_float(w.x);
            gc.g[k].v[1] = __uint_as_float(w.y);
          }
        }
      } else {
        if (!kF32) gc.g[k] = splat<V>(0.0f);
#pragma unroll
        for (int e = 0; e < V; ++e) {
          bool take = off + e < p.n;
#ifdef LA_DEBUG
          take = take && dbg_access_ok(reinterpret_cast<const void*>(g_addr + e * kElem), kElem);
#endif
          if (kF32) {
            gc.g[k].v[e] = take ? __ldcs(reinterpret_cast<const float*>(g_addr) + e) : 0.0f;
          } else {  // element by element into the packed form
            const uint32_t h = take ? (uint32_t)__ldcs(reinterpret_cast<const unsigned short*>(g_addr) + e) : 0u;
            gc.g[k].v[e / 2] = __uint_as_float(__float_as_uint(gc.g[k].v[e / 2]) | (h << (16 * (e & 1))));
          }
        }
      }
      advance(g_addr, row_bytes);
    }
}

// r = eta_t / sqrt(B^2_{t-t'} + t' eps^2): the step size all workers share (Section 4.2).
template <int V>
__device__ __forceinline__ Vec<V> step_size(const Vec<V>& bs, float q, float eta_t) {
  Vec<V> r;
#pragma unroll
  for (int k = 0; k < V; ++k) r.v[k] = __fdiv_rn(eta_t, __fsqrt_rn(__fadd_rn(bs.v[k], q)));
  return r;
}

// Gradient of V coordinates for one worker.  `xv` is the worker's own iterate
// (Algorithm 3: G_{i,t} = grad f(x_{i,t-1}; z_{i,t})).  `ctr0` = gamma (p0 + 1) for the
// group's first coordinate pair p0.
template <int GM, bool BF16, int V>
__device__ __forceinline__ Vec<V> gradient(const SweepParams& p, const CoordInputs<V>& in, const Vec<V>& xv,
                                           uint64_t key, uint64_t ctr0, uint32_t worker, uint64_t off) {
  Vec<V> g;
  if (GM == kGradConstant) {
    return in.s;
  } else {
    Vec<V> xi;
#pragma unroll
    for (int k = 0; k < V; k += 2) normal_pair(key, ctr0 + kGoldenGamma * (uint64_t)(k / 2), xi.v[k], xi.v[k + 1]);
#pragma unroll
    for (int k = 0; k < V; ++k) {
      if (GM == kGradNoise) {
        g.v[k] = xi.v[k];
      } else if (GM == kGradNoiseScaled) {
        g.v[k] = __fmul_rn(in.s.v[k], xi.v[k]);
      } else {  // quadratic
        g.v[k] = __fmaf_rn(in.a.v[k], __fsub_rn(xv.v[k], in.c.v[k]), __fmul_rn(p.sigma, xi.v[k]));
      }
    }
    if (BF16) {
#pragma unroll
      for (int k = 0; k < V; k += 2) round_pair_through_bf16(g.v[k], g.v[k + 1]);
    }
  }
  return g;
}

// y = x - r g ; A^2 = B^2 + g g   (Algorithm 3), one fused multiply-add each.
template <int V, bool ACC = true>
__device__ __forceinline__ void apply(const Vec<V>& r, const Vec<V>& g, Vec<V>& x, Vec<V>& b) {
#pragma unroll
  for (int k = 0; k < V; ++k) {
    x.v[k] = __fmaf_rn(-r.v[k], g.v[k], x.v[k]);
    if (ACC) b.v[k] = __fmaf_rn(g.v[k], g.v[k], b.v[k]);
  }
}

// ACC = true: Algorithm 3 (Local AdaAlter).  ACC = false: Algorithm 2 (Local SGD) — the same sweep
// without accumulators: y = x - eta_t G, and the synchronisation averages x only.
template <int W_, int V, int GM, bool BF16, bool PRE, bool STEP, bool POST, int MINB, bool ACC = true, int XCH = 0>
__global__ void __launch_bounds__(LA_BLOCK, MINB) la_sweep(const SweepParams p) {
  static_assert(!(PRE && POST), "one synchronisation per pass");
  static_assert(V == 2 || V == 4, "a thread owns 2 or 4 coordinates");
  static_assert(XCH == 0 || ACC, "the exchange carries x and B^2: Local AdaAlter only");
  static_assert(XCH != 1 || POST || (PRE && !STEP), "export: sums of a step's results or of the stored replicas");
  static_assert(XCH != 2 || PRE, "import: the averaged state is what the pass starts from");
  constexpr bool kExport = (XCH == 1), kImport = (XCH == 2);
  constexpr bool kNeedsNoise = STEP && (GM == kGradNoise || GM == kGradNoiseScaled || GM == kGradQuadratic);
  constexpr int WR_ = kImport ? 1 : W_;  // replicas on the READ side (import: the one row of totals)
  // replicas loaded before any is consumed (four-coordinate threads hold twice the data per replica)
  constexpr int kChunkMax = (V == 4) ? ((PRE || POST) ? LA_CH_V4 : LA_CH_V4_STEP) : LA_CH;
  constexpr int CH = (WR_ > 0) ? (WR_ < kChunkMax ? WR_ : kChunkMax) : 4;
  constexpr int kReadUnroll = (WR_ > 0) ? kMaxWorkers : 1;  // static counts: unroll fully, so that the
  constexpr int kWriteUnroll = (W_ > 0) ? kMaxWorkers : 4;  // reduction stack is indexed by constants; run-time
                                                            // counts: four gradient chains in flight
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;
  const uint32_t Wr = kImport ? 1u : W;

#ifdef LA_DEBUG
  dbg_begin(p.dbg);
#endif
  __shared__ uint64_t keys[kMaxWorkers];
  if (kNeedsNoise) {
    if (threadIdx.x < W) keys[threadIdx.x] = step_worker_key(p.seed, step_index(p), p.identical_workers ? 0u : p.worker_base + threadIdx.x);
    __syncthreads();
  }

  // per-step scalars (worker- and coordinate-independent)
  float q = 0.f, eta_t = 0.f;
  if (STEP) {
    const float eps2 = __fmul_rn(p.eps, p.eps);
    q = __fmul_rn(__uint2float_rn(p.tp), eps2);  // t' eps^2, the placeholder of Section 4.2
    eta_t = p.eta;
    if (p.warm_up_steps != 0u) {  // Section 6.2: eta_t = eta min(1, t / warm_up_steps)
      const float ratio = __fdiv_rn(__ull2float_rn(step_index(p)), __uint2float_rn(p.warm_up_steps));
      eta_t = __fmul_rn(p.eta, fminf(1.0f, ratio));
    }
  }

  // Grid-stride loop over coordinate groups, software-pipelined: while the replicas of one
  // chunk are being consumed, the loads of the next chunk (or of the next group's first chunk
  // and worker-independent data) are already in flight.  The empty asm statements pin that
  // order against the compiler's scheduler.
  const uint64_t ngroups = (p.n + (uint64_t)(V - 1)) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (grp >= ngroups) return;
  constexpr bool kLoadsBs = STEP && !PRE && ACC;

  const uint64_t x_base = reinterpret_cast<uint64_t>(p.X);
  const uint64_t b_delta = reinterpret_cast<uint64_t>(p.B2) - x_base;
  const uint64_t stride_bytes = p.stride * sizeof(float);
  // read side: the replicas, or (import) the sums seen as one replica whose "B^2" sits
  // xch_b_off floats after its "x"
  const uint64_t rd_base = kImport ? reinterpret_cast<uint64_t>(p.xch) : x_base;
  const uint64_t rd_b_delta = kImport ? p.xch_b_off * sizeof(float) : b_delta;

  constexpr bool kSupplied = STEP && (GM == kGradExternalF32 || GM == kGradExternalBF16);
  constexpr bool kExternal = kSupplied && !PRE;  // table rows fetched in the replica pipeline; a step that follows an
                                                 // average (PRE) fetches them in its write loop instead
  constexpr uint64_t kGradElem = (GM == kGradExternalBF16) ? 2 : 4;
  const uint64_t g_base = reinterpret_cast<uint64_t>(p.gext);
  const uint64_t g_row_bytes = p.n * kGradElem;

  // Static worker counts: one buffer of loads in flight (`nxt`), copied when consumed — the chunk
  // loop is fully unrolled, so the copies are register renaming.  Run-time worker counts: the loop
  // stays rolled, a copy would wait for the data BEFORE the next loads are issued, so there are
  // two buffers with compile-time roles (`rb[0]`, `rb[1]`: slots of even and odd position).
  ReplicaChunk<V, CH> nxt, rb[(WR_ > 0) ? 1 : 2];
  GradChunk<V, kExternal ? CH : 1> gnxt, gb[(WR_ > 0) ? 1 : 2];
  CoordInputs<V> in_next;
  load_coord<GM, STEP, kLoadsBs, V>(in_next, p, grp * V);
  uint64_t ld_addr = rd_base + grp * (V * sizeof(float));
  uint64_t g_addr = g_base + grp * (V * kGradElem);
  load_chunk<V, CH, ACC>((WR_ > 0) ? nxt : rb[0], ld_addr, rd_b_delta, stride_bytes, Wr, 0u
                         LA_DBG_ARG(rd_base + grp * (V * sizeof(float))));
  if (kExternal)
    load_grads<GM, V, kExternal ? CH : 1>((WR_ > 0) ? gnxt : gb[0], p, g_addr, g_row_bytes, W, 0u, grp * V);

  // A step that follows an average takes supplied gradients in its write loop, kWriteChunk table rows ahead.
  constexpr bool kSuppliedAfterAverage = kSupplied && PRE;
  constexpr int kWriteChunk = (V == 4) ? LA_WRITE_CH_V4 : 4;
  GradChunk<V, kSuppliedAfterAverage ? kWriteChunk : 1> gw_next;
  uint64_t gw_addr = g_base + grp * (V * kGradElem);
  if (kSuppliedAfterAverage)
    load_grads<GM, V, kSuppliedAfterAverage ? kWriteChunk : 1>(gw_next, p, gw_addr, g_row_bytes, W, 0u, grp * V);

  for (;;) {
    const uint64_t off = grp * V;
    const uint64_t next_grp = grp + nthreads;
    const bool has_next = next_grp < ngroups;
    const CoordInputs<V> in = in_next;
    const uint64_t ctr0 = kGoldenGamma * (((p.j_base + off) >> 1) + 1u);
    uint64_t st_addr = x_base + off * sizeof(float);

    Vec<V> r;
    if (kLoadsBs) r = step_size<V>(in.bs, q, eta_t);
    if (!ACC) r = splat<V>(eta_t);
    typename TreeFor<WR_, V, ACC>::type tree;

    // One chunk of CH replicas starting at replica i0: start the loads of what comes next, then
    // consume the chunk.  `tr` is the reduction the chunk's results enter, `local0` the index of
    // the chunk's first replica as that reduction counts it, `whole` whether all CH replicas exist.
    auto chunk = [&](const uint32_t i0, auto& tr, const uint32_t local0, const bool whole) __attribute__((always_inline)) {
      ReplicaChunk<V, CH> cur = nxt;
      GradChunk<V, kExternal ? CH : 1> gcur = gnxt;
      if (i0 + CH < Wr) {
        load_chunk<V, CH, ACC>(nxt, ld_addr, rd_b_delta, stride_bytes, Wr, i0 + CH LA_DBG_ARG(rd_base + off * sizeof(float)));
        if (kExternal) load_grads<GM, V, kExternal ? CH : 1>(gnxt, p, g_addr, g_row_bytes, W, i0 + CH, off);
      } else if (has_next) {
        load_coord<GM, STEP, kLoadsBs, V>(in_next, p, next_grp * V);
        ld_addr = rd_base + next_grp * (V * sizeof(float));
        load_chunk<V, CH, ACC>(nxt, ld_addr, rd_b_delta, stride_bytes, Wr, 0u LA_DBG_ARG(rd_base + next_grp * (V * sizeof(float))));
        if (kExternal) {
          g_addr = g_base + next_grp * (V * kGradElem);
          load_grads<GM, V, kExternal ? CH : 1>(gnxt, p, g_addr, g_row_bytes, W, 0u, next_grp * V);
        }
      }
      asm volatile("" ::: "memory");
#pragma unroll
      for (int k = 0; k < CH; ++k)
        if (whole || i0 + k < Wr) {
          const uint32_t i = i0 + k;
          if (PRE) {
            tr.push_in_chunk(local0 + k, k, whole, cur.x[k], cur.b[k]);
          } else {
            const Vec<V> g = kExternal ? unpack_grads<GM, V>(gcur.g[kExternal ? k : 0])
                                       : gradient<GM, BF16, V>(p, in, cur.x[k], kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
            apply<V, ACC>(r, g, cur.x[k], cur.b[k]);
            if (POST) {
              tr.push_in_chunk(local0 + k, k, whole, cur.x[k], cur.b[k]);
            } else {
              store_replica<V, ACC>(st_addr, b_delta, stride_bytes, cur.x[k], cur.b[k]
                                    LA_DBG_ARG(x_base + off * sizeof(float) + (uint64_t)i * stride_bytes));
            }
          }
        }
    };

    if constexpr (WR_ > 0) {
#pragma unroll kReadUnroll
      for (uint32_t i0 = 0; i0 < Wr; i0 += CH) chunk(i0, tree, i0, i0 + CH <= Wr);
    } else {
      // Worker count known only at run time.  The replicas are consumed in SLOTS of CH, always an
      // even number of them per coordinate group, so that every slot has a compile-time position
      // (even: buffer 0, odd: buffer 1): a slot first starts the loads of the slot that follows
      // into the other buffer, then consumes its own.  Only the last (odd) slot of a group has
      // nothing after it in the group; it fetches the first chunk of the thread's next group.
      auto slot = [&](auto position, const uint32_t i0, auto& tr, const uint32_t local0, const bool whole)
                      __attribute__((always_inline)) {
        constexpr int P = decltype(position)::value;
        ReplicaChunk<V, CH>& cur = rb[P];
        ReplicaChunk<V, CH>& ahead = rb[1 - P];
        GradChunk<V, kExternal ? CH : 1>& gcur = gb[P];
        GradChunk<V, kExternal ? CH : 1>& gahead = gb[1 - P];
        if (i0 + CH < Wr) {
          load_chunk<V, CH, ACC>(ahead, ld_addr, rd_b_delta, stride_bytes, Wr, i0 + CH LA_DBG_ARG(rd_base + off * sizeof(float)));
          if (kExternal) load_grads<GM, V, kExternal ? CH : 1>(gahead, p, g_addr, g_row_bytes, W, i0 + CH, off);
        } else if (P == 1 && has_next) {
          load_coord<GM, STEP, kLoadsBs, V>(in_next, p, next_grp * V);
          ld_addr = rd_base + next_grp * (V * sizeof(float));
          load_chunk<V, CH, ACC>(ahead, ld_addr, rd_b_delta, stride_bytes, Wr, 0u LA_DBG_ARG(rd_base + next_grp * (V * sizeof(float))));
          if (kExternal) {
            g_addr = g_base + next_grp * (V * kGradElem);
            load_grads<GM, V, kExternal ? CH : 1>(gahead, p, g_addr, g_row_bytes, W, 0u, next_grp * V);
          }
        }
        asm volatile("" ::: "memory");
#pragma unroll
        for (int k = 0; k < CH; ++k)
          if (whole || i0 + k < Wr) {
            const uint32_t i = i0 + k;
            if (PRE) {
              tr.push_in_chunk(local0 + k, k, whole, cur.x[k], cur.b[k]);
            } else {
              const Vec<V> g = kExternal ? unpack_grads<GM, V>(gcur.g[kExternal ? k : 0])
                                         : gradient<GM, BF16, V>(p, in, cur.x[k], kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
              apply<V, ACC>(r, g, cur.x[k], cur.b[k]);
              if (POST) {
                tr.push_in_chunk(local0 + k, k, whole, cur.x[k], cur.b[k]);
              } else {
                store_replica<V, ACC>(st_addr, b_delta, stride_bytes, cur.x[k], cur.b[k]
                                      LA_DBG_ARG(x_base + off * sizeof(float) + (uint64_t)i * stride_bytes));
              }
            }
          }
      };
      using Even = std::integral_constant<int, 0>;
      using Odd = std::integral_constant<int, 1>;
      // Passes that average first take whole tiles of kTile replicas: inside a tile every position
      // is a compile-time constant, so the tile is summed by the stack-form tree (constant register
      // indices, no predication) and enters the run-time counter as one aligned block — an aligned
      // block of 2^k workers is a complete subtree of the adjacent-pair tree.  What is left (fewer
      // than half a tile) goes through the counter in one last pair of slots.
      constexpr int kTile = 16, kTileLog = 4;
      static_assert(CH == 4, "tiles and half tiles are whole pairs of slots");
      uint32_t i0 = 0;
      if ((PRE || POST) && V == 2) {  // (four-coordinate threads have no registers to spare for a tile)
        for (; i0 + kTile <= Wr; i0 += kTile) {
          PairTree<V, ACC> tile;
          slot(Even{}, i0, tile, 0u, true);
          slot(Odd{}, i0 + CH, tile, (uint32_t)CH, true);
          slot(Even{}, i0 + 2 * CH, tile, (uint32_t)(2 * CH), true);
          slot(Odd{}, i0 + 3 * CH, tile, (uint32_t)(3 * CH), true);
          tile.finish(kTile);
          tree.template push_block<kTileLog>(tile.x[0], tile.b[0]);
        }
        if (i0 + kTile / 2 <= Wr) {  // one half tile, the same way
          PairTree<V, ACC> tile;
          slot(Even{}, i0, tile, 0u, true);
          slot(Odd{}, i0 + CH, tile, (uint32_t)CH, true);
          tile.finish(kTile / 2);
          tree.template push_block<kTileLog - 1>(tile.x[0], tile.b[0]);
          i0 += kTile / 2;
        }
      }
      // (a group that ended exactly on a tile has had its last odd slot; otherwise pairs of slots
      // until the replicas are used up — the odd slot of the last pair may be empty)
      for (; i0 < Wr; i0 += 2 * CH) {
        slot(Even{}, i0, tree, i0, i0 + CH <= Wr);
        slot(Odd{}, i0 + CH, tree, i0 + CH, i0 + 2 * CH <= Wr);
      }
    }

    if (PRE || POST) {
      tree.finish(Wr);
      if (kExport) {
        // the means are formed after the exchange, from the totals over all ranks
        st_stream<V>(p.xch + off, tree.x[0]);
        st_stream<V>(p.xch + p.xch_b_off + off, tree.b[0]);
      } else {
        // synchronisation branch of Algorithm 3: means over workers; the mean accumulator is
        // also the new stale denominator
        const Vec<V> xm = kImport ? div_by_workers<0, V>(tree.x[0], p.W_total) : div_by_workers<W_, V>(tree.x[0], W);
        Vec<V> bm = xm;
        if (ACC) {
          bm = kImport ? div_by_workers<0, V>(tree.b[0], p.W_total) : div_by_workers<W_, V>(tree.b[0], W);
          st_stream<V>(p.Bs + off, bm);
        }
        if (PRE && STEP) {
          // first step of the next period: every replica starts from the mean, t' = 1
          if (ACC) r = step_size<V>(bm, q, eta_t);
          if constexpr (kSuppliedAfterAverage) {
            // gradients from the caller's table, fetched a chunk of rows ahead (the last chunk of a
            // group already fetches the first rows of the next group)
#pragma unroll kWriteUnroll
            for (uint32_t i0 = 0; i0 < W; i0 += kWriteChunk) {
              const GradChunk<V, kWriteChunk> gcur = gw_next;
              if (i0 + kWriteChunk < W) {
                load_grads<GM, V, kWriteChunk>(gw_next, p, gw_addr, g_row_bytes, W, i0 + kWriteChunk, off);
              } else if (has_next) {
                gw_addr = g_base + next_grp * (V * kGradElem);
                load_grads<GM, V, kWriteChunk>(gw_next, p, gw_addr, g_row_bytes, W, 0u, next_grp * V);
              }
#pragma unroll
              for (int k = 0; k < kWriteChunk; ++k)
                if (i0 + k < W) {
                  Vec<V> xv = xm, bv = bm;
                  apply<V, ACC>(r, unpack_grads<GM, V>(gcur.g[k]), xv, bv);
                  store_replica<V, ACC>(st_addr, b_delta, stride_bytes, xv, bv
                                        LA_DBG_ARG(x_base + off * sizeof(float) + (uint64_t)(i0 + k) * stride_bytes));
                }
            }
          } else {
#pragma unroll kWriteUnroll
            for (uint32_t i = 0; i < W; ++i) {
              Vec<V> xv = xm, bv = bm;
              const Vec<V> g = gradient<GM, BF16, V>(p, in, xv, kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
              apply<V, ACC>(r, g, xv, bv);
              store_replica<V, ACC>(st_addr, b_delta, stride_bytes, xv, bv
                                    LA_DBG_ARG(x_base + off * sizeof(float) + (uint64_t)i * stride_bytes));
            }
          }
        } else {
#pragma unroll kWriteUnroll
          for (uint32_t i = 0; i < W; ++i)
            store_replica<V, ACC>(st_addr, b_delta, stride_bytes, xm, bm
                                  LA_DBG_ARG(x_base + off * sizeof(float) + (uint64_t)i * stride_bytes));
        }
      }
    }
    if (!has_next) break;
    grp = next_grp;
  }
}

// Algorithm 1 (Distributed AdaGrad), one iteration: every worker's gradient at the COMMON iterate,
// G_t = mean over workers (same adjacent-pair tree), B^2_t = B^2_{t-1} + G_t o G_t,
// x_t = x_{t-1} - eta_t G_t / sqrt(B^2_t + eps^2) with the UPDATED accumulator.  The iterate is
// shared by construction, so only replica 0 is kept; the accumulator is mirrored into Bs.
template <int W_, int V, int GM, int MINB>
__global__ void __launch_bounds__(LA_BLOCK, MINB) la_adagrad(const SweepParams p) {
  constexpr bool kNeedsNoise = (GM == kGradNoise || GM == kGradNoiseScaled || GM == kGradQuadratic);
  constexpr bool kExternal = (GM == kGradExternalF32 || GM == kGradExternalBF16);
  constexpr uint64_t kGradElem = (GM == kGradExternalBF16) ? 2 : 4;
  constexpr int kOuterUnroll = (W_ > 0) ? kMaxWorkers : 1;
  const uint32_t W = (W_ > 0) ? (uint32_t)W_ : p.W;
#ifdef LA_DEBUG
  dbg_begin(p.dbg);
#endif
  __shared__ uint64_t keys[kMaxWorkers];
  if (kNeedsNoise) {
    if (threadIdx.x < W) keys[threadIdx.x] = step_worker_key(p.seed, step_index(p), p.identical_workers ? 0u : p.worker_base + threadIdx.x);
    __syncthreads();
  }
  const float eps2 = __fmul_rn(p.eps, p.eps);
  float eta_t = p.eta;
  if (p.warm_up_steps != 0u) {
    const float ratio = __fdiv_rn(__ull2float_rn(step_index(p)), __uint2float_rn(p.warm_up_steps));
    eta_t = __fmul_rn(p.eta, fminf(1.0f, ratio));
  }
  const uint64_t ngroups = (p.n + (uint64_t)(V - 1)) / (uint64_t)V;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += nthreads) {
    const uint64_t off = grp * V;
    CoordInputs<V> in;
    load_coord<GM, true, false, V>(in, p, off);
    Vec<V> x = ld_stream<V>(p.X + off);
    Vec<V> b = ld_stream<V>(p.B2 + off);
    const uint64_t ctr0 = kGoldenGamma * (((p.j_base + off) >> 1) + 1u);
    typename TreeFor<W_, V, false>::type tree;
    uint64_t g_addr = reinterpret_cast<uint64_t>(p.gext) + off * kGradElem;  // supplied gradients, row by row
#pragma unroll kOuterUnroll
    for (uint32_t i = 0; i < W; ++i) {
      Vec<V> g;
      if (kExternal) {
        GradChunk<V, 1> gc;
        load_grads<GM, V, 1>(gc, p, g_addr, p.n * kGradElem, W, i, off);
        g = unpack_grads<GM, V>(gc.g[0]);
      } else {
        g = gradient<GM, false, V>(p, in, x, kNeedsNoise ? keys[i] : 0ull, ctr0, i, off);
      }
      tree.push(i, g, g);
    }
    tree.finish(W);
    const Vec<V> gm = div_by_workers<W_, V>(tree.x[0], W);
#pragma unroll
    for (int k = 0; k < V; ++k) {
      b.v[k] = __fmaf_rn(gm.v[k], gm.v[k], b.v[k]);
      const float r = __fdiv_rn(eta_t, __fsqrt_rn(__fadd_rn(b.v[k], eps2)));
      x.v[k] = __fmaf_rn(-r, gm.v[k], x.v[k]);
    }
    st_stream<V>(p.X + off, x);
    st_stream<V>(p.B2 + off, b);
    st_stream<V>(p.Bs + off, b);
  }
}

// Host-side launcher table entry: the kernel and the number of coordinates a thread owns.
using SweepFn = void (*)(const SweepParams);
struct SweepKernel {
  SweepFn fn;
  int vec;
};
// rule: 0 = Local AdaAlter, 1 = Local SGD, 2 = Distributed AdaGrad (one kernel per step)
// xch: 0 = single-GPU pass, 1 = export to / 2 = import from the exchange buffer (rule 0 only)
SweepKernel lookup_sweep(int W, int rule, int gm, bool bf16, bool pre, bool step, bool post, int xch = 0);

}  // namespace la
