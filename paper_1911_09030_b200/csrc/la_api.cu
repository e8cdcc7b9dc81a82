// C-ABI of the Local AdaAlter hot-path library: context, schedule (Algorithm 3's outer
// loop and its t / t' / sync bookkeeping), state upload/download and kernel dispatch.
// All arithmetic of the method lives in la_sweep.cuh; this file moves scalars and pointers.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/local_adaalter.h"
#include "la_exchange.cuh"
#include "la_period.cuh"
#include "la_sweep.cuh"

namespace la {

SweepKernel lookup_sweep_w0(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w1(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w2(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w4(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w8(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w16(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w3(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w6(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w12(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w32(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w64(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w5(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w7(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w9(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w10(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w11(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w13(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w14(int, int, bool, bool, bool, bool, int);
SweepKernel lookup_sweep_w15(int, int, bool, bool, bool, bool, int);

SweepKernel lookup_sweep(int W, int rule, int gm, bool bf16, bool pre, bool step, bool post, int xch) {
  switch (W) {
    case 1: return lookup_sweep_w1(rule, gm, bf16, pre, step, post, xch);
    case 2: return lookup_sweep_w2(rule, gm, bf16, pre, step, post, xch);
    case 4: return lookup_sweep_w4(rule, gm, bf16, pre, step, post, xch);
    case 8: return lookup_sweep_w8(rule, gm, bf16, pre, step, post, xch);
    case 16: return lookup_sweep_w16(rule, gm, bf16, pre, step, post, xch);
    case 3: return lookup_sweep_w3(rule, gm, bf16, pre, step, post, xch);
    case 6: return lookup_sweep_w6(rule, gm, bf16, pre, step, post, xch);
    case 12: return lookup_sweep_w12(rule, gm, bf16, pre, step, post, xch);
#ifndef LA_DEBUG   // the checked build keeps to the first set of instantiations; the rest runs as a run-time count
    case 32: return lookup_sweep_w32(rule, gm, bf16, pre, step, post, xch);
    case 64: return lookup_sweep_w64(rule, gm, bf16, pre, step, post, xch);
    case 5: return lookup_sweep_w5(rule, gm, bf16, pre, step, post, xch);
    case 7: return lookup_sweep_w7(rule, gm, bf16, pre, step, post, xch);
    case 9: return lookup_sweep_w9(rule, gm, bf16, pre, step, post, xch);
    case 10: return lookup_sweep_w10(rule, gm, bf16, pre, step, post, xch);
    case 11: return lookup_sweep_w11(rule, gm, bf16, pre, step, post, xch);
    case 13: return lookup_sweep_w13(rule, gm, bf16, pre, step, post, xch);
    case 14: return lookup_sweep_w14(rule, gm, bf16, pre, step, post, xch);
    case 15: return lookup_sweep_w15(rule, gm, bf16, pre, step, post, xch);
#endif
    default: return lookup_sweep_w0(rule, gm, bf16, pre, step, post, xch);
  }
}

// True for worker counts without an instantiation of their own.
bool lookup_sweep_is_runtime(int W) {
  switch (W) {
    case 1: case 2: case 3: case 4: case 6: case 8: case 12: case 16: return false;
#ifndef LA_DEBUG
    case 5: case 7: case 9: case 10: case 11: case 13: case 14: case 15: case 32: case 64: return false;
#endif
    default: return true;
  }
}

PeriodKernel lookup_period_w0(int, bool, bool);
PeriodKernel lookup_period_w1(int, bool, bool);
PeriodKernel lookup_period_w2(int, bool, bool);
PeriodKernel lookup_period_w4(int, bool, bool);
PeriodKernel lookup_period_w8(int, bool, bool);
PeriodKernel lookup_period_w16(int, bool, bool);
PeriodKernel lookup_period_w3(int, bool, bool);
PeriodKernel lookup_period_w6(int, bool, bool);
PeriodKernel lookup_period_w12(int, bool, bool);
PeriodKernel lookup_period_w32(int, bool, bool);
PeriodKernel lookup_period_w64(int, bool, bool);
PeriodKernel lookup_period_w5(int, bool, bool);
PeriodKernel lookup_period_w7(int, bool, bool);
PeriodKernel lookup_period_w9(int, bool, bool);
PeriodKernel lookup_period_w10(int, bool, bool);
PeriodKernel lookup_period_w11(int, bool, bool);
PeriodKernel lookup_period_w13(int, bool, bool);
PeriodKernel lookup_period_w14(int, bool, bool);
PeriodKernel lookup_period_w15(int, bool, bool);

PeriodKernel lookup_period(int W, int gm, bool bf16, bool post) {
  switch (W) {
    case 1: return lookup_period_w1(gm, bf16, post);
    case 2: return lookup_period_w2(gm, bf16, post);
    case 4: return lookup_period_w4(gm, bf16, post);
    case 8: return lookup_period_w8(gm, bf16, post);
    case 16: return lookup_period_w16(gm, bf16, post);
    case 3: return lookup_period_w3(gm, bf16, post);
    case 6: return lookup_period_w6(gm, bf16, post);
    case 12: return lookup_period_w12(gm, bf16, post);
#ifndef LA_DEBUG   // the checked build keeps to the first set of instantiations; the rest runs as a run-time count
    case 32: return lookup_period_w32(gm, bf16, post);
    case 64: return lookup_period_w64(gm, bf16, post);
    case 5: return lookup_period_w5(gm, bf16, post);
    case 7: return lookup_period_w7(gm, bf16, post);
    case 9: return lookup_period_w9(gm, bf16, post);
    case 10: return lookup_period_w10(gm, bf16, post);
    case 11: return lookup_period_w11(gm, bf16, post);
    case 13: return lookup_period_w13(gm, bf16, post);
    case 14: return lookup_period_w14(gm, bf16, post);
    case 15: return lookup_period_w15(gm, bf16, post);
#endif
    default: return lookup_period_w0(gm, bf16, post);
  }
}

constexpr int kExchangeVec = 2;  // coordinates per thread in the combine kernel

// Coordinates [0, count) of every replica: x0 (zeros from n on, or everywhere without x0), b0sq.
__global__ void la_fill(float* X, float* B2, float* Bs, const float* x0, float b0sq, uint64_t stride,
                        uint64_t n, uint64_t count, uint32_t W) {
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += nthreads) {
    const float v = (x0 != nullptr && j < n) ? x0[j] : 0.0f;
    for (uint32_t i = 0; i < W; ++i) {
      X[(uint64_t)i * stride + j] = v;
      B2[(uint64_t)i * stride + j] = b0sq;
    }
    Bs[j] = b0sq;
  }
}

// Copies replica 0's x and B^2 into replicas 1..W-1 (Algorithm 1 keeps one iterate that every
// worker holds; the AdaGrad kernel stores it once, and this materialises the other copies when
// a per-worker view is needed again).
__global__ void la_broadcast_replica0(float* X, float* B2, uint64_t stride, uint32_t W) {
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t nvec = stride / 4;  // stride is a multiple of 64 floats
  for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < nvec; j += nthreads) {
    const float4 x = reinterpret_cast<const float4*>(X)[j];
    const float4 b = reinterpret_cast<const float4*>(B2)[j];
    for (uint32_t i = 1; i < W; ++i) {
      reinterpret_cast<float4*>(X + (uint64_t)i * stride)[j] = x;
      reinterpret_cast<float4*>(B2 + (uint64_t)i * stride)[j] = b;
    }
  }
}

// The two building blocks of the noise source over their whole 24-bit domains, as the sweep
// kernels evaluate them: radius[k-1] = sqrt(-2 ln(k 2^-24)), k = 1..2^24; (cos, sin)(2 pi q 2^-24),
// q = 0..2^24-1.
__global__ void la_noise_tables_kernel(float* radius, float* cs, float* sn) {
  const uint32_t nthreads = gridDim.x * blockDim.x;
  for (uint32_t q = blockIdx.x * blockDim.x + threadIdx.x; q < (1u << 24); q += nthreads) {
    if (radius) radius[q] = radius_from_top24(q << 8);
    if (cs || sn) {
      float c, s;
      cossin_from_top24(q << 8, c, s);
      if (cs) cs[q] = c;
      if (sn) sn[q] = s;
    }
  }
}

// Device-resident step counter used by captured graphs (see la_set_graph).
__global__ void la_counter_set(uint64_t* ctr, uint64_t v) { *ctr = v; }
__global__ void la_counter_add(uint64_t* ctr, uint64_t v) { *ctr += v; }

// Diagnostics (off the hot path): with x-bar = mean over workers (plain left-to-right sum in
// double), out[0] += sum_j a_j (x-bar_j - c_j)^2 / 2  (the quadratic objective at the mean iterate,
// the quantity whose gradient norm Theorem 1 bounds) and out[1] += sum_i sum_j (x_ij - x-bar_j)^2 / W
// (how far the replicas have drifted apart since the last synchronisation; the term the proof
// in Appendix A controls by H).  a == nullptr skips the objective.
__global__ void la_diagnostics(const float* __restrict__ X, const float* __restrict__ a, const float* __restrict__ c,
                               uint64_t n, uint64_t stride, uint32_t W, double* __restrict__ out) {
  double f = 0.0, d = 0.0;
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += nthreads) {
    double m = 0.0;
    for (uint32_t i = 0; i < W; ++i) m += (double)X[(uint64_t)i * stride + j];
    m /= (double)W;
    double dev = 0.0;
    for (uint32_t i = 0; i < W; ++i) {
      const double e = (double)X[(uint64_t)i * stride + j] - m;
      dev += e * e;
    }
    d += dev / (double)W;
    if (a != nullptr) {
      const double e = m - (double)c[j];
      f += 0.5 * (double)a[j] * e * e;
    }
  }
  // block reduction, then one atomic pair per block
  __shared__ double sf[LA_BLOCK / 32], sd[LA_BLOCK / 32];
  for (int o = 16; o > 0; o >>= 1) {
    f += __shfl_down_sync(0xffffffffu, f, o);
    d += __shfl_down_sync(0xffffffffu, d, o);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sf[warp] = f; sd[warp] = d; }
  __syncthreads();
  if (warp == 0) {
    f = lane < (int)(blockDim.x >> 5) ? sf[lane] : 0.0;
    d = lane < (int)(blockDim.x >> 5) ? sd[lane] : 0.0;
    for (int o = 16; o > 0; o >>= 1) {
      f += __shfl_down_sync(0xffffffffu, f, o);
      d += __shfl_down_sync(0xffffffffu, d, o);
    }
    if (lane == 0) {
      atomicAdd(out, f);
      atomicAdd(out + 1, d);
    }
  }
}

}  // namespace la

namespace {

thread_local std::string g_create_error;
constexpr uint64_t kExchangeVecHost = la::kExchangeVec;

// kClassStepSync, kClassSyncStep and kClassPeriod are also counted in the aggregate "fused" class.
enum KernelClass { kClassLocal = 0, kClassSync = 1, kClassFused = 2, kClassOther = 3,
                   kClassStepSync = 4, kClassSyncStep = 5, kClassPeriod = 6 };

struct EventPair {
  cudaEvent_t a, b;
  int cls;
};

}  // namespace

struct la_ctx {
  // configuration
  std::vector<uint64_t> sizes, offsets;
  uint64_t N = 0, stride = 0, ngroups = 0, j_base = 0;
  uint32_t W = 0, H = 0;
  float eta = 0, eps = 0, b0sq = 0, sigma = 0;
  uint32_t warm_up_steps = 0;
  int grad_kind = la::kGradNoise;
  bool bf16 = false, identical = false;
  uint64_t seed = 0;
  int fusion = LA_FUSE_NONE;
  int rule = LA_RULE_ADAALTER;
  bool shared_iterate = false;  // AdaGrad steps ran: replica 0 holds x_t, B^2_t; replicas 1..W-1 are stale
  bool sums_in_replica0 = false;  // LA_FUSE_MEAN_ONCE between a closing step and the next one: replica 0's rows hold
                                  // the tree SUMS of that step's y, A^2; the other replicas and the stale array are
                                  // out of date until the sums are imported (by the next step, or on demand)
  bool profiling = false;
  int device = 0;
  cudaStream_t stream = nullptr;
  int num_sms = 148;
  int blocks_per_sm = 0;  // 0 = per-kernel default
  // device memory
  void* arena = nullptr;
  bool owns_arena = false;
  float *X = nullptr, *B2 = nullptr, *Bs = nullptr, *pa = nullptr, *pc = nullptr, *ps = nullptr;
  bool has_s = false;
  // sharding by worker: exchange buffer [2][stride], peers' buffers, global worker numbering
  uint32_t worker_base = 0, W_total = 0, rank = 0, world = 1;
  float* S = nullptr;
  float* peerS[la::kMaxRanks] = {};
  void* ipc_opened[la::kMaxRanks] = {};
  double* diag = nullptr;  // two doubles for la_diagnostics, allocated on its first call
  // la_run_streamed: copy streams and per-chunk events, created on first use
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  std::vector<cudaEvent_t> ev_in, ev_done;
  cudaEvent_t ev_idle = nullptr;
  // checked build (LA_DEBUG): device status words the kernels report address violations into,
  // and a test knob that makes the kernels treat the last `dbg_narrow` bytes of the arena as foreign
  unsigned long long* dbg_status = nullptr;
  uint64_t dbg_narrow = 0, arena_size = 0;
  // CUDA-graph replay of whole periods (la_set_graph)
  bool use_graph = false, capturing = false;
  uint64_t* sched = nullptr;       // device: global step count before the period being replayed
  uint64_t capture_base = 0;
  cudaGraphExec_t graph_exec = nullptr;
  uint64_t graph_key[8] = {};
  la_stats graph_delta{};          // what one replay adds to the statistics
  // schedule (Algorithm 3): t = local steps so far, tp = local steps since the last sync
  uint64_t t = 0, nsync = 0;
  uint32_t tp = 0;
  // statistics
  la_stats stats{};
  std::vector<EventPair> pending;
  std::vector<EventPair> pool;
  std::string err;
};

namespace {

int fail(la_ctx* c, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) c->err = buf; else g_create_error = buf;
  return code;
}

#define LA_CUDA(ctx, call)                                                                      \
  do {                                                                                          \
    cudaError_t e_ = (call);                                                                    \
    if (e_ != cudaSuccess) return fail((ctx), LA_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

uint64_t round_up(uint64_t v, uint64_t m) { return (v + m - 1) / m * m; }

// Layout of the arena, in floats: X[W][stride] | B2[W][stride] | Bs[stride] | a | c | s.
// stride = N rounded up to 64 floats, so every sub-array starts on a 256-byte boundary and
// the last group of four coordinates never leaves its array.
int validate(const la_config* cfg, uint64_t* N_out) {
  if (!cfg) return fail(nullptr, LA_EINVAL, "config is NULL");
  if (cfg->K == 0 || cfg->sizes == nullptr) return fail(nullptr, LA_EINVAL, "K must be >= 1 and sizes non-NULL");
  uint64_t N = 0;
  for (uint32_t k = 0; k < cfg->K; ++k) {
    if (cfg->sizes[k] == 0) return fail(nullptr, LA_EINVAL, "tensor %u has size 0", k);
    if (N + cfg->sizes[k] < N) return fail(nullptr, LA_EINVAL, "total size overflows");
    N += cfg->sizes[k];
  }
  if (N > (1ull << 40)) return fail(nullptr, LA_EINVAL, "N too large");
  if (cfg->W == 0 || cfg->W > LA_MAX_WORKERS) return fail(nullptr, LA_EINVAL, "W must be in 1..%u", LA_MAX_WORKERS);
  if (cfg->H == 0) return fail(nullptr, LA_EINVAL, "H must be >= 1");
  if (!std::isfinite(cfg->eta)) return fail(nullptr, LA_EINVAL, "eta must be finite");
  if (!(cfg->eps > 0.0f) || !std::isfinite(cfg->eps) || !(cfg->eps * cfg->eps > 0.0f))
    return fail(nullptr, LA_EINVAL, "eps must be finite and eps*eps > 0 in fp32");
  if (!(cfg->b0sq >= 0.0f) || !std::isfinite(cfg->b0sq)) return fail(nullptr, LA_EINVAL, "b0sq must be finite and >= 0");
  if (cfg->j_base % 4 != 0) return fail(nullptr, LA_EINVAL, "j_base must be a multiple of 4");
  *N_out = N;
  return LA_OK;
}

uint64_t arena_floats(uint64_t N, uint32_t W) {
  const uint64_t stride = round_up(N, 64);
  return stride * (2ull * W + 4ull);
}

// ---- profiling events -------------------------------------------------------------------
int drain_events(la_ctx* c) {
  if (c->pending.empty()) return LA_OK;
  LA_CUDA(c, cudaStreamSynchronize(c->stream));
  for (auto& p : c->pending) {
    float ms = 0.f;
    LA_CUDA(c, cudaEventElapsedTime(&ms, p.a, p.b));
    if (p.cls == kClassLocal) c->stats.ms_local += ms;
    else if (p.cls == kClassSync) c->stats.ms_sync += ms;
    else if (p.cls != kClassOther) c->stats.ms_fused += ms;
    if (p.cls == kClassStepSync) c->stats.ms_step_sync += ms;
    else if (p.cls == kClassSyncStep) c->stats.ms_sync_step += ms;
    else if (p.cls == kClassPeriod) c->stats.ms_period += ms;
    c->pool.push_back(p);
  }
  c->pending.clear();
  return LA_OK;
}

int begin_timed(la_ctx* c, int cls, EventPair* ep) {
  if (c->pending.size() >= 8192) {
    int rc = drain_events(c);
    if (rc) return rc;
  }
  if (!c->pool.empty()) {
    *ep = c->pool.back();
    c->pool.pop_back();
  } else {
    LA_CUDA(c, cudaEventCreate(&ep->a));
    LA_CUDA(c, cudaEventCreate(&ep->b));
  }
  ep->cls = cls;
  LA_CUDA(c, cudaEventRecord(ep->a, c->stream));
  return LA_OK;
}

// ---- checked build ---------------------------------------------------------------------------
#ifdef LA_DEBUG
void fill_debug_ranges(const la_ctx* c, la::DebugRanges* d, const void* gext, uint64_t gext_bytes) {
  const uint64_t a = reinterpret_cast<uint64_t>(c->arena);
  d->lo[0] = a; d->hi[0] = a + c->arena_size - c->dbg_narrow;
  d->lo[1] = reinterpret_cast<uint64_t>(gext); d->hi[1] = d->lo[1] + gext_bytes;
  d->lo[2] = reinterpret_cast<uint64_t>(c->S); d->hi[2] = d->lo[2] + (c->S ? 2 * c->stride * sizeof(float) : 0);
  d->status = c->dbg_status;
}
#endif

// After a synchronising call in the checked build: turn recorded violations into an error.
int debug_poll(la_ctx* c) {
#ifdef LA_DEBUG
  if (!c->dbg_status) return LA_OK;
  unsigned long long st[3] = {0, 0, 0};
  LA_CUDA(c, cudaMemcpyAsync(st, c->dbg_status, sizeof st, cudaMemcpyDeviceToHost, c->stream));
  LA_CUDA(c, cudaStreamSynchronize(c->stream));
  if (st[0] != 0) {
    LA_CUDA(c, cudaMemsetAsync(c->dbg_status, 0, sizeof st, c->stream));
    const char* kind = (st[2] & 0xFF) == 2 ? "is not the row its replica index and coordinate give" : "lies outside every range the pass may touch";
    return fail(c, LA_EBOUNDS, "checked build: %llu access(es) skipped; the first, at device address 0x%llx (%llu bytes), %s",
                st[0], st[1], (st[2] >> 8), kind);
  }
#else
  (void)c;
#endif
  return LA_OK;
}

// ---- kernel dispatch ------------------------------------------------------------------------
// Algorithmic bytes of one pass (what must cross HBM with the thread-per-coordinate mapping):
// every replica's x and B^2 read and written once, worker-independent arrays once.
double pass_bytes(const la_ctx* c, bool pre, bool step, bool post, int gm) {
  const double n = (double)c->N, W = (double)c->W;
  if (c->rule == LA_RULE_ADAGRAD) {                 // one shared x, B2: read + write, Bs written
    double b = 20.0 * n;
    if (gm == la::kGradExternalF32) b += 4.0 * W * n;
    if (gm == la::kGradExternalBF16) b += 2.0 * W * n;
    if (gm == la::kGradQuadratic) b += 8.0 * n;
    if (gm == la::kGradNoiseScaled || (gm == la::kGradConstant && c->has_s)) b += 4.0 * n;
    return b;
  }
  if (c->rule == LA_RULE_LOCAL_SGD) {               // X only: read + write
    double b = 8.0 * W * n;
    if (step) {
      if (gm == la::kGradExternalF32) b += 4.0 * W * n;
      if (gm == la::kGradExternalBF16) b += 2.0 * W * n;
      if (gm == la::kGradQuadratic) b += 8.0 * n;
      if (gm == la::kGradNoiseScaled || (gm == la::kGradConstant && c->has_s)) b += 4.0 * n;
    }
    return b;
  }
  double b = 16.0 * W * n;                          // X, B2: read + write
  if (pre || post) b += 4.0 * n;                    // stale accumulator written
  if (step && !pre) b += 4.0 * n;                   // stale accumulator read
  if (step) {
    if (gm == la::kGradQuadratic) b += 8.0 * n;
    if (gm == la::kGradNoiseScaled || (gm == la::kGradConstant && c->has_s)) b += 4.0 * n;
    if (gm == la::kGradExternalF32) b += 4.0 * W * n;
    if (gm == la::kGradExternalBF16) b += 2.0 * W * n;
  }
  return b;
}

// xch: 0 = a pass of the single-GPU path; 1 / 2 = the pass exports to / imports from the exchange
// buffer of the by-worker sharding (see la_exchange.cuh).
// in_replica0: the sums live in replica 0's own rows (single-GPU LA_FUSE_MEAN_ONCE) instead of the exchange buffer.
int launch_sweep(la_ctx* c, bool pre, bool step, bool post, uint64_t t, uint32_t tp, int gm, const void* gext,
                 int xch = 0, bool in_replica0 = false) {
  const la::SweepKernel k =
      la::lookup_sweep((int)c->W, c->rule, gm, c->bf16 && gm <= la::kGradQuadratic, pre, step, post, xch);
  la::SweepFn fn = k.fn;
  if (!fn)
    return fail(c, LA_ESTATE, "no kernel for this combination (W=%u rule=%d grad=%d bf16=%d)", c->W, c->rule, gm,
                (int)c->bf16);
  la::SweepParams p{};
  p.X = c->X; p.B2 = c->B2; p.Bs = c->Bs;
  p.a = c->pa; p.c = c->pc; p.s = c->has_s ? c->ps : nullptr;
  p.gext = gext;
  if (gext) {
    const uint64_t elem = (gm == la::kGradExternalBF16) ? 2 : 4;
    p.gext_vec = (c->N % (uint64_t)k.vec == 0 && (reinterpret_cast<uintptr_t>(gext) % ((uint64_t)k.vec * elem)) == 0) ? 1u : 0u;
  }
  p.n = c->N; p.stride = c->stride; p.j_base = c->j_base;
  p.seed = c->seed; p.W = c->W; p.tp = tp;
  p.t = c->capturing ? t - c->capture_base : t;
  p.t_dev = c->capturing ? c->sched : nullptr;
  p.warm_up_steps = c->warm_up_steps; p.identical_workers = c->identical ? 1u : 0u;
  p.worker_base = c->worker_base;
  p.eta = c->eta; p.eps = c->eps; p.sigma = c->sigma;
  p.xch = c->S; p.xch_b_off = c->stride; p.W_total = c->W_total;
  if (in_replica0) { p.xch = c->X; p.xch_b_off = (uint64_t)c->W * c->stride; p.W_total = c->W; }
#ifdef LA_DEBUG
  fill_debug_ranges(c, &p.dbg, gext, gext ? (uint64_t)c->W * c->N * (gm == la::kGradExternalBF16 ? 2u : 4u) : 0u);
#endif
  const unsigned block = la::kBlockThreads;
  const uint64_t ngroups = (c->N + (uint64_t)k.vec - 1) / (uint64_t)k.vec;
  uint64_t blocks = (ngroups + block - 1) / block;
  // Measured on B200 (sweeps of 4..4096 blocks per SM): kernels that take a step run best when a
  // block lives long enough to amortise its start (the software pipeline over coordinate groups
  // pays off) yet stays small enough to balance the SMs.  The work of a block grows with the
  // replicas and coordinates a thread owns, so the grid does too: 16 W blocks per SM for
  // two-coordinate threads (W = 4: 64; 96 from W = 6 on), half of that for four-coordinate
  // threads, never fewer than 32.  The pure averaging kernel runs best with one group per thread.
  int step_bps = 16 * (int)c->W * 2 / k.vec;
  step_bps = step_bps < 32 ? 32 : (step_bps > 96 ? 96 : step_bps);
  // (run-time worker counts: their averaging pass overlaps a group's tail with the next group's
  // first loads, so it wants a grid-stride grid too — W = 5 / 9 / 20: 0.72 / 0.83 / 0.98 of the copy
  // bandwidth at 32 blocks per SM against 0.58 / 0.65 / 0.86 with one group per thread)
  const bool runtime_w = la::lookup_sweep_is_runtime((int)c->W);
  const int bps = c->blocks_per_sm > 0 ? c->blocks_per_sm : (step ? step_bps : (runtime_w ? 32 : 4096));
  const uint64_t cap = (uint64_t)c->num_sms * (uint64_t)bps;
  if (blocks > cap) blocks = cap;
  int cls = !step ? kClassSync : (post ? kClassStepSync : (pre ? kClassSyncStep : kClassLocal));
  if (xch != 0 && !in_replica0) cls = step ? kClassFused : kClassOther;  // exchange passes: aggregate classes only
  EventPair ep{};
  if (c->profiling) {
    int rc = begin_timed(c, cls, &ep);
    if (rc) return rc;
  }
  fn<<<(unsigned)blocks, block, 0, c->stream>>>(p);
  LA_CUDA(c, cudaGetLastError());
  if (c->profiling) {
    LA_CUDA(c, cudaEventRecord(ep.b, c->stream));
    c->pending.push_back(ep);
  }
  double bytes = pass_bytes(c, pre, step, post, gm);
  const double rw = 8.0 * c->W * (double)c->N, ex = 8.0 * (double)c->N;  // replicas one way; the exchange buffer
  if (xch == 1) bytes += ex - rw - (post ? 4.0 * (double)c->N : 0.0);    // sums stored instead of W means (and no Bs)
  if (xch == 2) bytes += ex - rw;                                        // totals read instead of W replicas
  if (cls == kClassLocal) { c->stats.launches_local++; c->stats.bytes_local += bytes; }
  else if (cls == kClassSync) { c->stats.launches_sync++; c->stats.bytes_sync += bytes; }
  else if (cls == kClassOther) { c->stats.launches_other++; }
  else {
    c->stats.launches_fused++; c->stats.bytes_fused += bytes;
    if (cls == kClassStepSync) { c->stats.launches_step_sync++; c->stats.bytes_step_sync += bytes; }
    else if (cls == kClassSyncStep) { c->stats.launches_sync_step++; c->stats.bytes_sync_step += bytes; }
  }
  return LA_OK;
}

// h consecutive local steps (and, if `post`, the synchronisation that closes the period) in one pass.
int launch_period(la_ctx* c, uint32_t h, bool post) {
  const la::PeriodKernel k =
      la::lookup_period((int)c->W, c->grad_kind, c->bf16 && c->grad_kind <= la::kGradQuadratic, post);
  if (!k.fn) return fail(c, LA_ESTATE, "no period kernel for this combination (W=%u grad=%d)", c->W, c->grad_kind);
  la::PeriodParams pp{};
  la::SweepParams& p = pp.base;
  p.X = c->X; p.B2 = c->B2; p.Bs = c->Bs;
  p.a = c->pa; p.c = c->pc; p.s = c->has_s ? c->ps : nullptr;
  p.n = c->N; p.stride = c->stride; p.j_base = c->j_base;
  p.seed = c->seed; p.W = c->W; p.tp = c->tp;
  p.t = c->capturing ? c->t - c->capture_base : c->t;
  p.t_dev = c->capturing ? c->sched : nullptr;
  p.warm_up_steps = c->warm_up_steps; p.identical_workers = c->identical ? 1u : 0u;
  p.worker_base = c->worker_base;
  p.eta = c->eta; p.eps = c->eps; p.sigma = c->sigma;
  pp.h = h;
#ifdef LA_DEBUG
  fill_debug_ranges(c, &p.dbg, nullptr, 0);
#endif
  const unsigned block = (unsigned)k.block;
  const uint64_t ngroups = (c->N + (uint64_t)k.vec - 1) / (uint64_t)k.vec;
  uint64_t blocks = (ngroups + block - 1) / block;
  // issue-bound kernel: at the full configuration sizes 384..768 blocks per SM in the grid measured
  // best (few coordinate groups per thread); smaller grids lose up to 20 %
  const int bps = c->blocks_per_sm > 0 ? c->blocks_per_sm : 768;  // counted in 256-thread units
  const uint64_t cap = (uint64_t)c->num_sms * (uint64_t)bps * 256u / block;
  if (blocks > cap) blocks = cap;
  EventPair ep{};
  if (c->profiling) {
    int rc = begin_timed(c, kClassPeriod, &ep);
    if (rc) return rc;
  }
  k.fn<<<(unsigned)blocks, block, 0, c->stream>>>(pp);
  LA_CUDA(c, cudaGetLastError());
  if (c->profiling) {
    LA_CUDA(c, cudaEventRecord(ep.b, c->stream));
    c->pending.push_back(ep);
  }
  const double bytes = pass_bytes(c, false, true, post, c->grad_kind);
  c->stats.launches_fused++; c->stats.bytes_fused += bytes;
  c->stats.launches_period++; c->stats.bytes_period += bytes;
  return LA_OK;
}

int upload_padded(la_ctx* c, float* dst, const float* src_host, float pad) {
  // dst has `stride` floats; [0,N) from the host, the tail [N,stride) = pad.
  LA_CUDA(c, cudaMemcpyAsync(dst, src_host, c->N * sizeof(float), cudaMemcpyHostToDevice, c->stream));
  if (c->stride > c->N) {
    if (pad != 0.0f) return fail(c, LA_EINVAL, "internal: non-zero pad");
    LA_CUDA(c, cudaMemsetAsync(dst + c->N, 0, (c->stride - c->N) * sizeof(float), c->stream));
  }
  return LA_OK;
}

// count = 0: the whole arrays up to the replica stride (padding included).
int do_fill(la_ctx* c, const float* x0_dev, uint64_t count = 0) {
  const unsigned block = 256;
  if (count == 0) count = c->stride;
  uint64_t blocks = (count + block - 1) / block;
  const uint64_t cap = (uint64_t)c->num_sms * 16;
  if (blocks > cap) blocks = cap;
  la::la_fill<<<(unsigned)blocks, block, 0, c->stream>>>(c->X, c->B2, c->Bs, x0_dev, c->b0sq, c->stride, c->N, count, c->W);
  LA_CUDA(c, cudaGetLastError());
  c->stats.launches_other++;
  return LA_OK;
}

// Algorithm 1 has ONE iterate that every worker holds; la_adagrad stores it in replica 0 only.
// Before anything looks at replicas 1..W-1 individually again (another update rule, a per-worker
// write), replica 0 is copied into them.
int materialise_replicas(la_ctx* c) {
  if (!c->shared_iterate) return LA_OK;
  if (c->W > 1) {
    const unsigned block = 256;
    uint64_t blocks = (c->stride / 4 + block - 1) / block;
    const uint64_t cap = (uint64_t)c->num_sms * 32;
    if (blocks > cap) blocks = cap;
    la::la_broadcast_replica0<<<(unsigned)blocks, block, 0, c->stream>>>(c->X, c->B2, c->stride, c->W);
    LA_CUDA(c, cudaGetLastError());
    c->stats.launches_other++;
  }
  c->shared_iterate = false;
  return LA_OK;
}

// LA_FUSE_MEAN_ONCE leaves the sums of a closing step in replica 0's rows; whoever needs the
// synchronised state itself (a reader, a writer, another kind of step) first turns them into
// the means in every replica and the stale array: the import half of that synchronisation.
int import_pending_sums(la_ctx* c) {
  if (!c->sums_in_replica0) return LA_OK;
  int rc = launch_sweep(c, true, false, false, c->t, 0, la::kGradNoise, nullptr, 2, true);
  if (rc) return rc;
  c->sums_in_replica0 = false;
  return LA_OK;
}

}  // namespace

// =============================================================================== C surface
extern "C" {

const char* la_last_error(const la_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

int la_arena_bytes(const la_config* cfg, uint64_t* bytes) {
  uint64_t N = 0;
  int rc = validate(cfg, &N);
  if (rc) return rc;
  if (!bytes) return fail(nullptr, LA_EINVAL, "bytes is NULL");
  *bytes = arena_floats(N, cfg->W) * sizeof(float);
  return LA_OK;
}

int la_create_ex(la_ctx** out, const la_config* cfg) {
  if (!out) return fail(nullptr, LA_EINVAL, "out is NULL");
  *out = nullptr;
  uint64_t N = 0;
  int rc = validate(cfg, &N);
  if (rc) return rc;
  la_ctx* c = new (std::nothrow) la_ctx();
  if (!c) return fail(nullptr, LA_ENOMEM, "host allocation failed");
  auto bail = [&](int code, const char* what, cudaError_t e) {
    fail(nullptr, code, "%s%s%s", what, e != cudaSuccess ? ": " : "", e != cudaSuccess ? cudaGetErrorString(e) : "");
    if (c->owns_arena && c->arena) cudaFree(c->arena);
    if (c->dbg_status) cudaFree(c->dbg_status);
    delete c;
    return code;
  };
  cudaError_t e;
  int dev = cfg->device;
  if (dev < 0 && (e = cudaGetDevice(&dev)) != cudaSuccess) return bail(LA_ECUDA, "cudaGetDevice", e);
  c->device = dev;
  DeviceGuard guard(dev);
  if (!guard.ok) return bail(LA_ECUDA, "cannot select device", cudaSuccess);
  int sms = 0;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
    return bail(LA_ECUDA, "cudaDeviceGetAttribute", e);
  c->num_sms = sms > 0 ? sms : 148;
  c->sizes.assign(cfg->sizes, cfg->sizes + cfg->K);
  c->offsets.resize(cfg->K);
  uint64_t off = 0;
  for (uint32_t k = 0; k < cfg->K; ++k) { c->offsets[k] = off; off += c->sizes[k]; }
  c->N = N;
  c->stride = round_up(N, 64);
  c->ngroups = (N + 3) / 4;
  c->j_base = cfg->j_base;
  c->W = cfg->W; c->H = cfg->H; c->eta = cfg->eta; c->eps = cfg->eps; c->b0sq = cfg->b0sq;
  c->stream = (cudaStream_t)cfg->stream;
  const uint64_t need = arena_floats(N, cfg->W) * sizeof(float);
  if (cfg->dev_arena) {
    if (cfg->arena_bytes < need) return bail(LA_ENOMEM, "caller arena smaller than la_arena_bytes()", cudaSuccess);
    if (((uintptr_t)cfg->dev_arena & 255u) != 0) return bail(LA_EINVAL, "caller arena must be 256-byte aligned", cudaSuccess);
    c->arena = cfg->dev_arena;
  } else {
    if ((e = cudaMalloc(&c->arena, need)) != cudaSuccess) {
      c->arena = nullptr;
      cudaGetLastError();
      return bail(LA_ENOMEM, "cudaMalloc of the state arena failed", e);
    }
    c->owns_arena = true;
  }
  c->arena_size = need;
#ifdef LA_DEBUG
  if ((e = cudaMalloc((void**)&c->dbg_status, 4 * sizeof(unsigned long long))) != cudaSuccess) {
    c->dbg_status = nullptr;
    cudaGetLastError();
    return bail(LA_ENOMEM, "cudaMalloc of the checked build's status words failed", e);
  }
  if ((e = cudaMemsetAsync(c->dbg_status, 0, 4 * sizeof(unsigned long long), c->stream)) != cudaSuccess)
    return bail(LA_ECUDA, "cudaMemsetAsync", e);
#endif
  float* base = (float*)c->arena;
  c->X = base;
  c->B2 = c->X + (uint64_t)c->W * c->stride;
  c->Bs = c->B2 + (uint64_t)c->W * c->stride;
  c->pa = c->Bs + c->stride;
  c->pc = c->pa + c->stride;
  c->ps = c->pc + c->stride;
  // problem arrays start as zeros so that padded coordinates stay finite in every mode
  if ((e = cudaMemsetAsync(c->pa, 0, 3 * c->stride * sizeof(float), c->stream)) != cudaSuccess)
    return bail(LA_ECUDA, "cudaMemsetAsync", e);
  c->grad_kind = la::kGradNoise;
  rc = do_fill(c, nullptr);
  if (rc) { g_create_error = c->err; if (c->owns_arena) cudaFree(c->arena); if (c->dbg_status) cudaFree(c->dbg_status); delete c; return rc; }
  *out = c;
  return LA_OK;
}

int la_create(la_ctx** out, uint64_t N, uint32_t W, float eta, float eps, uint32_t H) {
  la_config cfg;
  std::memset(&cfg, 0, sizeof cfg);
  cfg.K = 1; cfg.sizes = &N; cfg.W = W; cfg.H = H; cfg.eta = eta; cfg.eps = eps; cfg.b0sq = 0.0f;
  cfg.device = -1;
  return la_create_ex(out, &cfg);
}

void la_destroy(la_ctx* c) {
  if (!c) return;
  DeviceGuard guard(c->device);
  cudaStreamSynchronize(c->stream);
  for (auto& p : c->pending) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  for (auto& p : c->pool) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  for (auto*& m : c->ipc_opened) if (m) { cudaIpcCloseMemHandle(m); m = nullptr; }
  if (c->S) cudaFree(c->S);
  if (c->diag) cudaFree(c->diag);
  if (c->dbg_status) cudaFree(c->dbg_status);
  for (auto e : c->ev_in) cudaEventDestroy(e);
  for (auto e : c->ev_done) cudaEventDestroy(e);
  if (c->ev_idle) cudaEventDestroy(c->ev_idle);
  if (c->copy_in) cudaStreamDestroy(c->copy_in);
  if (c->copy_out) cudaStreamDestroy(c->copy_out);
  if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
  if (c->sched) cudaFree(c->sched);
  if (c->owns_arena && c->arena) cudaFree(c->arena);
  delete c;
}

int la_set_init(la_ctx* c, const float* x0_host, float b0sq) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!(b0sq >= 0.0f) || !std::isfinite(b0sq)) return fail(c, LA_EINVAL, "b0sq must be finite and >= 0");
  DeviceGuard guard(c->device);
  c->b0sq = b0sq;
  const float* x0_dev = nullptr;
  if (x0_host) {
    // stage x0 in replica 0's own slot, then broadcast from there
    LA_CUDA(c, cudaMemcpyAsync(c->X, x0_host, c->N * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    x0_dev = c->X;
  }
  int rc = do_fill(c, x0_dev);
  if (rc) return rc;
  c->shared_iterate = false;
  c->sums_in_replica0 = false;
  c->t = 0; c->tp = 0; c->nsync = 0;
  return LA_OK;
}

int la_set_grad_noise(la_ctx* c, uint64_t seed, const float* s_host) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  DeviceGuard guard(c->device);
  c->seed = seed;
  c->has_s = s_host != nullptr;
  c->grad_kind = s_host ? la::kGradNoiseScaled : la::kGradNoise;
  if (s_host) return upload_padded(c, c->ps, s_host, 0.0f);
  return LA_OK;
}

int la_set_grad_quadratic(la_ctx* c, uint64_t seed, const float* a_host, const float* c_host, float sigma) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!a_host || !c_host) return fail(c, LA_EINVAL, "a and c must be non-NULL");
  if (!std::isfinite(sigma)) return fail(c, LA_EINVAL, "sigma must be finite");
  DeviceGuard guard(c->device);
  c->seed = seed; c->sigma = sigma; c->grad_kind = la::kGradQuadratic;
  int rc = upload_padded(c, c->pa, a_host, 0.0f);
  if (rc) return rc;
  return upload_padded(c, c->pc, c_host, 0.0f);
}

int la_set_grad_constant(la_ctx* c, const float* s_host) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  DeviceGuard guard(c->device);
  c->grad_kind = la::kGradConstant;
  c->has_s = s_host != nullptr;
  if (s_host) return upload_padded(c, c->ps, s_host, 0.0f);
  return LA_OK;
}

int la_set_grad_dtype(la_ctx* c, int dtype) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (dtype != LA_F32 && dtype != LA_BF16) return fail(c, LA_EINVAL, "dtype must be LA_F32 or LA_BF16");
  c->bf16 = dtype == LA_BF16;
  return LA_OK;
}

int la_set_identical_workers(la_ctx* c, int on) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  c->identical = on != 0;
  return LA_OK;
}

int la_set_warmup(la_ctx* c, uint32_t steps) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  c->warm_up_steps = steps;
  return LA_OK;
}

int la_set_fusion(la_ctx* c, int mode) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (mode != LA_FUSE_NONE && mode != LA_FUSE_STEP_SYNC && mode != LA_FUSE_SYNC_STEP && mode != LA_FUSE_PERIOD &&
      mode != LA_FUSE_MEAN_ONCE)
    return fail(c, LA_EINVAL, "unknown fusion mode %d", mode);
  c->fusion = mode;
  return LA_OK;
}

int la_set_rule(la_ctx* c, int rule) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (rule != LA_RULE_ADAALTER && rule != LA_RULE_LOCAL_SGD && rule != LA_RULE_ADAGRAD)
    return fail(c, LA_EINVAL, "unknown update rule %d", rule);
  if (c->tp != 0) return fail(c, LA_ESTATE, "the update rule can only change right after a synchronisation (t' = 0)");
  if (rule != c->rule) {
    DeviceGuard guard(c->device);
    int rc = import_pending_sums(c);
    if (rc) return rc;
  }
  if (c->rule == LA_RULE_ADAGRAD && rule != LA_RULE_ADAGRAD) {
    DeviceGuard guard(c->device);
    int rc = materialise_replicas(c);  // the other rules advance every replica on its own
    if (rc) return rc;
  }
  c->rule = rule;
  return LA_OK;
}

int la_set_graph(la_ctx* c, int on) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (on && c->stream == nullptr) return fail(c, LA_ESTATE, "graph replay needs a context on a non-default stream (the legacy default stream cannot be captured)");
  DeviceGuard guard(c->device);
  if (on && !c->sched) {
    cudaError_t e = cudaMalloc((void**)&c->sched, sizeof(uint64_t));
    if (e != cudaSuccess) { c->sched = nullptr; cudaGetLastError(); return fail(c, LA_ENOMEM, "cudaMalloc failed: %s", cudaGetErrorString(e)); }
  }
  c->use_graph = on != 0;
  return LA_OK;
}

int la_set_profiling(la_ctx* c, int on) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  DeviceGuard guard(c->device);
  if (!on) { int rc = drain_events(c); if (rc) return rc; }
  c->profiling = on != 0;
  return LA_OK;
}

int la_set_launch_shape(la_ctx* c, int blocks_per_sm) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (blocks_per_sm < 0 || blocks_per_sm > 4096) return fail(c, LA_EINVAL, "blocks_per_sm out of range");
  c->blocks_per_sm = blocks_per_sm;
  return LA_OK;
}

// ---- hot path ------------------------------------------------------------------------------
int la_local_step(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  int rc = launch_sweep(c, false, true, false, c->t + 1, c->tp + 1, c->grad_kind, nullptr);
  if (rc) return rc;
  c->t += 1;
  if (c->rule == LA_RULE_ADAGRAD) { c->nsync += 1; c->shared_iterate = true; }  // Algorithm 1 exchanges gradients every iteration
  else c->tp += 1;
  return LA_OK;
}

int la_local_step_grads(la_ctx* c, const void* g_dev, int dtype) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!g_dev) return fail(c, LA_EINVAL, "g_dev is NULL");
  if (dtype != LA_F32 && dtype != LA_BF16) return fail(c, LA_EINVAL, "dtype must be LA_F32 or LA_BF16");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  int rc = launch_sweep(c, false, true, false, c->t + 1, c->tp + 1,
                        dtype == LA_F32 ? la::kGradExternalF32 : la::kGradExternalBF16, g_dev);
  if (rc) return rc;
  c->t += 1;
  if (c->rule == LA_RULE_ADAGRAD) { c->nsync += 1; c->shared_iterate = true; }
  else c->tp += 1;
  return LA_OK;
}

int la_step_grads(la_ctx* c, const void* g_dev, int dtype) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!g_dev) return fail(c, LA_EINVAL, "g_dev is NULL");
  if (dtype != LA_F32 && dtype != LA_BF16) return fail(c, LA_EINVAL, "dtype must be LA_F32 or LA_BF16");
  if (c->rule == LA_RULE_ADAGRAD) return la_local_step_grads(c, g_dev, dtype);  // Algorithm 1: one pass is the whole iteration
  DeviceGuard guard(c->device);
  const int gm = dtype == LA_F32 ? la::kGradExternalF32 : la::kGradExternalBF16;
  if (c->fusion == LA_FUSE_MEAN_ONCE && c->rule == LA_RULE_ADAALTER && c->H >= 2u) {
    // the synchronised state is stored once (see run_steps): sums out at t' = H, one copy in at t' = 1
    if (c->sums_in_replica0) {
      int rc = launch_sweep(c, true, true, false, c->t + 1, 1u, gm, g_dev, 2, true);
      if (rc) return rc;
      c->sums_in_replica0 = false;
      c->t += 1; c->tp = 1;
      return LA_OK;
    }
    if (c->tp + 1 == c->H) {
      int rc = launch_sweep(c, false, true, true, c->t + 1, c->tp + 1, gm, g_dev, 1, true);
      if (rc) return rc;
      c->sums_in_replica0 = true;
      c->t += 1; c->tp = 0; c->nsync += 1;
      return LA_OK;
    }
  }
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  const bool closes = (c->tp + 1 == c->H);
  if (closes && c->fusion != LA_FUSE_NONE) {
    int rc = launch_sweep(c, false, true, true, c->t + 1, c->tp + 1, gm, g_dev);  // step and its sync in one pass
    if (rc) return rc;
    c->t += 1; c->tp = 0; c->nsync += 1;
    return LA_OK;
  }
  int rc = launch_sweep(c, false, true, false, c->t + 1, c->tp + 1, gm, g_dev);
  if (rc) return rc;
  c->t += 1; c->tp += 1;
  if (c->tp == c->H) return la_sync(c);
  return LA_OK;
}

int la_sync(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (c->rule == LA_RULE_ADAGRAD) return fail(c, LA_ESTATE, "Distributed AdaGrad keeps one shared iterate: nothing to synchronise");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  int rc = launch_sweep(c, true, false, false, c->t, 0, la::kGradNoise, nullptr);
  if (rc) return rc;
  c->tp = 0; c->nsync += 1;
  return LA_OK;
}

static int run_steps(la_ctx* c, uint64_t T);

// Capture one whole period (H iterations from t' = 0, exactly the launches run_steps would make)
// into a CUDA graph.  The kernels take the step index as "offset within the period + *sched", so
// the same graph serves every period; its last node advances *sched by H.
static int ensure_period_graph(la_ctx* c) {
  uint64_t key[8] = {(uint64_t)c->fusion | ((uint64_t)c->rule << 8) | ((uint64_t)c->grad_kind << 16) |
                         ((uint64_t)c->bf16 << 24) | ((uint64_t)c->identical << 25) | ((uint64_t)c->has_s << 26),
                     c->seed, (uint64_t)c->warm_up_steps | ((uint64_t)c->blocks_per_sm << 32),
                     (uint64_t)c->worker_base | ((uint64_t)c->H << 32), 0, 0, 0, 1};
  std::memcpy(&key[4], &c->sigma, sizeof(float));
  std::memcpy(&key[5], &c->eta, sizeof(float));
  std::memcpy(&key[6], &c->eps, sizeof(float));
  if (c->graph_exec && std::memcmp(key, c->graph_key, sizeof key) == 0) return LA_OK;
  if (c->graph_exec) { cudaGraphExecDestroy(c->graph_exec); c->graph_exec = nullptr; }
  const uint64_t t0 = c->t, ns0 = c->nsync;
  const uint32_t tp0 = c->tp;
  const la_stats st0 = c->stats;
  LA_CUDA(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
  c->capturing = true;
  c->capture_base = c->t;
  int rc = run_steps(c, c->H);
  if (rc == LA_OK) {
    la::la_counter_add<<<1, 1, 0, c->stream>>>(c->sched, (uint64_t)c->H);
    if (cudaGetLastError() != cudaSuccess) rc = fail(c, LA_ECUDA, "launch of the counter node failed");
  }
  c->capturing = false;
  cudaGraph_t graph = nullptr;
  cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
  // what one replay adds to the statistics; then undo the bookkeeping of the (unexecuted) capture
  c->graph_delta = la_stats{};
  c->graph_delta.launches_local = c->stats.launches_local - st0.launches_local;
  c->graph_delta.launches_sync = c->stats.launches_sync - st0.launches_sync;
  c->graph_delta.launches_fused = c->stats.launches_fused - st0.launches_fused;
  c->graph_delta.launches_step_sync = c->stats.launches_step_sync - st0.launches_step_sync;
  c->graph_delta.launches_period = c->stats.launches_period - st0.launches_period;
  c->graph_delta.launches_other = 1;
  c->graph_delta.bytes_local = c->stats.bytes_local - st0.bytes_local;
  c->graph_delta.bytes_sync = c->stats.bytes_sync - st0.bytes_sync;
  c->graph_delta.bytes_fused = c->stats.bytes_fused - st0.bytes_fused;
  c->graph_delta.bytes_step_sync = c->stats.bytes_step_sync - st0.bytes_step_sync;
  c->graph_delta.bytes_period = c->stats.bytes_period - st0.bytes_period;
  c->stats = st0; c->t = t0; c->tp = tp0; c->nsync = ns0;
  if (rc != LA_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
  if (e != cudaSuccess || !graph) { cudaGetLastError(); return fail(c, LA_ECUDA, "stream capture failed: %s", cudaGetErrorString(e)); }
  e = cudaGraphInstantiate(&c->graph_exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e != cudaSuccess) { c->graph_exec = nullptr; cudaGetLastError(); return fail(c, LA_ECUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(e)); }
  std::memcpy(c->graph_key, key, sizeof key);
  return LA_OK;
}

int la_run(la_ctx* c, uint64_t T) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  DeviceGuard guard(c->device);
  // Launch-bound regime (small N): replay whole periods from a captured graph.
  if (c->use_graph && !c->profiling && c->rule != LA_RULE_ADAGRAD && c->fusion != LA_FUSE_SYNC_STEP &&
      c->fusion != LA_FUSE_MEAN_ONCE && !c->sums_in_replica0 && c->tp == 0 &&
      c->H <= 4096u && T >= (uint64_t)c->H) {
    int rc = ensure_period_graph(c);
    if (rc) return rc;
    const uint64_t reps = T / c->H;
    la::la_counter_set<<<1, 1, 0, c->stream>>>(c->sched, c->t);
    LA_CUDA(c, cudaGetLastError());
    for (uint64_t k = 0; k < reps; ++k) LA_CUDA(c, cudaGraphLaunch(c->graph_exec, c->stream));
    c->t += reps * c->H;
    c->nsync += reps;
    c->stats.launches_local += reps * c->graph_delta.launches_local;
    c->stats.launches_sync += reps * c->graph_delta.launches_sync;
    c->stats.launches_fused += reps * c->graph_delta.launches_fused;
    c->stats.launches_other += reps * c->graph_delta.launches_other + 1;
    c->stats.bytes_local += (double)reps * c->graph_delta.bytes_local;
    c->stats.bytes_sync += (double)reps * c->graph_delta.bytes_sync;
    c->stats.bytes_fused += (double)reps * c->graph_delta.bytes_fused;
    c->stats.launches_step_sync += reps * c->graph_delta.launches_step_sync;
    c->stats.launches_period += reps * c->graph_delta.launches_period;
    c->stats.bytes_step_sync += (double)reps * c->graph_delta.bytes_step_sync;
    c->stats.bytes_period += (double)reps * c->graph_delta.bytes_period;
    T -= reps * c->H;
  }
  return run_steps(c, T);
}

static int run_steps(la_ctx* c, uint64_t T) {
  // Algorithm 3: for t in [T]: local step; if mod(t, H) == 0 (tracked as t' == H): synchronise.
  // `deferred` marks a synchronisation that is due but has been folded into the next step.
  if (c->fusion != LA_FUSE_MEAN_ONCE || c->rule != LA_RULE_ADAALTER || c->H < 2u) {
    int rc_ = import_pending_sums(c);
    if (rc_) return rc_;
  }
  if (c->rule == LA_RULE_ADAGRAD) {  // Algorithm 1: every iteration is one fully synchronous pass
    for (uint64_t k = 0; k < T; ++k) {
      int rc = la_local_step(c);
      if (rc) return rc;
    }
    return LA_OK;
  }
  if (c->fusion == LA_FUSE_PERIOD && c->rule == LA_RULE_ADAALTER) {
    // temporal blocking: up to kPeriodMax local steps per pass, the closing one with its sync
    uint64_t left = T;
    while (left > 0) {
      if (c->tp >= c->H) {  // only after manual stepping past H: behave like the plain loop
        int rc = la_local_step(c);
        if (rc) return rc;
        left -= 1;
        continue;
      }
      uint64_t h = (uint64_t)(c->H - c->tp);
      if (h > left) h = left;
      if (h > (uint64_t)la::kPeriodMax) h = la::kPeriodMax;
      const bool closes = (c->tp + h == c->H);
      // a single step gains nothing from the blocked kernel: use the step kernels (K1 / K3)
      int rc = (h == 1) ? launch_sweep(c, false, true, closes, c->t + 1, c->tp + 1, c->grad_kind, nullptr)
                        : launch_period(c, (uint32_t)h, closes);
      if (rc) return rc;
      c->t += h;
      if (closes) { c->tp = 0; c->nsync += 1; } else { c->tp += (uint32_t)h; }
      left -= h;
    }
    return LA_OK;
  }
  if (c->fusion == LA_FUSE_MEAN_ONCE && c->rule == LA_RULE_ADAALTER && c->H >= 2u) {
    // A synchronisation makes all replicas equal, so its result is stored ONCE: the step that
    // closes a period writes only the tree sums of its y, A^2 (into replica 0's rows), and the
    // first step of the next period reads that one copy, divides, and writes the W replicas it
    // produces.  Per period this saves one write and one read of all replicas but one.  The
    // sums stay pending across calls; anything else that needs the state imports them first.
    for (uint64_t k = 0; k < T; ++k) {
      int rc;
      if (c->sums_in_replica0) {
        rc = launch_sweep(c, true, true, false, c->t + 1, 1u, c->grad_kind, nullptr, 2, true);  // import, then step t' = 1
        if (rc) return rc;
        c->sums_in_replica0 = false;
        c->t += 1; c->tp = 1;
      } else if (c->tp + 1 == c->H) {
        rc = launch_sweep(c, false, true, true, c->t + 1, c->tp + 1, c->grad_kind, nullptr, 1, true);  // step t' = H, sums only
        if (rc) return rc;
        c->sums_in_replica0 = true;
        c->t += 1; c->tp = 0; c->nsync += 1;
      } else {
        rc = la_local_step(c);  // K1
        if (rc) return rc;
      }
    }
    return LA_OK;
  }
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  bool deferred = false;
  const int fusion = (c->fusion == LA_FUSE_PERIOD || c->fusion == LA_FUSE_MEAN_ONCE) ? LA_FUSE_STEP_SYNC
                                                                                      : c->fusion;  // fall-backs: step+sync
  for (uint64_t k = 0; k < T; ++k) {
    int rc;
    if (deferred) {
      rc = launch_sweep(c, true, true, false, c->t + 1, 1, c->grad_kind, nullptr);  // K4: sync, then step t'=1
      if (rc) return rc;
      c->nsync += 1; c->t += 1; c->tp = 1;
      deferred = false;
    } else if (fusion == LA_FUSE_STEP_SYNC && c->tp + 1 == c->H) {
      rc = launch_sweep(c, false, true, true, c->t + 1, c->tp + 1, c->grad_kind, nullptr);  // K3: step t'=H and its sync
      if (rc) return rc;
      c->t += 1; c->tp = 0; c->nsync += 1;
      continue;
    } else {
      rc = la_local_step(c);  // K1
      if (rc) return rc;
    }
    if (c->tp == c->H) {
      if (fusion == LA_FUSE_SYNC_STEP && k + 1 < T) {
        deferred = true;
      } else {
        rc = la_sync(c);  // K2
        if (rc) return rc;
      }
    }
  }
  return LA_OK;
}

// ---- a whole job from and to host memory, pipelined over coordinate ranges --------------------
// Algorithm 3 never mixes coordinates, so [upload, T iterations, download] of one coordinate range
// is independent of every other range: while range k computes on the context's stream, range k+1
// is uploaded on a second stream and range k-1 downloaded on a third.  During a range the
// context simply points at that part of its arrays (same replica stride, shifted coordinate base).
int la_run_streamed(la_ctx* c, uint64_t T, const la_stream_io* io, uint32_t chunks) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!io) return fail(c, LA_EINVAL, "io is NULL");
  if (io->worker >= c->W) return fail(c, LA_EINVAL, "worker %u out of range (W=%u)", io->worker, c->W);
  if (c->grad_kind == la::kGradQuadratic && (!io->a_host != !io->c_host))
    return fail(c, LA_EINVAL, "a_host and c_host come together");
  if (chunks == 0) chunks = 16;
  if (chunks > 4096) chunks = 4096;
  DeviceGuard guard(c->device);
  if (!c->copy_in) LA_CUDA(c, cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking));
  if (!c->copy_out) LA_CUDA(c, cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking));
  if (!c->ev_idle) LA_CUDA(c, cudaEventCreateWithFlags(&c->ev_idle, cudaEventDisableTiming));
  while (c->ev_in.size() < chunks) {
    cudaEvent_t a = nullptr, b = nullptr;
    LA_CUDA(c, cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
    c->ev_in.push_back(a);
    LA_CUDA(c, cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
    c->ev_done.push_back(b);
  }
  // the uploads overwrite the state: whatever the context's stream still does comes first
  LA_CUDA(c, cudaEventRecord(c->ev_idle, c->stream));
  LA_CUDA(c, cudaStreamWaitEvent(c->copy_in, c->ev_idle, 0));

  struct View { float *X, *B2, *Bs, *pa, *pc, *ps; uint64_t N, j_base; } full{c->X, c->B2, c->Bs, c->pa, c->pc, c->ps, c->N, c->j_base};
  const uint64_t per = round_up((full.N + chunks - 1) / chunks, 256);  // whole 1 KiB units: vector accesses stay aligned
  c->shared_iterate = false;
  c->sums_in_replica0 = false;
  int rc = LA_OK;
  uint32_t k = 0;
  for (uint64_t j0 = 0; j0 < full.N && rc == LA_OK; j0 += per, ++k) {
    const uint64_t n = (full.N - j0 < per) ? full.N - j0 : per;
    const bool last = (j0 + n == full.N);
    const uint64_t span = last ? c->stride - j0 : n;  // the last range also owns the padding up to the stride
    const size_t bytes = n * sizeof(float), tail = (span - n) * sizeof(float);
    auto up = [&](float* dst, const float* src) -> cudaError_t {
      cudaError_t e = cudaMemcpyAsync(dst + j0, src + j0, bytes, cudaMemcpyHostToDevice, c->copy_in);
      if (e == cudaSuccess && tail) e = cudaMemsetAsync(dst + j0 + n, 0, tail, c->copy_in);
      return e;
    };
    cudaError_t e = cudaSuccess;
    if (io->x0_host) e = cudaMemcpyAsync(full.X + j0, io->x0_host + j0, bytes, cudaMemcpyHostToDevice, c->copy_in);  // staged in replica 0
    if (e == cudaSuccess && io->a_host) e = up(full.pa, io->a_host);
    if (e == cudaSuccess && io->c_host) e = up(full.pc, io->c_host);
    if (e == cudaSuccess && io->s_host) e = up(full.ps, io->s_host);
    if (e == cudaSuccess) e = cudaEventRecord(c->ev_in[k], c->copy_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->stream, c->ev_in[k], 0);
    if (e != cudaSuccess) { rc = fail(c, LA_ECUDA, "upload of coordinate range %u failed: %s", k, cudaGetErrorString(e)); break; }

    c->X = full.X + j0; c->B2 = full.B2 + j0; c->Bs = full.Bs + j0;
    c->pa = full.pa + j0; c->pc = full.pc + j0; c->ps = full.ps + j0;
    c->N = n; c->j_base = full.j_base + j0;
    c->t = 0; c->tp = 0; c->nsync = 0;
    rc = do_fill(c, io->x0_host ? c->X : nullptr, span);
    if (rc == LA_OK) rc = run_steps(c, T);
    if (rc == LA_OK) rc = import_pending_sums(c);
    if (rc != LA_OK) break;
    e = cudaEventRecord(c->ev_done[k], c->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->copy_out, c->ev_done[k], 0);
    const uint64_t row = (uint64_t)(c->shared_iterate ? 0u : io->worker) * c->stride;
    if (e == cudaSuccess && io->x_host) e = cudaMemcpyAsync(io->x_host + j0, c->X + row, bytes, cudaMemcpyDeviceToHost, c->copy_out);
    if (e == cudaSuccess && io->b2_host) e = cudaMemcpyAsync(io->b2_host + j0, c->B2 + row, bytes, cudaMemcpyDeviceToHost, c->copy_out);
    if (e == cudaSuccess && io->bs_host) e = cudaMemcpyAsync(io->bs_host + j0, c->Bs, bytes, cudaMemcpyDeviceToHost, c->copy_out);
    if (e != cudaSuccess) { rc = fail(c, LA_ECUDA, "download of coordinate range %u failed: %s", k, cudaGetErrorString(e)); break; }
  }
  c->X = full.X; c->B2 = full.B2; c->Bs = full.Bs; c->pa = full.pa; c->pc = full.pc; c->ps = full.ps;
  c->N = full.N; c->j_base = full.j_base;
  if (io->s_host) c->has_s = true;
  // the call returns with the outputs complete and the state resident, like la_read_state
  cudaError_t e1 = cudaStreamSynchronize(c->copy_out), e2 = cudaStreamSynchronize(c->stream);
  if (rc != LA_OK) return rc;
  if (e1 != cudaSuccess || e2 != cudaSuccess) return fail(c, LA_ECUDA, "stream synchronisation failed: %s", cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
  return debug_poll(c);
}

// ---- state access ----------------------------------------------------------------------------
int la_read_range(la_ctx* c, uint32_t worker, uint64_t j0, uint64_t n, float* x_host, float* b2_host, float* bs_host) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (worker >= c->W) return fail(c, LA_EINVAL, "worker %u out of range (W=%u)", worker, c->W);
  if (j0 > c->N || n > c->N - j0) return fail(c, LA_EINVAL, "coordinate range out of bounds");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  if (c->shared_iterate) worker = 0;  // Algorithm 1: every worker holds the one iterate, stored in replica 0
  const size_t bytes = n * sizeof(float);
  if (n) {
    if (x_host) LA_CUDA(c, cudaMemcpyAsync(x_host, c->X + (uint64_t)worker * c->stride + j0, bytes, cudaMemcpyDeviceToHost, c->stream));
    if (b2_host) LA_CUDA(c, cudaMemcpyAsync(b2_host, c->B2 + (uint64_t)worker * c->stride + j0, bytes, cudaMemcpyDeviceToHost, c->stream));
    if (bs_host) LA_CUDA(c, cudaMemcpyAsync(bs_host, c->Bs + j0, bytes, cudaMemcpyDeviceToHost, c->stream));
  }
  LA_CUDA(c, cudaStreamSynchronize(c->stream));
  return debug_poll(c);
}

int la_read_state(la_ctx* c, uint32_t worker, float* x_host, float* b2_host, float* bs_host) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  return la_read_range(c, worker, 0, c->N, x_host, b2_host, bs_host);
}

int la_write_state(la_ctx* c, uint32_t worker, const float* x_host, const float* b2_host, const float* bs_host) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (worker >= c->W) return fail(c, LA_EINVAL, "worker %u out of range (W=%u)", worker, c->W);
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  if (x_host || b2_host) {
    int rc = materialise_replicas(c);  // a per-worker write: the replicas become individual again
    if (rc) return rc;
  }
  const size_t bytes = c->N * sizeof(float);
  if (x_host) LA_CUDA(c, cudaMemcpyAsync(c->X + (uint64_t)worker * c->stride, x_host, bytes, cudaMemcpyHostToDevice, c->stream));
  if (b2_host) LA_CUDA(c, cudaMemcpyAsync(c->B2 + (uint64_t)worker * c->stride, b2_host, bytes, cudaMemcpyHostToDevice, c->stream));
  if (bs_host) LA_CUDA(c, cudaMemcpyAsync(c->Bs, bs_host, bytes, cudaMemcpyHostToDevice, c->stream));
  LA_CUDA(c, cudaStreamSynchronize(c->stream));
  return LA_OK;
}

int la_tensor_range(const la_ctx* c, uint32_t k, uint64_t* offset, uint64_t* size) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (k >= c->sizes.size()) return fail(const_cast<la_ctx*>(c), LA_EINVAL, "tensor %u out of range", k);
  if (offset) *offset = c->offsets[k];
  if (size) *size = c->sizes[k];
  return LA_OK;
}

int la_get_counters(const la_ctx* c, uint64_t* t, uint32_t* t_prime, uint64_t* n_sync) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (t) *t = c->t;
  if (t_prime) *t_prime = c->tp;
  if (n_sync) *n_sync = c->nsync;
  return LA_OK;
}

int la_set_counters(la_ctx* c, uint64_t t, uint32_t t_prime, uint64_t n_sync) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  c->t = t; c->tp = t_prime; c->nsync = n_sync;
  return LA_OK;
}

int la_get_stats(la_ctx* c, la_stats* out, int reset) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!out) return fail(c, LA_EINVAL, "out is NULL");
  DeviceGuard guard(c->device);
  int rc = drain_events(c);
  if (rc) return rc;
  *out = c->stats;
  if (reset) c->stats = la_stats{};
  return debug_poll(c);
}

// ---- sharding by worker -------------------------------------------------------------------
int la_set_worker_range(la_ctx* c, uint32_t worker_base, uint32_t W_total) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (W_total == 0) { c->worker_base = 0; c->W_total = 0; return LA_OK; }
  if ((uint64_t)worker_base + c->W > W_total) return fail(c, LA_EINVAL, "worker range exceeds W_total");
  c->worker_base = worker_base; c->W_total = W_total;
  return LA_OK;
}

int la_comm_create(la_ctx* c, uint32_t rank, uint32_t world) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (world == 0 || world > la::kMaxRanks || rank >= world) return fail(c, LA_EINVAL, "need rank < world <= %d", la::kMaxRanks);
  if (c->rule != LA_RULE_ADAALTER) return fail(c, LA_ESTATE, "sharding by worker is implemented for Local AdaAlter only");
  // "tree over the local replicas, then tree over the ranks" is the adjacent-pair tree over all
  // workers only when every rank contributes a full power-of-two block of leaves
  if (world > 1 && (c->W & (c->W - 1)) != 0)
    return fail(c, LA_EINVAL, "with more than one rank the local worker count must be a power of two (W=%u)", c->W);
  DeviceGuard guard(c->device);
  if (!c->S) {
    cudaError_t e = cudaMalloc((void**)&c->S, 2 * c->stride * sizeof(float));
    if (e != cudaSuccess) { c->S = nullptr; cudaGetLastError(); return fail(c, LA_ENOMEM, "cudaMalloc of the exchange buffer failed: %s", cudaGetErrorString(e)); }
    LA_CUDA(c, cudaMemsetAsync(c->S, 0, 2 * c->stride * sizeof(float), c->stream));
  }
  c->rank = rank; c->world = world;
  for (auto& q : c->peerS) q = nullptr;
  c->peerS[rank] = c->S;
  if (c->W_total == 0) { c->W_total = c->W * world; c->worker_base = c->W * rank; }
  return LA_OK;
}

int la_comm_buffer(la_ctx* c, void** dev_ptr, uint64_t* bytes) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  if (dev_ptr) *dev_ptr = c->S;
  if (bytes) *bytes = 2 * c->stride * sizeof(float);
  return LA_OK;
}

int la_comm_ipc_handle(la_ctx* c, void* handle64) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  if (!handle64) return fail(c, LA_EINVAL, "handle buffer is NULL");
  static_assert(sizeof(cudaIpcMemHandle_t) == 64, "IPC handle size");
  DeviceGuard guard(c->device);
  cudaIpcMemHandle_t h;
  LA_CUDA(c, cudaIpcGetMemHandle(&h, c->S));
  std::memcpy(handle64, &h, sizeof h);
  return LA_OK;
}

int la_comm_set_peer(la_ctx* c, uint32_t peer_rank, void* dev_ptr) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  if (peer_rank >= c->world || peer_rank == c->rank || !dev_ptr) return fail(c, LA_EINVAL, "bad peer rank or pointer");
  c->peerS[peer_rank] = (float*)dev_ptr;
  return LA_OK;
}

int la_comm_open_peer(la_ctx* c, uint32_t peer_rank, const void* handle64) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  if (peer_rank >= c->world || peer_rank == c->rank || !handle64) return fail(c, LA_EINVAL, "bad peer rank or handle");
  DeviceGuard guard(c->device);
  cudaIpcMemHandle_t h;
  std::memcpy(&h, handle64, sizeof h);
  void* mapped = nullptr;
  LA_CUDA(c, cudaIpcOpenMemHandle(&mapped, h, cudaIpcMemLazyEnablePeerAccess));
  if (c->ipc_opened[peer_rank]) cudaIpcCloseMemHandle(c->ipc_opened[peer_rank]);
  c->ipc_opened[peer_rank] = mapped;
  c->peerS[peer_rank] = (float*)mapped;
  return LA_OK;
}

int la_comm_export(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  return launch_sweep(c, true, false, false, c->t, 0, la::kGradNoise, nullptr, 1);
}

int la_comm_combine(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  DeviceGuard guard(c->device);
  la::CombineParams p{};
  for (uint32_t r = 0; r < c->world; ++r) {
    if (!c->peerS[r]) return fail(c, LA_ESTATE, "exchange buffer of rank %u not attached", r);
    p.S[r] = c->peerS[r];
  }
  p.stride = c->stride; p.world = c->world;
  const uint64_t units = c->stride / 64;
  p.slice_lo = units * c->rank / c->world * 64;
  p.slice_hi = units * (c->rank + 1) / c->world * 64;
  if (p.slice_hi > p.slice_lo) {
    const uint64_t groups = (p.slice_hi - p.slice_lo) / kExchangeVecHost;
    uint64_t blocks = (groups + la::kBlockThreads - 1) / la::kBlockThreads;
    const uint64_t cap = (uint64_t)c->num_sms * 4096;
    if (blocks > cap) blocks = cap;
    la::la_combine_sums<la::kExchangeVec><<<(unsigned)blocks, la::kBlockThreads, 0, c->stream>>>(p);
    LA_CUDA(c, cudaGetLastError());
    c->stats.launches_other++;
  }
  return LA_OK;
}

int la_comm_import(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  int rc = launch_sweep(c, true, false, false, c->t, 0, la::kGradNoise, nullptr, 2);
  if (rc) return rc;
  c->tp = 0; c->nsync += 1;
  return LA_OK;
}

static int step_export_impl(la_ctx* c, int gm, const void* gext) {
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  if (c->rule != LA_RULE_ADAALTER) return fail(c, LA_ESTATE, "sharding by worker is implemented for Local AdaAlter only");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  int rc = launch_sweep(c, false, true, true, c->t + 1, c->tp + 1, gm, gext, 1);
  if (rc) return rc;
  c->t += 1; c->tp += 1;
  return LA_OK;
}

int la_comm_step_export(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  return step_export_impl(c, c->grad_kind, nullptr);
}

int la_comm_step_grads_export(la_ctx* c, const void* g_dev, int dtype) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!g_dev) return fail(c, LA_EINVAL, "g_dev is NULL");
  if (dtype != LA_F32 && dtype != LA_BF16) return fail(c, LA_EINVAL, "dtype must be LA_F32 or LA_BF16");
  return step_export_impl(c, dtype == LA_F32 ? la::kGradExternalF32 : la::kGradExternalBF16, g_dev);
}

int la_comm_import_step(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  if (c->rule != LA_RULE_ADAALTER) return fail(c, LA_ESTATE, "sharding by worker is implemented for Local AdaAlter only");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  int rc = launch_sweep(c, true, true, false, c->t + 1, 1u, c->grad_kind, nullptr, 2);
  if (rc) return rc;
  c->nsync += 1; c->t += 1; c->tp = 1;
  return LA_OK;
}

int la_comm_import_step_grads(la_ctx* c, const void* g_dev, int dtype) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  if (!c->S) return fail(c, LA_ESTATE, "call la_comm_create first");
  if (!g_dev) return fail(c, LA_EINVAL, "g_dev is NULL");
  if (dtype != LA_F32 && dtype != LA_BF16) return fail(c, LA_EINVAL, "dtype must be LA_F32 or LA_BF16");
  if (c->rule != LA_RULE_ADAALTER) return fail(c, LA_ESTATE, "sharding by worker is implemented for Local AdaAlter only");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  int rc = launch_sweep(c, true, true, false, c->t + 1, 1u, dtype == LA_F32 ? la::kGradExternalF32 : la::kGradExternalBF16,
                        g_dev, 2);
  if (rc) return rc;
  c->nsync += 1; c->t += 1; c->tp = 1;
  return LA_OK;
}

int la_diagnostics(la_ctx* c, double* objective, double* replica_spread) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  DeviceGuard guard(c->device);
  { int rc_ = import_pending_sums(c); if (rc_) return rc_; }
  if (!c->diag) {
    cudaError_t e = cudaMalloc((void**)&c->diag, 2 * sizeof(double));
    if (e != cudaSuccess) { c->diag = nullptr; cudaGetLastError(); return fail(c, LA_ENOMEM, "cudaMalloc failed: %s", cudaGetErrorString(e)); }
  }
  LA_CUDA(c, cudaMemsetAsync(c->diag, 0, 2 * sizeof(double), c->stream));
  const bool quad = c->grad_kind == la::kGradQuadratic;
  const uint32_t W = c->shared_iterate ? 1u : c->W;  // after AdaGrad steps all workers hold replica 0's iterate
  uint64_t blocks = (c->N + la::kBlockThreads - 1) / la::kBlockThreads;
  const uint64_t cap = (uint64_t)c->num_sms * 16;
  if (blocks > cap) blocks = cap;
  la::la_diagnostics<<<(unsigned)blocks, la::kBlockThreads, 0, c->stream>>>(c->X, quad ? c->pa : nullptr, c->pc, c->N,
                                                                             c->stride, W, c->diag);
  LA_CUDA(c, cudaGetLastError());
  c->stats.launches_other++;
  double host[2] = {0, 0};
  LA_CUDA(c, cudaMemcpyAsync(host, c->diag, sizeof host, cudaMemcpyDeviceToHost, c->stream));
  LA_CUDA(c, cudaStreamSynchronize(c->stream));
  if (objective) *objective = quad ? host[0] : NAN;
  if (replica_spread) *replica_spread = host[1];
  return LA_OK;
}

int la_noise_tables(float* radius_dev, float* cos_dev, float* sin_dev, void* stream) {
  if (!radius_dev && !cos_dev && !sin_dev) return LA_OK;
  la::la_noise_tables_kernel<<<148 * 8, 256, 0, (cudaStream_t)stream>>>(radius_dev, cos_dev, sin_dev);
  if (cudaGetLastError() != cudaSuccess) return fail(nullptr, LA_ECUDA, "launch of the table kernel failed");
  return LA_OK;
}

int la_stream_sync(la_ctx* c) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
  DeviceGuard guard(c->device);
  LA_CUDA(c, cudaStreamSynchronize(c->stream));
  return debug_poll(c);
}

int la_debug_build(void) {
#ifdef LA_DEBUG
  return 1;
#else
  return 0;
#endif
}

int la_debug_narrow(la_ctx* c, uint64_t bytes) {
  if (!c) return fail(nullptr, LA_EINVAL, "ctx is NULL");
#ifdef LA_DEBUG
  if (bytes > c->arena_size) return fail(c, LA_EINVAL, "more than the arena holds");
  c->dbg_narrow = bytes;
  return LA_OK;
#else
  (void)bytes;
  return fail(c, LA_ESTATE, "this is not the checked build (compile with -DLA_DEBUG)");
#endif
}

}  // extern "C"
