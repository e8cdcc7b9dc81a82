// Local AdaAlter reference oracle (CPU, single-threaded, deliberately plain).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct
// restatement of Algorithm 3 ("Local AdaAlter") of arXiv 1911.09030 that the
// CUDA library is checked against.  It shares no code, header, table or
// constant generator with the CUDA path; only tests, the smoke check and the
// benchmark's CPU-baseline leg may load it.  Nothing here is tuned.
//
// What follows the paper and where:
//   * initialisation x_{i,0}=x_0, B^2_{i,0}=b_0^2 1           Algorithm 3, init line
//   * t' = mod(t-1,H)+1, kept as "local steps since last sync"  Algorithm 3
//   * G_{i,t} evaluated at the worker's own x_{i,t-1}           Algorithm 3
//   * y = x - eta*G/sqrt(B^2_{i,t-t'} + t' eps^2)               Algorithm 3
//   * A^2 = B^2_{i,t-1} + G o G                                 Algorithm 3
//   * every H steps: x, B^2 <- mean over workers of y, A^2      Algorithm 3
//   * the denominator B^2_{i,t-t'} is the accumulator as of the last
//     synchronisation and is the same on every worker          Section 4.2,
//     "Lazy update of the denominators"; Appendix A (definition of B-bar)
//   * warm-up eta_t = eta*min(1, t/warm_up_steps)               Section 6.2
//   * baselines: Distributed AdaGrad (Algorithm 1), Local SGD (Algorithm 2)
//
// Two state copies advance side by side:
//   fp32 : the arithmetic contract (one IEEE-754 binary32 operation per line
//          below, fused multiply-add only where fmaf is written);
//   fp64 : a "shadow" that evaluates the paper's formulas literally in
//          double, on the same fp32 noise draws but its own state.
//
// The synthetic stochastic gradient (noise xi, diagonal quadratic) is not from
// the paper; it is a counter-based generator defined in prose in the design
// document and implemented here from that prose: splitmix64 finaliser keyed
// on (seed, step, worker, coordinate pair) -> two 24-bit uniforms ->
// Box-Muller with ln / sin / cos given by fixed fp32 polynomial recipes.
//
// Parity pins (tests, "not gpu"): hand-worked Algorithm-3 case, independent
// brute-force fp64 script, closed forms for constant gradients, H=1 / W=1 /
// identical-worker reductions, accumulator identity, mean-iterate recursion,
// exhaustive accuracy scans of the ln and sin/cos recipes against libm in
// double, published splitmix64 outputs, distribution tests of xi.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

namespace {

// ---------------------------------------------------------------- bit casts
inline uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float u2f(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// ------------------------------------------------------------ splitmix64 mix
// Output function of the splitmix64 generator (Steele, Lea, Flood 2014;
// Vigna's public-domain description): xor-shift 30, multiply, xor-shift 27,
// multiply, xor-shift 31, all modulo 2^64.
const uint64_t kGamma = 0x9E3779B97F4A7C15ull;  // golden-ratio increment

uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Stream key of (step t >= 1, worker i): k_t = M(seed + gamma*t),
// k_{t,i} = M(k_t + gamma*(i+1)).
uint64_t stream_key(uint64_t seed, uint64_t t, uint32_t worker) {
  uint64_t kt = mix64(seed + kGamma * t);
  return mix64(kt + kGamma * (uint64_t)(worker + 1));
}

// --------------------------------------------------------- -2 ln(u1) recipe
// u1 = k * 2^-24 with integer k in [1, 2^24].  Returns L ~= -2 ln(u1) >= 0.
// Steps: f = (float)k (exact); split f = m * 2^e with m in [sqrt(1/2), sqrt 2)
// by integer arithmetic on the bit pattern; t = m - 1 (exact);
// -2 ln m ~= -2 t + t^2 Q(t), Q a fixed degree-7 polynomial (Horner, fmaf);
// L = fma(24 - e, 2 ln 2, -2 ln m).
float neg2ln_u24(uint32_t k) {
  const uint32_t kSqrtHalfBits = 0x3F3504F3u;  // bit pattern of fl32(sqrt(1/2))
  float f = (float)k;
  uint32_t d = f2u(f) - kSqrtHalfBits;
  int e = (int)(d >> 23);                      // f >= 1 so d is non-negative
  float m = u2f((d & 0x007FFFFFu) + kSqrtHalfBits);
  float t = m - 1.0f;
  float q = -0x1.70cfe8p-3f;
  q = std::fmaf(q, t, 0x1.23ffe8p-2f);
  q = std::fmaf(q, t, -0x1.2f3c7ep-2f);
  q = std::fmaf(q, t, 0x1.5374fcp-2f);
  q = std::fmaf(q, t, -0x1.990c98p-2f);
  q = std::fmaf(q, t, 0x1.000438p-1f);
  q = std::fmaf(q, t, -0x1.555630p-1f);
  q = std::fmaf(q, t, 0x1.fffffcp-1f);
  float t2 = t * t;
  float lm = std::fmaf(t2, q, -2.0f * t);
  float ne = (float)(24 - e);
  return std::fmaf(ne, 0x1.62e430p+0f /* fl32(2 ln 2) */, lm);
}

// ------------------------------------------------- cos/sin(2 pi q / 2^24)
// q is a 24-bit integer.  Octant o = top 3 bits; r = low 21 bits, reflected to
// 2^21 - r in odd octants (exact); x = (float)r * fl32(pi) * 2^-23 in [0, pi/4];
// sin x ~= x + x*x2*S(x2), cos x ~= 1 + x2*C(x2) with fixed polynomials;
// octant symmetries restore cos and sin of the full angle.
void cossin_u24(uint32_t q, float* c_out, float* s_out) {
  uint32_t o = q >> 21;
  uint32_t r = q & 0x1FFFFFu;
  if (o & 1u) r = 0x200000u - r;
  float x = (float)r * 0x1.921fb6p-22f;
  float x2 = x * x;
  float sp = -0x1.9ac9fep-13f;
  sp = std::fmaf(sp, x2, 0x1.110c2ap-7f);
  sp = std::fmaf(sp, x2, -0x1.555552p-3f);
  float sn = std::fmaf(x * x2, sp, x);
  float cp = 0x1.9a6efep-16f;
  cp = std::fmaf(cp, x2, -0x1.6c0e08p-10f);
  cp = std::fmaf(cp, x2, 0x1.55554cp-5f);
  cp = std::fmaf(cp, x2, -0x1.000000p-1f);
  float cs = std::fmaf(x2, cp, 1.0f);
  // octant table (theta = o*pi/4 + x for even o, (o+1)*pi/4 - x for odd o)
  float c, s;
  switch (o) {
    case 0: c = cs;  s = sn;  break;
    case 1: c = sn;  s = cs;  break;
    case 2: c = -sn; s = cs;  break;
    case 3: c = -cs; s = sn;  break;
    case 4: c = -cs; s = -sn; break;
    case 5: c = -sn; s = -cs; break;
    case 6: c = sn;  s = -cs; break;
    default: c = cs; s = -sn; break;
  }
  *c_out = c;
  *s_out = s;
}

// ------------------------------------------------------ Box-Muller pair draw
// One 64-bit draw z per coordinate PAIR p = j >> 1 (j = global coordinate):
//   z  = M(key + gamma*(p+1)),
//   u1 = ((z >> 40) + 1) * 2^-24 in (0,1],  u2 = ((z >> 8) & 0xFFFFFF) * 2^-24,
//   R  = sqrt(-2 ln u1),  xi(even j) = R cos(2 pi u2),  xi(odd j) = R sin(2 pi u2).
void noise_pair(uint64_t key, uint64_t p, float* xi_even, float* xi_odd) {
  uint64_t z = mix64(key + kGamma * (p + 1));
  uint32_t k = (uint32_t)(z >> 40) + 1u;
  uint32_t q = (uint32_t)(z >> 8) & 0xFFFFFFu;
  float R = std::sqrt(neg2ln_u24(k));
  float c, s;
  cossin_u24(q, &c, &s);
  *xi_even = R * c;
  *xi_odd = R * s;
}

float noise_xi(uint64_t key, uint64_t j) {
  float a, b;
  noise_pair(key, j >> 1, &a, &b);
  return (j & 1) ? b : a;
}

// ------------------------------------------- bf16 round-to-nearest-even, widened
float bf16_round(float g) {
  uint32_t u = f2u(g);
  u += 0x7FFFu + ((u >> 16) & 1u);
  u &= 0xFFFF0000u;
  return u2f(u);
}

// ------------------------------------------------------------ pairwise tree
// Sum over workers: adjacent pairs, level by level; an odd element at a level
// is carried up unchanged.  (W=4: (v0+v1)+(v2+v3).)
template <typename T>
T tree_sum(std::vector<T>& v) {
  size_t n = v.size();
  while (n > 1) {
    size_t o = 0;
    for (size_t k = 0; k + 1 < n; k += 2) v[o++] = v[k] + v[k + 1];
    if (n & 1) v[o++] = v[n - 1];
    n = o;
  }
  return v[0];
}

enum GradMode { kNoise = 0, kQuadratic = 1, kConstant = 2 };
enum Rule { kRuleAdaAlter = 0, kRuleLocalSGD = 1, kRuleAdaGrad = 2 };

struct Oracle {
  uint64_t n = 0;        // coordinates simulated here
  uint64_t j_base = 0;   // global index of local coordinate 0
  uint32_t W = 0, H = 0;
  float eta = 0, eps = 0, b0sq = 0;
  uint32_t warm_up_steps = 0;  // 0 = no warm-up
  int rule = kRuleAdaAlter;    // Algorithm 3 by default; Algorithms 1 and 2 as baselines
  // gradient source
  int mode = kNoise;
  uint64_t seed = 0;
  float sigma = 0;
  bool bf16 = false;
  bool identical_workers = false;
  uint32_t worker_base = 0;    // global index of local worker 0 (workers sharded over ranks)
  std::vector<float> a, c, s;  // s empty => s == 1
  // state, fp32
  std::vector<float> X, B2, Bs;  // X,B2: [W][n]; Bs: [n]
  // state, fp64 shadow
  std::vector<double> Xd, B2d, Bsd;
  uint64_t t = 0;
  uint32_t tp = 0;
  uint64_t nsync = 0;

  float eta_t() const {  // Section 6.2 warm-up
    if (warm_up_steps == 0) return eta;
    float ratio = (float)t / (float)warm_up_steps;
    return eta * std::fmin(1.0f, ratio);
  }
  double eta_t_d() const {
    if (warm_up_steps == 0) return (double)eta;
    double ratio = (double)t / (double)warm_up_steps;
    return (double)eta * std::fmin(1.0, ratio);
  }

  // Stochastic gradient G_{i,t} of worker i at coordinate j, evaluated at the iterate stored at
  // index ix (fp32: g from X[ix]; shadow: gd from Xd[ix]).  `gext` prescribes it instead.
  void gradient(uint32_t i, uint64_t j, size_t ix, uint64_t key_i, const float* gext, float* g_out,
                double* gd_out) const {
    float g;
    double gd;
    if (gext) {
      g = gext[(size_t)i * n + j];
      gd = (double)g;
    } else if (mode == kConstant) {
      g = s.empty() ? 1.0f : s[j];
      gd = (double)g;
    } else {
      float xi = noise_xi(key_i, j_base + j);
      if (mode == kNoise) {
        g = s.empty() ? xi : s[j] * xi;
        gd = s.empty() ? (double)xi : (double)s[j] * (double)xi;
      } else {
        float dlt = X[ix] - c[j];
        float nz = sigma * xi;
        g = std::fmaf(a[j], dlt, nz);
        gd = (double)a[j] * (Xd[ix] - (double)c[j]) + (double)sigma * (double)xi;
      }
      if (bf16) {
        g = bf16_round(g);
        gd = (double)bf16_round((float)gd);
      }
    }
    *g_out = g;
    *gd_out = gd;
  }

  std::vector<uint64_t> step_keys() const {
    std::vector<uint64_t> key(W);
    for (uint32_t i = 0; i < W; ++i) key[i] = stream_key(seed, t, identical_workers ? 0u : worker_base + i);
    return key;
  }

  // One iteration of Algorithm 3 without the synchronisation branch.
  // `gext` (optional) supplies G_{i,t} as a [W][n] table instead of the source.
  void adaalter_step(const float* gext) {
    t += 1;
    tp += 1;
    const float eps2 = eps * eps;
    const float et = eta_t();
    const double etd = eta_t_d();
    const double eps2d = (double)eps * (double)eps;
    const std::vector<uint64_t> key = step_keys();
    for (uint64_t j = 0; j < n; ++j) {
      // shared, stale denominator: B^2 as of the last sync + t' eps^2
      float q = (float)tp * eps2;
      float d = Bs[j] + q;
      float r = et / std::sqrt(d);
      double dd = Bsd[j] + (double)tp * eps2d;
      for (uint32_t i = 0; i < W; ++i) {
        size_t ix = (size_t)i * n + j;
        float g;
        double gd;
        gradient(i, j, ix, key[i], gext, &g, &gd);
        X[ix] = std::fmaf(-r, g, X[ix]);     // y = x - eta G / sqrt(.)
        B2[ix] = std::fmaf(g, g, B2[ix]);    // A^2 = B^2 + G o G
        Xd[ix] = Xd[ix] - etd * gd / std::sqrt(dd);
        B2d[ix] = B2d[ix] + gd * gd;
      }
    }
  }

  // One iteration of Algorithm 2 (Local SGD) without its averaging branch:
  // y_{i,t} = x_{i,t-1} - eta G_{i,t}.  No accumulator is kept.
  void local_sgd_step(const float* gext) {
    t += 1;
    tp += 1;
    const float et = eta_t();
    const double etd = eta_t_d();
    const std::vector<uint64_t> key = step_keys();
    for (uint64_t j = 0; j < n; ++j)
      for (uint32_t i = 0; i < W; ++i) {
        size_t ix = (size_t)i * n + j;
        float g;
        double gd;
        gradient(i, j, ix, key[i], gext, &g, &gd);
        X[ix] = std::fmaf(-et, g, X[ix]);
        Xd[ix] = Xd[ix] - etd * gd;
      }
  }

  // One iteration of Algorithm 1 (Distributed AdaGrad): every worker evaluates its gradient at
  // the common iterate x_{t-1}; G_t = (1/n) sum_i G_{i,t}; B^2_t = B^2_{t-1} + G_t o G_t;
  // x_t = x_{t-1} - eta G_t / sqrt(B^2_t + eps^2)  (the UPDATED accumulator).  All replicas
  // stay equal; one gradient exchange per iteration is counted in nsync.
  void adagrad_step(const float* gext) {
    t += 1;
    const float eps2 = eps * eps;
    const float et = eta_t();
    const double etd = eta_t_d();
    const double eps2d = (double)eps * (double)eps;
    const std::vector<uint64_t> key = step_keys();
    std::vector<float> vg(W);
    for (uint64_t j = 0; j < n; ++j) {
      double gsum = 0;
      for (uint32_t i = 0; i < W; ++i) {
        float g;
        double gd;
        gradient(i, j, j /* replica 0 holds the common iterate */, key[i], gext, &g, &gd);
        vg[i] = g;
        gsum += gd;
      }
      float gm = tree_sum(vg) / (float)W;
      double gmd = gsum / (double)W;
      float b = std::fmaf(gm, gm, B2[j]);
      float d = b + eps2;
      float r = et / std::sqrt(d);
      float x = std::fmaf(-r, gm, X[j]);
      double bd = B2d[j] + gmd * gmd;
      double xd = Xd[j] - etd * gmd / std::sqrt(bd + eps2d);
      for (uint32_t i = 0; i < W; ++i) {
        size_t ix = (size_t)i * n + j;
        X[ix] = x; B2[ix] = b; Xd[ix] = xd; B2d[ix] = bd;
      }
      Bs[j] = b;
      Bsd[j] = bd;
    }
    nsync += 1;
  }

  void local_step(const float* gext) {
    if (rule == kRuleLocalSGD) local_sgd_step(gext);
    else if (rule == kRuleAdaGrad) adagrad_step(gext);
    else adaalter_step(gext);
  }

  // Synchronisation branch of Algorithm 3: means of y and A^2 over workers
  // replace every worker's x and B^2; the mean B^2 becomes the stale denominator.
  // (Algorithm 2's averaging branch is the same with the accumulator left out.)
  void sync() {
    if (rule == kRuleLocalSGD) { sync_x_only(); return; }
    std::vector<float> vx(W), vb(W);
    std::vector<double> vxd(W), vbd(W);
    for (uint64_t j = 0; j < n; ++j) {
      for (uint32_t i = 0; i < W; ++i) {
        vx[i] = X[(size_t)i * n + j];
        vb[i] = B2[(size_t)i * n + j];
      }
      float xm = tree_sum(vx) / (float)W;
      float bm = tree_sum(vb) / (float)W;
      double xs = 0, bs = 0;
      for (uint32_t i = 0; i < W; ++i) {
        xs += Xd[(size_t)i * n + j];
        bs += B2d[(size_t)i * n + j];
      }
      double xmd = xs / (double)W, bmd = bs / (double)W;
      for (uint32_t i = 0; i < W; ++i) {
        X[(size_t)i * n + j] = xm;
        B2[(size_t)i * n + j] = bm;
        Xd[(size_t)i * n + j] = xmd;
        B2d[(size_t)i * n + j] = bmd;
      }
      Bs[j] = bm;
      Bsd[j] = bmd;
    }
    tp = 0;
    nsync += 1;
  }

  // Algorithm 2, else-branch: x_{i,t} = (1/n) sum_k y_{k,t}.
  void sync_x_only() {
    std::vector<float> vx(W);
    for (uint64_t j = 0; j < n; ++j) {
      for (uint32_t i = 0; i < W; ++i) vx[i] = X[(size_t)i * n + j];
      float xm = tree_sum(vx) / (float)W;
      double xs = 0;
      for (uint32_t i = 0; i < W; ++i) xs += Xd[(size_t)i * n + j];
      double xmd = xs / (double)W;
      for (uint32_t i = 0; i < W; ++i) {
        X[(size_t)i * n + j] = xm;
        Xd[(size_t)i * n + j] = xmd;
      }
    }
    tp = 0;
    nsync += 1;
  }

  void run(uint64_t T) {
    for (uint64_t k = 0; k < T; ++k) {
      local_step(nullptr);
      if (rule != kRuleAdaGrad && tp == H) sync();
    }
  }
};

}  // namespace

// ------------------------------------------------------------------ C surface
extern "C" {

void* ora_create(uint64_t n, uint64_t j_base, uint32_t W, float eta, float eps,
                 uint32_t H, float b0sq, const float* x0 /* n or NULL */) {
  if (n == 0 || W == 0 || H == 0 || !(eps > 0.0f) || !std::isfinite(eta)) return nullptr;
  Oracle* o = new (std::nothrow) Oracle();
  if (!o) return nullptr;
  o->n = n; o->j_base = j_base; o->W = W; o->H = H;
  o->eta = eta; o->eps = eps; o->b0sq = b0sq;
  o->X.resize((size_t)W * n); o->B2.assign((size_t)W * n, b0sq); o->Bs.assign(n, b0sq);
  o->Xd.resize((size_t)W * n); o->B2d.assign((size_t)W * n, (double)b0sq);
  o->Bsd.assign(n, (double)b0sq);
  for (uint32_t i = 0; i < W; ++i)
    for (uint64_t j = 0; j < n; ++j) {
      float v = x0 ? x0[j] : 0.0f;
      o->X[(size_t)i * n + j] = v;
      o->Xd[(size_t)i * n + j] = (double)v;
    }
  return o;
}

void ora_destroy(void* h) { delete (Oracle*)h; }

void ora_set_grad_noise(void* h, uint64_t seed, const float* s /* n or NULL */) {
  Oracle* o = (Oracle*)h;
  o->mode = kNoise; o->seed = seed;
  if (s) o->s.assign(s, s + o->n); else o->s.clear();
}
void ora_set_grad_quadratic(void* h, uint64_t seed, const float* a, const float* c, float sigma) {
  Oracle* o = (Oracle*)h;
  o->mode = kQuadratic; o->seed = seed; o->sigma = sigma;
  o->a.assign(a, a + o->n); o->c.assign(c, c + o->n);
}
void ora_set_grad_constant(void* h, const float* s /* n or NULL => 1 */) {
  Oracle* o = (Oracle*)h;
  o->mode = kConstant;
  if (s) o->s.assign(s, s + o->n); else o->s.clear();
}
void ora_set_grad_bf16(void* h, int on) { ((Oracle*)h)->bf16 = on != 0; }
void ora_set_identical_workers(void* h, int on) { ((Oracle*)h)->identical_workers = on != 0; }
void ora_set_warmup(void* h, uint32_t steps) { ((Oracle*)h)->warm_up_steps = steps; }
void ora_set_rule(void* h, int rule) { ((Oracle*)h)->rule = rule; }
void ora_set_worker_base(void* h, uint32_t base) { ((Oracle*)h)->worker_base = base; }

void ora_local_step(void* h) { ((Oracle*)h)->local_step(nullptr); }
void ora_local_step_grads(void* h, const float* g /* [W][n] */) { ((Oracle*)h)->local_step(g); }
void ora_sync(void* h) { ((Oracle*)h)->sync(); }
void ora_run(void* h, uint64_t T) { ((Oracle*)h)->run(T); }

void ora_read(void* h, uint32_t worker, float* x, float* b2, float* bs) {
  Oracle* o = (Oracle*)h;
  size_t off = (size_t)worker * o->n;
  if (x) std::memcpy(x, o->X.data() + off, o->n * 4);
  if (b2) std::memcpy(b2, o->B2.data() + off, o->n * 4);
  if (bs) std::memcpy(bs, o->Bs.data(), o->n * 4);
}
void ora_read_shadow(void* h, uint32_t worker, double* x, double* b2, double* bs) {
  Oracle* o = (Oracle*)h;
  size_t off = (size_t)worker * o->n;
  if (x) std::memcpy(x, o->Xd.data() + off, o->n * 8);
  if (b2) std::memcpy(b2, o->B2d.data() + off, o->n * 8);
  if (bs) std::memcpy(bs, o->Bsd.data(), o->n * 8);
}
void ora_write(void* h, uint32_t worker, const float* x, const float* b2, const float* bs) {
  Oracle* o = (Oracle*)h;
  size_t off = (size_t)worker * o->n;
  for (uint64_t j = 0; j < o->n; ++j) {
    if (x) { o->X[off + j] = x[j]; o->Xd[off + j] = (double)x[j]; }
    if (b2) { o->B2[off + j] = b2[j]; o->B2d[off + j] = (double)b2[j]; }
    if (bs) { o->Bs[j] = bs[j]; o->Bsd[j] = (double)bs[j]; }
  }
}
void ora_get_counters(void* h, uint64_t* t, uint32_t* tp, uint64_t* nsync) {
  Oracle* o = (Oracle*)h;
  if (t) *t = o->t;
  if (tp) *tp = o->tp;
  if (nsync) *nsync = o->nsync;
}
void ora_set_counters(void* h, uint64_t t, uint32_t tp, uint64_t nsync) {
  Oracle* o = (Oracle*)h;
  o->t = t; o->tp = tp; o->nsync = nsync;
}

// ---- gradient-source primitives, exposed so tests can pin each one ----
uint64_t ora_mix64(uint64_t z) { return mix64(z); }
uint64_t ora_stream_key(uint64_t seed, uint64_t t, uint32_t worker) { return stream_key(seed, t, worker); }
float ora_neg2ln_u24(uint32_t k) { return neg2ln_u24(k); }
void ora_cossin_u24(uint32_t q, float* c, float* s) { cossin_u24(q, c, s); }
float ora_bf16_round(float g) { return bf16_round(g); }
void ora_noise_fill(uint64_t seed, uint64_t t, uint32_t worker, uint64_t j0, uint64_t n, float* out) {
  uint64_t key = stream_key(seed, t, worker);
  for (uint64_t j = 0; j < n; ++j) out[j] = noise_xi(key, j0 + j);
}
void ora_uniform_bits(uint64_t seed, uint64_t t, uint32_t worker, uint64_t p, uint32_t* k, uint32_t* q) {
  uint64_t z = mix64(stream_key(seed, t, worker) + kGamma * (p + 1));
  *k = (uint32_t)(z >> 40) + 1u;
  *q = (uint32_t)(z >> 8) & 0xFFFFFFu;
}

// Exhaustive scans of the two recipes against libm in double.
// out[0] = max abs error of L vs -2 ln(k 2^-24); out[1] = max relative error
// (k < 2^24); out[2] = min L over all k; out[3] = L at k = 2^24.
void ora_scan_neg2ln(double* out) {
  double maxabs = 0, maxrel = 0, minL = 1e30;
  for (uint32_t k = 1; k <= (1u << 24); ++k) {
    double L = (double)neg2ln_u24(k);
    double ref = -2.0 * std::log((double)k * 0x1p-24);
    double e = std::fabs(L - ref);
    if (e > maxabs) maxabs = e;
    if (k < (1u << 24) && e / ref > maxrel) maxrel = e / ref;
    if (L < minL) minL = L;
  }
  out[0] = maxabs; out[1] = maxrel; out[2] = minL; out[3] = (double)neg2ln_u24(1u << 24);
}
// Whole-domain tables of the two building blocks of the noise recipe, for element-by-element
// comparison with another implementation: L[k-1] = neg2ln_u24(k), k = 1..2^24, and
// (c[q], s[q]) = cossin_u24(q), q = 0..2^24-1.  Any pointer may be null.
void ora_table_neg2ln(float* L) {
  if (!L) return;
  for (uint32_t k = 1; k <= (1u << 24); ++k) L[k - 1] = neg2ln_u24(k);
}
void ora_table_cossin(float* c, float* s) {
  for (uint32_t q = 0; q < (1u << 24); ++q) {
    float cc, ss;
    cossin_u24(q, &cc, &ss);
    if (c) c[q] = cc;
    if (s) s[q] = ss;
  }
}
// out[0] = max abs error of cos, out[1] = of sin, out[2] = max |c^2+s^2-1|.
void ora_scan_cossin(double* out) {
  double ec = 0, es = 0, en = 0;
  const double two_pi = 6.283185307179586476925286766559;
  for (uint32_t q = 0; q < (1u << 24); ++q) {
    float c, s;
    cossin_u24(q, &c, &s);
    double th = two_pi * (double)q * 0x1p-24;
    double dc = std::fabs((double)c - std::cos(th)), ds = std::fabs((double)s - std::sin(th));
    double dn = std::fabs((double)c * c + (double)s * s - 1.0);
    if (dc > ec) ec = dc;
    if (ds > es) es = ds;
    if (dn > en) en = dn;
  }
  out[0] = ec; out[1] = es; out[2] = en;
}

}  // extern "C"
