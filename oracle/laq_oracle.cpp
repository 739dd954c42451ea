// LAQ reference ("oracle") -- TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded CPU statement of one LAQ iteration (Sun, Chen, Giannakis,
// Yang, "Communication-Efficient Distributed Learning via Lazily Aggregated Quantized
// Gradients", NeurIPS 2019), written from the paper.  It exists so that the CUDA library can
// be checked against something that is easy to compare with the paper by eye.  Nothing in the
// product path may call it, and it shares no code, header, table or constant with the CUDA
// sources.
//
// Two instantiations of the same template:
//   T = double : every elementwise quantity in fp64 ("fp64 oracle")
//   T = float  : every elementwise quantity in fp32, one IEEE operation at a time in the order
//                written below, no fused multiply-add ("fp32 mirror"); squared norms are
//                accumulated in fp64 from exact products, and the trigger is evaluated in fp64.
// Build with -O2 -ffp-contract=off -fno-fast-math so the compiler neither fuses nor reorders.
//
// Paper passages followed (section / equation / algorithm):
//   Sec. 2.1, Eq. (5)  codes     q_i = floor((g_i - Qp_i + R)/(2 tau R) + 1/2), tau = 1/(2^b - 1),
//                                R = || g - Qp ||_inf
//   Sec. 2.1, Eq. (6)  innovation dQ = 2 tau R q - R 1 ; message = (R, q) = 32 + b p bits ;
//                                server recovery Q_new = Q_prev + dQ
//   Sec. 2.1           error      eps = g - Q_new,  ||eps||_inf <= tau R
//   Sec. 2.2, Eq. (7a) skip rule  ||dQ||^2 <= (1/(alpha^2 M^2)) sum_d xi_d ||theta^{k+1-d}-theta^{k-d}||^2
//                                              + 3 (||eps^k||^2 + ||eps_hat^{k-1}||^2)
//   Sec. 2.2, Eq. (7b) clock      t_m <= t_bar
//   Eq. (4)            server     grad^k = grad^{k-1} + sum_{m in M^k} dQ_m ; theta^{k+1} = theta^k - alpha grad^k
//   Algorithm 2        the loop   (broadcast, compute, quantize, test, upload/skip, clock, update)
//   Supplement "Simulation details": softmax regression with cross-entropy + (lambda/2) Tr(theta^T theta)
//                                inside every sample loss, f = (1/N) sum_m f_m ; one-hidden-layer
//                                ReLU network 784-200-10.
//
// Readings where the paper is silent (all listed in the design notes of the repository):
//   * initial state: Q_m(theta_hat^0) = 0, ||eps_hat||^2 = 0, grad^0 = 0, all D stored parameter
//     differences 0, clocks t_m = t_bar + 1 so that every worker uploads at k = 1;
//   * R = 0 gives q = 0, dQ = 0, eps = 0;
//   * ||theta^{k+1} - theta^k||^2 is evaluated as ||alpha grad^k||^2;
//   * eps_hat is the error at the worker's last upload and is carried across skips;
//   * clock_mode 0 is Algorithm 2 as printed (skip allowed while t_m <= t_bar); clock_mode 1 is
//     the stricter reading of the prose (no copy older than t_bar - 1 iterations: skip needs
//     t_m + 2 <= t_bar), under which t_bar = 1 never skips;
//   * per-sample gradients are scaled by 1/N (N = all samples) and worker m carries the share
//     (N_m/N) lambda theta of the regulariser, so that sum_m g_m is the gradient of f.
//
// Parity unpinned: the iteration/upload/bit COUNTS of the paper's Tables 1-2 (they need MNIST).
// Everything else has a pin in tests/ (hand-worked quantizer case, brute-force nearest grid
// point, error bound, server recovery, aggregate invariant, GD/QGD limits, clock bound,
// Proposition 1 bound, Theorem 1 linear rate, finite-difference gradients, bit-count formula).

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <type_traits>
#include <vector>

namespace {

typedef int64_t i64;

enum Model { M_LOGREG_BIN = 0, M_SOFTMAX = 1, M_MLP2 = 2, M_SYNTH = 3, M_GIVEN = 4 };
enum Flags { F_QUANT_OFF = 1u, F_TRIGGER_OFF = 2u };

// ---------------------------------------------------------------------------------------------
// bf16 operand rounding (round to nearest, ties to even) of an fp32 value, returned as fp32.
// Used only by the network model, whose two large products take bf16 operands.
// ---------------------------------------------------------------------------------------------
float round_bf16(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) return x;  // inf / nan unchanged
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  u &= 0xffff0000u;
  float r;
  std::memcpy(&r, &u, 4);
  return r;
}

// ---------------------------------------------------------------------------------------------
// Quantizer, Sec. 2.1 Eq. (5)-(6).  One worker.
//   in : g[p]  local gradient,  qp[p]  Q_m(theta_hat^{k-1})
//   out: R, codes q[p] in [0, 2^b-1], dq[p] = 2 tau R q - R, qnew[p] = qp + dq, eps[p] = g - qnew,
//        n_dq = ||dq||^2, n_eps = ||eps||^2  (fp64 sums, index order)
// Operation order (each one IEEE operation in T):
//   d = g - qp ; R = max |d| ; tau = 1/(2^b-1) ; s = (2 tau) R ; t = (d + R)/s + 1/2 ;
//   q = clamp(floor(t), 0, 2^b-1) ; dq = s q - R ; qnew = qp + dq ; eps = g - qnew.
// Eq. (5) is 0/0 (or x/0) when the grid step s is zero: R = 0, or R so small that 2 tau R underflows in T.
// Then q = 0, and Eq. (6) is applied as printed (for R = 0 it gives dq = 0).
// ---------------------------------------------------------------------------------------------
template <typename T>
void quantize(const T* g, const T* qp, i64 p, int b, T* R_out, int32_t* q, T* dq, T* qnew, T* eps,
              double* n_dq, double* n_eps) {
  T R = 0;
  for (i64 i = 0; i < p; ++i) {
    T d = g[i] - qp[i];
    T a = std::fabs(d);
    if (a > R || a != a) R = a;  // NaN propagates into R so the caller can flag it
  }
  *R_out = R;
  const double levels_d = std::ldexp(1.0, b) - 1.0;  // 2^b - 1
  const T levels = (T)levels_d;
  const T tau = (T)1 / levels;
  const T s = ((T)2 * tau) * R;
  double sdq = 0.0, seps = 0.0;
  for (i64 i = 0; i < p; ++i) {
    int32_t qi = 0;
    if (s > (T)0) {
      T d = g[i] - qp[i];
      T t = (d + R) / s + (T)0.5;
      T f = std::floor(t);
      if (f < (T)0) f = 0;
      if (f > levels) f = levels;
      qi = (int32_t)f;
    }
    T dqi = s * (T)qi - R;  // Eq. (6): multiply, then subtract
    T qn = qp[i] + dqi;
    T e = g[i] - qn;
    if (q) q[i] = qi;
    if (dq) dq[i] = dqi;
    if (qnew) qnew[i] = qn;
    if (eps) eps[i] = e;
    sdq += (double)dqi * (double)dqi;
    seps += (double)e * (double)e;
  }
  *n_dq = sdq;
  *n_eps = seps;
}

// Server-side recovery (text after Eq. (6)): Q_new = Q_prev + (2 tau R q - R).
template <typename T>
void decode(T R, const int32_t* q, const T* qp, i64 p, int b, T* qnew, T* dq) {
  const T levels = (T)(std::ldexp(1.0, b) - 1.0);
  const T tau = (T)1 / levels;
  const T s = ((T)2 * tau) * R;
  for (i64 i = 0; i < p; ++i) {
    T d = s * (T)q[i] - R;
    if (dq) dq[i] = d;
    qnew[i] = qp[i] + d;
  }
}

// The upload message's code stream (the b p bits of the message, text after Eq. (6)): code i occupies
// bits [i b, (i+1) b) of the stream; stream bit j is bit (j mod 32) of 32-bit word floor(j / 32), least
// significant first.  Written bit by bit, so a code may straddle two words (b = 3).
void pack_codes(const int32_t* q, i64 p, int b, uint32_t* words, i64 n_words) {
  for (i64 w = 0; w < n_words; ++w) words[w] = 0;
  for (i64 i = 0; i < p; ++i)
    for (int t = 0; t < b; ++t) {
      i64 bit = i * (i64)b + t;
      if (((uint32_t)q[i] >> t) & 1u) words[bit / 32] |= 1u << (bit % 32);
    }
}
void unpack_codes(const uint32_t* words, i64 p, int b, int32_t* q) {
  for (i64 i = 0; i < p; ++i) {
    uint32_t v = 0;
    for (int t = 0; t < b; ++t) {
      i64 bit = i * (i64)b + t;
      v |= ((words[bit / 32] >> (bit % 32)) & 1u) << t;
    }
    q[i] = (int32_t)v;
  }
}

// ---------------------------------------------------------------------------------------------
// Trigger, Eq. (7a)+(7b), one worker.  dtheta2[0] is the newest difference
// ||theta^k - theta^{k-1}||^2 (d = 1), dtheta2[D-1] the oldest (d = D).
// Returns 1 to skip, 0 to upload; *rhs_out receives the right-hand side of (7a).
// ---------------------------------------------------------------------------------------------
int trigger(double n_dq, double n_eps, double n_epshat, const double* dtheta2, const float* xi,
            int D, float alpha, int M, int clock, int tbar, int clock_mode, double* rhs_out) {
  double acc = 0.0;
  for (int d = 0; d < D; ++d) {
    double term = (double)xi[d] * dtheta2[d];
    acc = acc + term;
  }
  double a = (double)alpha;
  double c = (a * a) * ((double)M * (double)M);
  double rhs = acc / c + 3.0 * (n_eps + n_epshat);
  *rhs_out = rhs;
  bool crit_a = n_dq <= rhs;
  bool crit_b = (clock_mode == 0) ? (clock <= tbar) : (clock + 2 <= tbar);
  return (crit_a && crit_b) ? 1 : 0;
}

// ---------------------------------------------------------------------------------------------
// Models (supplement, "Simulation details").  All in fp64 from fp32 data; the caller rounds the
// gradient to T.  `inv_N` = 1/N with N the total sample count over all workers; `share` = N_m/N.
// Each returns the worker's loss contribution (1/N) sum_n CE_n + share (lambda/2) ||theta||^2.
// ---------------------------------------------------------------------------------------------

// Binary logistic regression: z = x . theta, loss = softplus(z) - y z, grad = (sigma(z) - y) x.
double grad_logreg_bin(const float* X, const int32_t* y, i64 n, int F, const double* theta,
                       double inv_N, double share, double lambda, double* g) {
  for (int f = 0; f < F; ++f) g[f] = 0.0;
  double loss = 0.0;
  for (i64 r = 0; r < n; ++r) {
    const float* x = X + r * F;
    double z = 0.0;
    for (int f = 0; f < F; ++f) z += (double)x[f] * theta[f];
    double sp = (z > 0.0) ? z + std::log1p(std::exp(-z)) : std::log1p(std::exp(z));
    double sig = (z >= 0.0) ? 1.0 / (1.0 + std::exp(-z)) : std::exp(z) / (1.0 + std::exp(z));
    loss += sp - (double)y[r] * z;
    double res = sig - (double)y[r];
    for (int f = 0; f < F; ++f) g[f] += res * (double)x[f];
  }
  double nrm = 0.0;
  for (int f = 0; f < F; ++f) {
    g[f] = g[f] * inv_N + share * lambda * theta[f];
    nrm += theta[f] * theta[f];
  }
  return loss * inv_N + share * 0.5 * lambda * nrm;
}

// C-class softmax regression, theta is C x F row-major.
double grad_softmax(const float* X, const int32_t* y, i64 n, int F, int C, const double* theta,
                    double inv_N, double share, double lambda, double* g) {
  const i64 p = (i64)C * F;
  for (i64 i = 0; i < p; ++i) g[i] = 0.0;
  std::vector<double> z(C), pr(C);
  double loss = 0.0;
  for (i64 r = 0; r < n; ++r) {
    const float* x = X + r * F;
    double zmax = -std::numeric_limits<double>::infinity();
    for (int c = 0; c < C; ++c) {
      double acc = 0.0;
      const double* th = theta + (i64)c * F;
      for (int f = 0; f < F; ++f) acc += th[f] * (double)x[f];
      z[c] = acc;
      if (acc > zmax) zmax = acc;
    }
    double sum = 0.0;
    for (int c = 0; c < C; ++c) {
      pr[c] = std::exp(z[c] - zmax);
      sum += pr[c];
    }
    loss += (zmax + std::log(sum)) - z[y[r]];
    for (int c = 0; c < C; ++c) {
      double res = pr[c] / sum - (c == y[r] ? 1.0 : 0.0);
      double* gc = g + (i64)c * F;
      for (int f = 0; f < F; ++f) gc[f] += res * (double)x[f];
    }
  }
  double nrm = 0.0;
  for (i64 i = 0; i < p; ++i) {
    g[i] = g[i] * inv_N + share * lambda * theta[i];
    nrm += theta[i] * theta[i];
  }
  return loss * inv_N + share * 0.5 * lambda * nrm;
}

// One-hidden-layer ReLU network F-H-C with softmax cross-entropy.
// Parameter layout: W1 [H x F] row-major, b1 [H], W2 [C x H] row-major, b2 [C].
// With bf16_ops != 0 the operands of the two large products are rounded to bf16 first
// (X and W1 in the hidden pre-activation; dH and X in the W1 gradient); accumulation, the
// output layer, softmax, bias gradients and the regulariser are unrounded.
double grad_mlp2(const float* X, const int32_t* y, i64 n, int F, int H, int C, const double* theta,
                 double inv_N, double share, double lambda, int bf16_ops, double* g) {
  const i64 oW1 = 0, ob1 = (i64)H * F, oW2 = ob1 + H, ob2 = oW2 + (i64)C * H, p = ob2 + C;
  for (i64 i = 0; i < p; ++i) g[i] = 0.0;
  std::vector<double> W1r((size_t)H * F);
  for (i64 i = 0; i < (i64)H * F; ++i)
    W1r[i] = bf16_ops ? (double)round_bf16((float)theta[oW1 + i]) : theta[oW1 + i];
  std::vector<double> xr(F), h(H), z(C), pr(C), dz(C), dh(H);
  double loss = 0.0;
  for (i64 r = 0; r < n; ++r) {
    const float* x = X + r * F;
    for (int f = 0; f < F; ++f) xr[f] = bf16_ops ? (double)round_bf16(x[f]) : (double)x[f];
    for (int j = 0; j < H; ++j) {
      double acc = 0.0;
      const double* w = &W1r[(size_t)j * F];
      for (int f = 0; f < F; ++f) acc += xr[f] * w[f];
      acc += theta[ob1 + j];
      h[j] = acc > 0.0 ? acc : 0.0;
    }
    double zmax = -std::numeric_limits<double>::infinity();
    for (int c = 0; c < C; ++c) {
      double acc = 0.0;
      for (int j = 0; j < H; ++j) acc += theta[oW2 + (i64)c * H + j] * h[j];
      acc += theta[ob2 + c];
      z[c] = acc;
      if (acc > zmax) zmax = acc;
    }
    double sum = 0.0;
    for (int c = 0; c < C; ++c) {
      pr[c] = std::exp(z[c] - zmax);
      sum += pr[c];
    }
    loss += (zmax + std::log(sum)) - z[y[r]];
    for (int c = 0; c < C; ++c) dz[c] = pr[c] / sum - (c == y[r] ? 1.0 : 0.0);
    for (int c = 0; c < C; ++c) {
      for (int j = 0; j < H; ++j) g[oW2 + (i64)c * H + j] += dz[c] * h[j];
      g[ob2 + c] += dz[c];
    }
    for (int j = 0; j < H; ++j) {
      double acc = 0.0;
      for (int c = 0; c < C; ++c) acc += theta[oW2 + (i64)c * H + j] * dz[c];
      dh[j] = h[j] > 0.0 ? acc : 0.0;
      g[ob1 + j] += dh[j];
    }
    for (int j = 0; j < H; ++j) {
      if (dh[j] == 0.0) continue;
      double dj = bf16_ops ? (double)round_bf16((float)dh[j]) : dh[j];
      double* gw = g + oW1 + (i64)j * F;
      for (int f = 0; f < F; ++f) gw[f] += dj * xr[f];
    }
  }
  double nrm = 0.0;
  for (i64 i = 0; i < p; ++i) {
    g[i] = g[i] * inv_N + share * lambda * theta[i];
    nrm += theta[i] * theta[i];
  }
  return loss * inv_N + share * 0.5 * lambda * nrm;
}

// ---------------------------------------------------------------------------------------------
// Synthetic gradient stream for the large-p throughput workload (no data shard): a counter-based
// generator, so that both this file and the CUDA library can produce the same fp32 values from
// its definition alone.  Coordinates come in groups of four (group v = i / 4, e = i mod 4):
//   fmix32(x): the 32-bit finaliser of MurmurHash3 (A. Appleby, public domain):
//       x ^= x>>16; x *= 0x85ebca6b; x ^= x>>13; x *= 0xc2b2ae35; x ^= x>>16
//   key_m  = fmix32( seed_lo ^ fmix32( seed_hi + 0x9e3779b9 * (m+1) ) )
//   h0     = fmix32( (uint32) v ^ key_m ) ;  h1 = h0 * 0x9e3779b1 ;  h1 ^= h1 >> 15
//   with bytes b0..b3 of a word (b0 lowest):  S(h) = b0+b1+b2+b3-510 ,  A(h) = b0-b1+b2-b3
//       (sums of four uniform bytes: near-Gaussian, variance 21845 = 4 (256^2-1)/12, S and A uncorrelated)
//   z_0 = S(h0), z_1 = A(h0), z_2 = S(h1), z_3 = A(h1)
//   cz     = fp32( sigma / sqrt(21845) )
//   eta_m  = fp32( eta0 (m+1) / M )                 (heterogeneous drift speed)
//   g_m^k[i] = fl( fma( fl(k eta_m), z_{e xor 2}, z_e ) * cz )      fp32, k = 1, 2, ...
//       (the slowly growing drift term reuses the z of the partner coordinate e xor 2)
// ---------------------------------------------------------------------------------------------
uint32_t fmix32(uint32_t x) {
  x ^= x >> 16;
  x *= 0x85ebca6bu;
  x ^= x >> 13;
  x *= 0xc2b2ae35u;
  x ^= x >> 16;
  return x;
}
void synth_gradient(uint64_t seed, int m, int M, i64 p, i64 k, float sigma, float eta0, float* g) {
  uint32_t seed_lo = (uint32_t)(seed & 0xffffffffu), seed_hi = (uint32_t)(seed >> 32);
  uint32_t key = fmix32(seed_lo ^ fmix32(seed_hi + 0x9e3779b9u * (uint32_t)(m + 1)));
  float cz = (float)((double)sigma / std::sqrt(21845.0));
  float eta_m = (float)((double)eta0 * (double)(m + 1) / (double)M);
  float drift = (float)k * eta_m;
  for (i64 v = 0; 4 * v < p; ++v) {
    uint32_t h[2];
    h[0] = fmix32((uint32_t)v ^ key);
    h[1] = h[0] * 0x9e3779b1u;
    h[1] ^= h[1] >> 15;
    float z[4];
    for (int j = 0; j < 2; ++j) {
      int b0 = h[j] & 255, b1 = (h[j] >> 8) & 255, b2 = (h[j] >> 16) & 255, b3 = (h[j] >> 24) & 255;
      z[2 * j] = (float)(b0 + b1 + b2 + b3 - 510);
      z[2 * j + 1] = (float)(b0 - b1 + b2 - b3);
    }
    for (int e = 0; e < 4 && 4 * v + e < p; ++e) {
      float a = std::fmaf(drift, z[e ^ 2], z[e]);
      g[4 * v + e] = a * cz;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The LAQ loop (Algorithm 2), state and one iteration.
// ---------------------------------------------------------------------------------------------
// Start of worker m's minibatch window at iteration k = 1, 2, ..: a counter-based draw from (seed, m, k)
// with the 32-bit finalizer fmix32, reduced modulo the shard size n.
i64 batch_offset(uint64_t seed, int m, i64 k, i64 n) {
  const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
  const uint32_t h = fmix32(fmix32(lo + (uint32_t)k) ^ (hi + 0x9e3779b9u * (uint32_t)(m + 1)));
  return (i64)(h % (uint32_t)n);
}

struct Config {
  int model, M;
  i64 p;
  int n_features, n_classes, n_hidden;
  float alpha, lambda;
  int b, D;
  std::vector<float> xi;
  int tbar, clock_mode;
  uint32_t flags;
  uint64_t seed;
  float synth_sigma, synth_eta0;
  int bf16_ops;
  int batch = 0;  // 0: full local gradients; > 0: minibatch size per worker (the stochastic variant of Sec. 4)
};

struct IterStats {  // what one iteration reports, per worker unless noted
  std::vector<int32_t> skip;
  std::vector<double> R, n_dq, n_eps, rhs, loss_m;
  double dtheta2, loss;
  int uploads;
};

template <typename T>
struct Laq {
  Config c;
  std::vector<i64> N;  // samples per worker
  i64 Ntot = 0;
  std::vector<std::vector<float>> X;
  std::vector<std::vector<int32_t>> y;
  std::vector<T> theta, agg;      // theta^k, grad^{k-1}
  std::vector<T> qp;              // Q_m(theta_hat_m^{k-1}), M x p
  std::vector<double> n_epshat;   // ||eps_hat_m||^2
  std::vector<int32_t> clock;     // t_m
  std::vector<double> hist;       // hist[0] newest ... hist[D-1] oldest squared differences
  std::vector<int32_t> codes;     // last computed codes, M x p (b <= 31)
  std::vector<T> g;               // last gradients, M x p
  i64 k = 0;                      // iterations done
  i64 uploads = 0;
  i64 bits = 0;
  IterStats st;

  void init(const Config& cfg, const i64* Nm, const float* theta0) {
    c = cfg;
    N.assign(Nm, Nm + c.M);
    Ntot = 0;
    for (int m = 0; m < c.M; ++m) Ntot += N[m];
    X.resize(c.M);
    y.resize(c.M);
    theta.assign(c.p, (T)0);
    if (theta0)
      for (i64 i = 0; i < c.p; ++i) theta[i] = (T)theta0[i];
    agg.assign(c.p, (T)0);
    qp.assign((size_t)c.M * c.p, (T)0);
    n_epshat.assign(c.M, 0.0);
    clock.assign(c.M, c.tbar + 1);
    hist.assign(c.D, 0.0);
    codes.assign((size_t)c.M * c.p, 0);
    g.assign((size_t)c.M * c.p, (T)0);
    k = 0;
    uploads = 0;
    bits = 0;
  }

  // Algorithm 2, "worker m computes grad f_m(theta^k)": fills g (M x p) from the model.
  void compute_gradients() {
    st.loss_m.assign(c.M, 0.0);
    if (c.model == M_GIVEN) return;
    if (c.model == M_SYNTH) {
      std::vector<float> tmp(c.p);
      for (int m = 0; m < c.M; ++m) {
        synth_gradient(c.seed, m, c.M, c.p, k + 1, c.synth_sigma, c.synth_eta0, tmp.data());
        for (i64 i = 0; i < c.p; ++i) g[(size_t)m * c.p + i] = (T)tmp[i];
      }
      return;
    }
    std::vector<double> th(c.p), gd(c.p);
    for (i64 i = 0; i < c.p; ++i) th[i] = (double)theta[i];
    const double inv_N = 1.0 / (double)Ntot;
    std::vector<float> Xb;
    std::vector<int32_t> yb;
    for (int m = 0; m < c.M; ++m) {
      const double share = (double)N[m] / (double)Ntot;
      // The stochastic variant (Sec. 4, minibatch tests): the sum over the worker's samples is replaced by
      // N_m / B_m times the sum over a minibatch of B_m samples, here a cyclic window of consecutive samples
      // with a pseudo-random start; the regulariser's share is unchanged.
      const float* Xm = X[m].data();
      const int32_t* ym = y[m].data();
      i64 n_used = N[m];
      double inv_Nm = inv_N;
      if (c.batch > 0) {
        const i64 B = std::min<i64>(c.batch, N[m]);
        const i64 o = batch_offset(c.seed, m, k + 1, N[m]);
        const size_t F = (size_t)c.n_features;
        Xb.resize((size_t)B * F);
        yb.resize((size_t)B);
        for (i64 j = 0; j < B; ++j) {
          const i64 r = (o + j) % N[m];
          std::memcpy(&Xb[(size_t)j * F], Xm + (size_t)r * F, sizeof(float) * F);
          yb[(size_t)j] = ym[r];
        }
        Xm = Xb.data();
        ym = yb.data();
        n_used = B;
        inv_Nm = inv_N * ((double)N[m] / (double)B);
      }
      double loss = 0.0;
      if (c.model == M_LOGREG_BIN)
        loss = grad_logreg_bin(Xm, ym, n_used, c.n_features, th.data(), inv_Nm, share, (double)c.lambda,
                               gd.data());
      else if (c.model == M_SOFTMAX)
        loss = grad_softmax(Xm, ym, n_used, c.n_features, c.n_classes, th.data(), inv_Nm, share,
                            (double)c.lambda, gd.data());
      else
        loss = grad_mlp2(Xm, ym, n_used, c.n_features, c.n_hidden, c.n_classes, th.data(), inv_Nm, share,
                         (double)c.lambda, c.bf16_ops, gd.data());
      st.loss_m[m] = loss;
      for (i64 i = 0; i < c.p; ++i) g[(size_t)m * c.p + i] = (T)gd[i];
    }
  }

  // One pass of Algorithm 2's loop body with g already in place.
  void iterate() {
    const int M = c.M;
    const i64 p = c.p;
    st.skip.assign(M, 0);
    st.R.assign(M, 0.0);
    st.n_dq.assign(M, 0.0);
    st.n_eps.assign(M, 0.0);
    st.rhs.assign(M, 0.0);
    st.uploads = 0;
    std::vector<T> dq(p), qnew(p);
    std::vector<int32_t> q(p);
    // the server applies the uploads in ascending worker order: grad += dQ_m, one add each
    for (int m = 0; m < M; ++m) {
      const T* gm = &g[(size_t)m * p];
      T* qpm = &qp[(size_t)m * p];
      T R = 0;
      double n_dq = 0.0, n_eps = 0.0;
      if (c.flags & F_QUANT_OFF) {
        // unquantized innovation (the lazily aggregated gradient without a quantizer):
        // Q_m(theta^k) = grad f_m(theta^k), eps = 0, a coordinate costs 32 bits.
        for (i64 i = 0; i < p; ++i) {
          T d = gm[i] - qpm[i];
          T a = std::fabs(d);
          if (a > R || a != a) R = a;
          dq[i] = d;
          qnew[i] = gm[i];
          q[i] = 0;
          n_dq += (double)d * (double)d;
        }
      } else {
        quantize<T>(gm, qpm, p, c.b, &R, q.data(), dq.data(), qnew.data(), nullptr, &n_dq, &n_eps);
      }
      std::memcpy(&codes[(size_t)m * p], q.data(), sizeof(int32_t) * p);
      double rhs = 0.0;
      int skip = trigger(n_dq, n_eps, n_epshat[m], hist.data(), c.xi.data(), c.D, c.alpha, M,
                         clock[m], c.tbar, c.clock_mode, &rhs);
      if (c.flags & F_TRIGGER_OFF) skip = 0;
      st.skip[m] = skip;
      st.R[m] = (double)R;
      st.n_dq[m] = n_dq;
      st.n_eps[m] = n_eps;
      st.rhs[m] = rhs;
      if (skip) {
        clock[m] += 1;  // theta_hat unchanged
      } else {
        for (i64 i = 0; i < p; ++i) {
          qpm[i] = qnew[i];
          agg[i] = agg[i] + dq[i];
        }
        n_epshat[m] = n_eps;
        clock[m] = 0;
        st.uploads += 1;
        uploads += 1;
        bits += (c.flags & F_QUANT_OFF) ? 32 * p : 32 + (i64)c.b * p;
      }
    }
    // theta^{k+1} = theta^k - alpha grad^k ; newest squared difference = ||alpha grad^k||^2
    double d2 = 0.0;
    for (i64 i = 0; i < p; ++i) {
      T u = (T)c.alpha * agg[i];
      theta[i] = theta[i] - u;
      d2 += (double)u * (double)u;
    }
    for (int d = c.D - 1; d > 0; --d) hist[d] = hist[d - 1];
    if (c.D > 0) hist[0] = d2;
    st.dtheta2 = d2;
    k += 1;
  }

  void step_model() {
    compute_gradients();
    double l = 0.0;
    for (int m = 0; m < c.M; ++m) l += st.loss_m[m];
    st.loss = l;
    iterate();
  }
  void step_given(const T* gin) {
    std::memcpy(g.data(), gin, sizeof(T) * (size_t)c.M * c.p);
    st.loss_m.assign(c.M, 0.0);
    st.loss = 0.0;
    iterate();
  }
};

struct Handle {
  int prec;  // 32 or 64
  Laq<float> f;
  Laq<double> d;
};

}  // namespace

// =============================================================================================
// C interface (loaded with ctypes by the tests, the smoke check and the bench's CPU baseline).
// =============================================================================================
extern "C" {

// ---- stateless pieces ------------------------------------------------------------------------
void laqo_quantize_f64(const double* g, const double* qp, int64_t p, int b, double* R, int32_t* q,
                       double* dq, double* qnew, double* eps, double* n_dq, double* n_eps) {
  quantize<double>(g, qp, p, b, R, q, dq, qnew, eps, n_dq, n_eps);
}
void laqo_quantize_f32(const float* g, const float* qp, int64_t p, int b, float* R, int32_t* q,
                       float* dq, float* qnew, float* eps, double* n_dq, double* n_eps) {
  quantize<float>(g, qp, p, b, R, q, dq, qnew, eps, n_dq, n_eps);
}
void laqo_decode_f64(double R, const int32_t* q, const double* qp, int64_t p, int b, double* qnew,
                     double* dq) {
  decode<double>(R, q, qp, p, b, qnew, dq);
}
void laqo_decode_f32(float R, const int32_t* q, const float* qp, int64_t p, int b, float* qnew,
                     float* dq) {
  decode<float>(R, q, qp, p, b, qnew, dq);
}
int64_t laqo_code_words(int64_t p, int b) { return (p * (int64_t)b + 31) / 32; }
void laqo_pack_codes(const int32_t* q, int64_t p, int b, uint32_t* words) {
  pack_codes(q, p, b, words, laqo_code_words(p, b));
}
void laqo_unpack_codes(const uint32_t* words, int64_t p, int b, int32_t* q) {
  unpack_codes(words, p, b, q);
}
int laqo_trigger(double n_dq, double n_eps, double n_epshat, const double* dtheta2,
                 const float* xi, int D, float alpha, int M, int clock, int tbar, int clock_mode,
                 double* rhs) {
  return trigger(n_dq, n_eps, n_epshat, dtheta2, xi, D, alpha, M, clock, tbar, clock_mode, rhs);
}
double laqo_grad_logreg_bin(const float* X, const int32_t* y, int64_t n, int F, const double* theta,
                            double inv_N, double share, double lambda, double* g) {
  return grad_logreg_bin(X, y, n, F, theta, inv_N, share, lambda, g);
}
double laqo_grad_softmax(const float* X, const int32_t* y, int64_t n, int F, int C,
                         const double* theta, double inv_N, double share, double lambda, double* g) {
  return grad_softmax(X, y, n, F, C, theta, inv_N, share, lambda, g);
}
double laqo_grad_mlp2(const float* X, const int32_t* y, int64_t n, int F, int H, int C,
                      const double* theta, double inv_N, double share, double lambda, int bf16_ops,
                      double* g) {
  return grad_mlp2(X, y, n, F, H, C, theta, inv_N, share, lambda, bf16_ops, g);
}
void laqo_synth_gradient(uint64_t seed, int m, int M, int64_t p, int64_t k, float sigma, float eta0,
                         float* g) {
  synth_gradient(seed, m, M, p, k, sigma, eta0, g);
}
float laqo_round_bf16(float x) { return round_bf16(x); }

// ---- the loop ----------------------------------------------------------------------------------
void* laqo_new(int precision, int model, int M, int64_t p, const int64_t* N, int n_features,
               int n_classes, int n_hidden, float alpha, float lambda, int b, int D, const float* xi,
               int tbar, int clock_mode, uint32_t flags, uint64_t seed, float synth_sigma,
               float synth_eta0, int bf16_ops, const float* theta0) {
  if (precision != 32 && precision != 64) return nullptr;
  if (M < 1 || p < 1 || D < 0 || b < 1 || b > 31) return nullptr;
  Handle* h = new Handle();
  h->prec = precision;
  Config c;
  c.model = model;
  c.M = M;
  c.p = p;
  c.n_features = n_features;
  c.n_classes = n_classes;
  c.n_hidden = n_hidden;
  c.alpha = alpha;
  c.lambda = lambda;
  c.b = b;
  c.D = D;
  c.xi.assign(xi, xi + D);
  c.tbar = tbar;
  c.clock_mode = clock_mode;
  c.flags = flags;
  c.seed = seed;
  c.synth_sigma = synth_sigma;
  c.synth_eta0 = synth_eta0;
  c.bf16_ops = bf16_ops;
  if (precision == 32)
    h->f.init(c, N, theta0);
  else
    h->d.init(c, N, theta0);
  return h;
}
void laqo_free(void* hv) { delete (Handle*)hv; }
void laqo_set_batch(void* hv, int batch) {
  Handle* h = (Handle*)hv;
  if (h->prec == 32)
    h->f.c.batch = batch;
  else
    h->d.c.batch = batch;
}
int64_t laqo_batch_offset(uint64_t seed, int m, int64_t k, int64_t n) { return batch_offset(seed, m, k, n); }

int laqo_set_shard(void* hv, int m, const float* X, const int32_t* y, int64_t n, int row_len) {
  Handle* h = (Handle*)hv;
  auto set = [&](auto& L) -> int {
    if (m < 0 || m >= L.c.M || n != L.N[m]) return 1;
    L.X[m].assign(X, X + (size_t)n * row_len);
    L.y[m].assign(y, y + n);
    return 0;
  };
  return h->prec == 32 ? set(h->f) : set(h->d);
}

int laqo_step(void* hv) {
  Handle* h = (Handle*)hv;
  if (h->prec == 32)
    h->f.step_model();
  else
    h->d.step_model();
  return 0;
}
// g is M x p in the handle's own precision (float for 32, double for 64)
int laqo_step_given(void* hv, const void* g) {
  Handle* h = (Handle*)hv;
  if (h->prec == 32)
    h->f.step_given((const float*)g);
  else
    h->d.step_given((const double*)g);
  return 0;
}

// Last iteration's report.  Any pointer may be null.
void laqo_last_stats(void* hv, int32_t* skip, double* R, double* n_dq, double* n_eps, double* rhs,
                     double* loss_m, double* dtheta2, double* loss, int32_t* uploads) {
  Handle* h = (Handle*)hv;
  auto get = [&](auto& L) {
    const int M = L.c.M;
    for (int m = 0; m < M; ++m) {
      if (skip) skip[m] = L.st.skip[m];
      if (R) R[m] = L.st.R[m];
      if (n_dq) n_dq[m] = L.st.n_dq[m];
      if (n_eps) n_eps[m] = L.st.n_eps[m];
      if (rhs) rhs[m] = L.st.rhs[m];
      if (loss_m) loss_m[m] = L.st.loss_m[m];
    }
    if (dtheta2) *dtheta2 = L.st.dtheta2;
    if (loss) *loss = L.st.loss;
    if (uploads) *uploads = L.st.uploads;
  };
  if (h->prec == 32)
    get(h->f);
  else
    get(h->d);
}

// State, always delivered as fp64 (exact for the fp32 mirror).  Any pointer may be null.
void laqo_get_state(void* hv, double* theta, double* agg, double* qp, double* g, int32_t* codes,
                    double* n_epshat, int32_t* clock, double* hist, int64_t* counters /*k,uploads,bits*/) {
  Handle* h = (Handle*)hv;
  auto get = [&](auto& L) {
    const int M = L.c.M;
    const i64 p = L.c.p;
    if (theta)
      for (i64 i = 0; i < p; ++i) theta[i] = (double)L.theta[i];
    if (agg)
      for (i64 i = 0; i < p; ++i) agg[i] = (double)L.agg[i];
    if (qp)
      for (i64 i = 0; i < (i64)M * p; ++i) qp[i] = (double)L.qp[i];
    if (g)
      for (i64 i = 0; i < (i64)M * p; ++i) g[i] = (double)L.g[i];
    if (codes) std::memcpy(codes, L.codes.data(), sizeof(int32_t) * (size_t)M * p);
    if (n_epshat)
      for (int m = 0; m < M; ++m) n_epshat[m] = L.n_epshat[m];
    if (clock)
      for (int m = 0; m < M; ++m) clock[m] = L.clock[m];
    if (hist)
      for (int d = 0; d < L.c.D; ++d) hist[d] = L.hist[d];
    if (counters) {
      counters[0] = L.k;
      counters[1] = L.uploads;
      counters[2] = L.bits;
    }
  };
  if (h->prec == 32)
    get(h->f);
  else
    get(h->d);
}

// Overwrite pieces of the state (used by tests that start from a prescribed situation).
void laqo_set_state(void* hv, const double* theta, const double* agg, const double* qp,
                    const double* n_epshat, const int32_t* clock, const double* hist) {
  Handle* h = (Handle*)hv;
  auto set = [&](auto& L) {
    using T = typename std::decay<decltype(L.theta)>::type::value_type;
    const int M = L.c.M;
    const i64 p = L.c.p;
    if (theta)
      for (i64 i = 0; i < p; ++i) L.theta[i] = (T)theta[i];
    if (agg)
      for (i64 i = 0; i < p; ++i) L.agg[i] = (T)agg[i];
    if (qp)
      for (i64 i = 0; i < (i64)M * p; ++i) L.qp[i] = (T)qp[i];
    if (n_epshat)
      for (int m = 0; m < M; ++m) L.n_epshat[m] = n_epshat[m];
    if (clock)
      for (int m = 0; m < M; ++m) L.clock[m] = clock[m];
    if (hist)
      for (int d = 0; d < L.c.D; ++d) L.hist[d] = hist[d];
  };
  if (h->prec == 32)
    set(h->f);
  else
    set(h->d);
}

// Loss of the whole problem at the current theta (fp64), without stepping.
double laqo_loss(void* hv) {
  Handle* h = (Handle*)hv;
  auto run = [&](auto& L) -> double {
    auto saved_g = L.g;
    auto saved_st = L.st;
    L.compute_gradients();
    double l = 0.0;
    for (int m = 0; m < L.c.M; ++m) l += L.st.loss_m[m];
    L.g = saved_g;
    L.st = saved_st;
    return l;
  };
  return h->prec == 32 ? run(h->f) : run(h->d);
}

}  // extern "C"
