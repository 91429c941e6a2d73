// dmx_oracle.cpp — CPU oracle of the DYNAMIX data-parallel gradient step.
//
// TEST INFRASTRUCTURE, not product code: only the tests, the smoke check and the
// CPU-baseline leg of the benchmark may build, load or call this file. It shares no
// code, header, table or constant with the CUDA library; the state-vector layout and the
// return codes below are typed in again from the interface description on purpose.
//
// What it computes is the plain definition of the step, one parameter at a time, in
// fp64, in the order and notation of the method:
//   Algorithm 1, worker loop (each worker computes its gradient at its own batch size and the
//     global model is updated): the K workers' gradients x_k (each a mean over b_k samples) are combined into the mean
//     over all B = sum b_k samples, g_j = (sum_k b_k x_kj) / B, and the global model takes
//     one SGD-momentum step m <- beta m + g, theta <- theta - lr m (Section "Workloads
//     and Datasets" names SGD; the momentum form is the usual undampened one), or one Adam
//     step (the same section names ADAM; Kingma & Ba 2015, Algorithm 1):
//     m <- b1 m + (1-b1) g, v <- b2 v + (1-b2) g^2, theta <- theta - lr mhat/(sqrt(vhat)+eps)
//     with mhat = m/(1-b1^t), vhat = v/(1-b2^t). In Adam mode the state vector also carries
//     mean, variance and standard deviation over the parameters of g_j/(sqrt(vhat_j)+eps),
//     this library's reading of the gradient statistics normalized for an adaptive optimizer.
//   Section "State representation", "Training Statistical Efficiency Metrics": gradient
//     statistics, sigma_norm and sigma^2_norm; Section "RL Agent Inference Evaluation",
//     "Batch Size Adaptation Dynamics": the gradient noise scale.
// The paper prints no formula for any of these. The estimators follow from modelling x_k
// as the mean of b_k i.i.d. per-sample gradients with mean G and covariance Sigma:
//   E sum_k b_k |x_k - g|^2 = (K-1) tr Sigma      =>  trS = D / (K-1)
//   E |g|^2 = |G|^2 + tr Sigma / B                =>  G2  = A - trS / B
//   gns = trS / G2,   sigma^2_norm = (trS / B) / A  (noise-to-signal of the step taken).
//
// Pinned by tests/test_oracle_pins.py (closed forms, exact rational brute force, invariants,
// statistical expectations). Not pinned by anything in the paper: the choice of these
// estimators over other unbiased ones, and the sigma_norm reading ("parity unpinned" with
// respect to the paper for those two choices).
//
// Long sums use Neumaier-compensated fp64 accumulation so that the oracle's own error stays
// near 1e-15 relative at P = 3.4e8. The parameter range is processed in fixed blocks of 2^20
// elements whose partial sums are combined in block order, so the result does not depend
// on the number of threads.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <new>
#include <thread>
#include <vector>

namespace {

constexpr int kOk = 0, kErrArg = -1, kErrSegments = -2, kErrBatch = -3, kErrOrder = -8;
constexpr int kF32 = 0, kBF16 = 1;
constexpr int64_t kBlock = int64_t(1) << 20;

// out_state layout (fp32): header of 16, then q_k[K], V_s[S], N_s[S]
constexpr int iB = 0, iA = 1, iTrS = 2, iG2 = 3, iGns = 4, iCos = 5, iDot = 6, iPP = 7,
              iSig2 = 8, iSig = 9, iWq = 10, iFlags = 11, iHdr = 16;
constexpr int fNonFinite = 1, fG2NonPos = 2, fCosUndef = 4, fSingle = 8;

struct Sum {  // Neumaier compensated sum
  double s = 0.0, c = 0.0;
  void add(double v) {
    double t = s + v;
    if (std::fabs(s) >= std::fabs(v)) c += (s - t) + v; else c += (v - t) + s;
    s = t;
  }
  double value() const { return s + c; }
};

double widen(const void* base, int dtype, int64_t i) {
  if (dtype == kF32) return (double)static_cast<const float*>(base)[i];
  uint32_t bits = uint32_t(static_cast<const uint16_t*>(base)[i]) << 16;  // bf16 = top half of fp32
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}

struct Partial {
  std::vector<Sum> q;      // K
  Sum c, pp, su, su2;
  int seg_first = 0;       // V, N cover segments seg_first .. seg_first + V.size() - 1
  std::vector<Sum> V, N;
};

}  // namespace

struct dmxo {
  int K = 0, S = 0, dtype = 0;
  int64_t P = 0;
  std::vector<int64_t> o;  // S+1 offsets
  // per-step
  bool open = false;
  std::vector<double> b;
  double B = 0, lr = 0, beta = 0;
  bool adam = false;       // Adam update instead of SGD with momentum (beta is then beta1)
  double beta2 = 0, eps = 0;
  int64_t t = 0;           // 1-based step count (bias correction)
  int64_t next = 0;        // next element expected by dmxo_range
  std::vector<Sum> q, V, N;
  Sum c, pp, su, su2;
};

namespace {

// Segment containing element j: the unique s with o[s] <= j < o[s+1].
int segment_of(const dmxo& h, int64_t j) {
  int lo = 0, hi = h.S - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) / 2;
    if (h.o[mid] <= j) lo = mid; else hi = mid - 1;
  }
  while (h.o[lo + 1] <= j) ++lo;  // step over empty segments that start at the same offset
  return lo;
}

// Elements [j0, j1) of the step; pointers address element `base`.
void run_block(const dmxo& h, int64_t base, int64_t j0, int64_t j1, const void* const* grads,
               float* params, float* momentum, float* second, float* prev_agg, Partial& out) {
  const int K = h.K;
  out.q.assign(K, Sum());
  out.seg_first = segment_of(h, j0);
  int s_last = segment_of(h, j1 - 1);
  out.V.assign(s_last - out.seg_first + 1, Sum());
  out.N.assign(s_last - out.seg_first + 1, Sum());
  std::vector<double> x(K);
  int s = out.seg_first;
  for (int64_t j = j0; j < j1; ++j) {
    while (h.o[s + 1] <= j) ++s;
    const int64_t i = j - base;
    // weighted aggregate: mean over all B samples
    double num = 0.0;
    for (int k = 0; k < K; ++k) {
      x[k] = widen(grads[k], h.dtype, i);
      num += h.b[k] * x[k];
    }
    const double g = num / h.B;
    // batch-size-weighted spread of the workers around the aggregate; per-worker norms
    double d = 0.0;
    for (int k = 0; k < K; ++k) {
      const double e = x[k] - g;
      d += h.b[k] * e * e;
      out.q[k].add(x[k] * x[k]);
    }
    out.V[s - out.seg_first].add(d);
    out.N[s - out.seg_first].add(g * g);
    // similarity to the previous step's aggregate (as stored)
    const double a = (double)prev_agg[i];
    out.c.add(g * a);
    out.pp.add(a * a);
    if (!h.adam) {
      // SGD with momentum
      const double m_new = h.beta * (double)momentum[i] + g;
      const double th_new = (double)params[i] - h.lr * m_new;
      momentum[i] = (float)m_new;
      params[i] = (float)th_new;
    } else {
      // Adam with bias correction
      const double m_new = h.beta * (double)momentum[i] + (1.0 - h.beta) * g;
      const double v_new = h.beta2 * (double)second[i] + (1.0 - h.beta2) * g * g;
      const double m_hat = m_new / (1.0 - std::pow(h.beta, (double)h.t));
      const double v_hat = v_new / (1.0 - std::pow(h.beta2, (double)h.t));
      const double den = std::sqrt(v_hat) + h.eps;
      const double th_new = (double)params[i] - h.lr * m_hat / den;
      const double g_hat = g / den;
      out.su.add(g_hat);
      out.su2.add(g_hat * g_hat);
      momentum[i] = (float)m_new;
      second[i] = (float)v_new;
      params[i] = (float)th_new;
    }
    prev_agg[i] = (float)g;
  }
}

}  // namespace

extern "C" {

int dmxo_create(int K, int64_t P, const int64_t* seg_offsets, int S, int dtype, dmxo** out) {
  if (!out) return kErrArg;
  *out = nullptr;
  if (K < 1 || K > 64 || P < 1 || S < 1 || S > 65536 || !seg_offsets) return kErrArg;
  if (dtype != kF32 && dtype != kBF16) return kErrArg;
  if (seg_offsets[0] != 0 || seg_offsets[S] != P) return kErrSegments;
  for (int s = 0; s < S; ++s)
    if (seg_offsets[s] > seg_offsets[s + 1]) return kErrSegments;
  dmxo* h = new (std::nothrow) dmxo;
  if (!h) return kErrArg;
  h->K = K; h->P = P; h->S = S; h->dtype = dtype;
  h->o.assign(seg_offsets, seg_offsets + S + 1);
  *out = h;
  return kOk;
}

int dmxo_state_len(const dmxo* h) { return h ? iHdr + h->K + 2 * h->S : kErrArg; }

int dmxo_begin(dmxo* h, const int32_t* batch_sizes, float lr, float beta) {
  if (!h || !batch_sizes) return kErrArg;
  h->b.assign(h->K, 0.0);
  int64_t B = 0;
  for (int k = 0; k < h->K; ++k) {
    if (batch_sizes[k] < 1) return kErrBatch;
    h->b[k] = (double)batch_sizes[k];
    B += batch_sizes[k];
  }
  h->B = (double)B;
  h->lr = (double)lr;      // the fp32 values, widened exactly
  h->beta = (double)beta;
  h->q.assign(h->K, Sum());
  h->V.assign(h->S, Sum());
  h->N.assign(h->S, Sum());
  h->c = Sum(); h->pp = Sum(); h->su = Sum(); h->su2 = Sum();
  h->adam = false;
  h->next = 0;
  h->open = true;
  return kOk;
}

int dmxo_begin_adam(dmxo* h, const int32_t* batch_sizes, float lr, float beta1, float beta2, float eps, int64_t t) {
  if (t < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f)) return kErrArg;
  const int rc = dmxo_begin(h, batch_sizes, lr, beta1);
  if (rc != kOk) return rc;
  h->adam = true;
  h->beta2 = (double)beta2;
  h->eps = (double)eps;
  h->t = t;
  return kOk;
}

// Process elements [j0, j0+n). grads[k], params, momentum, prev_agg address element j0.
// Ranges must arrive in ascending order without gaps, each starting on a multiple of 2^20.
// `second` is Adam's second-moment array (element j0 first); null in SGD mode.
int dmxo_range_adam(dmxo* h, int64_t j0, int64_t n, const void* const* grads, float* params,
                    float* momentum, float* second, float* prev_agg, int nthreads) {
  if (!h || !h->open || !grads || !params || !momentum || !prev_agg) return kErrArg;
  if (h->adam != (second != nullptr)) return kErrArg;
  if (j0 != h->next || j0 % kBlock != 0 || n < 1 || j0 + n > h->P) return kErrOrder;
  const int64_t nblocks = (n + kBlock - 1) / kBlock;
  std::vector<Partial> parts(nblocks);
  if (nthreads < 1) nthreads = 1;
  if ((int64_t)nthreads > nblocks) nthreads = (int)nblocks;
  auto work = [&](int t) {
    for (int64_t blk = t; blk < nblocks; blk += nthreads) {
      int64_t a = j0 + blk * kBlock, e = a + kBlock < j0 + n ? a + kBlock : j0 + n;
      run_block(*h, j0, a, e, grads, params, momentum, second, prev_agg, parts[blk]);
    }
  };
  if (nthreads == 1) {
    work(0);
  } else {
    std::vector<std::thread> pool;
    for (int t = 0; t < nthreads; ++t) pool.emplace_back(work, t);
    for (auto& th : pool) th.join();
  }
  for (int64_t blk = 0; blk < nblocks; ++blk) {  // combine in block order
    const Partial& p = parts[blk];
    for (int k = 0; k < h->K; ++k) h->q[k].add(p.q[k].value());
    h->c.add(p.c.value());
    h->pp.add(p.pp.value());
    h->su.add(p.su.value());
    h->su2.add(p.su2.value());
    for (size_t i = 0; i < p.V.size(); ++i) {
      h->V[p.seg_first + i].add(p.V[i].value());
      h->N[p.seg_first + i].add(p.N[i].value());
    }
  }
  h->next = j0 + n;
  return kOk;
}

int dmxo_range(dmxo* h, int64_t j0, int64_t n, const void* const* grads, float* params,
               float* momentum, float* prev_agg, int nthreads) {
  return dmxo_range_adam(h, j0, n, grads, params, momentum, nullptr, prev_agg, nthreads);
}

int dmxo_end(dmxo* h, float* out_state) {
  if (!h || !h->open || !out_state) return kErrArg;
  if (h->next != h->P) return kErrOrder;
  const int K = h->K, S = h->S;
  Sum As, Ds, Qw;
  for (int s = 0; s < S; ++s) { As.add(h->N[s].value()); Ds.add(h->V[s].value()); }
  for (int k = 0; k < K; ++k) Qw.add(h->b[k] * h->q[k].value());
  const double A = As.value(), D = Ds.value(), B = h->B;
  const double c = h->c.value(), pp = h->pp.value();
  int flags = 0;
  double trS = 0.0;
  if (K >= 2) trS = D / (K - 1); else flags |= fSingle;
  const double G2 = A - trS / B;
  double gns = 0.0;
  if (G2 > 0.0) gns = trS / G2; else flags |= fG2NonPos;
  double cosv = 0.0;
  if (A > 0.0 && pp > 0.0) cosv = c / std::sqrt(A * pp); else flags |= fCosUndef;
  const double sig2 = A > 0.0 ? trS / (B * A) : 0.0;
  const double sig = std::sqrt(sig2 > 0.0 ? sig2 : 0.0);
  bool bad = !std::isfinite((float)A) || !std::isfinite((float)pp);
  for (int k = 0; k < K; ++k) bad = bad || !std::isfinite((float)h->q[k].value());
  if (bad) flags |= fNonFinite;

  const int n = iHdr + K + 2 * S;
  for (int i = 0; i < n; ++i) out_state[i] = 0.0f;
  out_state[iB] = (float)B;
  out_state[iA] = (float)A;
  out_state[iTrS] = (float)trS;
  out_state[iG2] = (float)G2;
  out_state[iGns] = (float)gns;
  out_state[iCos] = (float)cosv;
  out_state[iDot] = (float)c;
  out_state[iPP] = (float)pp;
  out_state[iSig2] = (float)sig2;
  out_state[iSig] = (float)sig;
  out_state[iWq] = (float)(Qw.value() / B);
  out_state[iFlags] = (float)flags;
  if (h->adam) {
    const double mean = h->su.value() / (double)h->P;
    const double var = h->su2.value() / (double)h->P - mean * mean;
    out_state[12] = (float)mean;
    out_state[13] = (float)var;
    out_state[14] = (float)std::sqrt(var > 0.0 ? var : 0.0);
  }
  for (int k = 0; k < K; ++k) out_state[iHdr + k] = (float)h->q[k].value();
  for (int s = 0; s < S; ++s) {
    out_state[iHdr + K + s] = K >= 2 ? (float)(h->V[s].value() / (K - 1)) : 0.0f;
    out_state[iHdr + K + S + s] = (float)h->N[s].value();
  }
  h->open = false;
  return kOk;
}

// One whole step on host arrays (all of length P).
int dmxo_step(dmxo* h, const void* const* grads, const int32_t* batch_sizes, float* params,
              float* momentum, float lr, float beta, float* prev_agg, float* out_state,
              int nthreads) {
  int rc = dmxo_begin(h, batch_sizes, lr, beta);
  if (rc != kOk) return rc;
  rc = dmxo_range(h, 0, h->P, grads, params, momentum, prev_agg, nthreads);
  if (rc != kOk) return rc;
  return dmxo_end(h, out_state);
}

int dmxo_step_adam(dmxo* h, const void* const* grads, const int32_t* batch_sizes, float* params,
                   float* momentum, float* second, float lr, float beta1, float beta2, float eps, int64_t t,
                   float* prev_agg, float* out_state, int nthreads) {
  int rc = dmxo_begin_adam(h, batch_sizes, lr, beta1, beta2, eps, t);
  if (rc != kOk) return rc;
  rc = dmxo_range_adam(h, 0, h->P, grads, params, momentum, second, prev_agg, nthreads);
  if (rc != kOk) return rc;
  return dmxo_end(h, out_state);
}

// Window statistics over k consecutive state vectors (row-major k x n): per entry the mean and
// the population standard deviation, by the two-pass definition in fp64; the flags entry (11)
// gets the OR of the k flag words and spread 0. out has 2n entries: means, then deviations.
// (Section "State representation": state vectors are built from metrics collected over k
// iterations, as averages and standard deviations.)
int dmxo_window_stats(const float* states, int k, int n, float* out) {
  if (!states || !out || k < 1 || n <= iFlags) return kErrArg;
  for (int i = 0; i < n; ++i) {
    if (i == iFlags) {
      unsigned f = 0;
      for (int t = 0; t < k; ++t) f |= (unsigned)(int)states[(int64_t)t * n + i];
      out[i] = (float)f;
      out[n + i] = 0.0f;
      continue;
    }
    double sum = 0.0;
    for (int t = 0; t < k; ++t) sum += (double)states[(int64_t)t * n + i];
    const double mean = sum / k;
    double ss = 0.0;
    for (int t = 0; t < k; ++t) {
      const double d = (double)states[(int64_t)t * n + i] - mean;
      ss += d * d;
    }
    out[i] = (float)mean;
    out[n + i] = (float)std::sqrt(ss / k);
  }
  return kOk;
}

int dmxo_destroy(dmxo* h) {
  delete h;
  return kOk;
}

}  // extern "C"
