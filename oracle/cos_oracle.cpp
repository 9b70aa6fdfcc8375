// Float64 CPU oracle for the CoS verification step, C++ twin of cos_oracle.py (TEST INFRASTRUCTURE, not
// product code: only tests, the smoke check and the CPU-baseline leg of the benchmark may load it; nothing in the
// CUDA library links or calls it, and it shares no code with it).
//
// Same definition, same order of steps as the Python oracle, one (row, position) at a time in IEEE double, with
// OpenMP over the rows.  No blocking, no vector tricks, no fast-math.  Passages followed:
//   per-model distributions p_i = softmax(l_i / T)                      Sec. 3.1
//   weighted ensemble r = sum_i w_i p_i                                 Eq. 4 (n models: Sec. 4.1, Alg. 2)
//   logit-level combine r = softmax_M((sum_i w_i l_i) / T)              Eq. 5 (the mask M is a reading of this build)
//   accept test u <= min(1, r(x) / q(x))                                Eq. 6
//   residual resample x ~ norm(max(0, r - q)), bonus token              Sec. 3.2 (text after Eq. 6), Sec. 3.1, App. A.1
//   first rejection discards the tail                                   Sec. 3.1, Alg. 1
//   T = 0: one-hot distributions, lowest index wins ties                Sec. 4.1
// Conventions of this build (not fixed by the paper): Philox4x32-10 words, u = (2 (w >> 9) + 1) 2^-24, index-order
// inverse CDF "smallest k with CDF_k >= u S"; q(x) = 0 gives ratio +inf iff r(x) > 0; an empty residual draws from r.
// Pinned through tests/test_oracle_native.py: identical rows to the Python oracle (which carries the pins against
// the paper's closed forms) on seeded cases of every mode.

#include <math.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <limits>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr int kEnsemble = 0, kLogitLinear = 1;
constexpr unsigned kNonFinite = 1, kBadDraft = 2, kQZero = 4, kResidualEmpty = 8;
constexpr double kBoundaryRatio = 1e-5, kBoundaryCdf = 1e-6;

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds, Weyl key schedule.
void philox4x32_10(uint32_t c[4], uint32_t k0, uint32_t k1) {
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    const uint64_t p0 = 0xD2511F53ull * c[0], p1 = 0xCD9E8D57ull * c[2];
    const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
    const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
    const uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
    c[0] = n0;
    c[1] = lo1;
    c[2] = n2;
    c[3] = lo0;
  }
}

double word_to_uniform(uint32_t w) { return (2.0 * static_cast<double>(w >> 9) + 1.0) * 5.9604644775390625e-08; }

double half_to_double(uint16_t h) {
  const int sign = h >> 15, ex = (h >> 10) & 31, man = h & 1023;
  double v;
  if (ex == 0)
    v = ldexp(static_cast<double>(man), -24);
  else if (ex == 31)
    v = man ? std::numeric_limits<double>::quiet_NaN() : std::numeric_limits<double>::infinity();
  else
    v = ldexp(1.0 + man / 1024.0, ex - 15);
  return sign ? -v : v;
}

double load_logit(const void* base, int dtype, long long idx) {
  if (dtype == 0) return static_cast<double>(static_cast<const float*>(base)[idx]);
  const uint16_t h = static_cast<const uint16_t*>(base)[idx];
  if (dtype == 1) {
    const uint32_t bits = static_cast<uint32_t>(h) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return static_cast<double>(f);
  }
  return half_to_double(h);
}

struct Config {
  int n, combine, gamma, V, mask_model, bonus_model;
  double T, alpha;
  double w[8];
};

int first_argmax(const std::vector<double>& v) {
  int best = 0;
  for (int x = 1; x < static_cast<int>(v.size()); ++x)
    if (v[x] > v[best] || (v[best] != v[best] && v[x] == v[x])) best = x;  // a leading NaN never wins (numpy: NaN is the max; callers reject NaN first)
  return best;
}

double vec_max(const std::vector<double>& v) {  // NaN propagates, as numpy's max does
  double m = v[0];
  for (size_t x = 1; x < v.size(); ++x) {
    if (v[x] != v[x]) return v[x];
    if (v[x] > m) m = v[x];
  }
  return m;
}

void softmax_T(const std::vector<double>& l, double T, std::vector<double>& out) {
  const size_t V = l.size();
  out.resize(V);
  for (size_t x = 0; x < V; ++x) out[x] = l[x] / T;
  const double m = vec_max(out);
  double sum = 0.0;
  for (size_t x = 0; x < V; ++x) {
    out[x] = exp(out[x] - m);
    sum += out[x];
  }
  for (size_t x = 0; x < V; ++x) out[x] /= sum;
}

bool all_finite(const std::vector<double>& v) {
  for (double x : v)
    if (!std::isfinite(x)) return false;
  return true;
}

// r, q of one (row, position); false when some value is not finite
bool position_distributions(const std::vector<std::vector<double>>& l, const Config& c, int proposer, std::vector<double>& r,
                            std::vector<double>& q) {
  const int V = c.V, n = c.n;
  r.assign(V, 0.0);
  q.assign(V, 0.0);
  std::vector<double> tmp;
  if (c.T > 0.0) {
    if (c.combine == kEnsemble) {
      for (int i = 0; i < n; ++i) {
        softmax_T(l[i], c.T, tmp);
        for (int x = 0; x < V; ++x) r[x] = r[x] + c.w[i] * tmp[x];
        if (i == proposer) q = tmp;
      }
    } else {
      std::vector<double> cmb(V, 0.0);
      for (int i = 0; i < n; ++i)
        for (int x = 0; x < V; ++x) cmb[x] = cmb[x] + c.w[i] * l[i][x];
      softmax_T(l[proposer], c.T, q);
      if (c.mask_model >= 0) {
        const double bound = vec_max(l[c.mask_model]) + log(c.alpha);
        std::vector<double> z(V);
        for (int x = 0; x < V; ++x) z[x] = (l[c.mask_model][x] >= bound) ? cmb[x] / c.T : -std::numeric_limits<double>::infinity();
        const double m = vec_max(z);
        double sum = 0.0;
        for (int x = 0; x < V; ++x) {
          r[x] = (l[c.mask_model][x] >= bound) ? exp(z[x] - m) : 0.0;
          sum += r[x];
        }
        for (int x = 0; x < V; ++x) r[x] /= sum;
      } else {
        softmax_T(cmb, c.T, r);
      }
    }
  } else {
    bool usable = true;
    for (int i = 0; i < n && usable; ++i) {
      for (int x = 0; x < V; ++x)
        if (!(l[i][x] < std::numeric_limits<double>::infinity())) usable = false;
      if (usable && !std::isfinite(vec_max(l[i]))) usable = false;
    }
    if (usable) {
      q[first_argmax(l[proposer])] = 1.0;
      if (c.combine == kEnsemble) {
        for (int i = 0; i < n; ++i) r[first_argmax(l[i])] += c.w[i];
      } else {
        std::vector<double> cmb(V, 0.0);
        for (int i = 0; i < n; ++i)
          for (int x = 0; x < V; ++x) cmb[x] = cmb[x] + c.w[i] * l[i][x];
        if (c.mask_model >= 0) {
          const double bound = vec_max(l[c.mask_model]) + log(c.alpha);
          for (int x = 0; x < V; ++x)
            if (!(l[c.mask_model][x] >= bound)) cmb[x] = -std::numeric_limits<double>::infinity();
        }
        usable = std::isfinite(vec_max(cmb));
        r[first_argmax(cmb)] = 1.0;
      }
    }
    if (!usable)
      for (int x = 0; x < V; ++x) r[x] = std::numeric_limits<double>::quiet_NaN();
  }
  return all_finite(r) && all_finite(q);
}

struct Sample {
  int k;
  double lo, hi;
};

// index-order inverse CDF on unnormalised mass: smallest k whose running sum reaches u * total
Sample inverse_cdf(const std::vector<double>& mass, double u) {
  const int V = static_cast<int>(mass.size());
  std::vector<double> cdf(V);
  double run = 0.0;
  for (int x = 0; x < V; ++x) {
    run += mass[x];
    cdf[x] = run;
  }
  const double total = cdf[V - 1], target = u * total;
  int k = static_cast<int>(std::lower_bound(cdf.begin(), cdf.end(), target) - cdf.begin());
  if (k >= V) {
    k = V - 1;
    while (k > 0 && !(mass[k] > 0.0)) --k;
  }
  Sample s;
  s.k = k;
  s.lo = k > 0 ? cdf[k - 1] / total : 0.0;
  s.hi = cdf[k] / total;
  return s;
}

struct PosResult {
  bool accept = false, b_acc = false, b_smp = false;
  long long cand = -1;
  double ratio = NAN, r_d = NAN, q_d = NAN, S = NAN, prob = NAN;
  unsigned status = 0;
};

PosResult verify_position(const std::vector<std::vector<double>>& l, const Config& c, int proposer, bool is_bonus, int draft,
                          double u_acc, double u_smp) {
  PosResult res;
  if (is_bonus && c.bonus_model >= 0) proposer = c.bonus_model;
  std::vector<double> r, q;
  if (!position_distributions(l, c, proposer, r, q)) {
    res.status |= kNonFinite;
    return res;
  }
  if (is_bonus) {
    const std::vector<double>& law = (c.bonus_model >= 0) ? q : r;
    const Sample s = inverse_cdf(law, u_smp);
    res.cand = s.k;
    res.prob = law[s.k];
    res.b_smp = std::min(fabs(s.lo - u_smp), fabs(s.hi - u_smp)) < kBoundaryCdf;
    return res;
  }
  if (draft >= 0 && draft < c.V) {
    res.r_d = r[draft];
    res.q_d = q[draft];
    if (res.q_d > 0.0) {
      res.ratio = res.r_d / res.q_d;
    } else {
      res.status |= kQZero;
      res.ratio = res.r_d > 0.0 ? std::numeric_limits<double>::infinity() : 0.0;
    }
    const double thr = std::min(1.0, res.ratio);
    res.accept = u_acc <= thr;
    res.b_acc = fabs(u_acc - thr) < kBoundaryRatio;
  } else {
    res.status |= kBadDraft;
  }
  std::vector<double> resid(c.V);
  double S = 0.0;
  for (int x = 0; x < c.V; ++x) {
    resid[x] = std::max(0.0, r[x] - q[x]);
    S += resid[x];
  }
  res.S = S;
  Sample s;
  if (S > 0.0) {
    s = inverse_cdf(resid, u_smp);
  } else {
    if (!res.accept) res.status |= kResidualEmpty;
    s = inverse_cdf(r, u_smp);
  }
  res.cand = s.k;
  res.b_smp = std::min(fabs(s.lo - u_smp), fabs(s.hi - u_smp)) < kBoundaryCdf;
  return res;
}

}  // namespace

extern "C" {

// Threads the OpenMP runtime would use by default (1 when built without OpenMP).
int cos_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Verify `nrows` rows (indices in `rows`, or all B when rows is null) of a batch.  Logits [n][B][gamma+1][V] with
// element strides; dtype 0 = f32, 1 = bf16 bit patterns, 2 = IEEE half bit patterns.  `proposer` is [B] or, with
// per_pos, [B][gamma+1].  Per-position outputs are [B][gamma+1]; any of them may be null.  Returns 0, or -1 on a
// bad argument.
int cos_oracle_verify(const void* logits, int dtype, long long s_model, long long s_row, long long s_pos, int n, int B, int gamma,
                      int V, int combine, const float* weights, float temperature, int mask_model, float mask_alpha,
                      int bonus_model, const int* drafts, const int* proposer, int per_pos, unsigned long long seed,
                      unsigned long long offset, long long row_base, const int* rows, int nrows, int threads, int* accept_count,
                      int* out_tokens, unsigned* row_status, double* bonus_prob, unsigned char* accept, long long* cand,
                      double* ratio, double* r_d, double* q_d, double* S, unsigned char* boundary_accept,
                      unsigned char* boundary_sample, unsigned* pos_status, double* u_acc_out, double* u_smp_out) {
  if (!logits || n < 1 || n > 8 || B < 1 || gamma < 0 || V < 1 || !proposer || (gamma > 0 && !drafts)) return -1;
  Config c;
  c.n = n;
  c.combine = combine;
  c.gamma = gamma;
  c.V = V;
  c.mask_model = mask_model;
  c.bonus_model = bonus_model;
  c.T = static_cast<double>(temperature);
  c.alpha = static_cast<double>(mask_alpha);
  for (int i = 0; i < 8; ++i) c.w[i] = i < n ? static_cast<double>(weights[i]) : 0.0;
  const int P = gamma + 1;
  const int count = rows ? nrows : B;
#ifdef _OPENMP
  if (threads > 0) omp_set_num_threads(threads);
#pragma omp parallel for schedule(dynamic, 1)
#endif
  for (int t = 0; t < count; ++t) {
    const int b = rows ? rows[t] : t;
    std::vector<std::vector<double>> l(n, std::vector<double>(V));
    std::vector<PosResult> pos(P);
    for (int j = 0; j < P; ++j) {
      for (int i = 0; i < n; ++i) {
        const long long at = i * s_model + b * s_row + j * s_pos;
        for (int x = 0; x < V; ++x) l[i][x] = load_logit(logits, dtype, at + x);
      }
      uint32_t ctr[4] = {static_cast<uint32_t>(static_cast<unsigned long long>(row_base + b)), static_cast<uint32_t>(j),
                         static_cast<uint32_t>(offset), static_cast<uint32_t>(offset >> 32)};
      philox4x32_10(ctr, static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32));
      const double ua = word_to_uniform(ctr[0]), us = word_to_uniform(ctr[1]);
      const int pi = proposer[per_pos ? b * P + j : b];
      const bool is_bonus = (j == gamma);
      pos[j] = verify_position(l, c, pi, is_bonus, is_bonus ? 0 : drafts[b * gamma + j], ua, us);
      const long long o = static_cast<long long>(b) * P + j;
      if (accept) accept[o] = pos[j].accept;
      if (cand) cand[o] = pos[j].cand;
      if (ratio) ratio[o] = pos[j].ratio;
      if (r_d) r_d[o] = pos[j].r_d;
      if (q_d) q_d[o] = pos[j].q_d;
      if (S) S[o] = pos[j].S;
      if (boundary_accept) boundary_accept[o] = pos[j].b_acc;
      if (boundary_sample) boundary_sample[o] = pos[j].b_smp;
      if (pos_status) pos_status[o] = pos[j].status;
      if (u_acc_out) u_acc_out[o] = ua;
      if (u_smp_out) u_smp_out[o] = us;
    }
    int a = gamma;
    for (int j = 0; j < gamma; ++j)
      if (!pos[j].accept) {
        a = j;
        break;
      }
    accept_count[b] = a;
    for (int j = 0; j < P; ++j) out_tokens[static_cast<long long>(b) * P + j] = j < a ? drafts[b * gamma + j] : -1;
    out_tokens[static_cast<long long>(b) * P + a] = static_cast<int>(pos[a].cand);
    if (bonus_prob) bonus_prob[b] = (a == gamma) ? pos[gamma].prob : NAN;
    unsigned st = 0;
    for (int j = 0; j <= a; ++j) st |= pos[j].status;
    row_status[b] = st;
  }
  return 0;
}

}  // extern "C"
