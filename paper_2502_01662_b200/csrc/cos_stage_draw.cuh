// Staged launches of the CoS verification step: what the drawing stages (residual resample of Sec. 3.2, bonus token
// of Sec. 3.1) keep out of the kernel body: masses of big tokens in fp64 and the two one-sweep forms of the sweep.
// Included by cos_verify.cu only.
#pragma once

#include "cos_stage_shared.cuh"

using namespace cosv;

namespace {

// Mass of one "big" token (more than 2^-8 of some normaliser) in fp64 from the stored logits: r - q
// clipped at zero, or r.  Rare; kept out of line so that the mass loop stays small.
// `staged`/`k`: where the token's logits sit in shared memory (null: read them from global memory).
template <int DT, int MODE>
__device__ __noinline__ double big_token_mass(const KParams& p, const SoftPart* fsoft, const char* base, int e, int draw,
                                              const uint4* staged, int k, bool masked, float thr, int pis) {
  if (e >= p.V) return 0.0;
  double r64 = 0.0, q64 = 0.0;
  float lv[COS_MAX_MODELS];
  if (staged != nullptr) {
    for (int i = 0; i < p.n; ++i) lv[i] = Elem<DT>::pick(staged + i * 32, k);
  } else {
    for (int i = 0; i < p.n; ++i)
      lv[i] = Elem<DT>::load1(base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes, e);  // all loads first
  }
  if (MODE == kEnsembleSample) {
    for (int i = 0; i < p.n; ++i) {
      double pr = exp2(static_cast<double>(lv[i]) * p.cT64 - static_cast<double>(fsoft[i].ref)) / fsoft[i].s;
      r64 += p.w64[i] * pr;
      if (i == pis) q64 = pr;
    }
  } else {
    double cd = 0.0;
    for (int i = 0; i < p.n; ++i) cd = fma(p.w64[i], static_cast<double>(lv[i]), cd);
    bool in = !masked || (lv[p.mask_model] >= thr);
    r64 = in ? exp2(cd * p.cT64 - static_cast<double>(fsoft[1].ref)) / fsoft[1].s : 0.0;
    q64 = exp2(static_cast<double>(lv[pis]) * p.cT64 - static_cast<double>(fsoft[0].ref)) / fsoft[0].s;
  }
  return draw == kDrawR ? r64 : (draw == kDrawQ ? q64 : fmax(0.0, r64 - q64));
}

// 2^a and, when `in`, 2^b in fp64: the two channel terms of a big entry.  Out of line.
__device__ __noinline__ double2 big_pair(double a, double b, bool in) {
  return make_double2(exp2(a), in ? exp2(b) : 0.0);
}

// One-sweep drawing stage, a vector that holds a big entry (more than 2^-8 of a normaliser), done again
// entry by entry from the stored logits: big entries in fp64 into the thread's slots `bigacc` ([0] Z_A,
// [kThreads] Z_B, [2 kThreads] and [3 kThreads] the sums over entries with a positive mass), the others as the
// sweep does them, returned as (Z_A, Z_B, sum A, sum B) of this vector.  Rare; out of line.
template <int DT, int MODE>
__device__ __noinline__ float4 one_sweep_big_vector(const KParams& p, const OneSweep& c, const char* base, int e0, int pis,
                                                    bool masked, float thr, double* bigacc) {
  constexpr int E = Elem<DT>::E;
  float4 out = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int k = 0; k < E; ++k) {
    const int e = e0 + k;
    if (e >= p.V) break;
    float xa, xb;
    double cb;
    bool in = true;
    if (MODE == kEnsembleSample) {
      xa = Elem<DT>::load1(base, e);
      xb = Elem<DT>::load1(base + p.s_model * Elem<DT>::bytes, e);
      cb = static_cast<double>(xb);
    } else {
      xb = 0.f;
      cb = 0.0;
      xa = 0.f;
      for (int i = 0; i < p.n; ++i) {
        const float x = Elem<DT>::load1(base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes, e);
        xb = fmaf(p.w[i], x, xb);
        cb = fma(p.w64[i], static_cast<double>(x), cb);
        if (i == pis) xa = x;
        if (masked && i == p.mask_model) in = (x >= thr);
      }
    }
    const float eA = ex2_approx(fmaf(xa, p.cT, c.nrefA));
    const float eB = in ? ex2_approx(fmaf(xb, p.cT, c.nrefB)) : 0.f;
    if (eA > c.btA || eB > c.btB) {
      const double dA = exp2(static_cast<double>(xa) * p.cT64 - c.drefA);
      const double dB = in ? exp2(cb * p.cT64 - c.drefB) : 0.0;
      bigacc[0] += dA;
      bigacc[kThreads] += dB;
      if (c.ctA64 * dA + c.ctB64 * dB > 0.0) {
        bigacc[2 * kThreads] += dA;
        bigacc[3 * kThreads] += dB;
      }
    } else {
      const bool pos = __fadd_rn(__fmul_rn(c.ctA, eA), __fmul_rn(c.ctB, eB)) > 0.f;
      out.x += eA;
      out.y += eB;
      out.z += pos ? eA : 0.f;
      out.w += pos ? eB : 0.f;
    }
  }
  return out;
}

// The one-sweep drawing stage with a channel per model (ensembles of three or four; Eq. 4): r - q, r and q are all
// sums over the models of k_i e_i / Z_i with e_i = 2^(l_i c - ref_i), so a token's mass is that sum clipped at zero.
// One big entry (more than 2^-8 of a normaliser) of that sweep, in fp64 from its logits: into the thread's slots
// `bigacc` ([i kThreads] Z_i, [(4 + i) kThreads] the sum of e_i where the mass is positive).  Rare; out of line.
__device__ __noinline__ void one_sweep_big_token_n(const KParams& p, const OneSweepN& c, float x0, float x1, float x2, float x3,
                                                   double* bigacc) {
  const float x[4] = {x0, x1, x2, x3};
  double d[4], tot = 0.0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    d[i] = exp2(static_cast<double>(x[i]) * p.cT64 - c.dref[i]);  // (a model the ensemble does not have: -inf, no term)
    tot += c.ct64[i] * d[i];
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    bigacc[i * kThreads] += d[i];
    if (tot > 0.0) bigacc[(4 + i) * kThreads] += d[i];
  }
}

// The sweep itself: this block's steps [rank, rank + 1) / lparts of the unit's steps, its warps taking them in
// turn; every step (32 lanes x E entries, in token order) leaves, per model, the sum of e_i over its tokens with a
// positive mass (the set is decided with the normalisers of stage 0, products rounded one by one so that equal
// terms cancel exactly; over that set the mass is linear in the 1/Z_i), and the warp's share of the refined
// normalisers goes to sh.wsoft.  `kc` returns the coefficients k_i of what is drawn: max(0, r - q), r, or q.
template <int DT>
__device__ __forceinline__ void one_sweep_channels(const KParams& p, Shared& sh, uint4* ring, const char* base, int b, int rank,
                                                   int lparts, int pis, bool is_bonus, bool draw_q, int emit, bool vec_ok,
                                                   double (&kc)[4]) {
  constexpr int E = Elem<DT>::E;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float ct[4], nref[4], bt[4];
  double ct64[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const bool live = i < p.n;
    const double sel = (i == pis) ? 1.0 : 0.0;
    kc[i] = !live ? 0.0 : (!is_bonus ? p.w64[i] - sel : (draw_q ? sel : p.w64[i]));
    ct64[i] = live ? kc[i] / sh.fsoft[i].s : 0.0;  // with the first estimates: signs only
    ct[i] = static_cast<float>(ct64[i]);
    nref[i] = live ? -sh.fsoft[i].ref : 0.f;
    bt[i] = live ? sh.big_thr[i] : INFINITY;
  }
  if (tid == 0) {
    OneSweepN& c = one_sweep_consts_n(sh);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      c.ct[i] = ct[i];
      c.nref[i] = nref[i];
      c.bt[i] = bt[i];
      c.ct64[i] = ct64[i];
      c.dref[i] = (i < p.n) ? static_cast<double>(sh.fsoft[i].ref) : 0.0;
    }
  }
  // the big terms sit in shared memory (the staging ring is idle during this sweep), one slot per thread and sum
  double* bigacc = reinterpret_cast<double*>(ring) + tid;
#pragma unroll
  for (int q = 0; q < 8; ++q) bigacc[q * kThreads] = 0.0;
  __syncthreads();
  const long long row_step = p.s_model * Elem<DT>::bytes;
  const int blk_lo = static_cast<int>(static_cast<long long>(rank) * p.nsteps / lparts);
  const int blk_hi = static_cast<int>(static_cast<long long>(rank + 1) * p.nsteps / lparts);
  const size_t rec_at = static_cast<size_t>(b) * p.nsteps;
  const int nfull = vec_ok ? p.V / (32 * E) : 0;  // steps below this are whole aligned vectors
  float zs[4] = {0.f, 0.f, 0.f, 0.f};
  bool hasbig = false;
  Raw4 nx;
#pragma unroll
  for (int i = 0; i < 4; ++i) nx.r[i] = make_uint4(0u, 0u, 0u, 0u);
  auto fetch = [&](int s) {
    const char* src = base + static_cast<long long>(s * 32 + lane) * 16;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (i < p.n) nx.r[i] = ldg_stream16(src + i * row_step);
  };
  if (blk_lo + warp < blk_hi && blk_lo + warp < nfull) fetch(blk_lo + warp);
  for (int s = blk_lo + warp; s < blk_hi; s += kWarps) {
    const int e0 = (s * 32 + lane) * E;
    const bool have_raw = s < nfull;
    const Raw4 cur = nx;
    float x[4][E];
    if (have_raw) {
      const int sn = s + kWarps;
      if (sn < blk_hi && sn < nfull) fetch(sn);
#pragma unroll
      for (int i = 0; i < 4; ++i) Elem<DT>::unpack(cur.r[i], x[i]);
    } else {
      // ragged or unaligned step: entry by entry; entries beyond V read as -inf (no mass, outside every set)
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (i < p.n) load_chunk<DT>(base + i * row_step, e0, p.V, vec_ok, x[i]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (i >= p.n) {
#pragma unroll
        for (int k = 0; k < E; ++k) x[i][k] = -INFINITY;
      }
    }
    float vz[4] = {0.f, 0.f, 0.f, 0.f}, va[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < E; ++k) {
      // (channels in pairs through the packed fp32 instructions: the same values, fewer instructions)
      float t[4], e[4], m[4];
      fma2(t[0], t[1], x[0][k], x[1][k], p.cT, p.cT, nref[0], nref[1]);
      fma2(t[2], t[3], x[2][k], x[3][k], p.cT, p.cT, nref[2], nref[3]);
#pragma unroll
      for (int i = 0; i < 4; ++i) e[i] = ex2_approx(t[i]);
      add2(vz[0], vz[1], vz[0], vz[1], e[0], e[1]);
      add2(vz[2], vz[3], vz[2], vz[3], e[2], e[3]);
      mul2(m[0], m[1], ct[0], ct[1], e[0], e[1]);
      mul2(m[2], m[3], ct[2], ct[3], e[2], e[3]);
      const float acc = __fadd_rn(__fadd_rn(__fadd_rn(m[0], m[1]), m[2]), m[3]);
      if (acc > 0.f) {
        add2(va[0], va[1], va[0], va[1], e[0], e[1]);
        add2(va[2], va[3], va[2], va[3], e[2], e[3]);
      }
    }
    // rare: the vector may hold a big entry (no term is negative, so a big entry makes its vector's sum big)
    const bool big = (vz[0] > bt[0]) || (vz[1] > bt[1]) || (vz[2] > bt[2]) || (vz[3] > bt[3]);
    if (big) {
      // the vector again, its big entries in fp64 (entries beyond V and models the ensemble does not have are -inf)
#pragma unroll
      for (int i = 0; i < 4; ++i) vz[i] = va[i] = 0.f;
#pragma unroll
      for (int k = 0; k < E; ++k) {
        float e[4], acc = 0.f;
        bool bigtok = false;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          e[i] = ex2_approx(fmaf(x[i][k], p.cT, nref[i]));
          bigtok |= e[i] > bt[i];
          acc = __fadd_rn(acc, __fmul_rn(ct[i], e[i]));
        }
        if (bigtok) {
          one_sweep_big_token_n(p, one_sweep_consts_n(sh), x[0][k], x[1][k], x[2][k], x[3][k], bigacc);
        } else {
          const float in_p = (acc > 0.f) ? 1.f : 0.f;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            vz[i] += e[i];
            va[i] = fmaf(in_p, e[i], va[i]);
          }
        }
      }
      hasbig = true;
    }
    // the step's sums over the warp
    double mine = 0.0;
    const bool anybig = __any_sync(0xffffffffu, hasbig);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      zs[i] += vz[i];
      float r = va[i];
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) r += __shfl_xor_sync(0xffffffffu, r, d);
      double dr = static_cast<double>(r);
      if (anybig) {
        double t = bigacc[(4 + i) * kThreads];
        bigacc[(4 + i) * kThreads] = 0.0;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) t += shfl_double(t, lane ^ d);
        dr += t;
      }
      if (lane == i) mine = dr;
    }
    if (emit && lane < 4) {
      double* dst = (lane == 0) ? p.srung : (lane == 1 ? p.srungB : (lane == 2 ? p.srungC : p.srungD));
      dst[rec_at + s] = mine;
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    double t = static_cast<double>(zs[i]) + bigacc[i * kThreads];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) t += shfl_double(t, lane ^ d);
    if (lane == 0) {
      sh.wsoft[warp][i].s = t;
      sh.wsoft[warp][i].ref = (i < p.n) ? sh.fsoft[i].ref : 0.f;
    }
  }
}

// The one-sweep drawing stage with two channel sums per step (stage 3), the sweep itself.  (Inline: as a function
// of its own, with or without copies of the launch parameters it uses, its loop was slower by a quarter to a half.)
template <int DT, int MODE>
__device__ __forceinline__ void one_sweep_pair(const KParams& p, Shared& sh, uint4* ring, const char* base, int b, int rank, int lparts,
                                            int pis, bool masked, float thr, bool is_bonus, bool draw_q, int emit, bool vec_ok,
                                            double (&kc)[4]) {
  constexpr int E = Elem<DT>::E;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  auto row_of = [&](int i) -> const void* { return base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes; };
  // what the loop needs of the launch parameters
  const float cT = p.cT, w0 = p.w[0], w1 = p.w[1];
  const int n = p.n, mask_model = p.mask_model;
  double* const rec_a = p.srung;
  double* const rec_b = p.srungB;
  // ---- the drawing stages in one sweep.  A token's mass is k_A e_A / Z_A + k_B e_B / Z_B clipped at zero,
  // where the two channels are the two models (ensemble, n = 2) or the proposer's and the combined logits
  // (logit level), and (k_A, k_B) says what is drawn: max(0, r - q), r, or q.  The set of tokens with a
  // positive mass is decided with the normalisers stage 0 left (they are good to 1e-7, and a token whose sign
  // that could change carries no mass to speak of); over that set the mass is LINEAR in 1/Z_A and 1/Z_B,
  // so this sweep only adds up e_A and e_B over that set, step by step, and over everything for the refined
  // normalisers of stage 1.  Whoever locates the token turns the sums into masses once the normalisers are
  // complete.
  // Terms above 2^-8 of a normaliser go through fp64, as in stage 1.
  double kA, kB;
  if (MODE == kEnsembleSample) {
    const double selA = (pis == 0) ? 1.0 : 0.0, selB = (pis == 1) ? 1.0 : 0.0;
    kA = !is_bonus ? p.w64[0] - selA : (draw_q ? selA : p.w64[0]);
    kB = !is_bonus ? p.w64[1] - selB : (draw_q ? selB : p.w64[1]);
  } else {
    kA = !is_bonus ? -1.0 : (draw_q ? 1.0 : 0.0);
    kB = (is_bonus && draw_q) ? 0.0 : 1.0;
  }
  const double ctA64 = kA / sh.fsoft[0].s, ctB64 = kB / sh.fsoft[1].s;  // with the first estimates: signs only
  const float ctA = static_cast<float>(ctA64), ctB = static_cast<float>(ctB64);
  const float nrefA = -sh.fsoft[0].ref, nrefB = -sh.fsoft[1].ref;
  const float btA = sh.big_thr[0], btB = sh.big_thr[1];
  const double drefA = static_cast<double>(sh.fsoft[0].ref), drefB = static_cast<double>(sh.fsoft[1].ref);
  const char* row0 = reinterpret_cast<const char*>(row_of(0));
  const long long row_step = p.s_model * Elem<DT>::bytes;
  // this block's steps [blk_lo, blk_hi); its warps take them in turn, so that the block reads 8 KB of
  // every row at a time; every step (32 lanes x E entries, in token order) leaves its two sums on record
  const int blk_lo = static_cast<int>(static_cast<long long>(rank) * p.nsteps / lparts);
  const int blk_hi = static_cast<int>(static_cast<long long>(rank + 1) * p.nsteps / lparts);
  const size_t rec_at = static_cast<size_t>(b) * p.nsteps;
  const int nfull = vec_ok ? p.V / (32 * E) : 0;  // steps below this are whole aligned vectors
  float zsA = 0.f, zsB = 0.f, aA = 0.f, aB = 0.f;  // small terms: normalisers (all steps), sums of the step
  // the big terms of the same four sums sit in shared memory (the staging ring is idle during this sweep),
  // one slot per thread and sum: [0] Z_A, [1] Z_B, [2] and [3] the step's sums
  double* bigacc = reinterpret_cast<double*>(ring) + tid;
#pragma unroll
  for (int q = 0; q < 4; ++q) bigacc[q * kThreads] = 0.0;
  bool hasbig = false;
  if (tid == 0) {
    OneSweep& c = one_sweep_consts(sh);
    c.ctA = ctA;
    c.ctB = ctB;
    c.nrefA = nrefA;
    c.nrefB = nrefB;
    c.btA = btA;
    c.btB = btB;
    c.ctA64 = ctA64;
    c.ctB64 = ctB64;
    c.drefA = drefA;
    c.drefB = drefB;
  }
  __syncthreads();
  // one vector of entries: channel arguments xa (proposer's or model 0's logits) and xb (model 1's or the
  // combined logits)
  // (entries outside the mask arrive with xb = -inf: their e_B is zero)
  const float nctA = -ctA;
  auto eat = [&](const float (&xa)[E], const float (&xb)[E]) -> bool {
    float vzA = 0.f, vzB = 0.f, vaA = 0.f, vaB = 0.f;
#pragma unroll
    for (int k = 0; k < E; ++k) {
      // k_A e_A / Z_A + k_B e_B / Z_B > 0 with the products rounded one by one: where r and q coincide
      // neither side exceeds the other, as in exact arithmetic
      // The two channels side by side in the packed fp32 instructions: the same values, half the instructions
      // (workload 3: 89.9 -> 89.0 us per call, workload 5: 549.0 -> 547.1; the combined logits of the logit level
      // stay scalar: in pairs they made workload 5 slower).
      float tA, tB, mA, mB;
      fma2(tA, tB, xa[k], xb[k], cT, cT, nrefA, nrefB);
      const float eA = ex2_approx(tA);
      const float eB = ex2_approx(tB);
      mul2(mA, mB, nctA, ctB, eA, eB);
      add2(vzA, vzB, vzA, vzB, eA, eB);
      if (mB > mA) add2(vaA, vaB, vaA, vaB, eA, eB);
    }
    // rare: the vector may hold a big entry (no term is negative, so a big entry makes its vector's sum
    // big); the caller does the vector again, big entries in fp64
    if (vzA > btA || vzB > btB) return true;
    zsA += vzA;
    zsB += vzB;
    aA += vaA;
    aB += vaB;
    return false;
  };
  // a vector with a big entry, entry by entry from the stored logits, out of line (ragged steps)
  auto redo_from_memory = [&](int e0) {
    const float4 r = one_sweep_big_vector<DT, MODE>(p, one_sweep_consts(sh), base, e0, pis, masked, thr, bigacc);
    zsA += r.x;
    zsB += r.y;
    aA += r.z;
    aB += r.w;
    hasbig = true;
  };
  // the same from the two vectors at hand (models beyond the second are read again, entry by entry)
  auto redo = [&](const uint4& r0, const uint4& r1, int e0) {
    float x0[E], x1[E];
    Elem<DT>::unpack(r0, x0);
    Elem<DT>::unpack(r1, x1);
    float vzA = 0.f, vzB = 0.f, vaA = 0.f, vaB = 0.f;
#pragma unroll
    for (int k = 0; k < E; ++k) {
      float xa, xb;
      bool in = true;
      if (MODE == kEnsembleSample) {
        xa = x0[k];
        xb = x1[k];
      } else {
        xb = fmaf(p.w[0], x0[k], 0.f);
        if (p.n >= 2) xb = fmaf(p.w[1], x1[k], xb);
        for (int i = 2; i < p.n; ++i) xb = fmaf(p.w[i], Elem<DT>::load1(row_of(i), e0 + k), xb);
        xa = (pis == 0) ? x0[k] : (pis == 1 ? x1[k] : Elem<DT>::load1(row_of(pis), e0 + k));
        if (masked) {
          const int mm = p.mask_model;
          const float xm = (mm == 0) ? x0[k] : (mm == 1 ? x1[k] : Elem<DT>::load1(row_of(mm), e0 + k));
          in = (xm >= thr);
        }
      }
      const float eA = ex2_approx(fmaf(xa, p.cT, nrefA));
      const float eB = in ? ex2_approx(fmaf(xb, p.cT, nrefB)) : 0.f;
      if (eA > btA || eB > btB) {
        double cb;
        if (MODE == kEnsembleSample) {
          cb = static_cast<double>(xb);
        } else {
          cb = fma(p.w64[0], static_cast<double>(x0[k]), 0.0);
          if (p.n >= 2) cb = fma(p.w64[1], static_cast<double>(x1[k]), cb);
          for (int i = 2; i < p.n; ++i) cb = fma(p.w64[i], static_cast<double>(Elem<DT>::load1(row_of(i), e0 + k)), cb);
        }
        const double2 d = big_pair(static_cast<double>(xa) * p.cT64 - drefA, cb * p.cT64 - drefB, in);
        bigacc[0] += d.x;
        bigacc[kThreads] += d.y;
        if (ctA64 * d.x + ctB64 * d.y > 0.0) {
          bigacc[2 * kThreads] += d.x;
          bigacc[3 * kThreads] += d.y;
        }
      } else {
        const bool pos = __fadd_rn(__fmul_rn(ctA, eA), __fmul_rn(ctB, eB)) > 0.f;
        vzA += eA;
        vzB += eB;
        vaA += pos ? eA : 0.f;
        vaB += pos ? eB : 0.f;
      }
    }
    zsA += vzA;
    zsB += vzB;
    aA += vaA;
    aB += vaB;
    hasbig = true;
  };
  // the channel arguments of one step from the lane's vectors (the first two models' fetched ahead)
  auto feed = [&](const uint4& r0, const uint4& r1, int s) {
    const int e0 = (s * 32 + lane) * E;
    if (MODE == kEnsembleSample) {
      float xa[E], xb[E];
      Elem<DT>::unpack(r0, xa);
      Elem<DT>::unpack(r1, xb);
      if (eat(xa, xb)) redo(r0, r1, e0);
    } else {
      float cmb[E], vq[E];
      unsigned inb = 0u;
#pragma unroll
      for (int k = 0; k < E; ++k) cmb[k] = 0.f;
      auto take = [&](int i, const uint4& raw) {
        float x[E];
        Elem<DT>::unpack(raw, x);
        const float wi = (i == 0) ? w0 : (i == 1 ? w1 : p.w[i]);
#pragma unroll
        for (int k = 0; k < E; ++k) {
          cmb[k] = fmaf(wi, x[k], cmb[k]);
          if (i == pis) vq[k] = x[k];
          if (masked && i == mask_model) inb |= (x[k] >= thr) ? (1u << k) : 0u;
        }
      };
      take(0, r0);
      if (n >= 2) take(1, r1);
      for (int i = 2; i < n; ++i) take(i, ldg_stream16(row0 + i * row_step + static_cast<long long>(s * 32 + lane) * 16));
      if (masked) {
#pragma unroll
        for (int k = 0; k < E; ++k) cmb[k] = ((inb >> k) & 1u) ? cmb[k] : -INFINITY;
      }
      if (eat(vq, cmb)) redo(r0, r1, e0);
    }
  };
  const bool pair = (MODE == kEnsembleSample) || (n >= 2);
  uint4 nx0 = make_uint4(0u, 0u, 0u, 0u), nx1 = nx0;
  if (blk_lo + warp < blk_hi && blk_lo + warp < nfull) {
    const char* src = row0 + static_cast<long long>((blk_lo + warp) * 32 + lane) * 16;
    nx0 = ldg_stream16(src);
    if (pair) nx1 = ldg_stream16(src + row_step);
  }
  for (int s = blk_lo + warp; s < blk_hi; s += kWarps) {
    if (s < nfull) {
      const uint4 a0 = nx0, a1 = nx1;
      const int sn = s + kWarps;
      if (sn < blk_hi && sn < nfull) {
        const char* src = row0 + static_cast<long long>(sn * 32 + lane) * 16;
        nx0 = ldg_stream16(src);
        if (pair) nx1 = ldg_stream16(src + row_step);
      }
      feed(a0, a1, s);
    } else {
      // ragged or unaligned step: entry by entry; entries beyond V read as -inf (no mass, outside every set)
      const int e0 = (s * 32 + lane) * E;
      if (MODE == kEnsembleSample) {
        float xa[E], xb[E];
        load_chunk<DT>(row_of(0), e0, p.V, vec_ok, xa);
        load_chunk<DT>(row_of(1), e0, p.V, vec_ok, xb);
        if (eat(xa, xb)) redo_from_memory(e0);
      } else {
        float cmb[E], vq[E];
        unsigned inb = 0u;
#pragma unroll
        for (int k = 0; k < E; ++k) cmb[k] = 0.f;
        for (int i = 0; i < p.n; ++i) {
          float x[E];
          load_chunk<DT>(row_of(i), e0, p.V, vec_ok, x);
#pragma unroll
          for (int k = 0; k < E; ++k) {
            cmb[k] = (e0 + k < p.V) ? fmaf(p.w[i], x[k], cmb[k]) : -INFINITY;
            if (i == pis) vq[k] = x[k];
            if (masked && i == p.mask_model) inb |= (x[k] >= thr) ? (1u << k) : 0u;
          }
        }
        if (masked) {
#pragma unroll
          for (int k = 0; k < E; ++k) cmb[k] = ((inb >> k) & 1u) ? cmb[k] : -INFINITY;
        }
        if (eat(vq, cmb)) redo_from_memory(e0);
      }
    }
    // the step's two sums over the warp: the lower half of the lanes ends up with the first, the upper half with the
    // second (one exchange, then one sum per lane instead of two)
    const bool upper = (lane & 16) != 0;
    float mine = (upper ? aB : aA) + __shfl_xor_sync(0xffffffffu, upper ? aA : aB, 16);
#pragma unroll
    for (int d = 8; d > 0; d >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, d);
    double dm = static_cast<double>(mine);
    if (__any_sync(0xffffffffu, hasbig)) {
      const double ta = bigacc[2 * kThreads], tb = bigacc[3 * kThreads];
      bigacc[2 * kThreads] = bigacc[3 * kThreads] = 0.0;
      double tm = (upper ? tb : ta) + shfl_double(upper ? ta : tb, lane ^ 16);
#pragma unroll
      for (int d = 8; d > 0; d >>= 1) tm += shfl_double(tm, lane ^ d);
      dm += tm;
    }
    if ((lane & 15) == 0 && emit) (upper ? rec_b : rec_a)[rec_at + s] = dm;
    aA = aB = 0.f;
  }
  {
    double tA = static_cast<double>(zsA) + bigacc[0], tB = static_cast<double>(zsB) + bigacc[kThreads];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      tA += shfl_double(tA, lane ^ d);
      tB += shfl_double(tB, lane ^ d);
    }
    if (lane == 0) {
      sh.wsoft[warp][0].s = tA;
      sh.wsoft[warp][0].ref = sh.fsoft[0].ref;
      sh.wsoft[warp][1].s = tB;
      sh.wsoft[warp][1].ref = sh.fsoft[1].ref;
    }
  }
  kc[0] = kA;
  kc[1] = kB;
}

}  // namespace
