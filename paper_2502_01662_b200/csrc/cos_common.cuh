// Shared device helpers of the CoS verification kernels: element types, streaming loads, Philox4x32-10,
// the base-2 softmax accumulators and their reductions, and the launch parameters.
#ifndef COS_COMMON_CUH
#define COS_COMMON_CUH
#include <cooperative_groups.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <string>

#include "cos_verify.h"

namespace cg = cooperative_groups;

namespace cosv {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxSlots = COS_MAX_MODELS + 2;
constexpr int kNoReject = 0x7fffffff;
constexpr int kPackedP = 13;  // rows of up to this many positions keep their accept flags in the arrival word
constexpr int kDrawResidual = 0, kDrawR = 1, kDrawQ = 2;  // what a token is drawn from: max(0, r - q), r, or q
constexpr double kBigShare = 1.0 / 256.0;  // probabilities above 2^-8 get fp64 treatment when tokens are drawn
constexpr int kRingVecs = 8;                 // 16-byte vectors per lane staged ahead in sweep 2 (4 KB per warp)
constexpr int kRingBytes = kWarps * kRingVecs * 32 * 16;
constexpr int kRecG = 16;                    // running totals per warp kept in global memory between the drawing stages
constexpr int kMaxParts = 16;                // blocks that share one unit in the drawing stages
constexpr int kRec = 64;                     // running totals recorded per warp in sweep 2

enum Mode { kEnsembleSample = 0, kLogitSample = 1, kEnsembleGreedy = 2, kLogitGreedy = 3 };

struct UnitStats {  // what stage 1 needs from stage 0 about one (row, position)
  double s[COS_MAX_MODELS];   // normalisers sum 2^(arg - ref)
  float ref[COS_MAX_MODELS];  // reference exponents
  float thr32;                // plausibility threshold
  int pad[3];
};

struct KParams {
  const void* logits;
  long long s_model, s_row, s_pos;  // element strides
  const int* drafts;
  const int* proposer;
  int n, V, gamma, P, B;
  int mask_model;
  int vec_ok;   // every row start is 16-byte aligned
  int nsteps;   // ceil(V / (32 * E))
  int flags;
  int num_units, num_clusters;
  int per_pos;      // proposer is [B][gamma+1] (the model that proposed each draft) instead of [B]
  int early_exit;   // positions after a row's known first rejection may be left unread (barrier-free form only)
  int greedy;       // T = 0: no drawing stages; the fourth word of a unit's result carries the bonus probability
  int bonus_model;  // >= 0: the token after gamma acceptances follows this model's own distribution; -1: the combined one
  int parts;     // blocks that share one unit in stages 1 and 2
  int early_dependents;  // stage 0: let the next launch in the stream take places while this one runs
  int inputs_settled;    // stage 0, barrier-free form: the inputs may be read before the kernel ahead in the stream is complete
  int draw_cluster;      // one-sweep drawing stages: the blocks of a unit are a thread-block cluster and meet at its barrier
  int max_jobs;  // capacity of the job list
  float w[COS_MAX_MODELS];
  double w64[COS_MAX_MODELS];
  float cT;       // log2(e) / T in fp32 (T > 0)
  double cT64;    // the same value widened: the decision uses the constant the sweeps used
  double ln_alpha;
  unsigned seed_lo, seed_hi, off_lo, off_hi;
  const unsigned long long* off_dev;  // when set, the counter offset is read from device memory instead
  long long row_base;
  int* accept_count;
  int* out_tokens;
  unsigned* row_status;
  float* diag;
  float* dump_r;
  float* bonus_prob;
  // scratch owned by the context
  unsigned* work_counter;  // units are handed out from here; grows by num_units every run
  unsigned* exit_count;    // [2]: blocks of stage 0 / stage 2 that have left; the last one clears the counters
  int* row_arrivals;       // [B], zero between runs
  int* row_reject;         // [B]: earliest rejected position published so far; kNoReject between runs
  int4* unit_res;          // [B*P]: x = accept flag, y = status bits, z = candidate token, w = a token can be drawn
  int* job_count;          // units the drawing stages must process; cleared by the last block of stage 2
  int2* jobs;              // x = b * P + j of a unit that draws a token (y unused)
  UnitStats* ustats;       // [B*P]: merged statistics of sweep 1, read back by the later stages
  double* zpart;           // [B*P][parts][8]: stage 1's partial normalisers
  double* wtotg;           // [B*P][parts*16]: stage 2's mass of every warp run
  double* srung;           // [B][parts*16][kRecG]: running totals inside the runs of the row's drawing unit
                           // (one-sweep drawing stage: [B][nsteps], first channel sum of every step)
  int* part_arrivals;      // [B*P]: blocks of the unit that finished stage 2; zero between runs
  double* srungB;          // the one-sweep drawing stage: second channel of srung (null where that stage is not used)
  double* srungC;          // ... third and fourth channel (ensembles of three or four models; null otherwise)
  double* srungD;
};

// ------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void cp_async16(void* smem, const void* g) {
  unsigned sa = static_cast<unsigned>(__cvta_generic_to_shared(smem));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int DT>
struct Elem;
template <>
struct Elem<COS_DTYPE_F32> {
  static constexpr int E = 4;  // entries per 16-byte vector
  static constexpr int bytes = 4;
  static __device__ __forceinline__ void unpack(const uint4& r, float (&v)[4]) {
    v[0] = __uint_as_float(r.x);
    v[1] = __uint_as_float(r.y);
    v[2] = __uint_as_float(r.z);
    v[3] = __uint_as_float(r.w);
  }
  static __device__ __forceinline__ float load1(const void* row, long long x) {
    return __ldg(reinterpret_cast<const float*>(row) + x);
  }
  static __device__ __forceinline__ float pick(const uint4* vec, int k) {  // entry k of a vector in shared memory
    return reinterpret_cast<const float*>(vec)[k];
  }
};
template <>
struct Elem<COS_DTYPE_F16> {  // IEEE half: 8 entries per 16-byte vector, widened exactly
  static constexpr int E = 8;
  static constexpr int bytes = 2;
  static __device__ __forceinline__ void unpack(const uint4& r, float (&v)[8]) {
    const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[k]));
      v[2 * k] = f.x;
      v[2 * k + 1] = f.y;
    }
  }
  static __device__ __forceinline__ float load1(const void* row, long long x) {
    return __half2float(__ldg(reinterpret_cast<const __half*>(row) + x));
  }
  static __device__ __forceinline__ float pick(const uint4* vec, int k) {  // entry k of a vector in shared memory
    return __half2float(reinterpret_cast<const __half*>(vec)[k]);
  }
};
template <>
struct Elem<COS_DTYPE_BF16> {
  static constexpr int E = 8;
  static constexpr int bytes = 2;
  static __device__ __forceinline__ void unpack(const uint4& r, float (&v)[8]) {
    v[0] = __uint_as_float(r.x << 16);
    v[1] = __uint_as_float(r.x & 0xffff0000u);
    v[2] = __uint_as_float(r.y << 16);
    v[3] = __uint_as_float(r.y & 0xffff0000u);
    v[4] = __uint_as_float(r.z << 16);
    v[5] = __uint_as_float(r.z & 0xffff0000u);
    v[6] = __uint_as_float(r.w << 16);
    v[7] = __uint_as_float(r.w & 0xffff0000u);
  }
  static __device__ __forceinline__ float load1(const void* row, long long x) {
    unsigned short h = __ldg(reinterpret_cast<const unsigned short*>(row) + x);
    return __uint_as_float(static_cast<unsigned>(h) << 16);
  }
  static __device__ __forceinline__ float pick(const uint4* vec, int k) {  // entry k of a vector in shared memory
    return __uint_as_float(static_cast<unsigned>(reinterpret_cast<const unsigned short*>(vec)[k]) << 16);
  }
};

// One lane's chunk of a step: E consecutive entries starting at entry0.  Entries at or
// beyond V read as -inf (probability zero, never a maximum).
template <int DT>
__device__ __forceinline__ void load_chunk(const void* row, int entry0, int V, bool vec_ok,
                                           float (&v)[Elem<DT>::E]) {
  constexpr int E = Elem<DT>::E;
  if (vec_ok && entry0 + E <= V) {
    uint4 raw = ldg_stream16(reinterpret_cast<const char*>(row) + static_cast<long long>(entry0) * Elem<DT>::bytes);
    Elem<DT>::unpack(raw, v);
  } else {
#pragma unroll
    for (int k = 0; k < E; ++k) v[k] = (entry0 + k < V) ? Elem<DT>::load1(row, entry0 + k) : -INFINITY;
  }
}

// Philox4x32-10 (Salmon et al., SC'11): 10 rounds of two 32x32->64 multiplies and a
// Weyl key schedule.
__device__ __forceinline__ void philox4x32_10(unsigned c0, unsigned c1, unsigned c2, unsigned c3, unsigned k0,
                                              unsigned k1, unsigned (&out)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    unsigned hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    unsigned hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    unsigned n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0;
    c1 = lo1;
    c2 = n2;
    c3 = lo0;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

__device__ __forceinline__ double word_to_uniform(unsigned w) {
  return (2.0 * static_cast<double>(w >> 9) + 1.0) * 5.9604644775390625e-08;  // 2^-24
}

__device__ __forceinline__ double shfl_double(double x, int src) {
  int lo = __double2loint(x), hi = __double2hiint(x);
  lo = __shfl_sync(0xffffffffu, lo, src);
  hi = __shfl_sync(0xffffffffu, hi, src);
  return __hiloint2double(hi, lo);
}
__device__ __forceinline__ double shfl_up_double(double x, int d) {
  int lo = __double2loint(x), hi = __double2hiint(x);
  lo = __shfl_up_sync(0xffffffffu, lo, d);
  hi = __shfl_up_sync(0xffffffffu, hi, d);
  return __hiloint2double(hi, lo);
}

// ------------------------------------------------------------------------------------
// partial results exchanged lane -> warp -> block -> cluster
// ------------------------------------------------------------------------------------
struct SoftPart {  // sum over a set of tokens of 2^(arg - ref)
  double s;
  float ref;
  int pad;
};
struct ArgPart {  // running maximum with the lowest index among equals
  double val;
  int idx;
  int bad;  // a NaN or +inf was seen
};

__device__ __forceinline__ bool arg_better(double v, int i, double bv, int bi) {
  return (v > bv) || (v == bv && i < bi);
}

// lane accumulator of a softmax normaliser in the base-2 domain: s = sum 2^(v*c - ref)
// Two fp32 operations in one instruction (sm_100 has packed forms of fma, add and mul: each half is the IEEE
// operation of its scalar twin, so results do not change; what is saved is an issue slot).
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n.reg .b64 ra, rb, rc, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\nmov.b64 rc, {%6, %7};\n"
      "fma.rn.f32x2 rd, ra, rb, rc;\nmov.b64 {%0, %1}, rd;\n}\n"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void mul2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n.reg .b64 ra, rb, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\nmul.rn.f32x2 rd, ra, rb;\nmov.b64 {%0, %1}, rd;\n}\n"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n.reg .b64 ra, rb, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\nadd.rn.f32x2 rd, ra, rb;\nmov.b64 {%0, %1}, rd;\n}\n"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

struct LaneSoft {
  float ref, s;
  __device__ __forceinline__ void init() {
    ref = -INFINITY;
    s = 0.f;
  }
  // reference exponent moves up with the running maximum (never overflows)
  template <int E>
  __device__ __forceinline__ void add_online(const float (&v)[E], float c) {
    float vmax = v[0];
#pragma unroll
    for (int k = 1; k < E; ++k) vmax = fmaxf(vmax, v[k]);
    float cand = vmax * c;
    if (cand > ref) {
      s *= ex2_approx(ref - cand);
      ref = cand;
    }
    float nref = (ref == -INFINITY) ? 0.f : -ref;
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < E; ++k) acc += ex2_approx(fmaf(v[k], c, nref));
    s += acc;
  }
  __device__ __forceinline__ void add_online1(float x, float c) {
    float cand = x * c;
    if (cand > ref) {
      s *= ex2_approx(ref - cand);
      ref = cand;
    }
    float nref = (ref == -INFINITY) ? 0.f : -ref;
    s += ex2_approx(fmaf(x, c, nref));
  }
  // reference exponent fixed (set from the first chunk); the caller checks s for overflow
  template <int E>
  __device__ __forceinline__ void seed(const float (&v)[E], float c) {
    float vmax = v[0];
#pragma unroll
    for (int k = 1; k < E; ++k) vmax = fmaxf(vmax, v[k]);
    float cand = vmax * c;
    ref = (fabsf(cand) < INFINITY) ? floorf(cand) : 0.f;  // a whole number: sums with such references rescale exactly
    s = 0.f;
  }
  // the same with the packed forms of fma and add (same values, fewer instructions)
  template <int E>
  __device__ __forceinline__ void add_fixed2(const float (&v)[E], float c) {
    const float nref = -ref;
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int k = 0; k < E; k += 2) {
      float t0, t1;
      fma2(t0, t1, v[k], v[k + 1], c, c, nref, nref);
      add2(a0, a1, a0, a1, ex2_approx(t0), ex2_approx(t1));
    }
    s += a0 + a1;
  }
  template <int E>
  __device__ __forceinline__ void add_fixed(const float (&v)[E], float c) {
    const float nref = -ref;
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int k = 0; k < E; k += 2) {
      a0 += ex2_approx(fmaf(v[k], c, nref));
      a1 += ex2_approx(fmaf(v[k + 1], c, nref));
    }
    s += a0 + a1;
  }
};

// sum of (ref, s) pairs held one per lane: common reference = the largest, fp64 sum
__device__ __forceinline__ SoftPart warp_reduce_soft(float ref, double s) {
  float R = ref;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) R = fmaxf(R, __shfl_xor_sync(0xffffffffu, R, d));
  // references seeded by the sweep are whole numbers: the factor is then an exact power of two and cheap
  const float d = ref - R;
  double t;
  if (ref == R)
    t = s;
  else if (d == floorf(d) && d > -1000.f)
    t = s * __hiloint2double((1023 + static_cast<int>(d)) << 20, 0);
  else
    t = s * exp2(static_cast<double>(ref) - static_cast<double>(R));
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    int lo = __shfl_xor_sync(0xffffffffu, __double2loint(t), d);
    int hi = __shfl_xor_sync(0xffffffffu, __double2hiint(t), d);
    t += __hiloint2double(hi, lo);
  }
  SoftPart o;
  o.s = t;
  o.ref = R;
  o.pad = 0;
  return o;
}

__device__ __forceinline__ void warp_merge_soft(LaneSoft a, SoftPart* dst, int lane) {
  // lanes of one warp: fp32 is enough here, the errors of the 32 scale factors average out
  float R = a.ref;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) R = fmaxf(R, __shfl_xor_sync(0xffffffffu, R, d));
  float t = (a.ref == R) ? a.s : a.s * ex2_approx(a.ref - R);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) t += __shfl_xor_sync(0xffffffffu, t, d);
  if (lane == 0) {
    dst->s = static_cast<double>(t);
    dst->ref = R;
  }
}

__device__ __forceinline__ ArgPart warp_reduce_arg(double val, int idx, int bad, int lane) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    double ov = shfl_double(val, lane ^ d);
    int oi = __shfl_xor_sync(0xffffffffu, idx, d);
    bad |= __shfl_xor_sync(0xffffffffu, bad, d);
    if (arg_better(ov, oi, val, idx)) {
      val = ov;
      idx = oi;
    }
  }
  ArgPart o;
  o.val = val;
  o.idx = idx;
  o.bad = bad;
  return o;
}

__device__ __forceinline__ void warp_merge_arg(double val, int idx, int bad, ArgPart* dst, int lane) {
  ArgPart o = warp_reduce_arg(val, idx, bad, lane);
  if (lane == 0) *dst = o;
}

// The model whose distribution is q at position j of row b: the row's proposer, or the proposer of that draft
// when the caller gave one per position (Algorithm 2 verifies tokens of several proposers in one sequence).
// At the bonus position of a call that names a bonus model, q is that model's distribution: the token is
// then drawn from q (Sec. 3.3) by the machinery that otherwise draws from r.
__device__ __forceinline__ int proposer_of(const KParams& p, int b, int j) {
  if (j == p.gamma && p.bonus_model >= 0) return p.bonus_model;
  return p.proposer[p.per_pos ? b * p.P + j : b];
}

// Counter words 2 and 3 of the Philox call: from the arguments, or from device memory when the caller keeps
// the offset there (so that a captured graph can be replayed with fresh uniforms).
__device__ __forceinline__ unsigned offset_lo(const KParams& p) {
  return p.off_dev ? static_cast<unsigned>(__ldcg(p.off_dev)) : p.off_lo;
}
__device__ __forceinline__ unsigned offset_hi(const KParams& p) {
  return p.off_dev ? static_cast<unsigned>(__ldcg(p.off_dev) >> 32) : p.off_hi;
}

// ------------------------------------------------------------------------------------
// sweep 1: a block's slice of the vocabulary, threads interleaved over 16-byte vectors
// ------------------------------------------------------------------------------------
// Sweep 1 only forms sums, maxima and argmaxes, so any assignment of tokens to threads
// will do: each block reads its slice as consecutive 8 KB pieces (one vector per thread),
// which keeps the DRAM accesses of a block contiguous.
struct Slice {
  int v_lo, v_hi;  // whole 16-byte vectors [v_lo, v_hi) of the row (aligned layouts only)
  int e_lo, e_hi;  // single entries [e_lo, e_hi): the ragged tail, or everything when unaligned
};

template <int DT>
__device__ __forceinline__ Slice slice_of(int rank, int C, int V, bool vec_ok) {
  constexpr int E = Elem<DT>::E;
  Slice s;
  if (vec_ok) {
    const int nvec = V / E;
    s.v_lo = static_cast<int>(static_cast<long long>(rank) * nvec / C);
    s.v_hi = static_cast<int>(static_cast<long long>(rank + 1) * nvec / C);
    s.e_lo = (rank == C - 1) ? nvec * E : V;
    s.e_hi = V;
  } else {
    s.v_lo = s.v_hi = 0;
    s.e_lo = static_cast<int>(static_cast<long long>(rank) * V / C);
    s.e_hi = static_cast<int>(static_cast<long long>(rank + 1) * V / C);
  }
  return s;
}

// Softmax normaliser of one row over the slice: fixed reference exponent (seeded from the
// thread's first vector) with four loads in flight; overflow or a non-finite input falls
// back to the running-maximum form.
// U: 16-byte loads a thread issues before it consumes them
template <int DT, int NT, int U = 4>
__device__ __forceinline__ LaneSoft soft_slice(const void* row, const Slice& sl, int tid, float c) {
  constexpr int E = Elem<DT>::E;
  const char* rowb = reinterpret_cast<const char*>(row);
  LaneSoft acc;
  acc.init();
  int v = sl.v_lo + tid;
  if (v < sl.v_hi) {
    float x[E];
    uint4 raw[U];
    raw[0] = ldg_stream16(rowb + static_cast<long long>(v) * 16);
    Elem<DT>::unpack(raw[0], x);
    acc.seed(x, c);
    for (; v + (U - 1) * NT < sl.v_hi; v += U * NT) {
#pragma unroll
      for (int u = 0; u < U; ++u) raw[u] = ldg_stream16(rowb + static_cast<long long>(v + u * NT) * 16);
#pragma unroll
      for (int u = 0; u < U; ++u) {
        Elem<DT>::unpack(raw[u], x);
        acc.add_fixed2(x, c);
      }
    }
    for (; v < sl.v_hi; v += NT) {
      raw[0] = ldg_stream16(rowb + static_cast<long long>(v) * 16);
      Elem<DT>::unpack(raw[0], x);
      acc.add_fixed2(x, c);
    }
  }
  for (int e = sl.e_lo + tid; e < sl.e_hi; e += NT) acc.add_online1(Elem<DT>::load1(row, e), c);
  if (!(acc.s < INFINITY)) {
    acc.init();
    for (v = sl.v_lo + tid; v < sl.v_hi; v += NT) {
      float x[E];
      uint4 raw = ldg_stream16(rowb + static_cast<long long>(v) * 16);
      Elem<DT>::unpack(raw, x);
      acc.add_online(x, c);
    }
    for (int e = sl.e_lo + tid; e < sl.e_hi; e += NT) acc.add_online1(Elem<DT>::load1(row, e), c);
  }
  return acc;
}

// Softmax statistics of a logit-level combine over the slice `sl` of one (row, position): accq = the proposer's
// softmax, accc = the softmax of the combined logits sum_i w_i l_i (entries outside the plausibility mask count
// as -inf).  Fast form: fixed reference exponents seeded from the thread's first vector, one vector of every model
// per trip, the first two models fetched one trip ahead; overflow or a non-finite input falls back to the
// running-maximum form.  `tid` in [0, NT): the threads that share the slice.
template <int DT, int NT>
__device__ __forceinline__ void logit_soft_slice(const KParams& p, const char* base, const Slice& sl, int tid, int pis,
                                                 bool masked, float thr, LaneSoft& accq, LaneSoft& accc) {
  constexpr int E = Elem<DT>::E;
  auto row_of = [&](int i) -> const void* { return base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes; };
    const char* row0 = reinterpret_cast<const char*>(row_of(0));
    const long long row_step = p.s_model * Elem<DT>::bytes;
    // Fast form: fixed reference exponents seeded from the thread's first vector, one vector of every model
    // per trip, the first two models fetched one trip ahead (four loads in flight per thread).
    bool settled = false;
    {
      accq.init();
      accc.init();
      const bool pair = (p.n >= 2);
      uint4 nx0 = make_uint4(0u, 0u, 0u, 0u), nx1 = nx0;
      const int v0 = sl.v_lo + tid;
      if (v0 < sl.v_hi) {
        nx0 = ldg_stream16(row0 + static_cast<long long>(v0) * 16);
        if (pair) nx1 = ldg_stream16(row0 + row_step + static_cast<long long>(v0) * 16);
      }
      bool first = true;
      for (int v = v0; v < sl.v_hi; v += NT) {
        const uint4 a0 = nx0, a1 = nx1;
        {
          const int vn = v + NT;
          if (vn < sl.v_hi) {
            nx0 = ldg_stream16(row0 + static_cast<long long>(vn) * 16);
            if (pair) nx1 = ldg_stream16(row0 + row_step + static_cast<long long>(vn) * 16);
          }
        }
        float cmb[E], xq[E];
        unsigned inbits = 0xffffffffu;
#pragma unroll
        for (int k = 0; k < E; ++k) cmb[k] = 0.f;
        auto take = [&](int i, const uint4& raw) {
          float x[E];
          Elem<DT>::unpack(raw, x);
          const float wi = p.w[i];
#pragma unroll
          for (int k = 0; k < E; k += 2) fma2(cmb[k], cmb[k + 1], wi, wi, x[k], x[k + 1], cmb[k], cmb[k + 1]);
          if (i == pis) {
#pragma unroll
            for (int k = 0; k < E; ++k) xq[k] = x[k];
          }
          if (masked && i == p.mask_model) {
            inbits = 0u;
#pragma unroll
            for (int k = 0; k < E; ++k) inbits |= (x[k] >= thr) ? (1u << k) : 0u;
          }
        };
        take(0, a0);
        if (pair) take(1, a1);
        for (int i = 2; i < p.n; ++i) take(i, ldg_stream16(row0 + i * row_step + static_cast<long long>(v) * 16));
        if (masked) {
#pragma unroll
          for (int k = 0; k < E; ++k) cmb[k] = (inbits & (1u << k)) ? cmb[k] : -INFINITY;
        }
        if (first) {
          accq.seed(xq, p.cT);
          accc.seed(cmb, p.cT);
          first = false;
        }
        accq.add_fixed2(xq, p.cT);
        accc.add_fixed2(cmb, p.cT);
      }
      for (int e = sl.e_lo + tid; e < sl.e_hi; e += NT) {
        float cmb = 0.f, xq = -INFINITY, xe = 0.f;
        for (int i = 0; i < p.n; ++i) {
          float x = Elem<DT>::load1(row_of(i), e);
          cmb = fmaf(p.w[i], x, cmb);
          if (i == pis) xq = x;
          if (i == p.mask_model) xe = x;
        }
        if (masked && !(xe >= thr)) cmb = -INFINITY;
        accq.add_online1(xq, p.cT);
        accc.add_online1(cmb, p.cT);
      }
      settled = (accq.s < INFINITY) && (accc.s < INFINITY);
    }
    // overflow or a non-finite input: the running-maximum form (two vectors of two models per trip)
    for (int pass = 1; pass < 2 && !settled; ++pass) {
      const bool fixed = (pass == 0);
      accq.init();
      accc.init();
      bool seeded_q = false, seeded_c = false;
      // one model's vector: add to the combined logits; the proposer's row also feeds its own softmax,
      // the expert's row yields the mask bits
      auto take = [&](int i, const uint4& raw, float (&cmb)[E], unsigned& inbits) {
        float x[E];
        Elem<DT>::unpack(raw, x);
        const float wi = p.w[i];
#pragma unroll
        for (int k = 0; k < E; ++k) cmb[k] = fmaf(wi, x[k], cmb[k]);
        if (i == pis) {
          if (fixed) {
            if (!seeded_q) {
              accq.seed(x, p.cT);
              seeded_q = true;
            }
            accq.add_fixed(x, p.cT);
          } else {
            accq.add_online(x, p.cT);
          }
        }
        if (masked && i == p.mask_model) {
          inbits = 0u;
#pragma unroll
          for (int k = 0; k < E; ++k) inbits |= (x[k] >= thr) ? (1u << k) : 0u;
        }
      };
      auto finish = [&](float (&cmb)[E], unsigned inbits) {
        if (masked) {
#pragma unroll
          for (int k = 0; k < E; ++k) cmb[k] = (inbits & (1u << k)) ? cmb[k] : -INFINITY;
        }
        if (fixed) {
          if (!seeded_c) {
            accc.seed(cmb, p.cT);
            seeded_c = true;
          }
          accc.add_fixed(cmb, p.cT);
        } else {
          accc.add_online(cmb, p.cT);
        }
      };
      for (int v = sl.v_lo + tid; v < sl.v_hi; v += 2 * NT) {
        const bool have_b = (v + NT < sl.v_hi);
        const long long oa = static_cast<long long>(v) * 16;
        const long long ob = have_b ? oa + static_cast<long long>(NT) * 16 : oa;
        float ca[E], cb[E];
        unsigned ba = 0xffffffffu, bb = 0xffffffffu;
#pragma unroll
        for (int k = 0; k < E; ++k) ca[k] = cb[k] = 0.f;
        int i = 0;
        for (; i + 1 < p.n; i += 2) {  // two models, two vectors: four loads in flight
          const char* r0 = row0 + i * row_step;
          const char* r1 = r0 + row_step;
          const uint4 a0 = ldg_stream16(r0 + oa), b0 = ldg_stream16(r0 + ob);
          const uint4 a1 = ldg_stream16(r1 + oa), b1 = ldg_stream16(r1 + ob);
          take(i, a0, ca, ba);
          take(i + 1, a1, ca, ba);
          if (have_b) {
            take(i, b0, cb, bb);
            take(i + 1, b1, cb, bb);
          }
        }
        if (i < p.n) {
          const char* r0 = row0 + i * row_step;
          const uint4 a0 = ldg_stream16(r0 + oa), b0 = ldg_stream16(r0 + ob);
          take(i, a0, ca, ba);
          if (have_b) take(i, b0, cb, bb);
        }
        finish(ca, ba);
        if (have_b) finish(cb, bb);
      }
      for (int e = sl.e_lo + tid; e < sl.e_hi; e += NT) {
        float cmb = 0.f, xq = -INFINITY, xe = 0.f;
        for (int i = 0; i < p.n; ++i) {
          float x = Elem<DT>::load1(row_of(i), e);
          cmb = fmaf(p.w[i], x, cmb);
          if (i == pis) xq = x;
          if (i == p.mask_model) xe = x;
        }
        if (masked && !(xe >= thr)) cmb = -INFINITY;
        accq.add_online1(xq, p.cT);
        accc.add_online1(cmb, p.cT);
      }
      if ((accq.s < INFINITY) && (accc.s < INFINITY)) break;
    }
}

}  // namespace cosv

#endif  // COS_COMMON_CUH
