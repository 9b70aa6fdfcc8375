// CoS verification step for sm_100a: fused combine + accept test + residual / bonus sample
// + first-rejection scan, one persistent kernel of thread-block clusters.
//
// Work unit = one (row b, position j).  A cluster of C thread blocks owns a unit; every
// warp of the cluster owns a contiguous run of the vocabulary, so prefix order equals
// token order.  Per unit:
//   sweep 1  stream the n logit rows once from HBM (128-bit loads), keep per-lane online
//            softmax statistics (reference exponent, sum of 2^(l*c - ref)) or argmaxes,
//            merge lane -> warp -> block -> cluster (the last two in fp64, across blocks
//            through distributed shared memory);
//   decide   the accept test of Eq. 6 in fp64 from the merged statistics and the logits at
//            the draft token; rank 0 records the row's earliest known rejection;
//   sweep 2  only where a token must be drawn (first rejected position of a row, or the
//            bonus position when nothing earlier was rejected): re-read the unit (it is
//            still in L2), form r and q per token, residual max(0, r - q), warp-ordered
//            fp64 prefix sums, locate u * S, rescan one warp's run for the token;
//   publish  per-unit result, and the last unit of a row to arrive runs the
//            first-rejection scan and writes the row's outputs.
// Nothing in the kernel spins on memory: blocks meet only at hardware cluster barriers.

#include <cooperative_groups.h>
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

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxSlots = COS_MAX_MODELS + 2;
constexpr int kMaxCluster = 16;
constexpr int kNoReject = 0x7fffffff;

enum Mode { kEnsembleSample = 0, kLogitSample = 1, kEnsembleGreedy = 2, kLogitGreedy = 3 };

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
  float w[COS_MAX_MODELS];
  double w64[COS_MAX_MODELS];
  float cT;       // log2(e) / T in fp32 (T > 0)
  double cT64;    // the same value widened: the decision uses the constant the sweeps used
  double ln_alpha;
  unsigned seed_lo, seed_hi, off_lo, off_hi;
  long long row_base;
  int* accept_count;
  int* out_tokens;
  unsigned* row_status;
  float* diag;
  float* dump_r;
  // scratch owned by the context
  unsigned* work_counter;  // monotonically increasing across runs
  unsigned work_base;      // its value when this run starts
  int* row_arrivals;       // [B], zero between runs
  int* first_rej;          // [B], kNoReject between runs
  int4* unit_res;          // [B*P]: x = accept flag, y = status bits, z = candidate token
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
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
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

struct Xchg {  // one per block and barrier parity; peers read it through DSMEM
  SoftPart soft[kMaxSlots];
  ArgPart arg[kMaxSlots];
  double cta_total;
  int bcast[4];
};

struct Decision {  // written by thread 0 of every block, identically
  int accept, status, want_sample, cand;
  int natoms;
  int atom_tok[COS_MAX_MODELS];
  double atom_mass[COS_MAX_MODELS];
  double ratio, r_d, q_d, S, u_smp;
};

struct Shared {
  Xchg x[2];
  SoftPart wsoft[kWarps][kMaxSlots];
  ArgPart warg[kWarps][kMaxSlots];
  double wtot[kWarps];       // this block's per-warp totals of sweep 2
  double wincl[kWarps];      // their running sum
  SoftPart fsoft[kMaxSlots]; // merged over the cluster
  ArgPart farg[kMaxSlots];
  float a_scale[COS_MAX_MODELS];  // w_i / Z_i (ensemble) for sweep 2
  float a_ref[COS_MAX_MODELS];
  Decision dec;
  double target, base;  // sweep-2 search: u*S and the mass before the winning warp
  int win_rank, win_warp;
  int need2, next_unit;
  float thr32;  // plausibility threshold rounded up to fp32
  float ldraft[COS_MAX_MODELS];  // the n logits at the draft token, fetched before sweep 1
};

// lane accumulator of the online softmax in the base-2 domain
struct LaneSoft {
  float ref, s;
  __device__ __forceinline__ void init() {
    ref = -INFINITY;
    s = 0.f;
  }
  template <int E>
  __device__ __forceinline__ void add(const float (&v)[E], float c) {
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
};

__device__ __forceinline__ void warp_merge_soft(LaneSoft a, SoftPart* dst, int lane) {
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

__device__ __forceinline__ void warp_merge_arg(double val, int idx, int bad, ArgPart* dst, int lane) {
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
  if (lane == 0) {
    dst->val = val;
    dst->idx = idx;
    dst->bad = bad;
  }
}

__device__ __forceinline__ SoftPart merge_soft_list(const SoftPart* parts, int count, int stride_bytes) {
  float R = -INFINITY;
  for (int k = 0; k < count; ++k) {
    const SoftPart* p = reinterpret_cast<const SoftPart*>(reinterpret_cast<const char*>(parts) + k * stride_bytes);
    R = fmaxf(R, p->ref);
  }
  double Z = 0.0;
  for (int k = 0; k < count; ++k) {
    const SoftPart* p = reinterpret_cast<const SoftPart*>(reinterpret_cast<const char*>(parts) + k * stride_bytes);
    float ref = p->ref;
    double s = p->s;
    Z += (ref == R) ? s : s * exp2(static_cast<double>(ref) - static_cast<double>(R));
  }
  SoftPart o;
  o.s = Z;
  o.ref = R;
  o.pad = 0;
  return o;
}

// Block merge of warp partials, publish for the peers, cluster barrier, merge over ranks.
// All threads of all blocks of the cluster call this; results land in sh.fsoft / sh.farg.
__device__ void cluster_merge(Shared& sh, cg::cluster_group& cluster, int& phase, int nsoft, const int* soft_slots,
                              int narg, const int* arg_slots) {
  const int tid = threadIdx.x;
  const int C = cluster.num_blocks();
  __syncthreads();
  Xchg& mine = sh.x[phase & 1];
  if (tid < nsoft) {
    int slot = soft_slots[tid];
    mine.soft[slot] = merge_soft_list(&sh.wsoft[0][slot], kWarps, sizeof(SoftPart) * kMaxSlots);
  } else if (tid >= 32 && tid < 32 + narg) {
    int slot = arg_slots[tid - 32];
    ArgPart best = sh.warg[0][slot];
    for (int w = 1; w < kWarps; ++w) {
      ArgPart o = sh.warg[w][slot];
      best.bad |= o.bad;
      if (arg_better(o.val, o.idx, best.val, best.idx)) {
        best.val = o.val;
        best.idx = o.idx;
      }
    }
    mine.arg[slot] = best;
  }
  cluster.sync();
  if (tid < nsoft) {
    int slot = soft_slots[tid];
    SoftPart tmp[kMaxCluster];
    for (int r = 0; r < C; ++r) tmp[r] = cluster.map_shared_rank(&sh.x[phase & 1], r)->soft[slot];
    sh.fsoft[slot] = merge_soft_list(tmp, C, sizeof(SoftPart));
  } else if (tid >= 32 && tid < 32 + narg) {
    int slot = arg_slots[tid - 32];
    ArgPart best = cluster.map_shared_rank(&sh.x[phase & 1], 0)->arg[slot];
    for (int r = 1; r < C; ++r) {
      ArgPart o = cluster.map_shared_rank(&sh.x[phase & 1], r)->arg[slot];
      best.bad |= o.bad;
      if (arg_better(o.val, o.idx, best.val, best.idx)) {
        best.val = o.val;
        best.idx = o.idx;
      }
    }
    sh.farg[slot] = best;
  }
  __syncthreads();
  ++phase;
}

// ------------------------------------------------------------------------------------
// publishing a unit and the per-row first-rejection scan (Sec. 3.1)
// ------------------------------------------------------------------------------------
__device__ void publish_unit(const KParams& p, int b, int j, int accept, int status, int cand, double ratio,
                             double r_d, double q_d, double S) {
  if (p.diag) {
    float* d = p.diag + (static_cast<long long>(b) * p.P + j) * 4;
    d[0] = static_cast<float>(ratio);
    d[1] = static_cast<float>(r_d);
    d[2] = static_cast<float>(q_d);
    d[3] = static_cast<float>(S);
  }
  int4 res = make_int4(accept, status, cand, 0);
  __stcg(&p.unit_res[b * p.P + j], res);
  __threadfence();
  int prev = atomicAdd(&p.row_arrivals[b], 1);
  if (prev != p.P - 1) return;
  // last unit of the row: every other unit's result is visible after the fence below
  __threadfence();
  int a = p.gamma;
  unsigned st = 0;
  int tok = -1;
  for (int k = 0; k < p.P; ++k) {
    int4 u = __ldcg(&p.unit_res[b * p.P + k]);
    st |= static_cast<unsigned>(u.y);
    if (k == p.gamma || !u.x) {
      a = k;
      tok = u.z;
      break;
    }
  }
  p.accept_count[b] = a;
  int* o = p.out_tokens + static_cast<long long>(b) * p.P;
  for (int k = 0; k < p.P; ++k) o[k] = (k < a) ? p.drafts[b * p.gamma + k] : (k == a ? tok : -1);
  p.row_status[b] = st;
  p.row_arrivals[b] = 0;  // leave the scratch ready for the next run
  p.first_rej[b] = kNoReject;
}

// ------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------
template <int DT, int MODE>
__global__ void __launch_bounds__(kThreads, 2) cos_verify_kernel(const __grid_constant__ KParams p) {
  constexpr int E = Elem<DT>::E;
  constexpr bool kSample = (MODE == kEnsembleSample || MODE == kLogitSample);
  cg::cluster_group cluster = cg::this_cluster();
  const int C = cluster.num_blocks();
  const int rank = cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gwarp = rank * kWarps + warp, G = C * kWarps;
  __shared__ Shared sh;
  __shared__ int slot_ids[2][kMaxSlots];
  int phase = 0;
  const bool vec_ok = p.vec_ok != 0;
  const bool masked = (MODE == kLogitSample || MODE == kLogitGreedy) && p.mask_model >= 0;

  // this warp's run of steps (a step = 32 lanes x E entries)
  const int s_begin = static_cast<int>(static_cast<long long>(gwarp) * p.nsteps / G);
  const int s_end = static_cast<int>(static_cast<long long>(gwarp + 1) * p.nsteps / G);

  int unit = blockIdx.x / C;
  while (unit < p.num_units) {
    const int j = unit / p.B, b = unit % p.B;  // earlier positions of every row come first
    const int pi = p.proposer[b];
    const bool pi_ok = (pi >= 0 && pi < p.n);
    const int pis = pi_ok ? pi : 0;
    const char* base = reinterpret_cast<const char*>(p.logits) +
                       (static_cast<long long>(b) * p.s_row + static_cast<long long>(j) * p.s_pos) * Elem<DT>::bytes;
    auto row_of = [&](int i) -> const void* { return base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes; };
    const bool is_bonus = (j == p.gamma);
    const int draft = is_bonus ? 0 : p.drafts[b * p.gamma + j];
    if (tid < p.n && !is_bonus && draft >= 0 && draft < p.V) sh.ldraft[tid] = Elem<DT>::load1(row_of(tid), draft);

    // ================================ sweep 1: statistics ================================
    if (MODE == kEnsembleSample) {
      for (int i = 0; i < p.n; ++i) {
        const void* row = row_of(i);
        LaneSoft acc;
        acc.init();
        int s = s_begin;
        for (; s + 2 <= s_end; s += 2) {
          float v0[E], v1[E];
          load_chunk<DT>(row, (s * 32 + lane) * E, p.V, vec_ok, v0);
          load_chunk<DT>(row, ((s + 1) * 32 + lane) * E, p.V, vec_ok, v1);
          acc.add(v0, p.cT);
          acc.add(v1, p.cT);
        }
        for (; s < s_end; ++s) {
          float v0[E];
          load_chunk<DT>(row, (s * 32 + lane) * E, p.V, vec_ok, v0);
          acc.add(v0, p.cT);
        }
        warp_merge_soft(acc, &sh.wsoft[warp][i], lane);
      }
      if (tid < p.n) slot_ids[0][tid] = tid;
      cluster_merge(sh, cluster, phase, p.n, slot_ids[0], 0, slot_ids[1]);
    } else if (MODE == kEnsembleGreedy) {
      for (int i = 0; i < p.n; ++i) {
        const void* row = row_of(i);
        float best = -INFINITY;
        int bidx = kNoReject, bad = 0;
        for (int s = s_begin; s < s_end; ++s) {
          float v[E];
          const int e0 = (s * 32 + lane) * E;
          load_chunk<DT>(row, e0, p.V, vec_ok, v);
#pragma unroll
          for (int k = 0; k < E; ++k) {
            if (e0 + k < p.V) {
              bad |= !(v[k] < INFINITY);
              if (v[k] > best) {
                best = v[k];
                bidx = e0 + k;
              }
            }
          }
        }
        warp_merge_arg(static_cast<double>(best), bidx, bad, &sh.warg[warp][i], lane);
      }
      if (tid < p.n) slot_ids[1][tid] = tid;
      cluster_merge(sh, cluster, phase, 0, slot_ids[0], p.n, slot_ids[1]);
    } else {
      // logit-level combine.  soft slot 0 = proposer, soft slot 1 = combined logits;
      // arg slot 0 = expert maximum (mask), arg slot 1 = proposer argmax, arg slot 2 = combined argmax.
      if (masked) {
        const void* row = row_of(p.mask_model);
        float best = -INFINITY;
        int bad = 0;
        for (int s = s_begin; s < s_end; ++s) {
          float v[E];
          const int e0 = (s * 32 + lane) * E;
          load_chunk<DT>(row, e0, p.V, vec_ok, v);
#pragma unroll
          for (int k = 0; k < E; ++k) {
            if (e0 + k < p.V) {
              bad |= (v[k] != v[k]);
              best = fmaxf(best, v[k]);
            }
          }
        }
        warp_merge_arg(static_cast<double>(best), 0, bad, &sh.warg[warp][0], lane);
        if (tid == 0) slot_ids[1][0] = 0;
        cluster_merge(sh, cluster, phase, 0, slot_ids[0], 1, slot_ids[1]);
        if (tid == 0) {
          // l >= max + ln(alpha) in fp64 is the same as l >= (that bound rounded up to fp32) for fp32 l
          double bound = sh.farg[0].val + p.ln_alpha;
          sh.thr32 = sh.farg[0].bad ? __int_as_float(0x7fc00000) : __double2float_ru(bound);
        }
        __syncthreads();
      }
      const float thr = masked ? sh.thr32 : -INFINITY;
      if (MODE == kLogitSample) {
        LaneSoft accq, accc;
        accq.init();
        accc.init();
        for (int s = s_begin; s < s_end; ++s) {
          const int e0 = (s * 32 + lane) * E;
          float cmb[E], vq[E], ve[E];
#pragma unroll
          for (int k = 0; k < E; ++k) {
            cmb[k] = 0.f;
            vq[k] = -INFINITY;
            ve[k] = 0.f;
          }
          for (int i = 0; i < p.n; i += 2) {
            float va[E], vb[E];
            const bool two = (i + 1 < p.n);
            load_chunk<DT>(row_of(i), e0, p.V, vec_ok, va);
            if (two) load_chunk<DT>(row_of(i + 1), e0, p.V, vec_ok, vb);
            const float wa = p.w[i], wb = two ? p.w[i + 1] : 0.f;
#pragma unroll
            for (int k = 0; k < E; ++k) {
              cmb[k] = fmaf(wa, va[k], cmb[k]);
              if (i == pis) vq[k] = va[k];
              if (i == p.mask_model) ve[k] = va[k];
              if (two) {
                cmb[k] = fmaf(wb, vb[k], cmb[k]);
                if (i + 1 == pis) vq[k] = vb[k];
                if (i + 1 == p.mask_model) ve[k] = vb[k];
              }
            }
          }
#pragma unroll
          for (int k = 0; k < E; ++k) {
            bool in = (e0 + k < p.V) && (!masked || ve[k] >= thr);
            cmb[k] = in ? cmb[k] : -INFINITY;
          }
          accq.add(vq, p.cT);
          accc.add(cmb, p.cT);
        }
        warp_merge_soft(accq, &sh.wsoft[warp][0], lane);
        warp_merge_soft(accc, &sh.wsoft[warp][1], lane);
        if (tid < 2) slot_ids[0][tid] = tid;
        cluster_merge(sh, cluster, phase, 2, slot_ids[0], 0, slot_ids[1]);
      } else {  // kLogitGreedy: combined logits in fp64, the same chain of fused multiply-adds on every token
        double cbest = -INFINITY;
        int cidx = kNoReject, bad = 0;
        float qbest = -INFINITY;
        int qidx = kNoReject;
        for (int s = s_begin; s < s_end; ++s) {
          const int e0 = (s * 32 + lane) * E;
          double cmb[E];
          float ve[E];
#pragma unroll
          for (int k = 0; k < E; ++k) {
            cmb[k] = 0.0;
            ve[k] = 0.f;
          }
          for (int i = 0; i < p.n; ++i) {
            float va[E];
            load_chunk<DT>(row_of(i), e0, p.V, vec_ok, va);
            const double wa = p.w64[i];
#pragma unroll
            for (int k = 0; k < E; ++k) {
              if (e0 + k < p.V) {
                bad |= !(va[k] < INFINITY);
                cmb[k] = fma(wa, static_cast<double>(va[k]), cmb[k]);
                if (i == p.mask_model) ve[k] = va[k];
                if (i == pis && va[k] > qbest) {
                  qbest = va[k];
                  qidx = e0 + k;
                }
              }
            }
          }
#pragma unroll
          for (int k = 0; k < E; ++k) {
            if (e0 + k < p.V && (!masked || ve[k] >= thr)) {
              bad |= (cmb[k] != cmb[k]);
              if (cmb[k] > cbest) {
                cbest = cmb[k];
                cidx = e0 + k;
              }
            }
          }
        }
        warp_merge_arg(static_cast<double>(qbest), qidx, bad, &sh.warg[warp][1], lane);
        warp_merge_arg(cbest, cidx, bad, &sh.warg[warp][2], lane);
        if (tid < 2) slot_ids[1][tid] = tid + 1;
        cluster_merge(sh, cluster, phase, 0, slot_ids[0], 2, slot_ids[1]);
      }
    }

    // ================================ decision (Eq. 6) ================================
    if (tid == 0) {
      Decision& d = sh.dec;
      unsigned rnd[4];
      const unsigned long long grow = static_cast<unsigned long long>(p.row_base + b);
      philox4x32_10(static_cast<unsigned>(grow), static_cast<unsigned>(j), p.off_lo, p.off_hi, p.seed_lo, p.seed_hi, rnd);
      const double u_acc = word_to_uniform(rnd[0]);
      d.u_smp = word_to_uniform(rnd[1]);
      d.accept = 0;
      d.status = 0;
      d.want_sample = 0;
      d.cand = -1;
      d.natoms = 0;
      d.ratio = d.r_d = d.q_d = d.S = __longlong_as_double(0x7ff8000000000000LL);
      const bool draft_ok = is_bonus || (draft >= 0 && draft < p.V);
      bool finite = pi_ok;
      if (kSample) {
        const int nsoft = (MODE == kEnsembleSample) ? p.n : 2;
        for (int k = 0; k < nsoft; ++k) {
          const SoftPart& f = sh.fsoft[k];
          finite = finite && isfinite(f.ref) && isfinite(f.s) && (f.s > 0.0);
        }
        if (masked && sh.farg[0].bad) finite = false;
        if (!finite) {
          d.status |= COS_ROW_NONFINITE;
        } else {
          if (MODE == kEnsembleSample) {
            for (int i = 0; i < p.n; ++i) {
              sh.a_scale[i] = static_cast<float>(p.w64[i] / sh.fsoft[i].s);
              sh.a_ref[i] = -sh.fsoft[i].ref;
            }
          }
          if (!is_bonus) {
            if (draft_ok) {
              double r_d = 0.0, q_d = 0.0;
              if (MODE == kEnsembleSample) {
                for (int i = 0; i < p.n; ++i) {
                  double l = static_cast<double>(sh.ldraft[i]);
                  double pr = exp2(l * p.cT64 - static_cast<double>(sh.fsoft[i].ref)) / sh.fsoft[i].s;
                  r_d += p.w64[i] * pr;
                  if (i == pi) q_d = pr;
                }
              } else {
                double cd = 0.0;
                for (int i = 0; i < p.n; ++i)
                  cd = fma(p.w64[i], static_cast<double>(sh.ldraft[i]), cd);
                bool in = !masked || (sh.ldraft[p.mask_model] >= sh.thr32);
                r_d = in ? exp2(cd * p.cT64 - static_cast<double>(sh.fsoft[1].ref)) / sh.fsoft[1].s : 0.0;
                double lq = static_cast<double>(sh.ldraft[pi]);
                q_d = exp2(lq * p.cT64 - static_cast<double>(sh.fsoft[0].ref)) / sh.fsoft[0].s;
              }
              d.r_d = r_d;
              d.q_d = q_d;
              if (q_d > 0.0) {
                d.ratio = r_d / q_d;
              } else {
                d.status |= COS_ROW_Q_ZERO;
                d.ratio = (r_d > 0.0) ? __longlong_as_double(0x7ff0000000000000LL) : 0.0;
              }
              d.accept = (u_acc <= fmin(1.0, d.ratio)) ? 1 : 0;
            } else {
              d.status |= COS_ROW_BAD_DRAFT;
            }
          }
          d.want_sample = is_bonus || !d.accept;
        }
      } else {
        // greedy: distributions are atoms at lowest-index argmaxes
        int qtok;
        if (MODE == kEnsembleGreedy) {
          for (int i = 0; i < p.n; ++i) finite = finite && !sh.farg[i].bad && isfinite(sh.farg[i].val);
          qtok = sh.farg[pis].idx;
        } else {
          finite = finite && !sh.farg[1].bad && !sh.farg[2].bad && isfinite(sh.farg[1].val) && isfinite(sh.farg[2].val);
          if (masked && sh.farg[0].bad) finite = false;
          qtok = sh.farg[1].idx;
        }
        if (!finite) {
          d.status |= COS_ROW_NONFINITE;
        } else {
          // atoms of r, sorted by token, masses accumulated in model order
          if (MODE == kEnsembleGreedy) {
            for (int i = 0; i < p.n; ++i) {
              int t = sh.farg[i].idx, pos = 0;
              while (pos < d.natoms && d.atom_tok[pos] < t) ++pos;
              if (pos < d.natoms && d.atom_tok[pos] == t) {
                d.atom_mass[pos] += p.w64[i];
              } else {
                for (int k = d.natoms; k > pos; --k) {
                  d.atom_tok[k] = d.atom_tok[k - 1];
                  d.atom_mass[k] = d.atom_mass[k - 1];
                }
                d.atom_tok[pos] = t;
                d.atom_mass[pos] = 0.0 + p.w64[i];
                ++d.natoms;
              }
            }
          } else {
            d.natoms = 1;
            d.atom_tok[0] = sh.farg[2].idx;
            d.atom_mass[0] = 1.0;
          }
          auto r_at = [&](int t) {
            for (int k = 0; k < d.natoms; ++k)
              if (d.atom_tok[k] == t) return d.atom_mass[k];
            return 0.0;
          };
          bool use_r = is_bonus;
          if (!is_bonus) {
            if (draft_ok) {
              d.r_d = r_at(draft);
              d.q_d = (draft == qtok) ? 1.0 : 0.0;
              if (d.q_d > 0.0) {
                d.ratio = d.r_d / d.q_d;
              } else {
                d.status |= COS_ROW_Q_ZERO;
                d.ratio = (d.r_d > 0.0) ? __longlong_as_double(0x7ff0000000000000LL) : 0.0;
              }
              d.accept = (u_acc <= fmin(1.0, d.ratio)) ? 1 : 0;
            } else {
              d.status |= COS_ROW_BAD_DRAFT;
            }
            // residual max(0, r - q) over the atoms, summed in token order
            double S = 0.0;
            for (int k = 0; k < d.natoms; ++k) S += fmax(0.0, d.atom_mass[k] - (d.atom_tok[k] == qtok ? 1.0 : 0.0));
            d.S = S;
            if (!(S > 0.0)) {
              use_r = true;
              if (!d.accept) d.status |= COS_ROW_RESIDUAL_EMPTY;
            }
          }
          // inverse CDF over the atoms (token order): smallest k with running sum >= u * total
          double total = 0.0;
          for (int k = 0; k < d.natoms; ++k)
            total += use_r ? d.atom_mass[k] : fmax(0.0, d.atom_mass[k] - (d.atom_tok[k] == qtok ? 1.0 : 0.0));
          const double target = d.u_smp * total;
          double run = 0.0;
          int lastpos = -1;
          d.cand = -1;
          for (int k = 0; k < d.natoms; ++k) {
            double m = use_r ? d.atom_mass[k] : fmax(0.0, d.atom_mass[k] - (d.atom_tok[k] == qtok ? 1.0 : 0.0));
            run += m;
            if (m > 0.0) lastpos = d.atom_tok[k];
            if (d.cand < 0 && m > 0.0 && run >= target) d.cand = d.atom_tok[k];
          }
          if (d.cand < 0) d.cand = lastpos;
        }
      }
      // rank 0 alone talks to global memory about the row and fetches the next unit
      if (rank == 0) {
        int known = kNoReject;
        if (!is_bonus && !d.accept)
          known = atomicMin(&p.first_rej[b], j);
        else
          known = atomicMin(&p.first_rej[b], kNoReject);
        const bool superseded = known < j;  // an earlier position of this row already rejected
        int need2 = 0;
        if (kSample && finite) {
          need2 = (d.want_sample && !superseded) || (p.dump_r != nullptr) ||
                  ((p.flags & COS_RUN_ALL_RESIDUALS) && !is_bonus);
        }
        unsigned t = atomicAdd(p.work_counter, 1u);
        int next = p.num_clusters + static_cast<int>(t - p.work_base);
        Xchg& mine = sh.x[phase & 1];
        mine.bcast[0] = need2;
        mine.bcast[1] = next;
      }
    }
    cluster.sync();
    if (tid == 0) {
      const Xchg* r0 = cluster.map_shared_rank(&sh.x[phase & 1], 0);
      sh.need2 = r0->bcast[0];
      sh.next_unit = r0->bcast[1];
    }
    __syncthreads();
    ++phase;
    const int need2 = sh.need2;
    const int next_unit = sh.next_unit;

    // greedy test hook: r is a handful of atoms
    if (!kSample && p.dump_r != nullptr) {
      float* out = p.dump_r + (static_cast<long long>(b) * p.P + j) * p.V;
      const bool nonfinite = (sh.dec.status & COS_ROW_NONFINITE) != 0;
      for (int x = rank * kThreads + tid; x < p.V; x += C * kThreads) {
        float val = nonfinite ? __int_as_float(0x7fc00000) : 0.f;
        for (int k = 0; k < sh.dec.natoms; ++k)
          if (sh.dec.atom_tok[k] == x) val = static_cast<float>(sh.dec.atom_mass[k]);
        out[x] = val;
      }
    }

    // ================================ sweep 2: draw a token ================================
    bool published = false;
    if (kSample && need2) {
      bool from_r = is_bonus;  // the bonus is drawn from r itself; a rejected draft from max(0, r - q)
      const float inv_zq = (MODE == kEnsembleSample) ? static_cast<float>(1.0 / sh.fsoft[pis].s)
                                                     : static_cast<float>(1.0 / sh.fsoft[0].s);
      const float ref_q = (MODE == kEnsembleSample) ? -sh.fsoft[pis].ref : -sh.fsoft[0].ref;
      const float inv_zc = (MODE == kLogitSample) ? static_cast<float>(1.0 / sh.fsoft[1].s) : 0.f;
      const float ref_c = (MODE == kLogitSample) ? -sh.fsoft[1].ref : 0.f;
      const float thr = masked ? sh.thr32 : -INFINITY;
      double S_report = __longlong_as_double(0x7ff8000000000000LL);

      // mass of one lane chunk: fills res[] and returns nothing else; used by both the totals and the rescan
      auto chunk_mass = [&](int e0, bool use_r, bool dump, float (&res)[E]) {
        float r[E], q[E];
        if (MODE == kEnsembleSample) {
#pragma unroll
          for (int k = 0; k < E; ++k) {
            r[k] = 0.f;
            q[k] = 0.f;
          }
          for (int i = 0; i < p.n; ++i) {
            float v[E];
            load_chunk<DT>(row_of(i), e0, p.V, vec_ok, v);
            const float sc = sh.a_scale[i], rf = sh.a_ref[i];
#pragma unroll
            for (int k = 0; k < E; ++k) {
              float e = ex2_approx(fmaf(v[k], p.cT, rf));
              r[k] = fmaf(sc, e, r[k]);
              if (i == pis) q[k] = e * inv_zq;
            }
          }
        } else {
          float cmb[E], ve[E];
#pragma unroll
          for (int k = 0; k < E; ++k) {
            cmb[k] = 0.f;
            ve[k] = 0.f;
            q[k] = 0.f;
          }
          for (int i = 0; i < p.n; ++i) {
            float v[E];
            load_chunk<DT>(row_of(i), e0, p.V, vec_ok, v);
            const float wi = p.w[i];
#pragma unroll
            for (int k = 0; k < E; ++k) {
              cmb[k] = fmaf(wi, v[k], cmb[k]);
              if (i == p.mask_model) ve[k] = v[k];
              if (i == pis) q[k] = ex2_approx(fmaf(v[k], p.cT, ref_q)) * inv_zq;
            }
          }
#pragma unroll
          for (int k = 0; k < E; ++k) {
            bool in = (e0 + k < p.V) && (!masked || ve[k] >= thr);
            r[k] = in ? ex2_approx(fmaf(cmb[k], p.cT, ref_c)) * inv_zc : 0.f;
          }
        }
#pragma unroll
        for (int k = 0; k < E; ++k) {
          bool valid = (e0 + k < p.V);
          float m = use_r ? r[k] : fmaxf(0.f, r[k] - q[k]);
          res[k] = valid ? m : 0.f;
        }
        if (dump) {
          float* out = p.dump_r + (static_cast<long long>(b) * p.P + j) * p.V;
#pragma unroll
          for (int k = 0; k < E; ++k)
            if (e0 + k < p.V) out[e0 + k] = r[k];
        }
      };
      // per-step prefix over the 32 lanes in fp64: exclusive prefix and the lane's own sum
      auto lane_prefix = [&](const float (&res)[E], double& excl, float& own) {
        float ls = 0.f;
#pragma unroll
        for (int k = 0; k < E; ++k) ls += res[k];
        own = ls;
        double inc = static_cast<double>(ls);
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          double o = shfl_up_double(inc, d);
          if (lane >= d) inc += o;
        }
        excl = shfl_up_double(inc, 1);
        if (lane == 0) excl = 0.0;
      };

      for (int attempt = 0; attempt < 2; ++attempt) {
        const bool dump = (p.dump_r != nullptr) && attempt == 0;
        double wrun = 0.0;  // this warp's total, accumulated step by step
        for (int s = s_begin; s < s_end; ++s) {
          float res[E];
          chunk_mass((s * 32 + lane) * E, from_r, dump, res);
          double excl;
          float own;
          lane_prefix(res, excl, own);
          double step_total = shfl_double(excl + static_cast<double>(own), 31);
          wrun += step_total;
        }
        if (lane == 0) sh.wtot[warp] = wrun;
        __syncthreads();
        if (tid == 0) {
          double run = 0.0;
          for (int w = 0; w < kWarps; ++w) {
            run += sh.wtot[w];
            sh.wincl[w] = run;
          }
          sh.x[phase & 1].cta_total = run;
        }
        cluster.sync();
        if (tid == 0) {
          double tot[kMaxCluster];
          for (int r = 0; r < C; ++r) tot[r] = cluster.map_shared_rank(&sh.x[phase & 1], r)->cta_total;
          double S = 0.0;
          for (int r = 0; r < C; ++r) S += tot[r];
          const double target = sh.dec.u_smp * S;
          double cp = 0.0;
          int wr = -1, ww = -1;
          double wbase = 0.0;
          for (int r = 0; r < C && wr < 0; ++r) {
            if (cp + tot[r] >= target && tot[r] > 0.0) {
              wr = r;
              wbase = cp;
            }
            cp += tot[r];
          }
          if (wr == rank) {
            for (int w = 0; w < kWarps; ++w) {
              if (wbase + sh.wincl[w] >= target && sh.wtot[w] > 0.0) {
                ww = w;
                break;
              }
            }
            if (ww < 0) {  // rounding corner: last warp with mass
              for (int w = kWarps - 1; w >= 0; --w)
                if (sh.wtot[w] > 0.0) {
                  ww = w;
                  break;
                }
            }
          }
          sh.dec.S = S;
          sh.target = target;
          sh.base = wbase;
          sh.win_rank = (S > 0.0) ? wr : -2;
          sh.win_warp = ww;
        }
        __syncthreads();
        ++phase;
        if (attempt == 0 && !from_r) S_report = sh.dec.S;
        if (sh.win_rank == -2 && !from_r) {
          // no residual mass although a token is needed: draw from r instead
          from_r = true;
          if (tid == 0 && !sh.dec.accept) sh.dec.status |= COS_ROW_RESIDUAL_EMPTY;
          __syncthreads();
          continue;
        }
        break;
      }

      // the winning warp walks its run again and finds the token
      if (sh.win_rank == rank && sh.win_warp == warp) {
        const double target = sh.target;
        const double lex = (warp > 0) ? sh.wincl[warp - 1] : 0.0;
        const double cbase = sh.base;
        double R = 0.0;
        int token = -1, last_pos = -1;
        for (int s = s_begin; s < s_end && token < 0; ++s) {
          float res[E];
          const int e0 = (s * 32 + lane) * E;
          chunk_mass(e0, from_r, false, res);
          double excl;
          float own;
          lane_prefix(res, excl, own);
          const double incl = excl + static_cast<double>(own);
          const double step_total = shfl_double(incl, 31);
          const bool hit = (own > 0.f) && (cbase + (lex + (R + incl)) >= target);
          unsigned hits = __ballot_sync(0xffffffffu, hit);
          unsigned pos_lanes = __ballot_sync(0xffffffffu, own > 0.f);
          const bool step_hit = (cbase + (lex + (R + step_total)) >= target) && pos_lanes != 0u;
          if (step_hit) {
            int src = hits ? (__ffs(hits) - 1) : (31 - __clz(pos_lanes));
            int found = -1;
            if (lane == src) {
              float part = 0.f;
              int lastk = -1;
#pragma unroll
              for (int k = 0; k < E; ++k) {
                part += res[k];
                if (res[k] > 0.f) {
                  lastk = k;
                  if (found < 0 && cbase + (lex + (R + (excl + static_cast<double>(part)))) >= target) found = e0 + k;
                }
              }
              if (found < 0) found = e0 + lastk;
            }
            token = __shfl_sync(0xffffffffu, found, src);
          } else if (pos_lanes) {
            int src = 31 - __clz(pos_lanes);
            int lp = -1;
#pragma unroll
            for (int k = 0; k < E; ++k)
              if (res[k] > 0.f) lp = e0 + k;
            last_pos = __shfl_sync(0xffffffffu, lp, src);
          }
          R += step_total;
        }
        if (token < 0) token = last_pos;
        if (lane == 0) {
          const Decision& d = sh.dec;
          publish_unit(p, b, j, d.accept, d.status, token, d.ratio, d.r_d, d.q_d, S_report);
        }
      }
      published = (sh.win_rank >= 0);  // otherwise nothing had mass: rank 0 reports token -1 below
    }
    if (!published && rank == 0 && tid == 0) {
      const Decision& d = sh.dec;
      publish_unit(p, b, j, d.accept, d.status, d.cand, d.ratio, d.r_d, d.q_d, d.S);
    }
    __syncthreads();
    unit = next_unit;
  }
  cluster.sync();  // no block leaves while a peer may still read its shared memory
}

// ------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------
thread_local std::string g_create_error;

}  // namespace

struct cos_verify_ctx {
  cos_verify_config cfg;
  int cluster;
  int max_clusters;
  int sm_count;
  unsigned work_base;
  bool scratch_dirty;
  // device scratch
  unsigned* d_work_counter;
  int* d_row_arrivals;
  int* d_first_rej;
  int4* d_unit_res;
  // optional staging for host-pointer runs
  void* d_logits;
  int* d_drafts;
  int* d_proposer;
  int* d_accept;
  int* d_tokens;
  unsigned* d_status;
  float* d_diag;
  std::string err;
};

namespace {

using KernelFn = void (*)(const KParams);

KernelFn pick_kernel(int dtype, int mode) {
#define COS_CASE(DT, M) \
  if (dtype == DT && mode == M) return cos_verify_kernel<DT, M>;
  COS_CASE(COS_DTYPE_F32, kEnsembleSample)
  COS_CASE(COS_DTYPE_F32, kLogitSample)
  COS_CASE(COS_DTYPE_F32, kEnsembleGreedy)
  COS_CASE(COS_DTYPE_F32, kLogitGreedy)
  COS_CASE(COS_DTYPE_BF16, kEnsembleSample)
  COS_CASE(COS_DTYPE_BF16, kLogitSample)
  COS_CASE(COS_DTYPE_BF16, kEnsembleGreedy)
  COS_CASE(COS_DTYPE_BF16, kLogitGreedy)
#undef COS_CASE
  return nullptr;
}

int mode_of(const cos_verify_config& c) {
  const bool greedy = (c.temperature == 0.0f);
  if (c.combine == COS_COMBINE_PROB_ENSEMBLE) return greedy ? kEnsembleGreedy : kEnsembleSample;
  return greedy ? kLogitGreedy : kLogitSample;
}

int entries_per_vec(int dtype) { return dtype == COS_DTYPE_BF16 ? 8 : 4; }
int elem_bytes(int dtype) { return dtype == COS_DTYPE_BF16 ? 2 : 4; }

bool fail(std::string* dst, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  *dst = buf;
  return false;
}

bool validate_config(const cos_verify_config& c, std::string* err) {
  if (c.n < 1 || c.n > COS_MAX_MODELS) return fail(err, "n = %d outside 1..%d", c.n, COS_MAX_MODELS);
  if (c.combine != COS_COMBINE_PROB_ENSEMBLE && c.combine != COS_COMBINE_LOGIT_LINEAR)
    return fail(err, "unknown combine %d", c.combine);
  if (c.dtype != COS_DTYPE_F32 && c.dtype != COS_DTYPE_BF16) return fail(err, "unknown dtype %d", c.dtype);
  if (!(c.temperature >= 0.0f) || !isfinite(c.temperature)) return fail(err, "temperature must be finite and >= 0");
  if (c.gamma < 0) return fail(err, "gamma = %d must be >= 0", c.gamma);
  if (c.vocab < 1) return fail(err, "vocab = %d must be >= 1", c.vocab);
  if (c.max_batch < 1) return fail(err, "max_batch = %d must be >= 1", c.max_batch);
  if (static_cast<long long>(c.max_batch) * (c.gamma + 1) > 0x3fffffffLL) return fail(err, "max_batch * (gamma + 1) too large");
  double sum = 0.0;
  for (int i = 0; i < c.n; ++i) {
    if (!isfinite(c.weights[i])) return fail(err, "weight %d is not finite", i);
    sum += static_cast<double>(c.weights[i]);
  }
  if (c.combine == COS_COMBINE_PROB_ENSEMBLE) {
    for (int i = 0; i < c.n; ++i)
      if (c.weights[i] < 0.0f) return fail(err, "ensemble weight %d is negative", i);
    if (fabs(sum - 1.0) > 1e-6) return fail(err, "ensemble weights sum to %.9g, not 1", sum);
    if (c.mask_model >= 0) return fail(err, "the plausibility mask needs the logit-level combine");
  } else if (c.mask_model >= 0) {
    if (c.mask_model >= c.n) return fail(err, "mask_model = %d outside 0..n-1", c.mask_model);
    if (!(c.mask_alpha > 0.0f && c.mask_alpha <= 1.0f)) return fail(err, "mask_alpha must lie in (0, 1]");
  }
  if (c.mask_model < -1) return fail(err, "mask_model must be -1 or a model index");
  const int cs = c.cluster_size;
  if (!(cs == 0 || cs == 1 || cs == 2 || cs == 4 || cs == 8 || cs == 16))
    return fail(err, "cluster_size must be 0, 1, 2, 4, 8 or 16");
  return true;
}

int choose_cluster(const cos_verify_config& c) {
  if (c.cluster_size > 0) return c.cluster_size;
  const int nsteps = (c.vocab + 32 * entries_per_vec(c.dtype) - 1) / (32 * entries_per_vec(c.dtype));
  int cs = 8;
  while (cs > 1 && nsteps / (cs * kWarps) < 2) cs >>= 1;  // keep at least two steps per warp
  return cs;
}

cos_status cuda_fail(cos_verify_ctx* ctx, const char* what, cudaError_t e) {
  char buf[256];
  snprintf(buf, sizeof(buf), "%s: %s", what, cudaGetErrorString(e));
  if (ctx)
    ctx->err = buf;
  else
    g_create_error = buf;
  return COS_ERR_CUDA;
}

cos_status init_scratch(cos_verify_ctx* ctx, cudaStream_t stream) {
  const size_t rows = static_cast<size_t>(ctx->cfg.max_batch);
  cudaError_t e = cudaMemsetAsync(ctx->d_work_counter, 0, sizeof(unsigned), stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_row_arrivals, 0, rows * sizeof(int), stream);
  // kNoReject = 0x7fffffff is not a byte pattern; 0x7f7f7f7f is large enough to mean "no rejection yet"
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_first_rej, 0x7f, rows * sizeof(int), stream);
  if (e != cudaSuccess) return cuda_fail(ctx, "scratch reset", e);
  ctx->work_base = 0;
  ctx->scratch_dirty = false;
  return COS_OK;
}

}  // namespace

extern "C" cos_status cos_verify_create(const cos_verify_config* config, cos_verify_ctx** out) {
  if (!config || !out) {
    g_create_error = "null argument";
    return COS_ERR_INVALID_ARG;
  }
  *out = nullptr;
  if (!validate_config(*config, &g_create_error)) return COS_ERR_INVALID_ARG;
  cudaError_t e = cudaSetDevice(config->device);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaSetDevice", e);
  cos_verify_ctx* ctx = new (std::nothrow) cos_verify_ctx();
  if (!ctx) {
    g_create_error = "out of host memory";
    return COS_ERR_NOMEM;
  }
  ctx->cfg = *config;
  ctx->cluster = choose_cluster(*config);
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, config->device);
  if (e != cudaSuccess) {
    delete ctx;
    return cuda_fail(nullptr, "cudaGetDeviceProperties", e);
  }
  ctx->sm_count = prop.multiProcessorCount;
  KernelFn fn = pick_kernel(config->dtype, mode_of(*config));
  if (ctx->cluster > 8) {
    e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) {
      delete ctx;
      return cuda_fail(nullptr, "cluster size above 8 not available", e);
    }
  }
  {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(ctx->cluster * ctx->sm_count, 1, 1);
    lc.blockDim = dim3(kThreads, 1, 1);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = ctx->cluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    int nc = 0;
    e = cudaOccupancyMaxActiveClusters(&nc, reinterpret_cast<const void*>(fn), &lc);
    if (e != cudaSuccess || nc < 1) {
      delete ctx;
      if (e == cudaSuccess) {
        g_create_error = "no cluster of the requested size fits on the device";
        return COS_ERR_UNSUPPORTED;
      }
      return cuda_fail(nullptr, "cudaOccupancyMaxActiveClusters", e);
    }
    ctx->max_clusters = nc;
  }
  const size_t rows = static_cast<size_t>(config->max_batch), P = static_cast<size_t>(config->gamma) + 1;
  bool ok = true;
  ok = ok && cudaMalloc(&ctx->d_work_counter, 256) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_row_arrivals, rows * sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_first_rej, rows * sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_unit_res, rows * P * sizeof(int4)) == cudaSuccess;
  if (ok && config->host_staging) {
    const size_t V = static_cast<size_t>(config->vocab);
    ok = ok && cudaMalloc(&ctx->d_logits, static_cast<size_t>(config->n) * rows * P * V * elem_bytes(config->dtype)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_drafts, rows * (P > 1 ? P - 1 : 1) * sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_proposer, rows * sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_accept, rows * sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_tokens, rows * P * sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_status, rows * sizeof(unsigned)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_diag, rows * P * 4 * sizeof(float)) == cudaSuccess;
  }
  if (!ok) {
    (void)cudaGetLastError();
    cos_verify_destroy(ctx);
    g_create_error = "device allocation failed";
    return COS_ERR_NOMEM;
  }
  cos_status st = init_scratch(ctx, nullptr);
  if (st == COS_OK) {
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) st = cuda_fail(ctx, "cudaDeviceSynchronize", e);
  }
  if (st != COS_OK) {
    g_create_error = ctx->err;
    cos_verify_destroy(ctx);
    return st;
  }
  *out = ctx;
  return COS_OK;
}

extern "C" cos_status cos_verify_run(cos_verify_ctx* ctx, const cos_verify_args* a, void* cuda_stream) {
  if (!ctx) return COS_ERR_INVALID_ARG;
  if (!a) {
    ctx->err = "null args";
    return COS_ERR_INVALID_ARG;
  }
  const cos_verify_config& c = ctx->cfg;
  auto bad = [&](const char* m) {
    ctx->err = m;
    return COS_ERR_INVALID_ARG;
  };
  if (a->batch < 1 || a->batch > c.max_batch) return bad("batch outside 1..max_batch");
  if (!a->logits || !a->proposer || !a->accept_count || !a->out_tokens || !a->row_status) return bad("null device pointer");
  if (c.gamma > 0 && !a->draft_tokens) return bad("draft_tokens is null although gamma > 0");
  if (a->stride_model < 0 || a->stride_row < 0 || a->stride_pos < 0) return bad("negative stride");
  if (a->flags & ~COS_RUN_ALL_RESIDUALS) return bad("unknown flag bits");
  const int eb = elem_bytes(c.dtype);
  if (reinterpret_cast<uintptr_t>(a->logits) % eb) {
    ctx->err = "logits pointer not aligned to its element type";
    return COS_ERR_ALIGNMENT;
  }
  if (reinterpret_cast<uintptr_t>(a->proposer) % 4 || reinterpret_cast<uintptr_t>(a->accept_count) % 4 ||
      reinterpret_cast<uintptr_t>(a->out_tokens) % 4 || reinterpret_cast<uintptr_t>(a->row_status) % 4 ||
      (a->draft_tokens && reinterpret_cast<uintptr_t>(a->draft_tokens) % 4) ||
      (a->diag && reinterpret_cast<uintptr_t>(a->diag) % 4) || (a->dump_r && reinterpret_cast<uintptr_t>(a->dump_r) % 4)) {
    ctx->err = "an int32/float pointer is not 4-byte aligned";
    return COS_ERR_ALIGNMENT;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaSetDevice(c.device);
  if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
  if (ctx->scratch_dirty) {
    cos_status st = init_scratch(ctx, stream);
    if (st != COS_OK) return st;
  }

  KParams p;
  memset(&p, 0, sizeof(p));
  p.logits = a->logits;
  p.s_model = a->stride_model;
  p.s_row = a->stride_row;
  p.s_pos = a->stride_pos;
  p.drafts = a->draft_tokens;
  p.proposer = a->proposer;
  p.n = c.n;
  p.V = c.vocab;
  p.gamma = c.gamma;
  p.P = c.gamma + 1;
  p.B = a->batch;
  p.mask_model = (c.combine == COS_COMBINE_LOGIT_LINEAR) ? c.mask_model : -1;
  const int E = entries_per_vec(c.dtype);
  p.vec_ok = (reinterpret_cast<uintptr_t>(a->logits) % 16 == 0) && ((a->stride_model * eb) % 16 == 0) &&
             ((a->stride_row * eb) % 16 == 0) && ((a->stride_pos * eb) % 16 == 0);
  p.nsteps = (c.vocab + 32 * E - 1) / (32 * E);
  p.flags = a->flags;
  p.num_units = a->batch * (c.gamma + 1);
  p.num_clusters = p.num_units < ctx->max_clusters ? p.num_units : ctx->max_clusters;
  for (int i = 0; i < COS_MAX_MODELS; ++i) {
    p.w[i] = (i < c.n) ? c.weights[i] : 0.f;
    p.w64[i] = static_cast<double>(p.w[i]);
  }
  if (c.temperature > 0.0f) {
    p.cT = static_cast<float>(1.4426950408889634 / static_cast<double>(c.temperature));
    p.cT64 = static_cast<double>(p.cT);
  }
  p.ln_alpha = (p.mask_model >= 0) ? log(static_cast<double>(c.mask_alpha)) : 0.0;
  p.seed_lo = static_cast<unsigned>(a->seed);
  p.seed_hi = static_cast<unsigned>(a->seed >> 32);
  p.off_lo = static_cast<unsigned>(a->offset);
  p.off_hi = static_cast<unsigned>(a->offset >> 32);
  p.row_base = a->row_base;
  p.accept_count = a->accept_count;
  p.out_tokens = a->out_tokens;
  p.row_status = a->row_status;
  p.diag = a->diag;
  p.dump_r = a->dump_r;
  p.work_counter = ctx->d_work_counter;
  p.work_base = ctx->work_base;
  p.row_arrivals = ctx->d_row_arrivals;
  p.first_rej = ctx->d_first_rej;
  p.unit_res = ctx->d_unit_res;

  KernelFn fn = pick_kernel(c.dtype, mode_of(c));
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(static_cast<unsigned>(p.num_clusters) * ctx->cluster, 1, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = ctx->cluster;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  ctx->scratch_dirty = true;  // cleared below once the launch is known to be queued
  e = cudaLaunchKernelEx(&lc, fn, p);
  if (e != cudaSuccess) return cuda_fail(ctx, "kernel launch", e);
  // every unit is fetched exactly once from the counter or assigned statically, and every
  // cluster that ran fetches once past the end
  ctx->work_base += static_cast<unsigned>(p.num_units);
  ctx->scratch_dirty = false;
  return COS_OK;
}

extern "C" cos_status cos_verify_run_host(cos_verify_ctx* ctx, const cos_verify_args* a, void* cuda_stream) {
  if (!ctx) return COS_ERR_INVALID_ARG;
  if (!a) {
    ctx->err = "null args";
    return COS_ERR_INVALID_ARG;
  }
  const cos_verify_config& c = ctx->cfg;
  if (!ctx->d_logits) {
    ctx->err = "context was created without host_staging";
    return COS_ERR_INVALID_ARG;
  }
  if (a->batch < 1 || a->batch > c.max_batch) {
    ctx->err = "batch outside 1..max_batch";
    return COS_ERR_INVALID_ARG;
  }
  if (a->dump_r) {
    ctx->err = "dump_r is not available for host-pointer runs";
    return COS_ERR_UNSUPPORTED;
  }
  if (!a->logits || !a->proposer || !a->accept_count || !a->out_tokens || !a->row_status || (c.gamma > 0 && !a->draft_tokens)) {
    ctx->err = "null host pointer";
    return COS_ERR_INVALID_ARG;
  }
  const long long V = c.vocab, P = c.gamma + 1, B = a->batch;
  if (a->stride_pos != V || a->stride_row != P * V || a->stride_model != B * P * V) {
    ctx->err = "host-pointer runs need contiguous [n][B][gamma+1][V] logits";
    return COS_ERR_INVALID_ARG;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaSetDevice(c.device);
  if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
  const size_t lbytes = static_cast<size_t>(c.n) * B * P * V * elem_bytes(c.dtype);
  e = cudaMemcpyAsync(ctx->d_logits, a->logits, lbytes, cudaMemcpyHostToDevice, stream);
  if (e == cudaSuccess && c.gamma > 0)
    e = cudaMemcpyAsync(ctx->d_drafts, a->draft_tokens, B * c.gamma * sizeof(int), cudaMemcpyHostToDevice, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_proposer, a->proposer, B * sizeof(int), cudaMemcpyHostToDevice, stream);
  if (e != cudaSuccess) return cuda_fail(ctx, "host to device copy", e);
  cos_verify_args d = *a;
  d.logits = ctx->d_logits;
  d.draft_tokens = ctx->d_drafts;
  d.proposer = ctx->d_proposer;
  d.accept_count = ctx->d_accept;
  d.out_tokens = ctx->d_tokens;
  d.row_status = ctx->d_status;
  d.diag = a->diag ? ctx->d_diag : nullptr;
  cos_status st = cos_verify_run(ctx, &d, stream);
  if (st != COS_OK) return st;
  e = cudaMemcpyAsync(a->accept_count, ctx->d_accept, B * sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(a->out_tokens, ctx->d_tokens, B * P * sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(a->row_status, ctx->d_status, B * sizeof(unsigned), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess && a->diag)
    e = cudaMemcpyAsync(a->diag, ctx->d_diag, B * P * 4 * sizeof(float), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) {
    ctx->scratch_dirty = true;
    return cuda_fail(ctx, "device to host copy", e);
  }
  return COS_OK;
}

extern "C" cos_status cos_verify_get_info(const cos_verify_ctx* ctx, cos_verify_info* info) {
  if (!ctx || !info) return COS_ERR_INVALID_ARG;
  memset(info, 0, sizeof(*info));
  info->cluster_size = ctx->cluster;
  info->threads_per_block = kThreads;
  info->max_clusters = ctx->max_clusters;
  info->sm_count = ctx->sm_count;
  info->launches_per_run = 1;
  return COS_OK;
}

extern "C" cos_status cos_verify_destroy(cos_verify_ctx* ctx) {
  if (!ctx) return COS_OK;
  (void)cudaSetDevice(ctx->cfg.device);
  (void)cudaDeviceSynchronize();
  cudaFree(ctx->d_work_counter);
  cudaFree(ctx->d_row_arrivals);
  cudaFree(ctx->d_first_rej);
  cudaFree(ctx->d_unit_res);
  cudaFree(ctx->d_logits);
  cudaFree(ctx->d_drafts);
  cudaFree(ctx->d_proposer);
  cudaFree(ctx->d_accept);
  cudaFree(ctx->d_tokens);
  cudaFree(ctx->d_status);
  cudaFree(ctx->d_diag);
  (void)cudaGetLastError();
  delete ctx;
  return COS_OK;
}

extern "C" const char* cos_verify_last_error(const cos_verify_ctx* ctx) {
  return ctx ? ctx->err.c_str() : g_create_error.c_str();
}
