// CoS verification step for sm_100a: combine (Eq. 3-5), accept test (Eq. 6), residual / bonus sample and
// first-rejection scan (Sec. 3.1) for every row of a batch and every one of its gamma + 1 positions.
//
// Work unit = one (row b, position j).  One kernel template, instantiated per stage:
//   stage 0  every unit: stream the n logit rows once from HBM (128-bit streaming loads), keep per-lane
//            softmax statistics (reference exponent, sum of 2^(l*c - ref)) or argmaxes, merge them, take
//            the accept test in fp64 from the merged statistics and the logits at the draft token, publish
//            the unit; the last unit of a row to arrive scans for the first rejection, writes the row's
//            outputs and lists the one unit of the row that must draw a token.  Two forms of the unit loop:
//            a barrier-free one (a block owns a unit, its warps run from unit to unit and meet through
//            volatile words in shared memory) and a cluster form (the blocks of a thread-block cluster
//            split the vocabulary and exchange partial results through distributed shared memory);
//   stage 1  listed units only: the normalisers again, terms above 2^-8 of a normaliser in fp64;
//   stage 2  listed units only: token masses max(0, r - q) (or the law of the bonus token), every warp on
//            a contiguous run of the vocabulary so that prefix order is token order, fp64 running totals;
//            the last block of a unit to finish locates u * S and walks to the token;
//   stage 3  stages 1 and 2 in one sweep, for logit-level combines and two-model ensembles: there a mass is
//            k_A e_A / Z_A + k_B e_B / Z_B clipped at zero, linear in 1/Z_A and 1/Z_B over the tokens where
//            it is positive; that set is decided with stage 0's normalisers, the sweep records the two sums
//            of every step (256 or 128 consecutive tokens) next to the refined normalisers, and the last
//            block of a unit turns the sums into masses, finds the step by a prefix and walks it.
// Units are handed out from a global counter.  Between blocks there are only fences and arrival counters;
// the launches of a run (stage 0, then 3 or 1 and 2) order the stages.  Waits exist only inside a block of the barrier-free form,
// and they are bounded: a wait that gave up marks every row with COS_ROW_FAULT and the block leaves.
// At T = 0 stage 0 is the whole run.

#include <mutex>

#include "cos_common.cuh"
#include "cos_fused.h"

using namespace cosv;

namespace {

// Optional timeline of the one-sweep drawing stage (build with -DCOS_STAGE_PROFILE): thread 0 of every block stamps
// the global timer at eight points into g_sprof[block][point].  Compiled out of ordinary builds.
#ifdef COS_STAGE_PROFILE
constexpr int kSprofBlocks = 1024;
__device__ unsigned long long g_sprof[kSprofBlocks * 8];
#define SPROF(k)                                                                                  \
  do {                                                                                            \
    if (threadIdx.x == 0 && blockIdx.x < kSprofBlocks) {                                          \
      unsigned long long t_;                                                                      \
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));                                       \
      g_sprof[blockIdx.x * 8 + (k)] = t_;                                                         \
    }                                                                                             \
  } while (0)
#else
#define SPROF(k)
#endif

struct Xchg {  // one per block and barrier parity; peers read it through DSMEM
  SoftPart soft[kMaxSlots];
  ArgPart arg[kMaxSlots];
  double cta_total;
  int pad;
  int next;   // rank 0 only: the unit this cluster takes after the current one
};

struct Decision {  // written by thread 0 of every block, identically
  int accept, status, want_sample, cand;
  int natoms, need2, drawable;
  int atom_tok[COS_MAX_MODELS];
  double atom_mass[COS_MAX_MODELS];
  double ratio, r_d, q_d, S;
  double prob;  // greedy, bonus position: probability of cand under the law it came from
};

// Stage 0 without block barriers: every warp streams its share of unit after unit; what the warps of
// a block tell each other goes through these words (volatile accesses, fences, bounded waits).
struct FreeRun {
  SoftPart wsoft[2][kWarps][kMaxSlots];  // warp partials, two units deep
  ArgPart warg[2][kWarps][kMaxSlots];
  int unit_of[4];   // the unit this block processes as its seq-th, at [seq & 3]
  int unit_tag[4];  // seq + 1 once unit_of[seq & 3] is valid
  int arrive[2];    // warps that have finished the unit of that parity
  int epi_done;     // units whose merge and decision are complete
  int fault;        // a wait gave up
  int left;         // warps that have left the loop
  int skip_state[2];  // unit of that parity: 0 undecided, 1 swept, 2 left unread (its row is already rejected earlier)
};

struct OneSweep {  // constants of the one-sweep drawing stage, for its out-of-line part
  float ctA, ctB;        // k / first-estimate normaliser of each channel: decides the sign of a mass
  float nrefA, nrefB;    // minus the reference exponents
  float btA, btB;        // terms above these are big
  double ctA64, ctB64, drefA, drefB;
};

struct OneSweepN {  // the same for the one-sweep stage that keeps a channel per model (ensembles of three or four)
  float ct[4], nref[4], bt[4];
  double ct64[4], dref[4];
};

struct Raw4 {  // one lane's vector of each of up to four models
  uint4 r[4];
};

struct Shared;
__device__ __forceinline__ OneSweep& one_sweep_consts(Shared& sh);
__device__ __forceinline__ double* one_sweep_coef(Shared& sh);

struct Shared {
  Xchg x[2];
  FreeRun fr;
  SoftPart wsoft[kWarps][kMaxSlots];
  ArgPart warg[kWarps][kMaxSlots];
  double wtot[kWarps];        // this block's per-warp totals of sweep 2
  double wincl[kWarps];       // their running sum
  double srun[kWarps][kRec];  // a warp's running total after each group of steps
  double gw[kMaxParts * kWarps];  // locating the token: mass of every warp run of the unit (the one-sweep stage,
                                  // which has no runs, keeps its constants here: see one_sweep_consts)
  int win_g;
  SoftPart fsoft[kMaxSlots];  // merged over the cluster
  ArgPart farg[kMaxSlots];
  double pdraft[kMaxSlots];   // probability of the draft token under each merged softmax
  float a_scale[COS_MAX_MODELS];  // w_i / Z_i (ensemble) for sweep 2
  float a_ref[COS_MAX_MODELS];
  float a_resid[COS_MAX_MODELS];  // coefficient of e_i in r - q
  float a_draw[COS_MAX_MODELS];   // coefficient of e_i in the law a bonus token is drawn from (r, or the named model's)
  Decision dec;
  double u_acc, u_smp;
  double target, base;  // sweep-2 search: u*S and the mass before the winning block
  int win_rank, win_warp;
  int next_local, next;
  float thr32;  // plausibility threshold rounded up to fp32
  float big_thr[kMaxSlots];  // sweep 2: terms above this share of a normaliser are redone in fp64
  float ldraft[COS_MAX_MODELS];  // the n logits at the draft token, fetched before sweep 1
};

// The one-sweep drawing stage never fills gw[]; its constants and the two exact coefficients of the channel
// sums live there, so that the layout of Shared is the same for every stage.
static_assert(sizeof(OneSweep) <= 16 * sizeof(double), "OneSweep must fit in front of the coefficients");
static_assert(sizeof(OneSweepN) <= 16 * sizeof(double), "OneSweepN must fit in front of the coefficients");
__device__ __forceinline__ OneSweepN& one_sweep_consts_n(Shared& sh) { return *reinterpret_cast<OneSweepN*>(&sh.gw[0]); }
__device__ __forceinline__ OneSweep& one_sweep_consts(Shared& sh) { return *reinterpret_cast<OneSweep*>(&sh.gw[0]); }
__device__ __forceinline__ double* one_sweep_coef(Shared& sh) { return &sh.gw[16]; }

// Block merge of the warp partials, publish for the peers, ONE cluster barrier, merge over
// the ranks.  Warp k handles soft slot k (k < nsoft); warp 8 + k handles arg slot a0 + k.
// All threads of all blocks of the cluster call this; results land in sh.fsoft / sh.farg,
// and the cluster's next unit (drawn by rank 0) in sh.next.
__device__ __forceinline__ void cluster_merge(Shared& sh, cg::cluster_group& cluster, int& phase, int nsoft, int a0,
                                              int narg) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int C = cluster.num_blocks();
  __syncthreads();
  Xchg& mine = sh.x[phase & 1];
  if (warp < nsoft) {
    float ref = (lane < kWarps) ? sh.wsoft[lane][warp].ref : -INFINITY;
    double s = (lane < kWarps) ? sh.wsoft[lane][warp].s : 0.0;
    SoftPart o = warp_reduce_soft(ref, s);
    if (lane == 0) mine.soft[warp] = o;
  } else if (warp >= 8 && warp < 8 + narg) {
    const int slot = a0 + warp - 8;
    ArgPart in;
    if (lane < kWarps) {
      in = sh.warg[lane][slot];
    } else {
      in.val = -INFINITY;
      in.idx = kNoReject;
      in.bad = 0;
    }
    ArgPart o = warp_reduce_arg(in.val, in.idx, in.bad, lane);
    if (lane == 0) mine.arg[slot] = o;
  } else if (warp == kWarps - 1 && lane == 0) {
    mine.next = sh.next_local;
  }
  cluster.sync();
  if (warp < nsoft) {
    float ref = -INFINITY;
    double s = 0.0;
    if (lane < C) {
      const Xchg* peer = cluster.map_shared_rank(&sh.x[phase & 1], lane);
      ref = peer->soft[warp].ref;
      s = peer->soft[warp].s;
    }
    SoftPart o = warp_reduce_soft(ref, s);
    if (lane == 0) sh.fsoft[warp] = o;
  } else if (warp >= 8 && warp < 8 + narg) {
    const int slot = a0 + warp - 8;
    ArgPart in;
    in.val = -INFINITY;
    in.idx = kNoReject;
    in.bad = 0;
    if (lane < C) in = cluster.map_shared_rank(&sh.x[phase & 1], lane)->arg[slot];
    ArgPart o = warp_reduce_arg(in.val, in.idx, in.bad, lane);
    if (lane == 0) sh.farg[slot] = o;
  } else if (warp == kWarps - 1 && lane == 0) {
    const Xchg* r0 = cluster.map_shared_rank(&sh.x[phase & 1], 0);
    sh.next = r0->next;
  }
  __syncthreads();
  ++phase;
}

// A block leaves stage 0 of a greedy run (which = 0) or stage 2 (which = 1).  The last block of the launch to
// leave puts the counter of that stage back to zero, so that every run starts from the same state with the same
// arguments (a run can then be captured in a graph and replayed).  One thread per block calls it, after the
// block's last use of the counter has returned its value; the end of the launch publishes the reset.
// (When stages follow, the work counter is cleared by stage 1 instead, which costs nothing.)
__device__ __forceinline__ void stage_exit(const KParams& p, int which) {
  const unsigned prev = atomicAdd(&p.exit_count[which], 1u);
  if (prev == gridDim.x - 1) {
    p.exit_count[which] = 0u;
    if (which == 0)
      *p.work_counter = 0u;
    else
      *p.job_count = 0;
    __threadfence();
  }
}

// ------------------------------------------------------------------------------------
// publishing a unit and the per-row first-rejection scan (Sec. 3.1)
// ------------------------------------------------------------------------------------
__device__ __forceinline__ void push_job(const KParams& p, int idx, int emit) {
  const int k = atomicAdd(p.job_count, 1);
  if (k < p.max_jobs) p.jobs[k] = make_int2(idx, emit);
}

// Stage 0: record a unit's decision; the last unit of a row to arrive scans for the first
// rejection, writes the row's outputs and, where a token has to be drawn, lists that unit
// for the drawing stages (stage 2 fills in out_tokens[b][a]).
// `word4`: sampling modes: whether a token can be drawn at this unit; greedy modes: the bits of the bonus
// token's probability (a float), NaN away from the bonus position.
__device__ void publish_unit(const KParams& p, int b, int j, int accept, int status, int cand, int word4,
                             double ratio, double r_d, double q_d, double S) {
  const int drawable = p.greedy ? 0 : word4;
  const int idx = b * p.P + j;
  if (p.diag) {
    float* d = p.diag + static_cast<long long>(idx) * 4;
    d[0] = static_cast<float>(ratio);
    d[1] = static_cast<float>(r_d);
    d[2] = static_cast<float>(q_d);
    d[3] = static_cast<float>(S);
  }
  int4 res = make_int4(accept, status, cand, word4);
  __stcg(&p.unit_res[idx], res);
  if (p.early_exit && !accept && j < p.gamma) atomicMin(&p.row_reject[b], j);  // later positions may be left unread
  // test hooks: the combined distribution everywhere, or the residual mass at every draft position
  if (drawable && (p.dump_r != nullptr || ((p.flags & COS_RUN_ALL_RESIDUALS) && j < p.gamma))) push_job(p, idx, 0);
  __threadfence();
  // The row's word counts its published positions (low six bits) and, for rows of up to kPackedP positions,
  // also carries one "not accepted" bit and one "has status bits" bit per position: the last position to
  // arrive then knows the first rejection from the value the atomic returns, without reading the others.
  const bool packed = (p.P <= kPackedP);
  int mine = 1;
  if (packed) {
    if (!accept || j == p.gamma) mine |= 1 << (6 + j);
    if (status) mine |= 1 << (6 + kPackedP + j);
  }
  const int prev = atomicAdd(&p.row_arrivals[b], mine);
  if ((packed ? (prev & 63) : prev) != p.P - 1) return;  // longer rows keep a plain count in the word
  // last unit of the row: every other unit's result is visible after the fence below
  __threadfence();
  int a = p.gamma;
  unsigned st = 0;
  int tok = -1, draw = 0;
  if (packed) {
    const int total = prev + mine;  // every position added its own bits once: no carries
    a = __ffs((total >> 6) & ((1 << kPackedP) - 1)) - 1;
    const int4 u = __ldcg(&p.unit_res[b * p.P + a]);
    tok = u.z;
    draw = u.w;
    int with_status = (total >> (6 + kPackedP)) & ((2 << a) - 1);
    while (with_status) {  // rare: some position up to the first rejection reported status bits
      const int k = __ffs(with_status) - 1;
      with_status &= with_status - 1;
      st |= static_cast<unsigned>(__ldcg(&p.unit_res[b * p.P + k]).y);
    }
  } else {
    for (int k = 0; k < p.P; ++k) {
      int4 u = __ldcg(&p.unit_res[b * p.P + k]);
      st |= static_cast<unsigned>(u.y);
      if (k == p.gamma || !u.x) {
        a = k;
        tok = u.z;
        draw = u.w;
        break;
      }
    }
  }
  if (p.bonus_prob != nullptr) {
    // sampling modes: the drawing stage fills it in after a full acceptance; greedy modes know it here
    const bool known = p.greedy && a == p.gamma && tok >= 0;
    p.bonus_prob[b] = known ? __int_as_float(draw) : __int_as_float(0x7fc00000);
  }
  if (p.greedy) draw = 0;
  p.accept_count[b] = a;
  int* o = p.out_tokens + static_cast<long long>(b) * p.P;
  for (int k = 0; k < p.P; ++k) o[k] = (k < a) ? p.drafts[b * p.gamma + k] : (k == a ? tok : -1);
  p.row_status[b] = st;
  p.row_arrivals[b] = 0;  // leave the scratch ready for the next run
  if (p.early_exit) p.row_reject[b] = kNoReject;
  // under the test hooks the unit may already be on the list: every unit is listed once at most
  const bool listed = (p.dump_r != nullptr) || ((p.flags & COS_RUN_ALL_RESIDUALS) && a < p.gamma);
  if (draw && !listed) push_job(p, b * p.P + a, 1);
}

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
      float e[4], acc = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        e[i] = ex2_approx(fmaf(x[i][k], p.cT, nref[i]));
        vz[i] += e[i];
        acc = __fadd_rn(acc, __fmul_rn(ct[i], e[i]));
      }
      const float in_p = (acc > 0.f) ? 1.f : 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) va[i] = fmaf(in_p, e[i], va[i]);
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
  // what the loop needs of the launch parameters, in registers (through `p` it would be read again after every store)
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
      const float eA = ex2_approx(fmaf(xa[k], cT, nrefA));
      const float eB = ex2_approx(fmaf(xb[k], cT, nrefB));
      // k_A e_A / Z_A + k_B e_B / Z_B > 0 with the products rounded one by one: where r and q coincide
      // neither side exceeds the other, as in exact arithmetic
      const float in_p = (__fmul_rn(ctB, eB) > __fmul_rn(nctA, eA)) ? 1.f : 0.f;
      vzA += eA;
      vzB += eB;
      vaA = fmaf(in_p, eA, vaA);
      vaB = fmaf(in_p, eB, vaB);
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
    // the step's two sums over the warp
    float ra = aA, rb = aB;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      ra += __shfl_xor_sync(0xffffffffu, ra, d);
      rb += __shfl_xor_sync(0xffffffffu, rb, d);
    }
    double da = static_cast<double>(ra), db = static_cast<double>(rb);
    if (__any_sync(0xffffffffu, hasbig)) {
      double ta = bigacc[2 * kThreads], tb = bigacc[3 * kThreads];
      bigacc[2 * kThreads] = bigacc[3 * kThreads] = 0.0;
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) {
        ta += shfl_double(ta, lane ^ d);
        tb += shfl_double(tb, lane ^ d);
      }
      da += ta;
      db += tb;
    }
    if (lane == 0 && emit) {
      rec_a[rec_at + s] = da;
      rec_b[rec_at + s] = db;
    }
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

// Combined logit of one token in fp64, from the stored logits: the chain of fused multiply-adds that
// defines the greedy argmax (Eq. 5 at T = 0).  Out of line: the sweep calls it for a handful of tokens.
template <int DT>
__device__ __noinline__ double exact_combined(const KParams& p, const char* base, int e) {
  double cm = 0.0;
  for (int i = 0; i < p.n; ++i) {
    const void* row = base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes;
    cm = fma(p.w64[i], static_cast<double>(Elem<DT>::load1(row, e)), cm);
  }
  return cm;
}

// Sweep 1 of one (row, position): this thread's share of the slice `sl` of every model's row, merged
// over the warp into the warp's slots.  Ensemble sampling: soft slot i = softmax statistics of model i.
// Ensemble greedy: arg slot i = argmax of model i.  Logit-level sampling: soft slot 0 = proposer,
// soft slot 1 = combined logits.  Logit-level greedy: arg slot 1 = proposer argmax, arg slot 2 =
// combined argmax.  `thr` is the plausibility threshold (logit-level modes with a mask).
template <int DT, int MODE>
__device__ __forceinline__ void sweep_unit(const KParams& p, const char* base, const Slice& sl, int pis, bool masked,
                                           float thr, SoftPart* wsoft, ArgPart* warg) {
  constexpr int E = Elem<DT>::E;
  const int tid = threadIdx.x, lane = tid & 31;
  auto row_of = [&](int i) -> const void* { return base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes; };
  if (MODE == kEnsembleSample) {
    for (int i = 0; i < p.n; ++i) {
      LaneSoft acc = soft_slice<DT, kThreads>(row_of(i), sl, tid, p.cT);
      warp_merge_soft(acc, &wsoft[i], lane);
    }
  } else if (MODE == kEnsembleGreedy) {
    for (int i = 0; i < p.n; ++i) {
      const void* row = row_of(i);
      float best = -INFINITY;
      int bidx = kNoReject, bad = 0;
      auto see = [&](float x, int e) {
        bad |= !(x < INFINITY);
        if (x > best) {
          best = x;
          bidx = e;
        }
      };
      for (int v = sl.v_lo + tid; v < sl.v_hi; v += kThreads) {
        float x[E];
        uint4 raw = ldg_stream16(reinterpret_cast<const char*>(row) + static_cast<long long>(v) * 16);
        Elem<DT>::unpack(raw, x);
#pragma unroll
        for (int k = 0; k < E; ++k) see(x[k], v * E + k);
      }
      for (int e = sl.e_lo + tid; e < sl.e_hi; e += kThreads) see(Elem<DT>::load1(row, e), e);
      warp_merge_arg(static_cast<double>(best), bidx, bad, &warg[i], lane);
    }
  } else if (MODE == kLogitSample) {
    LaneSoft accq, accc;
    logit_soft_slice<DT, kThreads>(p, base, sl, tid, pis, masked, thr, accq, accc);
    warp_merge_soft(accq, &wsoft[0], lane);
    warp_merge_soft(accc, &wsoft[1], lane);
  } else {
    // The argmax of the combined logits must be the fp64 one (the same chain of fused multiply-adds
    // on every token, lowest index among equals).  Every token gets an fp32 value and a bound on its
    // distance from the fp64 value; only tokens that could reach the best fp64 value seen so far are
    // evaluated in fp64.
    double cbest = -INFINITY;
    float cbest_lo = -INFINITY;  // a lower bound of the maximum in fp32: the best fp64 value seen by the warp, rounded down
    int cidx = kNoReject, bad = 0;
    float qbest = -INFINITY;
    int qidx = kNoReject;
    const char* row0 = reinterpret_cast<const char*>(row_of(0));
    const long long row_step = p.s_model * Elem<DT>::bytes;
    const float kSlack = static_cast<float>(p.n) * 1.1920929e-07f;  // n * 2^-23: rounding of the fp32 chain
    auto consider = [&](float c32, float bnd, int e) {  // token inside the mask
      bad |= (c32 != c32);
      if (__fmaf_ru(bnd, kSlack, c32) >= cbest_lo) {
        const double cm = exact_combined<DT>(p, base, e);
        if (cm > cbest) {  // tokens come in increasing order within a thread: ties keep the earlier one
          cbest = cm;
          cidx = e;
          const float lo = __double2float_rd(cm);
          if (lo > cbest_lo) cbest_lo = lo;
        }
      }
    };
    // the vectors of the first two models are fetched one trip ahead: four loads in flight per thread
    const bool pair = (p.n >= 2);
    uint4 nx0 = make_uint4(0u, 0u, 0u, 0u), nx1 = nx0;
    {
      const int v0 = sl.v_lo + tid;
      if (v0 < sl.v_hi) {
        nx0 = ldg_stream16(row0 + static_cast<long long>(v0) * 16);
        if (pair) nx1 = ldg_stream16(row0 + row_step + static_cast<long long>(v0) * 16);
      }
    }
    for (int v = sl.v_lo + tid; v < sl.v_hi; v += kThreads) {
      const uint4 a0 = nx0, a1 = nx1;
      {
        const int vn = v + kThreads;
        if (vn < sl.v_hi) {
          nx0 = ldg_stream16(row0 + static_cast<long long>(vn) * 16);
          if (pair) nx1 = ldg_stream16(row0 + row_step + static_cast<long long>(vn) * 16);
        }
      }
      float c32[E], bnd[E];
      unsigned inbits = 0xffffffffu;
#pragma unroll
      for (int k = 0; k < E; ++k) c32[k] = bnd[k] = 0.f;
      auto take = [&](int i, const uint4& raw) {
        float x[E];
        Elem<DT>::unpack(raw, x);
        const float wi = p.w[i], wa = fabsf(wi);
#pragma unroll
        for (int k = 0; k < E; ++k) {
          bad |= !(x[k] < INFINITY);
          c32[k] = fmaf(wi, x[k], c32[k]);
          bnd[k] = fmaf(wa, fabsf(x[k]), bnd[k]);
        }
        if (i == pis) {
          float xm = x[0];
#pragma unroll
          for (int k = 1; k < E; ++k) xm = fmaxf(xm, x[k]);
          if (xm > qbest) {  // rare after the first few vectors; the first of equal entries wins
            qbest = xm;
#pragma unroll
            for (int k = E - 1; k >= 0; --k)
              if (x[k] == xm) qidx = v * E + k;
          }
        }
        if (masked && i == p.mask_model) {
          inbits = 0u;
#pragma unroll
          for (int k = 0; k < E; ++k) inbits |= (x[k] >= thr) ? (1u << k) : 0u;
        }
      };
      take(0, a0);
      if (pair) take(1, a1);
      const long long off = static_cast<long long>(v) * 16;
      for (int i = 2; i < p.n; ++i) take(i, ldg_stream16(row0 + i * row_step + off));
      // upper bounds of the fp64 values; one comparison decides whether any entry of the vector can matter.
      // The sum only carries a NaN (or an infinity of each sign) to the check below.
      float tmax = -INFINITY, tsum = 0.f;
#pragma unroll
      for (int k = 0; k < E; ++k) {
        const float t = (inbits & (1u << k)) ? __fmaf_ru(bnd[k], kSlack, c32[k]) : -INFINITY;
        tmax = fmaxf(tmax, t);
        tsum += t;
      }
      if (tmax >= cbest_lo || tsum != tsum) {
#pragma unroll
        for (int k = 0; k < E; ++k)
          if (inbits & (1u << k)) consider(c32[k], bnd[k], v * E + k);
      }
      // any exact value found by a lane of the warp is a lower bound of the maximum for all of them:
      // share the largest (floats ordered as unsigned integers, one warp-wide max)
      {
        const unsigned bits = __float_as_uint(cbest_lo);
        const unsigned key = bits ^ ((bits >> 31) ? 0xffffffffu : 0x80000000u);
        const unsigned top = __reduce_max_sync(__activemask(), key);
        const unsigned back = top ^ ((top >> 31) ? 0x80000000u : 0xffffffffu);
        const float shared_lo = __uint_as_float(back);
        if (shared_lo > cbest_lo) cbest_lo = shared_lo;
      }
    }
    for (int e = sl.e_lo + tid; e < sl.e_hi; e += kThreads) {
      float c32 = 0.f, bnd = 0.f, xe = 0.f;
      for (int i = 0; i < p.n; ++i) {
        float x = Elem<DT>::load1(row_of(i), e);
        bad |= !(x < INFINITY);
        c32 = fmaf(p.w[i], x, c32);
        bnd = fmaf(fabsf(p.w[i]), fabsf(x), bnd);
        if (i == pis && x > qbest) {
          qbest = x;
          qidx = e;
        }
        if (i == p.mask_model) xe = x;
      }
      if (!masked || xe >= thr) consider(c32, bnd, e);
    }
    warp_merge_arg(static_cast<double>(qbest), qidx, bad, &warg[1], lane);
    warp_merge_arg(cbest, cidx, bad, &warg[2], lane);
  }
}

// The accept test of one (row, position) from the merged statistics in shared memory (Eq. 6), taken
// by one thread in fp64; greedy modes also settle the replacement token here.  Reads fsoft / farg /
// pdraft / ldraft / u_acc / u_smp / thr32, writes dec and big_thr.
template <int DT, int MODE>
__device__ __forceinline__ void decide_unit(const KParams& p, Shared& sh, bool is_bonus, int draft, bool draft_ok,
                                            int pi, bool pi_ok, int pis, bool masked) {
  constexpr bool kSample = (MODE == kEnsembleSample || MODE == kLogitSample);
  const double kNaN = __longlong_as_double(0x7ff8000000000000LL);
  const double kInf = __longlong_as_double(0x7ff0000000000000LL);
  Decision& d = sh.dec;
  const double u_acc = sh.u_acc;
  d.accept = 0;
  d.status = 0;
  d.want_sample = 0;
  d.cand = -1;
  d.natoms = 0;
  d.ratio = d.r_d = d.q_d = d.S = d.prob = kNaN;
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
      for (int k = 0; k < nsoft; ++k) sh.big_thr[k] = static_cast<float>(sh.fsoft[k].s * kBigShare);
      if (!is_bonus) {
        if (draft_ok) {
          double r_d = 0.0, q_d = 0.0;
          if (MODE == kEnsembleSample) {
            for (int i = 0; i < p.n; ++i) {
              r_d += p.w64[i] * sh.pdraft[i];
              if (i == pi) q_d = sh.pdraft[i];
            }
          } else {
            double cd = 0.0;
            for (int i = 0; i < p.n; ++i) cd = fma(p.w64[i], static_cast<double>(sh.ldraft[i]), cd);
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
            d.ratio = (r_d > 0.0) ? kInf : 0.0;
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
            d.ratio = (d.r_d > 0.0) ? kInf : 0.0;
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
      const double target = sh.u_smp * total;
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
      if (is_bonus) {
        if (p.bonus_model >= 0) {  // the named model's one-hot law (its argmax sits in the proposer's slot)
          d.cand = qtok;
          d.prob = 1.0;
        } else {
          d.prob = r_at(d.cand);
        }
      }
    }
  }
  d.need2 = 0;  // tokens are drawn by the later stages, for the one position per row that needs it
  d.drawable = (kSample && finite) ? 1 : 0;
}

// ------------------------------------------------------------------------------------
// stage 0, one block per unit, no block barriers
// ------------------------------------------------------------------------------------
constexpr int kWaitSpins = 1 << 20;  // polls before a wait gives up (each at least 100 ns apart)

// Wait until *flag >= want.  False when the wait gave up or another warp did.
__device__ __forceinline__ bool wait_reach(const volatile int* flag, int want, const volatile int* fault, int lane) {
  int ok = 0;
  if (lane == 0) {
    for (int it = 0; it < kWaitSpins; ++it) {
      if (*flag >= want) {
        ok = 1;
        break;
      }
      if (*fault) break;
      __nanosleep(100);
    }
    __threadfence_block();
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// A wait gave up (a defect, never the data): mark every row and let the other warps of the block leave.
__device__ __noinline__ void raise_fault(const KParams& p, FreeRun& fr, int lane) {
  if (lane == 0) *reinterpret_cast<volatile int*>(&fr.fault) = 1;
  for (int b = lane; b < p.B; b += 32) atomicOr(&p.row_status[b], static_cast<unsigned>(COS_ROW_FAULT));
}

// Every warp sweeps its share of the block's current unit and moves straight on to the next one.
// The last warp to finish a unit merges the sixteen partials, takes the decision (Eq. 6) and publishes
// it while the others are already streaming; the first warp to finish draws the unit after the next
// from the work counter.  Partials are kept two units deep; a warp may run at most one unit ahead.
template <int DT, int MODE>
__device__ __forceinline__ void stage0_free_running(const KParams& p, Shared& sh) {
  constexpr bool kSample = (MODE == kEnsembleSample || MODE == kLogitSample);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  FreeRun& fr = sh.fr;
  volatile int* unit_of = fr.unit_of;
  volatile int* unit_tag = fr.unit_tag;
  volatile int* epi_done = &fr.epi_done;
  volatile int* fault = &fr.fault;
  const Slice sl = slice_of<DT>(0, 1, p.V, p.vec_ok != 0);
  if (tid == 0) {
    for (int k = 0; k < 4; ++k) {
      fr.unit_of[k] = p.num_units;
      fr.unit_tag[k] = 0;
    }
    fr.unit_of[0] = blockIdx.x;
    fr.unit_tag[0] = 1;
    fr.arrive[0] = fr.arrive[1] = 0;
    fr.left = 0;
    fr.skip_state[0] = fr.skip_state[1] = 0;
    fr.epi_done = 0;
    fr.fault = 0;
  }
  __syncthreads();
  // The inputs may be read before the kernel ahead in the stream is complete (the caller's promise): every warp then
  // sweeps the block's first unit, which is the block's own by its index, and only then waits for that kernel;
  // nothing but the inputs is touched before.  (The hint to leave positions unread is not taken together with it.)
  const bool settled = p.inputs_settled != 0;
  auto first_draw = [&]() {  // the block's first unit is valid: one draw settles its second
    const int nx = p.num_clusters + static_cast<int>(atomicAdd(p.work_counter, 1u));
    unit_of[1] = nx;
    __threadfence_block();
    unit_tag[1] = 2;
  };
  if (!settled && tid == kThreads - 32) first_draw();
  for (int seq = 0;; ++seq) {
    const int par = seq & 1;
    if (!wait_reach(&unit_tag[seq & 3], seq + 1, fault, lane)) {
      raise_fault(p, fr, lane);
      return;
    }
    const int unit = unit_of[seq & 3];
    if (unit >= p.num_units) break;
    const int j = unit / p.B, b = unit % p.B;  // earlier positions of every row come first
    const int pi = proposer_of(p, b, j);
    const bool pi_ok = (pi >= 0 && pi < p.n);
    const int pis = pi_ok ? pi : 0;
    const char* base = reinterpret_cast<const char*>(p.logits) +
                       (static_cast<long long>(b) * p.s_row + static_cast<long long>(j) * p.s_pos) * Elem<DT>::bytes;
    // the partials of this parity are free once the unit two back has been merged
    if (seq >= 2 && !wait_reach(epi_done, seq - 1, fault, lane)) {
      raise_fault(p, fr, lane);
      return;
    }
    // Early exit: a position behind a rejection that its row has already published decides nothing
    // (Sec. 3.1: the tokens after the first rejection are discarded).  The first warp to get here settles
    // it for the block, so that all sixteen do the same.  (Letting every warp look for itself during its
    // sweep was tried: the polls slowed the ordinary path by 4-6 % and gained nothing over this.)
    bool skipped = false;
    if (p.early_exit) {
      int st = 0;
      if (lane == 0) {
        const int mine = (*reinterpret_cast<volatile int*>(&p.row_reject[b]) < j) ? 2 : 1;
        st = atomicCAS(&fr.skip_state[par], 0, mine);
        if (st == 0) st = mine;
      }
      skipped = (__shfl_sync(0xffffffffu, st, 0) == 2);
    }
    if (!skipped)
      sweep_unit<DT, MODE>(p, base, sl, pis, false, -INFINITY, &fr.wsoft[par][warp][0], &fr.warg[par][warp][0]);
    if (settled && seq == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");  // from here on as in an ordinary run
      if (tid == kThreads - 32) first_draw();
    }
    int prev = 0;
    if (lane == 0) {
      __threadfence_block();
      prev = atomicAdd(&fr.arrive[par], 1);
      __threadfence_block();
    }
    prev = __shfl_sync(0xffffffffu, prev, 0);
    __syncwarp();
    if (prev == 0) {
      // first to finish: one draw per valid unit, made one unit ahead of its use
      if (!wait_reach(&unit_tag[(seq + 1) & 3], seq + 2, fault, lane)) {
        raise_fault(p, fr, lane);
        return;
      }
      if (lane == 0) {
        int nx = p.num_units;
        if (unit_of[(seq + 1) & 3] < p.num_units)
          nx = p.num_clusters + static_cast<int>(atomicAdd(p.work_counter, 1u));
        unit_of[(seq + 2) & 3] = nx;
        __threadfence_block();
        unit_tag[(seq + 2) & 3] = seq + 3;
      }
    }
    if (prev == kWarps - 1 && skipped) {
      // nothing was read: the unit reports "not accepted, no candidate", which the row's scan never reaches
      if (lane == 0) {
        const double nan = __longlong_as_double(0x7ff8000000000000LL);
        publish_unit(p, b, j, 0, 0, -1, kSample ? 0 : __float_as_int(__int_as_float(0x7fc00000)), nan, nan, nan, nan);
        fr.arrive[par] = 0;
        fr.skip_state[par] = 0;
        __threadfence_block();
        *epi_done = seq + 1;
      }
      __syncwarp();
    } else if (prev == kWarps - 1) {
      // last to finish: merge, decide, publish
      const int uidx = b * p.P + j;
      const bool is_bonus = (j == p.gamma);
      const int draft = is_bonus ? 0 : p.drafts[b * p.gamma + j];
      const bool draft_ok = is_bonus || (draft >= 0 && draft < p.V);
      if (lane < p.n && !is_bonus && draft_ok)
        sh.ldraft[lane] = Elem<DT>::load1(base + static_cast<long long>(lane) * p.s_model * Elem<DT>::bytes, draft);
      if (lane == 31) {
        unsigned rnd[4];
        const unsigned long long grow = static_cast<unsigned long long>(p.row_base + b);
        philox4x32_10(static_cast<unsigned>(grow), static_cast<unsigned>(j), offset_lo(p), offset_hi(p), p.seed_lo, p.seed_hi,
                      rnd);
        sh.u_acc = word_to_uniform(rnd[0]);
        sh.u_smp = word_to_uniform(rnd[1]);
      }
      const int nsoft = (MODE == kEnsembleSample) ? p.n : (MODE == kLogitSample ? 2 : 0);
      const int arg_lo = (MODE == kLogitGreedy) ? 1 : 0;
      const int narg = (MODE == kEnsembleGreedy) ? p.n : (MODE == kLogitGreedy ? 2 : 0);
      for (int k = 0; k < nsoft; ++k) {
        const float ref = (lane < kWarps) ? fr.wsoft[par][lane][k].ref : -INFINITY;
        const double sum = (lane < kWarps) ? fr.wsoft[par][lane][k].s : 0.0;
        const SoftPart o = warp_reduce_soft(ref, sum);
        if (lane == 0) sh.fsoft[k] = o;
      }
      for (int k = arg_lo; k < arg_lo + narg; ++k) {
        ArgPart in;
        if (lane < kWarps) {
          in = fr.warg[par][lane][k];
        } else {
          in.val = -INFINITY;
          in.idx = kNoReject;
          in.bad = 0;
        }
        const ArgPart o = warp_reduce_arg(in.val, in.idx, in.bad, lane);
        if (lane == 0) sh.farg[k] = o;
      }
      __syncwarp();
      if (MODE == kEnsembleSample && lane < p.n && !is_bonus && draft_ok) {
        // probability of the draft under model `lane`, with the constant the sweep used
        sh.pdraft[lane] = exp2(static_cast<double>(sh.ldraft[lane]) * p.cT64 - static_cast<double>(sh.fsoft[lane].ref)) /
                          sh.fsoft[lane].s;
      }
      __syncwarp();
      if (lane == 0) decide_unit<DT, MODE>(p, sh, is_bonus, draft, draft_ok, pi, pi_ok, pis, false);
      __syncwarp();
      if (kSample && lane < nsoft) {  // kept for the drawing stages
        p.ustats[uidx].s[lane] = sh.fsoft[lane].s;
        p.ustats[uidx].ref[lane] = sh.fsoft[lane].ref;
      }
      if (kSample && lane == 31) p.ustats[uidx].thr32 = 0.f;
      if (lane == 0) {
        const Decision& d = sh.dec;
        publish_unit(p, b, j, d.accept, d.status, d.cand, kSample ? d.drawable : __float_as_int(static_cast<float>(d.prob)),
                     d.ratio, d.r_d, d.q_d, d.S);
        fr.arrive[par] = 0;
        fr.skip_state[par] = 0;
        __threadfence_block();
        *epi_done = seq + 1;
      }
      __syncwarp();
    }
  }
  // the last warp of the block to run out of units reports the block's departure
  if (p.greedy && lane == 0 && atomicAdd(&fr.left, 1) == kWarps - 1) stage_exit(p, 0);
}

// ------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------
// MINB = blocks per multiprocessor the register allocation must allow (2: 64 registers, 4: 32 registers)
template <int DT, int MODE, int STAGE, int MINB = 2>
__global__ void __launch_bounds__(kThreads, MINB) cos_verify_kernel(const __grid_constant__ KParams p) {
  constexpr int E = Elem<DT>::E;
  constexpr bool kSample = (MODE == kEnsembleSample || MODE == kLogitSample);
  // the drawing stages in one sweep: stage 3 with two channel sums per step, stage 4 with one per model of an
  // ensemble of three or four
  constexpr bool kOneSweep = (STAGE == 3 || STAGE == 4);
  constexpr int NCH = (STAGE == 4) ? 4 : 2;
  cg::cluster_group cluster = cg::this_cluster();
  // stage 0 shares a unit among the blocks of a cluster; stages 1 and 2 among `parts` independent
  // blocks (they meet only through global memory: partial sums between the launches, an arrival counter within stage 2)
  const int lparts = (STAGE >= 1) ? p.parts : 1;  // blocks per unit in this launch
  const int C = (STAGE == 0) ? static_cast<int>(cluster.num_blocks()) : p.parts;
  const int rank = (STAGE == 0) ? static_cast<int>(cluster.block_rank()) : static_cast<int>(blockIdx.x % lparts);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gwarp = rank * kWarps + warp, G = C * kWarps;
  __shared__ Shared sh;
  extern __shared__ uint4 ring[];  // kWarps * kRingVecs * 32 vectors: sweep-2 staging
  int phase = 0;
  const bool vec_ok = p.vec_ok != 0;
  const bool masked = (MODE == kLogitSample || MODE == kLogitGreedy) && p.mask_model >= 0;
  const double kNaN = __longlong_as_double(0x7ff8000000000000LL);
  const double kInf = __longlong_as_double(0x7ff0000000000000LL);

  // this warp's run of steps (a step = 32 lanes x E entries)
  const int s_begin = static_cast<int>(static_cast<long long>(gwarp) * p.nsteps / G);
  const int s_end = static_cast<int>(static_cast<long long>(gwarp + 1) * p.nsteps / G);
  // this block's slice of every row in sweep 1
  const Slice sl = slice_of<DT>(rank, C, p.V, vec_ok);

  const int cluster_id = (STAGE == 0) ? blockIdx.x / C : blockIdx.x / lparts;
  // Every stage is launched while the kernel before it in the stream drains (programmatic dependent launch): its
  // blocks take their places as that kernel's blocks leave and wait here until it is complete and its writes are
  // visible.  Nothing is read or written before this point.  (Without the launch attribute, and behind a kernel
  // that never signals, this is the ordinary order of a stream.)
  // (With COS_RUN_INPUTS_SETTLED the barrier-free streaming stage reads its inputs first and waits after the sweep
  // of its first position: see stage0_free_running.)
  if (!(STAGE == 0 && p.inputs_settled)) asm volatile("griddepcontrol.wait;" ::: "memory");
  // The streaming stage of a large run and stage 1 let the next launch take places from the start (all their
  // blocks are resident or done by the time every one of them has said so; runs of a few blocks were slower with
  // the drawing stage's blocks waiting beside them); the drawing stages say so after their sweep, when most of
  // their blocks are about to leave and one per row goes on alone.
  if (STAGE == 1 || (STAGE == 0 && p.early_dependents)) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (kOneSweep) SPROF(0);
  if ((STAGE == 1 || kOneSweep) && blockIdx.x == 0 && tid == 0) *p.work_counter = 0u;  // stage 0 is over: ready for the next run
  const int job_stride = gridDim.x / lparts;
  int unit = cluster_id, emit = 0, job_it = 0, njobs = 0;
  if (STAGE == 0) {
    // One block per unit and no step that needs the whole block twice (the plausibility mask does, and so
    // does the greedy form of the combined-distribution test hook): the warps run without block barriers.
    if (C == 1 && !masked && (kSample || p.dump_r == nullptr)) {
      stage0_free_running<DT, MODE>(p, sh);
      return;
    }
  } else {
    njobs = *p.job_count;
    njobs = njobs < p.max_jobs ? njobs : p.max_jobs;
  }
  while (true) {
    int j, b;
    if (STAGE == 0) {
      if (unit >= p.num_units) break;
      j = unit / p.B;  // earlier positions of every row come first
      b = unit % p.B;
    } else {
      const int job = cluster_id + job_it * job_stride;
      if (job >= njobs) break;
      const int2 jb = p.jobs[job];
      ++job_it;
      b = jb.x / p.P;
      j = jb.x % p.P;
      emit = (p.accept_count[b] == j) ? 1 : 0;  // the token drawn here is the row's output
    }
    const int uidx = b * p.P + j;
    const int pi = proposer_of(p, b, j);
    const bool pi_ok = (pi >= 0 && pi < p.n);
    const int pis = pi_ok ? pi : 0;
    const char* base = reinterpret_cast<const char*>(p.logits) +
                       (static_cast<long long>(b) * p.s_row + static_cast<long long>(j) * p.s_pos) * Elem<DT>::bytes;
    auto row_of = [&](int i) -> const void* { return base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes; };
    const bool is_bonus = (j == p.gamma);
    const bool draw_q = is_bonus && p.bonus_model >= 0;  // the bonus token follows the named model's own law
    const int draft = is_bonus ? 0 : p.drafts[b * p.gamma + j];
    const bool draft_ok = is_bonus || (draft >= 0 && draft < p.V);

    if (STAGE == 0) {
    // ---- small jobs issued before the sweep so that their latency hides behind it
    if (tid < p.n && !is_bonus && draft_ok) sh.ldraft[tid] = Elem<DT>::load1(row_of(tid), draft);
    if (warp == kWarps - 1) {
      if (lane == 2) {
        // rank 0 draws the cluster's next unit now; every block learns it with the merged statistics
        if (rank == 0) sh.next_local = p.num_clusters + static_cast<int>(atomicAdd(p.work_counter, 1u));
      } else if (lane == 1) {
        unsigned rnd[4];
        const unsigned long long grow = static_cast<unsigned long long>(p.row_base + b);
        philox4x32_10(static_cast<unsigned>(grow), static_cast<unsigned>(j), offset_lo(p), offset_hi(p), p.seed_lo, p.seed_hi,
                      rnd);
        sh.u_acc = word_to_uniform(rnd[0]);
        sh.u_smp = word_to_uniform(rnd[1]);
      }
    }

    // ================================ sweep 1: statistics ================================
    if (MODE == kEnsembleSample) {
      sweep_unit<DT, MODE>(p, base, sl, pis, false, 0.f, &sh.wsoft[warp][0], &sh.warg[warp][0]);
      cluster_merge(sh, cluster, phase, p.n, 0, 0);
      if (tid < p.n && !is_bonus && draft_ok) {
        // probability of the draft under model tid, with the constant the sweep used
        sh.pdraft[tid] = exp2(static_cast<double>(sh.ldraft[tid]) * p.cT64 - static_cast<double>(sh.fsoft[tid].ref)) /
                         sh.fsoft[tid].s;
      }
    } else if (MODE == kEnsembleGreedy) {
      sweep_unit<DT, MODE>(p, base, sl, pis, false, 0.f, &sh.wsoft[warp][0], &sh.warg[warp][0]);
      cluster_merge(sh, cluster, phase, 0, 0, p.n);
    } else {
      // logit-level combine.  soft slot 0 = proposer, soft slot 1 = combined logits;
      // arg slot 0 = expert maximum (mask), arg slot 1 = proposer argmax, arg slot 2 = combined argmax.
      if (masked) {
        const void* row = row_of(p.mask_model);
        float best = -INFINITY;
        int bad = 0;
        for (int v = sl.v_lo + tid; v < sl.v_hi; v += kThreads) {
          float x[E];
          uint4 raw = ldg_stream16(reinterpret_cast<const char*>(row) + static_cast<long long>(v) * 16);
          Elem<DT>::unpack(raw, x);
#pragma unroll
          for (int k = 0; k < E; ++k) {
            bad |= (x[k] != x[k]);
            best = fmaxf(best, x[k]);
          }
        }
        for (int e = sl.e_lo + tid; e < sl.e_hi; e += kThreads) {
          float x = Elem<DT>::load1(row, e);
          bad |= (x != x);
          best = fmaxf(best, x);
        }
        warp_merge_arg(static_cast<double>(best), 0, bad, &sh.warg[warp][0], lane);
        cluster_merge(sh, cluster, phase, 0, 0, 1);
        if (tid == 0) {
          // l >= max + ln(alpha) in fp64 is the same as l >= (that bound rounded up to fp32) for fp32 l
          double bound = sh.farg[0].val + p.ln_alpha;
          sh.thr32 = sh.farg[0].bad ? __int_as_float(0x7fc00000) : __double2float_ru(bound);
        }
        __syncthreads();
      }
      const float thr = masked ? sh.thr32 : -INFINITY;
      if (MODE == kLogitSample) {
        sweep_unit<DT, MODE>(p, base, sl, pis, masked, thr, &sh.wsoft[warp][0], &sh.warg[warp][0]);
        cluster_merge(sh, cluster, phase, 2, 0, 0);
      } else {  // kLogitGreedy
        sweep_unit<DT, MODE>(p, base, sl, pis, masked, thr, &sh.wsoft[warp][0], &sh.warg[warp][0]);
        cluster_merge(sh, cluster, phase, 0, 1, 2);
      }
    }
    if (MODE == kEnsembleSample) __syncthreads();  // pdraft

    // ================================ decision (Eq. 6) ================================
    // every block takes the same decision from the same merged numbers
    if (tid == 0) decide_unit<DT, MODE>(p, sh, is_bonus, draft, draft_ok, pi, pi_ok, pis, masked);
    __syncthreads();
    // rank 0 keeps the merged statistics for the drawing stages and reports the unit
    if (rank == 0) {
      const int nkeep = (MODE == kEnsembleSample) ? p.n : (MODE == kLogitSample ? 2 : 0);
      if (tid < nkeep) {
        p.ustats[uidx].s[tid] = sh.fsoft[tid].s;
        p.ustats[uidx].ref[tid] = sh.fsoft[tid].ref;
      }
      if (tid == 32 && nkeep > 0) p.ustats[uidx].thr32 = masked ? sh.thr32 : 0.f;
    }
    } else {
      // stage 1: the statistics of this unit were merged by stage 0
      const int nkeep = (MODE == kEnsembleSample) ? p.n : 2;
      if (tid < nkeep) {
        sh.fsoft[tid].s = p.ustats[uidx].s[tid];
        sh.fsoft[tid].ref = p.ustats[uidx].ref[tid];
        sh.big_thr[tid] = static_cast<float>(sh.fsoft[tid].s * kBigShare);  // from the first estimate, in every stage
        if (STAGE == 2) {
          double z = 0.0;
          for (int q = 0; q < p.parts; ++q) z += p.zpart[(static_cast<size_t>(uidx) * p.parts + q) * 8 + tid];
          sh.fsoft[tid].s = z;
        }
      }
      if (tid == 32) {
        const int4 ur = __ldcg(&p.unit_res[uidx]);
        Decision& d = sh.dec;
        d.accept = ur.x;
        d.status = ur.y;
        d.want_sample = 1;
        d.cand = -1;
        d.natoms = 0;
        d.need2 = 1;
        d.drawable = 1;
        d.ratio = d.r_d = d.q_d = d.S = kNaN;
        sh.thr32 = p.ustats[uidx].thr32;
        unsigned rnd[4];
        const unsigned long long grow = static_cast<unsigned long long>(p.row_base + b);
        philox4x32_10(static_cast<unsigned>(grow), static_cast<unsigned>(j), offset_lo(p), offset_hi(p), p.seed_lo, p.seed_hi,
                      rnd);
        sh.u_smp = word_to_uniform(rnd[1]);
        sh.next = 0;
      }
      __syncthreads();
    }
    const int need2 = sh.dec.need2;
    const int next_unit = sh.next;

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
    if (kSample && need2) {
      const float thr = masked ? sh.thr32 : -INFINITY;
      const int nsoft2 = (MODE == kEnsembleSample) ? p.n : 2;

      // ---- 2a: normalisers again, now that the references are known: terms holding more
      // than 2^-8 of a normaliser are evaluated in fp64 and kept out of the fp32 sums, so
      // a dominant token neither absorbs the small ones nor carries the fast exp's error
      if (STAGE == 1) {
      if (MODE == kEnsembleSample) {
        for (int i = 0; i < p.n; ++i) {
          const void* row = row_of(i);
          const char* rowb = reinterpret_cast<const char*>(row);
          const float nref = -sh.fsoft[i].ref, bt = sh.big_thr[i];
          const double dref = static_cast<double>(sh.fsoft[i].ref);
          float zs = 0.f;
          double zb = 0.0;
          auto eat = [&](const float (&v)[E]) {
            float e[E];
            bool any = false;
#pragma unroll
            for (int k = 0; k < E; ++k) {
              e[k] = ex2_approx(fmaf(v[k], p.cT, nref));
              const bool big = e[k] > bt;
              any |= big;
              zs += big ? 0.f : e[k];
            }
            if (any) {
#pragma unroll
              for (int k = 0; k < E; ++k)
                if (e[k] > bt) zb += exp2(static_cast<double>(v[k]) * p.cT64 - dref);
            }
          };
          int v = sl.v_lo + tid;
          for (; v + 3 * kThreads < sl.v_hi; v += 4 * kThreads) {
            uint4 raw[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) raw[u] = ldg_stream16(rowb + static_cast<long long>(v + u * kThreads) * 16);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              float x[E];
              Elem<DT>::unpack(raw[u], x);
              eat(x);
            }
          }
          for (; v < sl.v_hi; v += kThreads) {
            float x[E];
            uint4 raw = ldg_stream16(rowb + static_cast<long long>(v) * 16);
            Elem<DT>::unpack(raw, x);
            eat(x);
          }
          for (int e = sl.e_lo + tid; e < sl.e_hi; e += kThreads) {
            const float x = Elem<DT>::load1(row, e);
            const float ee = ex2_approx(fmaf(x, p.cT, nref));
            if (ee > bt)
              zb += exp2(static_cast<double>(x) * p.cT64 - dref);
            else
              zs += ee;
          }
          double t = static_cast<double>(zs) + zb;
#pragma unroll
          for (int d = 16; d > 0; d >>= 1) t += shfl_double(t, lane ^ d);
          if (lane == 0) {
            sh.wsoft[warp][i].s = t;
            sh.wsoft[warp][i].ref = sh.fsoft[i].ref;
          }
        }
      } else {
        const float nref_q = -sh.fsoft[0].ref, nref_c = -sh.fsoft[1].ref;
        const float bt_q = sh.big_thr[0], bt_c = sh.big_thr[1];
        const double dref_q = static_cast<double>(sh.fsoft[0].ref), dref_c = static_cast<double>(sh.fsoft[1].ref);
        float zsq = 0.f, zsc = 0.f;
        double zbq = 0.0, zbc = 0.0;
        auto big_c = [&](int e) {  // combined logit of one token in fp64
          double cd = 0.0;
          for (int i = 0; i < p.n; ++i) cd = fma(p.w64[i], static_cast<double>(Elem<DT>::load1(row_of(i), e)), cd);
          return exp2(cd * p.cT64 - dref_c);
        };
        // the vectors of the first two models are fetched one trip ahead: four loads in flight per thread
        const char* row0 = reinterpret_cast<const char*>(row_of(0));
        const long long row_step = p.s_model * Elem<DT>::bytes;
        const bool pair = (p.n >= 2);
        uint4 nx0 = make_uint4(0u, 0u, 0u, 0u), nx1 = nx0;
        {
          const int v0 = sl.v_lo + tid;
          if (v0 < sl.v_hi) {
            nx0 = ldg_stream16(row0 + static_cast<long long>(v0) * 16);
            if (pair) nx1 = ldg_stream16(row0 + row_step + static_cast<long long>(v0) * 16);
          }
        }
        for (int v = sl.v_lo + tid; v < sl.v_hi; v += kThreads) {
          const uint4 a0 = nx0, a1 = nx1;
          {
            const int vn = v + kThreads;
            if (vn < sl.v_hi) {
              nx0 = ldg_stream16(row0 + static_cast<long long>(vn) * 16);
              if (pair) nx1 = ldg_stream16(row0 + row_step + static_cast<long long>(vn) * 16);
            }
          }
          float cmb[E], vq[E], ve[E];
#pragma unroll
          for (int k = 0; k < E; ++k) {
            cmb[k] = 0.f;
            vq[k] = -INFINITY;
            ve[k] = 0.f;
          }
          auto take = [&](int i, const uint4& raw) {
            float x[E];
            Elem<DT>::unpack(raw, x);
            const float wi = p.w[i];
#pragma unroll
            for (int k = 0; k < E; ++k) {
              cmb[k] = fmaf(wi, x[k], cmb[k]);
              if (i == pis) vq[k] = x[k];
              if (i == p.mask_model) ve[k] = x[k];
            }
          };
          take(0, a0);
          if (pair) take(1, a1);
          for (int i = 2; i < p.n; ++i) take(i, ldg_stream16(row0 + i * row_step + static_cast<long long>(v) * 16));
          bool any = false;
          float eq[E], ec[E];
#pragma unroll
          for (int k = 0; k < E; ++k) {
            const bool in = !masked || ve[k] >= thr;
            eq[k] = ex2_approx(fmaf(vq[k], p.cT, nref_q));
            ec[k] = in ? ex2_approx(fmaf(cmb[k], p.cT, nref_c)) : 0.f;
            const bool bq = eq[k] > bt_q, bc = ec[k] > bt_c;
            any |= bq | bc;
            zsq += bq ? 0.f : eq[k];
            zsc += bc ? 0.f : ec[k];
          }
          if (any) {
#pragma unroll
            for (int k = 0; k < E; ++k) {
              if (eq[k] > bt_q) zbq += exp2(static_cast<double>(vq[k]) * p.cT64 - dref_q);
              if (ec[k] > bt_c) zbc += big_c(v * E + k);
            }
          }
        }
        for (int e = sl.e_lo + tid; e < sl.e_hi; e += kThreads) {
          float cmb = 0.f, xq = -INFINITY, xe = 0.f;
          for (int i = 0; i < p.n; ++i) {
            float x = Elem<DT>::load1(row_of(i), e);
            cmb = fmaf(p.w[i], x, cmb);
            if (i == pis) xq = x;
            if (i == p.mask_model) xe = x;
          }
          const bool in = !masked || xe >= thr;
          const float eq = ex2_approx(fmaf(xq, p.cT, nref_q));
          const float ec = in ? ex2_approx(fmaf(cmb, p.cT, nref_c)) : 0.f;
          if (eq > bt_q)
            zbq += exp2(static_cast<double>(xq) * p.cT64 - dref_q);
          else
            zsq += eq;
          if (ec > bt_c)
            zbc += big_c(e);
          else
            zsc += ec;
        }
        double tq = static_cast<double>(zsq) + zbq, tc = static_cast<double>(zsc) + zbc;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
          tq += shfl_double(tq, lane ^ d);
          tc += shfl_double(tc, lane ^ d);
        }
        if (lane == 0) {
          sh.wsoft[warp][0].s = tq;
          sh.wsoft[warp][0].ref = sh.fsoft[0].ref;
          sh.wsoft[warp][1].s = tc;
          sh.wsoft[warp][1].ref = sh.fsoft[1].ref;
        }
      }
      // this block's share of every normaliser goes to global memory; stage 2 adds the shares up
      __syncthreads();
      if (warp < nsoft2) {
        float ref = (lane < kWarps) ? sh.wsoft[lane][warp].ref : -INFINITY;
        double sum = (lane < kWarps) ? sh.wsoft[lane][warp].s : 0.0;
        SoftPart o = warp_reduce_soft(ref, sum);
        if (lane == 0) p.zpart[(static_cast<size_t>(uidx) * p.parts + rank) * 8 + warp] = o.s;
      }
      } else {
      bool do_locate = false;
      if (kOneSweep) {
        SPROF(1);
        double kc[4] = {0.0, 0.0, 0.0, 0.0};  // coefficient of every channel in what is drawn
        if (STAGE == 4) {
          one_sweep_channels<DT>(p, sh, ring, base, b, rank, lparts, pis, is_bonus, draw_q, emit, vec_ok, kc);
        } else {
          one_sweep_pair<DT, MODE>(p, sh, ring, base, b, rank, lparts, pis, masked, thr, is_bonus, draw_q, emit, vec_ok, kc);
        }
        __syncthreads();
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        SPROF(2);
        if (warp < NCH) {
          float ref = (lane < kWarps) ? sh.wsoft[lane][warp].ref : -INFINITY;
          double sum = (lane < kWarps) ? sh.wsoft[lane][warp].s : 0.0;
          SoftPart o = warp_reduce_soft(ref, sum);
          if (lane == 0) p.zpart[(static_cast<size_t>(uidx) * p.parts + rank) * 8 + warp] = o.s;
        }
        // the last block of the unit to get here completes the normalisers and locates the token
        __syncthreads();
        if (tid == 0) {
          __threadfence();
          const int prev = atomicAdd(&p.part_arrivals[uidx], 1);
          sh.win_g = (prev == p.parts - 1) ? 1 : 0;
          if (prev == p.parts - 1) {
            __threadfence();            // what the other blocks wrote before they arrived is visible from here on
            p.part_arrivals[uidx] = 0;  // ready for the next run (a later launch: nothing waits for this store)
          }
        }
        __syncthreads();
        do_locate = (sh.win_g != 0) && emit;  // (every unit listed for this stage is its row's drawing unit)
        __syncthreads();
        SPROF(3);
        if (do_locate) {
          if (tid < NCH) {
            double z = 0.0;
            for (int q = 0; q < p.parts; ++q) z += __ldcg(&p.zpart[(static_cast<size_t>(uidx) * p.parts + q) * 8 + tid]);
            double kmine = kc[0];
#pragma unroll
            for (int i = 1; i < NCH; ++i) kmine = (tid == i) ? kc[i] : kmine;
            const bool live = (STAGE != 4) || tid < p.n;  // an ensemble of three leaves the fourth channel empty
            if (live) sh.fsoft[tid].s = z;
            one_sweep_coef(sh)[tid] = live ? kmine / z : 0.0;
          }
          __syncthreads();
          SPROF(4);
        }
      }
      if (!kOneSweep || do_locate) {
      if (MODE == kEnsembleSample && tid < p.n) {
        // r - q = sum_i (w_i/Z_i - [i = proposer]/Z_i) e_i, and r = sum_i (w_i/Z_i) e_i
        const double a = p.w64[tid] / sh.fsoft[tid].s;
        sh.a_scale[tid] = static_cast<float>(a);
        sh.a_resid[tid] = static_cast<float>(a - (tid == pis ? 1.0 / sh.fsoft[tid].s : 0.0));
        sh.a_draw[tid] = draw_q ? static_cast<float>(tid == pis ? 1.0 / sh.fsoft[tid].s : 0.0) : sh.a_scale[tid];
        sh.a_ref[tid] = -sh.fsoft[tid].ref;
      }
      __syncthreads();
      const float inv_zq = (MODE == kLogitSample) ? static_cast<float>(1.0 / sh.fsoft[0].s) : 0.f;
      const float ref_q = (MODE == kLogitSample) ? -sh.fsoft[0].ref : 0.f;
      const float inv_zc = (MODE == kLogitSample) ? static_cast<float>(1.0 / sh.fsoft[1].s) : 0.f;
      const float ref_c = (MODE == kLogitSample) ? -sh.fsoft[1].ref : 0.f;

      // ---- 2b: token masses.  mass32[k] is max(0, r - q) (or r) of the lane's k-th token in fp32;
      // tokens holding more than 2^-8 of any normaliser are flagged in `bigbits`, get mass32 = 0
      // and are evaluated by big_mass() in fp64 from the stored logits.
      // `staged` points at this lane's staged vector of model 0 (models 32 vectors apart), or is null.
      auto chunk_mass = [&](int e0, bool use_r, float (&mass32)[E], unsigned& bigbits, const uint4* staged) {
        auto fetch = [&](int i, float (&v)[E]) {
          if (staged != nullptr) {
            uint4 raw = staged[i * 32];
            Elem<DT>::unpack(raw, v);
          } else {
            load_chunk<DT>(row_of(i), e0, p.V, vec_ok, v);  // entries beyond V read as -inf: mass 0
          }
        };
        float acc[E], rr[E];
        bool anybig = false;
        bigbits = 0u;
        const float* coef = use_r ? sh.a_draw : sh.a_resid;
        const bool from_q = use_r && draw_q;
#pragma unroll
        for (int k = 0; k < E; ++k) {
          acc[k] = 0.f;
          rr[k] = 0.f;
        }
        if (MODE == kEnsembleSample) {
          for (int i = 0; i < p.n; ++i) {
            float v[E];
            fetch(i, v);
            const float co = coef[i], rf = sh.a_ref[i];
            float emax = 0.f;
#pragma unroll
            for (int k = 0; k < E; ++k) {
              const float e = ex2_approx(fmaf(v[k], p.cT, rf));
              emax = fmaxf(emax, e);
              // products rounded one by one (no fused multiply-add): when r and q coincide the terms
              // cancel exactly, as they do in exact arithmetic
              acc[k] = __fadd_rn(acc[k], __fmul_rn(co, e));
            }
            anybig |= emax > sh.big_thr[i];
          }
        } else {
          float cmb[E], ve[E], eq[E];
#pragma unroll
          for (int k = 0; k < E; ++k) {
            cmb[k] = 0.f;
            ve[k] = 0.f;
            eq[k] = 0.f;
          }
          for (int i = 0; i < p.n; ++i) {
            float v[E];
            fetch(i, v);
            const float wi = p.w[i];
#pragma unroll
            for (int k = 0; k < E; ++k) {
              cmb[k] = fmaf(wi, v[k], cmb[k]);
              if (i == p.mask_model) ve[k] = v[k];
              if (i == pis) eq[k] = ex2_approx(fmaf(v[k], p.cT, ref_q));
            }
          }
          const float qco = use_r ? 0.f : inv_zq;
          const bool tail = (staged == nullptr);
          float emq = 0.f, emc = 0.f;
#pragma unroll
          for (int k = 0; k < E; ++k) {
            bool in = !masked || ve[k] >= thr;
            if (tail) in = in && (e0 + k < p.V);
            const float ec = in ? ex2_approx(fmaf(cmb[k], p.cT, ref_c)) : 0.f;
            emc = fmaxf(emc, ec);
            emq = fmaxf(emq, eq[k]);
            rr[k] = ec * inv_zc;
            // rounded product: r == q cancels exactly
            acc[k] = from_q ? __fmul_rn(eq[k], inv_zq) : __fsub_rn(rr[k], __fmul_rn(eq[k], qco));
          }
          anybig = (emc > sh.big_thr[1]) || (emq > sh.big_thr[0]);
        }
#pragma unroll
        for (int k = 0; k < E; ++k) mass32[k] = fmaxf(0.f, acc[k]);  // r - q clipped at zero; r itself is never negative
        if (anybig) {
          // rare: find which tokens are big under some distribution; big_mass evaluates those in fp64
          if (MODE == kEnsembleSample) {
            for (int i = 0; i < p.n; ++i) {
              float v[E];
              fetch(i, v);
              const float rf = sh.a_ref[i], bt = sh.big_thr[i];
#pragma unroll
              for (int k = 0; k < E; ++k) bigbits |= (ex2_approx(fmaf(v[k], p.cT, rf)) > bt) ? (1u << k) : 0u;
            }
          } else {
            const float zc = static_cast<float>(sh.fsoft[1].s);
#pragma unroll
            for (int k = 0; k < E; ++k) {
              const float ec = rr[k] * zc;  // rr = ec / Z_c
              const bool inside = (e0 + k < p.V);
              const float lq = Elem<DT>::load1(row_of(pis), inside ? e0 + k : p.V - 1);
              const float eqk = inside ? ex2_approx(fmaf(lq, p.cT, ref_q)) : 0.f;
              bigbits |= (ec > sh.big_thr[1] || eqk > sh.big_thr[0]) ? (1u << k) : 0u;
            }
          }
#pragma unroll
          for (int k = 0; k < E; ++k)
            if (bigbits & (1u << k)) mass32[k] = 0.f;
        }
      };
      auto big_mass = [&](int e, bool use_r, const uint4* staged, int k) -> double {
        const int draw = use_r ? (draw_q ? kDrawQ : kDrawR) : kDrawResidual;
        return big_token_mass<DT, MODE>(p, sh.fsoft, base, e, draw, staged, k, masked, thr, pis);
      };
      // a lane's mass of one step: fp32 sum of the small tokens in token order plus the big ones in fp64
      auto lane_mass = [&](int e0, const float (&mass32)[E], unsigned bigbits, bool use_r, const uint4* staged) -> double {
        float ls = 0.f;
#pragma unroll
        for (int k = 0; k < E; ++k) ls += mass32[k];
        double own = static_cast<double>(ls);
        while (bigbits) {  // big tokens in token order
          const int k = __ffs(bigbits) - 1;
          bigbits &= bigbits - 1;
          own += big_mass(e0 + k, use_r, staged, k);
        }
        return own;
      };

      uint4* myring = ring + static_cast<size_t>(warp) * kRingVecs * 32 + lane;
      // Mass of one warp run [sb, se) in token order; the running total after every gszv steps goes to
      // rec[] (lane 0 writes; rec may be null).  Vectors of the coming steps are staged in shared memory
      // with cp.async so that a warp keeps several loads in flight although it consumes its run in order.
      auto run_totals = [&](int sb, int se, int gszv, bool use_r, double* rec) -> double {
        double wrun = 0.0;  // the run's total, accumulated group by group
        double lacc = 0.0;  // this lane's mass within the current group
        const int depth = (p.n <= 2) ? 4 : (p.n <= 4 ? 2 : 1);
        const int nfull = vec_ok ? p.V / (32 * E) : 0;
        const int fe = (se < nfull) ? se : nfull;  // steps [sb, fe) go through the ring
        const char* row0 = reinterpret_cast<const char*>(row_of(0));
        const long long row_step = p.s_model * Elem<DT>::bytes;
        auto stage_in = [&](int s, int to_slot) {  // issue the loads of step s into a ring slot
          const char* src = row0 + static_cast<long long>(s * 32 + lane) * 16;
          uint4* dst = &myring[to_slot * p.n * 32];
          for (int i = 0; i < p.n; ++i) cp_async16(dst + i * 32, src + i * row_step);
        };
        int fill = 0;  // ring slot the next staged step goes to
        for (int t = 0; t < depth; ++t) {
          if (sb + t < fe) stage_in(sb + t, fill);
          fill = (fill + 1 == depth) ? 0 : fill + 1;
          cp_async_commit();
        }
        int slot = 0, in_group = 0, grp = 0;
        for (int s = sb; s < se; ++s) {
          float mass32[E];
          unsigned bigbits;
          const int e0 = (s * 32 + lane) * E;
          if (s < fe) {
            if (depth == 4)
              cp_async_wait<3>();
            else if (depth == 2)
              cp_async_wait<1>();
            else
              cp_async_wait<0>();
            chunk_mass(e0, use_r, mass32, bigbits, &myring[slot * p.n * 32]);
            lacc += lane_mass(e0, mass32, bigbits, use_r, &myring[slot * p.n * 32]);
            if (s + depth < fe) stage_in(s + depth, slot);
            slot = (slot + 1 == depth) ? 0 : slot + 1;
            cp_async_commit();
          } else {
            chunk_mass(e0, use_r, mass32, bigbits, nullptr);
            lacc += lane_mass(e0, mass32, bigbits, use_r, nullptr);
          }
          if (++in_group == gszv || s + 1 == se) {
            double t = lacc;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) t += shfl_double(t, lane ^ d);
            wrun += t;
            if (lane == 0 && rec != nullptr) rec[grp] = wrun;
            ++grp;
            in_group = 0;
            lacc = 0.0;
          }
        }
        cp_async_wait<0>();
        return wrun;
      };
      // One warp finds the token inside the run [sb, se): `base` is the mass before the run, rec[] its
      // recorded running totals.  It picks the group of steps from rec[], walks that group again step
      // by step with an fp64 prefix over the lanes, then walks the lane's tokens.
      auto walk = [&](int sb, int se, int gszv, double base, const double* rec, double target, bool use_r) -> int {
        const int ngrp = (se - sb + gszv - 1) / gszv;
        int grp = -1;
        for (int g0 = 0; g0 < ngrp && grp < 0; g0 += 32) {
          const int g = g0 + lane;
          const double cur = (g < ngrp) ? rec[g] : 0.0;
          const double prev = (g > 0 && g < ngrp) ? rec[g - 1] : 0.0;
          const bool ok = (g < ngrp) && (cur > prev) && (base + cur >= target);
          const unsigned m = __ballot_sync(0xffffffffu, ok);
          if (m) grp = g0 + __ffs(m) - 1;
        }
        if (grp < 0) {  // rounding corner: last group with mass
          for (int g = ngrp - 1; g >= 0 && grp < 0; --g)
            if (rec[g] > (g > 0 ? rec[g - 1] : 0.0)) grp = g;
          if (grp < 0) grp = 0;
        }
        double R = (grp > 0) ? rec[grp - 1] : 0.0;
        int token = -1, last_pos = -1;
        const int rs_begin = sb + grp * gszv;
        const int rs_end = (rs_begin + gszv < se) ? rs_begin + gszv : se;
        const int wfull = vec_ok ? p.V / (32 * E) : 0;  // steps below this are whole aligned vectors
        for (int s = rs_begin; s < rs_end && token < 0; ++s) {
          float mass32[E];
          unsigned bigbits;
          const int e0 = (s * 32 + lane) * E;
          // the lane's vectors of the step go through its slots of the staging ring (idle by now), so that the big
          // tokens, which are evaluated one by one, find their logits there instead of in global memory.  (Ensembles
          // only: at logit level the same made the whole stage 4 % slower on the largest workload; the compiler's
          // register allocation for the sweep changes with it.)
          const uint4* st = nullptr;
          if (MODE == kEnsembleSample && s < wfull && p.n <= kRingVecs) {
            const char* src = reinterpret_cast<const char*>(row_of(0)) + static_cast<long long>(s * 32 + lane) * 16;
            for (int i = 0; i < p.n; ++i) myring[i * 32] = ldg_stream16(src + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes);
            st = myring;
          }
          chunk_mass(e0, use_r, mass32, bigbits, st);
          if (kOneSweep) SPROF(7);
          // per-token masses of this lane in fp64 (big tokens from their fp64 evaluation)
          double m64[E];
#pragma unroll
          for (int k = 0; k < E; ++k) m64[k] = static_cast<double>(mass32[k]);
          if (bigbits) {
#pragma unroll
            for (int k = 0; k < E; ++k)
              if (bigbits & (1u << k)) m64[k] = big_mass(e0 + k, use_r, st, k);
          }
          // the lane's mass exactly as lane_mass() forms it (fp32 sum of the small tokens, then the big ones
          // in token order), from the values already at hand
          float ls = 0.f;
#pragma unroll
          for (int k = 0; k < E; ++k) ls += mass32[k];
          double own = static_cast<double>(ls);
          if (bigbits) {
#pragma unroll
            for (int k = 0; k < E; ++k)
              if (bigbits & (1u << k)) own += m64[k];
          }
          double inc = own;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            double o = shfl_up_double(inc, d);
            if (lane >= d) inc += o;
          }
          double excl = shfl_up_double(inc, 1);
          if (lane == 0) excl = 0.0;
          const double incl = excl + own;
          const double step_total = shfl_double(incl, 31);
          const bool hit = (own > 0.0) && (base + (R + incl) >= target);
          unsigned hits = __ballot_sync(0xffffffffu, hit);
          unsigned pos_lanes = __ballot_sync(0xffffffffu, own > 0.0);
          const bool last_chance = (s + 1 == rs_end);
          if (hits != 0u || (last_chance && pos_lanes != 0u)) {
            int src = hits ? (__ffs(hits) - 1) : (31 - __clz(pos_lanes));
            int found = -1;
            if (lane == src) {
              double part = 0.0;
              int lastk = -1;
#pragma unroll
              for (int k = 0; k < E; ++k) {
                part += m64[k];
                if (m64[k] > 0.0) {
                  lastk = k;
                  if (found < 0 && base + (R + (excl + part)) >= target) found = e0 + k;
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
              if (m64[k] > 0.0) lp = e0 + k;
            last_pos = __shfl_sync(0xffffffffu, lp, src);
          }
          R += step_total;
        }
        return (token < 0) ? last_pos : token;
      };
      // sequential sums over the runs in token order: picks the first run whose inclusive sum reaches
      // u * S and has mass; thread 0 only.  Results in sh.dec.S, sh.target, sh.base, sh.win_g (-1: no mass).
      auto pick_run = [&](const double* tot, int count) {
        double S = 0.0;
        for (int g = 0; g < count; ++g) S += tot[g];
        const double target = sh.u_smp * S;
        double run = 0.0, wbase = 0.0;
        int win = -1;
        for (int g = 0; g < count && win < 0; ++g) {
          if (tot[g] > 0.0 && run + tot[g] >= target) {
            win = g;
            wbase = run;
          }
          run += tot[g];
        }
        if (win < 0 && S > 0.0) {  // rounding corner: last run with mass
          run = 0.0;
          for (int g = 0; g < count; ++g) {
            if (tot[g] > 0.0) {
              win = g;
              wbase = run;
            }
            run += tot[g];
          }
        }
        sh.dec.S = S;
        sh.target = target;
        sh.base = wbase;
        sh.win_g = (S > 0.0) ? win : -1;
      };
      auto run_gsz = [&](int nst, int nrec) { return (nst + nrec - 1) / nrec > 1 ? (nst + nrec - 1) / nrec : 1; };

      if (STAGE == 2) {
        // ---- masses of this block's runs, to be added up and searched by the last block of the unit
        const int gszv = run_gsz(s_end - s_begin, kRecG);
        double* rec = emit ? p.srung + (static_cast<size_t>(b) * G + gwarp) * kRecG : nullptr;
        if (p.dump_r != nullptr) {
          // test hook: the combined distribution of this block's runs, token by token
          float* out = p.dump_r + (static_cast<long long>(b) * p.P + j) * p.V;
          for (int s = s_begin; s < s_end; ++s) {
            const int e0 = (s * 32 + lane) * E;
            float r[E];
#pragma unroll
            for (int k = 0; k < E; ++k) r[k] = 0.f;
            if (MODE == kEnsembleSample) {
              for (int i = 0; i < p.n; ++i) {
                float v[E];
                load_chunk<DT>(row_of(i), e0, p.V, vec_ok, v);
#pragma unroll
                for (int k = 0; k < E; ++k) r[k] = fmaf(sh.a_scale[i], ex2_approx(fmaf(v[k], p.cT, sh.a_ref[i])), r[k]);
              }
            } else {
              float cmb[E], ve[E];
#pragma unroll
              for (int k = 0; k < E; ++k) cmb[k] = ve[k] = 0.f;
              for (int i = 0; i < p.n; ++i) {
                float v[E];
                load_chunk<DT>(row_of(i), e0, p.V, vec_ok, v);
#pragma unroll
                for (int k = 0; k < E; ++k) {
                  cmb[k] = fmaf(p.w[i], v[k], cmb[k]);
                  if (i == p.mask_model) ve[k] = v[k];
                }
              }
#pragma unroll
              for (int k = 0; k < E; ++k)
                r[k] = (!masked || ve[k] >= thr) ? ex2_approx(fmaf(cmb[k], p.cT, ref_c)) * inv_zc : 0.f;
            }
#pragma unroll
            for (int k = 0; k < E; ++k)
              if (e0 + k < p.V) out[e0 + k] = r[k];
          }
        }
        const double t = run_totals(s_begin, s_end, gszv, is_bonus, rec);
        if (lane == 0) p.wtotg[static_cast<size_t>(uidx) * G + gwarp] = t;
        // the last block of the unit to get here goes on to locate the token (fence + counter, no waiting)
        __syncthreads();
        if (tid == 0) {
          __threadfence();
          const int prev = atomicAdd(&p.part_arrivals[uidx], 1);
          sh.win_g = (prev == p.parts - 1) ? 1 : 0;
          if (prev == p.parts - 1) {
            __threadfence();            // what the other blocks wrote before they arrived is visible from here on
            p.part_arrivals[uidx] = 0;  // ready for the next run (a later launch: nothing waits for this store)
          }
        }
        __syncthreads();
        do_locate = (sh.win_g != 0);
        __syncthreads();
      }
      if (do_locate) {
        // ---- one block per unit: add the runs up, find the run, walk it
        int one_step = -1;  // one-sweep stage: the step that holds the token
        if (kOneSweep) {
          // Every step's channel sums turn into its mass now that the normalisers are complete (products rounded
          // one by one, so that equal sums under opposite coefficients cancel exactly).  Threads own consecutive
          // steps; a prefix over threads in step order gives S and the first step whose running total reaches u S.
          const int per = (p.nsteps + kThreads - 1) / kThreads;
          const int lo = tid * per, hi = (lo + per < p.nsteps) ? lo + per : p.nsteps;
          const double* ra = p.srung + static_cast<size_t>(b) * p.nsteps;
          const double* rb = p.srungB + static_cast<size_t>(b) * p.nsteps;
          const double* rc = (STAGE == 4) ? p.srungC + static_cast<size_t>(b) * p.nsteps : nullptr;
          const double* rd = (STAGE == 4) ? p.srungD + static_cast<size_t>(b) * p.nsteps : nullptr;
          auto step_mass = [&](int st) {
            double acc = __dadd_rn(__dmul_rn(one_sweep_coef(sh)[0], __ldcg(ra + st)), __dmul_rn(one_sweep_coef(sh)[1], __ldcg(rb + st)));
            if (STAGE == 4) {
              acc = __dadd_rn(acc, __dmul_rn(one_sweep_coef(sh)[2], __ldcg(rc + st)));
              acc = __dadd_rn(acc, __dmul_rn(one_sweep_coef(sh)[3], __ldcg(rd + st)));
            }
            return fmax(0.0, acc);
          };
          // (the masses of a thread's first four steps stay in registers for the second pass)
          double mkeep[4] = {0.0, 0.0, 0.0, 0.0};
          double mine = 0.0;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (lo + q < hi) {
              mkeep[q] = step_mass(lo + q);
              mine += mkeep[q];
            }
          }
          for (int st = lo + 4; st < hi; ++st) mine += step_mass(st);
          double incl = mine;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            const double o = shfl_up_double(incl, d);
            if (lane >= d) incl += o;
          }
          if (lane == 31) sh.wtot[warp] = incl;
          if (tid == 0) {
            sh.win_g = 0x7fffffff;
            sh.win_rank = -1;
          }
          __syncthreads();
          if (tid == 0) {
            double run = 0.0;
            for (int w2 = 0; w2 < kWarps; ++w2) {
              sh.wincl[w2] = run;  // mass before the warp's steps
              run += sh.wtot[w2];
            }
            sh.dec.S = run;
            sh.target = sh.u_smp * run;
          }
          __syncthreads();
          const double target = sh.target;
          double before = sh.wincl[warp] + (incl - mine);
          int first = 0x7fffffff, last = -1;
          double first_base = 0.0, first_m = 0.0, last_base = 0.0, last_m = 0.0;
          auto look = [&](int st, double m) {
            if (m > 0.0) {
              last = st;
              last_base = before;
              last_m = m;
              if (first == 0x7fffffff && before + m >= target) {
                first = st;
                first_base = before;
                first_m = m;
              }
            }
            before += m;
          };
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (lo + q < hi) look(lo + q, mkeep[q]);
          for (int st = lo + 4; st < hi; ++st) look(st, step_mass(st));
          if (first != 0x7fffffff) atomicMin(&sh.win_g, first);
          if (last >= 0) atomicMax(&sh.win_rank, last);  // rounding corner: the last step with mass
          __syncthreads();
          const int wfirst = sh.win_g, wlast = sh.win_rank;
          __syncthreads();
          if (wfirst != 0x7fffffff) {
            if (first == wfirst) {
              sh.base = first_base;
              sh.srun[0][0] = first_m;
            }
            one_step = wfirst;
          } else if (wlast >= 0 && sh.dec.S > 0.0) {
            if (last == wlast) {
              sh.base = last_base;
              sh.srun[0][0] = last_m;
            }
            one_step = wlast;
          }
          if (tid == 0) sh.win_g = (one_step >= 0) ? 0 : -1;
          SPROF(5);
        } else {
          for (int g = tid; g < G; g += kThreads) sh.gw[g] = __ldcg(&p.wtotg[static_cast<size_t>(uidx) * G + g]);
          __syncthreads();
          if (tid == 0) pick_run(sh.gw, G);
        }
        __syncthreads();
        // the residual mass S (Eq. 7: 1 - alpha) is reported wherever it was computed
        if (tid == 0 && p.diag) p.diag[static_cast<long long>(uidx) * 4 + 3] = is_bonus ? __int_as_float(0x7fc00000) : static_cast<float>(sh.dec.S);
        if (sh.win_g >= 0) {
          if (emit && warp == 0) {
            const int g = sh.win_g;
            // one-sweep stage: the run is the one step found above, its mass the only running total
            const int sb = kOneSweep ? one_step : static_cast<int>(static_cast<long long>(g) * p.nsteps / G);
            const int se = kOneSweep ? one_step + 1 : static_cast<int>(static_cast<long long>(g + 1) * p.nsteps / G);
            const int gsz = run_gsz(se - sb, kRecG);
            const double* rec = kOneSweep ? &sh.srun[0][0] : p.srung + (static_cast<size_t>(b) * G + g) * kRecG;
            const int token = walk(sb, se, gsz, sh.base, rec, sh.target, is_bonus);
            if (lane == 0) {
              p.out_tokens[uidx] = token;  // the row's token at its first rejection, or the bonus
              // Algorithm 2's Score returns the bonus token with its probability under the law it came from
              if (is_bonus && p.bonus_prob != nullptr && token >= 0)
                p.bonus_prob[b] = static_cast<float>(big_mass(token, true, nullptr, 0));
            }
            SPROF(6);
          }
        } else if (!is_bonus && emit) {
          // no residual mass although a token is needed: this block draws from r instead, over the whole
          // vocabulary (sixteen runs, totals in shared memory)
          const int sb = static_cast<int>(static_cast<long long>(warp) * p.nsteps / kWarps);
          const int se = static_cast<int>(static_cast<long long>(warp + 1) * p.nsteps / kWarps);
          const int gszv = run_gsz(se - sb, kRec);
          const double t = run_totals(sb, se, gszv, true, &sh.srun[warp][0]);
          if (lane == 0) sh.wtot[warp] = t;
          __syncthreads();
          if (tid == 0) {
            pick_run(sh.wtot, kWarps);
            if (!sh.dec.accept) atomicOr(&p.row_status[b], static_cast<unsigned>(COS_ROW_RESIDUAL_EMPTY));
          }
          __syncthreads();
          if (sh.win_g == warp) {
            const int token = walk(sb, se, gszv, sh.base, &sh.srun[warp][0], sh.target, true);
            if (lane == 0) p.out_tokens[uidx] = token;
          }
        }
      }
      }
      }  // stages 2 and 3
    }
    if (STAGE == 0 && rank == 0 && tid == 0) {
      const Decision& d = sh.dec;
      publish_unit(p, b, j, d.accept, d.status, d.cand, kSample ? d.drawable : __float_as_int(static_cast<float>(d.prob)),
                   d.ratio, d.r_d, d.q_d, d.S);
    }
    // No barrier here: everything the next unit writes before its first block barrier
    // (ldraft, next_local, u_acc/u_smp, warp partials) is read only before this point; stage 1
    // starts every unit with a block barrier of its own.
    if (STAGE >= 1) __syncthreads();
    unit = next_unit;
  }
  cluster.sync();  // no block leaves while a peer may still read its shared memory
  if (((STAGE == 0 && p.greedy) || STAGE >= 2) && tid == 0) stage_exit(p, STAGE == 0 ? 0 : 1);
}

// The log-sum-exp behind every softmax of a position, from the merged statistics a run leaves per position:
// ln sum_x exp(l(x) / T) = (ref + log2 s) ln 2.  One thread per (position, slot).
__global__ void export_lse_kernel(const UnitStats* ustats, const int4* unit_res, float* lse, int units, int slots, int sampling) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= units * slots) return;
  const int u = t / slots, k = t % slots;
  float v = __int_as_float(0x7fc00000);
  if (sampling && !(__ldcg(&unit_res[u]).y & COS_ROW_NONFINITE)) {
    const double sum = ustats[u].s[k];
    v = static_cast<float>((static_cast<double>(ustats[u].ref[k]) + log2(sum)) * 0.6931471805599453);
  }
  lse[t] = v;
}

// ------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------
thread_local std::string g_create_error;

}  // namespace

struct cos_verify_ctx {
  cos_verify_config cfg;
  int parts;            // blocks per unit in the drawing stages
  int parts_one;        // the same in the one-sweep drawing stage
  int max_clusters[5];  // resident clusters for cluster sizes 1, 2, 4, 8, 16 (0 = not available)
  int dense_blocks;     // resident blocks of the four-per-multiprocessor build of stage 0 (0 = there is none)
  int sm_count;
  unsigned* d_work_counter;
  bool scratch_dirty;
  // device scratch
  int* d_row_arrivals;
  int* d_row_reject;
  int4* d_unit_res;
  int* d_job_count;
  int2* d_jobs;
  UnitStats* d_ustats;
  double* d_zpart;
  double* d_wtotg;
  double* d_srung;
  double* d_srungC;  // third and fourth channel of the one-sweep stage (ensembles of three or four models)
  double* d_srungD;
  double* d_srungB;  // second channel of d_srung, for the one-sweep drawing stage
  int* d_part_arrivals;
  // optional per-stage timing (cos_verify_set_stage_timing)
  bool timing;
  cudaEvent_t ev[4];
  int ev_used;  // events recorded by the last run
  // optional staging for host-pointer runs
  // the one-launch form of a run (sampling modes the fused kernel covers, no cluster size requested)
  bool fused;      // the one-launch kernel covers this configuration (its scratch is allocated)
  bool use_fused;  // and runs take it (cos_verify_set_one_launch)
  bool draw_fused; // staged runs draw their tokens with that kernel's drawing items
  FusedPlan fplan;
  FusedScratch fscr;
  void* fused_mem[9];
  size_t fused_bytes[9];
  unsigned wait_limit;  // idle polls after which a block of the one-launch kernel gives up
  int test_drop;        // test hook: one streaming warp never reports its first item
  void* d_logits;
  int* d_drafts;
  int* d_proposer;
  float* d_bonus;
  int* d_accept;
  int* d_tokens;
  unsigned* d_status;
  float* d_diag;
  std::string err;
};

namespace {

using KernelFn = void (*)(const KParams);

KernelFn pick_kernel(int dtype, int mode, int stage, bool dense = false) {
  // one instantiation per stage, so that each gets its own register allocation; greedy modes have stage 0 only.
  // `dense`: stage 0 of ensemble sampling compiled for four blocks per multiprocessor; its sweep fits in 32
  // registers, and with more units than two blocks per multiprocessor can hold the extra warps pay
  // (measured on workload 3: 77.5 -> 74.3 us); with fewer units the 64-register build is the faster one.
  if (dense && stage == 0 && mode == kEnsembleSample) {
    if (dtype == COS_DTYPE_F32) return cos_verify_kernel<COS_DTYPE_F32, kEnsembleSample, 0, 4>;
    if (dtype == COS_DTYPE_BF16) return cos_verify_kernel<COS_DTYPE_BF16, kEnsembleSample, 0, 4>;
    if (dtype == COS_DTYPE_F16) return cos_verify_kernel<COS_DTYPE_F16, kEnsembleSample, 0, 4>;
  }
#define COS_CASE(DT, M, S) \
  if (dtype == DT && mode == M && stage == S) return cos_verify_kernel<DT, M, S>;
#define COS_SAMPLING(DT, M) COS_CASE(DT, M, 0) COS_CASE(DT, M, 1) COS_CASE(DT, M, 2) COS_CASE(DT, M, 3)
  // (stage 4, the one-sweep drawing stage with a channel per model, exists for ensembles only)
  // its sweep holds four vectors per lane and the next four: built for one block per multiprocessor (the
  // 64-register build spills a kilobyte per thread and is slower than the two-stage form)
  if (mode == kEnsembleSample && stage == 4) {
    if (dtype == COS_DTYPE_F32) return cos_verify_kernel<COS_DTYPE_F32, kEnsembleSample, 4, 1>;
    if (dtype == COS_DTYPE_BF16) return cos_verify_kernel<COS_DTYPE_BF16, kEnsembleSample, 4, 1>;
    if (dtype == COS_DTYPE_F16) return cos_verify_kernel<COS_DTYPE_F16, kEnsembleSample, 4, 1>;
  }
  COS_SAMPLING(COS_DTYPE_F32, kEnsembleSample)
  COS_SAMPLING(COS_DTYPE_F32, kLogitSample)
  COS_CASE(COS_DTYPE_F32, kEnsembleGreedy, 0)
  COS_CASE(COS_DTYPE_F32, kLogitGreedy, 0)
  COS_SAMPLING(COS_DTYPE_BF16, kEnsembleSample)
  COS_SAMPLING(COS_DTYPE_BF16, kLogitSample)
  COS_CASE(COS_DTYPE_BF16, kEnsembleGreedy, 0)
  COS_CASE(COS_DTYPE_BF16, kLogitGreedy, 0)
  COS_SAMPLING(COS_DTYPE_F16, kEnsembleSample)
  COS_SAMPLING(COS_DTYPE_F16, kLogitSample)
  COS_CASE(COS_DTYPE_F16, kEnsembleGreedy, 0)
  COS_CASE(COS_DTYPE_F16, kLogitGreedy, 0)
#undef COS_SAMPLING
#undef COS_CASE
  return nullptr;
}

int mode_of(const cos_verify_config& c) {
  const bool greedy = (c.temperature == 0.0f);
  if (c.combine == COS_COMBINE_PROB_ENSEMBLE) return greedy ? kEnsembleGreedy : kEnsembleSample;
  return greedy ? kLogitGreedy : kLogitSample;
}

int entries_per_vec(int dtype) { return dtype == COS_DTYPE_F32 ? 4 : 8; }
int elem_bytes(int dtype) { return dtype == COS_DTYPE_F32 ? 4 : 2; }

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
  if (c.dtype != COS_DTYPE_F32 && c.dtype != COS_DTYPE_BF16 && c.dtype != COS_DTYPE_F16)
    return fail(err, "unknown dtype %d", c.dtype);
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

// Blocks per unit in the drawing stages: as many as fit on the device in one wave (two blocks per
// multiprocessor), at least two steps per warp.
// The stage that draws the tokens in one sweep: 3 where two channel sums describe every mass (the combine is at
// logit level: proposer and combined logits; or it mixes two models), 4 for ensembles of three or four models (a
// channel per model); 0: the two-stage form (more models, one model, greedy decoding).
int one_sweep_stage(const cos_verify_config& c) {
  if (c.temperature == 0.0f) return 0;
  if (c.combine != COS_COMBINE_PROB_ENSEMBLE) return 3;
  return c.n == 2 ? 3 : ((c.n == 3 || c.n == 4) ? 4 : 0);
}

int choose_parts(const cos_verify_config& c, int rows, int sm_count) {
  int parts = 1;
  while (parts < kMaxParts && rows * parts * 2 <= 2 * sm_count) parts <<= 1;
  const int E = entries_per_vec(c.dtype);
  const int nsteps = (c.vocab + 32 * E - 1) / (32 * E);
  while (parts > 1 && nsteps / (parts * kWarps) < 2) parts >>= 1;
  return parts;
}

// Blocks per unit in the one-sweep drawing stage.  Where a block still has enough to do (eight steps per
// warp), several times more blocks than the device holds at once, so that it hands them out as slots come
// free: one wave of whole units leaves some multiprocessors with twice the work of others.  Small units
// stay at one wave: their blocks are bound by latency, not by throughput.
int choose_parts_one(const cos_verify_config& c, int rows, int sm_count) {
  const bool channels = (one_sweep_stage(c) == 4);
  const long long slots = (channels ? 1LL : 2LL) * sm_count;  // blocks the device holds at once
  const int E = entries_per_vec(c.dtype);
  const int nsteps = (c.vocab + 32 * E - 1) / (32 * E);
  // (the stage with a channel per model, one block per multiprocessor: blocks on half of the multiprocessors
  // were faster than blocks on all of them: workload 4 went from 96.1 to 90.1 us per call with 64 instead of 128)
  int parts = choose_parts(c, rows, channels ? sm_count / 2 : sm_count);
  while (parts < 8 && static_cast<long long>(rows) * parts < 3 * slots && nsteps / (2 * parts * kWarps) >= 8) parts <<= 1;
  return parts;
}

int log2i(int c) { return c >= 16 ? 4 : (c >= 8 ? 3 : (c >= 4 ? 2 : (c >= 2 ? 1 : 0))); }

// Stage 0 streams best with one block per unit (long contiguous reads, no cluster barrier);
// more blocks per unit only when there are too few units to occupy the device.
int choose_stream_cluster(const cos_verify_config& c, int units, int sm_count) {
  if (c.cluster_size > 0) return c.cluster_size;
  const int cap = choose_cluster(c);
  int cs = 1;
  while (cs < cap && units * cs < sm_count) cs <<= 1;
  return cs;
}

cudaError_t query_clusters(KernelFn fn, int cluster, int sm_count, int* out) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(cluster * sm_count, 1, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = 0;  // only stage 0 runs in clusters, and it stages nothing
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cluster;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(out, reinterpret_cast<const void*>(fn), &lc);
}

// attributes the kernels of one (dtype, mode) need before their first launch
cudaError_t prepare_kernels(int dtype, int mode, int cluster_size);

int stage_smem(int stage) { return stage >= 2 ? kRingBytes : 0; }  // the staging ring of the token-mass sweep

cudaError_t launch_stage(int dtype, int mode, int stage, const KParams& p, int cluster, cudaStream_t stream,
                         bool overlap_prev = false, bool dense = false) {
  KernelFn fn = pick_kernel(dtype, mode, stage, dense);
  if (fn == nullptr) return cudaErrorInvalidDeviceFunction;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(static_cast<unsigned>(p.num_clusters) * cluster, 1, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = stage_smem(stage);
  lc.stream = stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cluster;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = overlap_prev ? 2 : 1;
  return cudaLaunchKernelEx(&lc, fn, p);
}

cudaError_t prepare_kernels(int dtype, int mode, int cluster_size) {
  const bool draws = (mode == kEnsembleSample || mode == kLogitSample);
  cudaError_t e = cudaSuccess;
  for (int st = 2; draws && st <= 4 && e == cudaSuccess; ++st) {
    KernelFn fn = pick_kernel(dtype, mode, st);
    if (fn != nullptr)
      e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize, stage_smem(st));
  }
  if (e == cudaSuccess && cluster_size > 8)
    e = cudaFuncSetAttribute(reinterpret_cast<const void*>(pick_kernel(dtype, mode, 0)),
                             cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  return e;
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

// What a launch needs from the configuration and the arguments of a run (everything but the scratch pointers).
void fill_params(const cos_verify_config& c, const cos_verify_args* a, KParams& p) {
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
  const int eb = elem_bytes(c.dtype);
  p.vec_ok = (reinterpret_cast<uintptr_t>(a->logits) % 16 == 0) && ((a->stride_model * eb) % 16 == 0) &&
             ((a->stride_row * eb) % 16 == 0) && ((a->stride_pos * eb) % 16 == 0);
  p.nsteps = (c.vocab + 32 * E - 1) / (32 * E);
  p.flags = a->flags;
  p.num_units = a->batch * (c.gamma + 1);
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
  p.off_dev = reinterpret_cast<const unsigned long long*>(a->offset_device);
  p.row_base = a->row_base;
  p.accept_count = a->accept_count;
  p.out_tokens = a->out_tokens;
  p.row_status = a->row_status;
  p.diag = a->diag;
  p.dump_r = a->dump_r;
  p.bonus_prob = a->bonus_prob;
  p.per_pos = (a->flags & COS_RUN_PROPOSER_PER_POSITION) ? 1 : 0;
  p.bonus_model = (a->flags & COS_RUN_BONUS_FROM_MODEL) ? a->bonus_model : -1;
  p.greedy = (c.temperature == 0.0f) ? 1 : 0;
}

cos_status init_scratch(cos_verify_ctx* ctx, cudaStream_t stream) {
  const size_t rows = static_cast<size_t>(ctx->cfg.max_batch);
  cudaError_t e = cudaMemsetAsync(ctx->d_work_counter, 0, 4 * sizeof(unsigned), stream);  // counter and the two exit counts
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_row_arrivals, 0, rows * sizeof(int), stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_row_reject, 0x7f, rows * sizeof(int), stream);  // "none yet"
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_job_count, 0, 2 * sizeof(int), stream);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(ctx->d_part_arrivals, 0, rows * (static_cast<size_t>(ctx->cfg.gamma) + 1) * sizeof(int), stream);
  if (ctx->fused) {
    // counters, row words, arrival counters and the queue start at zero; the rest is written before it is read
    static const int kClear[] = {0, 1, 2, 4, 5, 6};
    for (int k : kClear)
      if (e == cudaSuccess) e = cudaMemsetAsync(ctx->fused_mem[k], 0, ctx->fused_bytes[k], stream);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, "scratch reset", e);
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
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, config->device);
  if (e != cudaSuccess) {
    delete ctx;
    return cuda_fail(nullptr, "cudaGetDeviceProperties", e);
  }
  ctx->sm_count = prop.multiProcessorCount;
  ctx->parts = choose_parts(*config, config->max_batch, ctx->sm_count);
  ctx->parts_one = choose_parts_one(*config, config->max_batch, ctx->sm_count);
  const size_t pmax = static_cast<size_t>(ctx->parts > ctx->parts_one ? ctx->parts : ctx->parts_one);
  KernelFn fn = pick_kernel(config->dtype, mode_of(*config), 0);
  e = prepare_kernels(config->dtype, mode_of(*config), config->cluster_size);
  if (e != cudaSuccess) {
    delete ctx;
    return cuda_fail(nullptr, "cudaFuncSetAttribute (shared memory or cluster size)", e);
  }
  for (int k = 0; k < 5; ++k) {
    const int cs = 1 << k;
    ctx->max_clusters[k] = 0;
    if (cs == 16 && config->cluster_size != 16) continue;
    int nc = 0;
    e = query_clusters(fn, cs, ctx->sm_count, &nc);
    if (e != cudaSuccess) {
      (void)cudaGetLastError();
      nc = 0;
    }
    ctx->max_clusters[k] = nc;
  }
  ctx->dense_blocks = 0;
  if (mode_of(*config) == kEnsembleSample) {
    int nc = 0;
    e = query_clusters(pick_kernel(config->dtype, kEnsembleSample, 0, true), 1, ctx->sm_count, &nc);
    if (e != cudaSuccess) {
      (void)cudaGetLastError();
      nc = 0;
    }
    ctx->dense_blocks = nc;
  }
  {
    const int need = config->cluster_size > 0 ? config->cluster_size : 1;
    if (ctx->max_clusters[log2i(need)] < 1 || ctx->max_clusters[0] < 1) {
      delete ctx;
      g_create_error = "no cluster of the requested size fits on the device";
      return COS_ERR_UNSUPPORTED;
    }
  }
  const size_t rows = static_cast<size_t>(config->max_batch), P = static_cast<size_t>(config->gamma) + 1;
  bool ok = true;
  ok = ok && cudaMalloc(&ctx->d_work_counter, 256) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_row_arrivals, rows * sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_row_reject, rows * sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_unit_res, rows * P * sizeof(int4)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_job_count, 256) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_jobs, (rows * P + rows) * sizeof(int2)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_ustats, rows * P * sizeof(UnitStats)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_zpart, rows * P * pmax * 8 * sizeof(double)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_wtotg, rows * P * pmax * kWarps * sizeof(double)) == cudaSuccess;
  const size_t steps = (static_cast<size_t>(config->vocab) + 32 * entries_per_vec(config->dtype) - 1) / (32 * entries_per_vec(config->dtype));
  const size_t rec_per_row = steps > pmax * kWarps * kRecG ? steps : pmax * kWarps * kRecG;  // one record per step, or per group of a run
  ok = ok && cudaMalloc(&ctx->d_srung, rows * rec_per_row * sizeof(double)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_srungB, rows * rec_per_row * sizeof(double)) == cudaSuccess;
  if (one_sweep_stage(*config) == 4) {
    ok = ok && cudaMalloc(&ctx->d_srungC, rows * rec_per_row * sizeof(double)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_srungD, rows * rec_per_row * sizeof(double)) == cudaSuccess;
  }
  ok = ok && cudaMalloc(&ctx->d_part_arrivals, rows * P * sizeof(int)) == cudaSuccess;
  ctx->wait_limit = 1u << 20;
  ctx->test_drop = 0;
  ctx->fused = false;
  ctx->draw_fused = false;
  if (ok && config->cluster_size == 0 &&
      fused_covers(config->dtype, mode_of(*config), config->n, config->vocab, config->gamma,
                   config->combine == COS_COMBINE_LOGIT_LINEAR ? config->mask_model : -1,
                   static_cast<long long>(rows) * static_cast<long long>(P))) {
    int per_sm = 0;
    e = fused_occupancy(config->dtype, mode_of(*config), config->n, &per_sm);
    if (e != cudaSuccess || per_sm < 1) {
      (void)cudaGetLastError();
    } else {
      ctx->fplan = fused_plan(config->dtype, mode_of(*config), config->n, config->vocab, config->gamma, config->max_batch,
                              ctx->sm_count, per_sm);
      fused_scratch_bytes(ctx->fplan, config->vocab, config->dtype, config->gamma, config->max_batch, ctx->fused_bytes);
      for (int k = 0; k < 9; ++k) ok = ok && cudaMalloc(&ctx->fused_mem[k], ctx->fused_bytes[k]) == cudaSuccess;
      if (ok) {
        ctx->fscr.ctr = static_cast<unsigned*>(ctx->fused_mem[0]);
        ctx->fscr.row_word = static_cast<unsigned long long*>(ctx->fused_mem[1]);
        ctx->fscr.unit_arrivals = static_cast<int*>(ctx->fused_mem[2]);
        ctx->fscr.chunk_part = static_cast<SoftPart*>(ctx->fused_mem[3]);
        ctx->fscr.dq = static_cast<int*>(ctx->fused_mem[4]);
        ctx->fscr.row_draw = static_cast<int*>(ctx->fused_mem[5]);
        ctx->fscr.draw_arrivals = static_cast<int*>(ctx->fused_mem[6]);
        ctx->fscr.dzpart = static_cast<double*>(ctx->fused_mem[7]);
        ctx->fscr.srec = static_cast<double*>(ctx->fused_mem[8]);
        ctx->fused = true;
      }
    }
  }
  if (ok && config->host_staging) {
    const size_t V = static_cast<size_t>(config->vocab);
    ok = ok && cudaMalloc(&ctx->d_logits, static_cast<size_t>(config->n) * rows * P * V * elem_bytes(config->dtype)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_drafts, rows * (P > 1 ? P - 1 : 1) * sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_proposer, rows * P * sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_bonus, rows * sizeof(float)) == cudaSuccess;
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

namespace {
// the launches of one run (everything but the optional export of the log-sum-exps)
cos_status run_launches(cos_verify_ctx* ctx, const cos_verify_args* a, void* cuda_stream) {
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
  if (a->flags & ~(COS_RUN_ALL_RESIDUALS | COS_RUN_PROPOSER_PER_POSITION | COS_RUN_BONUS_FROM_MODEL | COS_RUN_EARLY_EXIT |
                   COS_RUN_INPUTS_SETTLED)) return bad("unknown flag bits");
  if ((a->flags & COS_RUN_BONUS_FROM_MODEL) && (a->bonus_model < 0 || a->bonus_model >= c.n))
    return bad("bonus_model outside [0, n)");
  if (a->bonus_prob && reinterpret_cast<uintptr_t>(a->bonus_prob) % 4) {
    ctx->err = "bonus_prob is not 4-byte aligned";
    return COS_ERR_ALIGNMENT;
  }
  if (a->offset_device && reinterpret_cast<uintptr_t>(a->offset_device) % 8) {
    ctx->err = "offset_device is not 8-byte aligned";
    return COS_ERR_ALIGNMENT;
  }
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
  fill_params(c, a, p);
  p.work_counter = ctx->d_work_counter;
  p.exit_count = ctx->d_work_counter + 1;
  p.row_arrivals = ctx->d_row_arrivals;
  p.row_reject = ctx->d_row_reject;
  p.early_exit = (a->flags & COS_RUN_EARLY_EXIT) ? 1 : 0;
  p.unit_res = ctx->d_unit_res;
  p.job_count = ctx->d_job_count;
  p.jobs = ctx->d_jobs;
  p.ustats = ctx->d_ustats;
  p.zpart = ctx->d_zpart;
  p.wtotg = ctx->d_wtotg;
  p.srung = ctx->d_srung;
  p.part_arrivals = ctx->d_part_arrivals;
  p.srungB = ctx->d_srungB;
  p.srungC = ctx->d_srungC;
  p.srungD = ctx->d_srungD;
  p.parts = ctx->parts;
  p.max_jobs = p.num_units + a->batch;

  const int mode = mode_of(c);
  const bool draws = (mode == kEnsembleSample || mode == kLogitSample);
  // One launch does the whole run where the fused kernel covers it: aligned rows, no test hook.  (The hint to
  // leave positions unread is not taken there: every position is read once.)
  if (ctx->fused && ctx->use_fused && p.vec_ok && a->dump_r == nullptr && !(a->flags & COS_RUN_ALL_RESIDUALS)) {
    p.early_exit = 0;
    ctx->scratch_dirty = true;
    if (ctx->timing) cudaEventRecord(ctx->ev[0], stream);
    e = fused_launch(c.dtype, mode, p, ctx->fplan, ctx->fscr, ctx->wait_limit, ctx->test_drop, false, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, "kernel launch (one-launch form)", e);
    if (ctx->timing) cudaEventRecord(ctx->ev[1], stream);
    ctx->ev_used = 2;
    ctx->scratch_dirty = (ctx->test_drop != 0);  // a run that was made to give up leaves its counters behind
    return COS_OK;
  }
  // stage 0: every unit once (statistics, accept tests, row scans)
  const int c0 = choose_stream_cluster(c, p.num_units, ctx->sm_count);
  const int mc0 = ctx->max_clusters[log2i(c0)];
  if (mc0 < 1) {
    ctx->err = "no cluster of the chosen size fits on the device";
    return COS_ERR_UNSUPPORTED;
  }
  p.num_clusters = p.num_units < mc0 ? p.num_units : mc0;
  // more units than the 64-register build keeps resident, in the barrier-free form: the dense build
  const bool dense = (mode == kEnsembleSample) && c0 == 1 && p.num_units > mc0 && ctx->dense_blocks > mc0;
  if (dense) p.num_clusters = p.num_units < ctx->dense_blocks ? p.num_units : ctx->dense_blocks;
  ctx->scratch_dirty = true;  // cleared below once the launches are known to be queued
  if (ctx->timing) cudaEventRecord(ctx->ev[0], stream);
  p.early_dependents = (c0 == 1 && p.num_units >= ctx->sm_count) ? 1 : 0;
  {
    const bool masked = (c.combine != COS_COMBINE_PROB_ENSEMBLE) && c.mask_model >= 0;
    const bool hooks = (a->dump_r != nullptr) || (a->flags & COS_RUN_ALL_RESIDUALS);
    // what it overlaps with is the end of the previous call's drawing stage, where one block per row goes on alone;
    // a drawing stage of several waves of blocks leaves nothing to fill (workload 5 was 12 us slower with it), and
    // greedy runs have no drawing stage
    const int sweep_stage = one_sweep_stage(c);
    const long long slots = (sweep_stage == 4 ? 1LL : 2LL) * ctx->sm_count;
    const bool one_wave = draws && sweep_stage != 0 && static_cast<long long>(a->batch) * ctx->parts_one <= slots;
    p.inputs_settled =
        ((a->flags & COS_RUN_INPUTS_SETTLED) && p.early_dependents && one_wave && !masked && !hooks && !p.early_exit) ? 1 : 0;
  }
  e = launch_stage(c.dtype, mode, 0, p, c0, stream, p.early_dependents != 0, dense);
  if (e != cudaSuccess) return cuda_fail(ctx, "kernel launch (stage 0)", e);
  if (ctx->timing) cudaEventRecord(ctx->ev[1], stream);
  ctx->ev_used = 2;
  if (draws) {
    // stages 1 and 2: the units listed by stage 0 (one per row, or all of them under the test hooks);
    // blocks of a launch are independent, the launches themselves order the steps
    const bool all = (a->dump_r != nullptr) || (a->flags & COS_RUN_ALL_RESIDUALS);
    const int most = all ? p.max_jobs : a->batch;
    const int cap = 4096;  // a block walks the job list with a stride, so the grid may be smaller than the list
    p.num_clusters = (most < cap ? most : cap) * p.parts;  // blocks of a drawing launch
    // Two channel sums describe every mass when the combine is at logit level (proposer, combined logits) or
    // mixes two models: then one sweep does the work of stages 1 and 2.  The test hooks keep the two-stage form.
    const int sweep_stage = one_sweep_stage(c);
    const bool one_sweep = !all && sweep_stage != 0;
    if (!all && ctx->fused && ctx->draw_fused && p.vec_ok) {
      // the tokens are drawn by the persistent kernel's drawing items (one sweep with a channel sum per model, any
      // block takes any chunk of any row) instead of the drawing stages
      e = fused_launch(c.dtype, mode, p, ctx->fplan, ctx->fscr, ctx->wait_limit, 0, true, stream);
      if (e != cudaSuccess) return cuda_fail(ctx, "kernel launch (drawing items)", e);
      if (ctx->timing) cudaEventRecord(ctx->ev[2], stream);
      ctx->ev_used = 3;
      ctx->scratch_dirty = false;
      return COS_OK;
    }
    if (one_sweep) {
      p.parts = ctx->parts_one;
      p.num_clusters = (most < cap ? most : cap) * p.parts;
      e = launch_stage(c.dtype, mode, sweep_stage, p, 1, stream, true);
      if (e != cudaSuccess) return cuda_fail(ctx, "kernel launch (drawing stage)", e);
      if (ctx->timing) cudaEventRecord(ctx->ev[2], stream);
      ctx->ev_used = 3;
    }
    for (int st = 1; st <= 2 && !one_sweep; ++st) {
      e = launch_stage(c.dtype, mode, st, p, 1, stream, true);
      if (e != cudaSuccess) return cuda_fail(ctx, "kernel launch (drawing stages)", e);
      if (ctx->timing) cudaEventRecord(ctx->ev[st + 1], stream);
      ctx->ev_used = st + 2;
    }
  }
  // the last block of stage 0 to leave clears the work counter, the last of stage 2 the job counter: every
  // run starts from the same scratch state with the same arguments, whatever ran before it
  ctx->scratch_dirty = false;
  return COS_OK;
}

}  // namespace

#ifdef COS_STAGE_PROFILE
extern "C" int cos_stage_profile_read(unsigned long long* out, int blocks) {  // 8 words per block
  const size_t n = static_cast<size_t>(blocks < kSprofBlocks ? blocks : kSprofBlocks) * 8 * sizeof(unsigned long long);
  return cudaMemcpyFromSymbol(out, g_sprof, n) == cudaSuccess ? 0 : -1;
}
#endif

extern "C" cos_status cos_verify_run(cos_verify_ctx* ctx, const cos_verify_args* a, void* cuda_stream) {
  if (ctx && a && a->lse && reinterpret_cast<uintptr_t>(a->lse) % 4) {
    ctx->err = "lse is not 4-byte aligned";
    return COS_ERR_ALIGNMENT;
  }
  const cos_status st = run_launches(ctx, a, cuda_stream);
  if (st != COS_OK || a->lse == nullptr) return st;
  const cos_verify_config& c = ctx->cfg;
  const int units = a->batch * (c.gamma + 1);
  const int slots = (c.combine == COS_COMBINE_PROB_ENSEMBLE) ? c.n : 2;
  const int total = units * slots;
  export_lse_kernel<<<(total + 255) / 256, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      ctx->d_ustats, ctx->d_unit_res, a->lse, units, slots, c.temperature > 0.0f ? 1 : 0);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "kernel launch (log-sum-exp export)", e);
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
  if (a->dump_r || a->lse) {
    ctx->err = "dump_r and lse are not available for host-pointer runs";
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
  const size_t nprop = (a->flags & COS_RUN_PROPOSER_PER_POSITION) ? static_cast<size_t>(B * P) : static_cast<size_t>(B);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_proposer, a->proposer, nprop * sizeof(int), cudaMemcpyHostToDevice, stream);
  if (e != cudaSuccess) return cuda_fail(ctx, "host to device copy", e);
  cos_verify_args d = *a;
  d.flags &= ~COS_RUN_INPUTS_SETTLED;  // the inputs are what the copies above have just written
  d.logits = ctx->d_logits;
  d.draft_tokens = ctx->d_drafts;
  d.proposer = ctx->d_proposer;
  d.accept_count = ctx->d_accept;
  d.out_tokens = ctx->d_tokens;
  d.row_status = ctx->d_status;
  d.diag = a->diag ? ctx->d_diag : nullptr;
  d.bonus_prob = a->bonus_prob ? ctx->d_bonus : nullptr;
  if (a->offset_device) {  // a host address here, like every other pointer of this call
    d.offset = *a->offset_device;
    d.offset_device = nullptr;
  }
  cos_status st = cos_verify_run(ctx, &d, stream);
  if (st != COS_OK) return st;
  e = cudaMemcpyAsync(a->accept_count, ctx->d_accept, B * sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(a->out_tokens, ctx->d_tokens, B * P * sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(a->row_status, ctx->d_status, B * sizeof(unsigned), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess && a->diag)
    e = cudaMemcpyAsync(a->diag, ctx->d_diag, B * P * 4 * sizeof(float), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess && a->bonus_prob)
    e = cudaMemcpyAsync(a->bonus_prob, ctx->d_bonus, B * sizeof(float), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) {
    ctx->scratch_dirty = true;
    return cuda_fail(ctx, "device to host copy", e);
  }
  return COS_OK;
}

extern "C" cos_status cos_verify_set_stage_timing(cos_verify_ctx* ctx, int enable) {
  if (!ctx) return COS_ERR_INVALID_ARG;
  if (enable && !ctx->ev[0]) {
    for (int k = 0; k < 4; ++k) {
      cudaError_t e = cudaEventCreate(&ctx->ev[k]);
      if (e != cudaSuccess) return cuda_fail(ctx, "cudaEventCreate", e);
    }
  }
  ctx->timing = enable != 0;
  ctx->ev_used = 0;
  return COS_OK;
}

extern "C" cos_status cos_verify_get_stage_ms(cos_verify_ctx* ctx, float* ms, int32_t* count) {
  if (!ctx || !ms || !count) return COS_ERR_INVALID_ARG;
  *count = 0;
  if (!ctx->timing || ctx->ev_used < 2) {
    ctx->err = "no timed run to report";
    return COS_ERR_INVALID_ARG;
  }
  cudaError_t e = cudaEventSynchronize(ctx->ev[ctx->ev_used - 1]);
  for (int k = 0; e == cudaSuccess && k + 1 < ctx->ev_used; ++k) e = cudaEventElapsedTime(&ms[k], ctx->ev[k], ctx->ev[k + 1]);
  if (e != cudaSuccess) return cuda_fail(ctx, "stage timing", e);
  *count = ctx->ev_used - 1;
  return COS_OK;
}

extern "C" cos_status cos_verify_set_one_launch(cos_verify_ctx* ctx, int32_t enable) {
  if (!ctx) return COS_ERR_INVALID_ARG;
  if (enable && !ctx->fused) {
    ctx->err = "the one-launch form does not cover this configuration";
    return COS_ERR_UNSUPPORTED;
  }
  ctx->use_fused = (enable == 1);
  ctx->draw_fused = (enable == 2);
  return COS_OK;
}

extern "C" cos_status cos_verify_set_wait_limit(cos_verify_ctx* ctx, uint32_t polls, int32_t test_drop_report) {
  if (!ctx) return COS_ERR_INVALID_ARG;
  if (polls < 16) {
    ctx->err = "wait limit below 16 polls";
    return COS_ERR_INVALID_ARG;
  }
  ctx->wait_limit = polls;
  ctx->test_drop = test_drop_report ? 1 : 0;
  return COS_OK;
}

extern "C" cos_status cos_verify_get_info(const cos_verify_ctx* ctx, cos_verify_info* info) {
  if (!ctx || !info) return COS_ERR_INVALID_ARG;
  memset(info, 0, sizeof(*info));
  info->cluster_size = choose_stream_cluster(ctx->cfg, ctx->cfg.max_batch * (ctx->cfg.gamma + 1), ctx->sm_count);
  info->threads_per_block = kThreads;
  info->max_clusters = ctx->max_clusters[log2i(info->cluster_size)];
  info->sm_count = ctx->sm_count;
  {
    // ordinary runs (no test hook): one launch at T = 0; else stage 0 and the one-sweep drawing stage where it
    // applies (see one_sweep_stage), stages 0, 1 and 2 otherwise
    const int mode = mode_of(ctx->cfg);
    const bool one_sweep = one_sweep_stage(ctx->cfg) != 0 || (ctx->fused && ctx->draw_fused);
    info->launches_per_run = (ctx->cfg.temperature > 0.0f && !(ctx->fused && ctx->use_fused)) ? (one_sweep ? 2 : 3) : 1;
  }
  info->reserved[0] = ctx->fused ? ctx->fplan.chunks : ctx->parts;
  info->reserved[1] = ctx->fused ? ctx->fplan.dchunks : ctx->parts_one;
  info->reserved[2] = ((ctx->fused && ctx->use_fused) ? 1 : 0) | ((ctx->fused && ctx->draw_fused) ? 2 : 0);
  return COS_OK;
}

extern "C" cos_status cos_verify_destroy(cos_verify_ctx* ctx) {
  if (!ctx) return COS_OK;
  (void)cudaSetDevice(ctx->cfg.device);
  (void)cudaDeviceSynchronize();
  cudaFree(ctx->d_work_counter);
  cudaFree(ctx->d_row_arrivals);
  cudaFree(ctx->d_row_reject);
  cudaFree(ctx->d_job_count);
  cudaFree(ctx->d_jobs);
  cudaFree(ctx->d_ustats);
  cudaFree(ctx->d_zpart);
  cudaFree(ctx->d_wtotg);
  cudaFree(ctx->d_srung);
  cudaFree(ctx->d_srungB);
  cudaFree(ctx->d_srungC);
  cudaFree(ctx->d_srungD);
  cudaFree(ctx->d_part_arrivals);
  for (int k = 0; k < 4; ++k)
    if (ctx->ev[k]) cudaEventDestroy(ctx->ev[k]);
  cudaFree(ctx->d_unit_res);
  for (int k = 0; k < 9; ++k) cudaFree(ctx->fused_mem[k]);
  cudaFree(ctx->d_logits);
  cudaFree(ctx->d_drafts);
  cudaFree(ctx->d_proposer);
  cudaFree(ctx->d_bonus);
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

// ------------------------------------------------------------------------------------
// verification without a context and without any device allocation
// ------------------------------------------------------------------------------------
namespace {

// Scratch of the context-free entry point.  It is part of the library image: every device
// that loads the library holds these COS_STATIC_SCRATCH_BYTES until the process exits.
// Layout: [0, 256) work and job counters | row arrival counters | unit results | job list | unit statistics |
// partial normalisers | run masses | running totals of the drawing unit of each row.
static __device__ __align__(256) unsigned char g_static_scratch[COS_STATIC_SCRATCH_BYTES];

constexpr int kStaticMaxDevices = 64;
// Device address of g_static_scratch per device.  In host code the symbol itself is only a
// stand-in, never an address a kernel may use, so the address is asked for once per device.
unsigned char* g_static_addr[kStaticMaxDevices];
bool g_static_ready[kStaticMaxDevices];
std::mutex g_static_mutex;  // first calls from several host threads look the address up once

cos_status static_fail(cos_status st, const char* msg) {
  g_create_error = msg;
  return st;
}

}  // namespace

extern "C" cos_status cos_verify_run_static(const cos_verify_config* config, const cos_verify_args* a,
                                            void* cuda_stream) {
  if (!config || !a) return static_fail(COS_ERR_INVALID_ARG, "null argument");
  cos_verify_config c = *config;
  c.max_batch = COS_STATIC_MAX_BATCH;  // the array, not the caller, bounds the batch here
  if (!validate_config(c, &g_create_error)) return COS_ERR_INVALID_ARG;
  if (a->batch < 1 || a->batch > COS_STATIC_MAX_BATCH)
    return static_fail(COS_ERR_INVALID_ARG, "batch exceeds COS_STATIC_MAX_BATCH (1024) of the built-in scratch");
  const long long units = static_cast<long long>(a->batch) * (c.gamma + 1);
  if (units > COS_STATIC_MAX_POSITIONS)
    return static_fail(COS_ERR_INVALID_ARG,
                       "batch * (gamma + 1) exceeds COS_STATIC_MAX_POSITIONS (8192) of the built-in scratch");
  if (c.device < 0 || c.device >= kStaticMaxDevices) return static_fail(COS_ERR_INVALID_ARG, "device ordinal out of range");
  if (!a->logits || !a->proposer || !a->accept_count || !a->out_tokens || !a->row_status)
    return static_fail(COS_ERR_INVALID_ARG, "null device pointer");
  if (c.gamma > 0 && !a->draft_tokens) return static_fail(COS_ERR_INVALID_ARG, "draft_tokens is null although gamma > 0");
  if (a->stride_model < 0 || a->stride_row < 0 || a->stride_pos < 0) return static_fail(COS_ERR_INVALID_ARG, "negative stride");
  if (a->flags & ~(COS_RUN_ALL_RESIDUALS | COS_RUN_PROPOSER_PER_POSITION | COS_RUN_BONUS_FROM_MODEL | COS_RUN_EARLY_EXIT |
                   COS_RUN_INPUTS_SETTLED)) return static_fail(COS_ERR_INVALID_ARG, "unknown flag bits");
  if ((a->flags & COS_RUN_BONUS_FROM_MODEL) && (a->bonus_model < 0 || a->bonus_model >= c.n))
    return static_fail(COS_ERR_INVALID_ARG, "bonus_model outside [0, n)");
  if (a->bonus_prob && reinterpret_cast<uintptr_t>(a->bonus_prob) % 4)
    return static_fail(COS_ERR_ALIGNMENT, "bonus_prob is not 4-byte aligned");
  if (a->offset_device && reinterpret_cast<uintptr_t>(a->offset_device) % 8)
    return static_fail(COS_ERR_ALIGNMENT, "offset_device is not 8-byte aligned");
  if (a->lse) return static_fail(COS_ERR_UNSUPPORTED, "lse is not available from the allocation-free entry point");
  const int eb = elem_bytes(c.dtype);
  if (reinterpret_cast<uintptr_t>(a->logits) % eb) return static_fail(COS_ERR_ALIGNMENT, "logits pointer not aligned to its element type");
  if (reinterpret_cast<uintptr_t>(a->proposer) % 4 || reinterpret_cast<uintptr_t>(a->accept_count) % 4 ||
      reinterpret_cast<uintptr_t>(a->out_tokens) % 4 || reinterpret_cast<uintptr_t>(a->row_status) % 4 ||
      (a->draft_tokens && reinterpret_cast<uintptr_t>(a->draft_tokens) % 4) ||
      (a->diag && reinterpret_cast<uintptr_t>(a->diag) % 4) || (a->dump_r && reinterpret_cast<uintptr_t>(a->dump_r) % 4))
    return static_fail(COS_ERR_ALIGNMENT, "an int32/float pointer is not 4-byte aligned");

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaSetDevice(c.device);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaSetDevice", e);
  KernelFn fn = pick_kernel(c.dtype, mode_of(c), 0);
  {
    std::lock_guard<std::mutex> guard(g_static_mutex);
    if (!g_static_ready[c.device]) {
      // once per device, with that device current: the device address of the built-in array
      void* addr = nullptr;
      e = cudaGetSymbolAddress(&addr, g_static_scratch);
      if (e != cudaSuccess || addr == nullptr) return cuda_fail(nullptr, "cudaGetSymbolAddress(built-in scratch)", e);
      g_static_addr[c.device] = static_cast<unsigned char*>(addr);
      g_static_ready[c.device] = true;
    }
  }
  e = prepare_kernels(c.dtype, mode_of(c), c.cluster_size);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaFuncSetAttribute", e);
  int sm_count = 0;
  e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, c.device);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaDeviceGetAttribute", e);
  const int c0 = choose_stream_cluster(c, static_cast<int>(units), sm_count);
  int mc0 = 0;
  e = query_clusters(fn, c0, sm_count, &mc0);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaOccupancyMaxActiveClusters", e);
  if (mc0 < 1) return static_fail(COS_ERR_UNSUPPORTED, "no cluster of the requested size fits on the device");

  // carve the array; what must start clean is cleared on the caller's stream before the kernels
  unsigned char* basep = g_static_addr[c.device];
  unsigned* d_counter = reinterpret_cast<unsigned*>(basep);
  int* d_job_count = reinterpret_cast<int*>(basep + 16);
  int* d_arrivals = reinterpret_cast<int*>(basep + 256);
  int4* d_unit_res = reinterpret_cast<int4*>(basep + 256 + 4 * COS_STATIC_MAX_BATCH);
  int2* d_jobs = reinterpret_cast<int2*>(reinterpret_cast<unsigned char*>(d_unit_res) + 16 * COS_STATIC_MAX_POSITIONS);
  UnitStats* d_ustats = reinterpret_cast<UnitStats*>(reinterpret_cast<unsigned char*>(d_jobs) +
                                                      8 * (COS_STATIC_MAX_POSITIONS + COS_STATIC_MAX_BATCH));
  static_assert(sizeof(UnitStats) == 112, "COS_STATIC_SCRATCH_BYTES assumes 112 bytes of statistics per position");
  // one block per unit in the drawing stages here (parts = 1), which keeps the built-in array small
  double* d_zpart = reinterpret_cast<double*>(reinterpret_cast<unsigned char*>(d_ustats) + 112 * COS_STATIC_MAX_POSITIONS);
  double* d_wtotg = d_zpart + 8 * COS_STATIC_MAX_POSITIONS;
  double* d_srung = d_wtotg + 16 * COS_STATIC_MAX_POSITIONS;
  int* d_part_arrivals = reinterpret_cast<int*>(d_srung + 16 * 16 * COS_STATIC_MAX_BATCH);
  static_assert(kWarps == 16 && kRecG == 16, "COS_STATIC_SCRATCH_BYTES assumes 16 runs and 16 recorded totals per run");
  e = cudaMemsetAsync(basep, 0, 256, stream);  // work counter and both job counters
  if (e == cudaSuccess) e = cudaMemsetAsync(d_arrivals, 0, static_cast<size_t>(a->batch) * sizeof(int), stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(d_part_arrivals, 0, static_cast<size_t>(units) * sizeof(int), stream);
  if (e != cudaSuccess) return cuda_fail(nullptr, "clearing the built-in scratch", e);

  KParams p;
  fill_params(c, a, p);
  p.num_units = static_cast<int>(units);
  p.work_counter = d_counter;
  p.exit_count = d_counter + 1;
  p.row_arrivals = d_arrivals;
  p.row_reject = nullptr;  // the hint to leave positions unread is not taken here
  p.early_exit = 0;
  p.unit_res = d_unit_res;
  p.job_count = d_job_count;
  p.jobs = d_jobs;
  p.ustats = d_ustats;
  p.zpart = d_zpart;
  p.wtotg = d_wtotg;
  p.srung = d_srung;
  p.part_arrivals = d_part_arrivals;
  p.parts = 1;
  p.max_jobs = p.num_units + a->batch;

  p.num_clusters = p.num_units < mc0 ? p.num_units : mc0;
  e = launch_stage(c.dtype, mode_of(c), 0, p, c0, stream);
  if (e != cudaSuccess) return cuda_fail(nullptr, "kernel launch (stage 0)", e);
  if (mode_of(c) == kEnsembleSample || mode_of(c) == kLogitSample) {
    const bool all = (a->dump_r != nullptr) || (a->flags & COS_RUN_ALL_RESIDUALS);
    const int most = all ? p.max_jobs : a->batch;
    for (int st = 1; st <= 2; ++st) {
      p.num_clusters = most < 4096 ? most : 4096;
      e = launch_stage(c.dtype, mode_of(c), st, p, 1, stream);
      if (e != cudaSuccess) return cuda_fail(nullptr, "kernel launch (drawing stages)", e);
    }
  }
  return COS_OK;
}
