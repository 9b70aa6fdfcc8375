// Staged launches of the CoS verification step: the block's shared-memory layout, the merge over a cluster, and
// publishing a (row, position) with the per-row first-rejection scan (Sec. 3.1).  Included by cos_verify.cu only.
#pragma once

#include "cos_common.cuh"

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
// (the same by lane 0 of whichever warp gets there: the barrier-free streaming stage)
#define SPROFL(k)                                                                                 \
  do {                                                                                            \
    if ((threadIdx.x & 31) == 0 && blockIdx.x < kSprofBlocks) {                                   \
      unsigned long long t_;                                                                      \
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));                                       \
      g_sprof[blockIdx.x * 8 + (k)] = t_;                                                         \
    }                                                                                             \
  } while (0)
#else
#define SPROF(k)
#define SPROFL(k)
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

}  // namespace
