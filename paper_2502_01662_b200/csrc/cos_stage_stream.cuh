// Staged launches of the CoS verification step: the streaming stage (stage 0): the sweep of one (row, position)
// (Eq. 3-5), the accept decision (Eq. 6) and the barrier-free form of the loop over positions.
// Included by cos_verify.cu only.
#pragma once

#include "cos_stage_shared.cuh"

using namespace cosv;

namespace {

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
// U: loads in flight per thread in the ensemble sweep (4 in the 32-register build, 6 where 64 registers allow it:
// workload 4 went from 88.0 to 86.0 us per call; the 32-register build spills with 6 and lost 1.9 us on workload 3)
template <int DT, int MODE, int U = 4>
__device__ __forceinline__ void sweep_unit(const KParams& p, const char* base, const Slice& sl, int pis, bool masked,
                                           float thr, SoftPart* wsoft, ArgPart* warg) {
  constexpr int E = Elem<DT>::E;
  const int tid = threadIdx.x, lane = tid & 31;
  auto row_of = [&](int i) -> const void* { return base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes; };
  if (MODE == kEnsembleSample) {
    for (int i = 0; i < p.n; ++i) {
      LaneSoft acc = soft_slice<DT, kThreads, U>(row_of(i), sl, tid, p.cT);
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
        for (int k = 0; k < E; ++k) bad |= !(x[k] < INFINITY);
#pragma unroll
        for (int k = 0; k < E; k += 2) {  // (packed fp32 pairs: the same values, half the instructions)
          fma2(c32[k], c32[k + 1], wi, wi, x[k], x[k + 1], c32[k], c32[k + 1]);
          bnd[k] = fmaf(wa, fabsf(x[k]), bnd[k]);
          bnd[k + 1] = fmaf(wa, fabsf(x[k + 1]), bnd[k + 1]);
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
template <int DT, int MODE, int U = 4>
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
  if (warp == 0) SPROFL(0);
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
      sweep_unit<DT, MODE, U>(p, base, sl, pis, false, -INFINITY, &fr.wsoft[par][warp][0], &fr.warg[par][warp][0]);
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
      SPROFL(1);
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
      SPROFL(2);
      if (lane == 0) decide_unit<DT, MODE>(p, sh, is_bonus, draft, draft_ok, pi, pi_ok, pis, false);
      __syncwarp();
      SPROFL(3);
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
      SPROFL(4);
    }
  }
  // the last warp of the block to run out of units reports the block's departure
  if (p.greedy && lane == 0 && atomicAdd(&fr.left, 1) == kWarps - 1) stage_exit(p, 0);
}

}  // namespace
