// Staged launches of the CoS verification step: the kernel template, one instantiation per (dtype, mode, stage).
// Included by cos_verify.cu only.
#pragma once

#include "cos_stage_shared.cuh"
#include "cos_stage_draw.cuh"
#include "cos_stage_stream.cuh"

using namespace cosv;

namespace {

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
      stage0_free_running<DT, MODE, (MINB >= 4) ? 4 : 6>(p, sh);
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
      sweep_unit<DT, MODE, (MINB >= 4) ? 4 : 6>(p, base, sl, pis, false, 0.f, &sh.wsoft[warp][0], &sh.warg[warp][0]);
      cluster_merge(sh, cluster, phase, p.n, 0, 0);
      if (tid < p.n && !is_bonus && draft_ok) {
        // probability of the draft under model tid, with the constant the sweep used
        sh.pdraft[tid] = exp2(static_cast<double>(sh.ldraft[tid]) * p.cT64 - static_cast<double>(sh.fsoft[tid].ref)) /
                         sh.fsoft[tid].s;
      }
    } else if (MODE == kEnsembleGreedy) {
      sweep_unit<DT, MODE, (MINB >= 4) ? 4 : 6>(p, base, sl, pis, false, 0.f, &sh.wsoft[warp][0], &sh.warg[warp][0]);
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
        if (p.draw_cluster) {
          // the blocks of a unit are one thread-block cluster: its hardware barrier (release on arrival, acquire on
          // leaving) makes the partial sums and step records of all of them visible, and the first block goes on
          cluster.sync();
          do_locate = (rank == 0) && emit;
        } else {
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
        }
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
  if (STAGE == 0) cluster.sync();  // no block leaves while a peer may still read its shared memory
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

}  // namespace
