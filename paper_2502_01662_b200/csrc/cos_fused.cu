// CoS verification in ONE persistent launch (sampling modes, T > 0): combine (Eq. 3-5), accept test (Eq. 6),
// first-rejection scan and the residual / bonus draw (Sec. 3.1-3.2) without a second pass over the batch.
//
// The run is cut into work items that any block can take:
//   streaming item  one (row, position), or one chunk of it (a contiguous range of steps of its n logit rows):
//                   per-model softmax statistics of the chunk.  The block that completes the last chunk of a
//                   position merges the chunks in order, takes the accept test and publishes the position.
//   drawing item    one chunk of the one position of a row that must emit a token (its first rejection, or the
//                   bonus position): per step (32 lanes x one 16-byte vector) the channel sums over the tokens
//                   with a positive mass, plus the refined normalisers.  The block that completes the last chunk
//                   turns the sums into masses, finds the step by a prefix and walks it to the token.
// Streaming items come from a counter in row-major order; a row is settled as soon as every position up to its
// first rejection has been published (rows resolve from the front), and its drawing items then go to a queue
// that blocks look at before they take the next streaming item.
//
// A block (one per multiprocessor) is fifteen streaming warps, a service warp, a producer warp and a locating warp.
// The producer (one thread) follows the block's items and fills a ring of five 30 KB stages in shared memory with
// 1-D bulk copies that complete on mbarriers, running ahead across item boundaries; the streaming warps consume the
// stages without block barriers and leave their partial sums in a ring of eight item slots.  Drawing items are read by
// the streaming warps themselves.  The service warp fetches items ahead, merges the partials, talks to the other
// blocks (fences, arrival counters, the queue) and decides positions; the locating warp turns a row's recorded step
// sums into its token, so none of the serial work sits on the streaming warps' path.
// No block depends on a particular other block: any item can be taken by any block, and a block with nothing to
// do looks at the queue (with a growing pause) until every position is published and every row has its token.
// All waits are bounded.

#include "cos_fused.h"

using namespace cosv;

namespace {

constexpr int kFT = 576;          // threads per block: fifteen streaming warps, then the service, producer and locating warps
constexpr int kSW = 15;           // streaming warps
constexpr int kST = kSW * 32;     // streaming threads
constexpr int kRing = 8;          // items a block may have open
constexpr int kSvcWarp = kSW, kProdWarp = kSW + 1;  // the last warp locates tokens
constexpr int kNST = 5;                    // stages of the shared-memory ring the producer fills with bulk copies
constexpr int kVPT = 4;                    // 16-byte vectors per streaming thread and stage
constexpr int kStageVecs = kST * kVPT;     // 1920 vectors
constexpr int kStageBytes = kStageVecs * 16;  // 30 KB
constexpr int kCh = 4;            // channels of a drawing sweep (ensembles of up to four models; logit level: two)
constexpr int kItemStream = 0, kItemDraw = 1, kItemJob = 2, kItemExit = 3;  // kItemJob: a drawing item named by its place in the job list
// counters, each on a 128-byte line of its own (the queue's head and tail share one: they are read together)
constexpr int kCtrNext = 0, kCtrEvents = 32, kCtrHead = 64, kCtrTail = 65, kCtrGone = 96, kCtrFault = 128;
constexpr int kCtrWords = 160;

// Optional timeline accounting (build with -DCOS_FUSED_PROFILE): cycles the service warp and streaming warp 0 of
// every block spend in each activity, summed over blocks into g_prof.  Compiled out of ordinary builds.
#ifdef COS_FUSED_PROFILE
__device__ unsigned long long g_prof[48];
__device__ unsigned long long g_prof_t0;  // globaltimer at the start of the launch (block 0)
#define PROF_DECL unsigned long long prof_acc[16] = {0}; long long prof_t0 = 0; (void)prof_t0
#define PROF_T0 prof_t0 = clock64()
#define PROF_ADD(k) do { const long long t1_ = clock64(); prof_acc[k] += static_cast<unsigned long long>(t1_ - prof_t0); prof_t0 = t1_; } while (0)
#define PROF_COUNT(k) prof_acc[k] += 1
__device__ __forceinline__ unsigned long long prof_now() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define PROF_FLUSH(base) do { if ((threadIdx.x & 31) == 0) for (int q_ = 0; q_ < 16; ++q_) if (prof_acc[q_]) atomicAdd(&g_prof[(base) + q_], prof_acc[q_]); } while (0)
#else
#define PROF_DECL
#define PROF_T0
#define PROF_ADD(k)
#define PROF_COUNT(k)
#define PROF_FLUSH(base)
#endif

struct FParams {
  KParams k;
  FusedPlan plan;
  FusedScratch s;
  int num_items;          // streaming items of this run
  int nvec;               // 16-byte vectors per logit row
  unsigned total_events;  // positions to publish + rows to settle
  unsigned poll_limit;
  int debug_drop;
  int draw_only;          // the positions were published by an earlier launch; this one draws the tokens of its job list
};

struct ItemCtx {
  int kind, b, j, chunk;
  int pis;          // model whose distribution is q (valid index)
  int lo, hi;       // streaming: vectors [lo, hi) of every row; drawing: steps [lo, hi)
  int dkind;        // drawing: what the token is drawn from
  float ct[kCh], nref[kCh], bt[kCh];
  double ct64[kCh], dref[kCh];
};

struct FShared {
  int tag[kRing];       // seq + 1 once ctx[seq % kRing] is valid
  int arrive[kRing];    // streaming warps that have finished the item of that slot
  int started;          // number of items some warp has begun
  int fault;
  int num_items;        // items handed out by the counter
  unsigned total_events;
  // drawing-only launch: rows whose drawing sweep is complete, handed from the service warp to the locating warp
  int loc_ring[8];
  int loc_tail, loc_head, loc_exit;
  // the ring of stages: `full` completes when a stage's bulk copies have landed, `empty` when the fifteen
  // streaming warps have read it
  unsigned long long full[kNST], empty[kNST];
  ItemCtx ctx[kRing];
  SoftPart part[kRing][kSW][kCh];
};

__device__ __forceinline__ int vol_load(const int* p) { return *reinterpret_cast<const volatile int*>(p); }
__device__ __forceinline__ unsigned vol_load(const unsigned* p) { return *reinterpret_cast<const volatile unsigned*>(p); }

// ---- mbarriers and 1-D bulk copies (global -> shared, completing on an mbarrier) --------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(void* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok)
               : "r"(smem_u32(bar)), "r"(parity)
               : "memory");
  return ok != 0;
}
// Bounded wait for the phase of `parity` to complete.  False when it gave up (it then raises the block's fault
// flag) or when another warp already has.
__device__ __forceinline__ bool mbar_wait(void* bar, unsigned parity, int* fault, unsigned limit) {
  for (unsigned long long it = 0; it < 64ull * limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (vol_load(fault)) return false;
  }
  *reinterpret_cast<volatile int*>(fault) = 1;
  return false;
}
// both addresses 16-byte aligned, `bytes` a multiple of 16
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, void* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

template <int DT>
__device__ __forceinline__ uint4 ninf_vec() {
  const unsigned w = (DT == COS_DTYPE_F32) ? 0xff800000u : (DT == COS_DTYPE_BF16 ? 0xff80ff80u : 0xfc00fc00u);
  return make_uint4(w, w, w, w);
}

__device__ __forceinline__ const char* unit_base(const KParams& p, int b, int j, int eb) {
  return reinterpret_cast<const char*>(p.logits) + (static_cast<long long>(b) * p.s_row + static_cast<long long>(j) * p.s_pos) * eb;
}

// coefficient of channel i in the mass that is drawn from: max(0, r - q), r, or q
template <int MODE>
__device__ __forceinline__ double channel_k(const KParams& p, int i, int pis, int dkind) {
  if (MODE == kEnsembleSample) {
    const double sel = (i == pis) ? 1.0 : 0.0;
    return dkind == kDrawResidual ? p.w64[i] - sel : (dkind == kDrawQ ? sel : p.w64[i]);
  }
  if (i == 0) return dkind == kDrawResidual ? -1.0 : (dkind == kDrawQ ? 1.0 : 0.0);
  return dkind == kDrawQ ? 0.0 : 1.0;
}

// ------------------------------------------------------------------------------------
// streaming warps
// ------------------------------------------------------------------------------------
// A streaming load that stays where it is written (a batch of loads is issued first, then consumed).
__device__ __forceinline__ uint4 ldg_ahead16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// One row's share of one thread again in the running-maximum form (after an overflow or a non-finite input).
template <int DT>
__device__ __noinline__ LaneSoft online_redo(const char* row, int v_first, int v_hi, float c) {
  constexpr int E = Elem<DT>::E;
  LaneSoft acc;
  acc.init();
  for (int v = v_first; v < v_hi; v += kST) {
    float x[E];
    Elem<DT>::unpack(ldg_stream16(row + static_cast<long long>(v) * 16), x);
    acc.add_online(x, c);
  }
  return acc;
}

// How a streaming item maps to stages of the ring.  The producer warp and the streaming warps walk the same sequence:
// ensemble: row after row, 1920 vectors of one row per stage; logit level with two models: 960 vectors of each of the
// two rows per stage (the second row in the stage's upper half).  `k` counts stages since the launch began.

// Ensemble: the softmax statistics of the chunk [lo, hi) of every model's row.  A thread's vectors are those at
// lo + stid + 480 m, four per stage, read from shared memory once the stage's bulk copy has landed.  Fixed reference
// exponent per row and thread, seeded from the thread's first vector (a whole number, so that sums rescale exactly);
// overflow or a non-finite input redoes the thread's share of that row from global memory in the running-maximum
// form.  False when a wait gave up.
template <int DT>
__device__ __forceinline__ bool stream_ensemble(const FParams& fp, const ItemCtx& it, SoftPart* part, int stid, FShared& sh,
                                                const unsigned char* ring, unsigned& k) {
  constexpr int E = Elem<DT>::E;
  const KParams& p = fp.k;
  const int lane = stid & 31;
  const char* base = unit_base(p, it.b, it.j, Elem<DT>::bytes);
  const long long row_step = p.s_model * Elem<DT>::bytes;
  for (int i = 0; i < p.n; ++i) {
    LaneSoft acc;
    acc.init();
    bool first = true;
    for (int v = it.lo; v < it.hi; v += kStageVecs, ++k) {
      const unsigned slot = k % kNST;
      if (!mbar_wait(&sh.full[slot], (k / kNST) & 1u, &sh.fault, fp.poll_limit)) return false;
      const int nv = (it.hi - v < kStageVecs) ? it.hi - v : kStageVecs;
      const uint4* st = reinterpret_cast<const uint4*>(ring + static_cast<size_t>(slot) * kStageBytes);
      uint4 raw[kVPT];
#pragma unroll
      for (int j = 0; j < kVPT; ++j)
        if (stid + j * kST < nv) raw[j] = st[stid + j * kST];
#pragma unroll
      for (int j = 0; j < kVPT; ++j) {
        if (stid + j * kST < nv) {
          float x[E];
          Elem<DT>::unpack(raw[j], x);
          if (j == 0 && first) {
            acc.seed(x, p.cT);
            first = false;
          }
          acc.add_fixed(x, p.cT);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.empty[slot]);
    }
    if (!(acc.s < INFINITY)) acc = online_redo<DT>(base + i * row_step, it.lo + stid, it.hi, p.cT);
    warp_merge_soft(acc, &part[i], lane);
  }
  return true;
}

// Logit level with two models: proposer's softmax and the softmax of the combined logits.  `settled` comes back
// false when some lane of the warp met an overflow or a non-finite input (the caller then takes the general form
// from global memory).  False when a wait gave up.
template <int DT>
__device__ __forceinline__ bool stream_logit2(const FParams& fp, const ItemCtx& it, SoftPart* part, int stid, FShared& sh,
                                              const unsigned char* ring, unsigned& k, bool& settled_all) {
  constexpr int E = Elem<DT>::E;
  constexpr int HV = kStageVecs / 2, HT = kVPT / 2;  // vectors of each row per stage, per thread
  const KParams& p = fp.k;
  const int lane = stid & 31;
  const float w0 = p.w[0], w1 = p.w[1];
  const bool q_is_0 = (it.pis == 0);
  LaneSoft accq, accc;
  accq.init();
  accc.init();
  bool first = true;
  for (int v = it.lo; v < it.hi; v += HV, ++k) {
    const unsigned slot = k % kNST;
    if (!mbar_wait(&sh.full[slot], (k / kNST) & 1u, &sh.fault, fp.poll_limit)) return false;
    const int nv = (it.hi - v < HV) ? it.hi - v : HV;
    const uint4* st0 = reinterpret_cast<const uint4*>(ring + static_cast<size_t>(slot) * kStageBytes);
    const uint4* st1 = st0 + HV;
    uint4 r0[HT], r1[HT];
#pragma unroll
    for (int j = 0; j < HT; ++j)
      if (stid + j * kST < nv) {
        r0[j] = st0[stid + j * kST];
        r1[j] = st1[stid + j * kST];
      }
#pragma unroll
    for (int j = 0; j < HT; ++j) {
      if (stid + j * kST < nv) {
        float x0[E], x1[E], cmb[E];
        Elem<DT>::unpack(r0[j], x0);
        Elem<DT>::unpack(r1[j], x1);
#pragma unroll
        for (int q = 0; q < E; ++q) cmb[q] = fmaf(w1, x1[q], fmaf(w0, x0[q], 0.f));
        if (j == 0 && first) {
          if (q_is_0) accq.seed(x0, p.cT); else accq.seed(x1, p.cT);
          accc.seed(cmb, p.cT);
          first = false;
        }
        if (q_is_0) accq.add_fixed(x0, p.cT); else accq.add_fixed(x1, p.cT);
        accc.add_fixed(cmb, p.cT);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.empty[slot]);
  }
  const bool settled = (accq.s < INFINITY) && (accc.s < INFINITY);
  settled_all = __all_sync(0xffffffffu, settled);
  if (settled_all) {
    warp_merge_soft(accq, &part[0], lane);
    warp_merge_soft(accc, &part[1], lane);
  }
  return true;
}

// The producer warp's side of a streaming item (one thread): the stages in the order the streaming warps read them.
// A stage is refilled once the fifteen warps have released its previous contents.  False when a wait gave up.
template <int MODE>
__device__ __forceinline__ bool produce_item(const FParams& fp, const ItemCtx& it, FShared& sh, unsigned char* ring, unsigned& k,
                                             int eb) {
  const KParams& p = fp.k;
  const char* base = unit_base(p, it.b, it.j, eb);
  const long long row_step = p.s_model * eb;
  auto acquire = [&](unsigned slot) -> bool {
    return k < static_cast<unsigned>(kNST) || mbar_wait(&sh.empty[slot], ((k / kNST) - 1u) & 1u, &sh.fault, fp.poll_limit);
  };
  if (MODE == kEnsembleSample) {
    for (int i = 0; i < p.n; ++i)
      for (int v = it.lo; v < it.hi; v += kStageVecs, ++k) {
        const unsigned slot = k % kNST;
        if (!acquire(slot)) return false;
        const unsigned bytes = static_cast<unsigned>((it.hi - v < kStageVecs ? it.hi - v : kStageVecs)) * 16u;
        mbar_expect_tx(&sh.full[slot], bytes);
        bulk_load(ring + static_cast<size_t>(slot) * kStageBytes, base + i * row_step + static_cast<long long>(v) * 16, bytes,
                  &sh.full[slot]);
      }
  } else {
    constexpr int HV = kStageVecs / 2;
    for (int v = it.lo; v < it.hi; v += HV, ++k) {
      const unsigned slot = k % kNST;
      if (!acquire(slot)) return false;
      const unsigned bytes = static_cast<unsigned>((it.hi - v < HV ? it.hi - v : HV)) * 16u;
      unsigned char* dst = ring + static_cast<size_t>(slot) * kStageBytes;
      mbar_expect_tx(&sh.full[slot], 2u * bytes);
      bulk_load(dst, base + static_cast<long long>(v) * 16, bytes, &sh.full[slot]);
      bulk_load(dst + HV * 16, base + row_step + static_cast<long long>(v) * 16, bytes, &sh.full[slot]);
    }
  }
  return true;
}

// Whether a streaming item goes through the ring (the producer and the streaming warps must agree).
template <int MODE>
__device__ __forceinline__ bool item_uses_ring(const KParams& p) {
  return MODE == kEnsembleSample || p.n == 2;
}

template <int DT, int MODE>
__device__ __forceinline__ bool stream_item(const FParams& fp, const ItemCtx& it, SoftPart* part, int stid, FShared& sh,
                                            const unsigned char* ring, unsigned& k) {
  const KParams& p = fp.k;
  const int lane = stid & 31;
  if (MODE == kEnsembleSample) return stream_ensemble<DT>(fp, it, part, stid, sh, ring, k);
  if (item_uses_ring<MODE>(p)) {
    bool settled = false;
    if (!stream_logit2<DT>(fp, it, part, stid, sh, ring, k, settled)) return false;
    if (settled) return true;
  }
  // any other number of models, and the warps that met an overflow or a non-finite input: from global memory
  const char* base = unit_base(p, it.b, it.j, Elem<DT>::bytes);
  Slice sl;
  sl.v_lo = it.lo;
  sl.v_hi = it.hi;
  sl.e_lo = sl.e_hi = 0;
  LaneSoft accq, accc;
  logit_soft_slice<DT, kST>(p, base, sl, stid, it.pis, false, -INFINITY, accq, accc);
  warp_merge_soft(accq, &part[0], lane);
  warp_merge_soft(accc, &part[1], lane);
  return true;
}

template <int N>
struct RawSet {
  uint4 r[N];
};

// A vector of a drawing sweep that holds a big entry (more than 2^-8 of a normaliser), done again entry by entry from
// the vectors at hand (models beyond those are read again): big entries in fp64 into the thread's slots
// (`bigacc[q * kST]`: q < NCH the normalisers, NCH <= q < 2 NCH the step sums), the others as the sweep does
// them, returned in zs / as.  Rare; out of line.
template <int DT, int MODE, int NCH, int NL>
__device__ __noinline__ void draw_big_vector(const KParams& p, const ItemCtx& c, RawSet<NL> raw, const char* base, int e0,
                                             double* bigacc, float* zs, float* as) {
  constexpr int E = Elem<DT>::E;
  float xs[NL][E];
#pragma unroll
  for (int i = 0; i < NL; ++i) Elem<DT>::unpack(raw.r[i], xs[i]);
  for (int k = 0; k < E; ++k) {
    const int e = e0 + k;
    if (e >= p.V) break;
    float x[NCH];
    double x64[NCH];
    if (MODE == kEnsembleSample) {
      for (int i = 0; i < NCH; ++i) {
        x[i] = xs[i < NL ? i : 0][k];
        x64[i] = static_cast<double>(x[i]);
      }
    } else {
      float xb = 0.f, xa = 0.f;
      double cb = 0.0;
      for (int i = 0; i < p.n; ++i) {
        const float v = (i < NL) ? xs[i][k] : Elem<DT>::load1(base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes, e);
        xb = fmaf(p.w[i], v, xb);
        cb = fma(p.w64[i], static_cast<double>(v), cb);
        if (i == c.pis) xa = v;
      }
      x[0] = xa;
      x[1] = xb;
      x64[0] = static_cast<double>(xa);
      x64[1] = cb;
    }
    float ee[NCH];
    bool big = false;
    for (int i = 0; i < NCH; ++i) {
      ee[i] = ex2_approx(fmaf(x[i], p.cT, c.nref[i]));
      big |= ee[i] > c.bt[i];
    }
    if (big) {
      double d[NCH], tot = 0.0;
      for (int i = 0; i < NCH; ++i) {
        d[i] = exp2(x64[i] * p.cT64 - c.dref[i]);
        tot += c.ct64[i] * d[i];
      }
      for (int i = 0; i < NCH; ++i) {
        bigacc[i * kST] += d[i];
        if (tot > 0.0) bigacc[(NCH + i) * kST] += d[i];
      }
    } else {
      float acc = 0.f;
      for (int i = 0; i < NCH; ++i) acc = __fadd_rn(acc, __fmul_rn(c.ct[i], ee[i]));
      const bool pos = acc > 0.f;
      for (int i = 0; i < NCH; ++i) {
        zs[i] += ee[i];
        as[i] += pos ? ee[i] : 0.f;
      }
    }
  }
}

// One chunk of a drawing sweep.  A token's mass is sum_i k_i e_i / Z_i clipped at zero, with the channels i the
// models (ensemble) or the proposer's and the combined logits (logit level), e_i = 2^(arg_i - ref_i).  Which tokens
// have a positive mass is decided with the normalisers of the streaming pass (products rounded one by one, so that
// r == q gives exactly zero); over those tokens the mass is linear in the 1/Z_i, so the sweep records, per step,
// the sums of e_i over them, and adds up the refined normalisers (terms above 2^-8 of one in fp64).
template <int DT, int MODE, int NCH>
__device__ __forceinline__ void draw_item(const FParams& fp, const ItemCtx& it, SoftPart* part, int stid, double* bigacc) {
  constexpr int E = Elem<DT>::E;
  const KParams& p = fp.k;
  const int lane = stid & 31, warp = stid >> 5;
  const char* base = unit_base(p, it.b, it.j, Elem<DT>::bytes);
  const long long row_step = p.s_model * Elem<DT>::bytes;
  float ct[NCH], nref[NCH], bt[NCH];
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    ct[i] = it.ct[i];
    nref[i] = it.nref[i];
    bt[i] = it.bt[i];
  }
  float zs[NCH], as[NCH];
#pragma unroll
  for (int i = 0; i < NCH; ++i) zs[i] = as[i] = 0.f;
#pragma unroll
  for (int q = 0; q < 2 * NCH; ++q) bigacc[q * kST] = 0.0;
  bool zbig = false;
  constexpr int NL = (MODE == kEnsembleSample) ? NCH : 2;  // rows fetched one step ahead
  const int nl = (MODE == kEnsembleSample) ? NCH : (p.n < 2 ? p.n : 2);
  uint4 nx[NL];
  auto fetch = [&](int s) {
    const int v = s * 32 + lane;
#pragma unroll
    for (int i = 0; i < NL; ++i)
      nx[i] = (v < fp.nvec && i < nl) ? ldg_ahead16(base + i * row_step + static_cast<long long>(v) * 16) : ninf_vec<DT>();
  };
  double* rec = fp.s.srec + static_cast<size_t>(it.b) * p.nsteps * NCH;
#ifdef COS_FUSED_PROFILE
  long long dt0 = clock64(), dt_first = 0;
  unsigned long long dsteps = 0;
#endif
  if (it.lo + warp < it.hi) fetch(it.lo + warp);
  for (int s = it.lo + warp; s < it.hi; s += kSW) {
    uint4 cur[NL];
#pragma unroll
    for (int i = 0; i < NL; ++i) cur[i] = nx[i];
    if (s + kSW < it.hi) fetch(s + kSW);
    const int v = s * 32 + lane;
    float xc[NCH][E];  // channel arguments
    if (MODE == kEnsembleSample) {
#pragma unroll
      for (int i = 0; i < NCH; ++i) Elem<DT>::unpack(cur[i], xc[i]);
    } else {
#pragma unroll
      for (int k = 0; k < E; ++k) xc[1][k] = 0.f;
      auto take = [&](int i, const uint4& raw) {
        float x[E];
        Elem<DT>::unpack(raw, x);
        const float wi = p.w[i];
#pragma unroll
        for (int k = 0; k < E; ++k) {
          xc[1][k] = fmaf(wi, x[k], xc[1][k]);
          if (i == it.pis) xc[0][k] = x[k];
        }
      };
      take(0, cur[0]);
      if (p.n >= 2) take(1, cur[1]);
      for (int i = 2; i < p.n; ++i)
        take(i, v < fp.nvec ? ldg_stream16(base + i * row_step + static_cast<long long>(v) * 16) : ninf_vec<DT>());
      if (v >= fp.nvec) {
#pragma unroll
        for (int k = 0; k < E; ++k) xc[0][k] = xc[1][k] = -INFINITY;
      }
    }
    float vz[NCH], va[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) vz[i] = va[i] = 0.f;
#pragma unroll
    for (int k = 0; k < E; ++k) {
      float e[NCH];
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < NCH; ++i) {
        e[i] = ex2_approx(fmaf(xc[i][k], p.cT, nref[i]));
        vz[i] += e[i];
        acc = __fadd_rn(acc, __fmul_rn(ct[i], e[i]));
      }
      const float in_p = (acc > 0.f) ? 1.f : 0.f;
#pragma unroll
      for (int i = 0; i < NCH; ++i) va[i] = fmaf(in_p, e[i], va[i]);
    }
    bool big = false;
#pragma unroll
    for (int i = 0; i < NCH; ++i) big |= vz[i] > bt[i];
    // rare: the vector may hold a big entry (no term is negative, so a big entry makes its vector's sum big)
    if (big) {
      float rz[NCH], ra[NCH];
      for (int i = 0; i < NCH; ++i) rz[i] = ra[i] = 0.f;
      RawSet<NL> rs;
#pragma unroll
      for (int i = 0; i < NL; ++i) rs.r[i] = cur[i];
      draw_big_vector<DT, MODE, NCH, NL>(p, it, rs, base, v * E, bigacc, rz, ra);
#pragma unroll
      for (int i = 0; i < NCH; ++i) {
        zs[i] += rz[i];
        as[i] = ra[i];
      }
      zbig = true;
    } else {
#pragma unroll
      for (int i = 0; i < NCH; ++i) {
        zs[i] += vz[i];
        as[i] = va[i];
      }
    }
    // the step's sums over the warp
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) as[i] += __shfl_xor_sync(0xffffffffu, as[i], d);
    }
    double da[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) da[i] = static_cast<double>(as[i]);
    if (__any_sync(0xffffffffu, big)) {
#pragma unroll
      for (int i = 0; i < NCH; ++i) {
        double t = bigacc[(NCH + i) * kST];
        bigacc[(NCH + i) * kST] = 0.0;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) t += shfl_double(t, lane ^ d);
        da[i] += t;
      }
    }
    if (lane < NCH) {
      double mine = da[0];
#pragma unroll
      for (int i = 1; i < NCH; ++i) mine = (lane == i) ? da[i] : mine;
      __stcg(rec + static_cast<size_t>(s) * NCH + lane, mine);
    }
#ifdef COS_FUSED_PROFILE
    if (dsteps == 0) dt_first = clock64();
    ++dsteps;
#endif
  }
#ifdef COS_FUSED_PROFILE
  const long long dt_loop = clock64();
#endif
  // this warp's share of the refined normalisers
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    double t = static_cast<double>(zs[i]) + (__any_sync(0xffffffffu, zbig) ? bigacc[i * kST] : 0.0);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) t += shfl_double(t, lane ^ d);
    if (lane == 0) {
      part[i].s = t;
      part[i].ref = 0.f;
    }
  }
#ifdef COS_FUSED_PROFILE
  if (warp == 0 && lane == 0 && dsteps > 0) {
    atomicAdd(&g_prof[8], static_cast<unsigned long long>(dt_first - dt0));   // up to the end of the first step
    atomicAdd(&g_prof[9], static_cast<unsigned long long>(dt_loop - dt_first)); // the other steps
    atomicAdd(&g_prof[10], static_cast<unsigned long long>(clock64() - dt_loop)); // normaliser shares
    atomicAdd(&g_prof[11], dsteps - 1);
    atomicAdd(&g_prof[12], 1ull);
  }
#endif
}

template <int DT, int MODE, int NCH, bool DRAW_ONLY>
__device__ __forceinline__ void stream_role(const FParams& fp, FShared& sh, double* bigacc_all, const unsigned char* ring) {
  const int stid = threadIdx.x, lane = stid & 31, warp = stid >> 5;
  double* bigacc = bigacc_all + stid;
  unsigned k = 0;  // stages of the ring consumed so far
  PROF_DECL;
  PROF_T0;
  for (int seq = 0;; ++seq) {
    const int slot = seq & (kRing - 1);
    // the service warp posts the item; it is normally there already (fetched one ahead)
    int ok = 0;
    if (lane == 0) {
      // (bounded, but longer than the service warp's own patience: when nothing moves it is the one that gives up)
      for (unsigned long long it = 0; it < 8ull * fp.poll_limit; ++it) {
        if (vol_load(&sh.tag[slot]) == seq + 1) {
          ok = 1;
          break;
        }
        if (vol_load(&sh.fault)) break;
        __nanosleep(100);
      }
      __threadfence_block();
      if (ok) atomicMax(&sh.started, seq + 1);
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    PROF_ADD(0);  // waiting for an item
    if (!ok) break;
    __syncwarp();
    const ItemCtx& it = sh.ctx[slot];
    if (it.kind == kItemExit) break;
    if (!DRAW_ONLY && it.kind == kItemStream) {
      if (!stream_item<DT, MODE>(fp, it, &sh.part[slot][warp][0], stid, sh, ring, k)) break;
#ifdef COS_FUSED_PROFILE
      if (warp == 0 && lane == 0) atomicMax(&g_prof[32], prof_now() - g_prof_t0);
#endif
      PROF_ADD(1);
      PROF_COUNT(4);
    } else {
      draw_item<DT, MODE, NCH>(fp, it, &sh.part[slot][warp][0], stid, bigacc);
      PROF_ADD(2);
      PROF_COUNT(5);
    }
    if (it.kind == kItemDraw) __threadfence();  // the step records of a drawing item are read by another block
    __syncwarp();
    if (lane == 0) {
      const bool drop = fp.debug_drop && blockIdx.x == 0 && warp == 0 && seq == 0;  // test hook: a report that never comes
      __threadfence_block();
      if (!drop) atomicAdd(&sh.arrive[slot], 1);
    }
    PROF_ADD(3);  // reporting
  }
  if (warp == 0) PROF_FLUSH(0);
}

// The producer warp: one thread follows the block's items in order and fills the ring with the stages of the
// streaming items, as far ahead of the streaming warps as the ring and the posted items allow (across the change
// from one item to the next, so that the stream never drains).  Drawing items are read by the streaming warps
// themselves.  Before it leaves it makes sure that every copy it issued has landed.
template <int DT, int MODE>
__device__ __forceinline__ void producer_role(const FParams& fp, FShared& sh, unsigned char* ring) {
  if ((threadIdx.x & 31) != 0) return;
  unsigned k = 0;
  for (int seq = 0;; ++seq) {
    const int slot = seq & (kRing - 1);
    bool ok = false;
    for (unsigned long long it = 0; it < 8ull * fp.poll_limit; ++it) {
      if (vol_load(&sh.tag[slot]) == seq + 1) {
        ok = true;
        break;
      }
      if (vol_load(&sh.fault)) break;
      __nanosleep(100);
    }
    if (!ok) break;
    __threadfence_block();
    atomicMax(&sh.started, seq + 1);
    const ItemCtx& it = sh.ctx[slot];
    const int kind = *reinterpret_cast<const volatile int*>(&it.kind);
    if (kind == kItemExit) break;
    if (kind != kItemStream || !item_uses_ring<MODE>(fp.k)) continue;
    if (!produce_item<MODE>(fp, it, sh, ring, k, Elem<DT>::bytes)) break;
  }
  // every stage issued completes its `full` phase when its bytes are in, whoever reads them: wait for the last
  // use of every slot (bounded), so that no copy is in flight when the block's shared memory is given back
  for (unsigned back = 0; back < static_cast<unsigned>(kNST) && back < k; ++back) {
    const unsigned use = k - 1u - back;
    for (unsigned it = 0; it < (1u << 20); ++it)
      if (mbar_try_wait(&sh.full[use % kNST], (use / kNST) & 1u)) break;
  }
}

// ------------------------------------------------------------------------------------
// service warp
// ------------------------------------------------------------------------------------
struct Unif {
  double u_acc, u_smp;
};
__device__ __forceinline__ Unif position_uniforms(const KParams& p, int b, int j) {
  unsigned rnd[4];
  const unsigned long long grow = static_cast<unsigned long long>(p.row_base + b);
  philox4x32_10(static_cast<unsigned>(grow), static_cast<unsigned>(j), offset_lo(p), offset_hi(p), p.seed_lo, p.seed_hi, rnd);
  Unif u;
  u.u_acc = word_to_uniform(rnd[0]);
  u.u_smp = word_to_uniform(rnd[1]);
  return u;
}

__device__ __forceinline__ SoftPart ldcg_part(const SoftPart* q) {
  const int4 raw = __ldcg(reinterpret_cast<const int4*>(q));
  SoftPart o;
  o.s = __hiloint2double(raw.y, raw.x);
  o.ref = __int_as_float(raw.z);
  o.pad = 0;
  return o;
}
__device__ __forceinline__ void stcg_part(SoftPart* q, const SoftPart& v) {
  __stcg(reinterpret_cast<int4*>(q), make_int4(__double2loint(v.s), __double2hiint(v.s), __float_as_int(v.ref), 0));
}

__device__ __forceinline__ void add_events(const FParams& fp, unsigned n) {
  __threadfence();
  atomicAdd(&fp.s.ctr[kCtrEvents], n);
}

// one thread: the drawing items of row b go to the queue
__device__ __forceinline__ void push_draw(const FParams& fp, int b) {
  __threadfence();
  const unsigned at = atomicAdd(&fp.s.ctr[kCtrTail], static_cast<unsigned>(fp.plan.dchunks));
  for (int c = 0; c < fp.plan.dchunks; ++c) {
    const int desc = (kItemDraw << 30) | (b << 8) | c;
    if (at + c < static_cast<unsigned>(fp.plan.dq_cap)) atomicExch(&fp.s.dq[at + c], desc + 1);
  }
}

// Publish a position (Sec. 3.1).  The row's 64-bit word holds four bits per position: published, "the row stops
// here" (rejected, or the bonus position), "reported status bits", "a token can be drawn here".  Every position
// adds its own bits once, so the value the atomic returns tells the publisher whether it was the one that settled
// the row: every position up to the first stop is in.  That publisher writes the row's outputs and queues the
// row's drawing items; positions behind the first stop are still verified but decide nothing.
__device__ __forceinline__ void publish_position(const FParams& fp, int b, int j, int accept, int status, int drawable) {
  const KParams& p = fp.k;
  const bool stop = (!accept) || (j == p.gamma);
  const unsigned long long nib = 1ull | (stop ? 2ull : 0ull) | (status ? 4ull : 0ull) | (drawable ? 8ull : 0ull);
  const unsigned long long mine = nib << (4 * j);
  __threadfence();
  const unsigned long long prev = atomicAdd(&fp.s.row_word[b], mine);
  const unsigned long long total = prev + mine;
  const unsigned long long ones = 0x1111111111111111ull;
  const unsigned long long rowmask = (p.P >= 16) ? ~0ull : ((1ull << (4 * p.P)) - 1ull);
  auto settled = [&](unsigned long long w, int* first_stop) -> bool {
    const unsigned long long stops = (w >> 1) & ones;
    if (stops == 0ull) return false;
    const int fs = (__ffsll(static_cast<long long>(stops)) - 1) >> 2;
    const unsigned long long missing = ~w & ones & rowmask;
    const int fm = missing ? ((__ffsll(static_cast<long long>(missing)) - 1) >> 2) : p.P;
    *first_stop = fs;
    return fs < fm;
  };
  int a = 0, a_prev = 0;
  const bool now = settled(total, &a), before = settled(prev, &a_prev);
  if ((total & ones & rowmask) == (ones & rowmask)) fp.s.row_word[b] = 0ull;  // the row's last position: clean for the next run
  unsigned events = 1;
  if (now && !before) {
    __threadfence();
    unsigned st = 0;
    for (int k = 0; k <= a; ++k)
      if ((total >> (4 * k + 2)) & 1ull) st |= static_cast<unsigned>(__ldcg(&p.unit_res[b * p.P + k]).y);
    const bool can_draw = ((total >> (4 * a + 3)) & 1ull) != 0ull;
    p.accept_count[b] = a;
    int* o = p.out_tokens + static_cast<long long>(b) * p.P;
    for (int k = 0; k < p.P; ++k) o[k] = (k < a) ? p.drafts[b * p.gamma + k] : -1;
    p.row_status[b] = st;
    if (p.bonus_prob != nullptr) p.bonus_prob[b] = __int_as_float(0x7fc00000);
    if (can_draw) {
      const int dkind = (a < p.gamma) ? kDrawResidual : (p.bonus_model >= 0 ? kDrawQ : kDrawR);
      __stcg(&fp.s.row_draw[b], a | (dkind << 8));
      push_draw(fp, b);
    } else {
      events += 1;  // nothing can be drawn (a non-finite position): the row is settled
    }
  }
  add_events(fp, events);
}

// The last chunk of a position has arrived: merge the chunks in order, take the accept test in fp64 (Eq. 6) and
// publish.  Whole warp; `own` (chunks == 1) are the block's merged statistics.
template <int DT, int MODE>
__device__ __forceinline__ void finish_position(const FParams& fp, int b, int j, const SoftPart* own) {
  const KParams& p = fp.k;
  const int lane = threadIdx.x & 31;
  const int ns = fp.plan.nslots, C = fp.plan.chunks;
  const int uidx = b * p.P + j;
  SoftPart fs[kCh > 2 ? kCh : 2];
  for (int k = 0; k < ns; ++k) {
    if (C == 1) {
      fs[k] = own[k];
    } else {
      SoftPart in;
      in.s = 0.0;
      in.ref = -INFINITY;
      if (lane < C) in = ldcg_part(&fp.s.chunk_part[(static_cast<size_t>(uidx) * C + lane) * ns + k]);
      fs[k] = warp_reduce_soft(in.ref, in.s);
    }
  }
  const bool is_bonus = (j == p.gamma);
  const int draft = is_bonus ? 0 : p.drafts[b * p.gamma + j];
  const bool draft_ok = is_bonus || (draft >= 0 && draft < p.V);
  const int pi = proposer_of(p, b, j);
  const bool pi_ok = (pi >= 0 && pi < p.n);
  const char* base = unit_base(p, b, j, Elem<DT>::bytes);
  float ld = 0.f;
  if (lane < p.n && !is_bonus && draft_ok) ld = Elem<DT>::load1(base + static_cast<long long>(lane) * p.s_model * Elem<DT>::bytes, draft);
  const Unif un = position_uniforms(p, b, j);
  const double kNaN = __longlong_as_double(0x7ff8000000000000LL);
  const double kInf = __longlong_as_double(0x7ff0000000000000LL);
  bool finite = pi_ok;
  for (int k = 0; k < ns; ++k) finite = finite && isfinite(fs[k].ref) && isfinite(fs[k].s) && (fs[k].s > 0.0);
  int accept = 0, status = 0;
  double ratio = kNaN, r_d = kNaN, q_d = kNaN;
  if (!finite) {
    status |= COS_ROW_NONFINITE;
  } else if (!is_bonus) {
    if (draft_ok) {
      double rr = 0.0, qq = 0.0;
      if (MODE == kEnsembleSample) {
        for (int i = 0; i < p.n; ++i) {
          const double li = static_cast<double>(__shfl_sync(0xffffffffu, ld, i));
          const double pd = exp2(li * p.cT64 - static_cast<double>(fs[i].ref)) / fs[i].s;
          rr += p.w64[i] * pd;
          if (i == pi) qq = pd;
        }
      } else {
        double cd = 0.0, lq = 0.0;
        for (int i = 0; i < p.n; ++i) {
          const double li = static_cast<double>(__shfl_sync(0xffffffffu, ld, i));
          cd = fma(p.w64[i], li, cd);
          if (i == pi) lq = li;
        }
        rr = exp2(cd * p.cT64 - static_cast<double>(fs[1].ref)) / fs[1].s;
        qq = exp2(lq * p.cT64 - static_cast<double>(fs[0].ref)) / fs[0].s;
      }
      r_d = rr;
      q_d = qq;
      if (qq > 0.0) {
        ratio = rr / qq;
      } else {
        status |= COS_ROW_Q_ZERO;
        ratio = (rr > 0.0) ? kInf : 0.0;
      }
      accept = (un.u_acc <= fmin(1.0, ratio)) ? 1 : 0;
    } else {
      status |= COS_ROW_BAD_DRAFT;
    }
  }
  const int drawable = finite ? 1 : 0;
  if (lane < ns) {
    double sv = fs[0].s;
    float rv = fs[0].ref;
    for (int k = 1; k < ns; ++k) {
      sv = (lane == k) ? fs[k].s : sv;
      rv = (lane == k) ? fs[k].ref : rv;
    }
    __stcg(&p.ustats[uidx].s[lane], sv);
    __stcg(&p.ustats[uidx].ref[lane], rv);
    __threadfence();
  }
  __syncwarp();
  if (lane == 0) {
    if (p.diag) {
      float* d = p.diag + static_cast<long long>(uidx) * 4;
      d[0] = static_cast<float>(ratio);
      d[1] = static_cast<float>(r_d);
      d[2] = static_cast<float>(q_d);
      d[3] = static_cast<float>(kNaN);
    }
    __stcg(&p.unit_res[uidx], make_int4(accept, status, -1, drawable));
    publish_position(fp, b, j, accept, status, drawable);
  }
  __syncwarp();
}

// ---- locating the token of a row once its drawing sweep is complete -------------------------------------------
struct WalkConst {
  double zs[kCh];    // refined normalisers (ensemble: per model; logit level: proposer, combined)
  float ref[kCh];    // reference exponents
  float big_thr[kCh];
  float a_resid[kCh], a_draw[kCh];  // ensemble: coefficient of e_i in r - q, and in the law a bonus token follows
  float inv_zq, inv_zc;             // logit level
  int pis;
  bool draw_q;
};

// Mass of one big token in fp64 from the stored logits: r - q clipped at zero, r, or q.  Rare; out of line.
template <int DT, int MODE>
__device__ __noinline__ double big_token(const KParams& p, const WalkConst& w, const char* base, int e, int draw) {
  if (e >= p.V) return 0.0;
  double r64 = 0.0, q64 = 0.0;
  float lv[COS_MAX_MODELS];
  for (int i = 0; i < p.n; ++i) lv[i] = Elem<DT>::load1(base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes, e);
  if (MODE == kEnsembleSample) {
    for (int i = 0; i < p.n; ++i) {
      const double pr = exp2(static_cast<double>(lv[i]) * p.cT64 - static_cast<double>(w.ref[i])) / w.zs[i];
      r64 += p.w64[i] * pr;
      if (i == w.pis) q64 = pr;
    }
  } else {
    double cd = 0.0;
    for (int i = 0; i < p.n; ++i) cd = fma(p.w64[i], static_cast<double>(lv[i]), cd);
    r64 = exp2(cd * p.cT64 - static_cast<double>(w.ref[1])) / w.zs[1];
    q64 = exp2(static_cast<double>(lv[w.pis]) * p.cT64 - static_cast<double>(w.ref[0])) / w.zs[0];
  }
  return draw == kDrawR ? r64 : (draw == kDrawQ ? q64 : fmax(0.0, r64 - q64));
}

// fp32 masses of the E tokens of one lane of a step (products rounded one by one, so that r == q cancels exactly);
// tokens holding more than 2^-8 of a normaliser are flagged in `bigbits` and get mass 0 here.
template <int DT, int MODE>
__device__ __forceinline__ void token_masses(const KParams& p, const WalkConst& w, const char* base, int e0, bool use_r,
                                             float (&mass32)[Elem<DT>::E], unsigned& bigbits) {
  constexpr int E = Elem<DT>::E;
  float acc[E];
  bool anybig = false;
  bigbits = 0u;
#pragma unroll
  for (int k = 0; k < E; ++k) acc[k] = 0.f;
  if (MODE == kEnsembleSample) {
    for (int i = 0; i < p.n; ++i) {
      float v[E];
      load_chunk<DT>(base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes, e0, p.V, true, v);
      const float co = use_r ? w.a_draw[i] : w.a_resid[i], rf = -w.ref[i];
      float emax = 0.f;
#pragma unroll
      for (int k = 0; k < E; ++k) {
        const float e = ex2_approx(fmaf(v[k], p.cT, rf));
        emax = fmaxf(emax, e);
        acc[k] = __fadd_rn(acc[k], __fmul_rn(co, e));
        bigbits |= (e > w.big_thr[i]) ? (1u << k) : 0u;
      }
      anybig |= emax > w.big_thr[i];
    }
  } else {
    float cmb[E], eq[E];
#pragma unroll
    for (int k = 0; k < E; ++k) cmb[k] = eq[k] = 0.f;
    for (int i = 0; i < p.n; ++i) {
      float v[E];
      load_chunk<DT>(base + static_cast<long long>(i) * p.s_model * Elem<DT>::bytes, e0, p.V, true, v);
      const float wi = p.w[i];
#pragma unroll
      for (int k = 0; k < E; ++k) {
        cmb[k] = fmaf(wi, v[k], cmb[k]);
        if (i == w.pis) eq[k] = ex2_approx(fmaf(v[k], p.cT, -w.ref[0]));
      }
    }
    const bool from_q = use_r && w.draw_q;
    const float qco = use_r ? 0.f : w.inv_zq;
#pragma unroll
    for (int k = 0; k < E; ++k) {
      const bool in = (e0 + k < p.V);
      const float ec = in ? ex2_approx(fmaf(cmb[k], p.cT, -w.ref[1])) : 0.f;
      const float eqk = in ? eq[k] : 0.f;
      const float rr = ec * w.inv_zc;
      acc[k] = from_q ? __fmul_rn(eqk, w.inv_zq) : __fsub_rn(rr, __fmul_rn(eqk, qco));
      const bool big = (ec > w.big_thr[1]) || (eqk > w.big_thr[0]);
      bigbits |= big ? (1u << k) : 0u;
      anybig |= big;
    }
  }
#pragma unroll
  for (int k = 0; k < E; ++k) mass32[k] = ((bigbits >> k) & 1u) ? 0.f : fmaxf(0.f, acc[k]);
  if (!anybig) bigbits = 0u;
}

// The token inside one step: `before` is the mass in front of the step.  An fp64 prefix over the lanes, then the
// lane's tokens one by one.  Whole warp; returns the token (or the step's last token with mass).
template <int DT, int MODE>
__device__ __forceinline__ int walk_step(const KParams& p, const WalkConst& w, const char* base, int step, double before,
                                         double target, bool use_r) {
  constexpr int E = Elem<DT>::E;
  const int lane = threadIdx.x & 31;
  const int e0 = (step * 32 + lane) * E;
  const int draw = use_r ? (w.draw_q ? kDrawQ : kDrawR) : kDrawResidual;
  float mass32[E];
  unsigned bigbits;
  token_masses<DT, MODE>(p, w, base, e0, use_r, mass32, bigbits);
  double m64[E];
#pragma unroll
  for (int k = 0; k < E; ++k) m64[k] = static_cast<double>(mass32[k]);
  float ls = 0.f;
#pragma unroll
  for (int k = 0; k < E; ++k) ls += mass32[k];
  double own = static_cast<double>(ls);
  if (bigbits) {
    for (int k = 0; k < E; ++k)
      if (bigbits & (1u << k)) {
        m64[k] = big_token<DT, MODE>(p, w, base, e0 + k, draw);
        own += m64[k];
      }
  }
  double inc = own;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const double o = shfl_up_double(inc, d);
    if (lane >= d) inc += o;
  }
  double excl = shfl_up_double(inc, 1);
  if (lane == 0) excl = 0.0;
  const double incl = excl + own;
  const bool hit = (own > 0.0) && (before + incl >= target);
  const unsigned hits = __ballot_sync(0xffffffffu, hit);
  const unsigned pos_lanes = __ballot_sync(0xffffffffu, own > 0.0);
  if (hits == 0u && pos_lanes == 0u) return -1;
  const int src = hits ? (__ffs(hits) - 1) : (31 - __clz(pos_lanes));
  int found = -1;
  if (lane == src) {
    double part = 0.0;
    int lastk = -1;
#pragma unroll
    for (int k = 0; k < E; ++k) {
      part += m64[k];
      if (m64[k] > 0.0) {
        lastk = k;
        if (found < 0 && before + (excl + part) >= target) found = e0 + k;
      }
    }
    if (found < 0) found = e0 + lastk;
  }
  return __shfl_sync(0xffffffffu, found, src);
}

// The drawing sweep of row b is complete.  Whole warp.
constexpr int kLocBufSteps = 2048;  // steps whose masses fit the locating warp's buffer in shared memory (16 KB)

template <int DT, int MODE, int NCH>
__device__ __forceinline__ void locate_token(const FParams& fp, int b, double* mbuf = nullptr) {
  const KParams& p = fp.k;
  const int lane = threadIdx.x & 31;
  const int rd = __ldcg(&fp.s.row_draw[b]);
  const int j = rd & 0xff, dkind = rd >> 8;
  const int uidx = b * p.P + j;
  const bool is_bonus = (j == p.gamma);
  const int pis = proposer_of(p, b, j);
  const char* base = unit_base(p, b, j, Elem<DT>::bytes);
#ifdef COS_FUSED_PROFILE
  unsigned long long lt0 = prof_now();
#define LOC_STAMP(k) do { const unsigned long long t_ = prof_now(); if (lane == 0) atomicAdd(&g_prof[k], t_ - lt0); lt0 = t_; } while (0)
#else
#define LOC_STAMP(k)
#endif
  WalkConst w;
  w.pis = pis;
  w.draw_q = (dkind == kDrawQ);
  double coef[NCH];
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    double z = 0.0;
    for (int c = 0; c < fp.plan.dchunks; ++c) z += __ldcg(&fp.s.dzpart[(static_cast<size_t>(b) * fp.plan.dchunks + c) * NCH + i]);
    w.zs[i] = z;
    w.ref[i] = __ldcg(&p.ustats[uidx].ref[i]);
    w.big_thr[i] = static_cast<float>(__ldcg(&p.ustats[uidx].s[i]) * kBigShare);  // from the first estimate, as in the sweep
    coef[i] = channel_k<MODE>(p, i, pis, dkind) / z;
  }
  if (MODE == kEnsembleSample) {
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const double a = p.w64[i] / w.zs[i];
      const double sel = (i == pis) ? 1.0 / w.zs[i] : 0.0;
      w.a_resid[i] = static_cast<float>(a - sel);
      w.a_draw[i] = w.draw_q ? static_cast<float>(sel) : static_cast<float>(a);
    }
  } else {
    w.inv_zq = static_cast<float>(1.0 / w.zs[0]);
    w.inv_zc = static_cast<float>(1.0 / w.zs[1]);
  }
  // Every step's channel sums turn into its mass (products rounded one by one: equal sums under opposite
  // coefficients cancel exactly).  Steps are taken 32 at a time (lane l has step 32 t + l, so the records are read
  // coalesced); an inclusive scan over the lanes and a running total over the tiles give the mass in front of every
  // step.  First pass: the total S.  Second pass, same arithmetic: the first step whose running total reaches u S.
  const double* rec = fp.s.srec + static_cast<size_t>(b) * p.nsteps * NCH;
  auto step_mass = [&](int st) {
    if (st >= p.nsteps) return 0.0;
    double acc = __dmul_rn(coef[0], __ldcg(rec + static_cast<size_t>(st) * NCH));
#pragma unroll
    for (int i = 1; i < NCH; ++i) acc = __dadd_rn(acc, __dmul_rn(coef[i], __ldcg(rec + static_cast<size_t>(st) * NCH + i)));
    return fmax(0.0, acc);
  };
  auto scan32 = [&](double m) {
    double incl = m;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const double o = shfl_up_double(incl, d);
      if (lane >= d) incl += o;
    }
    return incl;
  };
  LOC_STAMP(26);
  const int ntiles = (p.nsteps + 31) / 32;
  // With a buffer in shared memory (the locating warp has one) the masses are computed once, with nothing between
  // the loads of a lane, and the search runs on shared memory; without one the second pass reads the records again.
  const bool buffered = (mbuf != nullptr) && (p.nsteps <= kLocBufSteps);
  double mine = 0.0;
  if (buffered) {
#pragma unroll 8
    for (int t = 0; t < ntiles; ++t) {
      const double m = step_mass(t * 32 + lane);
      mbuf[t * 32 + lane] = m;
      mine += m;
    }
    __syncwarp();
  } else {
#pragma unroll 8
    for (int t = 0; t < ntiles; ++t) mine += step_mass(t * 32 + lane);
  }
  double S = mine;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) S += shfl_double(S, lane ^ d);
  LOC_STAMP(27);
  const Unif un = position_uniforms(p, b, j);
  const double target = un.u_smp * S;
  int step = -1, last = -1;
  double step_base = 0.0, last_base = 0.0, run = 0.0;
  for (int t = 0; t < ntiles && step < 0; ++t) {
    const int st = t * 32 + lane;
    const double m = buffered ? mbuf[st] : step_mass(st);
    const double incl = scan32(m);
    const double before = run + (incl - m);
    const unsigned hit = __ballot_sync(0xffffffffu, m > 0.0 && before + m >= target);
    const unsigned mass = __ballot_sync(0xffffffffu, m > 0.0);
    if (hit) {
      const int src = __ffs(hit) - 1;
      step = t * 32 + src;
      step_base = shfl_double(before, src);
    } else if (mass) {
      const int src = 31 - __clz(mass);
      last = t * 32 + src;
      last_base = shfl_double(before, src);
    }
    run += shfl_double(incl, 31);
  }
  if (step < 0 && last >= 0 && S > 0.0) {  // rounding corner: the last step with mass
    step = last;
    step_base = last_base;
  }
  LOC_STAMP(28);
  if (lane == 0 && p.diag && dkind == kDrawResidual)
    p.diag[static_cast<long long>(uidx) * 4 + 3] = static_cast<float>(S);
  if (step >= 0) {
    const bool use_r = (dkind != kDrawResidual);
    const int token = walk_step<DT, MODE>(p, w, base, step, step_base, target, use_r);
    LOC_STAMP(29);
    if (lane == 0) {
      p.out_tokens[uidx] = token;
      // Algorithm 2's Score returns the bonus token with its probability under the law it came from
      if (is_bonus && p.bonus_prob != nullptr && token >= 0)
        p.bonus_prob[b] = static_cast<float>(big_token<DT, MODE>(p, w, base, token, w.draw_q ? kDrawQ : kDrawR));
      add_events(fp, 1);
    }
  } else if (dkind == kDrawResidual) {
    // a token is needed although max(0, r - q) has no mass: the row draws from r instead, with the same uniform
    if (lane == 0) {
      atomicOr(&p.row_status[b], static_cast<unsigned>(COS_ROW_RESIDUAL_EMPTY));
      __stcg(&fp.s.row_draw[b], j | (kDrawR << 8));
      push_draw(fp, b);
    }
  } else {
    if (lane == 0) add_events(fp, 1);  // nothing to draw from: the row keeps -1
  }
  __syncwarp();
  LOC_STAMP(30);
#undef LOC_STAMP
}

__device__ __forceinline__ uint2 vol_load2(const unsigned* p) {
  uint2 v;
  asm volatile("ld.volatile.global.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}

// One thread: the next item of this block, or -1.  Drawing items first (their logits are still in L2).
// The queue hands out tickets: a block that sees entries beyond the head takes the next ticket with one atomic
// add.  Under a race the ticket may lie beyond the tail; it then names the entry this block takes as soon as
// somebody writes it (`ticket` is kept across calls; a block holds one ticket at most).  Nobody spins on the
// queue, and every entry has exactly one taker, who cannot leave before the run is complete.
__device__ __forceinline__ int take_item(const FParams& fp, int num_items, bool& static_left, int& ticket) {
  if (ticket < 0) {
    const uint2 ht = vol_load2(&fp.s.ctr[kCtrHead]);  // head, tail
    if (ht.y > ht.x) ticket = static_cast<int>(atomicAdd(&fp.s.ctr[kCtrHead], 1u));
  }
  if (ticket >= 0 && ticket < fp.plan.dq_cap) {
    const int v = vol_load(&fp.s.dq[ticket]);
    if (v != 0) {
      fp.s.dq[ticket] = 0;  // clean for the next run
      ticket = -1;
      __threadfence();
      return v - 1;
    }
  }
  if (static_left) {
    const unsigned t = atomicAdd(&fp.s.ctr[kCtrNext], 1u);
    if (t < static_cast<unsigned>(num_items)) {
      if (fp.draw_only) {
        const int job = static_cast<int>(t) / fp.plan.dchunks, c = static_cast<int>(t) % fp.plan.dchunks;
        return (kItemJob << 30) | (job << 8) | c;
      }
      const int unit = static_cast<int>(t) / fp.plan.chunks, c = static_cast<int>(t) % fp.plan.chunks;
      return (kItemStream << 30) | (unit << 8) | c;
    }
    static_left = false;
  }
  return -1;
}

template <int MODE>
__device__ __forceinline__ void fill_ctx(const FParams& fp, ItemCtx& cx, int desc) {
  const KParams& p = fp.k;
  const int lane = threadIdx.x & 31;
  const int kind = (desc >> 30) & 3, id = (desc >> 8) & 0x3fffff, c = desc & 0xff;
  if (kind == kItemStream) {
    // Row-major order: a row's positions one after the other.  A row settles as soon as the position of its first
    // rejection is decided (the earlier ones came before it), while its later positions are still being streamed.
    // (Position-major over the batch, and over groups of 32 rows, measured 10 % slower on workloads 3 and 4.)
    const int b = id / p.P, j = id % p.P;
    if (lane == 0) {
      cx.kind = kItemStream;
      cx.b = b;
      cx.j = j;
      cx.chunk = c;
      // (only the logit-level sweep needs to know whose distribution q is; the decision looks it up itself)
      const int pi = (MODE == kLogitSample) ? proposer_of(p, b, j) : 0;
      cx.pis = (pi >= 0 && pi < p.n) ? pi : 0;
      const int lo = c * fp.plan.chunk_steps * 32, hi = lo + fp.plan.chunk_steps * 32;
      cx.lo = lo;
      cx.hi = hi < fp.nvec ? hi : fp.nvec;
    }
  } else {
    int b = id, j, dkind;
    if (kind == kItemJob) {
      // the id-th entry of the job list an earlier launch left: the one position of its row that draws a token
      const int idx = __ldcg(&p.jobs[id]).x;
      b = idx / p.P;
      j = idx % p.P;
      dkind = (j < p.gamma) ? kDrawResidual : (p.bonus_model >= 0 ? kDrawQ : kDrawR);
      if (lane == 0) __stcg(&fp.s.row_draw[b], j | (dkind << 8));  // every chunk of the row writes the same word
    } else {
      const int rd = __ldcg(&fp.s.row_draw[b]);
      j = rd & 0xff;
      dkind = rd >> 8;
    }
    const int pis = proposer_of(p, b, j);
    const int uidx = b * p.P + j;
    if (lane == 0) {
      cx.kind = kItemDraw;
      cx.b = b;
      cx.j = j;
      cx.chunk = c;
      cx.pis = pis;
      cx.dkind = dkind;
      const int lo = c * fp.plan.dchunk_steps, hi = lo + fp.plan.dchunk_steps;
      cx.lo = lo;
      cx.hi = hi < p.nsteps ? hi : p.nsteps;
    }
    if (lane < fp.plan.nch) {
      const double z0 = __ldcg(&p.ustats[uidx].s[lane]);
      const float ref = __ldcg(&p.ustats[uidx].ref[lane]);
      const double c64 = channel_k<MODE>(p, lane, pis, dkind) / z0;  // with the first estimates: signs only
      cx.ct64[lane] = c64;
      cx.ct[lane] = static_cast<float>(c64);
      cx.nref[lane] = -ref;
      cx.dref[lane] = static_cast<double>(ref);
      cx.bt[lane] = static_cast<float>(z0 * kBigShare);
    }
  }
  __syncwarp();
}

constexpr int kLocateChunk = 0xff;  // a queue entry with this chunk number asks for a row's token to be located

// Service warp: hand row b to this block's locating warp if that warp has nothing else to do.  Whole warp.
__device__ __forceinline__ bool hand_to_locator(FShared& sh, int b, int lane) {
  int ok = 0;
  if (lane == 0) {
    const int tail = vol_load(&sh.loc_tail), head = vol_load(&sh.loc_head);
    if (tail == head) {
      *reinterpret_cast<volatile int*>(&sh.loc_ring[tail & 7]) = b;
      __threadfence_block();
      *reinterpret_cast<volatile int*>(&sh.loc_tail) = tail + 1;
      ok = 1;
    }
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

template <int DT, int MODE, int NCH, bool DRAW_ONLY>
__device__ __forceinline__ void service_role(const FParams& fp, FShared& sh) {
  const KParams& p = fp.k;
  const int lane = threadIdx.x & 31;
  int fetched = 0, processed = 0;
  bool static_left = true;
  int ticket = -1;
  unsigned idle = 0;
  bool failed = false;
  // Looking for work reads two lines of L2 that every block shares.  A block that found nothing looks again only
  // after a pause that grows with every empty look (to a few loop turns): hundreds of blocks asking every 100 ns keep one
  // L2 slice so busy that every load of the device that maps to it waits behind them.
  unsigned empty_looks = 0, skip = 0;
#ifdef COS_FUSED_PROFILE
  const unsigned long long t_begin = prof_now();
  bool stamped = false;
#endif
  PROF_DECL;
  PROF_T0;
  while (true) {
    bool did = false;
    // ---- fetch up to two items ahead of the fastest of the streaming and producer warps
    if (skip > 0) --skip;
    // (and where items are few and short, no block should sit on work another block is idle for)
    if (skip == 0 && fetched < processed + kRing && fetched <= vol_load(&sh.started) + (DRAW_ONLY ? 0 : 1)) {
      int desc = -1;
      if (lane == 0) desc = take_item(fp, sh.num_items, static_left, ticket);
      desc = __shfl_sync(0xffffffffu, desc, 0);
      static_left = __shfl_sync(0xffffffffu, static_left ? 1 : 0, 0) != 0;
      if (desc != -1 && ((desc >> 30) & 3) == kItemDraw && (desc & 0xff) == kLocateChunk) {
        // a row whose sweep is complete, passed on by a block whose locating warp was busy
        const int b = (desc >> 8) & 0x3fffff;
        if (!hand_to_locator(sh, b, lane)) locate_token<DT, MODE, NCH>(fp, b);
        did = true;
        empty_looks = 0;
      } else if (desc != -1) {
        PROF_ADD(0);  // taking an item
        fill_ctx<MODE>(fp, sh.ctx[fetched & (kRing - 1)], desc);
        PROF_ADD(1);
        if (lane == 0) {
          __threadfence_block();
          *reinterpret_cast<volatile int*>(&sh.tag[fetched & (kRing - 1)]) = fetched + 1;
        }
        ++fetched;
        did = true;
        empty_looks = 0;
      } else {
#ifdef COS_FUSED_PROFILE
        if (!stamped && !static_left && lane == 0) atomicMax(&g_prof[13], prof_now() - t_begin);
        if (!static_left) stamped = true;
#endif
        empty_looks = empty_looks < 4 ? empty_looks + 1 : 4;
        skip = empty_looks;  // loop turns (each sleeps 100 to 200 ns, in practice rather more)
      }
      if (desc == -1 && processed == fetched) {
        // nothing open here and nothing to take: done once every position is published and every row settled
        unsigned ev = 0;
        if (lane == 0) ev = vol_load(&fp.s.ctr[kCtrEvents]);
        ev = __shfl_sync(0xffffffffu, ev, 0);
        if (ev >= sh.total_events) break;
      }
    }
    // ---- the oldest open item, once every streaming warp has reported it
    if (processed < fetched) {
      const int slot = processed & (kRing - 1);
      int in = 0;
      if (lane == 0) in = vol_load(&sh.arrive[slot]);
      in = __shfl_sync(0xffffffffu, in, 0);
      if (in == kSW) {
        __threadfence_block();
        const ItemCtx& cx = sh.ctx[slot];
        const int b = cx.b, j = cx.j, c = cx.chunk;
        if (!DRAW_ONLY && cx.kind == kItemStream) {
          const int ns = fp.plan.nslots, C = fp.plan.chunks;
          const int uidx = b * p.P + j;
          SoftPart merged[kCh > 2 ? kCh : 2];
          for (int k = 0; k < ns; ++k) {
            const float ref = (lane < kSW) ? sh.part[slot][lane][k].ref : -INFINITY;
            const double s = (lane < kSW) ? sh.part[slot][lane][k].s : 0.0;
            merged[k] = warp_reduce_soft(ref, s);
          }
          bool last = true;
          if (C > 1) {
            int prev = 0;
            if (lane == 0) {
              for (int k = 0; k < ns; ++k) stcg_part(&fp.s.chunk_part[(static_cast<size_t>(uidx) * C + c) * ns + k], merged[k]);
              __threadfence();
              prev = atomicAdd(&fp.s.unit_arrivals[uidx], 1);
              if (prev == C - 1) {
                fp.s.unit_arrivals[uidx] = 0;  // clean for the next run
                __threadfence();
              }
            }
            prev = __shfl_sync(0xffffffffu, prev, 0);
            last = (prev == C - 1);
          }
          PROF_ADD(2);  // a streaming chunk reported
          if (last) {
            finish_position<DT, MODE>(fp, b, j, merged);
#ifdef COS_FUSED_PROFILE
            if (lane == 0) atomicMax(&g_prof[33], prof_now() - g_prof_t0);
#endif
            PROF_ADD(3);
            PROF_COUNT(8);
          }
        } else {
          // this block's share of the refined normalisers; the last chunk of the row locates the token
          for (int i = 0; i < NCH; ++i) {
            double t = (lane < kSW) ? sh.part[slot][lane][i].s : 0.0;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) t += shfl_double(t, lane ^ d);
            if (lane == 0) __stcg(&fp.s.dzpart[(static_cast<size_t>(b) * fp.plan.dchunks + c) * NCH + i], t);
          }
          int prev = 0;
          if (lane == 0) {
            __threadfence();
            prev = atomicAdd(&fp.s.draw_arrivals[b], 1);
            if (prev == fp.plan.dchunks - 1) {
              fp.s.draw_arrivals[b] = 0;
              __threadfence();
            }
          }
          prev = __shfl_sync(0xffffffffu, prev, 0);
#ifdef COS_FUSED_PROFILE
          if (lane == 0) atomicMax(&g_prof[34], prof_now() - g_prof_t0);
#endif
          PROF_ADD(4);  // a drawing chunk reported
          if (prev == fp.plan.dchunks - 1) {
            // the row's sweep is complete: its token is located by the block's locating warp, so that this warp
            // stays free to report other chunks; if that warp is busy the row goes to the queue, for any block to take
            bool handed = false;
            {
              handed = hand_to_locator(sh, b, lane);
              if (!handed) {
                if (lane == 0) {
                  __threadfence();
                  const unsigned at = atomicAdd(&fp.s.ctr[kCtrTail], 1u);
                  if (at < static_cast<unsigned>(fp.plan.dq_cap)) atomicExch(&fp.s.dq[at], ((kItemDraw << 30) | (b << 8) | kLocateChunk) + 1);
                }
                handed = true;
              }
            }
            if (!handed) locate_token<DT, MODE, NCH>(fp, b);
            PROF_ADD(5);
            PROF_COUNT(9);
          }
        }
        if (lane == 0) {
          *reinterpret_cast<volatile int*>(&sh.arrive[slot]) = 0;
          __threadfence_block();
        }
        ++processed;
        did = true;
      }
    }
    if (did) {
      idle = 0;
    } else {
      PROF_ADD(processed < fetched ? 6 : 7);  // waiting for the streaming warps / for work
      if (++idle > fp.poll_limit) {
        failed = true;
        break;
      }
      __nanosleep(processed < fetched ? 100 : 200);
    }
  }
  if (failed) {
    // no progress anywhere for the whole limit (a defect, never the data): mark every row, let everybody leave
    if (lane == 0) {
      *reinterpret_cast<volatile int*>(&sh.fault) = 1;
      atomicExch(&fp.s.ctr[kCtrFault], 1u);
    }
    for (int b = lane; b < p.B; b += 32) atomicOr(&p.row_status[b], static_cast<unsigned>(COS_ROW_FAULT));
  }
  PROF_FLUSH(16);
#ifdef COS_FUSED_PROFILE
  if (lane == 0) atomicMax(&g_prof[14], prof_now() - t_begin);
#endif
  // tell the streaming warps (and the locating warp) to leave
  if (lane == 0) {
    *reinterpret_cast<volatile int*>(&sh.loc_exit) = 1;
    ItemCtx& cx = sh.ctx[fetched & (kRing - 1)];
    cx.kind = kItemExit;
    __threadfence_block();
    *reinterpret_cast<volatile int*>(&sh.tag[fetched & (kRing - 1)]) = fetched + 1;
    // the last block to leave puts the counters back: every run starts from the same state
    __threadfence();
    const unsigned gone = atomicAdd(&fp.s.ctr[kCtrGone], 1u);
    if (gone == gridDim.x - 1) {
      const bool faulted = vol_load(&fp.s.ctr[kCtrFault]) != 0u;
      fp.s.ctr[kCtrNext] = 0u;
      fp.s.ctr[kCtrEvents] = 0u;
      fp.s.ctr[kCtrHead] = 0u;
      fp.s.ctr[kCtrTail] = 0u;
      fp.s.ctr[kCtrGone] = 0u;
      fp.s.ctr[kCtrFault] = faulted ? 2u : 0u;  // 2: the scratch may be dirty; the host clears it before the next run
      if (fp.draw_only) {  // what the staged launches leave clean for the next run
        *fp.k.job_count = 0;
        *fp.k.work_counter = 0u;
      }
      __threadfence();
    }
  }
}

// DRAW_ONLY: the launch that only draws tokens (after a staged launch published the positions); it is compiled
// without the streaming code.  One block per multiprocessor in both forms: the drawing sweep then keeps its working
// set in registers, and the ring of stages, not the number of resident warps, keeps the stream going.
template <int DT, int MODE, int NCH, bool DRAW_ONLY>
__global__ void __launch_bounds__(kFT, 1) cos_fused_kernel(const __grid_constant__ FParams fp) {
  __shared__ FShared sh;
  // dynamic shared memory: [2 * NCH][kST] fp64 sums of the big terms of a drawing sweep (one slot per thread), the
  // locating warp's buffer of step masses, then (one-launch form) the ring of kNST stages the producer fills
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  double* bigacc = reinterpret_cast<double*>(dyn_smem);
  double* locbuf = reinterpret_cast<double*>(dyn_smem + ((2 * NCH * kST * sizeof(double) + 127) / 128) * 128);
  unsigned char* ring = reinterpret_cast<unsigned char*>(locbuf + kLocBufSteps);
  const int tid = threadIdx.x;
  if (tid < kRing) {
    sh.tag[tid] = 0;
    sh.arrive[tid] = 0;
  }
  if (tid == 0) {
    for (int q = 0; q < kNST; ++q) {
      mbar_init(&sh.full[q], 1);       // the producer's arrival, with the bytes it announces
      mbar_init(&sh.empty[q], kSW);    // one arrival per streaming warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // (after a launch that published the positions: started while it drained; nothing it wrote is read before this)
  if (fp.draw_only) asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef COS_FUSED_PROFILE
  if (tid == 0 && blockIdx.x == 0) g_prof_t0 = prof_now();
#endif
  if (tid == 0) {
    sh.started = 0;
    sh.fault = 0;
    sh.loc_tail = sh.loc_head = sh.loc_exit = 0;
    if (fp.draw_only) {
      int njobs = __ldcg(fp.k.job_count);
      njobs = njobs < fp.k.max_jobs ? njobs : fp.k.max_jobs;
      sh.num_items = njobs * fp.plan.dchunks;
      sh.total_events = static_cast<unsigned>(njobs);
    } else {
      sh.num_items = fp.num_items;
      sh.total_events = fp.total_events;
    }
  }
  __syncthreads();
  const int role = tid >> 5;
  if (role < kSW) {
    stream_role<DT, MODE, NCH, DRAW_ONLY>(fp, sh, bigacc, ring);
  } else if (role == kSvcWarp) {
    service_role<DT, MODE, NCH, DRAW_ONLY>(fp, sh);
  } else if (role == kProdWarp) {
    if (!DRAW_ONLY) producer_role<DT, MODE>(fp, sh, ring);
  } else {
    // the locating warp: rows in the order the service warp hands them over
    const int lane = tid & 31;
    int head = 0;
    for (unsigned long long it = 0; it < 16ull * fp.poll_limit; ++it) {
      int tail = 0, leave = 0;
      if (lane == 0) {
        tail = vol_load(&sh.loc_tail);
        leave = vol_load(&sh.loc_exit) | vol_load(&sh.fault);
      }
      tail = __shfl_sync(0xffffffffu, tail, 0);
      leave = __shfl_sync(0xffffffffu, leave, 0);
      if (head < tail) {
        __syncwarp();
        const int b = vol_load(&sh.loc_ring[head & 7]);
#ifdef COS_FUSED_PROFILE
        const unsigned long long tl0 = prof_now();
#endif
        locate_token<DT, MODE, NCH>(fp, b, locbuf);
#ifdef COS_FUSED_PROFILE
        if (lane == 0) {
          atomicMax(&g_prof[35], prof_now() - g_prof_t0);
          atomicAdd(&g_prof[7], prof_now() - tl0);
          atomicAdd(&g_prof[15], 1ull);
        }
#endif
        ++head;
        if (lane == 0) {
          __threadfence_block();
          *reinterpret_cast<volatile int*>(&sh.loc_head) = head;
        }
        it = 0;
      } else if (leave) {
        break;
      } else {
        __nanosleep(100);
      }
    }
  }
}

using FusedFn = void (*)(const FParams);

template <int DT, bool DRAW_ONLY>
FusedFn pick_dt(int mode, int n) {
  if (mode == kLogitSample) return cos_fused_kernel<DT, kLogitSample, 2, DRAW_ONLY>;
  if (mode == kEnsembleSample) {
    if (n == 1) return cos_fused_kernel<DT, kEnsembleSample, 1, DRAW_ONLY>;
    if (n == 2) return cos_fused_kernel<DT, kEnsembleSample, 2, DRAW_ONLY>;
    if (n == 3) return cos_fused_kernel<DT, kEnsembleSample, 3, DRAW_ONLY>;
    if (n == 4) return cos_fused_kernel<DT, kEnsembleSample, 4, DRAW_ONLY>;
  }
  return nullptr;
}

FusedFn pick_fused(int dtype, int mode, int n, bool draw_only = false) {
  if (draw_only) {
    if (dtype == COS_DTYPE_F32) return pick_dt<COS_DTYPE_F32, true>(mode, n);
    if (dtype == COS_DTYPE_BF16) return pick_dt<COS_DTYPE_BF16, true>(mode, n);
    if (dtype == COS_DTYPE_F16) return pick_dt<COS_DTYPE_F16, true>(mode, n);
    return nullptr;
  }
  if (dtype == COS_DTYPE_F32) return pick_dt<COS_DTYPE_F32, false>(mode, n);
  if (dtype == COS_DTYPE_BF16) return pick_dt<COS_DTYPE_BF16, false>(mode, n);
  if (dtype == COS_DTYPE_F16) return pick_dt<COS_DTYPE_F16, false>(mode, n);
  return nullptr;
}

int channels_of(int mode, int n) { return mode == kEnsembleSample ? n : 2; }
size_t fused_smem(int mode, int n, bool draw_only) {
  const size_t big = ((static_cast<size_t>(2 * channels_of(mode, n)) * kST * sizeof(double) + 127) / 128) * 128;
  return big + kLocBufSteps * sizeof(double) + (draw_only ? 0 : static_cast<size_t>(kNST) * kStageBytes);
}

}  // namespace

#ifdef COS_FUSED_PROFILE
extern "C" int cos_fused_profile_read(unsigned long long* out32, int reset) {  // 48 words
  if (cudaMemcpyFromSymbol(out32, g_prof, sizeof(g_prof)) != cudaSuccess) return -1;
  if (reset) {
    unsigned long long z[48] = {0};
    if (cudaMemcpyToSymbol(g_prof, z, sizeof(z)) != cudaSuccess) return -1;
  }
  return 0;
}
#endif

namespace cosv {

bool fused_covers(int dtype, int mode, int n, int vocab, int gamma, int mask_model, long long max_units) {
  if (mode != kEnsembleSample && mode != kLogitSample) return false;
  if (mode == kEnsembleSample && n > kCh) return false;
  if (mask_model >= 0) return false;
  if (gamma + 1 > 16) return false;            // four bits per position in the row's word
  if (max_units > 0x3fffffLL) return false;    // item descriptors keep 22 bits for the position
  const int E = (dtype == COS_DTYPE_F32) ? 4 : 8;
  if (vocab % E != 0) return false;            // whole 16-byte vectors only
  return pick_fused(dtype, mode, n) != nullptr;
}

FusedPlan fused_plan(int dtype, int mode, int n, int vocab, int gamma, int max_batch, int sm_count, int blocks_per_sm) {
  FusedPlan pl;
  const int E = (dtype == COS_DTYPE_F32) ? 4 : 8;
  const int nvec = vocab / E;
  const int nsteps = (nvec + 31) / 32;
  // Streaming chunks.  A whole position per item where that still gives every block several items (one report to the
  // other blocks less per item); else just enough chunks of at least 256 KB (over all models) to give the persistent
  // blocks about four items each; 32 chunks at most, whole stages of the ring.
  const long long step_bytes = 512LL * n;
  const long long dchunk_kb = 64;
  const long long units = static_cast<long long>(max_batch) * (gamma + 1);
  const long long blocks_ll = sm_count;
  int chunks = 1;
  if (units * 2 < 7 * blocks_ll) {
    chunks = static_cast<int>((7 * blocks_ll + 2 * units - 1) / (2 * units));
    const long long most = (nsteps * step_bytes) / (256 * 1024);
    if (chunks > most) chunks = static_cast<int>(most);
    if (chunks > 32) chunks = 32;
    if (chunks < 1) chunks = 1;
  }
  int cs = (nsteps + chunks - 1) / chunks;
  pl.chunks = chunks;
  pl.chunk_steps = cs;
  // (a stage of the ring is 60 steps of one row, or 30 of each row of a logit-level pair)
  const int batch = (mode == kEnsembleSample) ? kStageVecs / 32 : kStageVecs / 64;
  if (chunks > 1) pl.chunk_steps = (pl.chunk_steps + batch - 1) / batch * batch;
  pl.chunks = (nsteps + pl.chunk_steps - 1) / pl.chunk_steps;
  // drawing chunks of about 64 KB, 64 at most
  int ds = static_cast<int>((dchunk_kb * 1024 + step_bytes - 1) / step_bytes);
  if (ds < kSW) ds = kSW;
  int dchunks = (nsteps + ds - 1) / ds;
  if (dchunks > 64) dchunks = 64;
  if (dchunks < 1) dchunks = 1;
  pl.dchunk_steps = (nsteps + dchunks - 1) / dchunks;
  pl.dchunks = (nsteps + pl.dchunk_steps - 1) / pl.dchunk_steps;
  pl.nslots = (mode == kEnsembleSample) ? n : 2;
  pl.nch = channels_of(mode, n);
  pl.blocks = sm_count * (blocks_per_sm > 0 ? blocks_per_sm : 1);
  pl.draw_blocks = sm_count;
  pl.dq_cap = 2 * max_batch * (pl.dchunks + 1);  // a row queues its items once (twice when the residual turns out empty), and may be queued for locating
  return pl;
}

void fused_scratch_bytes(const FusedPlan& pl, int vocab, int dtype, int gamma, int max_batch, size_t out[9]) {
  const size_t B = static_cast<size_t>(max_batch), P = static_cast<size_t>(gamma) + 1;
  const int E = (dtype == COS_DTYPE_F32) ? 4 : 8;
  const size_t nsteps = (static_cast<size_t>(vocab / E) + 31) / 32;
  out[0] = kCtrWords * sizeof(unsigned);
  out[1] = B * sizeof(unsigned long long);
  out[2] = B * P * sizeof(int);
  out[3] = B * P * pl.chunks * pl.nslots * sizeof(SoftPart);
  out[4] = static_cast<size_t>(pl.dq_cap) * sizeof(int);
  out[5] = B * sizeof(int);
  out[6] = B * sizeof(int);
  out[7] = B * pl.dchunks * pl.nch * sizeof(double);
  out[8] = B * nsteps * pl.nch * sizeof(double);
}

cudaError_t fused_occupancy(int dtype, int mode, int n, int* blocks_per_sm) {
  FusedFn fn = pick_fused(dtype, mode, n);
  if (fn == nullptr) return cudaErrorInvalidDeviceFunction;
  cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(fused_smem(mode, n, false)));
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(reinterpret_cast<const void*>(pick_fused(dtype, mode, n, true)),
                             cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(fused_smem(mode, n, true)));
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, reinterpret_cast<const void*>(fn), kFT,
                                                       fused_smem(mode, n, false));
}

cudaError_t fused_launch(int dtype, int mode, const KParams& p, const FusedPlan& plan, const FusedScratch& scratch,
                         unsigned poll_limit, int debug_drop, bool draw_only, cudaStream_t stream) {
  FusedFn fn = pick_fused(dtype, mode, p.n, draw_only);
  if (fn == nullptr) return cudaErrorInvalidDeviceFunction;
  FParams fp;
  fp.k = p;
  fp.plan = plan;
  fp.s = scratch;
  fp.num_items = p.num_units * plan.chunks;
  const int E = (dtype == COS_DTYPE_F32) ? 4 : 8;
  fp.nvec = p.V / E;
  fp.total_events = static_cast<unsigned>(p.num_units + p.B);
  fp.poll_limit = poll_limit;
  fp.debug_drop = debug_drop;
  fp.draw_only = draw_only ? 1 : 0;
  int blocks = draw_only ? plan.draw_blocks : plan.blocks;
  const int most = draw_only ? p.B * plan.dchunks : fp.num_items;
  if (blocks > most) blocks = most;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  lc.blockDim = dim3(kFT, 1, 1);
  lc.dynamicSmemBytes = fused_smem(mode, p.n, draw_only);
  lc.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = draw_only ? 1 : 0;  // a drawing launch starts while the launch before it drains
  return cudaLaunchKernelEx(&lc, fn, fp);
}

}  // namespace cosv
