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
//   stage 4  the same for ensembles of three or four models, with one sum per model and step.
// Units are handed out from a global counter.  Between blocks there are only fences and arrival counters;
// the launches of a run (stage 0, then 3 or 1 and 2) order the stages.  Waits exist only inside a block of the barrier-free form,
// and they are bounded: a wait that gave up marks every row with COS_ROW_FAULT and the block leaves.
// At T = 0 stage 0 is the whole run.
//
// This file is the host side of the library (contexts, launches, the C entry points).  The device code it compiles:
//   cos_common.cuh        constants, launch parameters, loads, Philox, softmax partials
//   cos_stage_shared.cuh  shared-memory layout of a block, cluster merge, publishing a position and the row scan
//   cos_stage_stream.cuh  stage 0: the sweep of a position, the accept decision, the barrier-free loop
//   cos_stage_draw.cuh    stages 1 to 4: big tokens in fp64, the two one-sweep forms
//   cos_stage_kernel.cuh  the kernel template
// (cos_fused.cu holds the persistent one-launch kernel, cos_probe.cu the two streaming ceilings.)

#include <mutex>

#include "cos_common.cuh"
#include "cos_fused.h"
#include "cos_stage_kernel.cuh"

using namespace cosv;

namespace {

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
  // keep a step per warp (small vocabularies are a chain of latencies: workload 1 went from 25.3 to 24.1 us per call
  // and workload 2 from 35.3 to 34.2 when this asked for one step instead of two)
  while (cs > 1 && nsteps / (cs * kWarps) < 1) cs >>= 1;
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
  // (choose_parts counts two blocks per multiprocessor; the stage with a channel per model holds one, so it is
  // asked for half the device: one wave of blocks instead of two.  Workload 4: 96.1 -> 90.1 us per call with 128
  // blocks instead of 256; 64 blocks: 104.8 us)
  int parts = choose_parts(c, rows, channels ? sm_count / 2 : sm_count);
  while (parts < 8 && static_cast<long long>(rows) * parts < 3 * slots && nsteps / (2 * parts * kWarps) >= 8) parts <<= 1;
  // few rows of a small vocabulary: the stage is a chain of latencies, and more blocks per row (one cluster, down
  // to a step per warp) shorten the sweep in it (workload 1: 26.5 -> 25.3 us per call, workload 2: 41.7 -> 36.0 us)
  while (parts < 8 && static_cast<long long>(rows) * parts * 2 <= slots && nsteps / (2 * parts) >= kWarps / 2) parts <<= 1;
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
  e = launch_stage(c.dtype, mode, 0, p, c0, stream, true, dense);
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
      int draw_cs = 1;
      // the blocks of a unit as one cluster (portable sizes), where the launch is a single wave of blocks: with
      // several waves the clusters wait for four free places at once (workload 5: +17 us per call), with one the
      // barrier is cheaper than fence and counter (workloads 1 to 4: -1.4 to -1.7 us)
      const long long draw_slots = (sweep_stage == 4 ? 1LL : 2LL) * ctx->sm_count;
      if (p.parts > 1 && p.parts <= 8 && static_cast<long long>(most) * p.parts <= draw_slots) {
        draw_cs = p.parts;
        p.draw_cluster = 1;
        p.num_clusters = (most < cap ? most : cap);
      }
      e = launch_stage(c.dtype, mode, sweep_stage, p, draw_cs, stream, true);
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
