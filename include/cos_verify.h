/*
 * cos_verify.h -- C ABI of the CoS verification step for NVIDIA B200 (sm_100a).
 *
 * The operation (paper: "Fast Large Language Model Collaborative Decoding via
 * Speculation", Sec. 3.1-3.2):
 *   for every row b of a batch and every one of the gamma+1 positions j, read the
 *   logits of n models over the vocabulary, form the combined distribution r
 *   (Eq. 3: weighted probability ensemble, Eq. 4, or a logit-level combination,
 *   Eq. 5, optionally restricted to a plausibility mask), test the draft token x
 *   with  u <= min(1, r(x) / q(x))  against the proposer's distribution q (Eq. 6),
 *   find the first rejected position of the row, and emit there a token drawn from
 *   norm(max(0, r - q)) (text after Eq. 6, App. A.1), or, when all gamma drafts pass,
 *   a bonus token for position gamma (Sec. 3.1).  Temperature T tempers every
 *   softmax; T = 0 is greedy decoding with one-hot distributions (Sec. 4.1).
 *
 * All pointers in cos_verify_args are DEVICE pointers owned by the caller unless a
 * function says otherwise.  No function here synchronises the device except
 * cos_verify_create, cos_verify_destroy and cos_verify_run_host.
 */
#ifndef COS_VERIFY_H
#define COS_VERIFY_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define COS_MAX_MODELS 8

typedef struct cos_verify_ctx cos_verify_ctx; /* opaque; owns only device scratch */

typedef enum {
  COS_OK = 0,
  COS_ERR_INVALID_ARG = 1, /* null pointer, value out of range, inconsistent config   */
  COS_ERR_UNSUPPORTED = 2, /* valid request this build does not implement             */
  COS_ERR_ALIGNMENT = 3,   /* a pointer is not aligned to its element type            */
  COS_ERR_CUDA = 4,        /* a CUDA runtime call failed; see cos_verify_last_error   */
  COS_ERR_NOMEM = 5        /* host or device allocation failed                        */
} cos_status;

/* combination function C / C' of Eq. 3 */
enum {
  COS_COMBINE_PROB_ENSEMBLE = 0, /* r = sum_i w_i softmax(l_i / T)              (Eq. 4)            */
  COS_COMBINE_LOGIT_LINEAR = 1   /* r = softmax_M((sum_i w_i l_i) / T)          (Eq. 5; also logit */
                                 /*     interpolation of an aligned / base model pair)             */
};

enum { COS_DTYPE_F32 = 0, COS_DTYPE_BF16 = 1, COS_DTYPE_F16 = 2 };

/* bits of row_status[b]; only positions up to and including the row's first rejection report */
enum {
  COS_ROW_NONFINITE = 1,      /* a distribution was NaN/Inf: that position counts as rejected, token -1 */
  COS_ROW_BAD_DRAFT = 2,      /* draft token outside [0, vocab): rejected, residual still sampled       */
  COS_ROW_Q_ZERO = 4,         /* q(draft) == 0: ratio taken as +inf if r(draft) > 0, else 0             */
  COS_ROW_RESIDUAL_EMPTY = 8, /* rejected but max(0, r - q) == 0 everywhere: token drawn from r         */
  COS_ROW_FAULT = 16          /* an internal wait of the kernel gave up (a defect, never the data): the */
                              /* call's outputs are undefined and the context must not be used again;   */
                              /* set on every row, reported whatever the row's first rejection          */
};

/* bits of cos_verify_args.flags */
enum {
  COS_RUN_ALL_RESIDUALS = 1,         /* compute the residual mass S = sum max(0, r - q) = 1 - alpha      */
                                     /* (Eq. 7) at every draft position and report it in diag, not only  */
                                     /* where it is needed                                               */
  COS_RUN_PROPOSER_PER_POSITION = 2, /* `proposer` is [B][gamma+1]: entry (b, j), j < gamma, is the model */
                                     /* that proposed draft j of row b, so q changes from position to    */
                                     /* position (Algorithm 2 verifies a cached sequence that holds      */
                                     /* tokens of several proposers).  Entry (b, gamma) must be a valid  */
                                     /* index; its distribution decides nothing.                         */
  COS_RUN_BONUS_FROM_MODEL = 4,      /* the token after gamma acceptances is drawn from model            */
                                     /* `bonus_model`'s own distribution instead of the combined one     */
                                     /* (Sec. 3.3: the verifier's bonus token, to be treated as that     */
                                     /* model's next proposal)                                           */
  COS_RUN_EARLY_EXIT = 8,            /* a hint: positions behind a rejection that their row has already  */
                                     /* reported may be left unread (Sec. 3.1 discards them anyway).     */
                                     /* accept_count, out_tokens, row_status and bonus_prob are those of */
                                     /* the full run; diag is NaN at a position that was left unread,    */
                                     /* and which positions those are depends on timing.  Taken by       */
                                     /* cos_verify_run when no cluster size and no mask is configured.   */
  COS_RUN_INPUTS_SETTLED = 16        /* a promise by the caller: logits, draft_tokens and proposer were  */
                                     /* complete in device memory before the work that precedes this     */
                                     /* call in its stream was submitted (they are not written by the    */
                                     /* kernel queued just before the call).  The streaming launch may   */
                                     /* then read them while that work drains - the drawing launch of    */
                                     /* the previous call, for one - and waits for it only before it     */
                                     /* touches anything else; calls queued back to back overlap.        */
                                     /* Outputs and results are those of an ordinary run.  Without the   */
                                     /* flag a run reads nothing before the work ahead of it in the      */
                                     /* stream is complete.  Taken by cos_verify_run at T > 0 for runs   */
                                     /* of at least one position per multiprocessor whose drawing launch */
                                     /* is a single wave of blocks, without cluster size, mask, test     */
                                     /* hook or COS_RUN_EARLY_EXIT; ignored otherwise (cos_verify_get_   */
                                     /* info does not tell).                                             */
};

typedef struct {
  int32_t n;                       /* number of models, 1..COS_MAX_MODELS                               */
  int32_t combine;                 /* COS_COMBINE_*                                                     */
  float weights[COS_MAX_MODELS];   /* w_i.  Ensemble: w_i >= 0, |sum - 1| <= 1e-6.  Logit-linear: any   */
                                   /* finite values (contrastive decoding is (1, -mu), Eq. 5).          */
  int32_t mask_model;              /* logit-linear only: index e of the model whose probabilities gate  */
                                   /* the vocabulary, or -1 for no mask                                 */
  float mask_alpha;                /* in (0, 1]: keep x with l_e(x) >= max_x l_e(x) + ln(mask_alpha)    */
  float temperature;               /* T >= 0; 0 = greedy (lowest index wins ties)                       */
  int32_t gamma;                   /* proposal length, >= 0; every row has gamma + 1 positions          */
  int32_t vocab;                   /* V >= 1                                                            */
  int32_t max_batch;               /* largest batch a run may pass, >= 1                                */
  int32_t dtype;                   /* COS_DTYPE_* of the logits                                         */
  int32_t device;                  /* CUDA device ordinal                                               */
  int32_t cluster_size;            /* thread blocks that share one (row, position) in the streaming     */
                                   /* stage: 1, 2, 4, 8 or 16; 0 lets the library choose                */
  int32_t host_staging;            /* non-zero: also allocate device staging for cos_verify_run_host    */
} cos_verify_config;

typedef struct {
  const void* logits;          /* [n][B][gamma+1][V], element (i,b,j,x) at                              */
                               /*   i*stride_model + b*stride_row + j*stride_pos + x   (in elements)    */
  int64_t stride_model, stride_row, stride_pos;
  const int32_t* draft_tokens; /* [B][gamma]; may be NULL when gamma == 0                               */
  const int32_t* proposer;     /* [B], index in [0, n) of the model that proposed the row's drafts      */
                               /* ([B][gamma+1] with COS_RUN_PROPOSER_PER_POSITION).  An index outside  */
                               /* [0, n) names no distribution q: the positions it governs report       */
                               /* COS_ROW_NONFINITE (rejected, token -1); nothing is read out of bounds */
  int32_t batch;               /* B, 1..max_batch                                                       */
  int32_t flags;               /* COS_RUN_* bits                                                        */
  int64_t row_base;            /* global index of row 0 (for row-sharded batches); enters the RNG only  */
  uint64_t seed, offset;       /* Philox4x32-10 key and counter words 2-3; counter words 0-1 are        */
                               /* (row_base + b, j).  Word 0 of the output feeds the accept test, word  */
                               /* 1 the residual / bonus sample, each as u = (2*(w>>9)+1) * 2^-24.      */
  int32_t* accept_count;       /* out [B]: number of accepted drafts a, 0..gamma                        */
  int32_t* out_tokens;         /* out [B][gamma+1]: a accepted drafts, then the resampled (a < gamma)   */
                               /* or bonus (a == gamma) token, then -1 padding                          */
  uint32_t* row_status;        /* out [B]: COS_ROW_* bits                                               */
  float* diag;                 /* optional out [B][gamma+1][4]: ratio r(x)/q(x), r(x), q(x) at the      */
                               /* draft, and S where it was computed (NaN elsewhere); may be NULL       */
  float* dump_r;               /* optional test hook, out [B][gamma+1][V]: the combined distribution;   */
                               /* forces the full second sweep everywhere; may be NULL                  */
  float* bonus_prob;           /* optional out [B]: where accept_count == gamma, the probability of the */
                               /* bonus token under the distribution it was drawn from (what Score of   */
                               /* Algorithm 2 returns beside the token); NaN elsewhere; may be NULL     */
  int32_t bonus_model;         /* read only with COS_RUN_BONUS_FROM_MODEL: index in [0, n)              */
  const uint64_t* offset_device; /* optional: device address of the counter offset, read by the kernels */
                               /* in place of `offset` (8-byte aligned); lets a captured run be         */
                               /* replayed with fresh uniforms; may be NULL                             */
  float* lse;                  /* optional out [B][gamma+1][S]: the log-sum-exp ln sum_x exp(l(x) / T)  */
                               /* behind every softmax of a position (Sec. 3.1).  Ensemble: S = n, one  */
                               /* per model; logit level: S = 2, the proposer's logits and the combined */
                               /* (masked) logits.  NaN at T = 0 and where the position is not finite.  */
                               /* One more small launch per run; may be NULL                            */
} cos_verify_args;

typedef struct {
  int32_t cluster_size;      /* thread blocks per (row, position)                                     */
  int32_t threads_per_block;
  int32_t max_clusters;      /* clusters that can be resident at once on the device                   */
  int32_t sm_count;
  int32_t launches_per_run;  /* kernels an ordinary cos_verify_run enqueues: 1 at T = 0 and where the     */
                             /* one-launch form was chosen (reserved[2] bit 0); else 2 for logit-level */
                             /* combines and ensembles of two to four models, 3 otherwise.  Every      */
                             /* launch takes its places on the device while the kernel before it in    */
                             /* the stream drains, and reads or writes nothing until that kernel is    */
                             /* complete (unless COS_RUN_INPUTS_SETTLED says the inputs may be read)   */
  int32_t reserved[3];       /* [0], [1]: work items per position when streaming / drawing; [2]: bit  */
                             /* 0: an ordinary run is one launch; bit 1: the tokens of a staged run   */
                             /* are drawn by the persistent kernel's drawing items                    */
} cos_verify_info;

/*
 * Validate the configuration, select the device, allocate scratch sized for
 * max_batch * (gamma + 1) positions and return a context in *out.
 * Errors: COS_ERR_INVALID_ARG (with the reason available from cos_verify_last_error(NULL)),
 * COS_ERR_CUDA, COS_ERR_NOMEM.  One context serves one stream at a time.
 */
cos_status cos_verify_create(const cos_verify_config* config, cos_verify_ctx** out);

/*
 * Enqueue one verification pass (Eq. 3-6 and the rejection / bonus rule of Sec. 3.1) for
 * args->batch rows on `cuda_stream` (a cudaStream_t; NULL is the default stream) and
 * return without waiting.  Outputs are valid once the stream has reached this point.
 * Host-detected problems return an error code and enqueue nothing; data-dependent
 * problems are reported per row in row_status and never trap the device.
 * Runs that share a context must be ordered on one stream.
 * The launches of a run depend on its arguments only (the kernels leave the context's scratch as they
 * found it), so a run may be captured into a CUDA graph and replayed; keep the counter offset in device
 * memory (offset_device) to give every replay its own uniforms.
 */
cos_status cos_verify_run(cos_verify_ctx* ctx, const cos_verify_args* args, void* cuda_stream);

/*
 * Same operation with every pointer in `args` a HOST pointer (pinned memory makes the
 * copies asynchronous): copies logits, drafts and proposers to staging owned by the
 * context, runs, copies accept_count / out_tokens / row_status (and diag if given)
 * back and waits for the stream.  Requires config.host_staging != 0 and contiguous
 * logits (stride_pos = V, stride_row = (gamma+1) V, stride_model = B (gamma+1) V).
 * dump_r and lse are not supported here.
 */
cos_status cos_verify_run_host(cos_verify_ctx* ctx, const cos_verify_args* args, void* cuda_stream);

/*
 * The same verification pass for callers that must not allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for deployment only.)
 *
 * cos_verify_create reserves its scratch with cudaMalloc.  Some hosts of this library cannot
 * do that at the point where they need a verification: an inference engine that has handed
 * the whole device to its own memory pool, or a serving loop in which the device-wide
 * synchronisation that cudaMalloc / cudaFree imply would stall every other stream.  This call
 * needs no context: the kernels' scratch (work and job counters, per-row arrival counters,
 * per-position results, statistics and partial sums, the list of positions that draw a token)
 * lives in an array that is part of the
 * library image, COS_STATIC_SCRATCH_BYTES long, resident on every device that loads the
 * library until the process exits.  The call performs no cudaMalloc, cudaFree or other
 * device allocation; `config` is read on every call (max_batch and host_staging are ignored).
 *
 * Limits: args->batch <= COS_STATIC_MAX_BATCH and args->batch * (gamma + 1) <=
 * COS_STATIC_MAX_POSITIONS; anything larger returns COS_ERR_INVALID_ARG with the reason in
 * cos_verify_last_error(NULL) and enqueues nothing.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and
 * sets kernel attributes; make that first call outside any stream capture.  Every call
 * re-initialises the part of the array that must start clean (memset on `cuda_stream`)
 * before the kernel, so a call does not depend on what the previous one left behind.
 * All calls on a device share the one array: two calls that overlap on the GPU (different
 * streams without an ordering between them) race and give undefined results.  Calls ordered
 * on one stream, or otherwise serialised, are safe.  Inputs, outputs and semantics are those
 * of cos_verify_run.
 */
#define COS_STATIC_MAX_BATCH 1024
#define COS_STATIC_MAX_POSITIONS 8192
#define COS_STATIC_SCRATCH_BYTES                                                                          \
  (256 + 4 * COS_STATIC_MAX_BATCH + 16 * COS_STATIC_MAX_POSITIONS +                                      \
   8 * (COS_STATIC_MAX_POSITIONS + COS_STATIC_MAX_BATCH) + 112 * COS_STATIC_MAX_POSITIONS +              \
   8 * 8 * COS_STATIC_MAX_POSITIONS + 8 * 16 * COS_STATIC_MAX_POSITIONS + 8 * 16 * 16 * COS_STATIC_MAX_BATCH +   \
   4 * COS_STATIC_MAX_POSITIONS)
cos_status cos_verify_run_static(const cos_verify_config* config, const cos_verify_args* args, void* cuda_stream);

/*
 * Measurement aid: with `enable` non-zero, every later cos_verify_run records CUDA events on its
 * stream around each of its launches (stage 0: every position, Eq. 3-6 and the row scan; then the
 * launches that draw the tokens).  cos_verify_get_stage_ms waits for the last timed run and
 * returns the duration of each of its launches in milliseconds (at most 3 values) and their
 * number.  Timing adds a few event records per run and changes no result.
 */
cos_status cos_verify_set_stage_timing(cos_verify_ctx* ctx, int enable);
cos_status cos_verify_get_stage_ms(cos_verify_ctx* ctx, float* ms, int32_t* count);

/*
 * The one-launch form of a run (Sec. 3.1-3.2 as ONE persistent kernel): streaming work items of about 128 KB,
 * rows settled as soon as every position up to their first rejection is published, the token draw queued inside
 * the same launch.  It covers sampling runs (T > 0) of ensembles of up to four models and of logit-level combines
 * without mask, with 16-byte aligned rows, at most 16 positions per row and no test hook.  `enable` = 1 makes
 * later runs of this context take it (COS_ERR_UNSUPPORTED when the configuration is not covered); `enable` = 2
 * keeps the staged streaming launch and lets the same persistent kernel draw the tokens in a second launch that
 * runs only its drawing items (one sweep with a channel sum per model, also for ensembles of three and four
 * models); 0 returns to the staged launches, which are the default because they are the faster form on the
 * measured workloads.  Results are those of the staged form (same arithmetic per position; sums are merged in
 * another order, so probabilities may differ in the last bits).  COS_RUN_EARLY_EXIT is ignored by form 1: every
 * position is read.
 */
cos_status cos_verify_set_one_launch(cos_verify_ctx* ctx, int32_t enable);

/*
 * Failure detection of the one-launch form of a run (sampling modes without mask or test hook): every wait
 * inside the kernel is a bounded poll.  A block that sees no progress for `polls` polls (about 0.2 us each; the
 * default of 2^20 is about a fifth of a second) sets COS_ROW_FAULT on every row and leaves; the kernel always
 * terminates and the device stays usable.  `polls` must be at least 16.  `test_drop_report` != 0 is a test
 * hook: one streaming warp of block 0 then never reports its first work item, so the waits of that block run
 * out and the run ends with COS_ROW_FAULT; the context clears its scratch before its next run.
 * The paper has no counterpart; this follows from running the whole step (Sec. 3.1-3.2) as one launch.
 */
cos_status cos_verify_set_wait_limit(cos_verify_ctx* ctx, uint32_t polls, int32_t test_drop_report);

/*
 * Measurement aid (the paper has no counterpart): the two ceilings the streaming pass is compared with, measured
 * on the current device.  kind 0 reads `bytes` of `device_buf` once with 128-bit streaming loads; kind 1 does the
 * same and evaluates one fast base-2 exponential per 16-bit entry, which is what a softmax normaliser (Sec. 3.1)
 * costs per bf16 logit.  Same launch shape as the verification kernels.  `device_out` is scratch of at least
 * 1024 floats per multiprocessor (`out_floats` says how many it holds).  Runs two untimed and `reps` timed
 * launches on `cuda_stream`, waits for them, and returns the fastest in *best_ms.  `device_buf` must be 16-byte
 * aligned; its contents only matter as numbers (any bf16 data will do).
 */
cos_status cos_verify_measure_ceiling(int32_t kind, const void* device_buf, uint64_t bytes, float* device_out,
                                      uint64_t out_floats, int32_t reps, float* best_ms, void* cuda_stream);

/* Launch geometry chosen at creation. */
cos_status cos_verify_get_info(const cos_verify_ctx* ctx, cos_verify_info* info);

/* Free the context and its scratch (waits for the device). NULL is allowed. */
cos_status cos_verify_destroy(cos_verify_ctx* ctx);

/* Text of the last error on this context, or of the last failed create when ctx is NULL. */
const char* cos_verify_last_error(const cos_verify_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* COS_VERIFY_H */
