// Internal interface between the translation units of the library: the one-launch form of a verification run.
#ifndef COS_FUSED_H
#define COS_FUSED_H

#include <cuda_runtime.h>
#include <stddef.h>

#include "cos_common.cuh"

namespace cosv {

// How a run is cut into work items, and where the one-launch kernel keeps its state.
struct FusedPlan {
  int chunks, chunk_steps;    // streaming: chunks per (row, position), steps (32 vectors of 16 bytes per model) per chunk
  int dchunks, dchunk_steps;  // drawing: the same for the one (row, position) of a row that draws a token
  int nslots;                 // softmax statistics per (row, position): n (ensemble) or 2 (logit level)
  int nch;                    // channel sums per step of a drawing sweep: n (ensemble) or 2
  int blocks;                 // persistent blocks of the one-launch form (two per multiprocessor)
  int draw_blocks;            // persistent blocks of a launch that only draws tokens (one per multiprocessor)
  int dq_cap;                 // entries of the queue of drawing items
};

// Device scratch of the one-launch kernel (all of it zero between runs).
struct FusedScratch {
  unsigned* ctr;                 // next streaming item, events done, queue head and tail, blocks gone, fault (a line each)
  unsigned long long* row_word;  // [B]
  int* unit_arrivals;            // [B * P]
  SoftPart* chunk_part;          // [B * P][chunks][nslots]
  int* dq;                       // [dq_cap]
  int* row_draw;                 // [B]
  int* draw_arrivals;            // [B]
  double* dzpart;                // [B][dchunks][nch]
  double* srec;                  // [B][nsteps][nch]
};

// Whether the one-launch kernel covers this configuration (mode: the Mode enum of the kernels).
bool fused_covers(int dtype, int mode, int n, int vocab, int gamma, int mask_model, long long max_units);

// Work decomposition for a context (sizes follow max_batch); `blocks_per_sm` from fused_occupancy.
FusedPlan fused_plan(int dtype, int mode, int n, int vocab, int gamma, int max_batch, int sm_count, int blocks_per_sm);

// Bytes of each scratch array for `plan` (same order as the members of FusedScratch).
void fused_scratch_bytes(const FusedPlan& plan, int vocab, int dtype, int gamma, int max_batch, size_t out[9]);

cudaError_t fused_occupancy(int dtype, int mode, int n, int* blocks_per_sm);

// Enqueue the launch.  `p` is filled as for the staged kernels; plan/scratch come from the context.
// `poll_limit`: idle polls after which a block that sees no progress gives up (COS_ROW_FAULT on every row).
// `debug_drop`: test hook; when non-zero, one streaming warp of block 0 never reports its first item.
// `draw_only`: the positions were published by the staged launch before this one (its job list names, per row, the
// position that draws a token); this launch then only draws those tokens.
cudaError_t fused_launch(int dtype, int mode, const KParams& p, const FusedPlan& plan, const FusedScratch& scratch,
                         unsigned poll_limit, int debug_drop, bool draw_only, cudaStream_t stream);

}  // namespace cosv

#endif  // COS_FUSED_H
