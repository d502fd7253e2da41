/*
 * sti_planner.h - the two-stage pipeline planner of STI (arXiv 2207.05022, Section 5), host only.
 *
 * It produces the plan that sti_plan_create (sti.h) executes.  A *shard* here is the paper's: vertical
 * slice i of a layer = attention head i plus FFN slice i, stored at versions 2,3,4,5,6 and 32 bits
 * (Section 4.2); the library's attention unit i and FFN unit i of that layer get the same keep flag,
 * bitwidth and residency.
 *
 * Inputs are the two offline profiles of Section 5.2: the IO delay of one shard per version and the
 * computation delay of one layer as a function of the number of shards m (at the padded input length
 * in use), plus the shard-importance table (one score per shard, larger = more important).
 *
 * Stage 1, compute planning (Section 5.3): among all (n, m) with n * T_comp(m) <= T pick the one with
 * the most shards n*m, the deeper one on a tie.  The submodel is layers 0..n-1 and, in each layer, the
 * m most important shards (lower index on ties).
 * Stage 2, IO planning (Section 5.4): accumulated IO budgets AIB(0) = IO delay of the preload buffer's
 * contents, AIB(k) = AIB(k-1) + T_comp(m); a shard of layer k costs its IO delay in AIB(k..n-1);
 * a plan is valid iff every AIB stays >= 0.  Pass 1 gives every shard outside the preload buffer the
 * highest uniform version that is valid (2 bits even if that is not); pass 2 walks the shards in
 * importance order and raises each to the highest version its budgets still allow.
 * Preload contents (Section 1): the first shards in layer order that fit in preload_bytes.  When the
 * request does not say what the buffer holds, the planner first plans with the buffer size as bonus
 * budget, picks those first shards, and then plans again with that buffer as given.
 */
#ifndef STI_PLANNER_H_
#define STI_PLANNER_H_

#include <stddef.h>
#include <stdint.h>

#include "sti.h"

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

#define STI_N_VERSIONS 6   /* bitwidths 2, 3, 4, 5, 6, 32 in this order */

typedef struct {
  int32_t n_layers;                    /* N of the stored model                                     */
  int32_t n_slices;                    /* M shards per layer                                         */
  const double* t_comp_us;             /* [n_slices + 1]; entry m = delay of one layer with m shards; [0] unused */
  double t_io_us[STI_N_VERSIONS];      /* IO delay of one shard at 2,3,4,5,6,32 bits                 */
  uint64_t shard_bytes[STI_N_VERSIONS];/* size of one shard at those versions                        */
  const float* importance;             /* [n_layers * n_slices], layer-major                         */
} sti_planner_profile;

typedef struct {
  double target_us;                    /* T                                                          */
  uint64_t preload_bytes;              /* |S|                                                        */
  const uint8_t* preloaded_bits;       /* optional [n_layers * n_slices]: 0 = not in the buffer, else the version held */
} sti_planner_request;

typedef struct {                       /* arrays are caller-allocated, [n_layers * n_slices], layer-major */
  int32_t n, m;                        /* submodel size                                              */
  int32_t pass1_bits;                  /* the uniform version of pass 1                              */
  int32_t valid;                       /* 1 = every AIB >= 0 (no stall expected), 0 = not even 2 bits fit */
  uint8_t* keep;                       /* 1 = shard is part of the submodel                          */
  uint8_t* bits;                       /* version of each kept shard                                 */
  uint8_t* preload;                    /* 1 = shard sits in the preload buffer                       */
  double* aib_us;                      /* [n_layers]: remaining budget per submodel layer (entries >= n are 0) */
} sti_planner_result;

/* Section 5.3 + 5.4.  Host only; no device is touched.  STI_ERR_ARG on null pointers or empty tables. */
sti_status sti_plan_auto(const sti_planner_profile* profile, const sti_planner_request* request,
                         sti_planner_result* result);

/* Back-to-back executions (Section 3.2) with the eviction rule of Section 5.5: after a run the loaded
 * shards may stay cached in an enlarged preload buffer.  Shards are evicted from the top layer downwards
 * until the rest fits, i.e. walking the executed submodel in layer order (layer 0 first, slices in index
 * order) shards are retained, at the version they ran with, while they fit in buffer_bytes; the walk
 * stops at the first shard that does not fit.  keep / bits are the executed plan's grids
 * ([n_layers * n_slices], layer-major); out_preloaded_bits (same shape, caller-allocated) receives 0 or the
 * retained version and is what sti_plan_auto takes as `preloaded_bits` for the next execution, whose
 * planner then spends the IO time no longer needed on higher versions of the other shards.
 * out_used_bytes (optional) receives the bytes retained.  STI_ERR_ARG on null pointers, empty grids or a
 * kept shard whose version is not one of 2,3,4,5,6,32.  Host only. */
sti_status sti_preload_after_run(int32_t n_layers, int32_t n_slices, const uint8_t* keep, const uint8_t* bits,
                                 const uint64_t shard_bytes[STI_N_VERSIONS], uint64_t buffer_bytes,
                                 uint8_t* out_preloaded_bits, uint64_t* out_used_bytes);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* STI_PLANNER_H_ */
