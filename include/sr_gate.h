/*
 * sr_gate.h -- C ABI of the Selective Rollout gate library (NVIDIA B200, sm_100a).
 *
 * The library evaluates, for many GRPO groups at once, the gate of the paper's
 * Section 3.2: the mean pairwise prefix edit distance d_K between the N partial
 * action sequences of a group, the decision Cut = [d_K < d_L] (Eq. 2), and the
 * group-relative advantages of Eq. 1 with the zero-variance flag of Section 2.1.
 *
 * Conventions (every entry point unless it says otherwise)
 *   - Pointers are DEVICE pointers.  The caller owns every buffer; the library
 *     allocates no device memory and keeps no state between calls.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work on it and return without synchronising.
 *   - Return value: SR_OK, or a negative SR_ERR_* code.  Every code except SR_ERR_CUDA
 *     comes from a check of the arguments made before anything is enqueued: no buffer
 *     was touched.  SR_ERR_CUDA reports a CUDA call or launch that failed part-way:
 *     earlier copies and kernels of the same call may already be on the stream, and the
 *     outputs, the workspace / arena and *status are then undefined.
 *   - Actions (or tokens) are int32 IDs compared for equality only; every 32-bit
 *     value is legal.  Mapping action strings to IDs is the caller's job.
 *   - Pairs of a group are ordered (0,1),(0,2),...,(0,N-1),(1,2),...,(N-2,N-1);
 *     P = N(N-1)/2.
 */
#ifndef SR_GATE_H_
#define SR_GATE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SR_VERSION 100

/* error codes */
#define SR_OK 0
#define SR_ERR_NULL (-1)           /* a required pointer is NULL */
#define SR_ERR_BAD_N (-2)          /* N < 2 or N > SR_MAX_N, or n_groups < 0 */
#define SR_ERR_BAD_K (-3)          /* K < 0, K > stride, K > SR_MAX_K, bad max_steps */
#define SR_ERR_ALIGN (-4)          /* seqs not 16-byte aligned or stride % 4 != 0 */
#define SR_ERR_STATE_SIZE (-5)     /* incremental state buffer too small */
#define SR_ERR_WORKSPACE (-6)      /* workspace NULL, misaligned or too small */
#define SR_ERR_CUDA (-7)           /* a CUDA call failed; see sr_last_cuda_error() */
#define SR_ERR_BAD_MODE (-8)       /* unknown norm_mode */
#define SR_ERR_SCRATCH_LIMIT (-9)  /* sr_gate_noalloc: problem needs more than the built-in scratch */
#define SR_ERR_BAD_OFFSETS (-10)   /* sr_gate_host_packed: row_start malformed */

/* limits */
#define SR_MAX_N 32                /* rollouts per group */
#define SR_MAX_K 1024              /* longest prefix (symbols) */
#define SR_MAX_INCR_STEPS 32       /* longest rollout the incremental state can hold */

/* norm_mode */
#define SR_NORM_MAXLEN 0           /* paper: each pair distance / longer prefix length */
#define SR_NORM_NONE 1             /* mean of the raw pair distances */

/* new_actions value meaning "this rollout emitted no action this step" */
#define SR_NO_ACTION INT32_MIN

/* bits OR-ed into *status by the kernels (the caller zeroes it when it wants to) */
#define SR_STATUS_NEG_LEN 1        /* a negative length was treated as 0 */
#define SR_STATUS_STEP_OVERFLOW 2  /* an action arrived for a rollout already at max_steps; ignored */
#define SR_STATUS_BAD_STATE 4      /* incremental state header does not match the call; step skipped */

int sr_version(void);
const char* sr_strerror(int code);      /* static string */
const char* sr_last_cuda_error(void);   /* text of the last CUDA failure seen by this thread */

/*
 * sr_gate -- d_K and the stop mask for every group (Section 3.2, Appendix B
 * "prefix_edit_distance_mean", Eq. 2).
 *
 * For each group g and each pair i<j: d_ij = unit-cost Levenshtein distance
 * (insert / delete / substitute) between the first m_i = min(len_i, K) IDs of
 * rollout i and the first m_j of rollout j.  With SR_NORM_MAXLEN each d_ij is
 * divided by max(m_i, m_j) (0 when both prefixes are empty); the terms are added
 * in fp64 in pair order and divided by P, giving mean[g] = d_K.  stop[g] =
 * (mean[g] < threshold), strictly.  Negative lengths count as 0 and set
 * SR_STATUS_NEG_LEN.
 *
 *   seqs       in  [n_groups][N][stride] int32, row-major, 16-byte aligned, stride % 4 == 0
 *   lens       in  [n_groups][N] int32 actions emitted so far; NULL = every length is K
 *   K              gate step, 0 <= K <= min(stride, SR_MAX_K)
 *   threshold      d_L
 *   pair_dist  out [n_groups][P] int32 raw distances; may be NULL
 *   pair_sum   out [n_groups] int32 sum of the raw distances; may be NULL
 *   mean       out [n_groups] fp64; may be NULL
 *   stop       out [n_groups] uint8, 1 = cut; required
 *   status     in/out 1 int32 of SR_STATUS_* bits; may be NULL
 *   workspace      device scratch of at least sr_gate_workspace_bytes(...) bytes,
 *                  256-byte aligned; contents are undefined before and after the
 *                  call; may be NULL when that size is 0 (K <= 32).  Two calls
 *                  that may overlap on the device need separate workspaces.
 *
 * n_groups == 0 is a valid no-op.  Prefixes of up to 32 symbols use one 32-bit
 * word of bit-parallel state per pair; longer ones use the blocked multi-word path,
 * which leaves the common prefix of a pair out of the computation (the distance of
 * two sequences equals that of what follows a common prefix), so groups whose
 * rollouts agree on their first symbols cost less.  Results do not depend on it.
 */
int sr_gate(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
            int32_t stride, int32_t K, double threshold, int32_t norm_mode,
            int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
            int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/* Host-only, pure.  Scratch bytes sr_gate needs for these sizes (0 when K <= 32);
 * returns 0 for invalid arguments as well (sr_gate then reports the error). */
size_t sr_gate_workspace_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K);

/*
 * sr_gate_decide -- the same stop mask as sr_gate for less work.  Eq. 2 only consumes the
 * comparison d_K < d_L, so a group can be dismissed as soon as a LOWER bound of its d_K
 * reaches the threshold.  For prefixes longer than 32 symbols the match-stream pass
 * yields such a bound per pair for free: max(|m_i - m_j|, number of symbols of one prefix
 * that do not occur in the other at all) <= d_ij.  The bounds go through the very same
 * ordered fp64 sum as the distances (every term is smaller or equal and rounded addition
 * is monotone), so a group whose bounded d_K is not below the threshold gets stop = 0
 * without a single column of the recurrence.  A group the bounds leave open is computed,
 * but only as far as the threshold can still be met: with every other pair at its lower
 * bound, a pair whose distance exceeds L (P d_L - sum of the others' bounded terms) settles
 * the group as "continue", so each pair runs in a diagonal band (Ukkonen's cut-off) that
 * is just wide enough for that cap, and for the number of positions at which the two
 * prefixes differ, an upper bound that prep also counts.  A pair that stays within its
 * band gets its exact distance; one that leaves it is reported as "more than the cap".
 *
 *   stop       identical to sr_gate's, always
 *   exact      out [n_groups] uint8 or NULL: 1 = pair_dist / pair_sum / mean of the group
 *              are the exact values (as sr_gate); 0 = the group was settled (stop = 0) by
 *              bounds or caps, and its values are lower bounds (each <= the exact value,
 *              mean >= threshold)
 *   other arguments and the workspace as for sr_gate (sr_gate_workspace_bytes applies).
 *
 * With K <= 32 every group is computed exactly.  The mode pays off where the bounds settle
 * much of the batch (token-level groups at the paper's d_L = 0.12: three times faster than
 * sr_gate); where most groups have to be computed anyway, sr_gate is the faster call.  The
 * paper has no counterpart; its gate is evaluated on a handful of groups per iteration and
 * never needed one.
 */
int sr_gate_decide(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                   int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                   int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                   uint8_t* exact, int32_t* status, void* workspace, size_t workspace_bytes,
                   void* stream);

/*
 * sr_gate_host -- the same computation on HOST buffers: copies seqs/lens to the
 * device, runs sr_gate, and copies the requested outputs back, all enqueued on
 * `stream`; the caller synchronises the stream before reading the outputs.
 * Every data pointer here is a HOST pointer (pinned memory makes the copies
 * asynchronous); outputs that are NULL are not copied.  `arena` is DEVICE scratch
 * of at least sr_gate_host_arena_bytes(...) bytes, 256-byte aligned, used for the
 * staged inputs, outputs and the gate workspace.
 * `copy_stream` (a second cudaStream_t, or NULL): when given, and different from
 * `stream`, the inputs are sent in four chunks on it so that the copy of one chunk
 * overlaps the kernels of the previous one; the outputs still arrive on `stream`, which
 * is the only stream the caller has to synchronise.  The chunked path creates and
 * releases a few CUDA events per call (no device memory).
 */
int sr_gate_host(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                 int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                 int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                 int32_t* status, void* arena, size_t arena_bytes, void* stream,
                 void* copy_stream);
size_t sr_gate_host_arena_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K);

/*
 * sr_gate_host_packed -- sr_gate_host for HOST input in packed (ragged) form: the
 * prefixes of all rollouts one after the other, without padding.  The operation is the
 * same d_K / stop mask of Section 3.2 and Eq. 2; only the input layout differs.  Token-
 * level prefixes of very different lengths fill a padded [rows][stride] array to about
 * two thirds, and over a host link the copy sets the time of a call, so sending only
 * the symbols that exist is what shortens it.
 *
 *   symbols    in  HOST int32: row r (= g * N + i) owns symbols[row_start[r] .. row_start[r+1])
 *   row_start  in  HOST int64 [n_groups * N + 1], row_start[0] = 0, non-decreasing; the
 *                  length of row r is row_start[r+1] - row_start[r] (plays the part of
 *                  lens; a row may be longer than K, only its first K symbols count).
 *                  Read on the host during the call, and again by the copy engine: keep
 *                  both arrays unchanged until the stream has passed the call.
 *   stride         row pitch of the padded device copy: a multiple of 4, >= K; the sum of
 *                  all lengths must not exceed n_groups * N * stride
 *   outputs, status, stream: as for sr_gate_host (HOST pointers)
 *   copy_stream    a second cudaStream_t, or NULL.  When given (and different from `stream`,
 *                  K > 32, at least 64 groups) the symbols are sent on it in four pieces of
 *                  whole groups, and the gate's per-group pass runs on each piece while the
 *                  next one is still on the link; the recurrence runs once over the whole
 *                  batch.  Outputs arrive on `stream`, the only stream to synchronise.  This
 *                  path creates and releases a few CUDA events per call (no device memory).
 *   arena          DEVICE scratch of sr_gate_host_packed_arena_bytes(...) bytes, 256-byte
 *                  aligned
 *
 * Errors (nothing enqueued): as sr_gate_host, and SR_ERR_BAD_OFFSETS for a malformed
 * row_start.
 */
int sr_gate_host_packed(const int32_t* symbols, const int64_t* row_start, int32_t n_groups,
                        int32_t N, int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                        int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                        int32_t* status, void* arena, size_t arena_bytes, void* stream,
                        void* copy_stream);
size_t sr_gate_host_packed_arena_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K);

/*
 * sr_gate_noalloc -- sr_gate for callers that cannot allocate device memory.  (The
 * paper has no counterpart: this is a deployment aid of this library.)
 *
 * Who needs it: a gate that runs inside someone else's process -- a rollout worker
 * embedded in an inference engine that claimed its GPU memory at start-up, a trainer
 * whose caching allocator owns the rest, a plug-in that is simply not allowed to
 * call cudaMalloc.  There sr_gate's `workspace` has nowhere to come from.  This
 * entry point takes the same inputs and outputs but no workspace: the multi-word
 * path (K > 32) works in a fixed array of SR_NOALLOC_SCRATCH_BYTES that is part of
 * the library's device image, so every GPU on which this entry point has been used
 * holds that much memory until the process exits.  It calls no allocation routine;
 * the CUDA runtime reserves the array when it loads the image on a device, which with
 * its default lazy loading happens inside the first call there.
 *
 *   - Limit: sr_gate_workspace_bytes(n_groups, N, stride, K) must not exceed
 *     SR_NOALLOC_SCRATCH_BYTES (also returned by sr_gate_noalloc_limit_bytes());
 *     otherwise SR_ERR_SCRATCH_LIMIT, nothing enqueued.  As a guide, 64 groups of
 *     N = 8 at K = 1024, or 1000 groups at K = 64, fit.  K <= 32 has no limit.
 *   - The first call on each device (with K > 32) looks up the array's device address
 *     (a cudaGetSymbolAddress with that device current), which is also when the 16 MiB
 *     are reserved.  Make that first call during set-up, before any stream capture is
 *     begun and while the memory is still to be had: if the device is already full it
 *     fails with SR_ERR_CUDA.  The address is remembered per device; after a
 *     cudaDeviceReset it is stale, so do not use this entry point on a device that the
 *     process has reset.
 *   - Arguments are checked exactly as sr_gate checks them, before the size limit.
 *   - All calls on a device share the one array.  It keeps whatever the last call
 *     left; each call clears the counters it needs zeroed before using them.  Two
 *     calls that can overlap on the device (different streams, no dependency) race
 *     on it: serialise them, or use sr_gate with separate workspaces.
 *   - Results are identical to sr_gate's.
 */
#define SR_NOALLOC_SCRATCH_BYTES (16u << 20)
int sr_gate_noalloc(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                    int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                    int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                    int32_t* status, void* stream);
size_t sr_gate_noalloc_limit_bytes(void);

/*
 * Incremental gate: the gate re-evaluated after every environment step while
 * each rollout appends one action per step.  The paper evaluates the gate at one
 * fixed step K (Appendix C.1) and names an adaptive K as future work (Section 5,
 * Limitations); this variant keeps, per pair, the boundary of the edit-distance
 * matrix (vertical deltas of the last column, horizontal deltas of the last row,
 * as +1 / -1 bit masks) in a caller-owned device buffer, so one step costs a
 * constant number of word operations per pair.  After every step the outputs
 * equal sr_gate(K = max_steps) on the prefixes emitted so far.
 *
 * The state is position independent: a byte copy of the buffer is a valid
 * snapshot and can be restored into any other buffer of the same size.
 *
 *   sr_incr_state_bytes  host-only, pure; 0 for invalid arguments
 *   sr_incr_init         formats `state` for n_groups x N rollouts of length 0;
 *                        max_steps in 1..SR_MAX_INCR_STEPS
 *   sr_gate_step_incremental
 *     new_actions in  [n_groups][N] int32; SR_NO_ACTION = no action this step.
 *                     An action for a rollout already holding max_steps actions is
 *                     ignored and sets SR_STATUS_STEP_OVERFLOW.
 *     outputs as for sr_gate (pair_dist, pair_sum, mean may be NULL).
 *     n_groups, N must match sr_incr_init, else SR_STATUS_BAD_STATE is set and
 *     the step does nothing.
 */
size_t sr_incr_state_bytes(int32_t n_groups, int32_t N, int32_t max_steps);
int sr_incr_init(void* state, size_t state_bytes, int32_t n_groups, int32_t N,
                 int32_t max_steps, void* stream);
int sr_gate_step_incremental(void* state, size_t state_bytes, const int32_t* new_actions,
                             int32_t n_groups, int32_t N, double threshold, int32_t norm_mode,
                             int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                             int32_t* status, void* stream);

/*
 * sr_gate_or_rule -- termination fraction tau_K (Appendix B, "termination_fraction")
 * and the two-clause gate of the OR-rule extension (Eq. 3):
 *     stop[g] = (mean[g] < threshold) || (tau[g] >= tau_high),
 * tau[g] = (finished rollouts of group g) / N in fp64.  A rollout counts as finished
 * by step K when its `done` byte is non-zero or, when done == NULL, when it has emitted
 * fewer than K actions (lens[g][i] < K).  tau_high > 1 reduces the rule to Eq. 2.
 *
 *   mean  in  [n_groups] fp64, d_K as written by sr_gate
 *   lens  in  [n_groups][N] int32; required when done == NULL
 *   done  in  [n_groups][N] uint8 or NULL
 *   tau   out [n_groups] fp64; may be NULL
 *   stop  out [n_groups] uint8; required
 */
int sr_gate_or_rule(const double* mean, const int32_t* lens, const uint8_t* done, int32_t n_groups,
                    int32_t N, int32_t K, double threshold, double tau_high, double* tau,
                    uint8_t* stop, void* stream);

/*
 * sr_grpo_advantage -- Eq. 1: A_i = (r_i - mean_r) / (sigma_r + eps) with the
 * population standard deviation (1/N), accumulated in fp64 and rounded once to
 * fp32.  zero_var[g] = 1 iff all N rewards of the group compare equal (Section
 * 2.1); such a group, and every group whose drop_mask byte is non-zero (a group
 * cut by the gate never enters the loss, Appendix C.1), gets A_i = +0.0 exactly.
 * NaN rewards compare unequal and propagate.
 *
 *   rewards    in  [n_groups][N] fp32
 *   drop_mask  in  [n_groups] uint8 or NULL
 *   adv        out [n_groups][N] fp32
 *   zero_var   out [n_groups] uint8; may be NULL
 */
int sr_grpo_advantage(const float* rewards, const uint8_t* drop_mask, int32_t n_groups,
                      int32_t N, float eps, float* adv, uint8_t* zero_var, void* stream);

/*
 * sr_group_signals -- the other action-only divergence signals of Appendix B, computed
 * on the same prefixes as d_K (prefix of rollout i = its first min(len_i, K) actions).
 * Every output is [n_groups] fp64 and may be NULL.
 *
 *   unique_prefix_ratio  distinct prefixes / N (equal = same length, same actions)
 *   unique_action_ratio  distinct values among the step-K actions a_{i,K}, / N; rollouts
 *                        that ended before step K share one extra value "no action"
 *   action_entropy       Shannon entropy of that empirical distribution (natural log)
 *                        divided by ln N, so that it lies in [0, 1] as Appendix B states
 *   bigram_jaccard_mean  mean over the pairs (fp64, pair order) of 1 - |A n B| / |A u B|,
 *                        A, B = the SETS of consecutive action pairs of the two prefixes;
 *                        a pair of prefixes without any bigram contributes 0
 *
 * seqs / lens / stride / K as for sr_gate, with K <= 32 (action-level prefixes).  The
 * ratios and the Jaccard mean are exact to the last bit of their definition; the entropy
 * goes through the device logarithm and agrees with a host libm to a few ulp.
 * (Not computed: obs_unique_ratio, which needs the environment's observations.)
 */
int sr_group_signals(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                     int32_t stride, int32_t K, double* unique_prefix_ratio,
                     double* unique_action_ratio, double* action_entropy,
                     double* bigram_jaccard_mean, void* stream);

/*
 * sr_batch_stats -- batch reductions behind two of the paper's figures: the share of
 * zero-advantage trajectories that dilutes the batch-mean loss (Section 4.5: about 40 %
 * without the gate, 28 % with it) and the advantage norm kept after cutting,
 * ||A_kept||_2 / ||A_full||_2 (Section 3.4: 96.7 % at the chosen threshold).
 *
 *   adv     in  [n_groups][N] fp32 advantages computed WITHOUT a drop mask
 *   stop    in  [n_groups] uint8 gate decisions, or NULL (every group kept)
 *   counts  out 3 int64: [0] advantages equal to zero over all groups,
 *                        [1] the same over kept groups (stop == 0), [2] kept groups
 *   sumsq   out 2 fp64:  [0] sum of squared advantages over all groups, [1] over kept
 *
 * The fp64 sums are accumulated in parallel (thread, block, then atomics), so they are
 * reproducible to about 1e-12 relative, not bit for bit; the counts are exact.
 */
int sr_batch_stats(const float* adv, const uint8_t* stop, int32_t n_groups, int32_t N,
                   int64_t* counts, double* sumsq, void* stream);

/*
 * sr_kept_groups -- the groups that stay in the training batch, as an index list.  The
 * trainer skips a group the gate cut (Appendix C.1); the dynamic-sampling baseline the
 * paper compares with (appendix on strong baselines) also drops the groups whose
 * advantages are all zero (Section 2.1).  This call writes the ascending indices g of the
 * groups with stop[g] == 0 and, when zero_var is given, zero_var[g] == 0.
 *
 *   stop       in  [n_groups] uint8 or NULL (no group cut)
 *   zero_var   in  [n_groups] uint8 or NULL (filter off)
 *   index      out [n_groups] int32; the first *count entries are written, ascending
 *   count      out 1 int32 (device)
 *   workspace      device scratch of sr_kept_groups_workspace_bytes(n_groups) bytes,
 *                  16-byte aligned; contents undefined before and after
 *
 * The order does not depend on how the kernels are scheduled.  n_groups == 0 writes
 * *count = 0.
 */
int sr_kept_groups(const uint8_t* stop, const uint8_t* zero_var, int32_t n_groups, int32_t* index,
                   int32_t* count, void* workspace, size_t workspace_bytes, void* stream);
size_t sr_kept_groups_workspace_bytes(int32_t n_groups);   /* host-only, pure */

/* Host-only, pure.  Step-token saving of cutting `cut` of `n_groups` groups at step K of
 * a horizon of T_max steps: cut * (T_max - K) / (n_groups * T_max) (caption of Table 1). */
double sr_savings_fraction(int64_t cut, int64_t n_groups, int32_t T_max, int32_t K);

/* Host-only, pure.  Gradient-norm gain predicted by the dilution argument when the
 * zero-advantage fraction goes from `before` to `after`: (1 - after) / (1 - before)
 * (Section 4.5: 0.72 / 0.60, about 1.20). */
double sr_dilution_gain(double zero_frac_before, double zero_frac_after);

#ifdef __cplusplus
}
#endif
#endif /* SR_GATE_H_ */
