/*
 * Data-parallel device ops of the same library (libssn.so): the elementwise steps of AsyncSPARTA
 * (Sec. 4.2, Eq. sparta, Eq. delta_rule; Algorithm 3, one worker's view of an averaging round)
 * and stage-wise gradient clipping (Sec. 4.3).  C ABI, raw DEVICE pointers unless a comment says
 * host, element counts, a cudaStream_t passed as void*; nothing is allocated, freed or
 * synchronised inside.  Parameter buffers are fp32, as the round's buffer is in Algorithm 3
 * (its first step refreshes an fp32 copy).  Status codes are those of ssn.h.  Buffers of one call must not overlap
 * unless stated; 16-byte aligned pointers get 128-bit accesses, others element-wise ones.
 */
#ifndef AGORA_DP_H_
#define AGORA_DP_H_

#include "ssn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * The index set of a round (Algorithm 3: a fraction s of the parameters that rotates with the step, the same on
 * every peer; consecutive rounds cover every parameter once per 1/s rounds): the contiguous
 * segment [*lo, *hi) with r = round mod R, R = rounds_per_cycle (20 for s = 5 %),
 *     lo = floor(n r / R) rounded down to a multiple of SPARTA_SEGMENT_ALIGN,
 *     hi = the lo of segment r + 1, or n for the last segment,
 * so that the R segments tile [0, n) and each starts on a 256-byte boundary of an aligned fp32
 * buffer (128-bit accesses for the ops below).  Host arithmetic only; lo and hi are host pointers.
 */
#define SPARTA_SEGMENT_ALIGN 64
ssn_status_t sparta_segment(int64_t n_params, int32_t rounds_per_cycle, int64_t round,
                            int64_t *lo, int64_t *hi);

/* Algorithm 3, the snapshot step of a sender: snap[0 : hi - lo] = buf[lo : hi]. */
ssn_status_t sparta_snapshot(const float *buf, int64_t lo, int64_t hi, float *snap, void *stream);

/* Algorithm 3, reducer, per arriving chunk c_i of sender i: acc[0:count] += w * chunk[0:count]
 * (a sender of weight 0 takes part in the round without contributing). */
ssn_status_t sparta_accumulate(float *acc, const float *chunk, float w, int64_t count, void *stream);

/*
 * Algorithm 3, reducer, all senders accounted: acc /= sum_w, and every sender i gets
 * deltas[i] = acc - chunks[i].  chunks and deltas are HOST arrays of `senders` device pointers
 * (1 <= senders <= SPARTA_MAX_SENDERS per call; deltas[i] may be chunks[i]: in place); acc is
 * left holding the weighted mean.  sum_w must be > 0.
 */
#define SPARTA_MAX_SENDERS 16
ssn_status_t sparta_deltas(float *acc, float sum_w, const float *const *chunks, float *const *deltas,
                           int32_t senders, int64_t count, void *stream);

/* Algorithm 3, sender, on receiving its deltas: buf[lo : hi] += delta[0 : hi - lo]. */
ssn_status_t sparta_add_delta(float *buf, int64_t lo, int64_t hi, const float *delta, void *stream);

/*
 * Eq. delta_rule / Algorithm 3 ApplyFinishedRound: the weights advanced while the round ran, so the
 * average is applied as a correction,
 *     theta[lo : hi] += lambda * (avg[0 : hi - lo] - snap[0 : hi - lo])
 * with avg the group average of the segment (buf[P] after the round) and snap the snapshot the
 * replica contributed; the paper uses lambda = 1.
 */
ssn_status_t sparta_apply_round(float *theta, int64_t lo, int64_t hi, const float *avg,
                                const float *snap, float lambda, void *stream);

/*
 * Stage-wise clipping threshold (Sec. 4.3): an equal split of a unit squared-norm budget over the
 * S stages, 1 / sqrt(S), doubled for the tail stage.  Host arithmetic; 0 when n_stages < 1.
 */
float stage_clip_threshold(int32_t n_stages, int32_t is_tail);

/*
 * Squared 2-norm of one gradient tensor added to *sumsq (DEVICE double, zeroed by the caller before
 * the first tensor of the stage): *sumsq += sum_i grad[i]^2, accumulated in fp64.  dtype is SSN_F32
 * or SSN_BF16.  The sums of the thread blocks are added atomically, so the last bits depend on
 * their order.
 */
ssn_status_t stage_clip_sumsq(const void *grad, int64_t count, int32_t dtype, double *sumsq, void *stream);

/*
 * Clips one gradient tensor of the stage in place by the stage's norm (the paper gives the
 * thresholds, not the formula; this is the usual clip-by-norm): with norm = sqrt(*sumsq),
 *     coef = min(1, threshold / (norm + 1e-6));   grad[i] *= coef
 * Nothing is written when coef == 1 (the kernel returns after reading *sumsq).
 */
ssn_status_t stage_clip_scale(void *grad, int64_t count, int32_t dtype, const double *sumsq,
                              float threshold, void *stream);

#ifdef __cplusplus
}
#endif

#endif /* AGORA_DP_H_ */
