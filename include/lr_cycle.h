/*
 * Host-side timing model and strategy search for Lookahead Reasoning cycles.
 * These calls run on the CPU only (no device, no context needed): they are what
 * a scheduler consults to pick its speculation depths and to predict what a
 * configuration is worth before it spends GPU time on it.
 *
 * Model (Section 3.2, "Theoretical Speedup Analysis", and Appendix B): the
 * target model needs T time units per reasoning step, the draft model c1 * T,
 * verification is free, one draft per position.  Time is integer: T = den and
 * one draft step costs num units (c1 = num / den).  The accept / reject outcome
 * of every draft is an input (a 0/1 byte stream), so a run is reproducible.
 */
#ifndef LR_CYCLE_H_
#define LR_CYCLE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lr_cycle_stats {
  int64_t stages;         /* whole cycles (sync) or stages (async) simulated */
  int64_t steps;          /* reasoning steps emitted */
  int64_t time;           /* wall time in units (T = den) */
  int64_t verdicts_used;  /* entries of the stream that were read */
  int64_t peak_in_flight; /* async: most target generations in flight at once; sync: gamma */
} lr_cycle_stats;

/*
 * Synchronous cycles (Algorithm 1): per cycle gamma - 1 drafts in sequence (num
 * units each), then the target's gamma steps in parallel (den units); the cycle
 * emits the drafts before the first rejected one plus the target's step at that
 * position.  A cycle reads gamma - 1 verdicts (verdicts_h: host uint8, nonzero
 * = accepted); with gamma == 1 it reads none and n_verdicts cycles are run.
 * Runs every whole cycle the stream allows.  LR_EINVAL (-1) for gamma < 1,
 * num < 0, den < 1 or a null pointer with n_verdicts > 0.
 */
int lr_cycle_simulate_sync(int32_t gamma, int64_t num, int64_t den, const uint8_t *verdicts_h, int64_t n_verdicts,
                           lr_cycle_stats *out);

/*
 * Asynchronous stages (Appendix B's three rules).  In a stage, position
 * i = 0, 1, ...: draft i is started as soon as draft i - 1 is written and fewer
 * than gamma target generations are in flight; the target's step i starts at
 * the same moment and takes den units; when it is done draft i is checked, and
 * a rejected draft ends the stage there (it emits drafts 0..i-1 and the
 * target's step i; the next stage starts at once).  A stage reads verdicts up
 * to and including its first zero; a stage the stream ends in is dropped.
 * Same errors as above.
 */
int lr_cycle_simulate_async(int32_t gamma, int64_t num, int64_t den, const uint8_t *verdicts_h, int64_t n_verdicts,
                            lr_cycle_stats *out);

/*
 * Closed forms of Section 3.2 / 3.3: mode 0 = f_sync(k), 1 = f_async(k) (S_1
 * when k >= ceil(1/c), else S_2), 2 = g(k), the token-level speedup.
 * NaN for arguments outside k >= 1, 0 < alpha < 1, 0 < c < 1.
 */
double lr_cycle_speedup(int32_t mode, int32_t k, double alpha, double c);

/*
 * Eq. 1 of Section 3.3: the (k1, k2) in 1..budget that maximise
 * h = f(k1) * g(k2) subject to ParallelDim_f * k2 <= budget, where
 * ParallelDim_f = k1 (sync) or min(ceil(1/c1), k1) (async).  Ties: smaller k1,
 * then smaller k2.  Outputs are host pointers.  LR_EINVAL (-1) for budget < 1,
 * rates or costs outside (0, 1), or a null output.
 */
int lr_cycle_best_strategy(int32_t budget, double alpha1, double c1, double alpha2, double c2, int32_t asynchronous,
                           int32_t *k1_out, int32_t *k2_out, double *h_out);

#ifdef __cplusplus
}
#endif
#endif /* LR_CYCLE_H_ */
