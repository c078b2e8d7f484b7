/*
 * concur_curate -- the arithmetic of the ConCuR data curation (arXiv 2510.07356) over a table of
 * generation records, on the GPU.
 *
 * A record is one generation j of one task i (N tasks x M generations, row-major [N][M]): whether
 * the generated kernel was correct, the run time of the PyTorch program and of the kernel, and the
 * length of the reasoning trace in tokens.  One call computes
 *
 *   speedup[i][j]    Eq. (1):  t_torch / t_kernel * 1[correct]        (float32, IEEE division)
 *   rule_a[i]        Sec. 3.5 (a): the generation with the shortest reasoning (first on ties) if it
 *                    is correct and no generation of the task has a higher speedup; else -1
 *   rule_b[i][j]     Sec. 3.5 (b): speedup > rule_b_speedup (5 in the paper)
 *   pick[s][i], keep[s][i]   Sec. 5, the four ablation selections s = 0 random, 1 longest,
 *                    2 shortest, 3 fastest: the correct generation of the task that the selection
 *                    takes (-1 if none is correct; first on ties), and whether the task is among
 *                    the top_k tasks by that key (ties: lower task index first).  The random
 *                    selection ranks by the keys the caller passes in; the library draws nothing.
 *   difficulty[i]    Sec. 6.1 / Table 4: 0 if the task's mean length < easy_below, 2 if it is
 *                    > hard_above, else 1 (compared exactly, as integer sums)
 *   stats[]          counts and sums, see CONCUR_STAT_*: Eq. (2) fast_p for the first generation
 *                    and for the best generation of every task, Eq. (3) the average reasoning
 *                    length, the Pearson correlation of length and speedup over correct samples
 *                    (Sec. 3.4), and how many samples each rule keeps
 *
 * All pointers are device pointers, caller-owned; the call is asynchronous on `cuda_stream`, keeps
 * nothing, allocates nothing and needs no handle.  Returns CONCUR_OK or a negative concur_status_t
 * (see concur_attn.h): CONCUR_ERR_INVALID_ARG for a null pointer or sizes outside 1 <= N,
 * 1 <= M <= 32, N * M < 2^31; CONCUR_ERR_CUDA if a launch fails.
 */
#ifndef CONCUR_CURATE_H_
#define CONCUR_CURATE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int32_t num_tasks;         /* N */
    int32_t gens;              /* M, generations per task (5 in synthesis, 10 in evaluation) */
    float   rule_b_speedup;    /* rule (b) keeps speedup > this; the paper uses 5 */
    float   fast_p;            /* p of Eq. (2); fast_1 is p = 1 */
    int32_t top_k;             /* tasks each ablation selection keeps; the paper uses 4,892 */
    int32_t easy_below;        /* Table 4: 4000 */
    int32_t hard_above;        /* Table 4: 8500 */
    int32_t reserved;          /* must be 0 */
} concur_curate_params_t;

enum {
    CONCUR_SEL_RANDOM = 0, CONCUR_SEL_MAX_LENGTH = 1, CONCUR_SEL_MIN_LENGTH = 2, CONCUR_SEL_SPEEDUP = 3,
    CONCUR_NUM_SELECTIONS = 4
};

enum {
    CONCUR_STAT_CORRECT = 0,          /* correct samples                                         */
    CONCUR_STAT_TASKS_CORRECT = 1,    /* tasks with at least one correct sample                  */
    CONCUR_STAT_RULE_A = 2,           /* samples kept by rule (a)                                */
    CONCUR_STAT_RULE_B = 3,           /* samples kept by rule (b)                                */
    CONCUR_STAT_LENGTH_SUM = 4,       /* sum of all reasoning lengths                            */
    CONCUR_STAT_ARL = 5,              /* Eq. (3)                                                 */
    CONCUR_STAT_FAST_FIRST_COUNT = 6, /* tasks whose first generation has speedup > p            */
    CONCUR_STAT_FAST_BEST_COUNT = 7,  /* tasks whose best generation has speedup > p             */
    CONCUR_STAT_EXEC_FIRST_COUNT = 8, /* tasks whose first generation is correct                 */
    CONCUR_STAT_N = 9,                /* samples in the correlation (= correct samples)          */
    CONCUR_STAT_SX = 10, CONCUR_STAT_SY = 11, CONCUR_STAT_SXX = 12, CONCUR_STAT_SYY = 13, CONCUR_STAT_SXY = 14,
    CONCUR_STAT_PEARSON_R = 15,       /* NaN with fewer than two samples or a constant column    */
    CONCUR_STAT_FAST_FIRST = 16,      /* Eq. (2) over first generations                          */
    CONCUR_STAT_FAST_BEST = 17,       /* Eq. (2) over best generations                           */
    CONCUR_CURATE_NUM_STATS = 24
};

int concur_curate(const concur_curate_params_t* params,
                  const uint8_t* correct, const float* t_torch, const float* t_kernel, const int32_t* length,
                  const float* sample_key,   /* [N][M] keys of the random selection's per-task choice */
                  const float* task_key,     /* [N]    keys of the random selection's task ranking     */
                  float* speedup,            /* [N][M] */
                  int32_t* rule_a,           /* [N]    */
                  uint8_t* rule_b,           /* [N][M] */
                  int32_t* pick,             /* [4][N] */
                  uint8_t* keep,             /* [4][N] */
                  uint8_t* difficulty,       /* [N]    */
                  double* stats,             /* [CONCUR_CURATE_NUM_STATS] */
                  void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* CONCUR_CURATE_H_ */
