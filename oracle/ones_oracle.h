/*
 * ones_oracle.h — CPU oracle for the ONES evolutionary batch-size search.
 *
 * TEST INFRASTRUCTURE.  This is the slow, single-threaded, plain-C statement of
 * what the search computes.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it; the CUDA library never does and shares no code,
 * header, table or constant generator with it.
 *
 * Parity pins: model, fitness, operators, elitism, repair and the Philox
 * generator are each pinned by the CPU test-suite (hand-worked values, exact
 * rational arithmetic, brute force, an exact knapsack DP, operator invariants,
 * an independently written Philox).  The evolutionary trajectory as a whole is
 * a randomised heuristic for which the paper prints no numbers:
 * "parity unpinned" beyond those per-step pins.
 *
 * All pointers are host pointers.  All functions return 0 on success or a
 * negative ORACLE_ERR_* code; nothing is printed, nothing aborts.
 */
#ifndef ONES_ORACLE_H
#define ONES_ORACLE_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* One job of the set J (paper, Table 1): the batch-size grid B_j = b0 << k, the
 * limit R_j = b0 << kmax, and the coefficients of its profiled throughput X_j. */
typedef struct {
    int32_t b0, max_per_gpu, kmin, kmax;
    double a, c, d, weight;
} oracle_job;

typedef struct {
    int32_t elitism, tournament;
    double p_mut, penalty;
    uint32_t flags;
} oracle_params;

#define ORACLE_FLAG_SRUF 1u /* score = -(sum_j weight_j * c_j / X_j): Alg. 1 score, negated */
/* bit 2 (value 2) only selects a launch sequence in the CUDA library; it means nothing here */
#define ORACLE_FLAG_TRUNCATION 4u /* the paper's selection: best K of K originals + 2K crossover children + K mutants */

/* bit 8 means nothing here either (launch sequence) */
#define ORACLE_FLAG_PER_GPU 16u /* the paper's own genome: one slot per GPU holding a job id (Eq. 1-2, Fig. 1) */

enum {
    ORACLE_OK = 0,
    ORACLE_ERR_NULL = -1,
    ORACLE_ERR_BAD_JOB = -2,
    ORACLE_ERR_BAD_PARAM = -3,
    ORACLE_ERR_NOMEM = -4,
    ORACLE_ERR_INFEASIBLE = -5
};

enum { ORACLE_STREAM_INIT = 0, ORACLE_STREAM_SEL_A = 1, ORACLE_STREAM_SEL_B = 2, ORACLE_STREAM_MUT = 3,
       ORACLE_STREAM_PICK = 4, ORACLE_STREAM_MUTANT = 5 };

typedef struct oracle_ctx oracle_ctx;

/* ---- stateless pieces (each is one step of the method) ---- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
/* random word for (absolute generation, row, column, stream) under a 64-bit seed */
uint32_t oracle_word(uint64_t seed, uint64_t gen_abs, uint32_t row, uint32_t col, uint32_t stream);
/* throughput model: X (samples/s) and g (= c_j, GPUs) of job at exponent k; a gene
 * outside [0, kmax] is a waiting job: X = 0, g = 0 */
int oracle_model(const oracle_job* job, int32_t k, double* X, int32_t* g);
/* per-gene score term (throughput, or the negated SRUF term when flags has SRUF) */
int oracle_term(const oracle_job* job, int32_t k, uint32_t flags, double* term, int32_t* g);
/* fitness and GPU demand of one genome */
int oracle_fitness(const oracle_job* jobs, int32_t n_jobs, int32_t capacity, double penalty,
                   uint32_t flags, const int32_t* genome, double* F, int32_t* gpus);
int oracle_validate_jobs(const oracle_job* jobs, int32_t n_jobs);
/* deterministic repair of one genome to GPU demand <= capacity; parked genes become -1 */
int oracle_repair(const oracle_job* jobs, int32_t n_jobs, int32_t capacity, int32_t* genome);
/* tournament of `tournament` draws among n candidates for pair q */
int32_t oracle_tournament(const double* F, int32_t n, int32_t tournament, uint64_t seed,
                          uint64_t gen_abs, uint32_t q, uint32_t stream);
/* indices of the e best candidates (F descending, index ascending) */
int oracle_top(const double* F, int32_t n, int32_t e, int32_t* idx);
/* per-GPU genome: `slots` holds one job id per GPU (anything outside [0, n_jobs) = idle).  Job j holds
 * c_j = the number of its slots (Eq. 2) and runs at the largest admissible batch whose GPU need fits:
 * the largest k in [kmin_j, kmax_j] with ceil(b0 << k / max_per_gpu) <= c_j; with none it waits.
 * exponents (nullable) receives that k per job, or -1. */
int oracle_fitness_per_gpu(const oracle_job* jobs, int32_t n_jobs, int32_t n_gpus, uint32_t flags,
                           const int32_t* slots, double* F, int32_t* gpus_used, int32_t* exponents);
/* "Reorder": the workers of a job become neighbours, jobs in the order of their first occurrence,
 * idle GPUs last */
int oracle_reorder(int32_t* slots, int32_t n_gpus, int32_t n_jobs);
/* "Refresh" of one per-GPU candidate when the job set changes (Section 3.2.2, Fig. 5), in four steps:
 * (1) slots of finished jobs become idle and surviving jobs take their new ids (inv[old id] = new id or -1);
 * (2) a job holding more GPUs than its batch-size limit needs gives up the surplus, last slots first;
 * (3) each new job (is_new) gets the GPUs of its smallest batch: the lowest idle slots, else the last slot of
 *     the lowest-index (longest present) surviving job that still holds one;
 * (4) while a GPU is idle: the job below its limit whose score term gains most from growing to the limit
 *     (ties: lower index) takes the GPUs it needs for that, or what is left, lowest idle slots first.
 * The row is not packed here (see oracle_reorder). */
int oracle_refresh(const oracle_job* jobs, int32_t n_jobs, uint32_t flags, const int32_t* inv, int32_t n_jobs_old,
                   const char* is_new, int32_t* slots, int32_t n_gpus);
/* the k best of n scores, as ascending indices (truncation selection, order preserved) */
int oracle_keep_best(const double* F, int32_t n, int32_t k, int32_t* kept);
/* mutation threshold on the 16-bit decision field for probability p */
uint32_t oracle_thr16(double p_mut);

/* ---- the search ---- */
int oracle_create(oracle_ctx** out, const oracle_job* jobs, int32_t n_jobs, int32_t capacity,
                  int32_t pop, const oracle_params* prm);
int oracle_destroy(oracle_ctx*);
int oracle_randomize(oracle_ctx*, uint64_t seed);
int oracle_set_population(oracle_ctx*, const int32_t* genomes, int64_t ld);
int oracle_get_population(oracle_ctx*, int32_t* genomes, int64_t ld);
/* genomes == NULL: the current population (n, ld ignored) */
int oracle_evaluate(oracle_ctx*, const int32_t* genomes, int64_t ld, int32_t n, double* fitness,
                    int32_t* gpus);
int oracle_evolve(oracle_ctx*, int32_t generations, uint64_t seed);
int oracle_best(oracle_ctx*, int repair, int32_t* genome, int32_t* gpus_per_job, double* rate_per_job,
                double* fitness, int32_t* total_gpus, int32_t* index);
int oracle_update_jobs(oracle_ctx*, const oracle_job* jobs, int32_t n_jobs, const int32_t* remap,
                       int32_t capacity);
int oracle_last_parents(oracle_ctx*, int32_t* parents /*[pairs][2]*/, int32_t* elites /*[E]*/);
int oracle_generation(const oracle_ctx*, uint64_t* gen_abs);
int oracle_set_generation(oracle_ctx*, uint64_t gen_abs); /* resume a saved search */
int32_t oracle_pairs(const oracle_ctx*);

#ifdef __cplusplus
}
#endif
#endif
