/*
 * ones.h — C ABI of the B200 evolutionary batch-size search (ONES, SC'21).
 *
 * One scheduling round of ONES scores a population of candidate schedules and
 * evolves it (paper, Section 3.2.2: initialisation, uniform crossover, uniform
 * mutation, selection, update with the best candidate S*).  This library runs
 * that loop on one GPU.  A candidate S (Eq. 1-2) is one row of int32 exponents,
 * one per job: job j runs with global batch B_j = b0_j << k_j on
 * c_j = ceil(B_j / max_per_gpu_j) GPUs; a gene outside [0, kmax_j] means the job
 * waits (B_j = c_j = 0, text after Eq. 2).
 *
 * Conventions
 *  - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global
 *    memory of the device that was current at ones_create.  The caller owns every
 *    buffer it passes, including the device workspace; the handle owns only small
 *    host-side state (including a few KiB of pinned host memory through which job tables
 *    are uploaded and the best schedule is downloaded).  Nothing here allocates or frees
 *    device memory.
 *  - Genome tables are row-major int32[n][ld], ld >= number of jobs, ld % 4 == 0,
 *    base address 16-byte aligned.  Columns >= number of jobs are never read as
 *    genes and never written.
 *  - Calls on a handle make the handle's device current for their duration and restore the
 *    caller's device before returning.
 *  - All work is enqueued on the CUDA stream given to ones_create.  Calls that
 *    return data to host memory synchronise that stream; the others do not.
 *  - Every function returns ONES_OK (0) or a negative ONES_ERR_* code.  Nothing is
 *    printed, nothing aborts.  An asynchronous CUDA fault surfaces as
 *    ONES_ERR_CUDA at the next synchronising call.
 *  - A handle is not thread-safe; different handles may be used from different
 *    threads.
 */
#ifndef ONES_H
#define ONES_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ones_ctx ones_ctx;

/* One job of the set J (Table 1).  b0 << k, k in [kmin, kmax], is the batch-size
 * grid and b0 << kmax the batch-size limit R_j (Section 3.2.2, "Evolution");
 * a, c, d are the coefficients of the job's profiled throughput X_j (Eq. 5):
 * seconds per iteration t = a + c * (B / g) + d * log2(g) on g GPUs, X = B / t.
 * log2(g) is the exact integer for a power of two; for any other g it is taken with the host's
 * math library when the job table is set and uploaded, not computed on the device.
 * weight is the per-job factor Y_processed * (1/rho - 1) of Alg. 1's score; it is
 * used only with ONES_FLAG_SRUF.  48 bytes. */
typedef struct {
    int32_t b0, max_per_gpu, kmin, kmax;
    double a, c, d, weight;
} ones_job;

/* Search parameters.  elitism: candidates that survive unchanged per generation;
 * tournament: draws per parent; p_mut: mutation rate theta per gene ("Uniform
 * mutation"); penalty: score lost per GPU above the cluster's capacity (Eq. 4 as a
 * soft constraint).  NULL where a ones_params* is expected means {2, 4, 0.1, 1e3, 0}.
 * p_mut is applied with a resolution of 1/65536: a gene mutates when a uniform 16-bit field is below
 * lround(p_mut * 65536), so the effective rate is that threshold / 65536 (0.1 -> 6554/65536).  A positive
 * p_mut that rounds to a threshold of 0 (below 2^-17) is rejected with ONES_ERR_BAD_PARAM rather than
 * silently switching mutation off. */
typedef struct {
    int32_t elitism, tournament;
    double p_mut, penalty;
    uint32_t flags;
} ones_params;

/* Score = -(sum_j weight_j * c_j / X_j): Alg. 1 / Eq. 8 (smallest remaining
 * utilisation first), negated so that higher is better.  Default score:
 * sum_j X_j (predicted cluster progress in samples per second). */
#define ONES_FLAG_SRUF 1u

/* Score each new population with a separate pass over it instead of inside the kernel that
 * writes it.  Results are identical; this only selects the launch sequence (used to time the
 * crossover/mutation and the fitness kernels on their own). */
#define ONES_FLAG_UNFUSED 2u

/* ones_evolve runs the paper's own scheme (Section 3.2.2 "Evolution", "Selection") instead of
 * tournament + elitism: per generation the pool G' = the pop current candidates (rows 0..pop-1),
 * 2*pop children of pop uniformly drawn parent pairs (uniform crossover, no mutation; rows
 * pop..3*pop-1) and pop mutants of pop uniformly drawn candidates (each job redrawn with rate p_mut;
 * rows 3*pop..4*pop-1) is scored and the best pop of the 4*pop (score descending, row ascending)
 * survive, in the order of their rows.  elitism and tournament are ignored.  The workspace must be
 * sized with ones_workspace_bytes_flags (the pool takes 4x the rows).  ones_last_parents then
 * returns [pop][2] parent rows. */
#define ONES_FLAG_TRUNCATION 4u

/* Small populations normally run all generations of a ones_evolve call in one launch of one
 * thread-block cluster, with the population in the cluster's shared memory.  This flag keeps the
 * launch-per-generation sequence instead (same results).  With ONES_FLAG_TRUNCATION the flag keeps the
 * survivors' gather into the second pool after every generation, where the default uses the pool in place
 * through a row map and orders the candidates only when they are read (same results). */
#define ONES_FLAG_NO_CLUSTER 8u

/* The paper's own genome (Eq. 1-2, Fig. 1): a candidate is one int32 per GPU of the cluster holding the
 * id of the job that runs there (anything outside [0, n_jobs) = idle), so genome tables are
 * int32[n][ld] with ld >= capacity.  Job j holds c_j = the number of its GPUs and runs at the largest
 * exponent in [kmin_j, kmax_j] whose GPU need fits into c_j; with none it waits.  The score is the sum
 * over jobs as before (no penalty: a candidate cannot exceed the cluster).  Crossover acts per GPU,
 * mutation puts a uniformly drawn job on a GPU with rate p_mut, and every new candidate goes through
 * the paper's "Reorder" (the workers of a job become neighbours, jobs in the order of their first
 * occurrence, idle GPUs last).  ones_create starts from an idle cluster.  ones_best returns the best
 * candidate as per-job exponents (h_genome[n_jobs], -1 = waits); the per-GPU rows come from
 * ones_get_population.  ones_update_jobs runs the paper's "Refresh" on every candidate (see there).
 * Not combinable with ONES_FLAG_TRUNCATION.  Size the workspace with ones_workspace_bytes_per_gpu. */
#define ONES_FLAG_PER_GPU 16u

/* The handle keeps its population as packed rows (one byte per gene, the tile layout described at
 * ones_pack_population) and ones_evolve reads parents and writes children as bytes: 2 bytes of device-memory
 * traffic per child gene instead of 8.  Random draws, operators, summation order and therefore children, scores
 * and selections are those of the int32 rows (Section 3.2.2 "Uniform crossover", "Uniform mutation"; Alg. 1's
 * score step).  Everything else keeps its interface: ones_set_population / ones_get_population take and return
 * int32 rows (converted on the way; a gene outside [0, 254] is stored as "waits" and reads back as -1),
 * ones_best and ones_update_jobs work as before, ones_pack_population(NULL) returns the rows as they are.
 * Needs model tables that fit the shared memory of one thread block (about 2300 jobs at kmax 7; otherwise
 * ones_create / ones_update_jobs return ONES_ERR_BAD_PARAM).  Not combinable with ONES_FLAG_TRUNCATION or
 * ONES_FLAG_PER_GPU; ONES_FLAG_UNFUSED and ONES_FLAG_NO_CLUSTER have no effect.  Size the workspace with
 * ones_workspace_bytes_flags. */
#define ONES_FLAG_PACKED 32u

#define ONES_MAX_EXPONENT 15  /* kmax <= 15 */
#define ONES_MAX_ELITES 256   /* elitism <= 256 */

enum {
    ONES_OK = 0,
    ONES_ERR_NULL = -1,       /* a required pointer is NULL */
    ONES_ERR_BAD_JOB = -2,    /* a job row violates the limits listed at ones_create */
    ONES_ERR_BAD_PARAM = -3,  /* a scalar argument or ones_params field is out of range */
    ONES_ERR_ALIGN = -4,      /* pointer not 16-byte aligned or ld % 4 != 0 */
    ONES_ERR_WORKSPACE = -5,  /* workspace too small for this population / job count */
    ONES_ERR_CUDA = -6,       /* a CUDA call failed; see ones_last_cuda_error */
    ONES_ERR_INFEASIBLE = -7, /* repair could not reach the capacity */
    ONES_ERR_NOMEM = -8       /* host allocation failed */
};

/* Bytes of device workspace needed for up to n_jobs_max jobs and a population of
 * pop candidates (two population buffers, fitness, parents, model tables,
 * scratch).  Returns 0 when an argument is out of range. */
size_t ones_workspace_bytes(int32_t n_jobs_max, int32_t pop);
/* The same for a handle created with `flags` (ONES_FLAG_TRUNCATION needs room for its candidate pool). */
size_t ones_workspace_bytes_flags(int32_t n_jobs_max, int32_t pop, uint32_t flags);
/* The same for a handle with ONES_FLAG_PER_GPU (rows hold `capacity` genes); n_jobs_max is the largest job
 * set that ones_update_jobs will be given. */
size_t ones_workspace_bytes_per_gpu(int32_t n_jobs_max, int32_t pop, int32_t capacity);

/* Create a search over `n_jobs` jobs on a cluster of `capacity` GPUs with a
 * population of `pop` candidates (Section 3.2.2 "Initialization": the population
 * G_0 of simple solutions — every job at its smallest batch, gene kmin_j).
 *   jobs        host, n_jobs rows.  Required per row: b0 > 0, max_per_gpu > 0,
 *               0 <= kmin <= kmax <= 15, b0 << kmax < 2^31, a, c, d finite and >= 0,
 *               t > 0 for every k; else ONES_ERR_BAD_JOB.
 *   capacity    |C| > 0.   pop >= elitism + 1.   tournament >= 1.   0 <= p_mut <= 1.
 *   d_workspace device, 256-byte aligned, at least ones_workspace_bytes(n_jobs, pop)
 *               bytes; a larger workspace lets ones_update_jobs grow the job set up
 *               to the n_jobs_max it was sized for.
 *   cuda_stream a cudaStream_t (NULL = the default stream).
 * Builds the per-(job, exponent) throughput table on the device. */
int ones_create(ones_ctx** out, const ones_job* jobs, int32_t n_jobs, int32_t capacity, int32_t pop,
                const ones_params* prm, void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/* Frees the handle's host state.  The workspace stays the caller's. */
int ones_destroy(ones_ctx* ctx);

/* Replace the population: candidate 0 keeps every job at kmin, every other gene is
 * drawn uniformly from [kmin_j, kmax_j] (Philox stream keyed by seed, row, job). */
int ones_randomize(ones_ctx* ctx, uint64_t seed);

/* Copy a population of pop rows in (out of) the handle.  `genomes` is device
 * memory if on_device != 0, host memory otherwise (then the call synchronises). */
int ones_set_population(ones_ctx* ctx, const int32_t* genomes, int64_t ld, int on_device);
int ones_get_population(ones_ctx* ctx, int32_t* genomes, int64_t ld, int on_device);

/* Score candidates (Alg. 1's score step, Eq. 8; capacity constraint Eq. 4):
 *   gpus[i]    = sum_j c_j                      (int32, wraps modulo 2^32)
 *   fitness[i] = sum_j term_j - penalty * max(0, gpus[i] - capacity)   (fp64)
 * with the sum taken in a fixed order: 32 partial sums, job j added to partial
 * (j / 4) % 32 in increasing j, then a pairwise tree (16, 8, 4, 2, 1) over them.
 *   d_genomes  device int32[n][ld], or NULL for the handle's current population
 *              (then ld and n are ignored and n = pop).
 *   d_fitness  device double[n];  d_gpus device int32[n] or NULL. */
int ones_evaluate(ones_ctx* ctx, const int32_t* d_genomes, int64_t ld, int32_t n, double* d_fitness,
                  int32_t* d_gpus);

/* Packed candidates: the same score step (Alg. 1, Eq. 8; Eq. 4) on rows of one byte per gene, a quarter of
 * the bytes of the int32 rows.  A byte holds the exponent (at most 15; any gene outside [0, 254] is stored as
 * 0xFF = the job waits).  A packed row is a sequence of tiles of 512 genes; the row stride ld8 is a multiple of
 * 512 bytes, at least ones_packed_row_bytes(n_jobs).  Inside a tile, byte 16*l + 4*b + s holds gene
 * 128*b + 4*l + s of the tile (l = 0..31, b = 0..3, s = 0..3; genes past n_jobs are 0xFF): one 16-byte load gives
 * a lane the genes it adds, in the order of the fixed summation, so fitness and gpus are bit-identical to
 * ones_evaluate on the int32 rows.
 *   ones_pack_population   d_genomes device int32[n][ld] (NULL: the handle's population, ld and n ignored)
 *                          -> d_packed device uint8[n][ld8], 16-byte aligned.
 *   ones_evaluate_packed   d_packed -> d_fitness device double[n], d_gpus device int32[n] or NULL.
 * Not available with ONES_FLAG_PER_GPU (job ids do not fit a byte).  Asynchronous. */
size_t ones_packed_row_bytes(int32_t n_jobs);
int ones_pack_population(ones_ctx* ctx, const int32_t* d_genomes, int64_t ld, int32_t n, uint8_t* d_packed,
                         int64_t ld8);
int ones_evaluate_packed(ones_ctx* ctx, const uint8_t* d_packed, int64_t ld8, int32_t n, double* d_fitness,
                         int32_t* d_gpus);

/* Run `generations` generations (Fig. 4: G_i -> G'_i -> G_{i+1}).  Each one: the
 * `elitism` best candidates (score descending, index ascending) move unchanged to
 * rows 0..E-1; for every pair of remaining rows two parents are chosen by
 * tournament, uniform crossover gives two complementary children ("Uniform
 * crossover"), each child gene is then redrawn uniformly in [kmin_j, kmax_j] with
 * probability p_mut ("Uniform mutation"), and the new population is scored.
 * Random draws come from Philox4x32-10 keyed by (seed; generation, row, job), the
 * generation counted from ones_create, so evolve(a + b) equals evolve(a) then
 * evolve(b).  Asynchronous. */
int ones_evolve(ones_ctx* ctx, int32_t generations, uint64_t seed);

/* The best candidate S* of the current population (Alg. 1, last step), optionally
 * repaired to fit the cluster: while the GPU demand exceeds the capacity the job
 * holding the most GPUs (lowest index on ties) that can still shrink goes down one
 * exponent; when none can, running jobs wait (gene -1) in increasing index.
 * Host outputs, each nullable: h_genome int32[n_jobs], h_gpus_per_job int32[n_jobs],
 * h_rate_per_job double[n_jobs] (X_j of the returned genes; with ONES_FLAG_SRUF the per-job score
 * terms -weight_j * c_j / X_j instead), fitness, total_gpus,
 * index (row of the population).  With repair the fitness is that of the repaired
 * row.  Synchronises. */
int ones_best(ones_ctx* ctx, int repair, int32_t* h_genome, int32_t* h_gpus_per_job,
              double* h_rate_per_job, double* fitness, int32_t* total_gpus, int32_t* index);

/* New scheduling round with a changed job set (Section 3.2.2 "Refresh": finished
 * jobs leave, new jobs arrive, limits R_j move).  Column j of the new population is
 * column remap[j] of the old one clamped into the new [kmin_j, kmax_j], or kmin_j
 * when remap[j] == -1; the model tables are rebuilt.  jobs, remap: host, n_jobs
 * entries; n_jobs must fit the workspace.  Asynchronous apart from argument checks: the job rows are checked on
 * the host (limits as at ones_create, and a positive, finite throughput for every exponent; else
 * ONES_ERR_BAD_JOB and the search is untouched).  The table kernel repeats the throughput check on the device;
 * should it ever disagree, ONES_ERR_BAD_JOB comes from the next call that synchronises (ones_best,
 * ones_get_population to host memory, ones_last_parents), like any asynchronous fault.
 * When the new set has the same jobs in the same columns (remap[j] == j) and no job's [kmin, kmax] shrinks, no
 * gene can move: the population is left where it is (after ones_set_population the full pass runs, since the
 * caller's genes may lie outside the limits), the tables are rebuilt and the scores are recomputed when next
 * needed; an identical job table and capacity change nothing at all.
 *
 * With ONES_FLAG_PER_GPU the candidates hold job ids, and every candidate goes through the four steps of
 * "Refresh" (Fig. 5) and then "Reorder":
 *   (1) the GPUs of finished jobs (old ids that no remap[j] names) become idle, surviving jobs take their
 *       new ids (should several new rows name one old job, the highest j keeps its GPUs);
 *   (2) a job holding more GPUs than its batch-size limit b0 << kmax needs gives up the surplus, its last
 *       GPUs first;
 *   (3) every new job (remap[j] == -1), in index order, gets the GPUs of its smallest batch: the lowest idle
 *       GPUs, and when none is idle the last GPU of the lowest-index (longest present) surviving job that
 *       still holds one;
 *   (4) while a GPU is idle, the job below its limit whose score term gains most from growing to the limit
 *       (ties: lower index) takes the GPUs it needs for that, or what is left, lowest idle GPUs first.
 * capacity must equal the cluster size of ones_create (ONES_ERR_BAD_PARAM otherwise).  The step keeps one
 * candidate and its per-job lists in the shared memory of a thread block: 8 * capacity + 16 * n_jobs + 16 * P
 * bytes, P = n_jobs rounded up to a power of two (512 for 129..256 jobs), must stay below 226 KiB, else
 * ONES_ERR_WORKSPACE (e.g. 4096 GPUs with up to 4220 jobs, 64 GPUs with up to 6236). */
int ones_update_jobs(ones_ctx* ctx, const ones_job* jobs, int32_t n_jobs, const int32_t* remap,
                     int32_t capacity);

/* Parents [pairs][2] and elites [elitism] chosen in the last generation (host
 * outputs, nullable); pairs = (pop - elitism + 1) / 2.  Synchronises. */
int ones_last_parents(ones_ctx* ctx, int32_t* h_parents, int32_t* h_elites);

/* The device-built model table: X[k][j] and g[k][j] for k = 0..kmax_max (host
 * outputs, row length n_jobs; entries with k > kmax_j are 0).  *planes receives
 * kmax_max + 1.  Pass NULL arrays to query *planes only.  Synchronises. */
int ones_model_table(ones_ctx* ctx, double* h_X, int32_t* h_g, int32_t* planes);

/* Indices of the e best of n scores (descending, ties to the lower index), the
 * selection step on its own.  d_scratch: device, >= ones_select_top_scratch_bytes(n, e),
 * 16-byte aligned.  1 <= e <= min(n, ONES_MAX_ELITES).  Asynchronous on `cuda_stream`. */
size_t ones_select_top_scratch_bytes(int32_t n, int32_t e);
int ones_select_top(const double* d_fitness, int32_t n, int32_t e, int32_t* d_index,
                    void* d_scratch, size_t scratch_bytes, void* cuda_stream);

/* The same selection for callers that cannot pass scratch memory.  (The paper has no counterpart:
 * this is a deployment variant of ones_select_top, not a step of the method.)  It is meant for
 * code that cannot obtain device memory when it runs — e.g. a scheduler plug-in inside a process
 * whose framework already owns the whole device, where cudaMalloc fails and the framework's
 * allocator is out of reach, or a round loop that cannot afford the device-wide synchronisation
 * an allocation implies.  The scratch is a fixed 128 KiB array inside the library's device image
 * (held by every GPU that loads the library until the process exits); the call allocates and
 * frees nothing.
 *   d_fitness, d_index  device, as for ones_select_top.   1 <= e <= min(n, ONES_NOALLOC_MAX_TOP);
 *   a larger e returns ONES_ERR_WORKSPACE (use ones_select_top with your own scratch).
 * The first call on each device looks up the array's device address (that device must be
 * current); make that first call before any stream capture begins.  The address is kept for the
 * life of the process: after cudaDeviceReset (or any other teardown of the device's primary
 * context) it no longer points at the array, so do not call this entry point again in a process
 * that reset the device.  All calls on a device share
 * the one array, which keeps whatever the last call left in it: no part of it needs clearing
 * (each call overwrites every record it later reads), but two calls whose kernels may overlap on
 * the GPU — different streams, or different threads — race on it; serialise them.
 * Asynchronous on `cuda_stream`; results equal those of ones_select_top. */
#define ONES_NOALLOC_MAX_TOP 64
int ones_select_top_noalloc(const double* d_fitness, int32_t n, int32_t e, int32_t* d_index,
                            void* cuda_stream);

/* Absolute generation counter, jobs and population of the handle. */
int ones_generation(const ones_ctx* ctx, uint64_t* gen_abs);
/* Resume a saved search: a handle created with the same jobs and parameters, given the saved
 * population (ones_set_population) and the saved generation counter, continues exactly as the
 * original would have (the random draws are keyed by the absolute generation). */
int ones_set_generation(ones_ctx* ctx, uint64_t gen_abs);
int ones_shape(const ones_ctx* ctx, int32_t* n_jobs, int32_t* pop, int32_t* capacity, int64_t* ld);

/* Kernel launches issued through this handle so far. */
int ones_kernel_launches(const ones_ctx* ctx, uint64_t* launches);

/* Per-stage device time.  With profiling on (on = 1: every generation, on = n > 1: every n-th
 * generation of a ones_evolve call), ones_evolve and ones_evaluate bracket
 * each kernel with CUDA events.  ones_stage_times synchronises and returns, for
 * stage s in {0 fitness (separate scoring passes), 1 select+elites, 2 evolve (crossover, mutation
 * and, unless ONES_FLAG_UNFUSED, the scoring of the children)}, the summed milliseconds
 * ms[s] and launch counts count[s] since the last call, then clears them. */
int ones_set_profiling(ones_ctx* ctx, int on);
int ones_stage_times(ones_ctx* ctx, double ms[3], uint64_t count[3]);

/* The cudaError_t of the last failed CUDA call of this handle (0 if none). */
int ones_last_cuda_error(const ones_ctx* ctx);
const char* ones_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif
