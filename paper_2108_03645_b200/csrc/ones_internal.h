// Internal interface between the C ABI (ones_api.cu) and the kernels (ones_kernels.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "ones.h"

namespace ones {

constexpr int kSMsDefault = 148;          // B200: 2 dies x 74 SMs (used only when the device cannot be asked)
constexpr int kSMsMax = 192;              // bound on the SM count that per-SM scratch lists are sized for
int sm_count();                           // SMs of the current device, at most kSMsMax
constexpr int kMaxSmemPerBlock = 232448;  // 227 KiB opt-in dynamic shared memory per CTA
constexpr int kTopBlocksMax = 128;        // partial top-k blocks

enum Stream : uint32_t {
    STREAM_INIT = 0, STREAM_SEL_A = 1, STREAM_SEL_B = 2, STREAM_MUT = 3, STREAM_PICK = 4, STREAM_MUTANT = 5
};

// Philox4x32-10 round keys for one 64-bit seed: key word pair of round r is
// (k[2r], k[2r+1]).  Passed to kernels by value so they sit in the constant bank.
struct RoundKeys {
    uint32_t k[20];
};
RoundKeys make_round_keys(uint64_t seed);

// Geometry of the per-(exponent, job) model tables on the device.
//   X[p * jpad + slot(j)], G[p * jpad + slot(j)], p = min(unsigned(k), k1): plane k1 is the
//   all-zero "job waits" plane; entries with k > kmax_j or j >= n_jobs are zero too.
//   slot(j) = (j & ~127) + (j & 3) * 32 + ((j >> 2) & 31): within a block of 128 jobs the
//   four genes of one int4 load land in four 32-entry runs, one entry per lane.
struct Tables {
    double* X;
    int32_t* G;
    int32_t* kmin;   // [jpad] lowest exponent of job j (0 for padding columns)
    int32_t* range;  // [jpad] kmax - kmin + 1 (1 for padding columns)
    int32_t jpad;    // n_jobs rounded up to a multiple of 128
    int32_t k1;      // max_j kmax_j + 1
};

struct BestOut {  // device record written by the best/repair kernel
    double fitness;
    int32_t total_gpus;
    int32_t index;
    int32_t status;  // 0 ok, 1 could not reach capacity
    int32_t steps;
};

// d_log2g: NULL, or log2 of the GPU count per (exponent, job) as double[k1][n_jobs] for job tables whose GPU counts
// are not all powers of two (computed by the caller's math library so that both sides of a comparison agree)
cudaError_t launch_build_tables(const ones_job* d_jobs, int32_t n_jobs, uint32_t flags, Tables t,
                                const double* d_log2g,
                                int32_t* d_bad /*set to 1 when a throughput is not positive and finite*/,
                                cudaStream_t s);
cudaError_t launch_fill_min(int32_t* pop, int64_t ld, int32_t n, int32_t n_jobs, Tables t, cudaStream_t s);
cudaError_t launch_randomize(int32_t* pop, int64_t ld, int32_t n, int32_t n_jobs, Tables t,
                             RoundKeys keys, cudaStream_t s);
cudaError_t launch_fitness(const int32_t* genomes, int64_t ld, int32_t n, int32_t n_jobs, Tables t,
                           int32_t capacity, double penalty, double* F, int32_t* G, cudaStream_t s);
// packed candidates (one byte per gene, tiles of 512 genes ordered for one 16-byte load per lane; ld8 % 512 == 0)
cudaError_t launch_pack_rows(const int32_t* src, int64_t ld, int32_t n, int32_t n_jobs, uint8_t* dst, int64_t ld8,
                             cudaStream_t s);
cudaError_t launch_fitness_packed(const uint8_t* rows, int64_t ld8, int32_t n, Tables t, int32_t capacity,
                                  double penalty, double* F, int32_t* G, cudaStream_t s);
// packed rows -> int32 rows (0xFF -> -1); row_index != NULL: only row *row_index, into the same row of dst
cudaError_t launch_unpack_rows(const uint8_t* src, int64_t ld8, int32_t n, int32_t n_jobs, int32_t* dst, int64_t ld,
                               const int32_t* row_index, cudaStream_t s);
// crossover + mutation + scoring on packed rows (as launch_evolve_score: same tables, same counter)
cudaError_t launch_evolve_score_packed(const uint8_t* src, uint8_t* dst, int64_t ld8, int32_t n, int32_t n_jobs, int32_t elitism,
                                       int32_t pairs, const int32_t* parents, const int32_t* elites, Tables t,
                                       RoundKeys keys, uint64_t gen, uint32_t thr16, int32_t capacity, double penalty,
                                       double* F, int32_t* G, unsigned int* work, cudaStream_t s);
// tournaments + top-e in one launch; *done must be 0 at launch (the kernel leaves it 0); done[1] is cleared for
// the work-item counter of launch_evolve_score
cudaError_t launch_select_stage(const double* F, int32_t n, int32_t tournament, int32_t pairs, RoundKeys keys,
                                uint64_t gen, int32_t* parents, int32_t e, int32_t* elites, void* scratch,
                                unsigned int* done, cudaStream_t s);
size_t top_scratch_bytes(int32_t n, int32_t e);
cudaError_t launch_top(const double* F, int32_t n, int32_t e, int32_t* idx_out, void* scratch,
                       cudaStream_t s, int* launches);
cudaError_t launch_evolve(const int32_t* src, int32_t* dst, int64_t ld, int32_t n, int32_t n_jobs,
                          int32_t elitism, int32_t pairs, const int32_t* parents, const int32_t* elites,
                          Tables t, RoundKeys keys, uint64_t gen, uint32_t thr16, cudaStream_t s);
// crossover + mutation + scoring of the children in one pass; needs evolve_score_smem(t) <= kMaxSmemPerBlock;
// *work: counter that is zero at launch (launch_select_stage clears done[1])
size_t evolve_score_smem(Tables t);
cudaError_t launch_evolve_score(const int32_t* src, int32_t* dst, int64_t ld, int32_t n, int32_t n_jobs,
                                int32_t elitism, int32_t pairs, const int32_t* parents, const int32_t* elites,
                                Tables t, RoundKeys keys, uint64_t gen, uint32_t thr16, int32_t capacity,
                                double penalty, double* F, int32_t* G, unsigned int* work,
                                bool in_limits /* every gene lies in its job's [kmin, kmax] */, cudaStream_t s);
// One launch per generation (tournaments + crossover + mutation + scoring + the next generation's elites).
struct GenerationShape {
    int blocks, threads;  // blocks == 0: not applicable, use the multi-launch sequence
    int32_t queue_cap;
    size_t smem;
};
size_t generation_scratch_bytes(int32_t e);
GenerationShape generation_shape(Tables t, int32_t pairs, int32_t elitism);
cudaError_t launch_generation(GenerationShape shape, const int32_t* src, int32_t* dst, int64_t ld, int32_t n,
                              int32_t n_jobs, int32_t elitism, int32_t pairs, int32_t tournament, const double* F_old,
                              double* F_new, int32_t* G, int32_t* parents, const int32_t* elites,
                              int32_t* elites_next, Tables t, RoundKeys keys, uint64_t gen, uint32_t thr16,
                              int32_t capacity, double penalty, void* scratch, unsigned int* done, cudaStream_t s);
// All generations of one call in one launch of one thread-block cluster (population in distributed shared memory)
struct ClusterShape {
    int cluster, threads;  // cluster == 0: not applicable
    int32_t rows_per_cta;
    int gs;                // lanes per pair of children
    size_t smem;
};
ClusterShape cluster_shape(Tables t, int64_t ld, int32_t n, int32_t elitism, int32_t pairs);
cudaError_t launch_evolve_cluster(ClusterShape shape, int32_t* pop_io, int64_t ld, int32_t n, int32_t n_jobs,
                                  int32_t elitism, int32_t pairs, int32_t tournament, double* F_io, int32_t* G_out,
                                  int32_t* parents_out, int32_t* elites_out, Tables t, RoundKeys keys, uint64_t gen0,
                                  int32_t generations, uint32_t thr16, int32_t capacity, double penalty, cudaStream_t s);
// The paper's truncation selection over a pool of 4K rows (ONES_FLAG_TRUNCATION)
size_t trunc_scratch_bytes(int32_t k);
cudaError_t launch_trunc_children(int32_t* pool, int64_t ld, int32_t k, int32_t* draws, Tables t, RoundKeys keys,
                                  uint64_t gen, uint32_t thr16, cudaStream_t s);  // 2 launches
// the same, scoring the 3K new rows in the same pass (needs evolve_score_smem(t) <= kMaxSmemPerBlock) and drawing
// the parents itself (written to draws[] for ones_last_parents); 1 launch
cudaError_t launch_trunc_children_score(int32_t* pool, int64_t ld, int32_t k, int32_t* draws, Tables t, RoundKeys keys,
                                        uint64_t gen, uint32_t thr16, int32_t capacity, double penalty, double* F,
                                        int32_t* G, const int32_t* rowmap /* nullptr: logical row = pool row */,
                                        cudaStream_t s);
// selection without copying a row: the pool is used in place through a map logical row -> pool row (4k entries)
bool trunc_inplace_available(int32_t k);
cudaError_t launch_trunc_select_inplace(int32_t k, const double* F, const int32_t* G, double* F_next, int32_t* G_next,
                                        const int32_t* oldmap, int32_t* newmap, cudaStream_t s);  // 1 launch
cudaError_t launch_trunc_compact(const int32_t* pool, int32_t* pool_next, int64_t ld, int32_t k, const int32_t* rowmap,
                                 cudaStream_t s);  // logical rows 0..k-1 -> rows 0..k-1 of pool_next
cudaError_t launch_trunc_select(const int32_t* pool, int32_t* pool_next, int64_t ld, int32_t k, const double* F,
                                const int32_t* G, double* F_next, int32_t* G_next, void* scratch,
                                cudaStream_t s, int* launches);  // 2 launches (pools up to 262144 rows) or 12
// The paper's per-GPU genome (ONES_FLAG_PER_GPU): scoring, the reorder operation, slot limits, best
// narrow: n_gpus * max_per_gpu < 2^31 for every job, so the exponent search may use 32-bit arithmetic
cudaError_t launch_fitness_per_gpu(const int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs,
                                   Tables t, const int4* fit, bool narrow, double* F, int32_t* G, cudaStream_t s);
cudaError_t launch_reorder(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, cudaStream_t s);
// reorder and score in one pass over the rows
cudaError_t launch_reorder_score(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, Tables t,
                                 const int4* fit, bool narrow, double* F, int32_t* G, cudaStream_t s);
cudaError_t launch_fill_slot_limits(int32_t* kmin, int32_t* range, int32_t len, int32_t n_gpus, int32_t n_jobs,
                                    const ones_job* jobs, int4* fit, int32_t jpad, cudaStream_t s);
cudaError_t launch_best_per_gpu(const int32_t* pop, int64_t ld, int32_t n_gpus, int32_t n_jobs, const int32_t* best_index,
                                Tables t, int32_t* work, int32_t* genome_out, int32_t* gpus_out, double* rate_out,
                                BestOut* out, cudaStream_t s);
// "Refresh" of every per-GPU candidate at a job-set change (tables, fit and remap are those of the new job
// set, n_old the size of the old one); inv: n_old entries, newcum: n_jobs + 1 entries of scratch.  Two launches.
// Needs refresh_smem(n_gpus, n_jobs) <= kMaxSmemPerBlock - 1024 bytes of shared memory per CTA.
size_t refresh_smem(int32_t n_gpus, int32_t n_jobs);
cudaError_t launch_refresh_per_gpu(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_old, int32_t n_jobs,
                                   Tables t, const int4* fit, const int32_t* remap, int32_t* inv, int32_t* newcum,
                                   cudaStream_t s);
cudaError_t launch_best(const int32_t* pop, int64_t ld, int32_t n_jobs, const int32_t* best_index, Tables t,
                        int32_t capacity, double penalty, int repair, int32_t* work /*3*jpad*/,
                        int32_t* genome_out, int32_t* gpus_out, double* rate_out, BestOut* out,
                        const int32_t* rowmap /* nullptr: row best_index[0] of pop */, cudaStream_t s);
cudaError_t launch_remap(const int32_t* src, int64_t ld_src, int32_t* dst, int64_t ld_dst, int32_t n,
                         int32_t n_jobs_new, const int32_t* remap, const int32_t* kmin_new,
                         const int32_t* range_new, cudaStream_t s);
// remap and score in one pass (tables of the new job set; needs remap_score_smem(t) <= kMaxSmemPerBlock and
// GPU counts that fit 16 bits)
size_t remap_score_smem(Tables t);
cudaError_t launch_remap_score(const int32_t* src, int64_t ld_src, int32_t* dst, int64_t ld_dst, int32_t n,
                               int32_t n_jobs_new, const int32_t* remap, Tables t, int32_t capacity, double penalty,
                               double* F, int32_t* G, cudaStream_t s);
cudaError_t launch_copy_rows(const int32_t* src, int64_t ld_src, int32_t* dst, int64_t ld_dst, int32_t n,
                             int32_t n_jobs, int zero_pad, cudaStream_t s);
cudaError_t launch_export_tables(Tables t, int32_t n_jobs, double* X_out, int32_t* G_out, cudaStream_t s);

}  // namespace ones
