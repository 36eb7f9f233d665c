// C ABI of the evolutionary batch-size search: argument checks, workspace layout, launch order.
// All arithmetic of the method runs in the kernels of ones_kernels.cu.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "ones.h"
#include "ones_internal.h"

using namespace ones;

namespace {

constexpr size_t kAlign = 256;
constexpr int32_t kPlanesMax = ONES_MAX_EXPONENT + 2;  // exponents 0..15 and the waiting plane
constexpr int32_t kJobsLimit = 1 << 20;
constexpr int32_t kPopLimit = 1 << 28;

inline size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int32_t ld_of(int32_t n_jobs) { return (n_jobs + 3) & ~3; }
inline int32_t jpad_of(int32_t n_jobs) { return (n_jobs + 127) & ~127; }

struct Layout {
    size_t pop0, pop1, P0, P1, F, F1, G, G1, trunc, rowmap0, rowmap1, slot_kmin, slot_range, fit, refresh, parents, elites, elites1, best_idx, X, Gt, kmin, range, jobs_in, top, work, out_pack, exp_X, exp_G,
        status, total;
};

Layout make_layout(int32_t jmax, int32_t pop, bool trunc = false, int32_t gpus = 0 /* > 0: per-GPU genome */,
                   bool packed = false /* the population also as one byte per gene */) {
    Layout L;
    size_t at = 0;
    auto take = [&](size_t bytes) {
        size_t here = at;
        at = up(at + bytes, kAlign);
        return here;
    };
    const size_t ldm = (size_t)ld_of(gpus > 0 ? gpus : jmax), jp = (size_t)jpad_of(jmax);
    const size_t sp = (size_t)jpad_of(gpus > 0 ? gpus : 1);  // slot limits of the per-GPU genome
    // the truncation scheme keeps a pool of 4 * pop rows (originals, crossover children, mutants)
    const size_t rows = trunc ? 4 * (size_t)pop : (size_t)pop;
    const size_t pairs = trunc ? 3 * (size_t)pop : ((size_t)pop + 1) / 2;  // 2K parents + K mutant sources
    L.pop0 = take(rows * ldm * 4);
    L.pop1 = take(rows * ldm * 4);
    const size_t p8 = packed ? rows * (((size_t)jmax + 511) / 512 * 512) : 16;
    L.P0 = take(p8);
    L.P1 = take(p8);
    L.F = take(rows * 8);
    L.F1 = take(rows * 8);
    L.G = take(rows * 4);
    L.G1 = take(rows * 4);
    L.trunc = take(trunc ? trunc_scratch_bytes(pop) : 16);
    L.rowmap0 = take(trunc ? rows * 4 : 16);  // pool used in place: logical row -> pool row, two maps in turn
    L.rowmap1 = take(trunc ? rows * 4 : 16);
    L.slot_kmin = take(sp * 4);
    L.slot_range = take(sp * 4);
    L.fit = take(gpus > 0 ? jp * 16 : 16);  // per-GPU genome: the jobs' limits in the tables' job order
    L.refresh = take(gpus > 0 ? (2 * (size_t)jmax + 2) * 4 : 16);  // per-GPU genome: old -> new ids, new jobs' needs
    L.parents = take(pairs * 2 * 4);
    L.elites = take((size_t)ONES_MAX_ELITES * 4);
    L.elites1 = take((size_t)ONES_MAX_ELITES * 4);
    L.best_idx = take(16);
    L.X = take((size_t)kPlanesMax * jp * 8);
    L.Gt = take((size_t)kPlanesMax * jp * 4);
    L.kmin = take(jp * 4);
    L.range = take(jp * 4);
    // job rows, then the remap entries of an update, then (only for job tables with GPU counts that are not powers
    // of two) log2 of the GPU count per exponent and job
    L.jobs_in = take((size_t)jmax * (sizeof(ones_job) + 8) + (size_t)(kPlanesMax - 1) * jmax * 8);
    {
        const size_t a = top_scratch_bytes(pop, ONES_MAX_ELITES), b = generation_scratch_bytes(ONES_MAX_ELITES);
        L.top = take(a > b ? a : b);
    }
    L.work = take(3 * jp * 4);
    L.out_pack = take(64 + (size_t)jmax * 16);  // BestOut, then rate, genome, gpus of the returned schedule
    L.exp_X = take((size_t)(kPlanesMax - 1) * jmax * 8);
    L.exp_G = take((size_t)(kPlanesMax - 1) * jmax * 4);
    L.status = take(16);
    L.total = at;
    return L;
}

struct Prof {
    bool on = false;
    int every = 1;        // bracket every n-th generation
    bool sample = true;   // this generation is bracketed
    std::vector<cudaEvent_t> ev;
    std::vector<int> stage;  // stage of event pair i
    size_t used = 0;         // events recorded since the last flush
    double ms[3] = {0, 0, 0};
    uint64_t count[3] = {0, 0, 0};
};

}  // namespace

struct ones_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int32_t J = 0, Jmax = 0, N = 0, cap = 0, pairs = 0;
    int64_t ld = 0;
    ones_params prm{};
    uint32_t thr16 = 0;
    char* ws = nullptr;
    Layout L{};
    int cur = 0;            // population buffer in force
    int fcur = 0;           // score buffer in force
    int gcur = 0;           // GPU-count buffer in force (only the truncation scheme alternates it)
    bool trunc = false;     // ONES_FLAG_TRUNCATION
    bool mapped = false;    // truncation scheme: the pool is in use in place, logical row r lives in pool row rowmap(mcur)[r]
    int mcur = 0;           // row map in force (if mapped)
    bool per_gpu = false;   // ONES_FLAG_PER_GPU: one gene per GPU (a job id) instead of one per job
    bool narrow = false;    // per-GPU genome: capacity * max_per_gpu < 2^31 for every job (32-bit exponent search)
    bool packed = false;    // ONES_FLAG_PACKED: the population lives as packed rows, the int32 buffers are scratch
    int pcur = 0;           // packed buffer in force
    int64_t ld8 = 0;        // stride of the packed rows
    bool int_valid = false; // packed handle: pop(cur) holds the unpacked population
    bool flag_pending = false;  // the device-side job-table flag of the last ones_update_jobs has not been read yet
    bool in_limits = false;     // every gene of the population is known to lie in its job's [kmin, kmax]
    int32_t W = 0;          // genes per candidate
    Tables tabS{};          // as tab, with the limits of a slot (any job id) for the shared operators
    int ecur = 0;           // elites buffer holding the elites of the population in force (if elites_valid)
    int elast = 0;          // elites buffer used by the last generation
    bool elites_valid = false;
    bool f_valid = false;
    uint64_t gen = 0;
    Tables tab{};
    bool fused = false;  // children are scored inside the evolve kernel
    ClusterShape cshape{0, 0, 0, 0, 0};  // one-cluster, one-launch path for small populations
    std::vector<ones_job> h_jobs;  // the job table the device tables were built from
    uint64_t launches = 0;
    int last_cuda = 0;
    Prof prof;
    unsigned char* staging = nullptr;  // small pinned host buffer: uploads and downloads go through it in one copy
    cudaEvent_t staging_read = nullptr;  // recorded after an upload from the staging buffer: the host waits for it
                                         // before it writes there again
    size_t staging_bytes = 0;

    int32_t* pop(int which) { return reinterpret_cast<int32_t*>(ws + (which ? L.pop1 : L.pop0)); }
    uint8_t* P(int which) { return reinterpret_cast<uint8_t*>(ws + (which ? L.P1 : L.P0)); }
    double* Fbuf(int which) { return reinterpret_cast<double*>(ws + (which ? L.F1 : L.F)); }
    double* F() { return Fbuf(fcur); }
    int32_t* Gbuf(int which) { return reinterpret_cast<int32_t*>(ws + (which ? L.G1 : L.G)); }
    int32_t* G() { return Gbuf(gcur); }
    int32_t* parents() { return reinterpret_cast<int32_t*>(ws + L.parents); }
    int32_t* rowmap(int which) { return reinterpret_cast<int32_t*>(ws + (which ? L.rowmap1 : L.rowmap0)); }
    int32_t* elites(int which) { return reinterpret_cast<int32_t*>(ws + (which ? L.elites1 : L.elites)); }
    int32_t* best_idx() { return reinterpret_cast<int32_t*>(ws + L.best_idx); }
    ones_job* jobs() { return reinterpret_cast<ones_job*>(ws + L.jobs_in); }
    int4* fit() { return reinterpret_cast<int4*>(ws + L.fit); }
    int32_t* refresh_inv() { return reinterpret_cast<int32_t*>(ws + L.refresh); }
    int32_t* refresh_cum() { return refresh_inv() + Jmax; }
    int32_t* remap(int32_t n_jobs) { return reinterpret_cast<int32_t*>(ws + L.jobs_in + (size_t)n_jobs * sizeof(ones_job)); }
    int32_t* status() { return reinterpret_cast<int32_t*>(ws + L.status); }
};

namespace {

int cuda_fail(ones_ctx* c, cudaError_t e);

int ensure_staging(ones_ctx* c, size_t bytes) {
    if (bytes <= c->staging_bytes) return ONES_OK;
    if (c->staging_read) cudaEventSynchronize(c->staging_read);  // no upload may still be reading the old buffer
    if (c->staging) cudaFreeHost(c->staging);
    c->staging = nullptr;
    c->staging_bytes = 0;
    const size_t want = bytes < 4096 ? 4096 : 2 * bytes;
    cudaError_t e = cudaMallocHost(reinterpret_cast<void**>(&c->staging), want);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->staging_bytes = want;
    return ONES_OK;
}

int cuda_fail(ones_ctx* c, cudaError_t e) {
    if (c) c->last_cuda = (int)e;
    return ONES_ERR_CUDA;
}

#define CU(c, call)                                     \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) return cuda_fail(c, e_); \
    } while (0)

int check_jobs(const ones_job* jobs, int32_t n) {
    if (!jobs) return ONES_ERR_NULL;
    if (n <= 0 || n > kJobsLimit) return ONES_ERR_BAD_JOB;
    for (int32_t j = 0; j < n; ++j) {
        const ones_job& q = jobs[j];
        if (q.b0 <= 0 || q.max_per_gpu <= 0) return ONES_ERR_BAD_JOB;
        if (q.kmin < 0 || q.kmin > q.kmax || q.kmax > ONES_MAX_EXPONENT) return ONES_ERR_BAD_JOB;
        if (((int64_t)q.b0 << q.kmax) >= ((int64_t)1 << 31)) return ONES_ERR_BAD_JOB;
        if (!(q.a >= 0.0) || !(q.c >= 0.0) || !(q.d >= 0.0)) return ONES_ERR_BAD_JOB;
        if (!isfinite(q.a) || !isfinite(q.c) || !isfinite(q.d) || !isfinite(q.weight)) return ONES_ERR_BAD_JOB;
    }
    return ONES_OK;
}

// Argument check: does every exponent of every job give a positive, finite throughput?  The tables themselves
// are built on the device (which sets a flag under the same condition); this check only lets ones_update_jobs
// reject a bad job table without waiting for the device.  Rows with ordinary magnitudes are accepted at
// once (seconds per iteration >= a > 0, everything far from the ends of the double range); the rest are
// evaluated exponent by exponent.
int check_throughput(const ones_job* jobs, int32_t n) {
    for (int32_t j = 0; j < n; ++j) {
        const ones_job& q = jobs[j];
        if (q.a > 1e-290 && q.a < 1e290 && q.c < 1e290 && q.d < 1e290) continue;
        for (int32_t k = 0; k <= q.kmax; ++k) {
            const int64_t b = (int64_t)q.b0 << k, m = q.max_per_gpu, g = (b + m - 1) / m;
            const double sec = (q.a + q.c * ((double)b / (double)g)) + q.d * log2((double)g);
            const double X = (double)b / sec;
            if (!(X > 0.0) || X > 1.7976931348623157e308) return ONES_ERR_BAD_JOB;
        }
    }
    return ONES_OK;
}

int check_params(const ones_params& p, int32_t pop) {
    if (p.elitism < 0 || p.elitism > ONES_MAX_ELITES || p.tournament < 1) return ONES_ERR_BAD_PARAM;
    if (pop < p.elitism + 1) return ONES_ERR_BAD_PARAM;
    if (!(p.p_mut >= 0.0 && p.p_mut <= 1.0)) return ONES_ERR_BAD_PARAM;
    if (p.p_mut > 0.0 && lround(p.p_mut * 65536.0) == 0) return ONES_ERR_BAD_PARAM;  // below the 16-bit resolution
    if (!isfinite(p.penalty)) return ONES_ERR_BAD_PARAM;
    return ONES_OK;
}

uint32_t threshold16(double p) {
    long t = lround(p * 65536.0);
    if (t < 0) t = 0;
    if (t > 65536) t = 65536;
    return (uint32_t)t;
}

void set_tables(ones_ctx* c, const ones_job* jobs, int32_t n_jobs) {
    int32_t kmax = 0;
    for (int32_t j = 0; j < n_jobs; ++j) kmax = jobs[j].kmax > kmax ? jobs[j].kmax : kmax;
    c->tab.X = reinterpret_cast<double*>(c->ws + c->L.X);
    c->tab.G = reinterpret_cast<int32_t*>(c->ws + c->L.Gt);
    c->tab.kmin = reinterpret_cast<int32_t*>(c->ws + c->L.kmin);
    c->tab.range = reinterpret_cast<int32_t*>(c->ws + c->L.range);
    c->tab.jpad = jpad_of(n_jobs);
    c->tab.k1 = kmax + 1;
    // the fused evolve+score kernel keeps GPU counts as 16-bit values in shared memory
    bool narrow = true;
    for (int32_t j = 0; j < n_jobs; ++j) {
        const int64_t b = (int64_t)jobs[j].b0 << jobs[j].kmax, m = jobs[j].max_per_gpu;
        if ((b + m - 1) / m > 65535) narrow = false;
    }
    c->fused = narrow && !(c->prm.flags & ONES_FLAG_UNFUSED) && evolve_score_smem(c->tab) <= (size_t)kMaxSmemPerBlock;
    c->tabS = c->tab;
    if (c->per_gpu) {
        c->narrow = true;
        for (int32_t j = 0; j < n_jobs; ++j)
            if ((int64_t)c->W * jobs[j].max_per_gpu >= ((int64_t)1 << 31)) c->narrow = false;
        c->tabS.kmin = reinterpret_cast<int32_t*>(c->ws + c->L.slot_kmin);
        c->tabS.range = reinterpret_cast<int32_t*>(c->ws + c->L.slot_range);
        c->fused = false;  // scoring a per-GPU candidate needs its job counts: separate kernel
    }
    c->cshape = ClusterShape{0, 0, 0, 0, 0};
    if (c->fused && !c->trunc && !c->packed && !(c->prm.flags & ONES_FLAG_NO_CLUSTER))
        c->cshape = cluster_shape(c->tab, ld_of(n_jobs), c->N, c->prm.elitism, c->pairs);
}

// ---- per-stage timing with CUDA events on the handle's stream ----
int prof_flush(ones_ctx* c) {
    Prof& p = c->prof;
    if (p.used == 0) return ONES_OK;
    CU(c, cudaStreamSynchronize(c->stream));
    for (size_t i = 0; i + 1 < p.used; i += 2) {
        float ms = 0.f;
        CU(c, cudaEventElapsedTime(&ms, p.ev[i], p.ev[i + 1]));
        const int s = p.stage[i / 2];
        p.ms[s] += (double)ms;
        p.count[s] += 1;
    }
    p.used = 0;
    return ONES_OK;
}

int prof_begin(ones_ctx* c, int stage) {
    Prof& p = c->prof;
    if (!p.on || !p.sample) return ONES_OK;
    if (p.used + 2 > p.ev.size()) {
        int rc = prof_flush(c);
        if (rc) return rc;
    }
    p.stage[p.used / 2] = stage;
    CU(c, cudaEventRecord(p.ev[p.used], c->stream));
    return ONES_OK;
}

int prof_end(ones_ctx* c) {
    Prof& p = c->prof;
    if (!p.on || !p.sample) return ONES_OK;
    CU(c, cudaEventRecord(p.ev[p.used + 1], c->stream));
    p.used += 2;
    return ONES_OK;
}

// Truncation scheme with the pool used in place: bring the K candidates, in order, to rows 0..K-1 of the other
// pool and go on there with logical row = pool row.  Everything that reads or replaces the population as rows
// calls this first; generations that follow one another never do.
int compact_pool(ones_ctx* c) {
    if (!c->mapped) return ONES_OK;
    CU(c, launch_trunc_compact(c->pop(c->cur), c->pop(c->cur ^ 1), c->ld, c->N, c->rowmap(c->mcur), c->stream));
    c->launches += 1;
    c->cur ^= 1;
    c->mapped = false;
    return ONES_OK;
}

int run_fitness(ones_ctx* c) {
    int rc = compact_pool(c);
    if (rc) return rc;
    rc = prof_begin(c, 0);
    if (rc) return rc;
    if (c->per_gpu)
        CU(c, launch_fitness_per_gpu(c->pop(c->cur), c->ld, c->N, c->W, c->J, c->tab, c->fit(), c->narrow, c->F(), c->G(), c->stream));
    else if (c->packed)
        CU(c, launch_fitness_packed(c->P(c->pcur), c->ld8, c->N, c->tab, c->cap, c->prm.penalty, c->F(), c->G(), c->stream));
    else
        CU(c, launch_fitness(c->pop(c->cur), c->ld, c->N, c->J, c->tab, c->cap, c->prm.penalty, c->F(), c->G(),
                             c->stream));
    c->launches += 1;
    c->f_valid = true;
    c->elites_valid = false;
    return prof_end(c);
}

// Packed handle: the int32 buffer in force -> packed rows, and back.
int pack_from_int(ones_ctx* c) {
    c->ld8 = (int64_t)(((size_t)c->J + 511) / 512 * 512);
    CU(c, launch_pack_rows(c->pop(c->cur), c->ld, c->N, c->J, c->P(c->pcur), c->ld8, c->stream));
    c->launches += 1;
    return ONES_OK;
}

int unpack_to_int(ones_ctx* c) {
    if (c->int_valid) return ONES_OK;
    CU(c, launch_unpack_rows(c->P(c->pcur), c->ld8, c->N, c->J, c->pop(c->cur), c->ld, nullptr, c->stream));
    c->launches += 1;
    c->int_valid = true;
    return ONES_OK;
}

int rebuild_tables(ones_ctx* c, const ones_job* h_jobs, int32_t n_jobs, const int32_t* h_remap = nullptr,
                   bool wait_for_flag = true) {
    // log2 of a GPU count that is not a power of two comes from the host's math library and is uploaded with the
    // job rows: the device routine may differ from it in the last bit, and a last bit decides tournaments
    int32_t kmax = 0;
    bool all_pow2 = true;
    for (int32_t j = 0; j < n_jobs; ++j) {
        kmax = h_jobs[j].kmax > kmax ? h_jobs[j].kmax : kmax;
        const int64_t b0 = h_jobs[j].b0, m = h_jobs[j].max_per_gpu;
        if ((b0 & (b0 - 1)) == 0 && (m & (m - 1)) == 0) continue;  // powers of two: so is every GPU count (no division)
        for (int32_t k = 0; k <= h_jobs[j].kmax && all_pow2; ++k) {
            const int64_t g = ((b0 << k) + m - 1) / m;
            all_pow2 = (g & (g - 1)) == 0;
        }
    }
    const size_t jb = sizeof(ones_job) * (size_t)n_jobs, rb = (size_t)n_jobs * 8;  // remap entries padded to 8 bytes each
    const size_t lb = all_pow2 ? 0 : (size_t)(kmax + 1) * n_jobs * 8;
    int rc = ensure_staging(c, jb + rb + lb);
    if (rc) return rc;
    if (!c->staging_read) CU(c, cudaEventCreateWithFlags(&c->staging_read, cudaEventDisableTiming));
    CU(c, cudaEventSynchronize(c->staging_read));  // the last upload has left the staging buffer
    memcpy(c->staging, h_jobs, jb);
    if (h_remap) memcpy(c->staging + jb, h_remap, (size_t)n_jobs * 4);
    if (lb) {
        double* lg = reinterpret_cast<double*>(c->staging + jb + rb);
        for (int32_t k = 0; k <= kmax; ++k)
            for (int32_t j = 0; j < n_jobs; ++j) {
                const int64_t b = (int64_t)h_jobs[j].b0 << (k <= h_jobs[j].kmax ? k : 0), m = h_jobs[j].max_per_gpu;
                lg[(size_t)k * n_jobs + j] = log2((double)((b + m - 1) / m));
            }
    }
    CU(c, cudaMemsetAsync(c->status(), 0, 16, c->stream));
    CU(c, cudaMemcpyAsync(c->jobs(), c->staging, (h_remap || lb) ? jb + rb + lb : jb, cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaEventRecord(c->staging_read, c->stream));
    const double* d_lg = lb ? reinterpret_cast<const double*>(reinterpret_cast<const unsigned char*>(c->jobs()) + jb + rb) : nullptr;
    set_tables(c, h_jobs, n_jobs);
    CU(c, launch_build_tables(c->jobs(), n_jobs, c->prm.flags, c->tab, d_lg, c->status(), c->stream));
    c->launches += 1;
    if (wait_for_flag) {
        int32_t bad = 0;
        CU(c, cudaMemcpyAsync(&bad, c->status(), 4, cudaMemcpyDeviceToHost, c->stream));
        CU(c, cudaStreamSynchronize(c->stream));
        if (bad) return ONES_ERR_BAD_JOB;  // some job has a non-positive or non-finite throughput
        c->flag_pending = false;
    } else {
        c->flag_pending = true;  // read at the next call that synchronises (the host check has passed already)
    }
    try {
        c->h_jobs.assign(h_jobs, h_jobs + n_jobs);
    } catch (...) {
        return ONES_ERR_NOMEM;
    }
    return ONES_OK;
}

// The job-table flag that ones_update_jobs left unread: fetched by the calls that synchronise anyway.
int enqueue_flag_read(ones_ctx* c) {
    if (!c->flag_pending) return ONES_OK;
    int rc = ensure_staging(c, 64);
    if (rc) return rc;
    CU(c, cudaMemcpyAsync(c->staging + c->staging_bytes - 16, c->status(), 4, cudaMemcpyDeviceToHost, c->stream));
    return ONES_OK;
}

int flag_after_sync(ones_ctx* c) {
    if (!c->flag_pending) return ONES_OK;
    c->flag_pending = false;
    int32_t bad = 0;
    memcpy(&bad, c->staging + c->staging_bytes - 16, 4);
    return bad ? ONES_ERR_BAD_JOB : ONES_OK;
}

// Work of a handle always goes to the device it was created on, whatever device the caller has current.
struct DeviceScope {
    int prev = -1;
    bool changed = false;
    explicit DeviceScope(const ones_ctx* c) {
        if (c && cudaGetDevice(&prev) == cudaSuccess && prev != c->device) changed = cudaSetDevice(c->device) == cudaSuccess;
    }
    ~DeviceScope() {
        if (changed) cudaSetDevice(prev);
    }
};

void free_ctx(ones_ctx* c) {
    if (!c) return;
    for (cudaEvent_t ev : c->prof.ev) cudaEventDestroy(ev);
    if (c->staging) cudaFreeHost(c->staging);
    if (c->staging_read) cudaEventDestroy(c->staging_read);
    delete c;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

size_t ones_workspace_bytes(int32_t n_jobs_max, int32_t pop) { return ones_workspace_bytes_flags(n_jobs_max, pop, 0u); }

size_t ones_workspace_bytes_flags(int32_t n_jobs_max, int32_t pop, uint32_t flags) {
    if (n_jobs_max <= 0 || n_jobs_max > kJobsLimit || pop <= 0 || pop > kPopLimit) return 0;
    const bool trunc = (flags & ONES_FLAG_TRUNCATION) != 0;
    if (trunc && pop > kPopLimit / 4) return 0;
    if (flags & ONES_FLAG_PER_GPU) return 0;  // needs the cluster size: ones_workspace_bytes_per_gpu
    const bool packed = (flags & ONES_FLAG_PACKED) != 0;
    if (packed && trunc) return 0;
    return make_layout(n_jobs_max, pop, trunc, 0, packed).total;
}

size_t ones_workspace_bytes_per_gpu(int32_t n_jobs, int32_t pop, int32_t capacity) {
    if (n_jobs <= 0 || n_jobs > kJobsLimit || pop <= 0 || pop > kPopLimit || capacity <= 0 || capacity > kJobsLimit) return 0;
    return make_layout(n_jobs, pop, false, capacity).total;
}

int ones_create(ones_ctx** out, const ones_job* jobs, int32_t n_jobs, int32_t capacity, int32_t pop,
                const ones_params* prm, void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!out) return ONES_ERR_NULL;
    *out = nullptr;
    if (!jobs || !d_workspace) return ONES_ERR_NULL;
    int rc = check_jobs(jobs, n_jobs);
    if (rc) return rc;
    ones_params p = {2, 4, 0.1, 1e3, 0};
    if (prm) p = *prm;
    if (capacity <= 0 || pop <= 0 || pop > kPopLimit) return ONES_ERR_BAD_PARAM;
    rc = check_params(p, pop);
    if (rc) return rc;
    if ((reinterpret_cast<uintptr_t>(d_workspace) & (kAlign - 1)) != 0) return ONES_ERR_ALIGN;
    const bool trunc = (p.flags & ONES_FLAG_TRUNCATION) != 0;
    const bool per_gpu = (p.flags & ONES_FLAG_PER_GPU) != 0;
    const bool packed = (p.flags & ONES_FLAG_PACKED) != 0;
    if (trunc && (pop > kPopLimit / 4 || per_gpu)) return ONES_ERR_BAD_PARAM;
    if (packed && (trunc || per_gpu)) return ONES_ERR_BAD_PARAM;
    if (per_gpu && capacity > kJobsLimit) return ONES_ERR_BAD_PARAM;
    const int32_t gpus = per_gpu ? capacity : 0;
    if (workspace_bytes < make_layout(n_jobs, pop, trunc, gpus, packed).total) return ONES_ERR_WORKSPACE;
    // the largest job count this workspace can hold
    int32_t lo = n_jobs, hi = kJobsLimit;
    while (lo < hi) {
        const int32_t mid = lo + (hi - lo + 1) / 2;
        if (make_layout(mid, pop, trunc, gpus, packed).total <= workspace_bytes) lo = mid;
        else hi = mid - 1;
    }
    ones_ctx* c = new (std::nothrow) ones_ctx();
    if (!c) return ONES_ERR_NOMEM;
    c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    c->J = n_jobs;
    c->Jmax = lo;
    c->per_gpu = per_gpu;
    c->packed = packed;
    c->W = per_gpu ? capacity : n_jobs;
    c->N = pop;
    c->cap = capacity;
    c->prm = p;
    c->thr16 = threshold16(p.p_mut);
    c->trunc = trunc;
    c->pairs = trunc ? pop : (pop - p.elitism + 1) / 2;
    c->ld = ld_of(c->W);
    c->ws = reinterpret_cast<char*>(d_workspace);
    c->L = make_layout(c->Jmax, pop, trunc, gpus, packed);
    cudaError_t e = cudaGetDevice(&c->device);
    if (e != cudaSuccess) {
        free_ctx(c);
        return ONES_ERR_CUDA;
    }
    if (trunc) {  // the radix search keeps its histogram and counters zero between launches
        e = cudaMemsetAsync(c->ws + c->L.trunc, 0, trunc_scratch_bytes(pop), c->stream);
        if (e != cudaSuccess) {
            free_ctx(c);
            return ONES_ERR_CUDA;
        }
    }
    rc = rebuild_tables(c, jobs, n_jobs);
    if (rc == ONES_OK) {
        if (per_gpu) {  // an idle cluster: every slot -1; slot limits for the shared operators
            e = cudaMemsetAsync(c->pop(0), 0xFF, (size_t)c->N * c->ld * 4, c->stream);
            if (e == cudaSuccess)
                e = launch_fill_slot_limits(c->tabS.kmin, c->tabS.range, jpad_of(c->W), c->W, c->J, c->jobs(), c->fit(),
                                            c->tab.jpad, c->stream);
        } else {
            e = launch_fill_min(c->pop(0), c->ld, c->N, c->J, c->tab, c->stream);
        }
        c->launches += 1;
        if (e != cudaSuccess) rc = cuda_fail(c, e);
    }
    c->cur = 0;
    c->in_limits = !per_gpu;
    if (rc == ONES_OK && packed) {
        // the one-byte rows need the tables in shared memory (no separate scoring pass exists for them)
        rc = c->fused ? pack_from_int(c) : ONES_ERR_BAD_PARAM;
        c->int_valid = true;
    }
    if (rc != ONES_OK) {
        free_ctx(c);
        return rc;
    }
    c->f_valid = false;
    c->elites_valid = false;
    *out = c;
    return ONES_OK;
}

int ones_destroy(ones_ctx* c) {
    if (!c) return ONES_OK;
    free_ctx(c);
    return ONES_OK;
}

int ones_randomize(ones_ctx* c, uint64_t seed) {
    DeviceScope scope(c);
    if (!c) return ONES_ERR_NULL;
    c->mapped = false;  // every candidate is replaced
    CU(c, launch_randomize(c->pop(c->cur), c->ld, c->N, c->W, c->tabS, make_round_keys(seed), c->stream));
    c->launches += 1;
    c->f_valid = false;
    c->elites_valid = false;
    c->in_limits = !c->per_gpu;
    if (c->packed) {
        c->int_valid = true;
        return pack_from_int(c);
    }
    return ONES_OK;
}

int ones_set_population(ones_ctx* c, const int32_t* genomes, int64_t ld, int on_device) {
    DeviceScope scope(c);
    if (!c || !genomes) return ONES_ERR_NULL;
    if (ld < c->W) return ONES_ERR_BAD_PARAM;
    c->mapped = false;  // every candidate is replaced
    if (on_device) {
        CU(c, launch_copy_rows(genomes, ld, c->pop(c->cur), c->ld, c->N, c->W, 1, c->stream));
        c->launches += 1;
    } else {
        if (c->ld != c->W) CU(c, cudaMemsetAsync(c->pop(c->cur), 0, (size_t)c->N * c->ld * 4, c->stream));
        CU(c, cudaMemcpy2DAsync(c->pop(c->cur), (size_t)c->ld * 4, genomes, (size_t)ld * 4, (size_t)c->W * 4,
                                (size_t)c->N, cudaMemcpyHostToDevice, c->stream));
        CU(c, cudaStreamSynchronize(c->stream));
    }
    c->f_valid = false;
    c->elites_valid = false;
    c->in_limits = false;
    if (c->packed) {  // genes outside [0, 254] become "waits": what is read back comes from the packed rows
        c->int_valid = false;
        return pack_from_int(c);
    }
    return ONES_OK;
}

int ones_get_population(ones_ctx* c, int32_t* genomes, int64_t ld, int on_device) {
    DeviceScope scope(c);
    if (!c || !genomes) return ONES_ERR_NULL;
    if (ld < c->W) return ONES_ERR_BAD_PARAM;
    if (c->packed) {
        int rc = unpack_to_int(c);
        if (rc) return rc;
    }
    {
        int rc = compact_pool(c);
        if (rc) return rc;
    }
    if (on_device) {
        CU(c, launch_copy_rows(c->pop(c->cur), c->ld, genomes, ld, c->N, c->W, 0, c->stream));
        c->launches += 1;
    } else {
        CU(c, cudaMemcpy2DAsync(genomes, (size_t)ld * 4, c->pop(c->cur), (size_t)c->ld * 4, (size_t)c->W * 4,
                                (size_t)c->N, cudaMemcpyDeviceToHost, c->stream));
        int rc = enqueue_flag_read(c);
        if (rc) return rc;
        CU(c, cudaStreamSynchronize(c->stream));
        return flag_after_sync(c);
    }
    return ONES_OK;
}

int ones_evaluate(ones_ctx* c, const int32_t* d_genomes, int64_t ld, int32_t n, double* d_fitness, int32_t* d_gpus) {
    DeviceScope scope(c);
    if (!c || !d_fitness) return ONES_ERR_NULL;
    if (!d_genomes) {
        if (!c->f_valid) {
            int rc = run_fitness(c);
            if (rc) return rc;
        }
        CU(c, cudaMemcpyAsync(d_fitness, c->F(), (size_t)c->N * 8, cudaMemcpyDeviceToDevice, c->stream));
        if (d_gpus) CU(c, cudaMemcpyAsync(d_gpus, c->G(), (size_t)c->N * 4, cudaMemcpyDeviceToDevice, c->stream));
        return ONES_OK;
    }
    if (n < 0 || ld < c->W) return ONES_ERR_BAD_PARAM;
    if ((ld & 3) != 0 || !aligned16(d_genomes)) return ONES_ERR_ALIGN;
    if (n == 0) return ONES_OK;
    int rc = prof_begin(c, 0);
    if (rc) return rc;
    if (c->per_gpu)
        CU(c, launch_fitness_per_gpu(d_genomes, ld, n, c->W, c->J, c->tab, c->fit(), c->narrow, d_fitness, d_gpus, c->stream));
    else
        CU(c, launch_fitness(d_genomes, ld, n, c->J, c->tab, c->cap, c->prm.penalty, d_fitness, d_gpus, c->stream));
    c->launches += 1;
    return prof_end(c);
}

size_t ones_packed_row_bytes(int32_t n_jobs) {
    if (n_jobs <= 0 || n_jobs > kJobsLimit) return 0;
    return ((size_t)n_jobs + 511) / 512 * 512;
}

int ones_pack_population(ones_ctx* c, const int32_t* d_genomes, int64_t ld, int32_t n, uint8_t* d_packed, int64_t ld8) {
    DeviceScope scope(c);
    if (!c || !d_packed) return ONES_ERR_NULL;
    if (c->per_gpu) return ONES_ERR_BAD_PARAM;  // job ids do not fit a byte
    if (!d_genomes && c->packed) {  // the handle's own rows are packed already
        if (ld8 < c->ld8) return ONES_ERR_BAD_PARAM;
        if ((ld8 & 511) != 0 || !aligned16(d_packed)) return ONES_ERR_ALIGN;
        if (ld8 != c->ld8) CU(c, cudaMemsetAsync(d_packed, 0xFF, (size_t)c->N * ld8, c->stream));
        CU(c, cudaMemcpy2DAsync(d_packed, (size_t)ld8, c->P(c->pcur), (size_t)c->ld8, (size_t)c->ld8, (size_t)c->N,
                                cudaMemcpyDeviceToDevice, c->stream));
        return ONES_OK;
    }
    if (!d_genomes) {
        int rc = compact_pool(c);
        if (rc) return rc;
        d_genomes = c->pop(c->cur);
        ld = c->ld;
        n = c->N;
    }
    if (n < 0 || ld < c->J || ld8 < (int64_t)ones_packed_row_bytes(c->J)) return ONES_ERR_BAD_PARAM;
    if ((ld & 3) != 0 || (ld8 & 511) != 0 || !aligned16(d_genomes) || !aligned16(d_packed)) return ONES_ERR_ALIGN;
    if (n == 0) return ONES_OK;
    CU(c, launch_pack_rows(d_genomes, ld, n, c->J, d_packed, ld8, c->stream));
    c->launches += 1;
    return ONES_OK;
}

int ones_evaluate_packed(ones_ctx* c, const uint8_t* d_packed, int64_t ld8, int32_t n, double* d_fitness,
                         int32_t* d_gpus) {
    DeviceScope scope(c);
    if (!c || !d_packed || !d_fitness) return ONES_ERR_NULL;
    if (c->per_gpu) return ONES_ERR_BAD_PARAM;
    if (n < 0 || ld8 < (int64_t)ones_packed_row_bytes(c->J)) return ONES_ERR_BAD_PARAM;
    if ((ld8 & 511) != 0 || !aligned16(d_packed)) return ONES_ERR_ALIGN;
    if (n == 0) return ONES_OK;
    int rc = prof_begin(c, 0);
    if (rc) return rc;
    CU(c, launch_fitness_packed(d_packed, ld8, n, c->tab, c->cap, c->prm.penalty, d_fitness, d_gpus, c->stream));
    c->launches += 1;
    return prof_end(c);
}

int ones_evolve(ones_ctx* c, int32_t generations, uint64_t seed) {
    DeviceScope scope(c);
    if (!c) return ONES_ERR_NULL;
    if (generations < 0) return ONES_ERR_BAD_PARAM;
    if (generations == 0) return ONES_OK;
    int rc;
    c->prof.sample = true;
    if (!c->f_valid && (rc = run_fitness(c)) != ONES_OK) return rc;
    const RoundKeys keys = make_round_keys(seed);
    if (c->trunc) {
        // the paper's scheme: pool of 4K rows, best K survive (elitism and tournament size do not apply)
        // Fused handles use the pool in place: survivors keep their pool rows, a map of 4K entries says where each
        // logical row lives, and no candidate is copied between generations (compact_pool() orders them when
        // someone asks for the population).  Otherwise the survivors are gathered into the other pool.
        const bool in_place = c->fused && !(c->prm.flags & ONES_FLAG_NO_CLUSTER) && trunc_inplace_available(c->N);
        if (!in_place && (rc = compact_pool(c)) != ONES_OK) return rc;
        for (int32_t it = 0; it < generations; ++it) {
            c->prof.sample = it % c->prof.every == 0;
            const int64_t K = c->N;
            if ((rc = prof_begin(c, 2)) != ONES_OK) return rc;
            if (c->fused) {  // the 3K new rows are scored while they are written
                CU(c, launch_trunc_children_score(c->pop(c->cur), c->ld, c->N, c->parents(), c->tab, keys, c->gen,
                                                  c->thr16, c->cap, c->prm.penalty, c->Fbuf(c->fcur), c->Gbuf(c->gcur),
                                                  c->mapped ? c->rowmap(c->mcur) : nullptr, c->stream));
                if ((rc = prof_end(c)) != ONES_OK) return rc;
            } else {
                CU(c, launch_trunc_children(c->pop(c->cur), c->ld, c->N, c->parents(), c->tab, keys, c->gen, c->thr16,
                                            c->stream));
                if ((rc = prof_end(c)) != ONES_OK) return rc;
                if ((rc = prof_begin(c, 0)) != ONES_OK) return rc;
                CU(c, launch_fitness(c->pop(c->cur) + K * c->ld, c->ld, 3 * c->N, c->J, c->tab, c->cap, c->prm.penalty,
                                     c->Fbuf(c->fcur) + K, c->Gbuf(c->gcur) + K, c->stream));
                if ((rc = prof_end(c)) != ONES_OK) return rc;
                c->launches += 1;
            }
            if ((rc = prof_begin(c, 1)) != ONES_OK) return rc;
            int sel_launches = 0;
            if (in_place) {
                const int next = c->mapped ? c->mcur ^ 1 : 0;
                CU(c, launch_trunc_select_inplace(c->N, c->Fbuf(c->fcur), c->Gbuf(c->gcur), c->Fbuf(c->fcur ^ 1),
                                                  c->Gbuf(c->gcur ^ 1), c->mapped ? c->rowmap(c->mcur) : nullptr,
                                                  c->rowmap(next), c->stream));
                sel_launches = 1;
                c->mapped = true;
                c->mcur = next;
            } else {
                CU(c, launch_trunc_select(c->pop(c->cur), c->pop(c->cur ^ 1), c->ld, c->N, c->Fbuf(c->fcur),
                                          c->Gbuf(c->gcur), c->Fbuf(c->fcur ^ 1), c->Gbuf(c->gcur ^ 1),
                                          c->ws + c->L.trunc, c->stream, &sel_launches));
                c->cur ^= 1;
            }
            if ((rc = prof_end(c)) != ONES_OK) return rc;
            c->launches += (c->fused ? 1u : 2u) + (uint64_t)sel_launches;
            c->fcur ^= 1;
            c->gcur ^= 1;
            c->gen += 1;
        }
        c->prof.sample = true;
        c->elites_valid = false;
        return ONES_OK;
    }
    const int32_t E = c->prm.elitism;
    if (c->packed) {
        // parents read and children written as bytes: selection stage, then crossover + mutation + scoring
        unsigned int* pdone = reinterpret_cast<unsigned int*>(c->status() + 1);
        for (int32_t it = 0; it < generations; ++it) {
            c->prof.sample = it % c->prof.every == 0;
            if ((rc = prof_begin(c, 1)) != ONES_OK) return rc;
            CU(c, launch_select_stage(c->F(), c->N, c->prm.tournament, c->pairs, keys, c->gen, c->parents(), E,
                                      c->elites(0), c->ws + c->L.top, pdone, c->stream));
            if ((rc = prof_end(c)) != ONES_OK) return rc;
            if ((rc = prof_begin(c, 2)) != ONES_OK) return rc;
            CU(c, launch_evolve_score_packed(c->P(c->pcur), c->P(c->pcur ^ 1), c->ld8, c->N, c->J, E, c->pairs, c->parents(),
                                             c->elites(0), c->tab, keys, c->gen, c->thr16, c->cap, c->prm.penalty, c->F(),
                                             c->G(), pdone + 1, c->stream));
            if ((rc = prof_end(c)) != ONES_OK) return rc;
            c->launches += 2;
            c->pcur ^= 1;
            c->gen += 1;
        }
        c->elast = 0;
        c->elites_valid = false;
        c->int_valid = false;
        c->prof.sample = true;
        return ONES_OK;
    }
    if (c->cshape.cluster > 0) {
        // small population: every generation of this call inside one cluster launch
        if ((rc = prof_begin(c, 2)) != ONES_OK) return rc;
        CU(c, launch_evolve_cluster(c->cshape, c->pop(c->cur), c->ld, c->N, c->J, E, c->pairs, c->prm.tournament, c->F(),
                                    c->G(), c->parents(), c->elites(0), c->tab, keys, c->gen, generations, c->thr16,
                                    c->cap, c->prm.penalty, c->stream));
        c->launches += 1;
        if ((rc = prof_end(c)) != ONES_OK) return rc;
        c->gen += (uint64_t)generations;
        c->elast = 0;
        c->elites_valid = false;
        return ONES_OK;
    }
    unsigned int* done = reinterpret_cast<unsigned int*>(c->status() + 1);
    const GenerationShape shape = c->fused ? generation_shape(c->tab, c->pairs, E) : GenerationShape{0, 0, 0, 0};
    if (shape.blocks > 0) {
        // one launch per generation; each launch also leaves the elites of the population it wrote
        if (E > 0 && !c->elites_valid) {
            if ((rc = prof_begin(c, 1)) != ONES_OK) return rc;
            int nl = 0;
            CU(c, launch_top(c->F(), c->N, E, c->elites(c->ecur), c->ws + c->L.top, c->stream, &nl));
            c->launches += (uint64_t)nl;
            if ((rc = prof_end(c)) != ONES_OK) return rc;
        }
        for (int32_t it = 0; it < generations; ++it) {
            c->prof.sample = it % c->prof.every == 0;
            if ((rc = prof_begin(c, 2)) != ONES_OK) return rc;
            CU(c, launch_generation(shape, c->pop(c->cur), c->pop(c->cur ^ 1), c->ld, c->N, c->J, E, c->pairs,
                                    c->prm.tournament, c->Fbuf(c->fcur), c->Fbuf(c->fcur ^ 1), c->G(), c->parents(),
                                    c->elites(c->ecur), c->elites(c->ecur ^ 1), c->tab, keys, c->gen, c->thr16, c->cap,
                                    c->prm.penalty, c->ws + c->L.top, done, c->stream));
            c->launches += 1;
            if ((rc = prof_end(c)) != ONES_OK) return rc;
            c->elast = c->ecur;
            c->cur ^= 1;
            c->fcur ^= 1;
            c->ecur ^= 1;
            c->elites_valid = true;
            c->gen += 1;
        }
        c->prof.sample = true;
        return ONES_OK;
    }
    for (int32_t it = 0; it < generations; ++it) {
        c->prof.sample = it % c->prof.every == 0;
        if ((rc = prof_begin(c, 1)) != ONES_OK) return rc;
        CU(c, launch_select_stage(c->F(), c->N, c->prm.tournament, c->pairs, keys, c->gen, c->parents(), E,
                                  c->elites(0), c->ws + c->L.top, done, c->stream));
        c->launches += 1;
        c->elast = 0;
        c->elites_valid = false;
        if ((rc = prof_end(c)) != ONES_OK) return rc;

        if ((rc = prof_begin(c, 2)) != ONES_OK) return rc;
        if (c->fused) {
            CU(c, launch_evolve_score(c->pop(c->cur), c->pop(c->cur ^ 1), c->ld, c->N, c->J, E, c->pairs,
                                      c->parents(), c->elites(0), c->tab, keys, c->gen, c->thr16, c->cap,
                                      c->prm.penalty, c->F(), c->G(), done + 1, c->in_limits, c->stream));
        } else {
            CU(c, launch_evolve(c->pop(c->cur), c->pop(c->cur ^ 1), c->ld, c->N, c->W, E, c->pairs, c->parents(),
                                c->elites(0), c->tabS, keys, c->gen, c->thr16, c->stream));
        }
        c->launches += 1;
        if ((rc = prof_end(c)) != ONES_OK) return rc;

        c->cur ^= 1;
        c->gen += 1;
        if (c->per_gpu) {
            // "Reorder" packs each job's workers in every new candidate; the same pass scores it
            if ((rc = prof_begin(c, 0)) != ONES_OK) return rc;
            CU(c, launch_reorder_score(c->pop(c->cur), c->ld, c->N, c->W, c->J, c->tab, c->fit(), c->narrow, c->F(), c->G(), c->stream));
            c->launches += 1;
            c->f_valid = true;
            if ((rc = prof_end(c)) != ONES_OK) return rc;
        } else if (!c->fused && (rc = run_fitness(c)) != ONES_OK) {
            return rc;
        }
    }
    c->prof.sample = true;
    return ONES_OK;
}

int ones_best(ones_ctx* c, int repair, int32_t* h_genome, int32_t* h_gpus_per_job, double* h_rate_per_job,
              double* fitness, int32_t* total_gpus, int32_t* index) {
    DeviceScope scope(c);
    if (!c) return ONES_ERR_NULL;
    int rc;
    if (!c->f_valid && (rc = run_fitness(c)) != ONES_OK) return rc;
    int nl = 0;
    CU(c, launch_top(c->F(), c->N, 1, c->best_idx(), c->ws + c->L.top, c->stream, &nl));
    const size_t J = (size_t)c->J;
    unsigned char* pack = reinterpret_cast<unsigned char*>(c->ws + c->L.out_pack);
    BestOut* d_rec = reinterpret_cast<BestOut*>(pack);
    double* d_rate = reinterpret_cast<double*>(pack + 64);
    int32_t* d_genome = reinterpret_cast<int32_t*>(pack + 64 + J * 8);
    int32_t* d_gpus = reinterpret_cast<int32_t*>(pack + 64 + J * 12);
    if (c->packed && !c->int_valid) {  // only the best row is needed as int32
        CU(c, launch_unpack_rows(c->P(c->pcur), c->ld8, 1, c->J, c->pop(c->cur), c->ld, c->best_idx(), c->stream));
        c->launches += 1;
    }
    if (c->per_gpu)
        CU(c, launch_best_per_gpu(c->pop(c->cur), c->ld, c->W, c->J, c->best_idx(), c->tab,
                                  reinterpret_cast<int32_t*>(c->ws + c->L.work), d_genome, d_gpus, d_rate, d_rec,
                                  c->stream));
    else
        CU(c, launch_best(c->pop(c->cur), c->ld, c->J, c->best_idx(), c->tab, c->cap, c->prm.penalty, repair,
                          reinterpret_cast<int32_t*>(c->ws + c->L.work), d_genome, d_gpus, d_rate, d_rec,
                          c->mapped ? c->rowmap(c->mcur) : nullptr, c->stream));
    c->launches += (uint64_t)nl + 1;
    const size_t bytes = 64 + J * 16;
    if ((rc = ensure_staging(c, bytes + 64)) != ONES_OK) return rc;
    CU(c, cudaMemcpyAsync(c->staging, pack, bytes, cudaMemcpyDeviceToHost, c->stream));
    if ((rc = enqueue_flag_read(c)) != ONES_OK) return rc;
    CU(c, cudaStreamSynchronize(c->stream));
    if ((rc = flag_after_sync(c)) != ONES_OK) return rc;
    BestOut rec;
    memcpy(&rec, c->staging, sizeof rec);
    if (h_rate_per_job) memcpy(h_rate_per_job, c->staging + 64, J * 8);
    if (h_genome) memcpy(h_genome, c->staging + 64 + J * 8, J * 4);
    if (h_gpus_per_job) memcpy(h_gpus_per_job, c->staging + 64 + J * 12, J * 4);
    if (fitness) *fitness = rec.fitness;
    if (total_gpus) *total_gpus = rec.total_gpus;
    if (index) *index = rec.index;
    return rec.status ? ONES_ERR_INFEASIBLE : ONES_OK;
}

int ones_update_jobs(ones_ctx* c, const ones_job* jobs, int32_t n_jobs, const int32_t* remap, int32_t capacity) {
    DeviceScope scope(c);
    if (!c || !jobs || !remap) return ONES_ERR_NULL;
    int rc = check_jobs(jobs, n_jobs);
    if (rc) return rc;
    if (capacity <= 0) return ONES_ERR_BAD_PARAM;
    if (n_jobs > c->Jmax) return ONES_ERR_WORKSPACE;
    for (int32_t j = 0; j < n_jobs; ++j)
        if (remap[j] < -1 || remap[j] >= c->J) return ONES_ERR_BAD_PARAM;
    if (c->per_gpu) {
        if (capacity != c->cap) return ONES_ERR_BAD_PARAM;  // a candidate has one gene per GPU of the cluster
        if (refresh_smem(c->W, n_jobs) > (size_t)kMaxSmemPerBlock - 1024) return ONES_ERR_WORKSPACE;
    }
    if ((rc = check_throughput(jobs, n_jobs)) != ONES_OK) return rc;
    if (!c->per_gpu && n_jobs == c->J && c->in_limits && (int32_t)c->h_jobs.size() == n_jobs) {
        // Same jobs in the same columns, and no job's range of exponents shrinks: no gene moves, so the
        // population stays where it is.  With an unchanged table even the scores stay; otherwise the tables are
        // rebuilt and the population is scored again when it is next needed.
        bool same_columns = true, same_table = capacity == c->cap;
        for (int32_t j = 0; j < n_jobs && same_columns; ++j) {
            const ones_job& was = c->h_jobs[j];
            same_columns = remap[j] == j && jobs[j].kmin <= was.kmin && jobs[j].kmax >= was.kmax;
            same_table = same_table && memcmp(&jobs[j], &was, sizeof(ones_job)) == 0;
        }
        if (same_columns) {
            if (same_table) return ONES_OK;
            if ((rc = rebuild_tables(c, jobs, n_jobs, nullptr, false)) != ONES_OK) return rc;
            if (c->packed && !c->fused) return ONES_ERR_BAD_PARAM;
            c->cap = capacity;
            c->f_valid = false;
            c->elites_valid = false;
            return ONES_OK;
        }
    }
    if (c->packed && (rc = unpack_to_int(c)) != ONES_OK) return rc;  // the column map works on the int32 rows
    if ((rc = compact_pool(c)) != ONES_OK) return rc;                // ... in the order of the candidates
    const int64_t old_ld = c->ld;
    const int32_t old_J = c->J;
    rc = rebuild_tables(c, jobs, n_jobs, remap, c->per_gpu);
    if (rc == ONES_OK && c->packed && !c->fused) rc = ONES_ERR_BAD_PARAM;  // tables of the new set do not fit shared memory
    if (rc != ONES_OK) {
        // put the tables of the job set in force back; the population is untouched
        const std::vector<ones_job> keep = c->h_jobs;
        int rc2 = rebuild_tables(c, keep.data(), (int32_t)keep.size());
        return rc2 == ONES_OK ? rc : rc2;
    }
    if (c->per_gpu) {
        // every candidate is refreshed in place (finished jobs leave, limits, new jobs, refill) and packed again
        CU(c, launch_fill_slot_limits(c->tabS.kmin, c->tabS.range, jpad_of(c->W), c->W, n_jobs, c->jobs(), c->fit(),
                                      c->tab.jpad, c->stream));
        CU(c, launch_refresh_per_gpu(c->pop(c->cur), c->ld, c->N, c->W, old_J, n_jobs, c->tab, c->fit(), c->remap(n_jobs),
                                     c->refresh_inv(), c->refresh_cum(), c->stream));
        // "Reorder" of the refreshed rows, scored under the new tables in the same pass
        CU(c, launch_reorder_score(c->pop(c->cur), c->ld, c->N, c->W, n_jobs, c->tab, c->fit(), c->narrow, c->F(), c->G(),
                                   c->stream));
        c->launches += 4;
        c->J = n_jobs;
        c->f_valid = true;
        c->elites_valid = false;
        return ONES_OK;
    }
    const int64_t new_ld = ld_of(n_jobs);
    // c->fused: the new job set's GPU counts fit the 16-bit table and the tables fit shared memory
    const bool scored = c->fused && remap_score_smem(c->tab) <= (size_t)kMaxSmemPerBlock;
    if (scored) {  // the new rows are scored while they are written
        CU(c, launch_remap_score(c->pop(c->cur), old_ld, c->pop(c->cur ^ 1), new_ld, c->N, n_jobs, c->remap(n_jobs),
                                 c->tab, capacity, c->prm.penalty, c->F(), c->G(), c->stream));
    } else {
        CU(c, launch_remap(c->pop(c->cur), old_ld, c->pop(c->cur ^ 1), new_ld, c->N, n_jobs, c->remap(n_jobs),
                           c->tab.kmin, c->tab.range, c->stream));
    }
    c->launches += 1;
    c->cur ^= 1;
    c->J = n_jobs;
    c->W = n_jobs;
    c->ld = new_ld;
    c->cap = capacity;
    c->f_valid = scored;
    c->elites_valid = false;
    c->in_limits = true;  // every gene was clamped into its job's new limits
    if (c->packed) {
        c->int_valid = true;
        return pack_from_int(c);
    }
    return ONES_OK;
}

int ones_last_parents(ones_ctx* c, int32_t* h_parents, int32_t* h_elites) {
    DeviceScope scope(c);
    if (!c) return ONES_ERR_NULL;
    if (h_parents && c->pairs > 0)
        CU(c, cudaMemcpyAsync(h_parents, c->parents(), (size_t)c->pairs * 8, cudaMemcpyDeviceToHost, c->stream));
    if (h_elites && c->prm.elitism > 0 && !c->trunc)
        CU(c, cudaMemcpyAsync(h_elites, c->elites(c->elast), (size_t)c->prm.elitism * 4, cudaMemcpyDeviceToHost, c->stream));
    int rc = enqueue_flag_read(c);
    if (rc) return rc;
    CU(c, cudaStreamSynchronize(c->stream));
    return flag_after_sync(c);
}

int ones_model_table(ones_ctx* c, double* h_X, int32_t* h_g, int32_t* planes) {
    DeviceScope scope(c);
    if (!c) return ONES_ERR_NULL;
    if (planes) *planes = c->tab.k1;
    if (!h_X && !h_g) return ONES_OK;
    double* dX = reinterpret_cast<double*>(c->ws + c->L.exp_X);
    int32_t* dG = reinterpret_cast<int32_t*>(c->ws + c->L.exp_G);
    CU(c, launch_export_tables(c->tab, c->J, dX, dG, c->stream));
    c->launches += 1;
    const size_t cells = (size_t)c->tab.k1 * c->J;
    if (h_X) CU(c, cudaMemcpyAsync(h_X, dX, cells * 8, cudaMemcpyDeviceToHost, c->stream));
    if (h_g) CU(c, cudaMemcpyAsync(h_g, dG, cells * 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    return ONES_OK;
}

size_t ones_select_top_scratch_bytes(int32_t n, int32_t e) {
    if (n <= 0 || e <= 0 || e > ONES_MAX_ELITES || e > n) return 0;
    return top_scratch_bytes(n, e);
}

int ones_select_top(const double* d_fitness, int32_t n, int32_t e, int32_t* d_index, void* d_scratch,
                    size_t scratch_bytes, void* cuda_stream) {
    if (!d_fitness || !d_index || !d_scratch) return ONES_ERR_NULL;
    if (n <= 0 || e <= 0 || e > ONES_MAX_ELITES || e > n) return ONES_ERR_BAD_PARAM;
    if (!aligned16(d_scratch)) return ONES_ERR_ALIGN;
    if (scratch_bytes < top_scratch_bytes(n, e)) return ONES_ERR_WORKSPACE;
    cudaError_t err = launch_top(d_fitness, n, e, d_index, d_scratch, reinterpret_cast<cudaStream_t>(cuda_stream),
                                 nullptr);
    return err == cudaSuccess ? ONES_OK : ONES_ERR_CUDA;
}

int ones_generation(const ones_ctx* c, uint64_t* gen_abs) {
    if (!c || !gen_abs) return ONES_ERR_NULL;
    *gen_abs = c->gen;
    return ONES_OK;
}

int ones_set_generation(ones_ctx* c, uint64_t gen_abs) {
    if (!c) return ONES_ERR_NULL;
    c->gen = gen_abs;
    return ONES_OK;
}

int ones_shape(const ones_ctx* c, int32_t* n_jobs, int32_t* pop, int32_t* capacity, int64_t* ld) {
    if (!c) return ONES_ERR_NULL;
    if (n_jobs) *n_jobs = c->J;
    if (pop) *pop = c->N;
    if (capacity) *capacity = c->cap;
    if (ld) *ld = c->ld;
    return ONES_OK;
}

int ones_kernel_launches(const ones_ctx* c, uint64_t* launches) {
    if (!c || !launches) return ONES_ERR_NULL;
    *launches = c->launches;
    return ONES_OK;
}

int ones_set_profiling(ones_ctx* c, int on) {
    DeviceScope scope(c);
    if (!c) return ONES_ERR_NULL;
    if (on && c->prof.ev.empty()) {
        const size_t want = 4096;
        c->prof.ev.reserve(want);
        for (size_t i = 0; i < want; ++i) {
            cudaEvent_t ev;
            CU(c, cudaEventCreate(&ev));
            c->prof.ev.push_back(ev);
        }
        c->prof.stage.assign(want / 2, 0);
    }
    if (!on) {
        int rc = prof_flush(c);
        if (rc) return rc;
    }
    c->prof.on = on != 0;
    c->prof.every = on > 1 ? on : 1;
    c->prof.sample = true;
    return ONES_OK;
}

int ones_stage_times(ones_ctx* c, double ms[3], uint64_t count[3]) {
    DeviceScope scope(c);
    if (!c || !ms || !count) return ONES_ERR_NULL;
    int rc = prof_flush(c);
    if (rc) return rc;
    for (int s = 0; s < 3; ++s) {
        ms[s] = c->prof.ms[s];
        count[s] = c->prof.count[s];
        c->prof.ms[s] = 0;
        c->prof.count[s] = 0;
    }
    return ONES_OK;
}

int ones_last_cuda_error(const ones_ctx* c) { return c ? c->last_cuda : 0; }

const char* ones_strerror(int code) {
    switch (code) {
        case ONES_OK: return "ok";
        case ONES_ERR_NULL: return "a required pointer is NULL";
        case ONES_ERR_BAD_JOB: return "a job row is out of range";
        case ONES_ERR_BAD_PARAM: return "an argument or parameter is out of range";
        case ONES_ERR_ALIGN: return "pointer not 16-byte aligned or ld not a multiple of 4";
        case ONES_ERR_WORKSPACE: return "workspace too small";
        case ONES_ERR_CUDA: return "a CUDA call failed";
        case ONES_ERR_INFEASIBLE: return "repair could not reach the capacity";
        case ONES_ERR_NOMEM: return "host allocation failed";
        default: return "unknown error code";
    }
}

}  // extern "C"
