// sm_100a kernels of the ONES evolutionary batch-size search.
//
// Data layout in HBM
//   population   int32[N][ld] row-major, one row per candidate schedule, ld = n_jobs rounded up
//                to 4 so that every row starts on a 16-byte boundary (int4 loads/stores)
//   F, G         double[N], int32[N]: score and GPU demand per candidate
//   model tables X (fp64) and G (int32), one plane per exponent, swizzled (see Tables)
// Nothing here is a dense contraction: the kernels are gathers, adds and a counter-based RNG,
// bounded by HBM bandwidth (fitness, evolve) or by launch latency (everything else).
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "ones_internal.h"

namespace ones {

// SMs of the current device (read once per device): persistent grids are sized from it.
int sm_count() {
    constexpr int kDevices = 64;
    static int cached[kDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kDevices) return kSMsDefault;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return kSMsDefault;
        cached[dev] = n < kSMsMax ? n : kSMsMax;
    }
    return cached[dev];
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  Round keys are precomputed on the host.
// ---------------------------------------------------------------------------------------------
RoundKeys make_round_keys(uint64_t seed) {
    RoundKeys rk;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        rk.k[2 * r] = a;
        rk.k[2 * r + 1] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return rk;
}

__device__ __forceinline__ uint4 philox(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                        const RoundKeys& rk) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned long long p0 = (unsigned long long)0xD2511F53u * c0;
        const unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k[2 * r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k[2 * r + 1];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Fourth counter word: stream id in the low 4 bits, high half of the generation above them.
__host__ __device__ __forceinline__ uint32_t counter3(uint32_t stream, uint64_t gen) {
    return stream | ((uint32_t)(gen >> 32) << 4);
}

// Uniform value in [kmin, kmin + range): kmin + floor(frac * range / 2^32).
__device__ __forceinline__ int32_t draw_gene(uint32_t frac, int32_t kmin, int32_t range) {
    return kmin + (int32_t)__umulhi(frac, (uint32_t)range);
}

__host__ __device__ __forceinline__ int32_t slot_of(int32_t j) {
    return (j & ~127) + ((j & 3) << 5) + ((j >> 2) & 31);
}

// Programmatic dependent launch.  A kernel launched with launch_after_previous() may become resident while
// the kernel before it in the stream is still running; everything it does before grid_dependency_wait()
// (staging the model tables, which no kernel of the generation loop writes) overlaps that kernel, and
// nothing written by it is touched until the wait returns, which is when the previous kernel has completed
// and its writes are visible.  grid_dependency_release() lets the next kernel's CTAs become resident early in
// the same way.  Launched normally, a kernel passes the wait at once.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... Params, typename... Args>
static cudaError_t launch_after_previous(void (*kernel)(Params...), int blocks, int threads, size_t smem, cudaStream_t s,
                                         Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// ---------------------------------------------------------------------------------------------
// Model tables: X_j(k), g_j(k) for every job and exponent (throughput model of the job table)
// ---------------------------------------------------------------------------------------------
__global__ void k_build_tables(const ones_job* __restrict__ jobs, int32_t n_jobs, uint32_t flags, Tables t,
                               const double* __restrict__ log2g, int32_t* __restrict__ bad) {
    const int32_t planes = t.k1 + 1;
    const int64_t total = (int64_t)planes * t.jpad;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t k = (int32_t)(i / t.jpad);
        const int32_t j = (int32_t)(i % t.jpad);
        double term = 0.0;
        int32_t gpus = 0;
        if (j < n_jobs) {
            const ones_job job = jobs[j];
            if (k <= job.kmax && k < t.k1) {
                const long long b = (long long)job.b0 << k;
                const long long m = job.max_per_gpu;
                const long long g = (b + m - 1) / m;
                const double local = __ddiv_rn((double)b, (double)g);
                // log2 of a power of two is its exponent, exactly; otherwise the value the caller supplies (its own
                // math library's, so that a comparison with host arithmetic is not decided by a last bit), else the
                // device routine
                const double lg = ((g & (g - 1)) == 0) ? (double)(63 - __clzll(g))
                                  : log2g       ? log2g[(int64_t)k * n_jobs + j]
                                                : log2((double)g);
                const double sec = __dadd_rn(__dadd_rn(job.a, __dmul_rn(job.c, local)), __dmul_rn(job.d, lg));
                const double X = __ddiv_rn((double)b, sec);
                if (!(X > 0.0) || X > 1.7976931348623157e308) atomicOr(bad, 1);  // needs seconds/iteration > 0
                gpus = (int32_t)g;
                term = (flags & ONES_FLAG_SRUF) ? -__ddiv_rn(__dmul_rn(job.weight, (double)gpus), X) : X;
            }
            if (k == 0) {
                t.kmin[j] = job.kmin;
                t.range[j] = job.kmax - job.kmin + 1;
            }
        } else if (k == 0) {
            t.kmin[j] = 0;
            t.range[j] = 1;
        }
        const int64_t at = (int64_t)k * t.jpad + slot_of(j);
        t.X[at] = term;
        t.G[at] = gpus;
    }
}

cudaError_t launch_build_tables(const ones_job* d_jobs, int32_t n_jobs, uint32_t flags, Tables t,
                                const double* d_log2g, int32_t* d_bad, cudaStream_t s) {
    const int64_t total = (int64_t)(t.k1 + 1) * t.jpad;
    const int grid = (int)((total + 255) / 256);
    k_build_tables<<<grid < 1024 ? grid : 1024, 256, 0, s>>>(d_jobs, n_jobs, flags, t, d_log2g, d_bad);
    return cudaGetLastError();
}

// X[k][j], g[k][j] in plain job order for the host (k < k1)
__global__ void k_export_tables(Tables t, int32_t n_jobs, double* __restrict__ X_out, int32_t* __restrict__ G_out) {
    const int64_t total = (int64_t)t.k1 * n_jobs;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t k = (int32_t)(i / n_jobs), j = (int32_t)(i % n_jobs);
        const int64_t at = (int64_t)k * t.jpad + slot_of(j);
        X_out[i] = t.X[at];
        G_out[i] = t.G[at];
    }
}

cudaError_t launch_export_tables(Tables t, int32_t n_jobs, double* X_out, int32_t* G_out, cudaStream_t s) {
    const int64_t total = (int64_t)t.k1 * n_jobs;
    const int grid = (int)((total + 255) / 256);
    k_export_tables<<<grid < 1024 ? grid : 1024, 256, 0, s>>>(t, n_jobs, X_out, G_out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Population set-up: all-minimum population, random population, row copies, column remap
// ---------------------------------------------------------------------------------------------
__global__ void k_fill_min(int32_t* __restrict__ pop, int64_t ld, int32_t n, int32_t n_jobs, Tables t) {
    const int64_t total = (int64_t)n * ld;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t j = (int32_t)(i % ld);
        pop[i] = j < n_jobs ? t.kmin[j] : 0;
    }
}

cudaError_t launch_fill_min(int32_t* pop, int64_t ld, int32_t n, int32_t n_jobs, Tables t, cudaStream_t s) {
    const int64_t total = (int64_t)n * ld;
    const int64_t grid = (total + 255) / 256;
    k_fill_min<<<(int)(grid < sm_count() * 8 ? grid : sm_count() * 8), 256, 0, s>>>(pop, ld, n, n_jobs, t);
    return cudaGetLastError();
}

// One thread per int4 of the population: four genes from one Philox call.
__global__ void k_randomize(int32_t* __restrict__ pop, int64_t ld, int32_t n, int32_t n_jobs, Tables t,
                            RoundKeys keys) {
    const int32_t nvec = (int32_t)(ld >> 2);
    const int64_t total = (int64_t)n * nvec;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t row = (int32_t)(i / nvec), v = (int32_t)(i % nvec);
        const int4 kmin = *reinterpret_cast<const int4*>(t.kmin + 4 * v);
        const int4 range = *reinterpret_cast<const int4*>(t.range + 4 * v);
        int4 out = kmin;  // candidate 0: every job at its smallest batch
        if (row > 0) {
            const uint4 w = philox((uint32_t)v, (uint32_t)row, 0u, counter3(STREAM_INIT, 0), keys);
            out.x = draw_gene(w.x, kmin.x, range.x);
            out.y = draw_gene(w.y, kmin.y, range.y);
            out.z = draw_gene(w.z, kmin.z, range.z);
            out.w = draw_gene(w.w, kmin.w, range.w);
        }
        *reinterpret_cast<int4*>(pop + (int64_t)row * ld + 4 * v) = out;
    }
}

cudaError_t launch_randomize(int32_t* pop, int64_t ld, int32_t n, int32_t n_jobs, Tables t,
                             RoundKeys keys, cudaStream_t s) {
    const int64_t total = (int64_t)n * (ld >> 2);
    const int64_t grid = (total + 255) / 256;
    k_randomize<<<(int)(grid < sm_count() * 8 ? grid : sm_count() * 8), 256, 0, s>>>(pop, ld, n, n_jobs, t, keys);
    return cudaGetLastError();
}

__global__ void k_copy_rows(const int32_t* __restrict__ src, int64_t ld_src, int32_t* __restrict__ dst,
                            int64_t ld_dst, int32_t n, int32_t n_jobs, int zero_pad) {
    const int64_t width = zero_pad ? ld_dst : n_jobs;
    const int64_t total = (int64_t)n * width;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / width;
        const int32_t j = (int32_t)(i % width);
        dst[row * ld_dst + j] = j < n_jobs ? src[row * ld_src + j] : 0;
    }
}

cudaError_t launch_copy_rows(const int32_t* src, int64_t ld_src, int32_t* dst, int64_t ld_dst, int32_t n,
                             int32_t n_jobs, int zero_pad, cudaStream_t s) {
    const int64_t total = (int64_t)n * (zero_pad ? ld_dst : n_jobs);
    const int64_t grid = (total + 255) / 256;
    if (grid == 0) return cudaSuccess;
    k_copy_rows<<<(int)(grid < sm_count() * 16 ? grid : sm_count() * 16), 256, 0, s>>>(src, ld_src, dst, ld_dst, n, n_jobs,
                                                                          zero_pad);
    return cudaGetLastError();
}

__global__ void k_remap(const int32_t* __restrict__ src, int64_t ld_src, int32_t* __restrict__ dst,
                        int64_t ld_dst, int32_t n, int32_t n_jobs_new, const int32_t* __restrict__ remap,
                        const int32_t* __restrict__ kmin_new, const int32_t* __restrict__ range_new) {
    const int64_t total = (int64_t)n * ld_dst;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / ld_dst;
        const int32_t j = (int32_t)(i % ld_dst);
        int32_t k = 0;
        if (j < n_jobs_new) {
            const int32_t lo = kmin_new[j], hi = lo + range_new[j] - 1;
            const int32_t from = remap[j];
            k = lo;
            if (from >= 0) k = min(max(src[row * ld_src + from], lo), hi);
        }
        dst[i] = k;
    }
}

cudaError_t launch_remap(const int32_t* src, int64_t ld_src, int32_t* dst, int64_t ld_dst, int32_t n,
                         int32_t n_jobs_new, const int32_t* remap, const int32_t* kmin_new,
                         const int32_t* range_new, cudaStream_t s) {
    const int64_t total = (int64_t)n * ld_dst;
    const int64_t grid = (total + 255) / 256;
    k_remap<<<(int)(grid < sm_count() * 16 ? grid : sm_count() * 16), 256, 0, s>>>(src, ld_src, dst, ld_dst, n, n_jobs_new,
                                                                      remap, kmin_new, range_new);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Fitness: one candidate per warp.  Lane l reads the int4 at genes 4l..4l+3 of every block of 128
// genes, looks each gene's (X, g) up in the tables and accumulates privately in increasing job
// order; a five-step butterfly over the 32 lanes finishes the fixed-order sum.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int4 ld_genes(const int4* p) {
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <bool SMEM, int UNROLL>
__global__ void __launch_bounds__(1024, 1)
k_fitness(const int32_t* __restrict__ genomes, int64_t ld, int32_t n, int32_t n_jobs, Tables t,
          int32_t capacity, double penalty, double* __restrict__ F, int32_t* __restrict__ G) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int32_t planes = t.k1 + 1;
    const double* __restrict__ lutX = t.X;
    const int32_t* __restrict__ lutG = t.G;
    if (SMEM) {
        // stage both tables in shared memory: X planes first, then g planes
        double* sX = reinterpret_cast<double*>(smem_raw);
        int32_t* sG = reinterpret_cast<int32_t*>(smem_raw + (size_t)planes * t.jpad * sizeof(double));
        const int32_t nX = planes * t.jpad / 2;  // int4 = two doubles
        const int32_t nG = planes * t.jpad / 4;  // int4 = four ints
        const int4* gX = reinterpret_cast<const int4*>(t.X);
        const int4* gG = reinterpret_cast<const int4*>(t.G);
        for (int32_t i = threadIdx.x; i < nX; i += blockDim.x) reinterpret_cast<int4*>(sX)[i] = gX[i];
        for (int32_t i = threadIdx.x; i < nG; i += blockDim.x) reinterpret_cast<int4*>(sG)[i] = gG[i];
        __syncthreads();
        lutX = sX;
        lutG = sG;
    }
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = blockDim.x >> 5;
    const int64_t total_warps = (int64_t)gridDim.x * warps_per_block;
    const int32_t nvec = (n_jobs + 3) >> 2;
    const uint32_t kcap = (uint32_t)t.k1;
    const int32_t jpad = t.jpad;

    for (int64_t cand = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); cand < n; cand += total_warps) {
        const int4* row = reinterpret_cast<const int4*>(genomes + cand * ld);
        double sum = 0.0;
        int32_t gpus = 0;
        for (int32_t v0 = 0; v0 < nvec; v0 += 32 * UNROLL) {
            int4 q[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int32_t v = v0 + u * 32 + lane;
                if (v < nvec) q[u] = ld_genes(row + v);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int32_t v = v0 + u * 32 + lane;
                if (v < nvec) {
                    const int32_t base = ((v0 >> 5) + u) * 128 + lane;  // slot of gene 4l of this block
                    const int32_t i0 = (int32_t)min((uint32_t)q[u].x, kcap) * jpad + base;
                    const int32_t i1 = (int32_t)min((uint32_t)q[u].y, kcap) * jpad + base + 32;
                    const int32_t i2 = (int32_t)min((uint32_t)q[u].z, kcap) * jpad + base + 64;
                    const int32_t i3 = (int32_t)min((uint32_t)q[u].w, kcap) * jpad + base + 96;
                    sum = __dadd_rn(sum, lutX[i0]); gpus += lutG[i0];
                    sum = __dadd_rn(sum, lutX[i1]); gpus += lutG[i1];
                    sum = __dadd_rn(sum, lutX[i2]); gpus += lutG[i2];
                    sum = __dadd_rn(sum, lutX[i3]); gpus += lutG[i3];
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
            gpus += __shfl_xor_sync(0xFFFFFFFFu, gpus, off);
        }
        if (lane == 0) {
            const int32_t over = gpus > capacity ? gpus - capacity : 0;
            F[cand] = __dsub_rn(sum, __dmul_rn(penalty, (double)over));
            if (G) G[cand] = gpus;
        }
    }
}

cudaError_t launch_fitness(const int32_t* genomes, int64_t ld, int32_t n, int32_t n_jobs, Tables t,
                           int32_t capacity, double penalty, double* F, int32_t* G, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const size_t lut_bytes = (size_t)(t.k1 + 1) * t.jpad * 12;
    const bool big = n >= sm_count() * 32;
    const int threads = big ? 1024 : 256;
    const int wpb = threads / 32;
    int64_t blocks = ((int64_t)n + wpb - 1) / wpb;
    if (lut_bytes <= (size_t)kMaxSmemPerBlock) {
        int per_sm = (int)(kMaxSmemPerBlock / (lut_bytes + 1024));
        if (per_sm < 1) per_sm = 1;
        const int by_threads = 2048 / threads;
        if (per_sm > by_threads) per_sm = by_threads;
        if (blocks > (int64_t)sm_count() * per_sm) blocks = (int64_t)sm_count() * per_sm;
        cudaError_t e = cudaFuncSetAttribute(k_fitness<true, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kMaxSmemPerBlock);
        if (e != cudaSuccess) return e;
        k_fitness<true, 4><<<(int)blocks, threads, lut_bytes, s>>>(genomes, ld, n, n_jobs, t, capacity, penalty, F, G);
    } else {
        // tables too large for shared memory: read them through L1/L2
        if (blocks > (int64_t)sm_count() * (2048 / threads)) blocks = (int64_t)sm_count() * (2048 / threads);
        k_fitness<false, 4><<<(int)blocks, threads, 0, s>>>(genomes, ld, n, n_jobs, t, capacity, penalty, F, G);
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Packed candidates: one byte per gene (exponents are at most 15; 0xFF = the job waits), a quarter of the
// bytes of the int32 rows.  A packed row is a sequence of tiles of 512 genes (row stride = jobs rounded up
// to 512 bytes).  Inside a tile the bytes are ordered so that ONE 16-byte load gives lane l exactly the
// genes it sums in the fixed order: byte 16*l + 4*b + s holds gene 128*b + 4*l + s of the tile (b = 0..3
// the 128-gene block, s = 0..3), i.e. the genes 4l..4l+3 of four consecutive blocks.  The lane adds them
// block after block, so partial sum l receives its jobs in increasing order and scores are bit-identical
// to those of the int32 rows.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_pack_rows(const int32_t* __restrict__ src, int64_t ld, int32_t n, int32_t n_jobs, uint8_t* __restrict__ dst, int64_t ld8) {
    const int32_t groups = (int32_t)(ld8 >> 4);  // 16-byte groups per packed row
    const int64_t total = (int64_t)n * groups;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / groups;
        const int32_t grp = (int32_t)(i % groups);
        const int32_t tile = grp >> 5, l = grp & 31;
        uint32_t w[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int32_t j0 = tile * 512 + b * 128 + 4 * l;
            int4 g = make_int4(-1, -1, -1, -1);
            if (j0 + 3 < n_jobs) {
                g = *reinterpret_cast<const int4*>(src + row * ld + j0);
            } else {
                if (j0 < n_jobs) g.x = src[row * ld + j0];
                if (j0 + 1 < n_jobs) g.y = src[row * ld + j0 + 1];
                if (j0 + 2 < n_jobs) g.z = src[row * ld + j0 + 2];
            }
            w[b] = min((uint32_t)g.x, 255u) | (min((uint32_t)g.y, 255u) << 8) | (min((uint32_t)g.z, 255u) << 16) |
                   (min((uint32_t)g.w, 255u) << 24);
        }
        *reinterpret_cast<uint4*>(dst + row * ld8 + 16 * (int64_t)grp) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

cudaError_t launch_pack_rows(const int32_t* src, int64_t ld, int32_t n, int32_t n_jobs, uint8_t* dst, int64_t ld8,
                             cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const int64_t total = (int64_t)n * (ld8 >> 4);
    const int64_t grid = (total + 255) / 256;
    k_pack_rows<<<(int)(grid < sm_count() * 16 ? grid : sm_count() * 16), 256, 0, s>>>(src, ld, n, n_jobs, dst, ld8);
    return cudaGetLastError();
}

// Packed rows back to int32 rows (0xFF -> -1, the waiting state).  One thread per int4 of the int32 row: its four
// genes are one aligned 32-bit word of the tile.  row_index != NULL: only row *row_index is unpacked, into the
// same row of dst.  Columns from n_jobs up to ld are written as 0.
__global__ void __launch_bounds__(256)
k_unpack_rows(const uint8_t* __restrict__ src, int64_t ld8, int32_t n, int32_t n_jobs, int32_t* __restrict__ dst, int64_t ld,
              const int32_t* __restrict__ row_index) {
    const int32_t nvec = (int32_t)(ld >> 2);
    const int64_t total = (int64_t)n * nvec;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = row_index ? (int64_t)*row_index : i / nvec;
        const int32_t j0 = 4 * (int32_t)(i % nvec);
        const int32_t tile = j0 >> 9, b = (j0 >> 7) & 3, l = (j0 >> 2) & 31;
        const uint32_t w = *reinterpret_cast<const uint32_t*>(src + row * ld8 + (int64_t)tile * 512 + 16 * l + 4 * b);
        int4 g;
        g.x = (int32_t)(w & 0xFFu);
        g.y = (int32_t)((w >> 8) & 0xFFu);
        g.z = (int32_t)((w >> 16) & 0xFFu);
        g.w = (int32_t)(w >> 24);
        g.x = j0 < n_jobs ? (g.x == 255 ? -1 : g.x) : 0;
        g.y = j0 + 1 < n_jobs ? (g.y == 255 ? -1 : g.y) : 0;
        g.z = j0 + 2 < n_jobs ? (g.z == 255 ? -1 : g.z) : 0;
        g.w = j0 + 3 < n_jobs ? (g.w == 255 ? -1 : g.w) : 0;
        *reinterpret_cast<int4*>(dst + row * ld + j0) = g;
    }
}

cudaError_t launch_unpack_rows(const uint8_t* src, int64_t ld8, int32_t n, int32_t n_jobs, int32_t* dst, int64_t ld,
                               const int32_t* row_index, cudaStream_t s) {
    if (row_index) n = 1;
    if (n <= 0) return cudaSuccess;
    const int64_t total = (int64_t)n * (ld >> 2);
    const int64_t grid = (total + 255) / 256;
    k_unpack_rows<<<(int)(grid < sm_count() * 16 ? grid : sm_count() * 16), 256, 0, s>>>(src, ld8, n, n_jobs, dst, ld, row_index);
    return cudaGetLastError();
}

// Fitness of packed candidates: one candidate per warp, one 16-byte load per lane and tile (UNROLL tiles in
// flight), tables in shared memory as for k_fitness.
template <bool SMEM, int UNROLL>
__global__ void __launch_bounds__(1024, 1)
k_fitness_packed(const uint8_t* __restrict__ rows, int64_t ld8, int32_t n, Tables t, int32_t capacity, double penalty,
                 double* __restrict__ F, int32_t* __restrict__ G) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int32_t planes = t.k1 + 1;
    const double* __restrict__ lutX = t.X;
    const int32_t* __restrict__ lutG = t.G;
    if (SMEM) {
        double* sX = reinterpret_cast<double*>(smem_raw);
        int32_t* sG = reinterpret_cast<int32_t*>(smem_raw + (size_t)planes * t.jpad * sizeof(double));
        const int32_t nX = planes * t.jpad / 2;
        const int32_t nG = planes * t.jpad / 4;
        const int4* gX = reinterpret_cast<const int4*>(t.X);
        const int4* gG = reinterpret_cast<const int4*>(t.G);
        for (int32_t i = threadIdx.x; i < nX; i += blockDim.x) reinterpret_cast<int4*>(sX)[i] = gX[i];
        for (int32_t i = threadIdx.x; i < nG; i += blockDim.x) reinterpret_cast<int4*>(sG)[i] = gG[i];
        __syncthreads();
        lutX = sX;
        lutG = sG;
    }
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = blockDim.x >> 5;
    const int64_t total_warps = (int64_t)gridDim.x * warps_per_block;
    const uint32_t kcap = (uint32_t)t.k1;
    const int32_t jpad = t.jpad;
    const int32_t tiles = (jpad + 511) >> 9;  // tiles that hold jobs (the tables end at jpad)

    for (int64_t cand = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); cand < n; cand += total_warps) {
        const uint4* row = reinterpret_cast<const uint4*>(rows + cand * ld8);
        double sum = 0.0;
        int32_t gpus = 0;
        for (int32_t t0 = 0; t0 < tiles; t0 += UNROLL) {
            uint4 q[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u)
                if (t0 + u < tiles) q[u] = __ldcs(row + (t0 + u) * 32 + lane);
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (t0 + u < tiles) {
                    const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const int32_t base = ((t0 + u) * 4 + b) * 128 + lane;  // slot of gene 4l of this block
                        if (base < jpad) {  // whole blocks past the tables hold no jobs (warp-uniform)
#pragma unroll
                            for (int s4 = 0; s4 < 4; ++s4) {
                                const uint32_t k = (w[b] >> (8 * s4)) & 0xFFu;
                                const int32_t at = (int32_t)min(k, kcap) * jpad + base + 32 * s4;
                                sum = __dadd_rn(sum, lutX[at]);
                                gpus += lutG[at];
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
            gpus += __shfl_xor_sync(0xFFFFFFFFu, gpus, off);
        }
        if (lane == 0) {
            const int32_t over = gpus > capacity ? gpus - capacity : 0;
            F[cand] = __dsub_rn(sum, __dmul_rn(penalty, (double)over));
            if (G) G[cand] = gpus;
        }
    }
}

cudaError_t launch_fitness_packed(const uint8_t* rows, int64_t ld8, int32_t n, Tables t, int32_t capacity,
                                  double penalty, double* F, int32_t* G, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const size_t lut_bytes = (size_t)(t.k1 + 1) * t.jpad * 12;
    const bool big = n >= sm_count() * 32;
    const int threads = big ? 1024 : 256;
    const int wpb = threads / 32;
    int64_t blocks = ((int64_t)n + wpb - 1) / wpb;
    if (lut_bytes <= (size_t)kMaxSmemPerBlock) {
        int per_sm = (int)(kMaxSmemPerBlock / (lut_bytes + 1024));
        if (per_sm < 1) per_sm = 1;
        const int by_threads = 2048 / threads;
        if (per_sm > by_threads) per_sm = by_threads;
        if (blocks > (int64_t)sm_count() * per_sm) blocks = (int64_t)sm_count() * per_sm;
        cudaError_t e = cudaFuncSetAttribute(k_fitness_packed<true, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kMaxSmemPerBlock);
        if (e != cudaSuccess) return e;
        k_fitness_packed<true, 4><<<(int)blocks, threads, lut_bytes, s>>>(rows, ld8, n, t, capacity, penalty, F, G);
    } else {
        if (blocks > (int64_t)sm_count() * (2048 / threads)) blocks = (int64_t)sm_count() * (2048 / threads);
        k_fitness_packed<false, 4><<<(int)blocks, threads, 0, s>>>(rows, ld8, n, t, capacity, penalty, F, G);
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Top-e selection (score descending, index ascending): per-block partial lists, then one block
// merges them.  Scores are mapped to order-preserving 64-bit keys; NaN ranks lowest.
// ---------------------------------------------------------------------------------------------
struct Rec {
    unsigned long long key;
    int32_t idx;
    int32_t pad;
};

__device__ __forceinline__ unsigned long long score_key(double f) {
    if (f != f) return 0ull;
    const unsigned long long b = (unsigned long long)__double_as_longlong(f + 0.0);  // -0 -> +0
    return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

// true when a ranks before b
__device__ __forceinline__ bool before(unsigned long long ka, int32_t ia, unsigned long long kb, int32_t ib) {
    return ka > kb || (ka == kb && ia < ib);
}

// Block-wide best record that ranks strictly after `prev` (or any record when !have_prev).
// SRC 0: items are scores F[i] with index lo + i; 1: Rec in global memory, possibly written by other
// CTAs of the same launch (read through L2); 2: Rec in shared memory.  s_warp holds one Rec per warp.
template <int SRC>
__device__ Rec block_next_best(const void* items, int32_t count, int32_t lo, bool have_prev, Rec prev,
                               Rec* s_warp) {
    Rec best;
    best.key = 0ull;
    best.idx = -1;
    best.pad = 0;
    for (int32_t i = threadIdx.x; i < count; i += blockDim.x) {
        unsigned long long k;
        int32_t id;
        if (SRC == 0) {
            k = score_key(reinterpret_cast<const double*>(items)[i]);
            id = lo + i;
        } else {
            int4 raw;
            if (SRC == 1) raw = __ldcg(reinterpret_cast<const int4*>(items) + i);
            else raw = reinterpret_cast<const int4*>(items)[i];
            k = ((unsigned long long)(uint32_t)raw.y << 32) | (uint32_t)raw.x;
            id = raw.z;
            if (id < 0) continue;
        }
        if (have_prev && !before(prev.key, prev.idx, k, id)) continue;
        if (best.idx < 0 || before(k, id, best.key, best.idx)) {
            best.key = k;
            best.idx = id;
        }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xFFFFFFFFu, best.key, off);
        const int32_t oi = __shfl_xor_sync(0xFFFFFFFFu, best.idx, off);
        if (oi >= 0 && (best.idx < 0 || before(ok, oi, best.key, best.idx))) {
            best.key = ok;
            best.idx = oi;
        }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
    __syncthreads();  // s_warp may still be read from the previous round
    if (lane == 0) s_warp[warp] = best;
    __syncthreads();
    // every warp reduces the per-warp winners again (same result everywhere, no third barrier)
    Rec r;
    r.key = 0ull;
    r.idx = -1;
    r.pad = 0;
    if (lane < nwarp) r = s_warp[lane];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xFFFFFFFFu, r.key, off);
        const int32_t oi = __shfl_xor_sync(0xFFFFFFFFu, r.idx, off);
        if (oi >= 0 && (r.idx < 0 || before(ok, oi, r.key, r.idx))) {
            r.key = ok;
            r.idx = oi;
        }
    }
    return r;
}

// Small e (at most E, E <= 4): every thread keeps the E best of its own items as a sorted list in registers
// and a warp pops its best e times (butterfly over the heads of the lists; the lane that owned the winner
// moves its list up), so a slice is read once and the block needs one barrier instead of two per rank.
template <int E>
struct TopList {
    unsigned long long key[E];
    int32_t idx[E];
};

// true when record a ranks before record b; a record with idx < 0 is empty and ranks last
__device__ __forceinline__ bool rec_before(unsigned long long ka, int32_t ia, unsigned long long kb, int32_t ib) {
    return ia >= 0 && (ib < 0 || before(ka, ia, kb, ib));
}

template <int E>
__device__ __forceinline__ void top_list_clear(TopList<E>& l) {
#pragma unroll
    for (int r = 0; r < E; ++r) {
        l.key[r] = 0ull;
        l.idx[r] = -1;
    }
}

template <int E>
__device__ __forceinline__ void top_list_insert(TopList<E>& l, unsigned long long k, int32_t id) {
    if (!rec_before(k, id, l.key[E - 1], l.idx[E - 1])) return;
    l.key[E - 1] = k;
    l.idx[E - 1] = id;
#pragma unroll
    for (int r = E - 1; r > 0; --r) {
        if (rec_before(l.key[r], l.idx[r], l.key[r - 1], l.idx[r - 1])) {
            const unsigned long long tk = l.key[r];
            const int32_t ti = l.idx[r];
            l.key[r] = l.key[r - 1];
            l.idx[r] = l.idx[r - 1];
            l.key[r - 1] = tk;
            l.idx[r - 1] = ti;
        }
    }
}

// The warp's best remaining record (to every lane); its owner drops it from its list.
template <int E>
__device__ __forceinline__ Rec warp_pop_best(TopList<E>& l) {
    Rec best;
    best.key = l.key[0];
    best.idx = l.idx[0];
    best.pad = 0;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xFFFFFFFFu, best.key, off);
        const int32_t oi = __shfl_xor_sync(0xFFFFFFFFu, best.idx, off);
        if (rec_before(ok, oi, best.key, best.idx)) {
            best.key = ok;
            best.idx = oi;
        }
    }
    if (best.idx >= 0 && l.idx[0] == best.idx) {
#pragma unroll
        for (int r = 0; r + 1 < E; ++r) {
            l.key[r] = l.key[r + 1];
            l.idx[r] = l.idx[r + 1];
        }
        l.key[E - 1] = 0ull;
        l.idx[E - 1] = -1;
    }
    return best;
}

// The e best (e <= E) of `count` items of one block of THREADS threads, in rank order, written by thread 0 to out[0..e)
// (empty records when there are fewer than e items).  SRC 0: the items are scores F[i] with index lo + i;
// 1: records in global memory, possibly written by other CTAs of the same launch (read through L2, four
// loads in flight per thread); 2: records in shared memory.  IDX_OUT: out is an int32 array that receives
// the indices only.  s_list: (THREADS / 32) * E records.
template <int E, int SRC, bool IDX_OUT = false, int THREADS = 256>
__device__ __forceinline__ void block_top_small(const void* __restrict__ items, int32_t count, int32_t lo, int32_t e,
                                                void* __restrict__ out, Rec* __restrict__ s_list) {
    TopList<E> l;
    top_list_clear(l);
    if (SRC == 1) {
        for (int32_t i0 = threadIdx.x; i0 < count; i0 += 4 * THREADS) {
            int4 raw[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i0 + u * THREADS < count) raw[u] = __ldcg(reinterpret_cast<const int4*>(items) + i0 + u * THREADS);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i0 + u * THREADS < count)
                    top_list_insert(l, ((unsigned long long)(uint32_t)raw[u].y << 32) | (uint32_t)raw[u].x, raw[u].z);
        }
    } else {
        for (int32_t i = threadIdx.x; i < count; i += THREADS) {
            if (SRC == 2) {
                const Rec q = reinterpret_cast<const Rec*>(items)[i];
                top_list_insert(l, q.key, q.idx);
            } else {
                top_list_insert(l, score_key(reinterpret_cast<const double*>(items)[i]), lo + i);
            }
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int32_t r = 0; r < e; ++r) {
        const Rec best = warp_pop_best(l);
        if (lane == 0) s_list[warp * E + r] = best;
    }
    __syncthreads();
    if (warp == 0) {
        TopList<E> m;
        top_list_clear(m);
        for (int32_t i = lane; i < (THREADS / 32) * E; i += 32) {
            const int32_t w = i / E, r = i % E;
            if (r < e) top_list_insert(m, s_list[w * E + r].key, s_list[w * E + r].idx);
        }
        for (int32_t r = 0; r < e; ++r) {
            const Rec best = warp_pop_best(m);
            if (lane == 0) {
                if (IDX_OUT) reinterpret_cast<int32_t*>(out)[r] = best.idx;
                else reinterpret_cast<Rec*>(out)[r] = best;
            }
        }
    }
}

// The same merge of at most 64 records in global memory by one warp alone (no barrier): idx_out[0..e).
template <int E>
__device__ __forceinline__ void warp_merge_small(const Rec* partial, int32_t count, int32_t e,
                                                 int32_t* __restrict__ idx_out) {
    const int lane = threadIdx.x & 31;
    TopList<E> m;
    top_list_clear(m);
    int4 raw[2];
#pragma unroll
    for (int u = 0; u < 2; ++u)
        if (lane + 32 * u < count) raw[u] = __ldcg(reinterpret_cast<const int4*>(partial) + lane + 32 * u);
#pragma unroll
    for (int u = 0; u < 2; ++u)
        if (lane + 32 * u < count)
            top_list_insert(m, ((unsigned long long)(uint32_t)raw[u].y << 32) | (uint32_t)raw[u].x, raw[u].z);
    for (int32_t r = 0; r < e; ++r) {
        const Rec best = warp_pop_best(m);
        if (lane == 0) idx_out[r] = best.idx;
    }
}

__global__ void __launch_bounds__(256) k_top_partial(const double* __restrict__ F, int32_t n, int32_t e,
                                                     int32_t per_block, Rec* __restrict__ partial) {
    __shared__ Rec s_warp[32];
    const int32_t lo = blockIdx.x * per_block;
    const int32_t count = min(per_block, n - lo);
    Rec prev;
    prev.key = 0;
    prev.idx = -1;
    prev.pad = 0;
    for (int32_t r = 0; r < e; ++r) {
        Rec best = block_next_best<0>(F + lo, count > 0 ? count : 0, lo, r > 0, prev, s_warp);
        if (threadIdx.x == 0) partial[(int64_t)blockIdx.x * e + r] = best;
        prev = best;
        if (best.idx < 0) {  // fewer than e items in this block: mark the rest empty
            for (int32_t r2 = r + 1 + threadIdx.x; r2 < e; r2 += blockDim.x)
                partial[(int64_t)blockIdx.x * e + r2] = best;
            break;
        }
    }
}

__global__ void __launch_bounds__(256) k_top_final(const Rec* __restrict__ partial, int32_t count, int32_t e,
                                                   int32_t* __restrict__ idx_out) {
    __shared__ Rec s_warp[32];
    Rec prev;
    prev.key = 0;
    prev.idx = -1;
    prev.pad = 0;
    for (int32_t r = 0; r < e; ++r) {
        Rec best = block_next_best<1>(partial, count, 0, r > 0, prev, s_warp);
        if (threadIdx.x == 0) idx_out[r] = best.idx;
        prev = best;
    }
}

static int top_blocks(int32_t n) {
    int b = (n + 1023) / 1024;
    if (b < 1) b = 1;
    if (b > kTopBlocksMax) b = kTopBlocksMax;
    return b;
}

size_t top_scratch_bytes(int32_t n, int32_t e) {
    (void)n;
    return (size_t)kTopBlocksMax * (size_t)e * sizeof(Rec);
}

cudaError_t launch_top(const double* F, int32_t n, int32_t e, int32_t* idx_out, void* scratch, cudaStream_t s,
                       int* launches) {
    if (e <= 0) return cudaSuccess;
    const int blocks = top_blocks(n);
    const int32_t per_block = (n + blocks - 1) / blocks;
    Rec* partial = reinterpret_cast<Rec*>(scratch);
    k_top_partial<<<blocks, 256, 0, s>>>(F, n, e, per_block, partial);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    k_top_final<<<1, 256, 0, s>>>(partial, blocks * e, e, idx_out);
    if (launches) *launches += 2;
    return cudaGetLastError();
}

static int top_blocks(int32_t n);

// Selection stage of one generation in a single launch: CTAs [0, top_blocks) build the partial
// top-e lists and the last of them to finish merges the lists into `elites`; the remaining CTAs run
// the tournaments.  `done` counts finished top CTAs; it must be zero at launch and is zero again
// at exit.  Nothing waits: the merging CTA is simply the one whose increment completes the count.
__device__ __forceinline__ void tournament_thread(const double* __restrict__ F, int32_t n, int32_t tournament,
                                                  int32_t i, const RoundKeys& keys, uint32_t gen_lo, uint32_t c3,
                                                  int32_t* __restrict__ parents) {
    const uint32_t q = (uint32_t)(i >> 1);
    int32_t win = -1;
    double fwin = 0.0;
    for (int32_t t0 = 0; t0 < tournament; t0 += 4) {
        const uint4 w4 = philox((uint32_t)(t0 >> 2), q, gen_lo, c3, keys);
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (t0 + u < tournament) {
                const int32_t idx = (int32_t)__umulhi(w[u], (uint32_t)n);
                const double f = F[idx];
                if (win < 0 || f > fwin || (f == fwin && idx < win)) {
                    win = idx;
                    fwin = f;
                }
            }
        }
    }
    parents[i] = win;
}

__global__ void __launch_bounds__(256)
k_select_stage(const double* __restrict__ F, int32_t n, int32_t tournament, int32_t pairs, RoundKeys keys,
               uint32_t gen_lo, uint32_t c3a, uint32_t c3b, int32_t* __restrict__ parents, int32_t e,
               int32_t top_blocks, int32_t per_block, Rec* __restrict__ partial, int32_t* __restrict__ elites,
               unsigned int* __restrict__ done) {
    grid_dependency_wait();  // the scores come from the kernel before
    if (blockIdx.x == 0 && threadIdx.x == 0) done[1] = 0u;  // work-item counter of the evolve kernel that follows
    if ((int32_t)blockIdx.x >= top_blocks) {
        const int32_t i = ((int32_t)blockIdx.x - top_blocks) * blockDim.x + threadIdx.x;
        if (i < 2 * pairs) tournament_thread(F, n, tournament, i, keys, gen_lo, (i & 1) ? c3b : c3a, parents);
        return;
    }
    __shared__ Rec s_warp[32];
    __shared__ bool s_last;
    const int32_t lo = blockIdx.x * per_block;
    const int32_t count = max(0, min(per_block, n - lo));
    const bool small = e <= 4;  // lists in registers, one barrier
    Rec prev;
    prev.key = 0;
    prev.idx = -1;
    prev.pad = 0;
    if (small) {
        if (e <= 2) block_top_small<2, 0>(F + lo, count, lo, e, partial + (int64_t)blockIdx.x * e, s_warp);
        else block_top_small<4, 0>(F + lo, count, lo, e, partial + (int64_t)blockIdx.x * e, s_warp);
    } else {
        for (int32_t r = 0; r < e; ++r) {
            Rec best = block_next_best<0>(F + lo, count, lo, r > 0, prev, s_warp);
            if (threadIdx.x == 0) partial[(int64_t)blockIdx.x * e + r] = best;
            prev = best;
            if (best.idx < 0) {  // fewer than e items in this slice: mark the rest empty
                for (int32_t r2 = r + 1 + threadIdx.x; r2 < e; r2 += blockDim.x)
                    partial[(int64_t)blockIdx.x * e + r2] = best;
                break;
            }
        }
    }
    // from here on only the merging CTA still works: the next kernel's CTAs may take the other SMs (they
    // arrive once every tournament CTA has ended and every top-e CTA is here)
    grid_dependency_release();
    __threadfence();  // every thread's records before the CTA is counted as finished
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(done, 1u) == (unsigned int)(top_blocks - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (small && top_blocks * e <= 64) {  // a handful of records: one warp, no barrier
        if (threadIdx.x < 32) {
            if (e <= 2) warp_merge_small<2>(partial, top_blocks * e, e, elites);
            else warp_merge_small<4>(partial, top_blocks * e, e, elites);
        }
    } else if (small) {
        if (e <= 2) block_top_small<2, 1, true>(partial, top_blocks * e, 0, e, elites, s_warp);
        else block_top_small<4, 1, true>(partial, top_blocks * e, 0, e, elites, s_warp);
    } else {
        prev.key = 0;
        prev.idx = -1;
        for (int32_t r = 0; r < e; ++r) {
            Rec best = block_next_best<1>(partial, top_blocks * e, 0, r > 0, prev, s_warp);
            if (threadIdx.x == 0) elites[r] = best.idx;
            prev = best;
        }
    }
    if (threadIdx.x == 0) *done = 0u;
}

cudaError_t launch_select_stage(const double* F, int32_t n, int32_t tournament, int32_t pairs, RoundKeys keys,
                                uint64_t gen, int32_t* parents, int32_t e, int32_t* elites, void* scratch,
                                unsigned int* done, cudaStream_t s) {
    const int top_b = e > 0 ? top_blocks(n) : 0;
    const int sel_b = (2 * pairs + 255) / 256;
    if (top_b + sel_b == 0) return cudaSuccess;
    const int32_t per_block = top_b ? (n + top_b - 1) / top_b : 0;
    return launch_after_previous(k_select_stage, top_b + sel_b, 256, 0, s, F, n, tournament, pairs, keys, (uint32_t)gen,
                                 counter3(STREAM_SEL_A, gen), counter3(STREAM_SEL_B, gen), parents, e, (int32_t)top_b,
                                 per_block, reinterpret_cast<Rec*>(scratch), elites, done);
}

// ---------------------------------------------------------------------------------------------
// Uniform crossover + uniform mutation, fused: one warp per pair of children.  Lane l handles the
// int4 at genes 4l..4l+3 of every block of 128 genes: two parent loads, one Philox call (counter =
// (int4 index, even child's row, generation, stream); each of its four words serves one job of both
// children), two child stores.  Warps past the last pair copy the elites to rows 0..E-1.
// ---------------------------------------------------------------------------------------------
// One random word W per job and pair of sibling children: low half = the even child's mutation
// field, high half = the odd child's, bit 0 = which child inherits the first parent's gene.  A child
// mutates when its field is below thr16, i.e. when the word with that field in its top half is below
// thr32 = thr16 << 16 (ALWAYS stands for thr16 = 65536).  Its new value uses the fraction
// (other field + own field * M) mod 2^16, placed in the top half by one multiply; the other child's
// field is uniform and independent of this child's decision, so the fraction is uniform.
template <bool ALWAYS>
__device__ __forceinline__ void sibling_gene(uint32_t W, int32_t a, int32_t b, int32_t kmin, int32_t range,
                                             uint32_t thr32, bool has1, int32_t& c0, int32_t& c1) {
    const bool flip = (W & 1u) != 0u;
    const uint32_t R = __funnelshift_l(W, W, 16);  // halves swapped: even child's field on top
    c0 = flip ? b : a;
    c1 = flip ? a : b;
    if (ALWAYS || R < thr32) c0 = draw_gene(W * 0x9E360001u, kmin, range);
    if (has1 && (ALWAYS || W < thr32)) c1 = draw_gene(R * 0x85EB0001u, kmin, range);
}

template <bool ALWAYS>
__device__ __forceinline__ void sibling_int4(const uint4 W, const int4 a, const int4 b, const int4 kmin,
                                             const int4 range, uint32_t thr32, bool has1, int4& c0, int4& c1) {
    sibling_gene<ALWAYS>(W.x, a.x, b.x, kmin.x, range.x, thr32, has1, c0.x, c1.x);
    sibling_gene<ALWAYS>(W.y, a.y, b.y, kmin.y, range.y, thr32, has1, c0.y, c1.y);
    sibling_gene<ALWAYS>(W.z, a.z, b.z, kmin.z, range.z, thr32, has1, c0.z, c1.z);
    sibling_gene<ALWAYS>(W.w, a.w, b.w, kmin.w, range.w, thr32, has1, c0.w, c1.w);
}

// Parent rows are asked to stay in L2 (tournament winners are read again by other pairs within the generation)
// and child rows are written as streaming data, so that the 0.5 GB of children do not push the parents out:
// measured 0.1785 -> 0.163 ms per generation at 2048 jobs x 65536 candidates.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ int4 ld_row(const unsigned char* p) {
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ int4 ld_row_hint(const unsigned char* p, uint64_t policy) {
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.s32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(policy));
    return v;
}
template <int UNROLL, bool ALWAYS, int MINB = 4>
__global__ void __launch_bounds__(256, MINB)
k_evolve(const int32_t* __restrict__ src, int32_t* __restrict__ dst, int64_t ld, int32_t n, int32_t n_jobs,
         int32_t elitism, int32_t pairs, const int32_t* __restrict__ parents, const int32_t* __restrict__ elites,
         Tables t, RoundKeys keys, uint32_t gen_lo, uint32_t c3, uint32_t thr32) {
    const int lane = threadIdx.x & 31;
    const uint64_t keep = l2_policy_evict_last();
    const int32_t warps_per_block = blockDim.x >> 5;
    const int64_t total_warps = (int64_t)gridDim.x * warps_per_block;
    const int32_t nvec = (int32_t)(ld >> 2);
    const int4* __restrict__ kminv = reinterpret_cast<const int4*>(t.kmin);
    const int4* __restrict__ rangev = reinterpret_cast<const int4*>(t.range);

    for (int64_t w = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); w < (int64_t)pairs + elitism;
         w += total_warps) {
        if (w >= pairs) {  // survivor: copy unchanged
            const int32_t r = (int32_t)(w - pairs);
            const int4* from = reinterpret_cast<const int4*>(src + (int64_t)elites[r] * ld);
            int4* to = reinterpret_cast<int4*>(dst + (int64_t)r * ld);
            for (int32_t v = lane; v < nvec; v += 32) to[v] = from[v];
            continue;
        }
        const int32_t q = (int32_t)w;
        const int32_t pa = parents[2 * q], pb = parents[2 * q + 1];
        const int32_t slot0 = elitism + 2 * q, slot1 = slot0 + 1;
        const bool has1 = slot1 < n;
        const int4* A = reinterpret_cast<const int4*>(src + (int64_t)pa * ld);
        const int4* B = reinterpret_cast<const int4*>(src + (int64_t)pb * ld);
        int4* C0 = reinterpret_cast<int4*>(dst + (int64_t)slot0 * ld);
        int4* C1 = reinterpret_cast<int4*>(dst + (int64_t)slot1 * ld);
        for (int32_t v0 = 0; v0 < nvec; v0 += 32 * UNROLL) {
            int4 a[UNROLL], b[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int32_t v = v0 + u * 32 + lane;
                if (v < nvec) {
                    a[u] = ld_row_hint(reinterpret_cast<const unsigned char*>(A + v), keep);
                    b[u] = ld_row_hint(reinterpret_cast<const unsigned char*>(B + v), keep);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int32_t v = v0 + u * 32 + lane;
                if (v < nvec) {
                    const int4 kmin = kminv[v];
                    const int4 range = rangev[v];
                    const uint4 W = philox((uint32_t)v, (uint32_t)slot0, gen_lo, c3, keys);
                    int4 c0, c1;
                    sibling_int4<ALWAYS>(W, a[u], b[u], kmin, range, thr32, has1, c0, c1);
                    __stcs(C0 + v, c0);
                    if (has1) __stcs(C1 + v, c1);
                }
            }
        }
    }
}

#ifndef ONES_EV_UNROLL
#define ONES_EV_UNROLL 2
#endif
cudaError_t launch_evolve(const int32_t* src, int32_t* dst, int64_t ld, int32_t n, int32_t n_jobs,
                          int32_t elitism, int32_t pairs, const int32_t* parents, const int32_t* elites,
                          Tables t, RoundKeys keys, uint64_t gen, uint32_t thr16, cudaStream_t s) {
    const int64_t warps = (int64_t)pairs + elitism;
    if (warps <= 0) return cudaSuccess;
    // one warp per pair, no grid-stride: measured faster than a persistent grid at population 65536
    int64_t blocks = (warps + 7) / 8;
    if (blocks > 0x7FFFFFFF) blocks = 0x7FFFFFFF;
    const uint32_t thr32 = thr16 >= 65536u ? 0xFFFFFFFFu : thr16 << 16;
    if (thr16 >= 65536u)
        k_evolve<ONES_EV_UNROLL, true><<<(int)blocks, 256, 0, s>>>(src, dst, ld, n, n_jobs, elitism, pairs, parents, elites, t, keys,
                                                      (uint32_t)gen, counter3(STREAM_MUT, gen), thr32);
    else
        k_evolve<ONES_EV_UNROLL, false><<<(int)blocks, 256, 0, s>>>(src, dst, ld, n, n_jobs, elitism, pairs, parents, elites, t, keys,
                                                       (uint32_t)gen, counter3(STREAM_MUT, gen), thr32);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Crossover + mutation + scoring in one pass: as k_evolve, and each child is scored from registers
// while it is written, so the new population is not read back for its fitness.  One persistent CTA
// per SM holds the model tables (and the per-job ranges, packed to bytes) in shared memory; a warp
// takes one pair of children at a time.  Scores are summed in the same fixed order as k_fitness
// (lane l accumulates the genes it owns in increasing job order, then the butterfly), so F and G
// are bit-identical to scoring the written rows afterwards.  Elite rows are copied and re-scored.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void score4(const int4 g, int32_t base, uint32_t kcap, int32_t jpad,
                                       const double* __restrict__ sX, const uint16_t* __restrict__ sG,
                                       double& sum, int32_t& gpus) {
    const int32_t i0 = (int32_t)min((uint32_t)g.x, kcap) * jpad + base;
    const int32_t i1 = (int32_t)min((uint32_t)g.y, kcap) * jpad + base + 32;
    const int32_t i2 = (int32_t)min((uint32_t)g.z, kcap) * jpad + base + 64;
    const int32_t i3 = (int32_t)min((uint32_t)g.w, kcap) * jpad + base + 96;
    sum = __dadd_rn(sum, sX[i0]); gpus += sG[i0];
    sum = __dadd_rn(sum, sX[i1]); gpus += sG[i1];
    sum = __dadd_rn(sum, sX[i2]); gpus += sG[i2];
    sum = __dadd_rn(sum, sX[i3]); gpus += sG[i3];
}

// What the pass is built around (each point measured at 2048 jobs x 65536 candidates):
//   - the 16-bit g planes are stored so that, for each of the four genes of a lane, the 32 lanes of a warp
//     read 32 different 4-byte bank words whatever their exponents: genes 0/1 and 2/3 of a lane share a word
//     (entry position within a plane: block * 128 + (sub >> 1) * 64 + lane * 2 + (sub & 1));
//   - work items (pairs of children, then survivors) are handed out through a counter in global memory after
//     the first round, so a warp whose parents came from DRAM does not hold the others up (a static
//     round-robin costs the same crossover pass 8 %);
//   - the next int4 of both parents (after a pair's last block: the first of the next pair's parents) is in
//     flight while the current one is worked on, the next pair's parent indices are fetched an item ahead, and
//     every fourth block the following four blocks of both parent rows are asked into L2 (asking further ahead
//     only adds DRAM reads: the lines are gone again before they are used);
//   - a child's mutated value is computed without a branch and selected.
// FULL: the row length is a multiple of 128 genes, so no lane ever falls outside a row.
#ifndef ONES_ES_THREADS
#define ONES_ES_THREADS 768  // threads per CTA when there are more items than warps
#endif
#ifndef ONES_ES_L2PF
#define ONES_ES_L2PF 2  // blocks of 128 genes asked into L2 at a time, that far ahead of the loads (0: off)
#endif

__device__ __forceinline__ void l2_prefetch(const unsigned char* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ int32_t g16_pos(int32_t slot) {  // position of table slot `slot` inside a 16-bit g plane
    return (slot & ~127) + ((slot >> 6) & 1) * 64 + (slot & 31) * 2 + ((slot >> 5) & 1);
}

// c = mutate ? kmin + hi32(frac * range) : c, with mutate = key < thr32 (or always)
template <bool ALWAYS>
__device__ __forceinline__ void mutate_gene(int32_t& c, uint32_t key, uint32_t thr32, uint32_t frac, int32_t range,
                                            int32_t kmin) {
    const int32_t m = kmin + (int32_t)__umulhi(frac, (uint32_t)range);
    c = (ALWAYS || key < thr32) ? m : c;
}

template <bool ALWAYS>
__device__ __forceinline__ void sibling_pair(uint32_t W, int32_t a, int32_t b, int32_t kmin, int32_t range,
                                             uint32_t thr32, int32_t& c0, int32_t& c1) {
    const bool flip = (W & 1u) != 0u;
    const uint32_t R = __funnelshift_l(W, W, 16);  // halves swapped: even child's field on top
    c0 = flip ? b : a;
    c1 = flip ? a : b;
    mutate_gene<ALWAYS>(c0, R, thr32, W * 0x9E360001u, range, kmin);
    mutate_gene<ALWAYS>(c1, W, thr32, R * 0x85EB0001u, range, kmin);
}

// One gene's table look-ups: xrow/grow point at the lane's entries of this gene in plane 0, strideX/strideG
// are the plane strides in bytes.
// CLAMP = false: the caller knows that every gene lies in [0, k1] (a population whose genes are inside their jobs'
// limits), so the gene itself is the plane.
template <bool CLAMP = true>
__device__ __forceinline__ void score_gene(int32_t k, uint32_t kcap, uint32_t strideX, uint32_t strideG,
                                           const unsigned char* __restrict__ xrow, const unsigned char* __restrict__ grow,
                                           double& sum, int32_t& gpus) {
    const uint32_t p = CLAMP ? min((uint32_t)k, kcap) : (uint32_t)k;
    sum = __dadd_rn(sum, *reinterpret_cast<const double*>(xrow + p * strideX));
    gpus += *reinterpret_cast<const uint16_t*>(grow + p * strideG);
}

template <bool CLAMP = true>
__device__ __forceinline__ void score_int4(const int4 g, uint32_t kcap, uint32_t strideX, uint32_t strideG,
                                           const unsigned char* __restrict__ xrow, const unsigned char* __restrict__ grow,
                                           double& sum, int32_t& gpus) {
    score_gene<CLAMP>(g.x, kcap, strideX, strideG, xrow, grow, sum, gpus);
    score_gene<CLAMP>(g.y, kcap, strideX, strideG, xrow + 256, grow + 2, sum, gpus);
    score_gene<CLAMP>(g.z, kcap, strideX, strideG, xrow + 512, grow + 128, sum, gpus);
    score_gene<CLAMP>(g.w, kcap, strideX, strideG, xrow + 768, grow + 130, sum, gpus);
}

// Shared memory: X planes (fp64), g planes narrowed to 16 bits (the host checks that every GPU count
// fits), kmin and range per job (int32).  `work` is the item counter: zero at launch (the selection stage
// clears it), it ends above the number of items.
template <int THREADS, bool ALWAYS, bool FULL, bool CLAMP>
__global__ void __launch_bounds__(THREADS, 1)
k_evolve_score(const int32_t* __restrict__ src, int32_t* __restrict__ dst, int64_t ld, int32_t n, int32_t n_jobs,
               int32_t elitism, int32_t pairs, const int32_t* __restrict__ parents,
               const int32_t* __restrict__ elites, Tables t, RoundKeys keys, uint32_t gen_lo, uint32_t c3,
               uint32_t thr32, int32_t capacity, double penalty, double* __restrict__ F, int32_t* __restrict__ G,
               unsigned int* __restrict__ work) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int32_t planes = t.k1 + 1;
    const int32_t jpad = t.jpad;
    unsigned char* sX = smem_raw;
    unsigned char* sG = smem_raw + (size_t)planes * jpad * 8;
    const int4* sKmin = reinterpret_cast<const int4*>(smem_raw + (size_t)planes * jpad * 10);
    const int4* sRange = sKmin + jpad / 4;
    {
        const int32_t nX = planes * jpad / 2, nG = planes * jpad / 4;
        const int4* gX = reinterpret_cast<const int4*>(t.X);
        const int4* gG = reinterpret_cast<const int4*>(t.G);
        for (int32_t i = threadIdx.x; i < nX; i += blockDim.x) reinterpret_cast<int4*>(sX)[i] = gX[i];
        for (int32_t i = threadIdx.x; i < nG; i += blockDim.x) {
            const int4 g = gG[i];  // slots 4i..4i+3 of one plane: same block and gene, four neighbouring lanes
            const int32_t plane = (4 * i) / jpad, slot = (4 * i) % jpad;
            uint16_t* to = reinterpret_cast<uint16_t*>(sG) + plane * jpad + g16_pos(slot);
            to[0] = (uint16_t)g.x;
            to[2] = (uint16_t)g.y;
            to[4] = (uint16_t)g.z;
            to[6] = (uint16_t)g.w;
        }
        for (int32_t i = threadIdx.x; i < jpad / 4; i += blockDim.x) {
            const_cast<int4*>(sKmin)[i] = reinterpret_cast<const int4*>(t.kmin)[i];
            const_cast<int4*>(sRange)[i] = reinterpret_cast<const int4*>(t.range)[i];
        }
        __syncthreads();
    }
    // parents and elites come from the selection stage, the rows from the generation before.  No early
    // release here: the next selection stage's CTAs would take SMs as they free up and the tail of this
    // kernel measured 3 % slower at the largest population.
    grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = THREADS >> 5;
    const int32_t total_warps = (int32_t)gridDim.x * warps_per_block;
    const int32_t nvec = (int32_t)(ld >> 2);
    const int32_t nblk = (nvec + 31) >> 5;
    const uint32_t kcap = (uint32_t)t.k1;
    const uint32_t strideX = (uint32_t)jpad * 8u, strideG = (uint32_t)jpad * 2u;
    const int64_t row_bytes = ld * 4;
    const unsigned char* srcb = reinterpret_cast<const unsigned char*>(src) + lane * 16;
    unsigned char* dstb = reinterpret_cast<unsigned char*>(dst) + lane * 16;
    const unsigned char* xlane = sX + lane * 8;
    const unsigned char* glane = sG + lane * 4;
    const int2* pp = reinterpret_cast<const int2*>(parents);
    const bool row_lane = FULL || lane < nvec;  // a lane past a short row's end never loads in block 0
    const uint64_t keep = l2_policy_evict_last();
    auto ldp = [&](const unsigned char* p) { return ld_row_hint(p, keep); };
    auto stc = [&](unsigned char* p, const int4 v) { __stcs(reinterpret_cast<int4*>(p), v); };
    // Items [0, pairs) are pairs of children, [pairs, pairs + elitism) survivors.  A warp's first item is its own
    // number; when there are more items than warps, every later one comes from the counter: lane 0 asks for a
    // ticket an item ahead and the warp reads it (one shuffle) half-way through the item it is working on, in
    // time to fetch the next pair's parent indices before that pair's first loads.
    const int32_t items = pairs + elitism;
    const bool dynamic = items > total_warps;
    unsigned int ticket = 0;
    auto ask = [&]() {
        if (dynamic && lane == 0) ticket = atomicAdd(work, 1u);
    };
    auto take = [&]() { return dynamic ? total_warps + (int32_t)__shfl_sync(0xFFFFFFFFu, ticket, 0) : items; };
    int32_t w = (int32_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    ask();
    int2 par = make_int2(0, 0);
    int4 a0 = make_int4(0, 0, 0, 0), b0 = a0, a1 = a0, b1 = a0;
    if (w < pairs) {
        par = pp[w];
        if (row_lane) {
            a0 = ldp(srcb + par.x * row_bytes);
            b0 = ldp(srcb + par.y * row_bytes);
        }
    }
    // One step = one int4 of each parent -> one int4 of each child, scored.
    auto step = [&](const int32_t blk, const int32_t slot0, const bool has1, unsigned char* __restrict__ C,
                    const int4& cura, const int4& curb, double& sum0, double& sum1, int32_t& gp0, int32_t& gp1) {
        const int32_t v = blk * 32 + lane;
        if (FULL || v < nvec) {
            const int4 kmin = sKmin[v];
            const int4 range = sRange[v];
            const uint4 W = philox((uint32_t)v, (uint32_t)slot0, gen_lo, c3, keys);
            int4 c0, c1;
            sibling_pair<ALWAYS>(W.x, cura.x, curb.x, kmin.x, range.x, thr32, c0.x, c1.x);
            sibling_pair<ALWAYS>(W.y, cura.y, curb.y, kmin.y, range.y, thr32, c0.y, c1.y);
            sibling_pair<ALWAYS>(W.z, cura.z, curb.z, kmin.z, range.z, thr32, c0.z, c1.z);
            sibling_pair<ALWAYS>(W.w, cura.w, curb.w, kmin.w, range.w, thr32, c0.w, c1.w);
            unsigned char* to = C + blk * 512;
            stc(to, c0);
            if (has1) stc(to + row_bytes, c1);
            const unsigned char* xrow = xlane + blk * 1024;
            const unsigned char* grow = glane + blk * 256;
            score_int4<CLAMP>(c0, kcap, strideX, strideG, xrow, grow, sum0, gp0);
            score_int4<CLAMP>(c1, kcap, strideX, strideG, xrow, grow, sum1, gp1);
        }
    };
    const int32_t take_at = (nblk / 2) & ~1;  // the block (even) at which the next item's number is read
    while (w < pairs) {
        const unsigned char* A = srcb + par.x * row_bytes;
        const unsigned char* B = srcb + par.y * row_bytes;
        const int32_t slot0 = elitism + 2 * w;
        const bool has1 = slot0 + 1 < n;
        unsigned char* C = dstb + slot0 * row_bytes;
        int32_t w_next = items;
        bool more = false;
        double sum0 = 0.0, sum1 = 0.0;
        int32_t gp0 = 0, gp1 = 0;
        // Fetch block `nb` of this pair's parents, or (after the last block) block 0 of the next pair's.
        auto fetch = [&](const int32_t nb, int4& na, int4& nb4) {
            na = make_int4(0, 0, 0, 0);
            nb4 = na;
            if (nb < nblk) {
                if (FULL || nb * 32 + lane < nvec) {
                    na = ldp(A + nb * 512);
                    nb4 = ldp(B + nb * 512);
                }
#if ONES_ES_L2PF > 0
                if ((nb % ONES_ES_L2PF) == 0 && nb + ONES_ES_L2PF < nblk) {
#pragma unroll
                    for (int d = 0; d < ONES_ES_L2PF; ++d) {
                        if (nb + ONES_ES_L2PF + d < nblk) {
                            l2_prefetch(A + (nb + ONES_ES_L2PF + d) * 512);
                            l2_prefetch(B + (nb + ONES_ES_L2PF + d) * 512);
                        }
                    }
                }
#endif
            } else if (more && row_lane) {
                na = ldp(srcb + par.x * row_bytes);
                nb4 = ldp(srcb + par.y * row_bytes);
            }
        };
        for (int32_t blk = 0; blk < nblk; blk += 2) {
            if (blk == take_at) {
                w_next = take();
                ask();
                more = w_next < pairs;
                if (more) par = pp[w_next];  // A and B keep this pair's rows
            }
            fetch(blk + 1, a1, b1);
            step(blk, slot0, has1, C, a0, b0, sum0, sum1, gp0, gp1);
            if (blk + 1 < nblk) {
                fetch(blk + 2, a0, b0);
                step(blk + 1, slot0, has1, C, a1, b1, sum0, sum1, gp0, gp1);
            } else {  // odd number of blocks: the next pair's first block sits in the other buffer
                a0 = a1;
                b0 = b1;
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum0 = __dadd_rn(sum0, __shfl_xor_sync(0xFFFFFFFFu, sum0, off));
            gp0 += __shfl_xor_sync(0xFFFFFFFFu, gp0, off);
            sum1 = __dadd_rn(sum1, __shfl_xor_sync(0xFFFFFFFFu, sum1, off));
            gp1 += __shfl_xor_sync(0xFFFFFFFFu, gp1, off);
        }
        if (lane == 0) {
            const int32_t over0 = gp0 > capacity ? gp0 - capacity : 0;
            F[slot0] = __dsub_rn(sum0, __dmul_rn(penalty, (double)over0));
            G[slot0] = gp0;
            if (has1) {
                const int32_t over1 = gp1 > capacity ? gp1 - capacity : 0;
                F[slot0 + 1] = __dsub_rn(sum1, __dmul_rn(penalty, (double)over1));
                G[slot0 + 1] = gp1;
            }
        }
        w = w_next;
    }
    // ---- survivors: copied unchanged and scored again ----
    while (w < items) {
        const int32_t w_next = take();
        ask();
        const int32_t r = w - pairs;
        const unsigned char* from = srcb + elites[r] * row_bytes;
        unsigned char* to = dstb + r * row_bytes;
        double sum = 0.0;
        int32_t gp = 0;
        for (int32_t blk = 0; blk < nblk; ++blk) {
            if (FULL || blk * 32 + lane < nvec) {
                const int4 g = *reinterpret_cast<const int4*>(from + blk * 512);
                *reinterpret_cast<int4*>(to + blk * 512) = g;
                score_int4<CLAMP>(g, kcap, strideX, strideG, xlane + blk * 1024, glane + blk * 256, sum, gp);
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
            gp += __shfl_xor_sync(0xFFFFFFFFu, gp, off);
        }
        if (lane == 0) {
            const int32_t over = gp > capacity ? gp - capacity : 0;
            F[r] = __dsub_rn(sum, __dmul_rn(penalty, (double)over));
            G[r] = gp;
        }
        w = w_next;
    }
}

// ---------------------------------------------------------------------------------------------
// The same pass on packed candidates (one byte per gene, tiles of 512 genes, see k_pack_rows): parents read and
// children written as bytes, 2 bytes of HBM traffic per child gene instead of 8.  One 16-byte load gives a lane
// the genes 4l..4l+3 of four consecutive 128-gene blocks; each of its four words is one block's int4 of the
// int32 rows, so the random words (one Philox call per block and lane, counter = the int4's index), the
// operators and the fixed summation order are those of k_evolve_score and the children equal the packed
// int32 children byte for byte.  Crossover takes the four genes of a word at once (a byte mask from bit 0 of
// the four random words); a mutated gene is inserted into its byte.  A parent byte of 0xFF (the job waits) is
// inherited as it is.  Work items and shared-memory tables as in k_evolve_score.
// ---------------------------------------------------------------------------------------------
template <bool ALWAYS>
__device__ __forceinline__ void mutate_byte(uint32_t& word, int s, uint32_t key, uint32_t thr32, uint32_t frac,
                                            int32_t range, int32_t kmin) {
    const uint32_t m = (uint32_t)(kmin + (int32_t)__umulhi(frac, (uint32_t)range));
    const uint32_t with = (word & ~(0xFFu << (8 * s))) | (m << (8 * s));
    word = (ALWAYS || key < thr32) ? with : word;
}

__device__ __forceinline__ void score_word(uint32_t w, uint32_t kcap, uint32_t strideX, uint32_t strideG,
                                           const unsigned char* __restrict__ xrow, const unsigned char* __restrict__ grow,
                                           double& sum, int32_t& gpus) {
    score_gene((int32_t)(w & 0xFFu), kcap, strideX, strideG, xrow, grow, sum, gpus);
    score_gene((int32_t)((w >> 8) & 0xFFu), kcap, strideX, strideG, xrow + 256, grow + 2, sum, gpus);
    score_gene((int32_t)((w >> 16) & 0xFFu), kcap, strideX, strideG, xrow + 512, grow + 128, sum, gpus);
    score_gene((int32_t)(w >> 24), kcap, strideX, strideG, xrow + 768, grow + 130, sum, gpus);
}

template <int THREADS, bool ALWAYS>
__global__ void __launch_bounds__(THREADS, 1)
k_evolve_score_packed(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int64_t ld8, int32_t n,
                      int32_t n_jobs, int32_t elitism, int32_t pairs, const int32_t* __restrict__ parents,
                      const int32_t* __restrict__ elites, Tables t, RoundKeys keys, uint32_t gen_lo, uint32_t c3,
                      uint32_t thr32, int32_t capacity, double penalty, double* __restrict__ F, int32_t* __restrict__ G,
                      unsigned int* __restrict__ work) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int32_t planes = t.k1 + 1;
    const int32_t jpad = t.jpad;
    unsigned char* sX = smem_raw;
    unsigned char* sG = smem_raw + (size_t)planes * jpad * 8;
    const int4* sKmin = reinterpret_cast<const int4*>(smem_raw + (size_t)planes * jpad * 10);
    const int4* sRange = sKmin + jpad / 4;
    {
        const int32_t nX = planes * jpad / 2, nG = planes * jpad / 4;
        const int4* gX = reinterpret_cast<const int4*>(t.X);
        const int4* gG = reinterpret_cast<const int4*>(t.G);
        for (int32_t i = threadIdx.x; i < nX; i += blockDim.x) reinterpret_cast<int4*>(sX)[i] = gX[i];
        for (int32_t i = threadIdx.x; i < nG; i += blockDim.x) {
            const int4 g = gG[i];
            const int32_t plane = (4 * i) / jpad, slot = (4 * i) % jpad;
            uint16_t* to = reinterpret_cast<uint16_t*>(sG) + plane * jpad + g16_pos(slot);
            to[0] = (uint16_t)g.x;
            to[2] = (uint16_t)g.y;
            to[4] = (uint16_t)g.z;
            to[6] = (uint16_t)g.w;
        }
        for (int32_t i = threadIdx.x; i < jpad / 4; i += blockDim.x) {
            int4 lo = reinterpret_cast<const int4*>(t.kmin)[i];
            // columns past the last job keep their 0xFF through a redraw (range 1, lower limit 255)
            if (4 * i >= n_jobs) lo.x = 255;
            if (4 * i + 1 >= n_jobs) lo.y = 255;
            if (4 * i + 2 >= n_jobs) lo.z = 255;
            if (4 * i + 3 >= n_jobs) lo.w = 255;
            const_cast<int4*>(sKmin)[i] = lo;
            const_cast<int4*>(sRange)[i] = reinterpret_cast<const int4*>(t.range)[i];
        }
        __syncthreads();
    }
    grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = THREADS >> 5;
    const int32_t total_warps = (int32_t)gridDim.x * warps_per_block;
    const int32_t tiles = (int32_t)(ld8 >> 9);
    const int32_t nblk = jpad >> 7;  // blocks of 128 genes that hold jobs; the blocks after them are copied
    const uint32_t kcap = (uint32_t)t.k1;
    const uint32_t strideX = (uint32_t)jpad * 8u, strideG = (uint32_t)jpad * 2u;
    const unsigned char* srcb = src + lane * 16;
    unsigned char* dstb = dst + lane * 16;
    const unsigned char* xlane = sX + lane * 8;
    const unsigned char* glane = sG + lane * 4;
    const int2* pp = reinterpret_cast<const int2*>(parents);

    const int32_t items = pairs + elitism;
    const bool dynamic = items > total_warps;
    unsigned int ticket = 0;
    auto ask = [&]() {
        if (dynamic && lane == 0) ticket = atomicAdd(work, 1u);
    };
    auto take = [&]() { return dynamic ? total_warps + (int32_t)__shfl_sync(0xFFFFFFFFu, ticket, 0) : items; };
    const uint64_t keep = l2_policy_evict_last();
    auto ld_tile = [&](const unsigned char* p) {
        const int4 v = ld_row_hint(p, keep);
        return make_uint4((uint32_t)v.x, (uint32_t)v.y, (uint32_t)v.z, (uint32_t)v.w);
    };
    int32_t w = (int32_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    ask();
    int2 par = make_int2(0, 0);
    uint4 qa = make_uint4(0, 0, 0, 0), qb = qa;
    if (w < pairs) {
        par = pp[w];
        qa = ld_tile(srcb + par.x * ld8);
        qb = ld_tile(srcb + par.y * ld8);
    }
    const int32_t take_at = tiles / 2;
    while (w < pairs) {
        const unsigned char* A = srcb + par.x * ld8;
        const unsigned char* B = srcb + par.y * ld8;
        const uint32_t slot0 = (uint32_t)(elitism + 2 * w);
        const bool has1 = (int32_t)slot0 + 1 < n;
        unsigned char* C = dstb + slot0 * ld8;
        int32_t w_next = items;
        bool more = false;
        double sum0 = 0.0, sum1 = 0.0;
        int32_t gp0 = 0, gp1 = 0;
        for (int32_t tile = 0; tile < tiles; ++tile) {
            if (tile == take_at) {
                w_next = take();
                ask();
                more = w_next < pairs;
                if (more) par = pp[w_next];  // A and B keep this pair's rows
            }
            // the next tile of both parents (after the last tile: the first of the next pair's) while this one is worked on
            uint4 na = make_uint4(0, 0, 0, 0), nb = na;
            if (tile + 1 < tiles) {
                na = ld_tile(A + (tile + 1) * 512);
                nb = ld_tile(B + (tile + 1) * 512);
            } else if (more) {
                na = ld_tile(srcb + par.x * ld8);
                nb = ld_tile(srcb + par.y * ld8);
            }
            const uint32_t aw[4] = {qa.x, qa.y, qa.z, qa.w}, bw[4] = {qb.x, qb.y, qb.z, qb.w};
            uint32_t c0w[4], c1w[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int32_t blk = tile * 4 + b;
                c0w[b] = aw[b];
                c1w[b] = bw[b];
                if (blk < nblk) {  // warp-uniform
                    const int32_t v = blk * 32 + lane;
                    const int4 kmin = sKmin[v];
                    const int4 range = sRange[v];
                    const uint4 W = philox((uint32_t)v, slot0, gen_lo, c3, keys);
                    // byte s of the even child comes from the second parent where bit 0 of random word s is set
                    const uint32_t flips = (W.x & 1u) | ((W.y & 1u) << 8) | ((W.z & 1u) << 16) | ((W.w & 1u) << 24);
                    const uint32_t m = flips * 0xFFu;
                    c0w[b] = (aw[b] & ~m) | (bw[b] & m);
                    c1w[b] = (bw[b] & ~m) | (aw[b] & m);
                    const uint32_t Ws[4] = {W.x, W.y, W.z, W.w};
                    const int32_t kmins[4] = {kmin.x, kmin.y, kmin.z, kmin.w}, ranges[4] = {range.x, range.y, range.z, range.w};
#pragma unroll
                    for (int s4 = 0; s4 < 4; ++s4) {
                        const uint32_t R = __funnelshift_l(Ws[s4], Ws[s4], 16);  // halves swapped: even child's field on top
                        mutate_byte<ALWAYS>(c0w[b], s4, R, thr32, Ws[s4] * 0x9E360001u, ranges[s4], kmins[s4]);
                        mutate_byte<ALWAYS>(c1w[b], s4, Ws[s4], thr32, R * 0x85EB0001u, ranges[s4], kmins[s4]);
                    }
                    const unsigned char* xrow = xlane + blk * 1024;
                    const unsigned char* grow = glane + blk * 256;
                    score_word(c0w[b], kcap, strideX, strideG, xrow, grow, sum0, gp0);
                    score_word(c1w[b], kcap, strideX, strideG, xrow, grow, sum1, gp1);
                }
            }
            unsigned char* to = C + tile * 512;
            __stcs(reinterpret_cast<uint4*>(to), make_uint4(c0w[0], c0w[1], c0w[2], c0w[3]));
            if (has1) __stcs(reinterpret_cast<uint4*>(to + ld8), make_uint4(c1w[0], c1w[1], c1w[2], c1w[3]));
            qa = na;
            qb = nb;
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum0 = __dadd_rn(sum0, __shfl_xor_sync(0xFFFFFFFFu, sum0, off));
            gp0 += __shfl_xor_sync(0xFFFFFFFFu, gp0, off);
            sum1 = __dadd_rn(sum1, __shfl_xor_sync(0xFFFFFFFFu, sum1, off));
            gp1 += __shfl_xor_sync(0xFFFFFFFFu, gp1, off);
        }
        if (lane == 0) {
            const int32_t over0 = gp0 > capacity ? gp0 - capacity : 0;
            F[slot0] = __dsub_rn(sum0, __dmul_rn(penalty, (double)over0));
            G[slot0] = gp0;
            if (has1) {
                const int32_t over1 = gp1 > capacity ? gp1 - capacity : 0;
                F[slot0 + 1] = __dsub_rn(sum1, __dmul_rn(penalty, (double)over1));
                G[slot0 + 1] = gp1;
            }
        }
        w = w_next;
    }
    // ---- survivors: copied unchanged and scored again ----
    while (w < items) {
        const int32_t w_next = take();
        ask();
        const int32_t r = w - pairs;
        const unsigned char* from = srcb + elites[r] * ld8;
        unsigned char* to = dstb + r * ld8;
        double sum = 0.0;
        int32_t gp = 0;
        for (int32_t tile = 0; tile < tiles; ++tile) {
            const uint4 q = *reinterpret_cast<const uint4*>(from + tile * 512);
            *reinterpret_cast<uint4*>(to + tile * 512) = q;
            const uint32_t qw[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int32_t blk = tile * 4 + b;
                if (blk < nblk) score_word(qw[b], kcap, strideX, strideG, xlane + blk * 1024, glane + blk * 256, sum, gp);
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
            gp += __shfl_xor_sync(0xFFFFFFFFu, gp, off);
        }
        if (lane == 0) {
            const int32_t over = gp > capacity ? gp - capacity : 0;
            F[r] = __dsub_rn(sum, __dmul_rn(penalty, (double)over));
            G[r] = gp;
        }
        w = w_next;
    }
}

cudaError_t launch_evolve_score_packed(const uint8_t* src, uint8_t* dst, int64_t ld8, int32_t n, int32_t n_jobs, int32_t elitism,
                                       int32_t pairs, const int32_t* parents, const int32_t* elites, Tables t,
                                       RoundKeys keys, uint64_t gen, uint32_t thr16, int32_t capacity, double penalty,
                                       double* F, int32_t* G, unsigned int* work, cudaStream_t s) {
    const int64_t warps = (int64_t)pairs + elitism;
    if (warps <= 0) return cudaSuccess;
    const size_t smem = evolve_score_smem(t);
    if (smem > (size_t)kMaxSmemPerBlock) return cudaErrorInvalidConfiguration;
    const uint32_t thr32 = thr16 >= 65536u ? 0xFFFFFFFFu : thr16 << 16;
    constexpr int kThreads = 1024;
    int64_t blocks = (warps + kThreads / 32 - 1) / (kThreads / 32);
    if (blocks > sm_count()) blocks = sm_count();
    auto kern = thr16 >= 65536u ? k_evolve_score_packed<kThreads, true> : k_evolve_score_packed<kThreads, false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemPerBlock);
    if (e != cudaSuccess) return e;
    return launch_after_previous(kern, (int)blocks, kThreads, smem, s, src, dst, ld8, n, n_jobs, elitism, pairs, parents, elites, t,
                                 keys, (uint32_t)gen, counter3(STREAM_MUT, gen), thr32, capacity, penalty, F, G, work);
}

// ---------------------------------------------------------------------------------------------
// Warm start across a changed job set, scored in the same pass: as k_remap (column j of the new row is
// column remap[j] of the old one clamped into the new limits, or the lower limit for a new job), one warp
// per candidate, the new row scored from registers in the fixed order while it is written.  One persistent
// CTA per SM with the new model tables, limits and the column map in shared memory.  A lane whose four
// columns come from four neighbouring old columns at the same place takes them as one int4.
// ---------------------------------------------------------------------------------------------
// shared memory: X planes (fp64), g planes (16 bits), column map (int32), limits as two bytes per job, one
// "same four columns" flag per int4
size_t remap_score_smem(Tables t) { return (size_t)(t.k1 + 1) * t.jpad * 10 + (size_t)t.jpad * 4 + (size_t)t.jpad * 2 + (size_t)t.jpad / 4; }

__global__ void __launch_bounds__(1024, 1)
k_remap_score(const int32_t* __restrict__ src, int64_t ld_src, int32_t* __restrict__ dst, int64_t ld_dst, int32_t n,
              int32_t n_jobs_new, const int32_t* __restrict__ remap, Tables t, int32_t capacity, double penalty,
              double* __restrict__ F, int32_t* __restrict__ G) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int32_t planes = t.k1 + 1;
    const int32_t jpad = t.jpad;
    double* sX = reinterpret_cast<double*>(smem_raw);
    uint16_t* sG = reinterpret_cast<uint16_t*>(smem_raw + (size_t)planes * jpad * 8);
    int4* sFrom = reinterpret_cast<int4*>(smem_raw + (size_t)planes * jpad * 10);
    uint2* sLim = reinterpret_cast<uint2*>(sFrom + jpad / 4);  // per job: lower limit | upper limit << 8 (both <= 15)
    uint8_t* sSame = reinterpret_cast<uint8_t*>(sLim + jpad / 4);  // per int4: its columns are the same four old columns
    {
        const int32_t nX = planes * jpad / 2, nG = planes * jpad / 4;
        const int4* gX = reinterpret_cast<const int4*>(t.X);
        const int4* gG = reinterpret_cast<const int4*>(t.G);
        for (int32_t i = threadIdx.x; i < nX; i += blockDim.x) reinterpret_cast<int4*>(sX)[i] = gX[i];
        for (int32_t i = threadIdx.x; i < nG; i += blockDim.x) {
            const int4 g = gG[i];
            reinterpret_cast<uint2*>(sG)[i] = make_uint2((uint32_t)g.x | ((uint32_t)g.y << 16),
                                                         (uint32_t)g.z | ((uint32_t)g.w << 16));
        }
        // padding columns: no source, limits [0, 0] (k_build_tables), so they come out as 0
        for (int32_t v = threadIdx.x; v < jpad / 4; v += blockDim.x) {
            int32_t from[4];
            uint32_t lim[4];
            bool same = true;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int32_t j = 4 * v + c;
                from[c] = j < n_jobs_new ? remap[j] : -1;
                const int32_t lo = t.kmin[j];
                lim[c] = (uint32_t)lo | ((uint32_t)(lo + t.range[j] - 1) << 8);
                same = same && from[c] == j;
            }
            sFrom[v] = make_int4(from[0], from[1], from[2], from[3]);
            sLim[v] = make_uint2(lim[0] | (lim[1] << 16), lim[2] | (lim[3] << 16));
            sSame[v] = same ? 1 : 0;
        }
        __syncthreads();
    }
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = blockDim.x >> 5;
    const int64_t total_warps = (int64_t)gridDim.x * warps_per_block;
    const int32_t nvec = (int32_t)(ld_dst >> 2);
    const uint32_t kcap = (uint32_t)t.k1;
    for (int64_t row = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); row < n; row += total_warps) {
        const int32_t* old_row = src + row * ld_src;
        int4* new_row = reinterpret_cast<int4*>(dst + row * ld_dst);
        double sum = 0.0;
        int32_t gpus = 0;
        constexpr int UN = 4;  // int4 of the old row in flight per lane
        for (int32_t v0 = lane; v0 < nvec; v0 += 32 * UN) {
            int4 k[UN];
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int32_t v = v0 + 32 * u;
                if (v < nvec) {
                    if (sSame[v]) {
                        k[u] = *reinterpret_cast<const int4*>(old_row + 4 * v);
                    } else {
                        const int4 from = sFrom[v];
                        const int32_t none = -0x7FFFFFFF;  // a new job: the clamp below puts it at its lower limit
                        k[u] = make_int4(none, none, none, none);
                        if (from.x >= 0) k[u].x = old_row[from.x];
                        if (from.y >= 0) k[u].y = old_row[from.y];
                        if (from.z >= 0) k[u].z = old_row[from.z];
                        if (from.w >= 0) k[u].w = old_row[from.w];
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int32_t v = v0 + 32 * u;
                if (v < nvec) {
                    const uint2 lim = sLim[v];
                    int4 c = k[u];
                    c.x = min(max(c.x, (int32_t)(lim.x & 0xFFu)), (int32_t)((lim.x >> 8) & 0xFFu));
                    c.y = min(max(c.y, (int32_t)((lim.x >> 16) & 0xFFu)), (int32_t)(lim.x >> 24));
                    c.z = min(max(c.z, (int32_t)(lim.y & 0xFFu)), (int32_t)((lim.y >> 8) & 0xFFu));
                    c.w = min(max(c.w, (int32_t)((lim.y >> 16) & 0xFFu)), (int32_t)(lim.y >> 24));
                    new_row[v] = c;
                    score4(c, (v >> 5) * 128 + lane, kcap, jpad, sX, sG, sum, gpus);
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
            gpus += __shfl_xor_sync(0xFFFFFFFFu, gpus, off);
        }
        if (lane == 0) {
            const int32_t over = gpus > capacity ? gpus - capacity : 0;
            F[row] = __dsub_rn(sum, __dmul_rn(penalty, (double)over));
            G[row] = gpus;
        }
    }
}

cudaError_t launch_remap_score(const int32_t* src, int64_t ld_src, int32_t* dst, int64_t ld_dst, int32_t n,
                               int32_t n_jobs_new, const int32_t* remap, Tables t, int32_t capacity, double penalty,
                               double* F, int32_t* G, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const size_t smem = remap_score_smem(t);
    if (smem > (size_t)kMaxSmemPerBlock) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(k_remap_score, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemPerBlock);
    if (e != cudaSuccess) return e;
    int64_t blocks = ((int64_t)n + 31) / 32;
    if (blocks > sm_count()) blocks = sm_count();
    k_remap_score<<<(int)blocks, 1024, smem, s>>>(src, ld_src, dst, ld_dst, n, n_jobs_new, remap, t, capacity, penalty, F, G);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// A whole generation in one launch: each warp runs the two tournaments of its pair (one draw per
// lane, butterfly for the winner), then crossover, mutation and scoring as k_evolve_score, and
// queues the scores it produced in shared memory; at the end every CTA reduces its queue to its e
// best and the last CTA to finish merges those lists into the elites of the NEXT generation.
// F_old is read (tournaments), F_new written: two score buffers.  `done` as in k_select_stage.
// ---------------------------------------------------------------------------------------------
// A tournament in two halves so that the score gathers of the NEXT pair are in flight while the
// current pair's rows are processed: draw (one draw per lane, private best) and reduce (butterfly).
struct Draw {
    int32_t idx;
    double f;
};

__device__ __forceinline__ Draw tournament_draw(const double* __restrict__ F, int32_t n, int32_t tournament, uint32_t q,
                                                uint32_t gen_lo, uint32_t c3, const RoundKeys& keys, int lane) {
    Draw d;
    d.idx = -1;
    d.f = 0.0;
    for (int32_t t0 = 0; t0 < tournament; t0 += 32) {
        const int32_t t = t0 + lane;
        if (t < tournament) {
            const uint4 w4 = philox((uint32_t)(t >> 2), q, gen_lo, c3, keys);
            const uint32_t w = (t & 2) ? ((t & 1) ? w4.w : w4.z) : ((t & 1) ? w4.y : w4.x);
            const int32_t idx = (int32_t)__umulhi(w, (uint32_t)n);
            const double f = F[idx];
            if (d.idx < 0 || f > d.f || (f == d.f && idx < d.idx)) {
                d.idx = idx;
                d.f = f;
            }
        }
    }
    return d;
}

__device__ __forceinline__ int32_t tournament_reduce(Draw d) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const int32_t oi = __shfl_xor_sync(0xFFFFFFFFu, d.idx, off);
        const double of = __shfl_xor_sync(0xFFFFFFFFu, d.f, off);
        if (oi >= 0 && (d.idx < 0 || of > d.f || (of == d.f && oi < d.idx))) {
            d.idx = oi;
            d.f = of;
        }
    }
    return d.idx;
}

template <int THREADS, int UNROLL, bool ALWAYS>
__global__ void __launch_bounds__(THREADS, 1)
k_generation(const int32_t* __restrict__ src, int32_t* __restrict__ dst, int64_t ld, int32_t n, int32_t n_jobs,
             int32_t elitism, int32_t pairs, int32_t tournament, const double* __restrict__ F_old,
             double* __restrict__ F_new, int32_t* __restrict__ G, int32_t* __restrict__ parents,
             const int32_t* __restrict__ elites, int32_t* __restrict__ elites_next, Tables t, RoundKeys keys,
             uint32_t gen_lo, uint32_t c3, uint32_t c3a, uint32_t c3b, uint32_t thr32, int32_t capacity,
             double penalty, Rec* __restrict__ partial, unsigned int* __restrict__ done, int32_t queue_cap) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ Rec s_warp[32];
    __shared__ int s_queued;
    __shared__ bool s_last;
    const int32_t planes = t.k1 + 1;
    const int32_t jpad = t.jpad;
    double* sX = reinterpret_cast<double*>(smem_raw);
    uint16_t* sG = reinterpret_cast<uint16_t*>(smem_raw + (size_t)planes * jpad * 8);
    int4* sKmin = reinterpret_cast<int4*>(smem_raw + (size_t)planes * jpad * 10);
    int4* sRange = sKmin + jpad / 4;
    Rec* queue = reinterpret_cast<Rec*>(smem_raw + (size_t)planes * jpad * 10 + (size_t)jpad * 8);
    {
        if (threadIdx.x == 0) s_queued = 0;
        const int32_t nX = planes * jpad / 2, nG = planes * jpad / 4;
        const int4* gX = reinterpret_cast<const int4*>(t.X);
        const int4* gG = reinterpret_cast<const int4*>(t.G);
        for (int32_t i = threadIdx.x; i < nX; i += blockDim.x) reinterpret_cast<int4*>(sX)[i] = gX[i];
        for (int32_t i = threadIdx.x; i < nG; i += blockDim.x) {
            const int4 g = gG[i];
            reinterpret_cast<uint2*>(sG)[i] = make_uint2((uint32_t)g.x | ((uint32_t)g.y << 16),
                                                         (uint32_t)g.z | ((uint32_t)g.w << 16));
        }
        for (int32_t i = threadIdx.x; i < jpad / 4; i += blockDim.x) {
            sKmin[i] = reinterpret_cast<const int4*>(t.kmin)[i];
            sRange[i] = reinterpret_cast<const int4*>(t.range)[i];
        }
        __syncthreads();
    }
    grid_dependency_wait();  // scores, elites and rows come from the generation before
    grid_dependency_release();  // measured: the next generation's CTAs best become resident as early as they can
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = blockDim.x >> 5;
    const int64_t total_warps = (int64_t)gridDim.x * warps_per_block;
    const int32_t nvec = (int32_t)(ld >> 2);
    const uint32_t kcap = (uint32_t)t.k1;

    const int64_t w_first = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    Draw da, db;
    da.idx = db.idx = -1;
    da.f = db.f = 0.0;
    if (w_first < pairs) {
        da = tournament_draw(F_old, n, tournament, (uint32_t)w_first, gen_lo, c3a, keys, lane);
        db = tournament_draw(F_old, n, tournament, (uint32_t)w_first, gen_lo, c3b, keys, lane);
    }
    for (int64_t w = w_first; w < (int64_t)pairs + elitism; w += total_warps) {
        double sum0 = 0.0, sum1 = 0.0;
        int32_t gp0 = 0, gp1 = 0;
        int32_t slot0, slot1;
        bool has1;
        if (w >= pairs) {  // survivor: copy unchanged and score again
            slot0 = (int32_t)(w - pairs);
            slot1 = slot0;
            has1 = false;
            const int4* from = reinterpret_cast<const int4*>(src + (int64_t)elites[slot0] * ld);
            int4* to = reinterpret_cast<int4*>(dst + (int64_t)slot0 * ld);
            for (int32_t v = lane; v < nvec; v += 32) {
                const int4 g = from[v];
                to[v] = g;
                score4(g, (v >> 5) * 128 + lane, kcap, jpad, sX, sG, sum0, gp0);
            }
        } else {
            const int32_t q = (int32_t)w;
            const int32_t pa = tournament_reduce(da);
            const int32_t pb = tournament_reduce(db);
            if (w + total_warps < pairs) {  // next pair's draws: their score gathers overlap this pair's rows
                da = tournament_draw(F_old, n, tournament, (uint32_t)(w + total_warps), gen_lo, c3a, keys, lane);
                db = tournament_draw(F_old, n, tournament, (uint32_t)(w + total_warps), gen_lo, c3b, keys, lane);
            }
            if (lane == 0) {
                parents[2 * q] = pa;
                parents[2 * q + 1] = pb;
            }
            slot0 = elitism + 2 * q;
            slot1 = slot0 + 1;
            has1 = slot1 < n;
            const int4* A = reinterpret_cast<const int4*>(src + (int64_t)pa * ld);
            const int4* B = reinterpret_cast<const int4*>(src + (int64_t)pb * ld);
            int4* C0 = reinterpret_cast<int4*>(dst + (int64_t)slot0 * ld);
            int4* C1 = reinterpret_cast<int4*>(dst + (int64_t)slot1 * ld);
            for (int32_t v0 = 0; v0 < nvec; v0 += 32 * UNROLL) {
                int4 a[UNROLL], b[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int32_t v = v0 + u * 32 + lane;
                    if (v < nvec) {
                        a[u] = A[v];
                        b[u] = B[v];
                    }
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int32_t v = v0 + u * 32 + lane;
                    if (v < nvec) {
                        const int4 kmin = sKmin[v];
                        const int4 range = sRange[v];
                        const uint4 W = philox((uint32_t)v, (uint32_t)slot0, gen_lo, c3, keys);
                        int4 c0, c1;
                        sibling_int4<ALWAYS>(W, a[u], b[u], kmin, range, thr32, has1, c0, c1);
                        C0[v] = c0;
                        const int32_t base = (v >> 5) * 128 + lane;
                        score4(c0, base, kcap, jpad, sX, sG, sum0, gp0);
                        if (has1) {
                            C1[v] = c1;
                            score4(c1, base, kcap, jpad, sX, sG, sum1, gp1);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum0 = __dadd_rn(sum0, __shfl_xor_sync(0xFFFFFFFFu, sum0, off));
            gp0 += __shfl_xor_sync(0xFFFFFFFFu, gp0, off);
            sum1 = __dadd_rn(sum1, __shfl_xor_sync(0xFFFFFFFFu, sum1, off));
            gp1 += __shfl_xor_sync(0xFFFFFFFFu, gp1, off);
        }
        if (lane == 0) {
            const int32_t over0 = gp0 > capacity ? gp0 - capacity : 0;
            const double f0 = __dsub_rn(sum0, __dmul_rn(penalty, (double)over0));
            F_new[slot0] = f0;
            G[slot0] = gp0;
            int32_t at = elitism > 0 ? atomicAdd(&s_queued, has1 ? 2 : 1) : queue_cap;
            if (at < queue_cap) {
                Rec r;
                r.key = score_key(f0);
                r.idx = slot0;
                r.pad = 0;
                queue[at] = r;
            }
            if (has1) {
                const int32_t over1 = gp1 > capacity ? gp1 - capacity : 0;
                const double f1 = __dsub_rn(sum1, __dmul_rn(penalty, (double)over1));
                F_new[slot1] = f1;
                G[slot1] = gp1;
                if (at + 1 < queue_cap) {
                    Rec r;
                    r.key = score_key(f1);
                    r.idx = slot1;
                    r.pad = 0;
                    queue[at + 1] = r;
                }
            }
        }
    }
    if (elitism <= 0) return;
    // this CTA's e best of what it produced, then the last CTA merges all lists
    __syncthreads();
    const int32_t queued = min(s_queued, queue_cap);
    Rec prev;
    prev.key = 0;
    prev.idx = -1;
    prev.pad = 0;
    for (int32_t r = 0; r < elitism; ++r) {
        Rec best = block_next_best<2>(queue, queued, 0, r > 0, prev, s_warp);
        if (threadIdx.x == 0) partial[(int64_t)blockIdx.x * elitism + r] = best;
        prev = best;
        if (best.idx < 0) {
            for (int32_t r2 = r + 1 + threadIdx.x; r2 < elitism; r2 += blockDim.x)
                partial[(int64_t)blockIdx.x * elitism + r2] = best;
            break;
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(done, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    prev.key = 0;
    prev.idx = -1;
    for (int32_t r = 0; r < elitism; ++r) {
        Rec best = block_next_best<1>(partial, (int32_t)gridDim.x * elitism, 0, r > 0, prev, s_warp);
        if (threadIdx.x == 0) elites_next[r] = best.idx;
        prev = best;
    }
    if (threadIdx.x == 0) *done = 0u;
}

size_t generation_scratch_bytes(int32_t e) { return (size_t)kSMsMax * (size_t)e * sizeof(Rec); }

// Launch shape of k_generation for this problem, or blocks = 0 when it does not apply (tables or the
// score queue do not fit shared memory, or the merge scratch would overflow).
GenerationShape generation_shape(Tables t, int32_t pairs, int32_t elitism) {
    GenerationShape g{0, 0, 0, 0};
    const int64_t warps = (int64_t)pairs + elitism;
    if (warps <= 0) return g;
    // Large populations are HBM-bound and measured faster as two launches (k_select_stage, then
    // k_evolve_score with the parents known up front); the single launch pays off when the generation is
    // launch-latency-bound.
    if (warps >= (int64_t)sm_count() * 16) return g;
    g.threads = 256;
    const int wpb = g.threads / 32;
    int64_t blocks = (warps + wpb - 1) / wpb;
    if (blocks > sm_count()) blocks = sm_count();  // the merge scratch holds up to kSMsMax lists (generation_scratch_bytes)
    const int64_t total_warps = blocks * wpb;
    const int64_t per_warp = (warps + total_warps - 1) / total_warps;
    g.queue_cap = (int32_t)(2 * per_warp * wpb);
    g.smem = evolve_score_smem(t) + (size_t)g.queue_cap * sizeof(Rec);
    if (g.smem + 1024 > (size_t)kMaxSmemPerBlock) return g;  // 1 KiB for the kernel's static shared memory
    g.blocks = (int)blocks;
    return g;
}

cudaError_t launch_generation(GenerationShape shape, const int32_t* src, int32_t* dst, int64_t ld, int32_t n,
                              int32_t n_jobs, int32_t elitism, int32_t pairs, int32_t tournament, const double* F_old,
                              double* F_new, int32_t* G, int32_t* parents, const int32_t* elites,
                              int32_t* elites_next, Tables t, RoundKeys keys, uint64_t gen, uint32_t thr16,
                              int32_t capacity, double penalty, void* scratch, unsigned int* done, cudaStream_t s) {
    if (shape.blocks <= 0) return cudaErrorInvalidConfiguration;
    const uint32_t thr32 = thr16 >= 65536u ? 0xFFFFFFFFu : thr16 << 16;
    const bool always = thr16 >= 65536u;
    void (*kern)(const int32_t*, int32_t*, int64_t, int32_t, int32_t, int32_t, int32_t, int32_t, const double*,
                 double*, int32_t*, int32_t*, const int32_t*, int32_t*, Tables, RoundKeys, uint32_t, uint32_t,
                 uint32_t, uint32_t, uint32_t, int32_t, double, Rec*, unsigned int*, int32_t);
    kern = always ? k_generation<256, 1, true> : k_generation<256, 1, false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)shape.smem);
    if (e != cudaSuccess) return e;
    return launch_after_previous(kern, shape.blocks, shape.threads, shape.smem, s, src, dst, ld, n, n_jobs, elitism, pairs,
                                 tournament, F_old, F_new, G, parents, elites, elites_next, t, keys, (uint32_t)gen,
                                 counter3(STREAM_MUT, gen), counter3(STREAM_SEL_A, gen), counter3(STREAM_SEL_B, gen), thr32,
                                 capacity, penalty, reinterpret_cast<Rec*>(scratch), done, shape.queue_cap);
}

size_t evolve_score_smem(Tables t) { return (size_t)(t.k1 + 1) * t.jpad * 10 + (size_t)t.jpad * 8; }

cudaError_t launch_evolve_score(const int32_t* src, int32_t* dst, int64_t ld, int32_t n, int32_t n_jobs,
                                int32_t elitism, int32_t pairs, const int32_t* parents, const int32_t* elites,
                                Tables t, RoundKeys keys, uint64_t gen, uint32_t thr16, int32_t capacity,
                                double penalty, double* F, int32_t* G, unsigned int* work, bool in_limits,
                                cudaStream_t s) {
    const int64_t warps = (int64_t)pairs + elitism;
    if (warps <= 0) return cudaSuccess;
    const size_t smem = evolve_score_smem(t);
    if (smem > (size_t)kMaxSmemPerBlock) return cudaErrorInvalidConfiguration;
    const uint32_t thr32 = thr16 >= 65536u ? 0xFFFFFFFFu : thr16 << 16;
    const bool always = thr16 >= 65536u, full = (ld & 127) == 0;
    // One persistent CTA per SM.  32 warps when that gives every item a warp of its own; otherwise 24 warps with
    // 80 registers each (measured 3 % faster than 32 x 64 at 2048 jobs x 65536 candidates).
    const bool wide = warps <= (int64_t)sm_count() * 32;
    const int threads = wide ? 1024 : ONES_ES_THREADS;
    int64_t blocks = (warps + threads / 32 - 1) / (threads / 32);
    if (blocks > sm_count()) blocks = sm_count();
    void (*kern)(const int32_t*, int32_t*, int64_t, int32_t, int32_t, int32_t, int32_t, const int32_t*, const int32_t*,
                 Tables, RoundKeys, uint32_t, uint32_t, uint32_t, int32_t, double, double*, int32_t*, unsigned int*);
    // the clamp of a gene to the tables' planes is only needed when genes may lie outside their jobs' limits
    const bool clamp = !in_limits;
#define ONES_ES_PICK(T)                                                                                              \
    (always ? (full ? (clamp ? k_evolve_score<T, true, true, true> : k_evolve_score<T, true, true, false>)          \
                    : (clamp ? k_evolve_score<T, true, false, true> : k_evolve_score<T, true, false, false>))       \
            : (full ? (clamp ? k_evolve_score<T, false, true, true> : k_evolve_score<T, false, true, false>)        \
                    : (clamp ? k_evolve_score<T, false, false, true> : k_evolve_score<T, false, false, false>)))
    if (wide) kern = ONES_ES_PICK(1024);
    else kern = ONES_ES_PICK(ONES_ES_THREADS);
#undef ONES_ES_PICK
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemPerBlock);
    if (e != cudaSuccess) return e;
    return launch_after_previous(kern, (int)blocks, threads, smem, s, src, dst, ld, n, n_jobs, elitism, pairs, parents,
                                 elites, t, keys, (uint32_t)gen, counter3(STREAM_MUT, gen), thr32, capacity, penalty, F, G,
                                 work);
}

// ---------------------------------------------------------------------------------------------
// Small populations: all generations of one ones_evolve call in ONE launch of one thread-block
// cluster.  Both population buffers, the scores and the model tables live in the shared memory of
// the cluster's CTAs (CTA r owns rows r*rows_per_cta ...); parents of other CTAs are read, and children
// that belong to a neighbour written, through distributed shared memory.  Every CTA keeps all scores of
// both populations: before the generation's cluster barrier a CTA stores the scores of the children it
// produced into every CTA's copy, so nothing is fetched after the barrier.  The elites of a new population
// are its rows 0..E-1 (the old elites, copied) or children that beat the old E-th best: a CTA lists those
// children (at most kClusterCand per generation, else every CTA falls back to the search over all
// scores), the lists travel with the scores, and one warp merges them.  One hardware cluster barrier per
// generation replaces the kernel boundaries; nothing spins.  Lanes are grouped so that one group of `gs` lanes (gs = int4 per
// row rounded up to a power of two, at most 32) handles one pair of children: with 6 jobs a warp
// runs 16 pairs at once.  Draws, operators, summation order and elites are those of the other paths.
// ---------------------------------------------------------------------------------------------
namespace cg = cooperative_groups;

constexpr int kClusterCand = 8;  // children of one CTA and generation that may enter the elites without the full search

struct ClusterSmem {  // byte offsets into dynamic shared memory
    size_t X, Fall0, Fall1, G16, pop0, pop1, Gc0, Gc1, kmin, range, elit, cand_cnt, cand_in, total;
};

__host__ __device__ inline ClusterSmem cluster_smem(int32_t planes, int32_t jpad, int64_t ld, int32_t rows,
                                                    int32_t elitism, int32_t n) {
    ClusterSmem m;
    size_t at = 0;
    const size_t e = (size_t)(elitism > 0 ? elitism : 1);
#define ONES_TAKE(field, bytes) m.field = at; at = (at + (size_t)(bytes) + 15) & ~(size_t)15
    ONES_TAKE(X, (size_t)planes * jpad * 8);
    ONES_TAKE(Fall0, (size_t)n * 8);  // every candidate's score, population 0 / 1
    ONES_TAKE(Fall1, (size_t)n * 8);
    ONES_TAKE(pop0, (size_t)rows * ld * 4);
    ONES_TAKE(pop1, (size_t)rows * ld * 4);
    ONES_TAKE(Gc0, (size_t)rows * 4);  // GPU counts of this CTA's rows, population 0 / 1
    ONES_TAKE(Gc1, (size_t)rows * 4);
    ONES_TAKE(kmin, (size_t)jpad * 4);
    ONES_TAKE(range, (size_t)jpad * 4);
    ONES_TAKE(elit, e * 4);
    ONES_TAKE(G16, (size_t)planes * jpad * 2);
    ONES_TAKE(cand_cnt, (size_t)2 * 16 * 4);                   // [population][producing CTA]
    ONES_TAKE(cand_in, (size_t)2 * 16 * kClusterCand * 16);    // [population][producing CTA][kClusterCand] records
#undef ONES_TAKE
    m.total = (at + 15) & ~(size_t)15;
    return m;
}

template <bool ALWAYS>
__global__ void __launch_bounds__(512, 1)
k_evolve_cluster(int32_t* __restrict__ pop_io, int64_t ld, int32_t n, int32_t n_jobs, int32_t elitism, int32_t pairs,
                 int32_t tournament, double* __restrict__ F_io, int32_t* __restrict__ G_out,
                 int32_t* __restrict__ parents_out, int32_t* __restrict__ elites_out, Tables t, RoundKeys keys,
                 uint64_t gen0, int32_t generations, uint32_t thr32, int32_t capacity, double penalty,
                 int32_t rows_shift /* rows per CTA = 1 << rows_shift */, int32_t gs) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ Rec s_warp[64];
    __shared__ Rec s_top[4];
    __shared__ int s_full;  // the elites of this generation need the search over all scores
    cg::cluster_group cluster = cg::this_cluster();
    const int32_t C = (int32_t)cluster.num_blocks(), me = (int32_t)cluster.block_rank();
    const int32_t planes = t.k1 + 1, jpad = t.jpad;
    const int32_t rows_per_cta = 1 << rows_shift, rows_mask = rows_per_cta - 1;
    const ClusterSmem m = cluster_smem(planes, jpad, ld, rows_per_cta, elitism, n);
    double* sX = reinterpret_cast<double*>(smem_raw + m.X);
    uint16_t* sG = reinterpret_cast<uint16_t*>(smem_raw + m.G16);
    double* sFall[2] = {reinterpret_cast<double*>(smem_raw + m.Fall0), reinterpret_cast<double*>(smem_raw + m.Fall1)};
    int32_t* sCandCnt = reinterpret_cast<int32_t*>(smem_raw + m.cand_cnt);
    Rec* sCandIn = reinterpret_cast<Rec*>(smem_raw + m.cand_in);
    int32_t* sPop[2] = {reinterpret_cast<int32_t*>(smem_raw + m.pop0), reinterpret_cast<int32_t*>(smem_raw + m.pop1)};
    int32_t* sGc[2] = {reinterpret_cast<int32_t*>(smem_raw + m.Gc0), reinterpret_cast<int32_t*>(smem_raw + m.Gc1)};
    int4* sKmin = reinterpret_cast<int4*>(smem_raw + m.kmin);
    int4* sRange = reinterpret_cast<int4*>(smem_raw + m.range);
    int32_t* sElit = reinterpret_cast<int32_t*>(smem_raw + m.elit);

    const int32_t lo = me * rows_per_cta, hi = min(n, lo + rows_per_cta), mine = max(0, hi - lo);
    const int32_t nvec = (int32_t)(ld >> 2);
    {   // stage tables, my rows and their scores
        const int32_t cells = planes * jpad;
        for (int32_t i = threadIdx.x; i < cells; i += blockDim.x) {
            sX[i] = t.X[i];
            sG[i] = (uint16_t)t.G[i];
        }
        for (int32_t i = threadIdx.x; i < jpad; i += blockDim.x) {
            reinterpret_cast<int32_t*>(sKmin)[i] = t.kmin[i];
            reinterpret_cast<int32_t*>(sRange)[i] = t.range[i];
        }
        const int4* src = reinterpret_cast<const int4*>(pop_io + (int64_t)lo * ld);
        for (int32_t i = threadIdx.x; i < mine * nvec; i += blockDim.x) reinterpret_cast<int4*>(sPop[0])[i] = src[i];
        for (int32_t i = threadIdx.x; i < n; i += blockDim.x) sFall[0][i] = F_io[i];  // every CTA takes all scores
        for (int32_t i = threadIdx.x; i < mine; i += blockDim.x) sGc[0][i] = G_out[lo + i];
    }
    __syncthreads();
    cluster.sync();  // everybody's rows and scores are staged

    const uint32_t kcap = (uint32_t)t.k1;
    const int32_t groups = (int32_t)blockDim.x / gs;
    const int32_t gi = (int32_t)threadIdx.x / gs, gl = (int32_t)threadIdx.x % gs;
    // child rows owned by this CTA: elite rows r < elitism, then pairs whose even child (row elitism + 2q) is mine
    const int32_t elite_lo = min(lo, elitism), elite_hi = min(hi, elitism);
    const int32_t first_child = max(lo, elitism);
    const int32_t q_lo = (first_child - elitism + 1) >> 1;                    // first q with elitism + 2q >= first_child
    const int32_t q_hi = hi > elitism ? min(pairs, (hi - elitism + 1) >> 1) : 0;  // first q with elitism + 2q >= hi
    // work items of a group: a pair of children, or (after the pairs, where the last trip usually has idle groups)
    // the copy of this CTA's elite rows, which keep their scores and GPU counts: all of them in one item when the
    // elites come from the lists (at most four), else one row per item
    const int32_t n_pairs = max(0, q_hi - q_lo);
    const int32_t elite_span = (elitism > 0 && elitism <= 4) ? 4 : 1;
    const int32_t n_elite_items = (max(0, elite_hi - elite_lo) + elite_span - 1) / elite_span;
    // the copies start at a warp of their own, so that no warp runs both kinds of item one after the other
    // (where that does not cost a trip)
    const int32_t groups_per_warp = gs < 32 ? 32 / gs : 1;
    const int32_t aligned0 = (n_pairs + groups_per_warp - 1) / groups_per_warp * groups_per_warp;
    const int32_t trips = (n_pairs + n_elite_items + groups - 1) / groups;
    const int32_t elite_item0 = aligned0 + n_elite_items <= trips * groups ? aligned0 : n_pairs;
    // the rows this CTA produces: its elite rows and both children of its pairs (the last odd child may be
    // a neighbour's row); over the cluster these ranges cover every row exactly once
    const int32_t made_elites = max(0, elite_hi - elite_lo);
    const int32_t child_lo = elitism + 2 * q_lo, child_hi = q_hi > q_lo ? min(n, elitism + 2 * q_hi) : child_lo;
    const int32_t made = made_elites + (child_hi - child_lo);
    const bool lists = elitism > 0 && elitism <= 4;  // elites by merging lists of promising children
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for (int32_t g = 0; g < generations; ++g) {
        const int cur = g & 1, nxt = cur ^ 1;
        const uint64_t gen = gen0 + (uint64_t)g;
        const uint32_t gen_lo = (uint32_t)gen;
        const uint32_t c3 = counter3(STREAM_MUT, gen), c3a = counter3(STREAM_SEL_A, gen), c3b = counter3(STREAM_SEL_B, gen);
        // ---- every CTA finds the elites of the population in force for itself ----
        const double* Fcur = sFall[cur];
        // With lists, warp 0 merges while the other warps already run their tournaments; everybody meets in
        // settle_elites() before the first thing that needs the elites (the end of the first trip).
        auto settle_elites = [&]() {
            bool full = g == 0;  // nothing is known about a population that came from outside
            if (!full) {
                __syncthreads();
                full = s_full != 0;
            }
            if (full) {  // sorted lists in registers over all scores, one barrier
                if (elitism <= 2) block_top_small<2, 0, false, 512>(Fcur, n, 0, elitism, s_top, s_warp);
                else block_top_small<4, 0, false, 512>(Fcur, n, 0, elitism, s_top, s_warp);
                __syncthreads();
            }
            if ((int32_t)threadIdx.x < elitism) {
                sElit[threadIdx.x] = s_top[threadIdx.x].idx;
                if (me == 0) elites_out[threadIdx.x] = s_top[threadIdx.x].idx;
            }
        };
        if (lists) {
            if (threadIdx.x == 0) sCandCnt[nxt * 16 + me] = 0;  // this generation's own list
            if (g > 0) {
                if (warp == 0) {
                    // rows 0..E-1 hold the old elites; a child enters only with a score above the old E-th best
                    const int32_t cnt = lane < C ? sCandCnt[cur * 16 + lane] : 0;
                    const bool over = __any_sync(0xFFFFFFFFu, cnt > kClusterCand);
                    if (!__any_sync(0xFFFFFFFFu, cnt > 0)) {
                        // no child beat the old elites: they stay, in their order, now as rows 0..E-1
                        if (lane < elitism) {
                            Rec q;
                            q.key = score_key(Fcur[lane]);
                            q.idx = lane;
                            q.pad = 0;
                            s_top[lane] = q;
                        }
                    } else if (!over) {
                        TopList<4> top;
                        top_list_clear(top);
                        if (lane < elitism) top_list_insert(top, score_key(Fcur[lane]), lane);
                        for (int32_t c = 0; c < cnt; ++c) {
                            const Rec q = sCandIn[(cur * 16 + lane) * kClusterCand + c];
                            top_list_insert(top, q.key, q.idx);
                        }
                        for (int32_t r = 0; r < elitism; ++r) {
                            const Rec best = warp_pop_best(top);
                            if (lane == 0) s_top[r] = best;
                        }
                    }
                    if (lane == 0) s_full = over;
                }
            }
            if (trips == 0) settle_elites();
        } else if (elitism > 0) {
            Rec prev;
            prev.key = 0;
            prev.idx = -1;
            prev.pad = 0;
            for (int32_t r = 0; r < elitism; ++r) {
                Rec best = block_next_best<0>(Fcur, n, 0, r > 0, prev, s_warp);
                if (threadIdx.x == 0) {
                    sElit[r] = best.idx;
                    if (me == 0) elites_out[r] = best.idx;
                }
                prev = best;
            }
            __syncthreads();
        }
        // ---- children ----
        for (int32_t trip = 0; trip < trips; ++trip) {
            const int32_t item = trip * groups + gi;
            const bool is_elite = item >= elite_item0 && item < elite_item0 + n_elite_items;
            const bool live = item < n_pairs || is_elite;
            int32_t pa = 0, pb = 0, slot0 = 0, slot1 = 0;
            bool has1 = false;
            uint32_t thr = 0u;
            auto copy_elites = [&]() {
                const int32_t ea = elite_lo + (item - elite_item0) * elite_span, eb = min(elite_hi, ea + elite_span);
                for (int32_t r = ea; r < eb; ++r) {  // rows of this CTA
                    const int32_t idx = elitism <= 4 ? s_top[r].idx : sElit[r];
                    const int4* A = reinterpret_cast<const int4*>(cluster.map_shared_rank(
                        sPop[cur] + (int64_t)(idx & rows_mask) * ld, (unsigned int)(idx >> rows_shift)));
                    int4* Cd = reinterpret_cast<int4*>(sPop[nxt] + (int64_t)(r & rows_mask) * ld);
                    for (int32_t v = gl; v < nvec; v += gs) Cd[v] = A[v];
                    if (gl == 0) {
                        sFall[nxt][r] = Fcur[idx];
                        sGc[nxt][r & rows_mask] = *cluster.map_shared_rank(sGc[cur] + (idx & rows_mask), (unsigned int)(idx >> rows_shift));
                    }
                }
            };
            const bool late = lists && trip == 0;  // the elites are settled at the end of this trip
            if (is_elite) {
                if (!late) copy_elites();
            } else if (live) {
                const int32_t q = q_lo + item;
                // the two tournaments: the lower half of the group's lanes runs the first parent's, the upper half
                // the second's (a group of one lane runs both), every lane for itself (same draws, same winner)
                for (int which = gs > 1 ? (gl >= (gs >> 1) ? 1 : 0) : 0; which < 2; ++which) {
                    int32_t win = -1;
                    double fwin = 0.0;
                    for (int32_t t0 = 0; t0 < tournament; t0 += 4) {
                        const uint4 w4 = philox((uint32_t)(t0 >> 2), (uint32_t)q, gen_lo, which ? c3b : c3a, keys);
                        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (t0 + u < tournament) {
                                const int32_t idx = (int32_t)__umulhi(w[u], (uint32_t)n);
                                const double f = Fcur[idx];
                                if (win < 0 || f > fwin || (f == fwin && idx < win)) {
                                    win = idx;
                                    fwin = f;
                                }
                            }
                        }
                    }
                    if (which) pb = win; else pa = win;
                    if (gs > 1) break;
                }
                slot0 = elitism + 2 * q;
                slot1 = slot0 + 1;
                has1 = slot1 < n;
                thr = thr32;
            }
            if (gs > 1) {  // each half of a group learns the other half's winner (all lanes of the warp take part)
                const int first = lane & ~(gs - 1);
                const int32_t wa = __shfl_sync(0xFFFFFFFFu, pa, first), wb = __shfl_sync(0xFFFFFFFFu, pb, first + (gs >> 1));
                if (live && !is_elite) {
                    pa = wa;
                    pb = wb;
                }
            }
            if (live && !is_elite && gl == 0) {
                const int32_t q = (slot0 - elitism) >> 1;
                parents_out[2 * q] = pa;
                parents_out[2 * q + 1] = pb;
            }
            double sum0 = 0.0, sum1 = 0.0;
            int32_t gp0 = 0, gp1 = 0;
            if (live && !is_elite) {
                const int32_t oa = pa >> rows_shift, ob = pb >> rows_shift;
                const int4* A = reinterpret_cast<const int4*>(cluster.map_shared_rank(sPop[cur] + (int64_t)(pa & rows_mask) * ld, (unsigned int)oa));
                const int4* B = reinterpret_cast<const int4*>(cluster.map_shared_rank(sPop[cur] + (int64_t)(pb & rows_mask) * ld, (unsigned int)ob));
                const int32_t o0 = slot0 >> rows_shift, o1 = has1 ? slot1 >> rows_shift : o0;
                int4* C0 = reinterpret_cast<int4*>(cluster.map_shared_rank(sPop[nxt] + (int64_t)(slot0 & rows_mask) * ld, (unsigned int)o0));
                int4* C1 = reinterpret_cast<int4*>(cluster.map_shared_rank(sPop[nxt] + (int64_t)((has1 ? slot1 : slot0) & rows_mask) * ld, (unsigned int)o1));
                for (int32_t v = gl; v < nvec; v += gs) {
                    const int4 a = A[v], b = B[v];
                    int4 c0, c1;
                    const uint4 W = philox((uint32_t)v, (uint32_t)slot0, gen_lo, c3, keys);
                    if (ALWAYS) sibling_int4<true>(W, a, b, sKmin[v], sRange[v], thr, has1, c0, c1);
                    else sibling_int4<false>(W, a, b, sKmin[v], sRange[v], thr, has1, c0, c1);
                    C0[v] = c0;
                    const int32_t base = (v >> 5) * 128 + (v & 31);
                    score4(c0, base, kcap, jpad, sX, sG, sum0, gp0);
                    if (has1) {
                        C1[v] = c1;
                        score4(c1, base, kcap, jpad, sX, sG, sum1, gp1);
                    }
                }
            }
            if (late) {
                settle_elites();
                if (is_elite) copy_elites();
            }
            // fixed-order sum over the group's lanes (partials of absent lanes are +0)
            for (int off = gs >> 1; off >= 1; off >>= 1) {
                sum0 = __dadd_rn(sum0, __shfl_xor_sync(0xFFFFFFFFu, sum0, off));
                gp0 += __shfl_xor_sync(0xFFFFFFFFu, gp0, off);
                sum1 = __dadd_rn(sum1, __shfl_xor_sync(0xFFFFFFFFu, sum1, off));
                gp1 += __shfl_xor_sync(0xFFFFFFFFu, gp1, off);
            }
            if (live && !is_elite && gl == 0) {
                // scores go to this CTA's copy first (sent to the others below); a child that beats the old
                // E-th best is listed for the next generation's elites
                const unsigned long long bar = lists ? s_top[elitism - 1].key : ~0ull;
                auto leave = [&](int32_t slot, double sum, int32_t gp) {
                    const int32_t over = gp > capacity ? gp - capacity : 0;
                    const double f = __dsub_rn(sum, __dmul_rn(penalty, (double)over));
                    sFall[nxt][slot] = f;
                    *cluster.map_shared_rank(sGc[nxt] + (slot & rows_mask), (unsigned int)(slot >> rows_shift)) = gp;
                    const unsigned long long key = score_key(f);
                    if (key > bar) {
                        const int32_t c = atomicAdd(&sCandCnt[nxt * 16 + me], 1);
                        if (c < kClusterCand) {
                            Rec q;
                            q.key = key;
                            q.idx = slot;
                            q.pad = 0;
                            sCandIn[(nxt * 16 + me) * kClusterCand + c] = q;
                        }
                    }
                };
                leave(slot0, sum0, gp0);
                if (has1) leave(slot1, sum1, gp1);
            }
        }
        __syncthreads();  // this CTA's scores and list are complete
        if (C > 1) {
            // what this CTA produced, to every other CTA's copy of the scores (and its list, one lane per CTA)
            double* Fnext = sFall[nxt];
            for (int32_t w = threadIdx.x; w < made * C; w += blockDim.x) {  // neighbouring lanes: neighbouring rows
                const int32_t r = w / made, i = w - r * made;
                const int32_t slot = i < made_elites ? elite_lo + i : child_lo + (i - made_elites);
                if (r != me) *cluster.map_shared_rank(Fnext + slot, (unsigned int)r) = Fnext[slot];
            }
            if (lists && warp == 1 && lane < C && lane != me) {
                const int32_t cnt = sCandCnt[nxt * 16 + me];
                *cluster.map_shared_rank(sCandCnt + nxt * 16 + me, (unsigned int)lane) = cnt;
                for (int32_t c = 0; c < min(cnt, kClusterCand); ++c) {
                    Rec* at = sCandIn + (nxt * 16 + me) * kClusterCand + c;
                    *cluster.map_shared_rank(at, (unsigned int)lane) = *at;
                }
            }
        }
        cluster.sync();  // all children, their scores and the lists are where they belong
    }
    // ---- write my rows back ----
    const int fin = generations & 1;
    int4* dst = reinterpret_cast<int4*>(pop_io + (int64_t)lo * ld);
    for (int32_t i = threadIdx.x; i < mine * nvec; i += blockDim.x) dst[i] = reinterpret_cast<const int4*>(sPop[fin])[i];
    for (int32_t i = threadIdx.x; i < mine; i += blockDim.x) {
        F_io[lo + i] = sFall[fin][lo + i];
        G_out[lo + i] = sGc[fin][i];
    }
}

template <bool ALWAYS>
static cudaError_t cluster_config(ClusterShape shape, cudaStream_t s, cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr) {
    auto kern = k_evolve_cluster<ALWAYS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)shape.smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, shape.cluster > 8 ? 1 : 0);
    if (e != cudaSuccess) return e;
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3((unsigned)shape.cluster, 1, 1);
    cfg->blockDim = dim3((unsigned)shape.threads, 1, 1);
    cfg->dynamicSmemBytes = shape.smem;
    cfg->stream = s;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)shape.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg->attrs = attr;
    cfg->numAttrs = 1;
    return cudaSuccess;
}

// cluster == 0: the population does not fit the shared memory of one cluster that the device can host (or is
// large enough for the HBM paths).  rows_per_cta >= 32 keeps every CTA busy.
ClusterShape cluster_shape(Tables t, int64_t ld, int32_t n, int32_t elitism, int32_t pairs) {
    ClusterShape shape{0, 0, 0, 0, 0};
    if ((int64_t)pairs + elitism >= (int64_t)sm_count() * 16) return shape;
    const int32_t nvec = (int32_t)(ld >> 2);
    int gs = 1;
    while (gs < nvec && gs < 32) gs <<= 1;
    for (int c = 16; c >= 1; c >>= 1) {
        int32_t rows = 1;  // rows per CTA: a power of two (owners and offsets by shift and mask)
        while (rows < (n + c - 1) / c) rows <<= 1;
        if (c > 1 && (rows < 32 || (int64_t)rows * (c - 1) >= n)) continue;  // keep every CTA busy
        const size_t bytes = cluster_smem(t.k1 + 1, t.jpad, ld, rows, elitism, n).total;
        if (bytes + 2048 > (size_t)kMaxSmemPerBlock) continue;
        ClusterShape trial{c, 512, rows, gs, bytes};
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr[1];
        int max_clusters = 0;
        if (cluster_config<false>(trial, nullptr, &cfg, attr) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&max_clusters, k_evolve_cluster<false>, &cfg) != cudaSuccess ||
            max_clusters < 1) {
            cudaGetLastError();  // this size cannot be hosted: try a smaller cluster
            continue;
        }
        return trial;
    }
    return shape;
}

template <bool ALWAYS>
static cudaError_t launch_cluster_t(ClusterShape shape, int32_t* pop_io, int64_t ld, int32_t n, int32_t n_jobs,
                                    int32_t elitism, int32_t pairs, int32_t tournament, double* F_io, int32_t* G_out,
                                    int32_t* parents_out, int32_t* elites_out, Tables t, RoundKeys keys, uint64_t gen0,
                                    int32_t generations, uint32_t thr32, int32_t capacity, double penalty,
                                    cudaStream_t s) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    cudaError_t e = cluster_config<ALWAYS>(shape, s, &cfg, attr);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, k_evolve_cluster<ALWAYS>, pop_io, ld, n, n_jobs, elitism, pairs, tournament, F_io,
                              G_out, parents_out, elites_out, t, keys, gen0, generations, thr32, capacity, penalty,
                              (int32_t)(31 - __builtin_clz((unsigned)shape.rows_per_cta)), (int32_t)shape.gs);
}

cudaError_t launch_evolve_cluster(ClusterShape shape, int32_t* pop_io, int64_t ld, int32_t n, int32_t n_jobs,
                                  int32_t elitism, int32_t pairs, int32_t tournament, double* F_io, int32_t* G_out,
                                  int32_t* parents_out, int32_t* elites_out, Tables t, RoundKeys keys, uint64_t gen0,
                                  int32_t generations, uint32_t thr16, int32_t capacity, double penalty, cudaStream_t s) {
    if (shape.cluster <= 0) return cudaErrorInvalidConfiguration;
    const uint32_t thr32 = thr16 >= 65536u ? 0xFFFFFFFFu : thr16 << 16;
    if (thr16 >= 65536u)
        return launch_cluster_t<true>(shape, pop_io, ld, n, n_jobs, elitism, pairs, tournament, F_io, G_out, parents_out,
                                      elites_out, t, keys, gen0, generations, thr32, capacity, penalty, s);
    return launch_cluster_t<false>(shape, pop_io, ld, n, n_jobs, elitism, pairs, tournament, F_io, G_out, parents_out,
                                   elites_out, t, keys, gen0, generations, thr32, capacity, penalty, s);
}

// ---------------------------------------------------------------------------------------------
// The paper's own selection (Section 3.2.2 "Evolution" / "Selection"): the candidate pool G'_i holds
// the K current candidates (rows 0..K-1), 2K crossover children of K uniformly drawn parent pairs
// (rows K..3K-1, no mutation) and K mutants of K uniformly drawn candidates (rows 3K..4K-1); the best K
// of the 4K (score descending, row ascending) survive in the order of their rows.
// ---------------------------------------------------------------------------------------------
// draws[0..2K): parents of pair q at 2q, 2q+1; draws[2K..3K): source row of mutant m
__global__ void k_trunc_draws(int32_t k, RoundKeys keys, uint32_t gen_lo, uint32_t c3a, uint32_t c3b, uint32_t c3pick,
                              int32_t* __restrict__ draws) {
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 3 * k) return;
    uint32_t row, c3;
    if (i < 2 * k) {
        row = (uint32_t)(i >> 1);
        c3 = (i & 1) ? c3b : c3a;
    } else {
        row = (uint32_t)(i - 2 * k);
        c3 = c3pick;
    }
    const uint4 w = philox(0u, row, gen_lo, c3, keys);
    draws[i] = (int32_t)__umulhi(w.x, (uint32_t)k);
}

// one warp per work item: items 0..K-1 are crossover pairs, K..2K-1 mutants
template <bool ALWAYS>
__global__ void __launch_bounds__(256, 4)
k_trunc_children(int32_t* __restrict__ pool, int64_t ld, int32_t k, const int32_t* __restrict__ draws, Tables t,
                 RoundKeys keys, uint32_t gen_lo, uint32_t c3cross, uint32_t c3mutant, uint32_t thr32) {
    const int lane = threadIdx.x & 31;
    const int64_t item = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (item >= 2 * (int64_t)k) return;
    const int32_t nvec = (int32_t)(ld >> 2);
    const int4* __restrict__ kminv = reinterpret_cast<const int4*>(t.kmin);
    const int4* __restrict__ rangev = reinterpret_cast<const int4*>(t.range);
    if (item < k) {
        const int32_t q = (int32_t)item;
        const int4* A = reinterpret_cast<const int4*>(pool + (int64_t)draws[2 * q] * ld);
        const int4* B = reinterpret_cast<const int4*>(pool + (int64_t)draws[2 * q + 1] * ld);
        int4* C0 = reinterpret_cast<int4*>(pool + ((int64_t)k + 2 * q) * ld);
        int4* C1 = reinterpret_cast<int4*>(pool + ((int64_t)k + 2 * q + 1) * ld);
        for (int32_t v = lane; v < nvec; v += 32) {
            const uint4 W = philox((uint32_t)v, (uint32_t)(2 * q), gen_lo, c3cross, keys);
            int4 c0, c1;
            sibling_int4<false>(W, A[v], B[v], kminv[v], rangev[v], 0u, true, c0, c1);  // threshold 0: no mutation
            C0[v] = c0;
            C1[v] = c1;
        }
    } else {
        const int32_t m = (int32_t)(item - k);
        const int4* S = reinterpret_cast<const int4*>(pool + (int64_t)draws[2 * k + m] * ld);
        int4* C = reinterpret_cast<int4*>(pool + ((int64_t)3 * k + m) * ld);
        for (int32_t v = lane; v < nvec; v += 32) {
            const uint4 W = philox((uint32_t)v, (uint32_t)m, gen_lo, c3mutant, keys);
            const int4 g = S[v];
            int4 c0, c1;
            sibling_int4<ALWAYS>(W, g, g, kminv[v], rangev[v], thr32, false, c0, c1);  // the even child's draws
            C[v] = c0;
        }
    }
}

// The same children, scored while they are written (as k_evolve_score: one persistent CTA per SM with the
// model tables in shared memory, one warp per work item, the fixed summation order), so the 3K new rows are
// not read back for their fitness.  F, G: the pool's score arrays (4K entries; rows K..4K-1 are written).
// Measured at 65536 candidates of 2048 jobs (ms per generation): 1024 threads 0.639, with the next step's parent
// genes loaded one step ahead 0.630; 768 threads (more registers) 0.691 and 0.673.
#ifndef ONES_TC_THREADS
#define ONES_TC_THREADS 1024
#endif
#ifndef ONES_TC_PREFETCH
#define ONES_TC_PREFETCH 1
#endif
template <bool ALWAYS>
__global__ void __launch_bounds__(ONES_TC_THREADS, 1)
k_trunc_children_score(int32_t* __restrict__ pool, int64_t ld, int32_t k, int32_t* __restrict__ draws, Tables t,
                       RoundKeys keys, uint32_t gen_lo, uint32_t c3a, uint32_t c3b, uint32_t c3pick, uint32_t c3cross,
                       uint32_t c3mutant, uint32_t thr32, int32_t capacity, double penalty, double* __restrict__ F,
                       int32_t* __restrict__ G, const int32_t* __restrict__ rowmap) {
    // (no early release of the selection that follows: measured 0.711-0.715 ms per generation with it against
    // 0.686 without, 65536 candidates of 2048 jobs)
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int32_t planes = t.k1 + 1;
    const int32_t jpad = t.jpad;
    double* sX = reinterpret_cast<double*>(smem_raw);
    uint16_t* sG = reinterpret_cast<uint16_t*>(smem_raw + (size_t)planes * jpad * 8);
    int4* sKmin = reinterpret_cast<int4*>(smem_raw + (size_t)planes * jpad * 10);
    int4* sRange = sKmin + jpad / 4;
    {
        const int32_t nX = planes * jpad / 2, nG = planes * jpad / 4;
        const int4* gX = reinterpret_cast<const int4*>(t.X);
        const int4* gG = reinterpret_cast<const int4*>(t.G);
        for (int32_t i = threadIdx.x; i < nX; i += blockDim.x) reinterpret_cast<int4*>(sX)[i] = gX[i];
        for (int32_t i = threadIdx.x; i < nG; i += blockDim.x) {
            const int4 g = gG[i];
            reinterpret_cast<uint2*>(sG)[i] = make_uint2((uint32_t)g.x | ((uint32_t)g.y << 16),
                                                         (uint32_t)g.z | ((uint32_t)g.w << 16));
        }
        for (int32_t i = threadIdx.x; i < jpad / 4; i += blockDim.x) {
            sKmin[i] = reinterpret_cast<const int4*>(t.kmin)[i];
            sRange[i] = reinterpret_cast<const int4*>(t.range)[i];
        }
        __syncthreads();
    }
    grid_dependency_wait();  // the pool, its row map and the scores come from the kernels before
    constexpr int UN = 1;  // int4 per source row in flight per lane (2 measured 2 % slower)
    const uint64_t keep = l2_policy_evict_last();  // the K current candidates are read about three times each
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = blockDim.x >> 5;
    const int64_t total_warps = (int64_t)gridDim.x * warps_per_block;
    const int32_t nvec = (int32_t)(ld >> 2);
    const uint32_t kcap = (uint32_t)t.k1;
    // pool row of a logical row (the pool is used in place: survivors stay where they are)
    auto row_of = [&](int64_t logical) -> int64_t { return rowmap ? (int64_t)rowmap[logical] : logical; };
    for (int64_t item = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); item < 2 * (int64_t)k;
         item += total_warps) {
        double sum0 = 0.0, sum1 = 0.0;
        int32_t gp0 = 0, gp1 = 0;
        int64_t slot0;
        const bool pair = item < k;
        if (pair) {
            const int32_t q = (int32_t)item;
            // the pair's two uniformly drawn parents (as k_trunc_draws; kept for ones_last_parents)
            const int32_t pa = (int32_t)__umulhi(philox(0u, (uint32_t)q, gen_lo, c3a, keys).x, (uint32_t)k);
            const int32_t pb = (int32_t)__umulhi(philox(0u, (uint32_t)q, gen_lo, c3b, keys).x, (uint32_t)k);
            if (lane == 0) {
                draws[2 * q] = pa;
                draws[2 * q + 1] = pb;
            }
            const int4* A = reinterpret_cast<const int4*>(pool + row_of(pa) * ld);
            const int4* B = reinterpret_cast<const int4*>(pool + row_of(pb) * ld);
            slot0 = (int64_t)k + 2 * q;
            int4* C0 = reinterpret_cast<int4*>(pool + row_of(slot0) * ld);
            int4* C1 = reinterpret_cast<int4*>(pool + row_of(slot0 + 1) * ld);
#if ONES_TC_PREFETCH
            int4 an = make_int4(0, 0, 0, 0), bn = an;  // the next step's parent genes are in flight while this one works
            if (lane < nvec) {
                an = ld_row_hint(reinterpret_cast<const unsigned char*>(A + lane), keep);
                bn = ld_row_hint(reinterpret_cast<const unsigned char*>(B + lane), keep);
            }
#endif
            for (int32_t v0 = lane; v0 < nvec; v0 += 32 * UN) {
                int4 a[UN], b[UN];
#if ONES_TC_PREFETCH
                a[0] = an;
                b[0] = bn;
                if (v0 + 32 < nvec) {
                    an = ld_row_hint(reinterpret_cast<const unsigned char*>(A + v0 + 32), keep);
                    bn = ld_row_hint(reinterpret_cast<const unsigned char*>(B + v0 + 32), keep);
                }
#else
#pragma unroll
                for (int u = 0; u < UN; ++u) {
                    const int32_t v = v0 + 32 * u;
                    if (v < nvec) {
                        a[u] = ld_row_hint(reinterpret_cast<const unsigned char*>(A + v), keep);
                        b[u] = ld_row_hint(reinterpret_cast<const unsigned char*>(B + v), keep);
                    }
                }
#endif
#pragma unroll
                for (int u = 0; u < UN; ++u) {
                    const int32_t v = v0 + 32 * u;
                    if (v < nvec) {
                        const uint4 W = philox((uint32_t)v, (uint32_t)(2 * q), gen_lo, c3cross, keys);
                        int4 c0, c1;
                        sibling_int4<false>(W, a[u], b[u], sKmin[v], sRange[v], 0u, true, c0, c1);  // threshold 0: no mutation
                        __stcs(C0 + v, c0);
                        __stcs(C1 + v, c1);
                        const int32_t base = (v >> 5) * 128 + lane;
                        score4(c0, base, kcap, jpad, sX, sG, sum0, gp0);
                        score4(c1, base, kcap, jpad, sX, sG, sum1, gp1);
                    }
                }
            }
        } else {
            const int32_t m = (int32_t)(item - k);
            const int32_t ps = (int32_t)__umulhi(philox(0u, (uint32_t)m, gen_lo, c3pick, keys).x, (uint32_t)k);
            if (lane == 0) draws[2 * k + m] = ps;
            const int4* S = reinterpret_cast<const int4*>(pool + row_of(ps) * ld);
            slot0 = (int64_t)3 * k + m;
            int4* C = reinterpret_cast<int4*>(pool + row_of(slot0) * ld);
#if ONES_TC_PREFETCH
            int4 gn = make_int4(0, 0, 0, 0), gn2 = gn;  // two steps ahead: a mutant reads one row only
            if (lane < nvec) gn = ld_row_hint(reinterpret_cast<const unsigned char*>(S + lane), keep);
            if (lane + 32 < nvec) gn2 = ld_row_hint(reinterpret_cast<const unsigned char*>(S + lane + 32), keep);
#endif
            for (int32_t v0 = lane; v0 < nvec; v0 += 32 * UN) {
                int4 g[UN];
#if ONES_TC_PREFETCH
                g[0] = gn;
                gn = gn2;
                if (v0 + 64 < nvec) gn2 = ld_row_hint(reinterpret_cast<const unsigned char*>(S + v0 + 64), keep);
#else
#pragma unroll
                for (int u = 0; u < UN; ++u)
                    if (v0 + 32 * u < nvec) g[u] = ld_row_hint(reinterpret_cast<const unsigned char*>(S + v0 + 32 * u), keep);
#endif
#pragma unroll
                for (int u = 0; u < UN; ++u) {
                    const int32_t v = v0 + 32 * u;
                    if (v < nvec) {
                        const uint4 W = philox((uint32_t)v, (uint32_t)m, gen_lo, c3mutant, keys);
                        int4 c0, c1;
                        sibling_int4<ALWAYS>(W, g[u], g[u], sKmin[v], sRange[v], thr32, false, c0, c1);  // the even child's draws
                        __stcs(C + v, c0);
                        score4(c0, (v >> 5) * 128 + lane, kcap, jpad, sX, sG, sum0, gp0);
                    }
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum0 = __dadd_rn(sum0, __shfl_xor_sync(0xFFFFFFFFu, sum0, off));
            gp0 += __shfl_xor_sync(0xFFFFFFFFu, gp0, off);
            sum1 = __dadd_rn(sum1, __shfl_xor_sync(0xFFFFFFFFu, sum1, off));
            gp1 += __shfl_xor_sync(0xFFFFFFFFu, gp1, off);
        }
        if (lane == 0) {
            const int32_t over0 = gp0 > capacity ? gp0 - capacity : 0;
            F[slot0] = __dsub_rn(sum0, __dmul_rn(penalty, (double)over0));
            G[slot0] = gp0;
            if (pair) {
                const int32_t over1 = gp1 > capacity ? gp1 - capacity : 0;
                F[slot0 + 1] = __dsub_rn(sum1, __dmul_rn(penalty, (double)over1));
                G[slot0 + 1] = gp1;
            }
        }
    }
}

struct TruncPick {  // result of the selection threshold search
    unsigned long long key;  // key of the K-th best candidate
    int32_t quota;           // how many candidates with exactly that key survive (lowest rows first)
    int32_t pad;
};

// K-th largest of n score keys by an 8-pass radix search.  One launch per pass: every CTA histograms the
// current digit of the keys that match the prefix found so far; the last CTA to finish picks the digit
// that holds the K-th key, narrows the prefix and clears the histogram for the next pass.
struct TruncState {
    unsigned long long prefix;
    int32_t remaining;
    unsigned int done;
    unsigned int hist[256];
};

__global__ void __launch_bounds__(256) k_trunc_radix_pass(const double* __restrict__ F, int32_t n, int32_t k, int pass,
                                                          TruncState* __restrict__ st, TruncPick* __restrict__ out) {
    grid_dependency_wait();  // launched as a programmatic dependent: only the launch latency overlaps
    __shared__ unsigned int hist[256];
    __shared__ bool s_last;
    hist[threadIdx.x] = 0u;
    __syncthreads();
    const int shift = 56 - 8 * pass;
    const unsigned long long mask = pass == 0 ? 0ull : ~0ull << (shift + 8);
    const unsigned long long prefix = pass == 0 ? 0ull : st->prefix;
    for (int32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const unsigned long long key = score_key(F[i]);
        if ((key & mask) == prefix) {
            // similar scores share their leading digits: one atomic per distinct digit in the warp
            const unsigned int digit = (unsigned int)(key >> shift) & 255u;
            const unsigned int peers = __match_any_sync(__activemask(), digit);
            if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[digit], (unsigned int)__popc(peers));
        }
    }
    __syncthreads();
    if (hist[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], hist[threadIdx.x]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&st->done, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    hist[threadIdx.x] = __ldcg(&st->hist[threadIdx.x]);
    st->hist[threadIdx.x] = 0u;
    __syncthreads();
    if (threadIdx.x == 0) {
        int32_t remaining = pass == 0 ? k : st->remaining;
        int32_t above = 0, d = 255;
        for (; d > 0; --d) {
            if (above + (int32_t)hist[d] >= remaining) break;
            above += (int32_t)hist[d];
        }
        remaining -= above;
        const unsigned long long np = prefix | ((unsigned long long)d << shift);
        st->prefix = np;
        st->remaining = remaining;
        st->done = 0u;
        if (pass == 7) {
            out->key = np;
            out->quota = remaining;
            out->pad = 0;
        }
    }
}

// per block of `per_block` consecutive rows: how many rank above the threshold, how many tie with it
__global__ void __launch_bounds__(256) k_trunc_count(const double* __restrict__ F, int32_t n, int32_t per_block,
                                                     const TruncPick* __restrict__ pick, int32_t* __restrict__ bsum) {
    grid_dependency_wait();  // launched as a programmatic dependent: only the launch latency overlaps
    __shared__ int32_t s_gt, s_eq;
    if (threadIdx.x == 0) s_gt = s_eq = 0;
    __syncthreads();
    const unsigned long long T = pick->key;
    const int32_t lo = blockIdx.x * per_block, hi = min(n, lo + per_block);
    int32_t gt = 0, eq = 0;
    for (int32_t i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        const unsigned long long key = score_key(F[i]);
        gt += key > T;
        eq += key == T;
    }
    atomicAdd(&s_gt, gt);
    atomicAdd(&s_eq, eq);
    __syncthreads();
    if (threadIdx.x == 0) {
        bsum[2 * blockIdx.x] = s_gt;
        bsum[2 * blockIdx.x + 1] = s_eq;
    }
}

// exclusive scan of the per-block counts (one CTA, blocks <= 1024)
__global__ void __launch_bounds__(1024) k_trunc_scan(int32_t* __restrict__ bsum, int32_t blocks) {
    grid_dependency_wait();  // launched as a programmatic dependent: only the launch latency overlaps
    __shared__ int32_t sg[1024], se[1024];
    const int t = threadIdx.x;
    sg[t] = t < blocks ? bsum[2 * t] : 0;
    se[t] = t < blocks ? bsum[2 * t + 1] : 0;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        const int32_t a = t >= off ? sg[t - off] : 0, b = t >= off ? se[t - off] : 0;
        __syncthreads();
        sg[t] += a;
        se[t] += b;
        __syncthreads();
    }
    if (t < blocks) {
        bsum[2 * t] = sg[t] - (t < blocks ? bsum[2 * t] : 0);      // exclusive
        bsum[2 * t + 1] = se[t] - (t < blocks ? bsum[2 * t + 1] : 0);
    }
}

// kept[p] = row of the p-th survivor (rows ascending): p = (#above before row) + min(#ties before row, quota)
__global__ void __launch_bounds__(256) k_trunc_place(const double* __restrict__ F, int32_t n, int32_t per_block,
                                                     const TruncPick* __restrict__ pick,
                                                     const int32_t* __restrict__ bsum, int32_t* __restrict__ kept) {
    grid_dependency_wait();  // launched as a programmatic dependent: only the launch latency overlaps
    __shared__ int32_t tg[256], te[256];
    const unsigned long long T = pick->key;
    const int32_t quota = pick->quota;
    const int32_t lo = blockIdx.x * per_block, hi = min(n, lo + per_block);
    const int32_t per_thread = per_block / 256;  // per_block is a multiple of 256
    const int32_t mylo = lo + threadIdx.x * per_thread, myhi = min(hi, mylo + per_thread);
    int32_t gt = 0, eq = 0;
    for (int32_t i = mylo; i < myhi; ++i) {
        const unsigned long long key = score_key(F[i]);
        gt += key > T;
        eq += key == T;
    }
    tg[threadIdx.x] = gt;
    te[threadIdx.x] = eq;
    __syncthreads();
    for (int off = 1; off < 256; off <<= 1) {
        const int32_t a = (int)threadIdx.x >= off ? tg[threadIdx.x - off] : 0;
        const int32_t b = (int)threadIdx.x >= off ? te[threadIdx.x - off] : 0;
        __syncthreads();
        tg[threadIdx.x] += a;
        te[threadIdx.x] += b;
        __syncthreads();
    }
    int32_t g_before = bsum[2 * blockIdx.x] + tg[threadIdx.x] - gt;
    int32_t e_before = bsum[2 * blockIdx.x + 1] + te[threadIdx.x] - eq;
    for (int32_t i = mylo; i < myhi; ++i) {
        const unsigned long long key = score_key(F[i]);
        if (key > T) {
            kept[g_before + min(e_before, quota)] = i;
            ++g_before;
        } else if (key == T) {
            if (e_before < quota) kept[g_before + e_before] = i;
            ++e_before;
        }
    }
}

// The whole threshold search and the survivors' places in ONE launch of one thread-block cluster, for pools of
// up to 16 x 1024 x 16 rows.  Every warp owns a contiguous run of 32 x kpt rows and every thread keeps the keys of
// its (up to 16) rows, 32 apart, in registers, so that scores, GPU counts and the row map are read and written by
// whole warps side by side.  The eight radix passes exchange their 256-bin histograms through distributed shared
// memory (one hardware cluster barrier per pass, the histograms alternating between two buffers; nothing spins);
// a thread remembers which of its keys still match the prefix, and a pass visits only the slots where some lane
// of the warp has one.  Then the counts above / at the threshold are scanned over warps and CTAs (inside a warp a
// ballot gives every row its rank) and every survivor's row is written to kept[] as k_trunc_place does.
// Replaces 11 launches (8 passes, count, scan, place).  With `newmap` the kernel is the whole selection: the pool
// is used in place, logical row -> pool row through a map of n entries; survivors keep their pool rows and become
// logical rows 0..K-1 (in the order of their logical rows, as the scheme asks), the rows given up become the
// places of the next generation's new candidates, and the survivors' scores and GPU counts move to the other
// score arrays.  No candidate row is copied.
// KEYS: rows a thread can hold (1, 4 or 16; the launch takes the smallest that covers the pool, so that small
// pools do not pay for the unrolled slots of large ones).
constexpr int kPickCtas = 16, kPickThreads = 1024, kPickKeys = 16;

template <int KEYS, int NCTA>
__global__ void __launch_bounds__(kPickThreads, 1)
k_trunc_pick_place(const double* __restrict__ F, int32_t n, int32_t k, int32_t* __restrict__ kept,
                   const int32_t* __restrict__ oldmap, int32_t* __restrict__ newmap, const int32_t* __restrict__ G,
                   double* __restrict__ F_new, int32_t* __restrict__ G_new) {
    grid_dependency_release();  // the next generation's CTAs stage their tables on the SMs this cluster leaves free
    grid_dependency_wait();
    cg::cluster_group cluster = cg::this_cluster();
    auto sync_all = [&]() {  // every CTA of the launch
        if (NCTA == 1) __syncthreads();
        else cluster.sync();
    };
    __shared__ unsigned int hist[2][256];  // by pass parity: a histogram is cleared two passes after it was read
    __shared__ unsigned int tot[256];
    __shared__ unsigned long long s_prefix;
    __shared__ int32_t s_remaining;
    __shared__ int32_t s_warp_g[32], s_warp_e[32];
    __shared__ int32_t s_cta[2];  // this CTA's counts above / at the threshold
    const unsigned int rank = cluster.block_rank();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // rows per thread, so that all CTAs share the work whatever the pool's size; the warp's rows are
    // wbase ... wbase + 32 * kpt - 1, slot u of lane l is row wbase + 32 u + l
    constexpr int32_t ncta = NCTA;  // 16, or 1 for small pools (the passes then cost block barriers only)
    const int32_t kpt = (n + ncta * kPickThreads - 1) / (ncta * kPickThreads);
    const int32_t wbase = ((int32_t)rank * (kPickThreads / 32) + warp) * 32 * kpt;
    unsigned long long key[KEYS];
    unsigned int alive = 0u;  // bit u: key u is a row of the pool and still matches the prefix
    // the scores were written throughout the kernel before and have mostly left L2: ask for all of this warp's
    // lines at once (one lane per 128 bytes), and for what the last step reads of the map and the GPU counts
    for (int32_t i = lane; i < kpt * 2; i += 32) {
        const int32_t row = wbase + 16 * i;
        if (row < n) {
            l2_prefetch(reinterpret_cast<const unsigned char*>(F + row));
            if (newmap && !(i & 1)) {
                l2_prefetch(reinterpret_cast<const unsigned char*>(G + row));
                if (oldmap) l2_prefetch(reinterpret_cast<const unsigned char*>(oldmap + row));
            }
        }
    }
#pragma unroll
    for (int u = 0; u < KEYS; ++u) {  // all the loads first, so that they are in flight together
        const int32_t row = wbase + 32 * u + lane;
        const bool have = u < kpt && row < n;
        key[u] = have ? (unsigned long long)__double_as_longlong(F[row]) : 0ull;
        alive |= have ? 1u << u : 0u;
    }
#pragma unroll
    for (int u = 0; u < KEYS; ++u)
        key[u] = ((alive >> u) & 1u) ? score_key(__longlong_as_double((long long)key[u])) : 0ull;
    const unsigned int rows_here = alive;
    unsigned long long prefix = 0ull;
    int32_t remaining = k;
    for (int pass = 0; pass < 8; ++pass) {
        unsigned int* myhist = hist[pass & 1];
        if (threadIdx.x < 256) myhist[threadIdx.x] = 0u;
        __syncthreads();
        const int shift = 56 - 8 * pass;
        const unsigned long long mask = pass == 0 ? 0ull : ~0ull << (shift + 8);
        const unsigned int warp_alive = __reduce_or_sync(0xFFFFFFFFu, alive);
        unsigned int run_digit = 0u, run_count = 0u;  // (uniform) slots in a row whose live keys all share one digit
#pragma unroll
        for (int u = 0; u < KEYS; ++u) {
            if (!((warp_alive >> u) & 1u)) continue;  // uniform: no lane of the warp has a matching key in this slot
            const bool in = ((alive >> u) & 1u) && (key[u] & mask) == prefix;
            if (!in) alive &= ~(1u << u);
            const unsigned int live = __ballot_sync(0xFFFFFFFFu, in);
            if (live == 0u) continue;
            // similar scores share their leading digits: when all live lanes of a slot agree the warp counts in a
            // register and adds once per run of such slots, else one atomic per key (grouping equal digits with a
            // warp match first measured 4 % slower)
            const unsigned int digit = (unsigned int)(key[u] >> shift) & 255u;
            const unsigned int lead = __shfl_sync(0xFFFFFFFFu, digit, __ffs(live) - 1);
            if (__all_sync(0xFFFFFFFFu, !in || digit == lead)) {
                if (lead != run_digit && run_count) {
                    if (lane == 0) atomicAdd(&myhist[run_digit], run_count);
                    run_count = 0u;
                }
                run_digit = lead;
                run_count += (unsigned int)__popc(live);
            } else if (in) {
                atomicAdd(&myhist[digit], 1u);
            }
        }
        if (run_count && lane == 0) atomicAdd(&myhist[run_digit], run_count);
        sync_all();  // every CTA's histogram of this digit is complete
        if (threadIdx.x < 256) {
            unsigned int sum = 0u;
#pragma unroll
            for (unsigned int r = 0; r < (unsigned int)NCTA; ++r) sum += *cluster.map_shared_rank(&myhist[threadIdx.x], r);
            tot[threadIdx.x] = sum;
        }
        __syncthreads();
        if (warp == 0) {
            // the digit that holds the remaining-th best key, bins taken from 255 downwards (every CTA finds the
            // same one): lane l owns the eight bins 255 - 8l ... 248 - 8l
            unsigned int c[8], mine = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                c[i] = tot[255 - (8 * lane + i)];
                mine += c[i];
            }
            unsigned int incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned int a = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += a;
            }
            const unsigned int reached = __ballot_sync(0xFFFFFFFFu, (int32_t)incl >= remaining);
            const int owner = reached ? __ffs(reached) - 1 : 31;
            if (lane == owner) {
                int32_t above = (int32_t)(incl - mine), d = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int32_t bin = 255 - (8 * lane + i);
                    if (bin == 0 || above + (int32_t)c[i] >= remaining) {
                        d = bin;
                        break;
                    }
                    above += (int32_t)c[i];
                }
                s_remaining = remaining - above;
                s_prefix = prefix | ((unsigned long long)d << shift);
            }
        }
        __syncthreads();
        prefix = s_prefix;
        remaining = s_remaining;
        // no second barrier: the other histogram is the one cleared next, and every CTA finished reading it before
        // it arrived at this pass's barrier
    }
    // prefix = key of the k-th best, remaining = how many rows with exactly that key survive (lowest rows first)
    const unsigned long long T = prefix;
    const int32_t quota = remaining;
    // counts above / at the threshold: per warp by ballots, then an exclusive scan over the CTA's warps (rows ascend
    // with the warp index), then over the CTAs
    int32_t wg = 0, we = 0;
#pragma unroll
    for (int u = 0; u < KEYS; ++u) {
        if (u >= kpt) break;  // uniform
        const bool have = (rows_here >> u) & 1u;
        wg += __popc(__ballot_sync(0xFFFFFFFFu, have && key[u] > T));
        we += __popc(__ballot_sync(0xFFFFFFFFu, have && key[u] == T));
    }
    if (lane == 0) {
        s_warp_g[warp] = wg;
        s_warp_e[warp] = we;
    }
    __syncthreads();
    if (warp == 0) {
        int32_t sg = s_warp_g[lane], se = s_warp_e[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t a = __shfl_up_sync(0xFFFFFFFFu, sg, off), b = __shfl_up_sync(0xFFFFFFFFu, se, off);
            if (lane >= off) {
                sg += a;
                se += b;
            }
        }
        s_warp_g[lane] = sg;  // inclusive over warps
        s_warp_e[lane] = se;
        if (lane == 31) {
            s_cta[0] = sg;
            s_cta[1] = se;
        }
    }
    sync_all();  // every CTA's totals are in place
    int32_t g_before = warp > 0 ? s_warp_g[warp - 1] : 0;  // rows of the warps (then CTAs) below this warp
    int32_t e_before = warp > 0 ? s_warp_e[warp - 1] : 0;
#pragma unroll
    for (unsigned int r = 0; r < (unsigned int)NCTA; ++r) {  // unrolled: the remote reads are all in flight at once
        if (r < rank) {
            const int32_t* other = cluster.map_shared_rank(s_cta, r);
            g_before += other[0];
            e_before += other[1];
        }
    }
    const unsigned int below = (1u << lane) - 1u;
    // eight slots at a time: what the slots read of the map and of the GPU counts is loaded first, so that a warp
    // waits for memory twice and not once per slot; a score is taken back from its key where the key has an
    // inverse (not for NaN and zero, whose sign or payload the key does not keep)
    constexpr int BATCH = KEYS < 8 ? KEYS : 8;
#pragma unroll
    for (int h = 0; h < KEYS; h += BATCH) {
        if (h >= kpt) break;  // uniform
        int32_t from[BATCH], gpus[BATCH];
#pragma unroll
        for (int v = 0; v < BATCH; ++v) {
            const int u = h + v;
            const int32_t row = wbase + 32 * u + lane;
            const bool have = (rows_here >> u) & 1u;
            from[v] = (newmap && oldmap && have) ? oldmap[row] : row;
            gpus[v] = (newmap && have && key[u] >= T) ? G[row] : 0;
        }
#pragma unroll
        for (int v = 0; v < BATCH; ++v) {
            const int u = h + v;
            if (u >= kpt) break;  // uniform
            const bool have = (rows_here >> u) & 1u;
            const bool gt = have && key[u] > T, eq = have && key[u] == T;
            const unsigned int bg = __ballot_sync(0xFFFFFFFFu, gt), be = __ballot_sync(0xFFFFFFFFu, eq);
            if (have) {
                const int32_t row = wbase + 32 * u + lane;
                const int32_t eb = e_before + __popc(be & below);
                const int32_t before = g_before + __popc(bg & below) + min(eb, quota);  // survivors among the rows below
                const bool keep = gt || (eq && eb < quota);
                if (newmap) {
                    // pool used in place: the survivor becomes logical row `before`, any other row becomes the
                    // place of a new candidate (logical rows K..n-1, in the order of the rows given up)
                    const int32_t place = keep ? before : k + (row - before);
                    newmap[place] = from[v];
                    if (keep) {
                        const unsigned long long kk = key[u];
                        const bool plain = kk != 0ull && kk != 0x8000000000000000ull;
                        const unsigned long long bits = (kk >> 63) ? kk ^ 0x8000000000000000ull : ~kk;
                        F_new[place] = plain ? __longlong_as_double((long long)bits) : F[row];
                        G_new[place] = gpus[v];
                    }
                } else if (keep) {
                    kept[before] = row;
                }
            }
            g_before += __popc(bg);
            e_before += __popc(be);
        }
    }
    sync_all();  // no CTA leaves while a neighbour may still read its totals
}

// Can the device host that cluster (asked once per device)?
static bool pick_cluster_available() {
    static int state[64] = {};  // 0 unknown, 1 yes, 2 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (state[dev] == 0) {
        int clusters = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kPickCtas, 1, 1);
        cfg.blockDim = dim3(kPickThreads, 1, 1);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kPickCtas;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        bool ok = cudaFuncSetAttribute(k_trunc_pick_place<1, kPickCtas>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
                  cudaFuncSetAttribute(k_trunc_pick_place<4, kPickCtas>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
                  cudaFuncSetAttribute(k_trunc_pick_place<kPickKeys, kPickCtas>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
                  cudaOccupancyMaxActiveClusters(&clusters, k_trunc_pick_place<kPickKeys, kPickCtas>, &cfg) == cudaSuccess && clusters >= 1;
        if (!ok) (void)cudaGetLastError();
        state[dev] = ok ? 1 : 2;
    }
    return state[dev] == 1;
}

// survivors move to rows 0..K-1 of the other pool, with their scores and GPU counts
__global__ void __launch_bounds__(256) k_trunc_gather(const int32_t* __restrict__ src, int32_t* __restrict__ dst,
                                                      int64_t ld, int32_t k, const int32_t* __restrict__ kept,
                                                      const double* __restrict__ F, const int32_t* __restrict__ G,
                                                      double* __restrict__ F_new, int32_t* __restrict__ G_new) {
    grid_dependency_wait();  // launched as a programmatic dependent: only the launch latency overlaps
    const int lane = threadIdx.x & 31;
    const int64_t p = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (p >= k) return;
    const int32_t from = kept[p];
    const int4* S = reinterpret_cast<const int4*>(src + (int64_t)from * ld);
    int4* D = reinterpret_cast<int4*>(dst + p * ld);
    const int32_t nvec = (int32_t)(ld >> 2);
    for (int32_t v = lane; v < nvec; v += 32) D[v] = S[v];
    if (lane == 0 && F_new) {
        F_new[p] = F[from];
        G_new[p] = G[from];
    }
}

size_t trunc_scratch_bytes(int32_t k) {
    return 64 + sizeof(TruncState) + 2 * 1024 * sizeof(int32_t) + (size_t)k * sizeof(int32_t);
}

// Can the selection of the best k of 4k rows run in place (one cluster launch, no row copied)?
bool trunc_inplace_available(int32_t k) {
    return 4 * (int64_t)k <= (int64_t)kPickCtas * kPickThreads * kPickKeys && pick_cluster_available();
}

// Derive the 3K new candidates of one generation into rows K..4K-1 of the pool.  draws: 3K ints.
cudaError_t launch_trunc_children(int32_t* pool, int64_t ld, int32_t k, int32_t* draws, Tables t, RoundKeys keys,
                                  uint64_t gen, uint32_t thr16, cudaStream_t s) {
    const uint32_t thr32 = thr16 >= 65536u ? 0xFFFFFFFFu : thr16 << 16;
    k_trunc_draws<<<(3 * k + 255) / 256, 256, 0, s>>>(k, keys, (uint32_t)gen, counter3(STREAM_SEL_A, gen),
                                                      counter3(STREAM_SEL_B, gen), counter3(STREAM_PICK, gen), draws);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int child_blocks = (int)((2 * (int64_t)k + 7) / 8);
    if (thr16 >= 65536u)
        k_trunc_children<true><<<child_blocks, 256, 0, s>>>(pool, ld, k, draws, t, keys, (uint32_t)gen,
                                                            counter3(STREAM_MUT, gen), counter3(STREAM_MUTANT, gen), thr32);
    else
        k_trunc_children<false><<<child_blocks, 256, 0, s>>>(pool, ld, k, draws, t, keys, (uint32_t)gen,
                                                             counter3(STREAM_MUT, gen), counter3(STREAM_MUTANT, gen), thr32);
    return cudaGetLastError();
}

cudaError_t launch_trunc_children_score(int32_t* pool, int64_t ld, int32_t k, int32_t* draws, Tables t, RoundKeys keys,
                                        uint64_t gen, uint32_t thr16, int32_t capacity, double penalty, double* F,
                                        int32_t* G, const int32_t* rowmap, cudaStream_t s) {
    const size_t smem = evolve_score_smem(t);
    if (smem > (size_t)kMaxSmemPerBlock) return cudaErrorInvalidConfiguration;
    const uint32_t thr32 = thr16 >= 65536u ? 0xFFFFFFFFu : thr16 << 16;
    cudaError_t e;
    constexpr int kThreads = ONES_TC_THREADS;
    int64_t blocks = (2 * (int64_t)k + kThreads / 32 - 1) / (kThreads / 32);
    if (blocks > sm_count()) blocks = sm_count();
    auto kern = thr16 >= 65536u ? k_trunc_children_score<true> : k_trunc_children_score<false>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemPerBlock);
    if (e != cudaSuccess) return e;
    return launch_after_previous(kern, (int)blocks, kThreads, smem, s, pool, ld, k, draws, t, keys, (uint32_t)gen,
                                 counter3(STREAM_SEL_A, gen), counter3(STREAM_SEL_B, gen), counter3(STREAM_PICK, gen),
                                 counter3(STREAM_MUT, gen), counter3(STREAM_MUTANT, gen), thr32, capacity, penalty, F,
                                 G, rowmap);
}

static cudaError_t launch_pick_place(const double* F, int32_t n, int32_t k, int32_t* kept, const int32_t* oldmap,
                                     int32_t* newmap, const int32_t* G, double* F_next, int32_t* G_next, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    // pools of up to 4096 rows: one CTA with up to four rows per thread (the eight passes then cost block barriers
    // only: 27 -> 19 us per selection at 4096 rows, 25 -> 12.5 at 128; with 16 rows per thread one CTA took 61 us
    // where the cluster takes 25); larger ones: the 16-CTA cluster
    const int ncta = n <= kPickThreads * 4 ? 1 : kPickCtas;
    cfg.gridDim = dim3(ncta, 1, 1);
    cfg.blockDim = dim3(kPickThreads, 1, 1);
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ncta;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const int32_t kpt = (n + ncta * kPickThreads - 1) / (ncta * kPickThreads);
    auto kern = ncta == 1 ? (kpt <= 1 ? k_trunc_pick_place<1, 1> : k_trunc_pick_place<4, 1>)
                          : kpt <= 1 ? k_trunc_pick_place<1, kPickCtas>
                                     : kpt <= 4 ? k_trunc_pick_place<4, kPickCtas> : k_trunc_pick_place<kPickKeys, kPickCtas>;
    return cudaLaunchKernelEx(&cfg, kern, F, n, k, kept, oldmap, newmap, G, F_next, G_next);
}

// The selection in place (see k_trunc_pick_place): oldmap (nullptr: logical row = pool row) -> newmap, both of
// 4k entries; F, G: 4k scores and GPU counts by logical row; F_next, G_next receive the survivors'.  One launch.
cudaError_t launch_trunc_select_inplace(int32_t k, const double* F, const int32_t* G, double* F_next, int32_t* G_next,
                                        const int32_t* oldmap, int32_t* newmap, cudaStream_t s) {
    if (!newmap || !trunc_inplace_available(k)) return cudaErrorNotSupported;
    return launch_pick_place(F, 4 * k, k, nullptr, oldmap, newmap, G, F_next, G_next, s);
}

// Logical rows 0..k-1 of a pool used in place, copied in order to rows 0..k-1 of pool_next.
cudaError_t launch_trunc_compact(const int32_t* pool, int32_t* pool_next, int64_t ld, int32_t k, const int32_t* rowmap,
                                 cudaStream_t s) {
    k_trunc_gather<<<(k + 7) / 8, 256, 0, s>>>(pool, pool_next, ld, k, rowmap, nullptr, nullptr, nullptr, nullptr);
    return cudaGetLastError();
}

// Keep the best K of the 4K scored rows: F, G hold 4K entries; the survivors become rows 0..K-1 of
// pool_next with F_next, G_next.  2 launches for pools of up to 262144 rows, 12 beyond.
cudaError_t launch_trunc_select(const int32_t* pool, int32_t* pool_next, int64_t ld, int32_t k, const double* F,
                                const int32_t* G, double* F_next, int32_t* G_next, void* scratch, cudaStream_t s,
                                int* launches) {
    const int32_t n = 4 * k;
    if (launches) *launches = 12;
    const int32_t per_block = ((n + 1023) / 1024 + 255) / 256 * 256;  // rows per block: multiple of 256, <= 1024 blocks
    const int32_t blocks = (n + per_block - 1) / per_block;
    TruncPick* pick = reinterpret_cast<TruncPick*>(scratch);
    TruncState* state = reinterpret_cast<TruncState*>(reinterpret_cast<char*>(scratch) + 64);
    int32_t* bsum = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(scratch) + 64 + sizeof(TruncState));
    int32_t* kept = bsum + 2 * 1024;
    cudaError_t e;
    if (n <= kPickCtas * kPickThreads * kPickKeys && pick_cluster_available()) {
        // threshold search and places in one cluster launch, then the gather
        e = launch_pick_place(F, n, k, kept, nullptr, nullptr, nullptr, nullptr, nullptr, s);
        if (e != cudaSuccess) return e;
        if (launches) *launches = 2;
        return launch_after_previous(k_trunc_gather, (k + 7) / 8, 256, 0, s, pool, pool_next, ld, k, (const int32_t*)kept,
                                     F, G, F_next, G_next);
    }
    int rb = (n + 2047) / 2048;
    if (rb > sm_count()) rb = sm_count();
    for (int pass = 0; pass < 8; ++pass) {
        e = launch_after_previous(k_trunc_radix_pass, rb, 256, 0, s, F, n, k, pass, state, pick);
        if (e != cudaSuccess) return e;
    }
    e = launch_after_previous(k_trunc_count, blocks, 256, 0, s, F, n, per_block, (const TruncPick*)pick, bsum);
    if (e != cudaSuccess) return e;
    e = launch_after_previous(k_trunc_scan, 1, 1024, 0, s, bsum, blocks);
    if (e != cudaSuccess) return e;
    e = launch_after_previous(k_trunc_place, blocks, 256, 0, s, F, n, per_block, (const TruncPick*)pick,
                              (const int32_t*)bsum, kept);
    if (e != cudaSuccess) return e;
    return launch_after_previous(k_trunc_gather, (k + 7) / 8, 256, 0, s, pool, pool_next, ld, k, (const int32_t*)kept, F,
                                 G, F_next, G_next);
}

// ---------------------------------------------------------------------------------------------
// The paper's own genome (Eq. 1-2, Fig. 1): one slot per GPU holding a job id (anything outside
// [0, n_jobs) = idle).  Job j holds c_j = the number of its slots and runs at the largest exponent in
// [kmin_j, kmax_j] whose GPU need g_j(k) fits into c_j; with none it waits.  Scores are summed over jobs
// in the same fixed order as everywhere else.
// ---------------------------------------------------------------------------------------------
// per job: the exponent it can run at on `count` GPUs (-1: waits).  g_j(k) does not decrease with k, so
// the search stops at the first exponent that needs more GPUs than the job holds.
__device__ __forceinline__ int32_t exponent_that_fits(const Tables& t, int32_t j, int32_t count) {
    const int32_t lo = t.kmin[j], hi = lo + t.range[j] - 1;
    const int32_t at = slot_of(j);
    int32_t best = -1;
    for (int32_t k = lo; k <= hi; ++k) {
        if (t.G[(int64_t)k * t.jpad + at] > count) break;
        best = k;
    }
    return best;
}

// The same from the job's own limits, without the table: ceil((b0 << k) / m) <= count exactly when
// (b0 << k) <= count * m, so the largest such k is floor(log2(count * m / b0)), found from the leading bits.
__device__ __forceinline__ int32_t exponent_that_fits(int32_t b0, int32_t m, int32_t kmin, int32_t kmax, int32_t count) {
    const unsigned long long room = (unsigned long long)count * (unsigned long long)m;
    if (room < (unsigned long long)b0) return -1;
    int32_t k = (63 - __clzll((long long)room)) - (31 - __clz(b0));
    if (((unsigned long long)b0 << k) > room) --k;
    k = min(k, kmax);
    return k >= kmin ? k : -1;
}

// The same in 32-bit arithmetic, for clusters with count * max_per_gpu < 2^31 for every job.
__device__ __forceinline__ int32_t exponent_that_fits32(int32_t b0, int32_t m, int32_t kmin, int32_t kmax, int32_t count) {
    const uint32_t room = (uint32_t)count * (uint32_t)m;
    if (room < (uint32_t)b0) return -1;
    int32_t k = __clz(b0) - __clz((int32_t)room);
    if (((uint32_t)b0 << k) > room) --k;
    k = min(k, kmax);
    return k >= kmin ? k : -1;
}

// Per-job terms of one per-GPU candidate from its job counts (shared memory), 256 threads.  A thread
// takes jobs 4v..4v+3: their counts are one int4, and for each of the four the lanes of a warp read
// neighbouring entries of the limits and of the model tables (the tables' job order).  Returns the GPUs used.
template <bool NARROW = false>
__device__ __forceinline__ int32_t per_gpu_terms(const int32_t* __restrict__ count, double* __restrict__ term,
                                                 int32_t jpad4, const Tables& t, const int4* __restrict__ fit) {
    int32_t used = 0;
    for (int32_t v0 = threadIdx.x; 4 * v0 < jpad4; v0 += 2 * 256) {
        // eight jobs per step: all their limits first, then all their table entries, so the loads overlap
        int32_t c[8], at[8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int32_t v = v0 + 256 * h;
            int4 cnt = make_int4(0, 0, 0, 0);
            if (4 * v < jpad4) cnt = *reinterpret_cast<const int4*>(count + 4 * v);
            c[4 * h + 0] = cnt.x; c[4 * h + 1] = cnt.y; c[4 * h + 2] = cnt.z; c[4 * h + 3] = cnt.w;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int32_t v = v0 + 256 * (e >> 2);
            const int32_t entry = ((4 * v) & ~127) + (v & 31) + 32 * (e & 3);
            at[e] = -1;
            if (c[e] > 0) {
                const int4 q = __ldg(fit + entry);  // b0, max_per_gpu, kmin, kmax
                const int32_t k = NARROW ? exponent_that_fits32(q.x, q.y, q.z, q.w, c[e])
                                         : exponent_that_fits(q.x, q.y, q.z, q.w, c[e]);
                if (k >= 0) at[e] = k * t.jpad + entry;
            }
        }
        double x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            x[e] = 0.0;
            if (at[e] >= 0) {
                x[e] = __ldg(t.X + at[e]);
                used += __ldg(t.G + at[e]);
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int32_t v = v0 + 256 * h;
            if (4 * v < jpad4)
                *reinterpret_cast<double4*>(term + 4 * v) = make_double4(x[4 * h], x[4 * h + 1], x[4 * h + 2], x[4 * h + 3]);
        }
    }
    return used;
}

// Count the GPUs of every job in one row held in shared memory.  A thread walks a contiguous piece of
// the row and adds a whole run of equal ids at once: after "Reorder" the workers of a job are neighbours,
// so one atomic per run instead of one per GPU.  FIRST also records each job's first slot.
template <bool FIRST>
__device__ __forceinline__ void count_runs(const int32_t* __restrict__ rowbuf, int32_t from, int32_t to, int32_t n_jobs,
                                           int32_t* __restrict__ count, int32_t* __restrict__ first) {
    int32_t run_id = -1, run_len = 0, run_at = 0;
    for (int32_t i = from; i < to; ++i) {
        const int32_t id = rowbuf[i];
        if (id != run_id) {
            if (run_id >= 0) {
                atomicAdd(&count[run_id], run_len);
                if (FIRST) atomicMin(&first[run_id], run_at);
            }
            run_id = (uint32_t)id < (uint32_t)n_jobs ? id : -1;
            run_len = 0;
            run_at = i;
        }
        ++run_len;
    }
    if (run_id >= 0) {
        atomicAdd(&count[run_id], run_len);
        if (FIRST) atomicMin(&first[run_id], run_at);
    }
}

// Per-GPU candidates, one CTA per candidate.  SCORE: the candidate's fitness and GPU demand from the
// job counts.  REORDER: the row rewritten with every job's workers side by side, jobs in order of first
// occurrence, idle GPUs last; the counts do not change, so both come from one counting pass.
// Shared memory: count[J] | first[J] start[J] (later the per-job terms, fp64) | the row.
template <bool REORDER, bool SCORE>
__global__ void __launch_bounds__(256)
k_per_gpu(int32_t* __restrict__ slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, Tables t,
          const int4* __restrict__ fit, double* __restrict__ F, int32_t* __restrict__ G) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int32_t s_warp[8];
    __shared__ int32_t s_used;
    const int32_t jpad4 = (n_jobs + 3) & ~3;
    int32_t* count = reinterpret_cast<int32_t*>(smem_raw);
    int32_t* first = count + jpad4;
    int32_t* start = first + jpad4;
    double* term = reinterpret_cast<double*>(first);
    int32_t* rowbuf = start + jpad4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t piece = ((n_gpus + 255) / 256) | 1;  // odd: neighbouring threads' pieces start in different banks
    const int32_t from = min(n_gpus, tid * piece), to = min(n_gpus, (tid + 1) * piece);
    for (int64_t cand = blockIdx.x; cand < n; cand += gridDim.x) {
        int32_t* row = slots + cand * ld;
        for (int32_t j = tid; j < n_jobs; j += 256) {
            count[j] = 0;
            if (REORDER) first[j] = 0x7FFFFFFF;
        }
        if (tid == 0) s_used = 0;
        for (int32_t i = tid; i < n_gpus; i += 256) rowbuf[i] = row[i];
        __syncthreads();
        count_runs<REORDER>(rowbuf, from, to, n_jobs, count, first);
        __syncthreads();
        if (REORDER) {
            // a job's run starts where the runs of the jobs that occurred earlier end: scan over the slots
            int32_t mine = 0;
            for (int32_t i = from; i < to; ++i) {
                const int32_t id = rowbuf[i];
                if ((uint32_t)id < (uint32_t)n_jobs && first[id] == i) mine += count[id];
            }
            int32_t incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += up;
            }
            if (lane == 31) s_warp[warp] = incl;
            __syncthreads();
            int32_t offset = incl - mine, total = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                const int32_t v = s_warp[w];
                if (w < warp) offset += v;
                total += v;
            }
            for (int32_t i = from; i < to; ++i) {
                const int32_t id = rowbuf[i];
                if ((uint32_t)id < (uint32_t)n_jobs && first[id] == i) {
                    start[id] = offset;
                    offset += count[id];
                }
            }
            __syncthreads();
            // fill: job j occupies [start, start + count); idle GPUs after the last run
            for (int32_t i = total + tid; i < n_gpus; i += 256) rowbuf[i] = -1;
            for (int32_t j = tid; j < n_jobs; j += 256) {
                const int32_t c = count[j];
                if (c > 0) {
                    const int32_t s0 = start[j];
                    for (int32_t u = 0; u < c; ++u) rowbuf[s0 + u] = j;
                }
            }
            __syncthreads();
            for (int32_t i = tid; i < n_gpus; i += 256) row[i] = rowbuf[i];
        }
        if (SCORE) {
            int32_t used = per_gpu_terms(count, term, jpad4, t, fit);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) used += __shfl_xor_sync(0xFFFFFFFFu, used, off);
            if (lane == 0 && used) atomicAdd(&s_used, used);
            __syncthreads();
            if (warp == 0) {
                // fixed summation order: lane l adds jobs 4l..4l+3 of every block of 128 jobs in turn,
                // then the 32 partial sums pairwise; a waiting job adds +0.0, which changes nothing
                double sum = 0.0;
                for (int32_t v = lane; 4 * v < jpad4; v += 32) {
                    const double4 q = *reinterpret_cast<const double4*>(term + 4 * v);
                    sum = __dadd_rn(__dadd_rn(__dadd_rn(__dadd_rn(sum, q.x), q.y), q.z), q.w);
                }
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
                if (lane == 0) {
                    F[cand] = sum;
                    if (G) G[cand] = s_used;
                }
            }
        }
        __syncthreads();
    }
}

// The same for rows of at most 256 * PIECE slots: every thread keeps its PIECE neighbouring slots in
// registers, so the row is read once from global memory and walked without loops over shared memory.
// RUNS: a thread adds a whole run of equal ids at once (few jobs on many GPUs: long runs, where one atomic
// per slot would hit the same counter from every lane); otherwise one atomic per slot (after crossover the
// runs are one or two slots long and the run bookkeeping costs more instructions than it saves).
// Reorder: the first slot of every job learns where the job's run starts (exclusive scan, over the slots, of
// the GPU counts of the jobs that start there) and leaves it in first[]; then every slot (or run) takes its
// place in the job's run with one atomic add on that cursor, so no thread loops over a job's whole run.
// NARROW: the exponent search in 32-bit arithmetic.
// Shared memory: count[J] | first[J] | the reordered row, later the per-job terms (fp64).
template <int PIECE, bool REORDER, bool SCORE, bool RUNS, bool NARROW>
__global__ void __launch_bounds__(256, 4)
k_per_gpu_regs(int32_t* __restrict__ slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, Tables t,
               const int4* __restrict__ fit, double* __restrict__ F, int32_t* __restrict__ G) {
    static_assert(PIECE % 4 == 0, "a thread's slots are whole int4");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int32_t s_warp[8];
    __shared__ int32_t s_used;
    const int32_t jpad4 = (n_jobs + 3) & ~3;
    int32_t* count = reinterpret_cast<int32_t*>(smem_raw);
    int32_t* first = count + jpad4;
    int32_t* out = first + jpad4;
    double* term = reinterpret_cast<double*>(out);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t from = tid * PIECE;
    int32_t id[PIECE];
    // this thread's slots of one row (rows are padded to int4); the next row is fetched while the current
    // one is still being worked on
    auto fetch = [&](int64_t cand) {
        const int32_t* src = slots + cand * ld + from;
#pragma unroll
        for (int q = 0; q < PIECE / 4; ++q) {
            int4 v = make_int4(-1, -1, -1, -1);
            if (from + 4 * q < n_gpus) v = __ldcs(reinterpret_cast<const int4*>(src + 4 * q));
            id[4 * q + 0] = v.x; id[4 * q + 1] = v.y; id[4 * q + 2] = v.z; id[4 * q + 3] = v.w;
        }
    };
    if (blockIdx.x < n) fetch(blockIdx.x);
    for (int64_t cand = blockIdx.x; cand < n; cand += gridDim.x) {
        int32_t* row = slots + cand * ld;
#pragma unroll
        for (int u = 0; u < PIECE; ++u)
            if (from + u >= n_gpus || (uint32_t)id[u] >= (uint32_t)n_jobs) id[u] = -1;  // idle
        for (int32_t j = 4 * tid; j < jpad4; j += 4 * 256) {
            *reinterpret_cast<int4*>(count + j) = make_int4(0, 0, 0, 0);
            if (REORDER) *reinterpret_cast<int4*>(first + j) = make_int4(0x7FFFFFFF, 0x7FFFFFFF, 0x7FFFFFFF, 0x7FFFFFFF);
        }
        if (tid == 0) s_used = 0;
        __syncthreads();
        if (RUNS) {  // one atomic per run of equal ids
            int32_t run_id = -1, run_len = 0, run_at = 0;
#pragma unroll
            for (int u = 0; u <= PIECE; ++u) {
                const int32_t v = u < PIECE ? id[u] : -2;
                if (v != run_id) {
                    if (run_id >= 0) {
                        atomicAdd(&count[run_id], run_len);
                        if (REORDER) atomicMin(&first[run_id], run_at);
                    }
                    run_id = v;
                    run_len = 0;
                    run_at = from + u;
                }
                ++run_len;
            }
        } else {
#pragma unroll
            for (int u = 0; u < PIECE; ++u)
                if (id[u] >= 0) {
                    atomicAdd(&count[id[u]], 1);
                    if (REORDER) atomicMin(&first[id[u]], from + u);
                }
        }
        __syncthreads();
        if (REORDER) {
            // a job's run starts where the runs of the jobs that occurred earlier end: scan over the slots
            int32_t c[PIECE];
            int32_t mine = 0;
#pragma unroll
            for (int u = 0; u < PIECE; ++u) {
                c[u] = 0;
                if (id[u] >= 0 && first[id[u]] == from + u) c[u] = count[id[u]];
                mine += c[u];
            }
            int32_t incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += up;
            }
            if (lane == 31) s_warp[warp] = incl;
            __syncthreads();  // every thread has read first[] by now: it becomes the jobs' write cursors
            int32_t offset = incl - mine, total = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                const int32_t v = s_warp[w];
                if (w < warp) offset += v;
                total += v;
            }
#pragma unroll
            for (int u = 0; u < PIECE; ++u)
                if (c[u] > 0) {
                    first[id[u]] = offset;
                    offset += c[u];
                }
            for (int32_t i = total + tid; i < n_gpus; i += 256) out[i] = -1;  // idle GPUs last
            __syncthreads();
            if (RUNS) {
                int32_t run_id = -1, run_len = 0;
#pragma unroll
                for (int u = 0; u <= PIECE; ++u) {
                    const int32_t v = u < PIECE ? id[u] : -2;
                    if (v != run_id) {
                        if (run_id >= 0) {
                            const int32_t dest = atomicAdd(&first[run_id], run_len);
                            for (int32_t r = 0; r < run_len; ++r) out[dest + r] = run_id;
                        }
                        run_id = v;
                        run_len = 0;
                    }
                    ++run_len;
                }
            } else {
#pragma unroll
                for (int u = 0; u < PIECE; ++u)
                    if (id[u] >= 0) out[atomicAdd(&first[id[u]], 1)] = id[u];
            }
            if (cand + gridDim.x < n) fetch(cand + gridDim.x);
            __syncthreads();
            for (int32_t i = 4 * tid; i < n_gpus; i += 4 * 256) {
                if (i + 3 < n_gpus) {
                    *reinterpret_cast<int4*>(row + i) = *reinterpret_cast<const int4*>(out + i);
                } else {
                    for (int32_t r = i; r < n_gpus; ++r) row[r] = out[r];
                }
            }
            if (SCORE) __syncthreads();  // the terms take the row's place
        }
        if (!REORDER && cand + gridDim.x < n) fetch(cand + gridDim.x);
        if (SCORE) {
            int32_t used = per_gpu_terms<NARROW>(count, term, jpad4, t, fit);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) used += __shfl_xor_sync(0xFFFFFFFFu, used, off);
            if (lane == 0 && used) atomicAdd(&s_used, used);
            __syncthreads();
            if (warp == 0) {
                // fixed summation order: lane l adds jobs 4l..4l+3 of every block of 128 jobs in turn,
                // then the 32 partial sums pairwise; a waiting job adds +0.0, which changes nothing
                double sum = 0.0;
                for (int32_t v = lane; 4 * v < jpad4; v += 32) {
                    const double4 q = *reinterpret_cast<const double4*>(term + 4 * v);
                    sum = __dadd_rn(__dadd_rn(__dadd_rn(__dadd_rn(sum, q.x), q.y), q.z), q.w);
                }
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
                if (lane == 0) {
                    F[cand] = sum;
                    if (G) G[cand] = s_used;
                }
            }
        }
        __syncthreads();
    }
}

static size_t per_gpu_regs_smem(int32_t n_gpus, int32_t n_jobs) {
    const size_t jpad4 = (size_t)((n_jobs + 3) & ~3), wpad = (size_t)((n_gpus + 3) & ~3);
    const size_t tail = wpad * 4 > jpad4 * 8 ? wpad * 4 : jpad4 * 8;
    return 2 * jpad4 * 4 + tail;
}

template <int PIECE, bool REORDER, bool SCORE, bool RUNS, bool NARROW>
static cudaError_t launch_per_gpu_regs_t(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, Tables t,
                                         const int4* fit, double* F, int32_t* G, cudaStream_t s) {
    const size_t smem = per_gpu_regs_smem(n_gpus, n_jobs);
    cudaError_t e = cudaFuncSetAttribute(k_per_gpu_regs<PIECE, REORDER, SCORE, RUNS, NARROW>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int64_t blocks = n;
    if (blocks > (int64_t)sm_count() * 8) blocks = (int64_t)sm_count() * 8;
    k_per_gpu_regs<PIECE, REORDER, SCORE, RUNS, NARROW><<<(int)blocks, 256, smem, s>>>(slots, ld, n, n_gpus, n_jobs, t, fit,
                                                                                        F, G);
    return cudaGetLastError();
}

template <int PIECE, bool REORDER, bool SCORE>
static cudaError_t launch_per_gpu_regs(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, Tables t,
                                       const int4* fit, bool narrow, double* F, int32_t* G, cudaStream_t s) {
    // long runs of equal ids when a job holds many GPUs on average
    const bool runs = (int64_t)n_gpus >= 8 * (int64_t)n_jobs;
    narrow = narrow && SCORE;
    if (runs)
        return narrow ? launch_per_gpu_regs_t<PIECE, REORDER, SCORE, true, SCORE>(slots, ld, n, n_gpus, n_jobs, t, fit, F, G, s)
                      : launch_per_gpu_regs_t<PIECE, REORDER, SCORE, true, false>(slots, ld, n, n_gpus, n_jobs, t, fit, F, G, s);
    return narrow ? launch_per_gpu_regs_t<PIECE, REORDER, SCORE, false, SCORE>(slots, ld, n, n_gpus, n_jobs, t, fit, F, G, s)
                  : launch_per_gpu_regs_t<PIECE, REORDER, SCORE, false, false>(slots, ld, n, n_gpus, n_jobs, t, fit, F, G, s);
}

static size_t per_gpu_smem(int32_t n_gpus, int32_t n_jobs) {
    return ((size_t)3 * ((n_jobs + 3) & ~3) + n_gpus) * 4;
}

template <bool REORDER, bool SCORE>
static cudaError_t launch_per_gpu(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, Tables t,
                                  const int4* fit, bool narrow, double* F, int32_t* G, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    if (per_gpu_regs_smem(n_gpus, n_jobs) <= (size_t)kMaxSmemPerBlock - 2048) {
        if (n_gpus <= 256 * 4) return launch_per_gpu_regs<4, REORDER, SCORE>(slots, ld, n, n_gpus, n_jobs, t, fit, narrow, F, G, s);
        if (n_gpus <= 256 * 16) return launch_per_gpu_regs<16, REORDER, SCORE>(slots, ld, n, n_gpus, n_jobs, t, fit, narrow, F, G, s);
    }
    const size_t smem = per_gpu_smem(n_gpus, n_jobs);
    if (smem > (size_t)kMaxSmemPerBlock - 2048) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(k_per_gpu<REORDER, SCORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int64_t blocks = n;
    if (blocks > (int64_t)sm_count() * 8) blocks = (int64_t)sm_count() * 8;
    k_per_gpu<REORDER, SCORE><<<(int)blocks, 256, smem, s>>>(slots, ld, n, n_gpus, n_jobs, t, fit, F, G);
    return cudaGetLastError();
}

cudaError_t launch_fitness_per_gpu(const int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs,
                                   Tables t, const int4* fit, bool narrow, double* F, int32_t* G, cudaStream_t s) {
    return launch_per_gpu<false, true>(const_cast<int32_t*>(slots), ld, n, n_gpus, n_jobs, t, fit, narrow, F, G, s);
}

cudaError_t launch_reorder(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, cudaStream_t s) {
    Tables none{};
    return launch_per_gpu<true, false>(slots, ld, n, n_gpus, n_jobs, none, nullptr, false, nullptr, nullptr, s);
}

cudaError_t launch_reorder_score(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_jobs, Tables t,
                                 const int4* fit, bool narrow, double* F, int32_t* G, cudaStream_t s) {
    return launch_per_gpu<true, true>(slots, ld, n, n_gpus, n_jobs, t, fit, narrow, F, G, s);
}

// admissible values of a slot: any job id (kmin 0, range n_jobs), for the shared operators; and the
// jobs' limits (b0, max_per_gpu, kmin, kmax) in the model tables' job order, for the exponent search
__global__ void k_fill_slot_limits(int32_t* __restrict__ kmin, int32_t* __restrict__ range, int32_t len, int32_t n_gpus,
                                   int32_t n_jobs, const ones_job* __restrict__ jobs, int4* __restrict__ fit, int32_t jpad) {
    for (int32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < len; i += gridDim.x * blockDim.x) {
        kmin[i] = 0;
        range[i] = i < n_gpus ? n_jobs : 1;
    }
    for (int32_t j = blockIdx.x * blockDim.x + threadIdx.x; j < jpad; j += gridDim.x * blockDim.x) {
        int4 q = make_int4(1, 1, 1, 0);  // no job: no exponent fits
        if (j < n_jobs) q = make_int4(jobs[j].b0, jobs[j].max_per_gpu, jobs[j].kmin, jobs[j].kmax);
        fit[slot_of(j)] = q;
    }
}

cudaError_t launch_fill_slot_limits(int32_t* kmin, int32_t* range, int32_t len, int32_t n_gpus, int32_t n_jobs,
                                    const ones_job* jobs, int4* fit, int32_t jpad, cudaStream_t s) {
    const int32_t most = len > jpad ? len : jpad;
    k_fill_slot_limits<<<(most + 255) / 256, 256, 0, s>>>(kmin, range, len, n_gpus, n_jobs, jobs, fit, jpad);
    return cudaGetLastError();
}

// best candidate of a per-GPU population as per-job exponents (one CTA); work: n_jobs counters
__global__ void __launch_bounds__(256)
k_best_per_gpu(const int32_t* __restrict__ pop, int64_t ld, int32_t n_gpus, int32_t n_jobs,
               const int32_t* __restrict__ best_index, Tables t, int32_t* __restrict__ work,
               int32_t* __restrict__ genome_out, int32_t* __restrict__ gpus_out, double* __restrict__ rate_out,
               BestOut* __restrict__ out) {
    const int32_t best = best_index[0];
    const int32_t* row = pop + (int64_t)best * ld;
    for (int32_t j = threadIdx.x; j < n_jobs; j += blockDim.x) work[j] = 0;
    __syncthreads();
    for (int32_t i = threadIdx.x; i < n_gpus; i += blockDim.x) {
        const int32_t id = row[i];
        if ((uint32_t)id < (uint32_t)n_jobs) atomicAdd(&work[id], 1);
    }
    __syncthreads();
    for (int32_t j = threadIdx.x; j < n_jobs; j += blockDim.x) {
        const int32_t k = exponent_that_fits(t, j, work[j]);
        const int64_t at = (int64_t)(k >= 0 ? k : t.k1) * t.jpad + slot_of(j);
        genome_out[j] = k;
        gpus_out[j] = t.G[at];
        rate_out[j] = t.X[at];
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        double sum = 0.0;
        int32_t used = 0;
        const int32_t nvec = (n_jobs + 3) >> 2;
        for (int32_t v = lane; v < nvec; v += 32)
            for (int s = 0; s < 4; ++s) {
                const int32_t j = 4 * v + s;
                if (j < n_jobs) {
                    sum = __dadd_rn(sum, rate_out[j]);
                    used += gpus_out[j];
                }
            }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
            used += __shfl_xor_sync(0xFFFFFFFFu, used, off);
        }
        if (lane == 0) {
            out->fitness = sum;
            out->total_gpus = used;
            out->index = best;
            out->status = 0;
            out->steps = 0;
        }
    }
}

cudaError_t launch_best_per_gpu(const int32_t* pop, int64_t ld, int32_t n_gpus, int32_t n_jobs, const int32_t* best_index,
                                Tables t, int32_t* work, int32_t* genome_out, int32_t* gpus_out, double* rate_out,
                                BestOut* out, cudaStream_t s) {
    k_best_per_gpu<<<1, 256, 0, s>>>(pop, ld, n_gpus, n_jobs, best_index, t, work, genome_out, gpus_out, rate_out, out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// "Refresh" of per-GPU candidates when the job set changes (Section 3.2.2, Fig. 5), one CTA per candidate:
//   (1) GPUs of finished jobs become idle, surviving jobs take their new ids (inv[old id] = new id or -1);
//   (2) a job holding more GPUs than its batch-size limit needs gives up the surplus, last GPUs first;
//   (3) every new job, in index order, gets the GPUs of its smallest batch: the lowest idle GPUs, and once
//       none is idle the last GPU of the lowest-index surviving job that still holds one;
//   (4) the idle GPUs that remain go to the jobs below their limit in the order of the score they would
//       gain by growing to it (ties: lower index), each taking what it needs for that, lowest GPUs first.
// Each step is a sequential rule; here every GPU slot decides on its own from three numbers: its rank among
// the slots of its job (which of them are "last"), its rank among the idle slots (which are "lowest"), and
// prefix sums over the jobs in the order they are served ("unit" u of step (3) belongs to the new job whose
// range of the running sum of smallest-batch needs holds u; units beyond the idle GPUs are taken from the
// surviving jobs in index order, each job's GPUs from its last one down).  Step (4) serves every job at most
// once and a job's gain does not change while others are served, so it is one sort by gain.
// The row is not packed here: "Reorder" runs afterwards.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kScanSat = 1u << 30;  // prefix sums saturate here (far above any GPU count)

__device__ __forceinline__ int32_t sat_add(int32_t a, int32_t b) {
    return (int32_t)min((uint32_t)a + (uint32_t)b, kScanSat);
}

// Exclusive prefix sums of the non-negative a[0..n) in shared memory, in place, by a block of 256 threads;
// returns the total to every thread.
__device__ int32_t block_scan_excl(int32_t* __restrict__ a, int32_t n, int32_t* __restrict__ s_warp) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t chunk = ((n + 255) / 256) | 1;
    const int32_t from = min(n, tid * chunk), to = min(n, from + chunk);
    int32_t mine = 0;
    for (int32_t i = from; i < to; ++i) mine = sat_add(mine, a[i]);
    int32_t incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl = sat_add(incl, up);
    }
    int32_t excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
    if (lane == 0) excl = 0;
    __syncthreads();
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int32_t offset = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        const int32_t v = s_warp[w];
        if (w < warp) offset = sat_add(offset, v);
        total = sat_add(total, v);
    }
    int32_t run = sat_add(offset, excl);
    for (int32_t i = from; i < to; ++i) {
        const int32_t v = a[i];
        a[i] = run;
        run = sat_add(run, v);
    }
    __syncthreads();
    return total;
}

// largest p in [0, n) with a[p] <= v, for non-decreasing a with a[0] <= v
__device__ __forceinline__ int32_t last_at_most(const int32_t* __restrict__ a, int32_t n, int32_t v) {
    int32_t lo = 0, hi = n;
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (a[mid] <= v) lo = mid; else hi = mid;
    }
    return lo;
}

// Order of service in step (4): larger gain first, lower job index on equal gains
__device__ __forceinline__ bool served_first(double ga, int32_t ja, double gb, int32_t jb) {
    return ga > gb || (ga == gb && ja < jb);
}

// Bitonic sort of 256 * PER (gain, job) records in shared memory into the order of service, by a block of
// 256 threads.  Thread t keeps records PER*t .. PER*t + PER-1 in registers: steps at distance < PER are
// compare-exchanges between its own registers, steps at distance < 32 * PER exchange with another lane of
// the warp by shuffles, and only the remaining steps (6 of 66 for 2048 records) go through shared memory,
// stored transposed (record r of thread t at r * 256 + t) so that lanes touch neighbouring words.
// The job indices are distinct, so of two records exactly one is served first.
template <int PER>
__device__ void block_sort_service_order(double* __restrict__ key, int32_t* __restrict__ who) {
    static_assert(PER >= 2 && (PER & (PER - 1)) == 0, "at least two records per thread, a power of two");
    const int tid = threadIdx.x;
    constexpr int32_t n = 256 * PER;
    double g[PER];
    int32_t w[PER];
#pragma unroll
    for (int r = 0; r < PER; ++r) {
        g[r] = key[PER * tid + r];
        w[r] = who[PER * tid + r];
    }
    for (int32_t k = 2; k <= n; k <<= 1) {
        // in the run of k records that holds position s the lower half keeps the records served first
        // when (s & k) == 0, the upper half otherwise
        for (int32_t d = k >> 1; d >= PER; d >>= 1) {
            const int32_t hop = d / PER;  // the partner record sits in thread t ^ hop, same register
            if (hop >= 32) {
                __syncthreads();
#pragma unroll
                for (int r = 0; r < PER; ++r) {
                    key[r * 256 + tid] = g[r];
                    who[r * 256 + tid] = w[r];
                }
                __syncthreads();
            }
#pragma unroll
            for (int r = 0; r < PER; ++r) {
                double og;
                int32_t ow;
                if (hop >= 32) {
                    og = key[r * 256 + (tid ^ hop)];
                    ow = who[r * 256 + (tid ^ hop)];
                } else {
                    og = __shfl_xor_sync(0xFFFFFFFFu, g[r], hop);
                    ow = __shfl_xor_sync(0xFFFFFFFFu, w[r], hop);
                }
                const int32_t s = PER * tid + r;
                const bool keep_first = ((s & k) == 0) == ((s & d) == 0);
                if (served_first(g[r], w[r], og, ow) != keep_first) {
                    g[r] = og;
                    w[r] = ow;
                }
            }
        }
#pragma unroll
        for (int dd = PER / 2; dd >= 1; dd >>= 1) {
            if (dd < k) {
#pragma unroll
                for (int r = 0; r < PER; ++r) {
                    if ((r & dd) == 0) {
                        const bool low_keeps_first = ((PER * tid + r) & k) == 0;
                        if (served_first(g[r | dd], w[r | dd], g[r], w[r]) == low_keeps_first) {
                            const double tg = g[r];
                            const int32_t tw = w[r];
                            g[r] = g[r | dd];
                            w[r] = w[r | dd];
                            g[r | dd] = tg;
                            w[r | dd] = tw;
                        }
                    }
                }
            }
        }
    }
    __syncthreads();  // the last transposed copy may still be read
#pragma unroll
    for (int r = 0; r < PER; ++r) {
        key[PER * tid + r] = g[r];
        who[PER * tid + r] = w[r];
    }
    __syncthreads();
}

// Step (4) needs the order of service only as far as the idle GPUs reach: every job that is served takes at
// least one GPU, so the first `need` = min(idle GPUs, jobs below their limit) records of the order are enough.
// This finds the key of the need-th record by an eight-pass radix search over the gains (records in registers,
// 256-bin histograms in shared memory), moves the records at or above it (all ties included: still a prefix
// of the order) to the front of key[] / who[], pads to a power of two and sorts only those.  Returns the
// length sorted, or 0 when more than kServeMax records would have to be sorted (the caller then sorts all).
// hist: 256 + 2 words of shared memory; records beyond n_jobs carry gain -inf and are never selected.
constexpr int32_t kServeMax = 1024;
#ifndef ONES_SERVE_PASSES
#define ONES_SERVE_PASSES 2
#endif

template <int PER>
__device__ int32_t block_select_service_prefix(double* __restrict__ key, int32_t* __restrict__ who, int32_t need,
                                               unsigned int* __restrict__ hist, int32_t* __restrict__ s_warp) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long k[PER];
    double g[PER];
    int32_t w[PER];
#pragma unroll
    for (int r = 0; r < PER; ++r) {  // record r of thread t: r * 256 + t (neighbouring lanes, neighbouring words)
        g[r] = key[r * 256 + tid];
        w[r] = who[r * 256 + tid];
        // the search runs on the gain rounded down to fp32 (a monotone map: the records kept are still a prefix
        // of the order, with a few more ties) and stops after ONES_SERVE_PASSES digits of that key
        const uint32_t fb = __float_as_uint(__double2float_rd(g[r]) + 0.0f);
        const uint32_t fk = g[r] != g[r] ? 0u : ((fb >> 31) ? ~fb : (fb | 0x80000000u));
        k[r] = (unsigned long long)fk << 32;
    }
    unsigned long long prefix = 0ull;
    int32_t remaining = need;
    unsigned int alive = (1u << PER) - 1u;
    for (int pass = 0; pass < ONES_SERVE_PASSES; ++pass) {
        hist[tid] = 0u;
        __syncthreads();
        const int shift = 56 - 8 * pass;
        const unsigned long long mask = pass == 0 ? 0ull : ~0ull << (shift + 8);
#pragma unroll
        for (int r = 0; r < PER; ++r) {
            if (((alive >> r) & 1u) && (k[r] & mask) == prefix) atomicAdd(&hist[(unsigned int)(k[r] >> shift) & 255u], 1u);
            else alive &= ~(1u << r);
        }
        __syncthreads();
        if (warp == 0) {  // the digit that holds the remaining-th largest key, bins taken from 255 downwards
            unsigned int c[8], mine = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                c[i] = hist[255 - (8 * lane + i)];
                mine += c[i];
            }
            unsigned int incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned int a = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += a;
            }
            const unsigned int reached = __ballot_sync(0xFFFFFFFFu, (int32_t)incl >= remaining);
            const int owner = reached ? __ffs(reached) - 1 : 31;
            if (lane == owner) {
                int32_t above = (int32_t)(incl - mine), d = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int32_t bin = 255 - (8 * lane + i);
                    if (bin == 0 || above + (int32_t)c[i] >= remaining) {
                        d = bin;
                        break;
                    }
                    above += (int32_t)c[i];
                }
                hist[256] = (unsigned int)d;
                hist[257] = (unsigned int)(remaining - above);
            }
        }
        __syncthreads();
        prefix |= (unsigned long long)hist[256] << shift;
        remaining = (int32_t)hist[257];
        __syncthreads();  // hist[256..257] are rewritten by the next pass
    }
    // prefix = key of the need-th record of the order: every record at or above it is kept
    int32_t mine = 0;
#pragma unroll
    for (int r = 0; r < PER; ++r) mine += k[r] >= prefix;
    int32_t incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += up;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();  // also: every thread holds its records in registers, key[] and who[] may be rewritten
    int32_t at = incl - mine, total = 0;
#pragma unroll
    for (int v = 0; v < 8; ++v) {
        const int32_t c = s_warp[v];
        if (v < warp) at += c;
        total += c;
    }
    if (total > kServeMax) return 0;  // block-uniform
    int32_t m2 = 2;
    while (m2 < total) m2 <<= 1;
#pragma unroll
    for (int r = 0; r < PER; ++r)
        if (k[r] >= prefix) {
            key[at] = g[r];
            who[at] = w[r];
            ++at;
        }
    for (int32_t i = total + tid; i < m2; i += 256) {
        key[i] = -CUDART_INF;
        who[i] = 0x40000000 + i;
    }
    __syncthreads();
    if (m2 == 1024) {
        block_sort_service_order<4>(key, who);
    } else if (m2 == 512) {
        block_sort_service_order<2>(key, who);
    } else {  // at most 256 records, one per thread, every step through shared memory
        for (int32_t kk = 2; kk <= m2; kk <<= 1)
            for (int32_t d = kk >> 1; d > 0; d >>= 1) {
                const int32_t s = tid, p = tid ^ d;
                if (s < m2 && p > s) {
                    const double ka = key[s], kb = key[p];
                    const int32_t ja = who[s], jb = who[p];
                    if (served_first(kb, jb, ka, ja) == ((s & kk) == 0)) {
                        key[s] = kb; key[p] = ka;
                        who[s] = jb; who[p] = ja;
                    }
                }
                __syncthreads();
            }
    }
    return m2;
}

// Once per job-set change: inv[old id] = the new id of a surviving job (the highest, should several claim
// one old job) or -1, and newcum[j] = the GPUs that the new jobs before j need for their smallest batch
// (newcum[n_jobs] = all of them), capped at the cluster's size: needs beyond it can never be met.
__global__ void __launch_bounds__(256)
k_refresh_prepare(const int32_t* __restrict__ remap, int32_t n_old, int32_t n_jobs, const int4* __restrict__ fit,
                  int32_t n_gpus, int32_t* __restrict__ inv, int32_t* __restrict__ newcum) {
    __shared__ int32_t s_warp[8];
    __shared__ int32_t s_carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int32_t o = tid; o < n_old; o += 256) inv[o] = -1;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int32_t j = tid; j < n_jobs; j += 256) {
        const int32_t r = remap[j];
        if (r >= 0 && r < n_old) atomicMax(&inv[r], j);
    }
    for (int32_t base = 0; base < n_jobs; base += 256) {
        const int32_t j = base + tid;
        int32_t want = 0;
        if (j < n_jobs && remap[j] < 0) {
            const int4 q = fit[slot_of(j)];  // b0, max_per_gpu, kmin, kmax
            const long long b = (long long)q.x << q.z, m = q.y;
            const long long g = (b + m - 1) / m;
            want = (int32_t)(g < (long long)n_gpus ? g : (long long)n_gpus);
        }
        int32_t incl = want;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl = sat_add(incl, up);
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        int32_t offset = s_carry, total = s_carry;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const int32_t v = s_warp[w];
            if (w < warp) offset = sat_add(offset, v);
            total = sat_add(total, v);
        }
        const int32_t before = sat_add(offset, incl - want);  // incl - want is exact unless incl saturated,
        if (j < n_jobs) newcum[j] = min(before, n_gpus);      // and then both exceed the cap anyway
        __syncthreads();
        if (tid == 0) s_carry = total;
        __syncthreads();
    }
    if (tid == 0) newcum[n_jobs] = min(s_carry, n_gpus);
}

static int32_t refresh_sort_len(int32_t n_jobs) {
    int32_t j2 = 2;
    while (j2 < n_jobs) j2 <<= 1;
    return j2 == 256 ? 512 : j2;  // from 512 records on the sort keeps at least two records per thread in registers
}

size_t refresh_smem(int32_t n_gpus, int32_t n_jobs) {
    const size_t jp = (size_t)((n_jobs + 3) & ~3), wp = (size_t)((n_gpus + 3) & ~3), j2 = (size_t)refresh_sort_len(n_jobs);
    return 12 * j2 + 4 * (j2 + 4) + 4 * (4 * jp + 2 * wp);
}

__global__ void __launch_bounds__(256)
k_refresh_per_gpu(int32_t* __restrict__ slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_old, int32_t n_jobs,
                  Tables t, const int4* __restrict__ fit, const int32_t* __restrict__ remap,
                  const int32_t* __restrict__ inv, const int32_t* __restrict__ newcum, int32_t j2) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int32_t s_warp[8];
    const int32_t jp = (n_jobs + 3) & ~3, wp = (n_gpus + 3) & ~3;
    double* key = reinterpret_cast<double*>(smem_raw);  // step (4): gain of the job at this place of the order
    int32_t* sj = reinterpret_cast<int32_t*>(key + j2);  //           and the job itself
    int32_t* cum = sj + j2;                              // prefix sums over jobs (j2 + 4 entries)
    int32_t* count = cum + j2 + 4;                       // GPUs held by each job
    int32_t* first = count + jp;                         // its first and last slot
    int32_t* last = first + jp;
    int32_t* lim = last + jp;                            // GPUs its batch-size limit needs
    int32_t* row = lim + jp;                             // the candidate
    int32_t* rk = row + wp;                              // occupied slot: rank among its job's slots; idle: among the idle
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t U = newcum[n_jobs];
    const int32_t chunk = ((n_gpus + 255) / 256) | 1;
    const int32_t from = min(n_gpus, tid * chunk), to = min(n_gpus, from + chunk);
    for (int32_t j = tid; j < n_jobs; j += 256) {
        const int32_t at = slot_of(j);
        lim[j] = t.G[(int64_t)fit[at].w * t.jpad + at];
    }
    for (int64_t cand = blockIdx.x; cand < n; cand += gridDim.x) {
        int32_t* grow = slots + cand * ld;
        for (int32_t j = tid; j < n_jobs; j += 256) {
            count[j] = 0;
            first[j] = 0x7FFFFFFF;
            last[j] = -1;
        }
        __syncthreads();
        // (1) new ids; GPUs, first and last slot of every job
        for (int32_t i = tid; i < n_gpus; i += 256) {
            const int32_t o = grow[i];
            const int32_t id = (uint32_t)o < (uint32_t)n_old ? __ldg(inv + o) : -1;
            row[i] = id;
            if (id >= 0) {
                atomicAdd(&count[id], 1);
                atomicMin(&first[id], i);
                atomicMax(&last[id], i);
            }
        }
        __syncthreads();
        // rank of a slot among the slots of its job: the distance from the first one when they are neighbours
        // (every row this library writes is packed), else counted by one thread per such job
        for (int32_t i = tid; i < n_gpus; i += 256) {
            const int32_t id = row[i];
            rk[i] = id >= 0 ? i - first[id] : 0;
        }
        __syncthreads();
        for (int32_t j = tid; j < n_jobs; j += 256) {
            const int32_t c = count[j];
            if (c > 0 && last[j] - first[j] + 1 != c) {
                int32_t r = 0;
                for (int32_t i = first[j]; i <= last[j]; ++i)
                    if (row[i] == j) rk[i] = r++;
            }
        }
        __syncthreads();
        // (2) scale down to the limit: the slots of rank >= limit are the last ones
        for (int32_t i = tid; i < n_gpus; i += 256) {
            const int32_t id = row[i];
            if (id >= 0 && rk[i] >= lim[id]) row[i] = -1;
        }
        for (int32_t j = tid; j < n_jobs; j += 256) {
            const int32_t kept = min(count[j], lim[j]);
            count[j] = kept;
            cum[j] = __ldg(remap + j) < 0 ? 0 : kept;  // what step (3) may take from the jobs before j
        }
        __syncthreads();
        const int32_t V = block_scan_excl(cum, n_jobs, s_warp);
        // rank of every idle slot among the idle ones
        int32_t idle_mine = 0;
        for (int32_t i = from; i < to; ++i) idle_mine += row[i] < 0;
        int32_t incl = idle_mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        int32_t idle_before = incl - idle_mine, n_idle = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const int32_t v = s_warp[w];
            if (w < warp) idle_before += v;
            n_idle += v;
        }
        for (int32_t i = from; i < to; ++i)
            if (row[i] < 0) rk[i] = idle_before++;
        __syncthreads();
        // (3) the new jobs' units: u < n_idle is the u-th idle slot, the others are taken from surviving jobs
        const int32_t granted = min(U, n_idle + V);
        const int32_t taken = max(0, granted - n_idle);
        for (int32_t i = tid; i < n_gpus; i += 256) {
            const int32_t id = row[i];
            int32_t unit = -1;
            if (id < 0) {
                if (rk[i] < U) unit = rk[i];
            } else if (__ldg(remap + id) >= 0) {
                const int32_t turn = cum[id] + (count[id] - 1 - rk[i]);  // its place in the order GPUs are taken
                if (turn < taken) unit = n_idle + turn;
            }
            if (unit >= 0) row[i] = last_at_most(newcum, n_jobs + 1, unit);
        }
        __syncthreads();
        for (int32_t j = tid; j < n_jobs; j += 256) {
            if (__ldg(remap + j) < 0) count[j] = min(newcum[j + 1], granted) - min(newcum[j], granted);
            else count[j] -= min(max(taken - cum[j], 0), count[j]);
        }
        __syncthreads();
        // (4) refill what is still idle (block-uniform condition)
        if (n_idle > U) {
            for (int32_t s0 = tid; s0 < j2; s0 += 4 * 256) {
                // four jobs per step, each kind of load issued for all four before the next kind
                int4 q[4];
                int32_t at[4], have[4];
                bool cand[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int32_t s = s0 + 256 * u;
                    cand[u] = s < n_jobs && count[s] < lim[s];
                    at[u] = slot_of(cand[u] ? s : 0);
                    have[u] = cand[u] ? count[s] : 0;
                    q[u] = cand[u] ? __ldg(fit + at[u]) : make_int4(1, 1, 0, 0);
                }
                double now[4], top[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int32_t k = (cand[u] && have[u] > 0) ? exponent_that_fits(q[u].x, q[u].y, q[u].z, q[u].w, have[u]) : -1;
                    now[u] = k >= 0 ? __ldg(t.X + (int64_t)k * t.jpad + at[u]) : 0.0;
                    top[u] = cand[u] ? __ldg(t.X + (int64_t)q[u].w * t.jpad + at[u]) : 0.0;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int32_t s = s0 + 256 * u;
                    if (s < j2) {
                        key[s] = cand[u] ? __dsub_rn(top[u], now[u]) : -CUDART_INF;
                        sj[s] = cand[u] ? s : 0x40000000 + s;
                    }
                }
            }
            __syncthreads();
            // only as much of the order as the idle GPUs can reach (every served job takes at least one)
            int32_t len = 0;
            if (j2 >= 512 && j2 <= 4096) {
                const int32_t need = min(n_idle - U, j2);
                unsigned int* hist = reinterpret_cast<unsigned int*>(cum);  // free until the prefix sums below
                if (j2 == 512) len = block_select_service_prefix<2>(key, sj, need, hist, s_warp);
                else if (j2 == 1024) len = block_select_service_prefix<4>(key, sj, need, hist, s_warp);
                else if (j2 == 2048) len = block_select_service_prefix<8>(key, sj, need, hist, s_warp);
                else len = block_select_service_prefix<16>(key, sj, need, hist, s_warp);
            }
            if (len > 0) {
                // sorted already
            } else if (j2 == 512) block_sort_service_order<2>(key, sj);
            else if (j2 == 1024) block_sort_service_order<4>(key, sj);
            else if (j2 == 2048) block_sort_service_order<8>(key, sj);
            else if (j2 == 4096) block_sort_service_order<16>(key, sj);
            else  // a few records (or more than fit registers): every step through shared memory
                for (int32_t k = 2; k <= j2; k <<= 1)
                    for (int32_t d = k >> 1; d > 0; d >>= 1) {
                        for (int32_t s = tid; s < j2; s += 256) {
                            const int32_t p = s ^ d;
                            if (p > s) {
                                const double ka = key[s], kb = key[p];
                                const int32_t ja = sj[s], jb = sj[p];
                                // ascending runs put the record served first at the lower place
                                if (served_first(kb, jb, ka, ja) == ((s & k) == 0)) {
                                    key[s] = kb; key[p] = ka;
                                    sj[s] = jb; sj[p] = ja;
                                }
                            }
                        }
                        __syncthreads();
                    }
            if (len == 0) len = j2;
            for (int32_t s = tid; s < len; s += 256) {
                const int32_t j = sj[s];
                cum[s] = j < n_jobs ? min(lim[j] - count[j], n_gpus) : 0;
            }
            __syncthreads();
            const int32_t wanted = block_scan_excl(cum, len, s_warp);
            for (int32_t i = tid; i < n_gpus; i += 256) {
                if (row[i] < 0) {
                    const int32_t r = rk[i] - U;
                    if (r >= 0 && r < wanted) row[i] = sj[last_at_most(cum, len, r)];
                }
            }
            __syncthreads();
        }
        for (int32_t i = tid; i < n_gpus; i += 256) grow[i] = row[i];
        __syncthreads();
    }
}

cudaError_t launch_refresh_per_gpu(int32_t* slots, int64_t ld, int32_t n, int32_t n_gpus, int32_t n_old, int32_t n_jobs,
                                   Tables t, const int4* fit, const int32_t* remap, int32_t* inv, int32_t* newcum,
                                   cudaStream_t s) {
    const size_t smem = refresh_smem(n_gpus, n_jobs);
    if (smem > (size_t)kMaxSmemPerBlock - 1024) return cudaErrorInvalidConfiguration;
    k_refresh_prepare<<<1, 256, 0, s>>>(remap, n_old, n_jobs, fit, n_gpus, inv, newcum);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || n <= 0) return e;
    e = cudaFuncSetAttribute(k_refresh_per_gpu, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int64_t blocks = n;
    if (blocks > (int64_t)sm_count() * 4) blocks = (int64_t)sm_count() * 4;
    k_refresh_per_gpu<<<(int)blocks, 256, smem, s>>>(slots, ld, n, n_gpus, n_old, n_jobs, t, fit, remap, inv, newcum,
                                                      refresh_sort_len(n_jobs));
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Best candidate and its repair to the cluster's capacity: one block.
// work[0..jpad) exponent, work[jpad..2jpad) GPUs now, work[2jpad..3jpad) GPUs one exponent lower
// (-1 when the job cannot shrink).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int2 block_arg_best(int2 mine /*(value, j); value < 0: none*/, int2* s_warp, bool want_max_value) {
    // max value, ties to the lower j (want_max_value) — or lowest j among value >= 0 otherwise
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        int2 o;
        o.x = __shfl_xor_sync(0xFFFFFFFFu, mine.x, off);
        o.y = __shfl_xor_sync(0xFFFFFFFFu, mine.y, off);
        bool take;
        if (want_max_value) take = o.x > mine.x || (o.x == mine.x && o.x >= 0 && o.y < mine.y);
        else take = o.x >= 0 && (mine.x < 0 || o.y < mine.y);
        if (take) mine = o;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
    __syncthreads();
    if (lane == 0) s_warp[warp] = mine;
    __syncthreads();
    int2 r = s_warp[0];
    for (int w = 1; w < nwarp; ++w) {
        const int2 o = s_warp[w];
        bool take;
        if (want_max_value) take = o.x > r.x || (o.x == r.x && o.x >= 0 && o.y < r.y);
        else take = o.x >= 0 && (r.x < 0 || o.y < r.y);
        if (take) r = o;
    }
    return r;
}

__global__ void __launch_bounds__(256)
k_best(const int32_t* __restrict__ pop, int64_t ld, int32_t n_jobs, const int32_t* __restrict__ best_index, Tables t,
       int32_t capacity, double penalty, int repair, int32_t* __restrict__ work, int32_t* __restrict__ genome_out,
       int32_t* __restrict__ gpus_out, double* __restrict__ rate_out, BestOut* __restrict__ out,
       const int32_t* __restrict__ rowmap) {
    __shared__ int2 s_warp[8];
    __shared__ long long s_total;
    __shared__ int s_status;
    const int32_t best = best_index[0];
    const int32_t* row = pop + (int64_t)(rowmap ? rowmap[best] : best) * ld;  // a pool used in place keeps a row map
    int32_t* wk = work;
    int32_t* wg = work + t.jpad;
    int32_t* wl = work + 2 * t.jpad;
    const uint32_t kcap = (uint32_t)t.k1;

    if (threadIdx.x == 0) { s_total = 0; s_status = 0; }
    __syncthreads();
    long long part = 0;
    for (int32_t j0 = threadIdx.x; j0 < n_jobs; j0 += 4 * blockDim.x) {
        // four jobs per step, each kind of load issued for all four before the next kind (the row lives in HBM)
        int32_t k[4], lo[4], g[4], less[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t j = j0 + u * (int32_t)blockDim.x;
            k[u] = j < n_jobs ? row[j] : -1;
            lo[u] = j < n_jobs ? t.kmin[j] : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t j = j0 + u * (int32_t)blockDim.x;
            const int32_t p = (int32_t)min((uint32_t)k[u], kcap);
            g[u] = j < n_jobs ? t.G[(int64_t)p * t.jpad + slot_of(j)] : 0;
            less[u] = -1;
            if (j < n_jobs && p > 0 && k[u] > lo[u]) less[u] = t.G[(int64_t)(p - 1) * t.jpad + slot_of(j)];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t j = j0 + u * (int32_t)blockDim.x;
            if (j < n_jobs) {
                wk[j] = k[u];  // genes that already mean "waiting" are returned as stored
                wg[j] = g[u];
                wl[j] = (g[u] > 0 && less[u] >= 0 && less[u] < g[u]) ? less[u] : -1;
                part += g[u];
            }
        }
    }
    atomicAdd(reinterpret_cast<unsigned long long*>(&s_total), (unsigned long long)part);
    __syncthreads();
    long long total = s_total;
    int32_t steps = 0;

    if (repair) {
        while (total > capacity) {
            // the job holding the most GPUs among those that can give some back
            int2 mine = make_int2(-1, 0x7FFFFFFF);
            for (int32_t j = threadIdx.x; j < n_jobs; j += blockDim.x)
                if (wl[j] >= 0 && wg[j] > mine.x) mine = make_int2(wg[j], j);
            int2 pick = block_arg_best(mine, s_warp, true);
            if (pick.x >= 0) {
                const int32_t j = pick.y;
                if (threadIdx.x == 0) {
                    const int32_t k = wk[j] - 1;
                    const int32_t g = wl[j];
                    total -= wg[j] - g;
                    int32_t less = -1;
                    if (k > t.kmin[j]) less = t.G[(int64_t)(k - 1) * t.jpad + slot_of(j)];
                    wk[j] = k;
                    wg[j] = g;
                    wl[j] = (less >= 0 && less < g) ? less : -1;
                    s_total = total;
                }
            } else {
                // nothing can shrink: the lowest-indexed running job waits
                int2 run = make_int2(-1, 0x7FFFFFFF);
                for (int32_t j = threadIdx.x; j < n_jobs; j += blockDim.x)
                    if (wg[j] > 0 && j < run.y) run = make_int2(1, j);
                int2 park = block_arg_best(run, s_warp, false);
                if (park.x < 0) {
                    if (threadIdx.x == 0) s_status = 1;
                    __syncthreads();
                    break;
                }
                if (threadIdx.x == 0) {
                    const int32_t j = park.y;
                    total -= wg[j];
                    wk[j] = -1;
                    wg[j] = 0;
                    wl[j] = -1;
                    s_total = total;
                }
            }
            __syncthreads();
            total = s_total;
            ++steps;
        }
    }
    __syncthreads();

    // outputs, then the score of the (repaired) row summed in the fixed order by warp 0.  Every thread
    // looks its jobs' terms up and leaves them where the GPU counts were (2 * jpad int32 = jpad doubles),
    // so that the summing warp reads one contiguous array, sixteen terms in flight per lane.
    for (int32_t j = threadIdx.x; j < n_jobs; j += blockDim.x) {
        if (genome_out) genome_out[j] = wk[j];
        if (gpus_out) gpus_out[j] = wg[j];
    }
    __syncthreads();
    double* term = reinterpret_cast<double*>(wg);
    for (int32_t j0 = threadIdx.x; j0 < n_jobs; j0 += 4 * blockDim.x) {
        int32_t p[4];
        double x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t j = j0 + u * (int32_t)blockDim.x;
            p[u] = j < n_jobs ? (int32_t)min((uint32_t)wk[j], kcap) : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t j = j0 + u * (int32_t)blockDim.x;
            x[u] = j < n_jobs ? t.X[(int64_t)p[u] * t.jpad + slot_of(j)] : 0.0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int32_t j = j0 + u * (int32_t)blockDim.x;
            if (j < n_jobs) {
                term[j] = x[u];
                if (rate_out) rate_out[j] = x[u];
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        double sum = 0.0;
        const int32_t nvec = (n_jobs + 3) >> 2;
        for (int32_t v0 = lane; v0 < nvec; v0 += 32 * 4) {
            double x[4][4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int s = 0; s < 4; ++s) {
                    const int32_t j = 4 * (v0 + 32 * u) + s;
                    x[u][s] = j < n_jobs ? term[j] : 0.0;
                }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    if (4 * (v0 + 32 * u) + s < n_jobs) sum = __dadd_rn(sum, x[u][s]);
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) sum = __dadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, off));
        if (lane == 0) {
            const int32_t g32 = (int32_t)total;
            const int32_t over = g32 > capacity ? g32 - capacity : 0;
            out->fitness = __dsub_rn(sum, __dmul_rn(penalty, (double)over));
            out->total_gpus = g32;
            out->index = best;
            out->status = s_status;
            out->steps = steps;
        }
    }
}

cudaError_t launch_best(const int32_t* pop, int64_t ld, int32_t n_jobs, const int32_t* best_index, Tables t,
                        int32_t capacity, double penalty, int repair, int32_t* work, int32_t* genome_out,
                        int32_t* gpus_out, double* rate_out, BestOut* out, const int32_t* rowmap, cudaStream_t s) {
    k_best<<<1, 256, 0, s>>>(pop, ld, n_jobs, best_index, t, capacity, penalty, repair, work, genome_out, gpus_out,
                             rate_out, out, rowmap);
    return cudaGetLastError();
}

}  // namespace ones
