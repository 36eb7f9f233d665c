/*
 * ones_oracle.c — CPU oracle for the ONES evolutionary batch-size search.
 *
 * TEST INFRASTRUCTURE (see ones_oracle.h).  Plain C, single thread, fp64, built
 * with -O2 -ffp-contract=off so every floating-point operation is rounded once.
 * It follows the steps of the search in the order the paper's Section 3.2.2
 * gives them (initialise, derive new candidates by crossover and mutation,
 * score, select, keep the best) with no blocking, caching or fusion: the
 * throughput model is re-evaluated for every gene of every candidate.
 *
 * Reading of the paper used here
 *  - A candidate S (Eq. 1-2) is stored as one exponent k_j per job:
 *    B_j = b0_j << k_j, c_j = ceil(B_j / max_per_gpu_j); k_j outside [0, kmax_j]
 *    is the waiting state B_j = c_j = 0 of the text after Eq. 2.
 *  - X_j (Table 1, Eq. 5) comes from an iteration-time model
 *    t = a + c*(B/c_j) + d*log2(c_j), X = B / t.
 *  - The score of a candidate is a sum over jobs of a per-job term (Alg. 1,
 *    Eq. 8), here the predicted progress sum_j X_j, and the one-job-per-GPU
 *    constraint (Eq. 4) enters as a penalty on sum_j c_j - |C|.
 *  - Uniform crossover gives two complementary children (Section 3.2.2, "Uniform
 *    crossover"); uniform mutation touches each job independently with rate
 *    theta ("Uniform mutation"), never leaving [kmin_j, kmax_j] (limit R_j).  One random word
 *    per job and pair of siblings carries the crossover bit and both children's mutation draws.
 *  - Selection: tournament for parents, the E best survive unchanged, S* is the
 *    best-scored candidate (Alg. 1, last step).
 */
#include "ones_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as     */
/* easy as 1, 2, 3", SC'11): ten rounds; each round multiplies words 0 and 2   */
/* by two fixed odd constants, the high halves are xored with the neighbouring */
/* words and the round key, the low halves move over; the key is bumped by two */
/* Weyl constants between rounds.                                              */
/* ------------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t MUL_A = 0xD2511F53u, MUL_B = 0xCD9E8D57u;
    const uint32_t WEYL_A = 0x9E3779B9u, WEYL_B = 0xBB67AE85u;
    uint32_t x0 = ctr[0], x1 = ctr[1], x2 = ctr[2], x3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += WEYL_A;
            k1 += WEYL_B;
        }
        uint64_t pa = (uint64_t)MUL_A * (uint64_t)x0;
        uint64_t pb = (uint64_t)MUL_B * (uint64_t)x2;
        uint32_t y0 = (uint32_t)(pb >> 32) ^ x1 ^ k0;
        uint32_t y1 = (uint32_t)pb;
        uint32_t y2 = (uint32_t)(pa >> 32) ^ x3 ^ k1;
        uint32_t y3 = (uint32_t)pa;
        x0 = y0; x1 = y1; x2 = y2; x3 = y3;
    }
    out[0] = x0; out[1] = x1; out[2] = x2; out[3] = x3;
}

/* Random word for (generation, row, column) on a stream.  Key = the 64-bit
 * seed; counter = (column / 4, row, generation low word, stream + 16 *
 * generation high word); the word taken is column % 4. */
uint32_t oracle_word(uint64_t seed, uint64_t gen_abs, uint32_t row, uint32_t col, uint32_t stream) {
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t ctr[4] = {col >> 2, row, (uint32_t)gen_abs, stream | ((uint32_t)(gen_abs >> 32) << 4)};
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    return out[col & 3u];
}

/* ------------------------------------------------------------------------- */
/* Throughput model and score                                                 */
/* ------------------------------------------------------------------------- */
int oracle_model(const oracle_job* job, int32_t k, double* X, int32_t* g) {
    if (!job || !X || !g) return ORACLE_ERR_NULL;
    *X = 0.0;
    *g = 0;
    if (k < 0 || k > job->kmax) return ORACLE_OK; /* the job waits: B = c = 0 */
    int64_t b = (int64_t)job->b0 << k;            /* global batch size B_j */
    int64_t m = job->max_per_gpu;
    int64_t gpus = (b + m - 1) / m;               /* c_j = ceil(B_j / max local batch) */
    double local = (double)b / (double)gpus;      /* local batch size b_j */
    double lg = log2((double)gpus);
    double t = (job->a + job->c * local) + job->d * lg; /* seconds per iteration */
    *X = (double)b / t;                           /* samples per second */
    *g = (int32_t)gpus;
    return ORACLE_OK;
}

int oracle_term(const oracle_job* job, int32_t k, uint32_t flags, double* term, int32_t* g) {
    double X;
    int rc = oracle_model(job, k, &X, g);
    if (rc) return rc;
    if (flags & ORACLE_FLAG_SRUF) {
        /* Alg. 1 score term Y_processed*(1/rho - 1) * c_j / X_j with the first two
         * factors folded into weight_j; negated so that higher is better. */
        *term = (*g > 0) ? -((job->weight * (double)*g) / X) : 0.0;
    } else {
        *term = X;
    }
    return ORACLE_OK;
}

int oracle_fitness(const oracle_job* jobs, int32_t n_jobs, int32_t capacity, double penalty,
                   uint32_t flags, const int32_t* genome, double* F, int32_t* gpus) {
    if (!jobs || !genome || !F) return ORACLE_ERR_NULL;
    /* Fixed summation order: 32 partial sums, job j goes to partial (j / 4) % 32
     * in increasing j, then a pairwise tree over the partials. */
    double part[32];
    for (int l = 0; l < 32; ++l) part[l] = 0.0;
    int64_t demand = 0;
    for (int32_t j = 0; j < n_jobs; ++j) {
        double term;
        int32_t g;
        oracle_term(&jobs[j], genome[j], flags, &term, &g);
        part[(j >> 2) & 31] += term;
        demand += g;
    }
    for (int off = 16; off >= 1; off >>= 1)
        for (int l = 0; l < off; ++l) part[l] = part[l] + part[l + off];
    int32_t demand32 = (int32_t)demand; /* two's-complement wrap, as 32-bit adds would give */
    int32_t over = demand32 > capacity ? demand32 - capacity : 0;
    *F = part[0] - penalty * (double)over;
    if (gpus) *gpus = demand32;
    return ORACLE_OK;
}

int oracle_validate_jobs(const oracle_job* jobs, int32_t n_jobs) {
    if (!jobs) return ORACLE_ERR_NULL;
    if (n_jobs <= 0) return ORACLE_ERR_BAD_JOB;
    for (int32_t j = 0; j < n_jobs; ++j) {
        const oracle_job* q = &jobs[j];
        if (q->b0 <= 0 || q->max_per_gpu <= 0) return ORACLE_ERR_BAD_JOB;
        if (q->kmin < 0 || q->kmin > q->kmax || q->kmax > 15) return ORACLE_ERR_BAD_JOB;
        if (((int64_t)q->b0 << q->kmax) >= ((int64_t)1 << 31)) return ORACLE_ERR_BAD_JOB;
        if (!(q->a >= 0.0) || !(q->c >= 0.0) || !(q->d >= 0.0)) return ORACLE_ERR_BAD_JOB;
        if (!isfinite(q->a) || !isfinite(q->c) || !isfinite(q->d) || !isfinite(q->weight))
            return ORACLE_ERR_BAD_JOB;
        for (int32_t k = 0; k <= q->kmax; ++k) {
            double X;
            int32_t g;
            oracle_model(q, k, &X, &g);
            if (!(X > 0.0) || !isfinite(X)) return ORACLE_ERR_BAD_JOB; /* t must be > 0 */
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------- */
/* Order, elites, tournament                                                  */
/* ------------------------------------------------------------------------- */
static int better(const double* F, int32_t x, int32_t y) {
    return F[x] > F[y] || (F[x] == F[y] && x < y);
}

int oracle_top(const double* F, int32_t n, int32_t e, int32_t* idx) {
    if (!F || !idx) return ORACLE_ERR_NULL;
    if (e < 0 || e > n) return ORACLE_ERR_BAD_PARAM;
    /* selection by repeated scan: rank r = best candidate not already taken */
    for (int32_t r = 0; r < e; ++r) {
        int32_t best = -1;
        for (int32_t i = 0; i < n; ++i) {
            int taken = 0;
            for (int32_t s = 0; s < r; ++s)
                if (idx[s] == i) taken = 1;
            if (taken) continue;
            if (best < 0 || better(F, i, best)) best = i;
        }
        idx[r] = best;
    }
    return ORACLE_OK;
}

int32_t oracle_tournament(const double* F, int32_t n, int32_t tournament, uint64_t seed,
                          uint64_t gen_abs, uint32_t q, uint32_t stream) {
    int32_t win = -1;
    for (int32_t t = 0; t < tournament; ++t) {
        uint32_t w = oracle_word(seed, gen_abs, q, (uint32_t)t, stream);
        int32_t idx = (int32_t)(((uint64_t)w * (uint64_t)(uint32_t)n) >> 32); /* uniform in [0, n) */
        if (win < 0 || better(F, idx, win)) win = idx;
    }
    return win;
}

uint32_t oracle_thr16(double p_mut) {
    long t = lround(p_mut * 65536.0);
    if (t < 0) t = 0;
    if (t > 65536) t = 65536;
    return (uint32_t)t;
}

/* uniform value in [kmin, kmax] from a 32-bit fraction: kmin + floor(frac * range / 2^32) */
static int32_t draw_gene(uint32_t frac, int32_t kmin, int32_t kmax) {
    uint64_t range = (uint64_t)(kmax - kmin + 1);
    return kmin + (int32_t)(((uint64_t)frac * range) >> 32);
}

/* One random word W serves one job of a pair of sibling children.  Its low half e is the
 * even child's 16-bit mutation field, its high half o the odd child's; bit 0 decides which
 * child inherits the first parent's gene.  A child mutates when its field is below the
 * threshold; its new value is drawn with the fraction (other field + own field * M) mod 2^16
 * in the top half of a 32-bit word, which is uniform because the other child's field is. */
static uint32_t even_fraction(uint32_t W) { return W * 0x9E360001u; }            /* top half: o + e*0x9E36 */
static uint32_t odd_fraction(uint32_t W) { return ((W << 16) | (W >> 16)) * 0x85EB0001u; } /* e + o*0x85EB */

/* ------------------------------------------------------------------------- */
/* Repair                                                                      */
/* ------------------------------------------------------------------------- */
int oracle_repair(const oracle_job* jobs, int32_t n_jobs, int32_t capacity, int32_t* genome) {
    if (!jobs || !genome) return ORACLE_ERR_NULL;
    for (;;) {
        int64_t demand = 0;
        for (int32_t j = 0; j < n_jobs; ++j) {
            double X; int32_t g;
            oracle_model(&jobs[j], genome[j], &X, &g);
            demand += g;
        }
        if (demand <= capacity) return ORACLE_OK;
        /* scale down the job holding the most GPUs among those that can give some back */
        int32_t pick = -1, pick_g = 0;
        for (int32_t j = 0; j < n_jobs; ++j) {
            int32_t k = genome[j];
            if (k < 0 || k > jobs[j].kmax || k <= jobs[j].kmin) continue;
            double X; int32_t g_now, g_less;
            oracle_model(&jobs[j], k, &X, &g_now);
            oracle_model(&jobs[j], k - 1, &X, &g_less);
            if (g_now > g_less && g_now > pick_g) { pick = j; pick_g = g_now; }
        }
        if (pick >= 0) { genome[pick] -= 1; continue; }
        /* nothing can shrink: the longest-present running job (lowest index) waits */
        int32_t park = -1;
        for (int32_t j = 0; j < n_jobs; ++j) {
            double X; int32_t g;
            oracle_model(&jobs[j], genome[j], &X, &g);
            if (g > 0) { park = j; break; }
        }
        if (park < 0) return ORACLE_ERR_INFEASIBLE;
        genome[park] = -1;
    }
}

/* ------------------------------------------------------------------------- */
/* Per-GPU genome (the paper's own encoding) and the reorder operation          */
/* ------------------------------------------------------------------------- */
int oracle_fitness_per_gpu(const oracle_job* jobs, int32_t n_jobs, int32_t n_gpus, uint32_t flags,
                           const int32_t* slots, double* F, int32_t* gpus_used, int32_t* exponents) {
    if (!jobs || !slots || !F) return ORACLE_ERR_NULL;
    int32_t* count = (int32_t*)calloc((size_t)n_jobs, sizeof(int32_t));
    if (!count) return ORACLE_ERR_NOMEM;
    for (int32_t i = 0; i < n_gpus; ++i)
        if (slots[i] >= 0 && slots[i] < n_jobs) count[slots[i]] += 1; /* c_j = sum_i min(1, b_j^i) */
    double part[32];
    for (int l = 0; l < 32; ++l) part[l] = 0.0;
    int64_t used = 0;
    for (int32_t j = 0; j < n_jobs; ++j) {
        int32_t kbest = -1;
        for (int32_t k = jobs[j].kmin; k <= jobs[j].kmax; ++k) {
            double X; int32_t g;
            oracle_model(&jobs[j], k, &X, &g);
            if (g <= count[j]) kbest = k;
        }
        double term = 0.0;
        int32_t g = 0;
        if (kbest >= 0) oracle_term(&jobs[j], kbest, flags, &term, &g);
        part[(j >> 2) & 31] = part[(j >> 2) & 31] + term; /* same summation order as oracle_fitness */
        used += g;
        if (exponents) exponents[j] = kbest;
    }
    for (int off = 16; off >= 1; off >>= 1)
        for (int l = 0; l < off; ++l) part[l] = part[l] + part[l + off];
    *F = part[0];
    if (gpus_used) *gpus_used = (int32_t)used;
    free(count);
    return ORACLE_OK;
}

int oracle_reorder(int32_t* slots, int32_t n_gpus, int32_t n_jobs) {
    if (!slots) return ORACLE_ERR_NULL;
    int32_t* out = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n_gpus > 0 ? n_gpus : 1));
    char* done = (char*)calloc((size_t)(n_jobs > 0 ? n_jobs : 1), 1);
    if (!out || !done) { free(out); free(done); return ORACLE_ERR_NOMEM; }
    int32_t at = 0;
    for (int32_t i = 0; i < n_gpus; ++i) { /* jobs in the order of their first occurrence */
        int32_t j = slots[i];
        if (j < 0 || j >= n_jobs || done[j]) continue;
        done[j] = 1;
        for (int32_t i2 = i; i2 < n_gpus; ++i2)
            if (slots[i2] == j) out[at++] = j;
    }
    while (at < n_gpus) out[at++] = -1; /* idle GPUs last */
    memcpy(slots, out, sizeof(int32_t) * (size_t)n_gpus);
    free(out);
    free(done);
    return ORACLE_OK;
}

/* "Refresh" of one per-GPU candidate at a change of the job set (Section 3.2.2).
 * inv[o] = new id of old job o, or -1 when it has finished; is_new[j] != 0 for a job that was not there. */
int oracle_refresh(const oracle_job* jobs, int32_t n_jobs, uint32_t flags, const int32_t* inv, int32_t n_jobs_old,
                   const char* is_new, int32_t* slots, int32_t n_gpus) {
    if (!jobs || !inv || !is_new || !slots) return ORACLE_ERR_NULL;
    int32_t* count = (int32_t*)calloc((size_t)(n_jobs > 0 ? n_jobs : 1), sizeof(int32_t));
    int32_t* limit = (int32_t*)calloc((size_t)(n_jobs > 0 ? n_jobs : 1), sizeof(int32_t));
    if (!count || !limit) { free(count); free(limit); return ORACLE_ERR_NOMEM; }
    /* (1) GPUs of finished jobs become idle; surviving jobs are known by their new ids */
    for (int32_t i = 0; i < n_gpus; ++i) {
        int32_t o = slots[i];
        slots[i] = (o >= 0 && o < n_jobs_old) ? inv[o] : -1;
        if (slots[i] >= 0) count[slots[i]] += 1;
    }
    /* (2) scale down: a job gives up the GPUs beyond those its batch-size limit needs, last ones first */
    for (int32_t j = 0; j < n_jobs; ++j) {
        double X;
        oracle_model(&jobs[j], jobs[j].kmax, &X, &limit[j]);
    }
    for (int32_t i = n_gpus - 1; i >= 0; --i) {
        int32_t j = slots[i];
        if (j >= 0 && count[j] > limit[j]) { slots[i] = -1; count[j] -= 1; }
    }
    /* (3) every new job gets the GPUs of its smallest batch: idle GPUs first (lowest first), then the
     * last GPU of the job that has been here longest (lowest index) among those that still hold one */
    for (int32_t j = 0; j < n_jobs; ++j) {
        if (!is_new[j]) continue;
        double X; int32_t want;
        oracle_model(&jobs[j], jobs[j].kmin, &X, &want);
        for (int32_t u = 0; u < want; ++u) {
            int32_t at = -1;
            for (int32_t i = 0; i < n_gpus && at < 0; ++i) if (slots[i] < 0) at = i;
            if (at < 0) {
                int32_t v = -1;
                for (int32_t q = 0; q < n_jobs && v < 0; ++q) if (!is_new[q] && count[q] > 0) v = q;
                if (v < 0) break;
                for (int32_t i = n_gpus - 1; i >= 0 && at < 0; --i) if (slots[i] == v) at = i;
                count[v] -= 1;
            }
            slots[at] = j;
            count[j] += 1;
        }
    }
    /* (4) fill the idle GPUs: the job whose score term gains most from growing to its limit goes first
     * (ties: lower index) and takes what it needs for that, or what is left */
    for (;;) {
        int32_t idle = 0;
        for (int32_t i = 0; i < n_gpus; ++i) idle += slots[i] < 0;
        if (idle == 0) break;
        int32_t pick = -1;
        double best = 0.0;
        for (int32_t j = 0; j < n_jobs; ++j) {
            if (count[j] >= limit[j]) continue;
            int32_t know = -1, g;
            for (int32_t k = jobs[j].kmin; k <= jobs[j].kmax; ++k) {
                double X;
                oracle_model(&jobs[j], k, &X, &g);
                if (g <= count[j]) know = k;
            }
            double now = 0.0, top;
            if (know >= 0) oracle_term(&jobs[j], know, flags, &now, &g);
            oracle_term(&jobs[j], jobs[j].kmax, flags, &top, &g);
            double gain = top - now;
            if (pick < 0 || gain > best) { pick = j; best = gain; }
        }
        if (pick < 0) break;
        int32_t take = limit[pick] - count[pick];
        if (take > idle) take = idle;
        for (int32_t i = 0; i < n_gpus && take > 0; ++i)
            if (slots[i] < 0) { slots[i] = pick; count[pick] += 1; take -= 1; }
    }
    free(count);
    free(limit);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------- */
/* The search                                                                  */
/* ------------------------------------------------------------------------- */
struct oracle_ctx {
    int32_t J, cap, N, pairs;
    int32_t W; /* genes per candidate: one per job, or one per GPU with ORACLE_FLAG_PER_GPU */
    oracle_params prm;
    oracle_job* jobs;
    int32_t* pop;   /* N x J */
    int32_t* next;  /* N x J */
    double* F;
    int32_t* G;
    int f_valid;
    uint64_t gen_abs;
    int32_t* parents; /* pairs x 2 of the last generation */
    int32_t* elites;  /* E of the last generation */
};

/* admissible values of gene j: the job's exponents, or (per-GPU genome) any job id */
static int32_t gene_lo(const oracle_ctx* c, int32_t j) { return (c->prm.flags & ORACLE_FLAG_PER_GPU) ? 0 : c->jobs[j].kmin; }
static int32_t gene_hi(const oracle_ctx* c, int32_t j) { return (c->prm.flags & ORACLE_FLAG_PER_GPU) ? c->J - 1 : c->jobs[j].kmax; }

static int check_params(const oracle_params* p, int32_t pop) {
    if ((p->flags & ORACLE_FLAG_PER_GPU) && (p->flags & ORACLE_FLAG_TRUNCATION)) return ORACLE_ERR_BAD_PARAM;
    if (p->elitism < 0 || p->tournament < 1) return ORACLE_ERR_BAD_PARAM;
    if (pop < p->elitism + 1) return ORACLE_ERR_BAD_PARAM;
    if (!(p->p_mut >= 0.0 && p->p_mut <= 1.0)) return ORACLE_ERR_BAD_PARAM;
    if (!isfinite(p->penalty)) return ORACLE_ERR_BAD_PARAM;
    return ORACLE_OK;
}

static void free_ctx(oracle_ctx* c) {
    if (!c) return;
    free(c->jobs); free(c->pop); free(c->next); free(c->F); free(c->G);
    free(c->parents); free(c->elites); free(c);
}

int oracle_create(oracle_ctx** out, const oracle_job* jobs, int32_t n_jobs, int32_t capacity,
                  int32_t pop, const oracle_params* prm) {
    if (!out || !jobs) return ORACLE_ERR_NULL;
    *out = NULL;
    oracle_params p = {2, 4, 0.1, 1e3, 0};
    if (prm) p = *prm;
    int rc = oracle_validate_jobs(jobs, n_jobs);
    if (rc) return rc;
    if (capacity <= 0 || pop <= 0) return ORACLE_ERR_BAD_PARAM;
    rc = check_params(&p, pop);
    if (rc) return rc;
    oracle_ctx* c = (oracle_ctx*)calloc(1, sizeof *c);
    if (!c) return ORACLE_ERR_NOMEM;
    c->J = n_jobs; c->cap = capacity; c->N = pop; c->prm = p;
    c->W = (p.flags & ORACLE_FLAG_PER_GPU) ? capacity : n_jobs;
    c->pairs = (p.flags & ORACLE_FLAG_TRUNCATION) ? pop : (pop - p.elitism + 1) / 2;
    size_t cells = (size_t)pop * (size_t)c->W;
    c->jobs = (oracle_job*)malloc(sizeof(oracle_job) * (size_t)n_jobs);
    c->pop = (int32_t*)malloc(sizeof(int32_t) * cells);
    c->next = (int32_t*)malloc(sizeof(int32_t) * cells);
    c->F = (double*)malloc(sizeof(double) * (size_t)pop);
    c->G = (int32_t*)malloc(sizeof(int32_t) * (size_t)pop);
    c->parents = (int32_t*)calloc((size_t)(c->pairs > 0 ? c->pairs : 1) * 2, sizeof(int32_t));
    c->elites = (int32_t*)calloc((size_t)(p.elitism > 0 ? p.elitism : 1), sizeof(int32_t));
    if (!c->jobs || !c->pop || !c->next || !c->F || !c->G || !c->parents || !c->elites) {
        free_ctx(c);
        return ORACLE_ERR_NOMEM;
    }
    memcpy(c->jobs, jobs, sizeof(oracle_job) * (size_t)n_jobs);
    /* initial population G_0 of simple solutions: every job at its smallest batch */
    for (int32_t i = 0; i < pop; ++i)
        for (int32_t j = 0; j < c->W; ++j)
            c->pop[(size_t)i * c->W + j] = (p.flags & ORACLE_FLAG_PER_GPU) ? -1 : jobs[j].kmin; /* per GPU: all idle */
    c->f_valid = 0;
    c->gen_abs = 0;
    *out = c;
    return ORACLE_OK;
}

int oracle_destroy(oracle_ctx* c) {
    free_ctx(c);
    return ORACLE_OK;
}

int oracle_randomize(oracle_ctx* c, uint64_t seed) {
    if (!c) return ORACLE_ERR_NULL;
    for (int32_t i = 0; i < c->N; ++i)
        for (int32_t j = 0; j < c->W; ++j) {
            int32_t k = gene_lo(c, j); /* candidate 0 stays the all-minimum schedule */
            if (i > 0) k = draw_gene(oracle_word(seed, 0, (uint32_t)i, (uint32_t)j, ORACLE_STREAM_INIT),
                                     gene_lo(c, j), gene_hi(c, j));
            c->pop[(size_t)i * c->W + j] = k;
        }
    c->f_valid = 0;
    return ORACLE_OK;
}

int oracle_set_population(oracle_ctx* c, const int32_t* genomes, int64_t ld) {
    if (!c || !genomes) return ORACLE_ERR_NULL;
    if (ld < c->W) return ORACLE_ERR_BAD_PARAM;
    for (int32_t i = 0; i < c->N; ++i)
        memcpy(&c->pop[(size_t)i * c->W], &genomes[(size_t)i * (size_t)ld], sizeof(int32_t) * (size_t)c->W);
    c->f_valid = 0;
    return ORACLE_OK;
}

int oracle_get_population(oracle_ctx* c, int32_t* genomes, int64_t ld) {
    if (!c || !genomes) return ORACLE_ERR_NULL;
    if (ld < c->W) return ORACLE_ERR_BAD_PARAM;
    for (int32_t i = 0; i < c->N; ++i)
        memcpy(&genomes[(size_t)i * (size_t)ld], &c->pop[(size_t)i * c->W], sizeof(int32_t) * (size_t)c->W);
    return ORACLE_OK;
}

static void score_row(const oracle_ctx* c, const int32_t* row, double* F, int32_t* G) {
    if (c->prm.flags & ORACLE_FLAG_PER_GPU)
        oracle_fitness_per_gpu(c->jobs, c->J, c->cap, c->prm.flags, row, F, G, NULL);
    else
        oracle_fitness(c->jobs, c->J, c->cap, c->prm.penalty, c->prm.flags, row, F, G);
}

static void score_population(oracle_ctx* c) {
    for (int32_t i = 0; i < c->N; ++i) score_row(c, &c->pop[(size_t)i * c->W], &c->F[i], &c->G[i]);
    c->f_valid = 1;
}

int oracle_evaluate(oracle_ctx* c, const int32_t* genomes, int64_t ld, int32_t n, double* fitness,
                    int32_t* gpus) {
    if (!c || !fitness) return ORACLE_ERR_NULL;
    if (!genomes) {
        if (!c->f_valid) score_population(c);
        memcpy(fitness, c->F, sizeof(double) * (size_t)c->N);
        if (gpus) memcpy(gpus, c->G, sizeof(int32_t) * (size_t)c->N);
        return ORACLE_OK;
    }
    if (ld < c->W || n < 0) return ORACLE_ERR_BAD_PARAM;
    for (int32_t i = 0; i < n; ++i) {
        int32_t g;
        score_row(c, &genomes[(size_t)i * (size_t)ld], &fitness[i], &g);
        if (gpus) gpus[i] = g;
    }
    return ORACLE_OK;
}

/* Indices of the k best of n scores (score descending, index ascending), returned in ascending index
 * order: truncation selection that keeps the survivors in the order they had. */
int oracle_keep_best(const double* F, int32_t n, int32_t k, int32_t* kept) {
    if (!F || !kept) return ORACLE_ERR_NULL;
    if (k < 0 || k > n) return ORACLE_ERR_BAD_PARAM;
    int32_t* order = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    char* keep = (char*)calloc((size_t)(n > 0 ? n : 1), 1);
    if (!order || !keep) { free(order); free(keep); return ORACLE_ERR_NOMEM; }
    for (int32_t i = 0; i < n; ++i) order[i] = i;
    /* heap sort under better(): the heap's root is the candidate that ranks last */
    for (int32_t i = 1; i < n; ++i) {
        int32_t c = i;
        while (c > 0) {
            int32_t p = (c - 1) / 2;
            if (!better(F, order[p], order[c])) break;
            int32_t t = order[p]; order[p] = order[c]; order[c] = t;
            c = p;
        }
    }
    for (int32_t end = n; end > 1; --end) {
        int32_t t = order[0]; order[0] = order[end - 1]; order[end - 1] = t;
        int32_t c = 0;
        for (;;) {
            int32_t l = 2 * c + 1, r = l + 1, w = c;
            if (l < end - 1 && better(F, order[w], order[l])) w = l;
            if (r < end - 1 && better(F, order[w], order[r])) w = r;
            if (w == c) break;
            t = order[c]; order[c] = order[w]; order[w] = t;
            c = w;
        }
    }
    for (int32_t r = 0; r < k; ++r) keep[order[r]] = 1; /* order[] is best first */
    int32_t at = 0;
    for (int32_t i = 0; i < n; ++i)
        if (keep[i]) kept[at++] = i;
    free(order);
    free(keep);
    return ORACLE_OK;
}

/* One generation of the paper's own scheme (Section 3.2.2 "Evolution" and "Selection"): from the K
 * candidates of G_i derive G'_i = the K candidates themselves, 2K children of K uniformly drawn
 * parent pairs (uniform crossover, no mutation) and K mutants of K uniformly drawn candidates
 * (each job redrawn with rate theta); score all 4K and keep the best K (score descending, position
 * in G'_i ascending), in the order they had in G'_i. */
static int truncation_generation(oracle_ctx* c, uint64_t seed) {
    const int32_t K = c->N, J = c->J;
    const uint64_t gen = c->gen_abs;
    const uint32_t thr = oracle_thr16(c->prm.p_mut);
    const size_t rows = (size_t)4 * K;
    int32_t* pool = (int32_t*)malloc(sizeof(int32_t) * rows * (size_t)J);
    double* F = (double*)malloc(sizeof(double) * rows);
    int32_t* G = (int32_t*)malloc(sizeof(int32_t) * rows);
    char* keep = NULL;
    if (!pool || !F || !G) { free(pool); free(F); free(G); return ORACLE_ERR_NOMEM; }
    memcpy(pool, c->pop, sizeof(int32_t) * (size_t)K * J);
    for (int32_t q = 0; q < K; ++q) { /* crossover children at rows K + 2q, K + 2q + 1 */
        int32_t pa = oracle_tournament(c->F, K, 1, seed, gen, (uint32_t)q, ORACLE_STREAM_SEL_A);
        int32_t pb = oracle_tournament(c->F, K, 1, seed, gen, (uint32_t)q, ORACLE_STREAM_SEL_B);
        c->parents[2 * q] = pa;
        c->parents[2 * q + 1] = pb;
        for (int32_t j = 0; j < J; ++j) {
            uint32_t W = oracle_word(seed, gen, (uint32_t)(2 * q), (uint32_t)j, ORACLE_STREAM_MUT);
            int flip = (int)(W & 1u);
            int32_t ga = c->pop[(size_t)pa * J + j], gb = c->pop[(size_t)pb * J + j];
            pool[((size_t)K + 2 * q) * J + j] = flip ? gb : ga;
            pool[((size_t)K + 2 * q + 1) * J + j] = flip ? ga : gb;
        }
    }
    for (int32_t m = 0; m < K; ++m) { /* mutants at rows 3K + m */
        int32_t from = oracle_tournament(c->F, K, 1, seed, gen, (uint32_t)m, ORACLE_STREAM_PICK);
        for (int32_t j = 0; j < J; ++j) {
            uint32_t W = oracle_word(seed, gen, (uint32_t)m, (uint32_t)j, ORACLE_STREAM_MUTANT);
            int32_t g = c->pop[(size_t)from * J + j];
            if ((W & 0xFFFFu) < thr) g = draw_gene(even_fraction(W), c->jobs[j].kmin, c->jobs[j].kmax);
            pool[((size_t)3 * K + m) * J + j] = g;
        }
    }
    for (size_t i = 0; i < rows; ++i)
        oracle_fitness(c->jobs, J, c->cap, c->prm.penalty, c->prm.flags, &pool[i * J], &F[i], &G[i]);
    int32_t* order = (int32_t*)malloc(sizeof(int32_t) * (size_t)K);
    if (!order) { free(pool); free(F); free(G); free(keep); return ORACLE_ERR_NOMEM; }
    int rc = oracle_keep_best(F, (int32_t)rows, K, order);
    if (rc) { free(order); free(pool); free(F); free(G); free(keep); return rc; }
    for (int32_t at = 0; at < K; ++at) {
        const size_t i = (size_t)order[at];
        memcpy(&c->next[(size_t)at * J], &pool[i * J], sizeof(int32_t) * (size_t)J);
        c->F[at] = F[i];
        c->G[at] = G[i];
    }
    int32_t* tmp = c->pop; c->pop = c->next; c->next = tmp;
    c->gen_abs = gen + 1;
    c->f_valid = 1;
    free(order); free(pool); free(F); free(G); free(keep);
    return ORACLE_OK;
}

int oracle_evolve(oracle_ctx* c, int32_t generations, uint64_t seed) {
    if (!c) return ORACLE_ERR_NULL;
    if (generations < 0) return ORACLE_ERR_BAD_PARAM;
    if (c->prm.flags & ORACLE_FLAG_TRUNCATION) {
        if (!c->f_valid) score_population(c);
        for (int32_t it = 0; it < generations; ++it) {
            int rc = truncation_generation(c, seed);
            if (rc) return rc;
        }
        return ORACLE_OK;
    }
    const int32_t N = c->N, J = c->W /* genes per candidate */, E = c->prm.elitism, T = c->prm.tournament;
    const uint32_t thr = oracle_thr16(c->prm.p_mut);
    if (!c->f_valid) score_population(c);
    for (int32_t it = 0; it < generations; ++it) {
        const uint64_t gen = c->gen_abs;
        /* survivors: the E best, unchanged, in rank order */
        oracle_top(c->F, N, E, c->elites);
        for (int32_t r = 0; r < E; ++r)
            memcpy(&c->next[(size_t)r * J], &c->pop[(size_t)c->elites[r] * J], sizeof(int32_t) * (size_t)J);
        /* every parent pair gives two complementary children, then each child mutates */
        for (int32_t q = 0; q < c->pairs; ++q) {
            int32_t pa = oracle_tournament(c->F, N, T, seed, gen, (uint32_t)q, ORACLE_STREAM_SEL_A);
            int32_t pb = oracle_tournament(c->F, N, T, seed, gen, (uint32_t)q, ORACLE_STREAM_SEL_B);
            c->parents[2 * q] = pa;
            c->parents[2 * q + 1] = pb;
            const int32_t slot0 = E + 2 * q, slot1 = slot0 + 1;
            const int32_t* A = &c->pop[(size_t)pa * J];
            const int32_t* B = &c->pop[(size_t)pb * J];
            for (int32_t j = 0; j < J; ++j) {
                const int32_t lo = gene_lo(c, j), hi = gene_hi(c, j);
                uint32_t W = oracle_word(seed, gen, (uint32_t)slot0, (uint32_t)j, ORACLE_STREAM_MUT);
                int flip = (int)(W & 1u); /* which child inherits the first parent's gene */
                int32_t child0 = flip ? B[j] : A[j];
                int32_t child1 = flip ? A[j] : B[j];
                if ((W & 0xFFFFu) < thr) child0 = draw_gene(even_fraction(W), lo, hi);
                c->next[(size_t)slot0 * J + j] = child0;
                if (slot1 < N) {
                    if ((W >> 16) < thr) child1 = draw_gene(odd_fraction(W), lo, hi);
                    c->next[(size_t)slot1 * J + j] = child1;
                }
            }
        }
        if (c->prm.flags & ORACLE_FLAG_PER_GPU) /* "Reorder": pack each job's workers, every new candidate */
            for (int32_t i = 0; i < N; ++i) oracle_reorder(&c->next[(size_t)i * J], J, c->J);
        int32_t* tmp = c->pop; c->pop = c->next; c->next = tmp;
        c->gen_abs = gen + 1;
        score_population(c);
    }
    return ORACLE_OK;
}

int oracle_best(oracle_ctx* c, int repair, int32_t* genome, int32_t* gpus_per_job, double* rate_per_job,
                double* fitness, int32_t* total_gpus, int32_t* index) {
    if (!c) return ORACLE_ERR_NULL;
    if (!c->f_valid) score_population(c);
    int32_t best;
    oracle_top(c->F, c->N, 1, &best);
    int32_t* row = (int32_t*)malloc(sizeof(int32_t) * (size_t)c->J);
    if (!row) return ORACLE_ERR_NOMEM;
    int rc = ORACLE_OK;
    double F = c->F[best];
    int32_t G = c->G[best];
    if (c->prm.flags & ORACLE_FLAG_PER_GPU) {
        /* the schedule as per-job exponents: what each job can run on the GPUs it holds; always fits */
        oracle_fitness_per_gpu(c->jobs, c->J, c->cap, c->prm.flags, &c->pop[(size_t)best * c->W], &F, &G, row);
    } else {
        memcpy(row, &c->pop[(size_t)best * c->J], sizeof(int32_t) * (size_t)c->J);
        if (repair) {
            rc = oracle_repair(c->jobs, c->J, c->cap, row);
            /* score of the repaired schedule: no penalty is left when it fits */
            oracle_fitness(c->jobs, c->J, c->cap, c->prm.penalty, c->prm.flags, row, &F, &G);
        }
    }
    for (int32_t j = 0; j < c->J; ++j) {
        double X; int32_t g;
        oracle_model(&c->jobs[j], row[j], &X, &g);
        if (gpus_per_job) gpus_per_job[j] = g;
        if (rate_per_job) rate_per_job[j] = X;
        if (genome) genome[j] = row[j];
    }
    if (fitness) *fitness = F;
    if (total_gpus) *total_gpus = G;
    if (index) *index = best;
    free(row);
    return rc;
}

int oracle_update_jobs(oracle_ctx* c, const oracle_job* jobs, int32_t n_jobs, const int32_t* remap,
                       int32_t capacity) {
    if (!c || !jobs || !remap) return ORACLE_ERR_NULL;
    int rc = oracle_validate_jobs(jobs, n_jobs);
    if (rc) return rc;
    if (capacity <= 0) return ORACLE_ERR_BAD_PARAM;
    for (int32_t j = 0; j < n_jobs; ++j)
        if (remap[j] < -1 || remap[j] >= c->J) return ORACLE_ERR_BAD_PARAM;
    oracle_job* nj = (oracle_job*)malloc(sizeof(oracle_job) * (size_t)n_jobs);
    if (!nj) return ORACLE_ERR_NOMEM;
    memcpy(nj, jobs, sizeof(oracle_job) * (size_t)n_jobs);
    if (c->prm.flags & ORACLE_FLAG_PER_GPU) {
        /* the cluster keeps its size; every candidate is refreshed and packed again */
        if (capacity != c->cap) { free(nj); return ORACLE_ERR_BAD_PARAM; }
        int32_t* inv = (int32_t*)malloc(sizeof(int32_t) * (size_t)c->J);
        char* is_new = (char*)calloc((size_t)n_jobs, 1);
        if (!inv || !is_new) { free(inv); free(is_new); free(nj); return ORACLE_ERR_NOMEM; }
        for (int32_t o = 0; o < c->J; ++o) inv[o] = -1;
        for (int32_t j = 0; j < n_jobs; ++j) {
            if (remap[j] >= 0) inv[remap[j]] = j; else is_new[j] = 1;
        }
        for (int32_t i = 0; i < c->N; ++i) {
            int32_t* row = &c->pop[(size_t)i * c->W];
            oracle_refresh(jobs, n_jobs, c->prm.flags, inv, c->J, is_new, row, c->W);
            oracle_reorder(row, c->W, n_jobs);
        }
        free(inv); free(is_new); free(c->jobs);
        c->jobs = nj;
        c->J = n_jobs;
        c->f_valid = 0;
        return ORACLE_OK;
    }
    size_t cells = (size_t)c->N * (size_t)n_jobs;
    int32_t* np = (int32_t*)malloc(sizeof(int32_t) * cells);
    int32_t* nn = (int32_t*)malloc(sizeof(int32_t) * cells);
    if (!np || !nn) { free(np); free(nn); free(nj); return ORACLE_ERR_NOMEM; }
    /* refresh: finished jobs' columns vanish, surviving jobs keep their gene
     * (clamped into the new limits), new jobs start at their smallest batch */
    for (int32_t i = 0; i < c->N; ++i)
        for (int32_t j = 0; j < n_jobs; ++j) {
            int32_t k = jobs[j].kmin;
            if (remap[j] >= 0) {
                k = c->pop[(size_t)i * c->J + remap[j]];
                if (k < jobs[j].kmin) k = jobs[j].kmin;
                if (k > jobs[j].kmax) k = jobs[j].kmax;
            }
            np[(size_t)i * n_jobs + j] = k;
        }
    free(c->pop); free(c->next); free(c->jobs);
    c->pop = np; c->next = nn; c->jobs = nj;
    c->J = n_jobs; c->W = n_jobs; c->cap = capacity;
    c->f_valid = 0;
    return ORACLE_OK;
}

int oracle_last_parents(oracle_ctx* c, int32_t* parents, int32_t* elites) {
    if (!c) return ORACLE_ERR_NULL;
    if (parents) memcpy(parents, c->parents, sizeof(int32_t) * 2 * (size_t)c->pairs);
    if (elites) memcpy(elites, c->elites, sizeof(int32_t) * (size_t)c->prm.elitism);
    return ORACLE_OK;
}

int oracle_generation(const oracle_ctx* c, uint64_t* gen_abs) {
    if (!c || !gen_abs) return ORACLE_ERR_NULL;
    *gen_abs = c->gen_abs;
    return ORACLE_OK;
}

int oracle_set_generation(oracle_ctx* c, uint64_t gen_abs) {
    if (!c) return ORACLE_ERR_NULL;
    c->gen_abs = gen_abs;
    return ORACLE_OK;
}

int32_t oracle_pairs(const oracle_ctx* c) { return c ? c->pairs : 0; }
