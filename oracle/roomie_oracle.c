/*
 * CPU oracle for the Roomie interference-model hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, step-by-step
 * statement of what the path computes, written from the paper.  It shares no
 * code with the CUDA implementation and must never be called from the product
 * path; only the tests, the smoke check and the benchmark's CPU-baseline leg
 * may load it.
 *
 * Arithmetic: integers for occupancy and time (1 tick = 1 ns), double for the
 * walk, the median, gamma and the pairwise slowdown; float (fixed summation
 * order) for the multi-model estimate and placement, where the method's
 * decision is taken in float32, with a double shadow kept beside it.
 *
 * Parity status: every function below is pinned by tests that do not call
 * back into this file (hand-derived values of Eq. 1, a block-by-block SM
 * filler, a 1-tick timeline stepper, closed forms, the printed count of
 * 112 500 alignment scenarios, brute-force argmin).  The one quantity the
 * paper gives no way to pin is the *quality* of the pairwise approximation
 * for three or more models (its 7-8 % / 90 % figures need its model set):
 * parity unpinned for that claim only; the N-way checker reports the gap.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_RANGE 2

typedef struct {
    uint32_t num_sms, regs_per_sm, smem_per_sm, threads_per_sm, blocks_per_sm;
} oracle_gpu_spec;

/* ------------------------------------------------------------------ *
 * Section 3.1, Eq. 1: theoretical occupancy o = W_b * b / W, where b is
 * the most restrictive of the per-SM limits.  The paper names warps,
 * registers and shared memory; the block-slot limit is added because the
 * modelled GPU states one.  The grid bounds how many blocks ever reach
 * one SM (ceil(grid / SMs) under round-robin distribution), which gives
 * the resident count b_res used downstream; o_theo keeps pure Eq. 1.
 *
 * limiter: 0 warps, 1 block slots, 2 registers, 3 shared memory (first
 * minimum in that order), 4 grid (only when the grid bound is stricter).
 * phi: per-SM demand at b_res, component-major [4][n]:
 *      warps, registers, shared-memory bytes, block slots.
 * ------------------------------------------------------------------ */
void oracle_occupancy(uint32_t n, const uint32_t *grid, const uint32_t *threads,
                      const uint32_t *regs, const uint32_t *smem,
                      const oracle_gpu_spec *spec,
                      uint32_t *b_lim, uint32_t *b_res, uint32_t *limiter,
                      uint32_t *warps, float *occ, float *occ_theo, uint32_t *phi,
                      uint32_t *n_unlaunchable)
{
    const uint64_t W = spec->threads_per_sm / 32;
    uint32_t bad = 0;
    for (uint32_t k = 0; k < n; ++k) {
        const uint64_t Wb = ((uint64_t)threads[k] + 31) / 32;
        const uint64_t INF = UINT64_MAX;
        uint64_t lim[4];
        lim[0] = Wb ? W / Wb : 0;                                   /* warp limit       */
        lim[1] = spec->blocks_per_sm;                               /* block-slot limit */
        const uint64_t regs_block = (uint64_t)regs[k] * 32 * Wb;    /* whole warps      */
        lim[2] = regs_block ? spec->regs_per_sm / regs_block : INF; /* register limit   */
        lim[3] = smem[k] ? spec->smem_per_sm / smem[k] : INF;       /* smem limit       */
        uint64_t b = lim[0];
        uint32_t which = 0;
        for (uint32_t c = 1; c < 4; ++c)
            if (lim[c] < b) { b = lim[c]; which = c; }
        const uint64_t b_grid = ((uint64_t)grid[k] + spec->num_sms - 1) / spec->num_sms;
        uint64_t br = b;
        if (b_grid < b) { br = b_grid; which = 4; }
        if (b == 0) ++bad;
        b_lim[k] = (uint32_t)b;
        b_res[k] = (uint32_t)br;
        limiter[k] = which;
        warps[k] = (uint32_t)(Wb * br);
        occ[k] = W ? (float)(Wb * br) / (float)W : 0.0f;
        occ_theo[k] = W ? (float)(Wb * b) / (float)W : 0.0f;
        phi[0 * (size_t)n + k] = (uint32_t)(Wb * br);
        phi[1 * (size_t)n + k] = (uint32_t)(br * regs_block);
        phi[2 * (size_t)n + k] = (uint32_t)(br * smem[k]);
        phi[3 * (size_t)n + k] = (uint32_t)br;
    }
    if (n_unlaunchable) *n_unlaunchable = bad;
}

/* ------------------------------------------------------------------ *
 * Timeline of one model's kernel sequence (Section 3.2, "Performance
 * drop": kernels run one after the other).  Durations and gaps are
 * quantised to integer nanosecond ticks with a float32 multiply and
 * round-half-even; a kernel lasts at least one tick.  start[k] is the
 * isolated start time; T = sum of kernel durations only (Eq. 4's
 * denominator), not the makespan.
 * Returns ORACLE_RANGE if a value is negative/non-finite or a profile's
 * timeline reaches 2^31 ticks.
 * ------------------------------------------------------------------ */
int oracle_timeline(uint32_t P, const uint32_t *offsets, const float *dur_us,
                    const float *gap_us, uint32_t *start, uint32_t *dt, uint64_t *T)
{
    int status = ORACLE_OK;
    for (uint32_t m = 0; m < P; ++m) {
        uint64_t t = 0, sum_d = 0;
        for (uint32_t k = offsets[m]; k < offsets[m + 1]; ++k) {
            float fd = dur_us[k] * 1000.0f, fg = gap_us[k] * 1000.0f;
            if (!(fd >= 0.0f && fd < 2147483648.0f)) { status = ORACLE_RANGE; fd = 0.0f; }
            if (!(fg >= 0.0f && fg < 2147483648.0f)) { status = ORACLE_RANGE; fg = 0.0f; }
            uint64_t d = (uint64_t)llrintf(fd), g = (uint64_t)llrintf(fg);
            if (d < 1) d = 1;
            start[k] = (uint32_t)t;
            dt[k] = (uint32_t)d;
            sum_d += d;
            t += d + g;
            if (t >= 2147483648ull) { status = ORACLE_RANGE; t = 0; }
        }
        T[m] = sum_d;
    }
    return status;
}

/* One model profile as the walk sees it. */
typedef struct {
    uint32_t q;
    const uint32_t *start, *dt;       /* ticks                                  */
    const uint32_t *phi;              /* base of [4][n_total], already offset   */
    size_t phi_stride;                /* n_total                                */
} prof_view;

/* Eq. 2 for two active kernels: some resource's combined demand exceeds the SM. */
static int interferes(const prof_view *a, uint32_t ka, const prof_view *b, uint32_t kb,
                      const uint64_t cap[4])
{
    for (int c = 0; c < 4; ++c) {
        uint64_t s = (uint64_t)a->phi[c * a->phi_stride + ka] + b->phi[c * b->phi_stride + kb];
        if (s > cap[c]) return 1;
    }
    return 0;
}

/* ------------------------------------------------------------------ *
 * Algorithm 1, inner while loop, for one alignment (s_i, s_j).
 *
 * mode 0 (TIMELINE): both suffixes start at time 0; the pairing (k_i, k_j)
 * is scored on the time both kernels run together; the kernel that ends
 * first is replaced by its model's next kernel (Section 3.2), both on a
 * tie.  When the predicate of Eq. 2 holds, the overlapped time is charged
 * in proportion to occupancy, d * o_i / (o_i + o_j) with d the overlap
 * (Algorithm 1 line 13; the two-phase paragraph ends interference when the
 * shorter kernel ends).  o_i/(o_i+o_j) = warps_i/(warps_i+warps_j).
 *
 * mode 1 (LOCKSTEP): Algorithm 1 to the letter: both indices advance
 * together and the whole duration d_{k_i} is charged.
 * ------------------------------------------------------------------ */
static void walk(const prof_view *A, const prof_view *B, uint32_t si, uint32_t sj,
                 const uint64_t cap[4], int mode,
                 double *delta_i, double *delta_j, uint64_t *V, uint64_t *evals)
{
    uint32_t ki = si, kj = sj;
    const int64_t base_i = A->start[si], base_j = B->start[sj];
    double di = 0.0, dj = 0.0;
    uint64_t v = 0, ev = 0;
    while (ki < A->q && kj < B->q) {
        const int64_t a0 = (int64_t)A->start[ki] - base_i, a1 = a0 + A->dt[ki];
        const int64_t b0 = (int64_t)B->start[kj] - base_j, b1 = b0 + B->dt[kj];
        const double wa = A->phi[ki], wb = B->phi[kj];            /* warps component */
        ++ev;
        if (mode == 0) {
            const int64_t ov = (a1 < b1 ? a1 : b1) - (a0 > b0 ? a0 : b0);
            if (ov > 0 && wa > 0 && wb > 0 && interferes(A, ki, B, kj, cap)) {
                di += (double)ov * wa / (wa + wb);
                dj += (double)ov * wb / (wa + wb);
                v += (uint64_t)ov;
            }
            if (a1 < b1) ++ki;
            else if (b1 < a1) ++kj;
            else { ++ki; ++kj; }
        } else {
            if (wa > 0 && wb > 0 && interferes(A, ki, B, kj, cap)) {
                di += (double)A->dt[ki] * wa / (wa + wb);
                dj += (double)B->dt[kj] * wb / (wa + wb);
                v += (uint64_t)A->dt[ki] + B->dt[kj];
            }
            ++ki; ++kj;
        }
    }
    *delta_i = di; *delta_j = dj; *V = v; *evals = ev;
}

/* ------------------------------------------------------------------ *
 * Section 3.2 in full ("Adjusted occupancy", "Two-phase execution",
 * "Performance drop") for one alignment: the two kernel sequences are run
 * together from (s_i, s_j); whenever the two active kernels' combined demand
 * exceeds the SM (Eq. 2) each runs with the blocks b~ the partition policy
 * leaves it, i.e. at occupancy o~ = W_b * b~ / W, and progresses at the rate
 * o~/o = b~/b (its execution time is inversely proportional to its adjusted
 * occupancy); the interference ends when the first of the two completes, and
 * the other continues at full occupancy with what is left of it (two-phase
 * execution), possibly against the finished model's next kernel.  Idle gaps
 * between kernels are not stretched.  The delay of a model is the time its
 * kernels took beyond their isolated durations; the run ends when either
 * model has completed its last kernel.
 *
 * Time is in integer ticks here as everywhere else, so that the order of
 * events (which kernel completes first, which one started earlier) is a
 * matter of integers and not of floating-point rounding.  The work of a
 * kernel is counted in block-ticks: d_k * b in all; in one tick a kernel
 * running with b~ blocks does b~ of them, so it completes after
 * ceil(work left / b~) ticks (its last tick may be only partly used) and a
 * kernel that keeps all its blocks takes exactly d_k.  A tick in which a
 * kernel runs with b~ of its b blocks delays it by (b - b~) / b.
 *
 * Policies for b~ (the paper names them, it does not spell them out):
 *   2 EQUAL    each kernel may use half of every SM resource;
 *   3 PRIORITY model i's kernel keeps its blocks, model j's kernel gets what
 *              is left of every resource;
 *   4 FCFS     the same with priority to the kernel that started earlier
 *              (model i on a tie).
 * A kernel left without a single block waits while the other runs at full
 * occupancy; under EQUAL, when neither fits into half an SM, the kernel
 * that started earlier (model i on a tie) runs alone.
 * Per-block demands come from phi at the resident block count b.  A kernel
 * without a resident block (b = 0) never interferes and takes d_k.
 * ------------------------------------------------------------------ */
typedef struct { uint64_t wb, regs, smem, b; } block_need;

static block_need need_of(const prof_view *p, uint32_t k)
{
    block_need n;
    n.b = p->phi[3 * p->phi_stride + k];
    n.wb = n.b ? p->phi[0 * p->phi_stride + k] / n.b : 0;
    n.regs = n.b ? p->phi[1 * p->phi_stride + k] / n.b : 0;
    n.smem = n.b ? p->phi[2 * p->phi_stride + k] / n.b : 0;
    return n;
}

/* blocks of a kernel that fit into the given amounts of the four resources, at most its own b */
static uint64_t blocks_in(const block_need *n, uint64_t warps, uint64_t regs, uint64_t smem, uint64_t slots)
{
    uint64_t b = n->b;
    if (n->wb && warps / n->wb < b) b = warps / n->wb;
    if (n->regs && regs / n->regs < b) b = regs / n->regs;
    if (n->smem && smem / n->smem < b) b = smem / n->smem;
    if (slots < b) b = slots;
    return b;
}

/* one model during the co-run */
typedef struct {
    const prof_view *p;
    uint32_t k;        /* its active kernel, or the next one while it idles              */
    uint64_t b;        /* blocks that kernel runs with alone (1 stands in for b = 0)     */
    uint64_t left;     /* work left, block-ticks                                         */
    uint64_t idle;     /* ticks of gap left before kernel k starts                       */
    uint64_t began;    /* tick at which kernel k started                                 */
    double delay;      /* ticks lost so far                                              */
} corun;

static void corun_start_kernel(corun *m, uint64_t now)
{
    const uint64_t b = m->p->phi[3 * m->p->phi_stride + m->k];
    m->b = b ? b : 1;
    m->left = (uint64_t)m->p->dt[m->k] * m->b;
    if (m->idle == 0) m->began = now;
}

static void walk_detailed(const prof_view *A, const prof_view *B, uint32_t si, uint32_t sj,
                          const uint64_t cap[4], int policy,
                          double *delta_i, double *delta_j, uint64_t *V, uint64_t *evals)
{
    corun M[2];
    uint64_t now = 0, ev = 0;
    memset(M, 0, sizeof(M));
    M[0].p = A; M[0].k = si; M[1].p = B; M[1].k = sj;
    corun_start_kernel(&M[0], 0);
    corun_start_kernel(&M[1], 0);
    while (M[0].k < A->q && M[1].k < B->q) {
        ++ev;
        /* blocks each active kernel runs with until the next event */
        uint64_t bt[2] = { M[0].b, M[1].b };
        if (M[0].idle == 0 && M[1].idle == 0 && A->phi[M[0].k] > 0 && B->phi[M[1].k] > 0 &&
            interferes(A, M[0].k, B, M[1].k, cap)) {
            const block_need n0 = need_of(A, M[0].k), n1 = need_of(B, M[1].k);
            if (policy == 2) {
                bt[0] = blocks_in(&n0, cap[0] / 2, cap[1] / 2, cap[2] / 2, cap[3] / 2);
                bt[1] = blocks_in(&n1, cap[0] / 2, cap[1] / 2, cap[2] / 2, cap[3] / 2);
                if (bt[0] == 0 && bt[1] == 0) { if (M[0].began <= M[1].began) bt[0] = n0.b; else bt[1] = n1.b; }
                else if (bt[0] == 0) bt[1] = n1.b;
                else if (bt[1] == 0) bt[0] = n0.b;
            } else {
                const int first = (policy == 3 || M[0].began <= M[1].began) ? 0 : 1;
                const block_need *hi = first == 0 ? &n0 : &n1, *lo = first == 0 ? &n1 : &n0;
                bt[1 - first] = blocks_in(lo, cap[0] - hi->wb * hi->b, cap[1] - hi->regs * hi->b,
                                          cap[2] - hi->smem * hi->b, cap[3] - hi->b);
            }
        }
        /* ticks to the next event: a gap ends or a kernel completes */
        uint64_t until[2], step = UINT64_MAX;
        for (int m = 0; m < 2; ++m) {
            until[m] = M[m].idle > 0 ? M[m].idle
                     : bt[m] > 0 ? (M[m].left + bt[m] - 1) / bt[m] : UINT64_MAX;
            if (until[m] < step) step = until[m];
        }
        if (step == UINT64_MAX) break;                          /* cannot happen: one of the two always runs */
        now += step;
        for (int m = 0; m < 2; ++m) {
            corun *c = &M[m];
            if (c->idle > 0) {
                c->idle -= step;
                if (c->idle == 0) c->began = now;
                continue;
            }
            c->delay += (double)(step * (c->b - bt[m])) / (double)c->b;
            if (until[m] == step) {                                /* this kernel completes */
                const uint32_t done = c->k++;
                if (c->k < c->p->q) {
                    c->idle = (uint64_t)c->p->start[c->k] - ((uint64_t)c->p->start[done] + c->p->dt[done]);
                    corun_start_kernel(c, now);
                }
            } else {
                c->left -= step * bt[m];
            }
        }
    }
    *delta_i = M[0].delay; *delta_j = M[1].delay; *V = 0; *evals = ev;   /* V is not defined in this mode */
}

static int cmp_double(const void *x, const void *y)
{
    double a = *(const double *)x, b = *(const double *)y;
    return (a > b) - (a < b);
}

/* median; even count -> mean of the two middle values; empty -> 0 */
static double median(double *v, size_t n)
{
    if (n == 0) return 0.0;
    qsort(v, n, sizeof(double), cmp_double);
    return (n & 1) ? v[n / 2] : 0.5 * (v[n / 2 - 1] + v[n / 2]);
}

/* candidate start indices of one model: evenly spaced grid of n_align
 * points, duplicates removed; n_align = 0 -> every index */
static uint32_t start_grid(uint32_t q, uint32_t n_align, uint32_t *out)
{
    if (n_align == 0) { for (uint32_t t = 0; t < q; ++t) out[t] = t; return q; }
    uint32_t n = 0;
    for (uint32_t t = 0; t < n_align; ++t) {
        uint32_t s = (uint32_t)(((uint64_t)t * q) / n_align);
        if (n == 0 || out[n - 1] != s) out[n++] = s;
    }
    return n;
}

typedef struct {
    uint32_t P, K;
    const uint32_t *offsets, *start, *dt, *phi;
    const uint64_t *T;
    oracle_gpu_spec spec;
} oracle_library;

static prof_view view(const oracle_library *L, uint32_t m)
{
    prof_view v;
    v.q = L->offsets[m + 1] - L->offsets[m];
    v.start = L->start + L->offsets[m];
    v.dt = L->dt + L->offsets[m];
    v.phi = L->phi + L->offsets[m];
    v.phi_stride = L->K;
    return v;
}

/* ------------------------------------------------------------------ *
 * Algorithm 1, lines 6-20, for one unordered pair (both directions come
 * from the same walks): alignment set C_ij, delay set D_ij, median, the
 * overlap factor gamma_ij = max(q_i/q_j, 1), and the pairwise relative
 * slowdown gamma_ij * median(D_ij) / T_i (Eq. 4's form of mu for M={i,j}).
 *
 * Optional per-alignment outputs (capacity `cap_align` entries each):
 * s_i, s_j, delta_i, delta_j, V, evals.  Returns the number of alignments
 * kept; *evals_total gets the number of scored pairings.
 * ------------------------------------------------------------------ */
uint32_t oracle_pair(const oracle_library *L, uint32_t a, uint32_t b,
                     int mode, uint32_t n_align, int start_filter,
                     double *P_ab, double *P_ba, uint64_t *evals_total,
                     uint32_t cap_align, uint32_t *out_si, uint32_t *out_sj,
                     double *out_di, double *out_dj, uint64_t *out_V, uint64_t *out_evals)
{
    const prof_view A = view(L, a), B = view(L, b);
    const uint64_t cap[4] = { L->spec.threads_per_sm / 32, L->spec.regs_per_sm,
                              L->spec.smem_per_sm, L->spec.blocks_per_sm };
    uint32_t *ga = (uint32_t *)malloc(sizeof(uint32_t) * (A.q + n_align + 1));
    uint32_t *gb = (uint32_t *)malloc(sizeof(uint32_t) * (B.q + n_align + 1));
    const uint32_t na = start_grid(A.q, n_align, ga), nb = start_grid(B.q, n_align, gb);
    double *Di = (double *)malloc(sizeof(double) * ((size_t)na * nb + 1));
    double *Dj = (double *)malloc(sizeof(double) * ((size_t)na * nb + 1));
    uint32_t kept = 0;
    uint64_t ev_sum = 0;
    for (uint32_t x = 0; x < na; ++x)
        for (uint32_t y = 0; y < nb; ++y) {
            const uint32_t si = ga[x], sj = gb[y];
            if (start_filter &&
                !(A.phi[si] > 0 && B.phi[sj] > 0 && interferes(&A, si, &B, sj, cap)))
                continue;                        /* not an interference starting point */
            double di, dj; uint64_t v, ev;
            if (mode >= 2) walk_detailed(&A, &B, si, sj, cap, mode, &di, &dj, &v, &ev);
            else walk(&A, &B, si, sj, cap, mode, &di, &dj, &v, &ev);
            if (kept < cap_align) {
                if (out_si) out_si[kept] = si;
                if (out_sj) out_sj[kept] = sj;
                if (out_di) out_di[kept] = di;
                if (out_dj) out_dj[kept] = dj;
                if (out_V) out_V[kept] = v;
                if (out_evals) out_evals[kept] = ev;
            }
            Di[kept] = di; Dj[kept] = dj; ++kept;
            ev_sum += ev;
        }
    const double med_i = median(Di, kept), med_j = median(Dj, kept);
    const double qa = A.q, qb = B.q;
    const double g_ab = qa / qb > 1.0 ? qa / qb : 1.0;
    const double g_ba = qb / qa > 1.0 ? qb / qa : 1.0;
    *P_ab = L->T[a] ? g_ab * med_i / (double)L->T[a] : 0.0;
    *P_ba = L->T[b] ? g_ba * med_j / (double)L->T[b] : 0.0;
    if (evals_total) *evals_total = ev_sum;
    free(ga); free(gb); free(Di); free(Dj);
    return kept;
}

/* ------------------------------------------------------------------ *
 * All pairs of the library: Pm[i*P + j] = slowdown of i caused by j.
 * Unordered pairs a <= b with index in [pair_begin, pair_end) of the
 * row-major upper triangle (diagonal included: two replicas of one model)
 * are evaluated; others are left untouched.  The diagonal takes the
 * i-side median.  Returns the number of scored pairings.  Pairs are
 * independent, so they are spread over the host's cores.
 * ------------------------------------------------------------------ */
uint64_t oracle_pair_matrix(const oracle_library *L, int mode, uint32_t n_align,
                            int start_filter, uint64_t pair_begin, uint64_t pair_end,
                            double *Pm, int num_threads)
{
    const uint64_t P = L->P, total = P * (P + 1) / 2;
    if (pair_end > total) pair_end = total;
    uint64_t evals = 0;
    /* pair index -> (a, b) table for the requested range */
    const uint64_t npairs = pair_end > pair_begin ? pair_end - pair_begin : 0;
    uint32_t *pa = (uint32_t *)malloc(sizeof(uint32_t) * (npairs + 1));
    uint32_t *pb = (uint32_t *)malloc(sizeof(uint32_t) * (npairs + 1));
    uint64_t idx = 0, w = 0;
    for (uint32_t a = 0; a < P; ++a)
        for (uint32_t b = a; b < P; ++b, ++idx)
            if (idx >= pair_begin && idx < pair_end) { pa[w] = a; pb[w] = b; ++w; }
#ifdef _OPENMP
    if (num_threads > 0) omp_set_num_threads(num_threads);
#else
    (void)num_threads;
#endif
    #pragma omp parallel for schedule(dynamic, 1) reduction(+ : evals)
    for (int64_t p = 0; p < (int64_t)npairs; ++p) {
        double ab, ba; uint64_t ev;
        oracle_pair(L, pa[p], pb[p], mode, n_align, start_filter, &ab, &ba, &ev,
                    0, NULL, NULL, NULL, NULL, NULL, NULL);
        Pm[(size_t)pa[p] * P + pb[p]] = ab;
        if (pa[p] != pb[p]) Pm[(size_t)pb[p] * P + pa[p]] = ba;
        evals += ev;
    }
    free(pa); free(pb);
    return evals;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ *
 * Algorithm 1, outer loops, given the pairwise terms: for the model set
 * M = residents (in slot order) followed by the incoming model,
 *   mu_i = sum over the other members j of Pm[id_i][id_j]
 * (T~_i = T_i + sum_j gamma_ij * Delta_ij divided through by T_i), and
 * the mean over M.  float32 with additions in slot order, as the method
 * defines it; mu64 / mean64 are the same sums in double.
 * ------------------------------------------------------------------ */
void oracle_multi_estimate(const float *Pm, uint32_t P, const int32_t *ids, uint32_t r,
                           int32_t incoming, float *mu, float *mean,
                           double *mu64, double *mean64)
{
    int32_t M[65];
    uint32_t m = 0;
    for (uint32_t t = 0; t < r && m < 64; ++t) M[m++] = ids[t];
    M[m++] = incoming;
    float tot = 0.0f; double tot64 = 0.0;
    for (uint32_t i = 0; i < m; ++i) {
        float s = 0.0f; double s64 = 0.0;
        for (uint32_t j = 0; j < m; ++j) {
            if (j == i) continue;
            const float p = Pm[(size_t)M[i] * P + M[j]];
            s = s + p; s64 += (double)p;
        }
        if (mu) mu[i] = s;
        if (mu64) mu64[i] = s64;
        tot = tot + s; tot64 += s64;
    }
    if (mean) *mean = tot / (float)m;
    if (mean64) *mean64 = tot64 / (double)m;
}

/* ------------------------------------------------------------------ *
 * Algorithm 2 applied to a stream of arrivals.  For arrival n (tick =
 * tick0 + n): residents whose expiry tick has come are removed (order
 * kept); every GPU with a free slot is scored what-if with the incoming
 * model added; a GPU is admissible when its mean drop is < lambda; the
 * admissible GPU with the lowest mean wins, lowest index on ties; no
 * admissible GPU -> -1 (deferred) and nothing is added.
 *
 * near_tie[n] (optional) = 1 when, in the double shadow, the winner's score
 * is within 1e-5 relative of another candidate's or of lambda: decisions
 * that float rounding of the pairwise matrix could legitimately flip.
 *
 * Variants (Section 3.4: the objective "can be easily substituted"; the
 * comment in Algorithm 2 asks that "no variant has a performance drop beyond
 * lambda"):
 *   admit_rule 0: mean drop < lambda (Algorithm 2 as printed), 1: the
 *                 largest member drop < lambda;
 *   objective  0: lowest mean drop (as printed), 1: lowest largest member
 *                 drop, 2: lowest drop of the arriving model.
 * ------------------------------------------------------------------ */
void oracle_place(const float *Pm, uint32_t P, uint32_t G, uint32_t R,
                  int32_t *ids, uint32_t *expiry, uint32_t *count, uint32_t *tick,
                  const int32_t *arr_id, const uint32_t *arr_life, uint32_t n,
                  float lambda, int admit_rule, int objective,
                  int32_t *gpu_out, float *mean_out, float *mu_arr_out,
                  uint8_t *near_tie)
{
    float *mu = (float *)malloc(sizeof(float) * (R + 1));
    double *mu64 = (double *)malloc(sizeof(double) * (R + 1));
    double *admit64_g = (double *)malloc(sizeof(double) * (G ? G : 1));   /* shadow; < 0: no free slot */
    double *score64_g = (double *)malloc(sizeof(double) * (G ? G : 1));
    for (uint32_t a = 0; a < n; ++a) {
        const uint32_t now = *tick + a;
        for (uint32_t g = 0; g < G; ++g) {                 /* departures */
            uint32_t w = 0;
            for (uint32_t s = 0; s < count[g]; ++s) {
                const uint32_t e = expiry[g * R + s];
                if (e != 0 && e <= now) continue;
                ids[g * R + w] = ids[g * R + s];
                expiry[g * R + w] = e;
                ++w;
            }
            for (uint32_t s = w; s < R; ++s) { ids[g * R + s] = -1; expiry[g * R + s] = 0; }
            count[g] = w;
        }
        int32_t best = -1; float best_mean = 0.0f, best_mu = 0.0f, best_score = 0.0f;
        for (uint32_t g = 0; g < G; ++g) {
            admit64_g[g] = -1.0; score64_g[g] = -1.0;
            if (count[g] >= R) continue;                   /* no free slot */
            float mean; double mean64;
            oracle_multi_estimate(Pm, P, ids + g * R, count[g], arr_id[a], mu, &mean, mu64, &mean64);
            float worst = 0.0f; double worst64 = 0.0;
            for (uint32_t i = 0; i <= count[g]; ++i) {
                if (mu[i] > worst) worst = mu[i];
                if (mu64[i] > worst64) worst64 = mu64[i];
            }
            const float admit = admit_rule == 1 ? worst : mean;
            const float score = objective == 1 ? worst : objective == 2 ? mu[count[g]] : mean;
            admit64_g[g] = admit_rule == 1 ? worst64 : mean64;
            score64_g[g] = objective == 1 ? worst64 : objective == 2 ? mu64[count[g]] : mean64;
            if (!(admit < lambda)) continue;               /* Algorithm 2 line 7 */
            if (best < 0 || score < best_score) {
                best = (int32_t)g; best_score = score; best_mean = mean; best_mu = mu[count[g]];
            }
        }
        if (near_tie) {
            uint8_t nt = 0;
            const double tol = 1e-5, lam = (double)lambda;
            for (uint32_t g = 0; g < G; ++g) {
                if (admit64_g[g] < 0.0) continue;
                if (fabs(admit64_g[g] - lam) <= tol * fabs(lam)) nt = 1;       /* admission within rounding */
                if (best >= 0 && (int32_t)g != best && admit64_g[g] < lam * (1.0 + tol)) {
                    const double x = score64_g[g], y = score64_g[best];
                    if (fabs(x - y) <= tol * fmax(fabs(x), fabs(y))) nt = 1;     /* two candidates within rounding */
                }
            }
            near_tie[a] = nt;
        }
        gpu_out[a] = best;
        if (mean_out) mean_out[a] = best >= 0 ? best_mean : 0.0f;
        if (mu_arr_out) mu_arr_out[a] = best >= 0 ? best_mu : 0.0f;
        if (best >= 0) {
            const uint32_t s = count[best]++;
            ids[best * R + s] = arr_id[a];
            expiry[best * R + s] = arr_life[a] ? now + arr_life[a] : 0;
        }
    }
    *tick += n;
    free(mu); free(mu64); free(admit64_g); free(score64_g);
}

/* ------------------------------------------------------------------ *
 * Placement quality (Section 5, "Deployment accuracy evaluation against
 * optimal strategies"): the deployment of n models on G identical GPUs
 * (at most R per GPU) with the lowest average predicted drop, found by
 * trying every assignment.  With the pairwise-sum estimate of Algorithm 1
 * the drop of model i is the sum of Pm[m_i][m_j] over the other models j
 * on its GPU, so the average drop of a deployment is
 *     cost = ( sum over i < j on the same GPU of (Pm[m_i][m_j] + Pm[m_j][m_i]) ) / n.
 * The value is DEFINED in float32: each pair term is one float add, terms are
 * accumulated model by model (j ascending, and for each j its partners
 * i < j ascending), one division at the end; cost64 is the same in double.
 * ------------------------------------------------------------------ */
float oracle_assignment_cost(const float *Pm, uint32_t P, const int32_t *models, uint32_t n,
                             const int32_t *gpu_of, double *cost64)
{
    float tot = 0.0f; double tot64 = 0.0;
    for (uint32_t j = 1; j < n; ++j)
        for (uint32_t i = 0; i < j; ++i) {
            if (gpu_of[i] < 0 || gpu_of[i] != gpu_of[j]) continue;
            const float a = Pm[(size_t)models[i] * P + models[j]], b = Pm[(size_t)models[j] * P + models[i]];
            tot = tot + (a + b);
            tot64 += (double)a + (double)b;
        }
    if (cost64) *cost64 = tot64 / (double)n;
    return tot / (float)n;
}

/* every assignment of models 1..n-1 (model 0 sits on GPU 0: the GPUs are identical) */
static void optimal_rec(const float *Pm, uint32_t P, const int32_t *models, uint32_t n, uint32_t G, uint32_t R,
                        uint32_t k, int32_t *gpu_of, uint32_t *load, float *best, int32_t *best_assign,
                        uint64_t *tried)
{
    if (k == n) {
        const float c = oracle_assignment_cost(Pm, P, models, n, gpu_of, NULL);
        ++*tried;
        if (*best < 0.0f || c < *best) { *best = c; memcpy(best_assign, gpu_of, sizeof(int32_t) * n); }
        return;
    }
    for (uint32_t g = 0; g < G; ++g) {
        if (load[g] >= R) continue;
        gpu_of[k] = (int32_t)g; ++load[g];
        optimal_rec(Pm, P, models, n, G, R, k + 1, gpu_of, load, best, best_assign, tried);
        --load[g];
    }
}

/* returns the lowest cost (float32) over all feasible assignments, -1 if none exists (n > G*R);
 * best_assign[n] gets one optimal assignment (the first found in lexicographic order), tried the count */
float oracle_optimal_assignment(const float *Pm, uint32_t P, const int32_t *models, uint32_t n,
                                uint32_t G, uint32_t R, int32_t *best_assign, uint64_t *tried)
{
    int32_t *gpu_of = (int32_t *)malloc(sizeof(int32_t) * (n + 1));
    uint32_t *load = (uint32_t *)calloc(G + 1, sizeof(uint32_t));
    float best = -1.0f;
    uint64_t t = 0;
    if (n > 0 && R > 0 && G > 0) {
        gpu_of[0] = 0; load[0] = 1;
        optimal_rec(Pm, P, models, n, G, R, 1, gpu_of, load, &best, best_assign, &t);
    }
    if (tried) *tried = t;
    free(gpu_of); free(load);
    return best;
}
