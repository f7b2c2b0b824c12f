/*
 * CPU oracle for the dense tensor contraction
 *
 *     C[Pi_C(I_m u I_n)] <- alpha * sum_{I_k} A[Pi_A(I_m u I_k)] * B[Pi_B(I_k u I_n)]
 *                           + beta * C[Pi_C(I_m u I_n)]                       (Eq. 2 / Eq. 3)
 *
 * written out as the naive loop nest of Listing 3: one loop per free index,
 * an accumulator, one loop per contracted index inside, and the alpha/beta
 * update of C after the contracted loops.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is deliberately plain and slow, it shares no
 * code with the CUDA library, and only the tests, the smoke check and the
 * benchmark's cpu-baseline leg may call it.  Nothing here is blocked, fused,
 * packed or reordered; the only concession to run time is that the outermost
 * free loop may be split across threads (each output is still produced by one
 * thread running the plain inner loops).
 *
 * Conventions: every operand value is widened exactly to double, the
 * accumulator is double, the result is returned as double.  A tensor is
 * described by (nmodes, extent[], stride[] in elements, label[]); a label that
 * occurs in A and C is free in A (I_m), in B and C free in B (I_n), in A and B
 * contracted (I_k) (Sec. 2.2).  Where the paper is silent: beta == 0 means the
 * old C is not read; alpha == 0 takes no shortcut.
 *
 * Parity pins (tests/test_oracle_*.py): brute-force flatten-to-matrix multiply
 * on small-integer inputs (exact), numpy einsum, the 2-D case against Listing 1,
 * all-ones / identity-B / rank-one / index-encoding closed forms, relabelling,
 * storage-permutation, A<->B swap and alpha/beta linearity invariants.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAX_MODES 32

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_F16 = 2, ORACLE_F64 = 3 /* A, B and the old C stored as double */ };

enum {
    ORACLE_OK = 0,
    ORACLE_ERR_ARG = 1,      /* NULL pointer, bad mode count, bad extent or stride */
    ORACLE_ERR_LABELS = 2,   /* label twice in a tensor, in all three, or in only one */
    ORACLE_ERR_EXTENT = 3    /* the two carriers of a label disagree on its extent */
};

typedef struct {
    int32_t nmodes;
    const int64_t *extent;
    const int64_t *stride;
    const int32_t *label;
} oracle_tensor_t;

/* the old value of C: stored as float, except for ORACLE_F64 */
static double load_c_old(const void *base, int64_t off, int dtype)
{
    return dtype == ORACLE_F64 ? ((const double *)base)[off] : (double)((const float *)base)[off];
}

/* exact widening of one stored operand element */
static double load_operand(const void *base, int64_t off, int dtype)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)base)[off];
    if (dtype == ORACLE_F64)
        return ((const double *)base)[off];
    uint16_t h = ((const uint16_t *)base)[off];
    if (dtype == ORACLE_BF16) {
        uint32_t u = (uint32_t)h << 16;
        float f;
        memcpy(&f, &u, 4);
        return (double)f;
    }
    /* IEEE binary16 */
    int sign = (h >> 15) & 1, ex = (h >> 10) & 0x1f, man = h & 0x3ff;
    double v;
    if (ex == 0)
        v = ldexp((double)man, -24);
    else if (ex == 31)
        v = man ? NAN : INFINITY;
    else
        v = ldexp((double)(man | 0x400), ex - 25);
    return sign ? -v : v;
}

static int find_label(const oracle_tensor_t *t, int32_t label)
{
    for (int i = 0; i < t->nmodes; ++i)
        if (t->label[i] == label)
            return i;
    return -1;
}

static int check_tensor(const oracle_tensor_t *t)
{
    if (!t || t->nmodes < 0 || t->nmodes > ORACLE_MAX_MODES)
        return ORACLE_ERR_ARG;
    if (t->nmodes > 0 && (!t->extent || !t->stride || !t->label))
        return ORACLE_ERR_ARG;
    for (int i = 0; i < t->nmodes; ++i) {
        if (t->extent[i] < 1 || t->stride[i] < 1)
            return ORACLE_ERR_ARG;
        for (int j = 0; j < i; ++j)
            if (t->label[i] == t->label[j])
                return ORACLE_ERR_LABELS;
    }
    return ORACLE_OK;
}

/* The loop structure of one contraction: which modes are free (they index C)
 * and which are contracted, each with its stride in the tensors carrying it. */
typedef struct {
    int nfree;                         /* = d_C, in C's storage order           */
    int64_t free_ext[ORACLE_MAX_MODES];
    int64_t free_sA[ORACLE_MAX_MODES]; /* 0 when the mode is not in A           */
    int64_t free_sB[ORACLE_MAX_MODES];
    int64_t free_sC[ORACLE_MAX_MODES];
    int ncon;                          /* contracted modes, in A's order        */
    int64_t con_ext[ORACLE_MAX_MODES];
    int64_t con_sA[ORACLE_MAX_MODES];
    int64_t con_sB[ORACLE_MAX_MODES];
} loops_t;

static int build_loops(const oracle_tensor_t *A, const oracle_tensor_t *B,
                       const oracle_tensor_t *C, loops_t *L)
{
    int rc;
    if ((rc = check_tensor(A)) || (rc = check_tensor(B)) || (rc = check_tensor(C)))
        return rc;
    memset(L, 0, sizeof *L);
    /* free modes: every mode of C must be in exactly one of A, B */
    for (int i = 0; i < C->nmodes; ++i) {
        int ia = find_label(A, C->label[i]), ib = find_label(B, C->label[i]);
        if ((ia >= 0) == (ib >= 0))
            return ORACLE_ERR_LABELS; /* in all three, or only in C */
        int64_t e = ia >= 0 ? A->extent[ia] : B->extent[ib];
        if (e != C->extent[i])
            return ORACLE_ERR_EXTENT;
        int f = L->nfree++;
        L->free_ext[f] = e;
        L->free_sA[f] = ia >= 0 ? A->stride[ia] : 0;
        L->free_sB[f] = ib >= 0 ? B->stride[ib] : 0;
        L->free_sC[f] = C->stride[i];
    }
    /* contracted modes: in A and B, not in C */
    for (int i = 0; i < A->nmodes; ++i) {
        if (find_label(C, A->label[i]) >= 0)
            continue;
        int ib = find_label(B, A->label[i]);
        if (ib < 0)
            return ORACLE_ERR_LABELS; /* only in A */
        if (A->extent[i] != B->extent[ib])
            return ORACLE_ERR_EXTENT;
        int c = L->ncon++;
        L->con_ext[c] = A->extent[i];
        L->con_sA[c] = A->stride[i];
        L->con_sB[c] = B->stride[ib];
    }
    for (int i = 0; i < B->nmodes; ++i)
        if (find_label(C, B->label[i]) < 0 && find_label(A, B->label[i]) < 0)
            return ORACLE_ERR_LABELS; /* only in B */
    return ORACLE_OK;
}

/* Listing 3, lines 9-16, for one tuple of free indices: the contracted loops
 * with their accumulator, then the update of C.  abs_out gets sum |a||b|. */
static void one_output(const loops_t *L, const void *A, const void *B, int dtype,
                       int64_t offA, int64_t offB, double *acc_out, double *abs_out)
{
    int64_t k[ORACLE_MAX_MODES] = {0};
    double acc = 0.0, aacc = 0.0;
    for (;;) {
        int64_t oa = offA, ob = offB;
        for (int c = 0; c < L->ncon; ++c) {
            oa += k[c] * L->con_sA[c];
            ob += k[c] * L->con_sB[c];
        }
        double a = load_operand(A, oa, dtype), b = load_operand(B, ob, dtype);
        acc += a * b;
        aacc += fabs(a) * fabs(b);
        int c = 0;
        for (; c < L->ncon; ++c) { /* advance the contracted odometer */
            if (++k[c] < L->con_ext[c])
                break;
            k[c] = 0;
        }
        if (c == L->ncon)
            break; /* also the single pass taken when there is no contracted mode */
    }
    *acc_out = acc;
    *abs_out = aacc;
}

typedef struct {
    const loops_t *L;
    const void *A, *B;
    const void *C_old;
    int dtype;
    double alpha, beta;
    double *C_ref, *absacc;
    int64_t outer_lo, outer_hi; /* range of the outermost (last) free index */
} job_t;

static void *run_job(void *arg)
{
    const job_t *J = (const job_t *)arg;
    const loops_t *L = J->L;
    int nf = L->nfree;
    int64_t idx[ORACLE_MAX_MODES] = {0};
    if (nf > 0) {
        if (J->outer_lo >= J->outer_hi)
            return NULL;
        idx[nf - 1] = J->outer_lo;
    }
    for (;;) {
        int64_t oa = 0, ob = 0, oc = 0;
        for (int f = 0; f < nf; ++f) {
            oa += idx[f] * L->free_sA[f];
            ob += idx[f] * L->free_sB[f];
            oc += idx[f] * L->free_sC[f];
        }
        double acc, aacc;
        one_output(L, J->A, J->B, J->dtype, oa, ob, &acc, &aacc);
        double r = J->alpha * acc;
        if (J->beta != 0.0)
            r += J->beta * load_c_old(J->C_old, oc, J->dtype);
        J->C_ref[oc] = r;
        if (J->absacc)
            J->absacc[oc] = aacc;
        int f = 0;
        for (; f < nf; ++f) { /* advance the free odometer, first mode fastest */
            int64_t hi = (f == nf - 1) ? J->outer_hi : L->free_ext[f];
            if (++idx[f] < hi)
                break;
            idx[f] = 0;
        }
        if (f == nf)
            break;
    }
    return NULL;
}

/*
 * Full contraction.  C_ref and absacc (optional) are arrays over C's storage
 * span, written only at the offsets C's modes address.  C_old may be NULL when
 * beta == 0.  nthreads <= 1 runs in the calling thread.
 */
int gett_oracle_contract(const oracle_tensor_t *A, const oracle_tensor_t *B,
                         const oracle_tensor_t *C, int dtype, double alpha, const void *A_data,
                         const void *B_data, double beta, const void *C_old, double *C_ref,
                         double *absacc, int nthreads)
{
    loops_t L;
    int rc = build_loops(A, B, C, &L);
    if (rc)
        return rc;
    if (!A_data || !B_data || !C_ref || (beta != 0.0 && !C_old))
        return ORACLE_ERR_ARG;
    if (dtype < ORACLE_F32 || dtype > ORACLE_F64)
        return ORACLE_ERR_ARG;
    int64_t outer = L.nfree ? L.free_ext[L.nfree - 1] : 1;
    if (nthreads < 1)
        nthreads = 1;
    if (nthreads > outer)
        nthreads = (int)outer;
    if (nthreads > 256)
        nthreads = 256;
    job_t jobs[256];
    pthread_t th[256];
    for (int t = 0; t < nthreads; ++t) {
        job_t j = {&L, A_data, B_data, C_old, dtype, alpha, beta, C_ref, absacc,
                   outer * t / nthreads, outer * (t + 1) / nthreads};
        jobs[t] = j;
    }
    if (nthreads == 1) {
        run_job(&jobs[0]);
        return ORACLE_OK;
    }
    for (int t = 0; t < nthreads; ++t)
        pthread_create(&th[t], NULL, run_job, &jobs[t]);
    for (int t = 0; t < nthreads; ++t)
        pthread_join(th[t], NULL);
    return ORACLE_OK;
}

typedef struct {
    const loops_t *L;
    const void *A, *B;
    const void *C_old;
    int dtype;
    double alpha, beta;
    const int64_t *points;
    double *out, *absacc;
    int64_t lo, hi;
} pjob_t;

static void *run_points(void *arg)
{
    const pjob_t *J = (const pjob_t *)arg;
    const loops_t *L = J->L;
    for (int64_t p = J->lo; p < J->hi; ++p) {
        const int64_t *idx = J->points + p * L->nfree;
        int64_t oa = 0, ob = 0, oc = 0;
        for (int f = 0; f < L->nfree; ++f) {
            oa += idx[f] * L->free_sA[f];
            ob += idx[f] * L->free_sB[f];
            oc += idx[f] * L->free_sC[f];
        }
        double acc, aacc;
        one_output(L, J->A, J->B, J->dtype, oa, ob, &acc, &aacc);
        double r = J->alpha * acc;
        if (J->beta != 0.0)
            r += J->beta * load_c_old(J->C_old, oc, J->dtype);
        J->out[p] = r;
        if (J->absacc)
            J->absacc[p] = aacc;
    }
    return NULL;
}

/*
 * The same computation for a chosen list of outputs: points[p*d_C + i] is the
 * index of C's i-th mode for output p.  out[p] / absacc[p] receive the values.
 */
int gett_oracle_points(const oracle_tensor_t *A, const oracle_tensor_t *B,
                       const oracle_tensor_t *C, int dtype, double alpha, const void *A_data,
                       const void *B_data, double beta, const void *C_old, int64_t npoints,
                       const int64_t *points, double *out, double *absacc, int nthreads)
{
    loops_t L;
    int rc = build_loops(A, B, C, &L);
    if (rc)
        return rc;
    if (!A_data || !B_data || !out || (npoints > 0 && L.nfree > 0 && !points) ||
        (beta != 0.0 && !C_old))
        return ORACLE_ERR_ARG;
    if (dtype < ORACLE_F32 || dtype > ORACLE_F64)
        return ORACLE_ERR_ARG;
    for (int64_t p = 0; p < npoints; ++p)
        for (int f = 0; f < L.nfree; ++f)
            if (points[p * L.nfree + f] < 0 || points[p * L.nfree + f] >= L.free_ext[f])
                return ORACLE_ERR_ARG;
    if (nthreads < 1)
        nthreads = 1;
    if (nthreads > 256)
        nthreads = 256;
    if (nthreads > npoints)
        nthreads = npoints > 0 ? (int)npoints : 1;
    pjob_t jobs[256];
    pthread_t th[256];
    for (int t = 0; t < nthreads; ++t) {
        pjob_t j = {&L, A_data, B_data, C_old, dtype, alpha, beta, points, out, absacc,
                    npoints * t / nthreads, npoints * (t + 1) / nthreads};
        jobs[t] = j;
    }
    if (nthreads == 1) {
        run_points(&jobs[0]);
        return ORACLE_OK;
    }
    for (int t = 0; t < nthreads; ++t)
        pthread_create(&th[t], NULL, run_points, &jobs[t]);
    for (int t = 0; t < nthreads; ++t)
        pthread_join(th[t], NULL);
    return ORACLE_OK;
}
