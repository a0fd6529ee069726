/*
 * CPU oracle for the general binary tensor contraction
 *
 *     D := alpha * op(A) * op(B) + beta * op(C)
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow evaluation of the
 * paper's definition used to check the GPU library; it shares no code with it
 * and nothing in the product path may call it.
 *
 * What it follows in the paper
 *   - Sec. "Operations", Eq. (case2) with Case 3 (repeated labels) and the
 *     Case 4 extension (isolated labels of A / B are summed): for every
 *     multi-index over D's labels
 *         D[.] = alpha * sum_{labels not in D} op(A)[.] * op(B)[.] + beta * op(C)[.]
 *     (sum_IA A)(sum_IB B) equals one sum over P u IA u IB of the product
 *     because an IA label does not index B and vice versa.
 *   - Note 6: a label that occurs several times in one tensor acts as one mode
 *     whose stride is the sum of the strides of its occurrences.
 *   - Sec. "Algorithm Structure": labels absent from a tensor get stride 0;
 *     multi-indices advance like an odometer whose FIRST position is fastest;
 *     an element lives at base + sum_k index_k * stride_k (Glossary, "Strided
 *     layout"); error checks come first (equal extents per label, C matches D,
 *     no aliasing inside D; Appendix "Testing" items 26-28).
 *   - Eq. (FreeD): a label that occurs only in D is rejected (Case 5).
 *
 * Readings where the paper is silent (kept identical to the library's):
 *   - op(X) is the element-wise complex conjugate when the flag is set.
 *   - beta == 0: C is never read (may be NULL); alpha == 0: A and B are never read.
 *   - alpha multiplies the finished sum once.
 *   - C must have D's rank, extents, strides and label order.
 *   - a label repeated inside D is not supported.
 *   - "aliasing inside D": sufficient test on D's modes of extent > 1 sorted by
 *     |stride|: |s_k| >= 1 + sum_{l<k} |s_l| (e_l - 1), zero stride is an error.
 *
 * Accumulation: one accumulator per D element, wider than the element type
 * (long double for 64-bit parts, double for 32-bit parts) unless `native_acc`
 * asks for the element's own precision (that build of the same loops is the
 * timed CPU baseline).  Beside every value it returns
 *     scale = |alpha| * sum |a||b| + |beta| * |c|
 * which the parity tests use to normalise the error.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_RANK 32
#define ORC_MAX_LABELS 96

enum { ORC_F32 = 0, ORC_F64 = 1, ORC_C32 = 2, ORC_C64 = 3 };

enum {
    ORC_OK = 0,
    ORC_ERR_INVALID_ARGUMENT = 1,
    ORC_ERR_INVALID_EXTENT = 2,
    ORC_ERR_EXTENT_MISMATCH = 3,
    ORC_ERR_C_D_MISMATCH = 4,
    ORC_ERR_D_ALIASING = 5,
    ORC_ERR_LABEL_ONLY_IN_D = 6,
    ORC_ERR_NOT_SUPPORTED = 7
};

typedef struct {
    int32_t rank;
    const int64_t *extent; /* rank entries */
    const int64_t *stride; /* rank entries, in elements, signed */
    const int64_t *label;  /* rank entries */
    int32_t conj;
    void *data; /* address of logical element (0,...,0) */
} orc_tensor;

/* One row per unique label: extent and the (summed) stride in each tensor. */
typedef struct {
    int64_t label, extent;
    int64_t sA, sB, sD;
    int inA, inB, inD;
} orc_mode;

typedef struct {
    int nD, nS; /* number of D labels, number of summed labels */
    orc_mode d[ORC_MAX_LABELS];
    orc_mode s[ORC_MAX_LABELS];
    int64_t sizeD, sizeS;
} orc_loops;

static int find_label(const orc_mode *t, int n, int64_t label)
{
    for (int i = 0; i < n; ++i)
        if (t[i].label == label) return i;
    return -1;
}

static int cmp_abs_stride(const void *x, const void *y)
{
    const int64_t *a = (const int64_t *)x, *b = (const int64_t *)y;
    int64_t sa = a[0] < 0 ? -a[0] : a[0], sb = b[0] < 0 ? -b[0] : b[0];
    return (sa > sb) - (sa < sb);
}

/* Error checks and label bookkeeping (Sec. "Algorithm Structure", first two paragraphs). */
static int orc_prepare(const orc_tensor *A, const orc_tensor *B, const orc_tensor *C,
                       const orc_tensor *D, int c_is_used, orc_loops *L)
{
    const orc_tensor *T[3] = {A, B, D};
    orc_mode all[ORC_MAX_LABELS];
    int n_all = 0;

    if (!A || !B || !D) return ORC_ERR_INVALID_ARGUMENT;
    for (int t = 0; t < 3; ++t) {
        if (T[t]->rank < 0 || T[t]->rank > ORC_MAX_RANK) return ORC_ERR_INVALID_ARGUMENT;
        if (T[t]->rank > 0 && (!T[t]->extent || !T[t]->stride || !T[t]->label))
            return ORC_ERR_INVALID_ARGUMENT;
        for (int i = 0; i < T[t]->rank; ++i)
            if (T[t]->extent[i] < 1) return ORC_ERR_INVALID_EXTENT;
    }
    /* a label repeated inside D would write only a diagonal of D */
    for (int i = 0; i < D->rank; ++i)
        for (int j = 0; j < i; ++j)
            if (D->label[i] == D->label[j]) return ORC_ERR_NOT_SUPPORTED;

    /* one row per unique label; strides of repeated labels add up (Note 6) */
    for (int t = 0; t < 3; ++t) {
        for (int i = 0; i < T[t]->rank; ++i) {
            int k = find_label(all, n_all, T[t]->label[i]);
            if (k < 0) {
                if (n_all == ORC_MAX_LABELS) return ORC_ERR_INVALID_ARGUMENT;
                k = n_all++;
                memset(&all[k], 0, sizeof all[k]);
                all[k].label = T[t]->label[i];
                all[k].extent = T[t]->extent[i];
            } else if (all[k].extent != T[t]->extent[i]) {
                return ORC_ERR_EXTENT_MISMATCH;
            }
            if (t == 0) { all[k].sA += T[t]->stride[i]; all[k].inA = 1; }
            if (t == 1) { all[k].sB += T[t]->stride[i]; all[k].inB = 1; }
            if (t == 2) { all[k].sD += T[t]->stride[i]; all[k].inD = 1; }
        }
    }
    /* Eq. (FreeD): every label of D occurs in A or in B */
    for (int k = 0; k < n_all; ++k)
        if (all[k].inD && !all[k].inA && !all[k].inB) return ORC_ERR_LABEL_ONLY_IN_D;

    /* C has D's structure (Note 5 and the reading stated above) */
    if (c_is_used) {
        if (!C) return ORC_ERR_INVALID_ARGUMENT;
        if (C->rank != D->rank) return ORC_ERR_C_D_MISMATCH;
        for (int i = 0; i < D->rank; ++i)
            if (C->extent[i] != D->extent[i] || C->stride[i] != D->stride[i] ||
                C->label[i] != D->label[i])
                return ORC_ERR_C_D_MISMATCH;
    }

    /* no two multi-indices of D may address the same element */
    {
        int64_t se[ORC_MAX_RANK][2];
        int n = 0;
        for (int i = 0; i < D->rank; ++i)
            if (D->extent[i] > 1) {
                if (D->stride[i] == 0) return ORC_ERR_D_ALIASING;
                se[n][0] = D->stride[i];
                se[n][1] = D->extent[i];
                ++n;
            }
        qsort(se, (size_t)n, sizeof se[0], cmp_abs_stride);
        int64_t span = 0; /* sum_{l<k} |s_l| (e_l - 1) */
        for (int k = 0; k < n; ++k) {
            int64_t s = se[k][0] < 0 ? -se[k][0] : se[k][0];
            if (s < 1 + span) return ORC_ERR_D_ALIASING;
            span += s * (se[k][1] - 1);
        }
    }

    /* D's labels in D's own order; every other label is summed */
    L->nD = L->nS = 0;
    L->sizeD = L->sizeS = 1;
    for (int i = 0; i < D->rank; ++i) {
        L->d[L->nD] = all[find_label(all, n_all, D->label[i])];
        L->sizeD *= L->d[L->nD].extent;
        ++L->nD;
    }
    for (int k = 0; k < n_all; ++k)
        if (!all[k].inD) {
            L->s[L->nS] = all[k];
            L->sizeS *= all[k].extent;
            ++L->nS;
        }
    return ORC_OK;
}

/*
 * The loop nest, once per (element type, accumulator type, real/complex).
 * `want` is NULL (all of D, written through D's strides) or a list of
 * column-major linear indices over D's labels (values go to out_val, D untouched).
 */
#define ORC_DEFINE_LOOPS(NAME, T, ACC, NCOMP, SQRT, FABS)                                        \
    static void NAME(const orc_loops *L, const orc_tensor *A, const orc_tensor *B,               \
                     const orc_tensor *C, const orc_tensor *D, const T *alpha, const T *beta,    \
                     int64_t n_want, const int64_t *want, T *out_val, double *out_scale)         \
    {                                                                                            \
        const T *pa = (const T *)A->data, *pb = (const T *)B->data;                              \
        const T *pc = C ? (const T *)C->data : NULL;                                             \
        T *pd = (T *)D->data;                                                                    \
        const ACC al_r = alpha[0], al_i = (NCOMP == 2) ? alpha[NCOMP - 1] : (ACC)0;              \
        const ACC be_r = beta[0], be_i = (NCOMP == 2) ? beta[NCOMP - 1] : (ACC)0;                \
        const int use_ab = (al_r != 0 || al_i != 0);                                             \
        const int use_c = (be_r != 0 || be_i != 0);                                              \
        const ACC abs_al = SQRT(al_r * al_r + al_i * al_i);                                      \
        const ACC abs_be = SQRT(be_r * be_r + be_i * be_i);                                      \
        const ACC sgnA = A->conj ? (ACC)-1 : (ACC)1, sgnB = B->conj ? (ACC)-1 : (ACC)1;          \
        const ACC sgnC = (C && C->conj) ? (ACC)-1 : (ACC)1;                                      \
        const int64_t total = want ? n_want : L->sizeD;                                          \
        _Pragma("omp parallel for schedule(static)")                                             \
        for (int64_t e = 0; e < total; ++e) {                                                    \
            int64_t lin = want ? want[e] : e;                                                    \
            int64_t offA = 0, offB = 0, offD = 0;                                                \
            for (int k = 0; k < L->nD; ++k) { /* first label of D fastest */                     \
                int64_t i = lin % L->d[k].extent;                                                \
                lin /= L->d[k].extent;                                                           \
                offA += i * L->d[k].sA;                                                          \
                offB += i * L->d[k].sB;                                                          \
                offD += i * L->d[k].sD;                                                          \
            }                                                                                    \
            ACC acc_r = 0, acc_i = 0, absacc = 0;                                                \
            if (use_ab) {                                                                        \
                int64_t idx[ORC_MAX_LABELS];                                                     \
                int64_t oa = offA, ob = offB;                                                    \
                for (int k = 0; k < L->nS; ++k) idx[k] = 0;                                      \
                for (int64_t s = 0; s < L->sizeS; ++s) {                                         \
                    const ACC ar = pa[NCOMP * oa];                                               \
                    const ACC br = pb[NCOMP * ob];                                               \
                    if (NCOMP == 2) {                                                            \
                        const ACC ai = sgnA * (ACC)pa[NCOMP * oa + (NCOMP - 1)];                 \
                        const ACC bi = sgnB * (ACC)pb[NCOMP * ob + (NCOMP - 1)];                 \
                        acc_r += ar * br - ai * bi;                                              \
                        acc_i += ar * bi + ai * br;                                              \
                        absacc += SQRT(ar * ar + ai * ai) * SQRT(br * br + bi * bi);             \
                    } else {                                                                     \
                        acc_r += ar * br;                                                        \
                        absacc += FABS(ar) * FABS(br);                                           \
                    }                                                                            \
                    /* odometer over the summed labels, first fastest */                         \
                    for (int k = 0; k < L->nS; ++k) {                                            \
                        oa += L->s[k].sA;                                                        \
                        ob += L->s[k].sB;                                                        \
                        if (++idx[k] < L->s[k].extent) break;                                    \
                        oa -= idx[k] * L->s[k].sA;                                               \
                        ob -= idx[k] * L->s[k].sB;                                               \
                        idx[k] = 0;                                                              \
                    }                                                                            \
                }                                                                                \
            }                                                                                    \
            ACC d_r = al_r * acc_r - al_i * acc_i;                                               \
            ACC d_i = al_r * acc_i + al_i * acc_r;                                               \
            ACC sc = abs_al * absacc;                                                            \
            if (use_c) {                                                                         \
                const ACC cr = pc[NCOMP * offD];                                                 \
                const ACC ci = (NCOMP == 2) ? sgnC * (ACC)pc[NCOMP * offD + (NCOMP - 1)] : 0;    \
                d_r += be_r * cr - be_i * ci;                                                    \
                d_i += be_r * ci + be_i * cr;                                                    \
                sc += abs_be * SQRT(cr * cr + ci * ci);                                          \
            }                                                                                    \
            if (want) {                                                                          \
                out_val[NCOMP * e] = (T)d_r;                                                     \
                if (NCOMP == 2) out_val[NCOMP * e + (NCOMP - 1)] = (T)d_i;                       \
            } else {                                                                             \
                pd[NCOMP * offD] = (T)d_r;                                                       \
                if (NCOMP == 2) pd[NCOMP * offD + (NCOMP - 1)] = (T)d_i;                         \
            }                                                                                    \
            if (out_scale) out_scale[e] = (double)sc;                                            \
        }                                                                                        \
    }

ORC_DEFINE_LOOPS(loops_f32_wide, float, double, 1, sqrt, fabs)
ORC_DEFINE_LOOPS(loops_f32_native, float, float, 1, sqrtf, fabsf)
ORC_DEFINE_LOOPS(loops_f64_wide, double, long double, 1, sqrtl, fabsl)
ORC_DEFINE_LOOPS(loops_f64_native, double, double, 1, sqrt, fabs)
ORC_DEFINE_LOOPS(loops_c32_wide, float, double, 2, sqrt, fabs)
ORC_DEFINE_LOOPS(loops_c32_native, float, float, 2, sqrtf, fabsf)
ORC_DEFINE_LOOPS(loops_c64_wide, double, long double, 2, sqrtl, fabsl)
ORC_DEFINE_LOOPS(loops_c64_native, double, double, 2, sqrt, fabs)

/*
 * Entry point.
 *   dtype        one of ORC_F32, ORC_F64, ORC_C32 (2 x float), ORC_C64 (2 x double)
 *   A, B, D      operands; C may be NULL when beta == 0
 *   alpha, beta  host scalars of the element type (2 parts when complex)
 *   native_acc   0: wide accumulator (verification), 1: element precision (timed baseline)
 *   n_want/want  NULL: evaluate all of D in place through D's strides; otherwise
 *                evaluate only these column-major linear indices over D's labels
 *                and store them in out_val (D's memory is not touched)
 *   out_scale    NULL, or one double per evaluated element (same order as the
 *                evaluation: column-major over D's labels, or the order of `want`)
 * Returns ORC_OK or an error code; nothing is written on error.
 */
int orc_contract(int dtype, const orc_tensor *A, const orc_tensor *B, const orc_tensor *C,
                 const orc_tensor *D, const void *alpha, const void *beta, int native_acc,
                 int64_t n_want, const int64_t *want, void *out_val, double *out_scale)
{
    orc_loops L;
    int c_is_used;
    if (!alpha || !beta || !D) return ORC_ERR_INVALID_ARGUMENT;
    if (want && !out_val) return ORC_ERR_INVALID_ARGUMENT;
    switch (dtype) {
    case ORC_F32: c_is_used = ((const float *)beta)[0] != 0; break;
    case ORC_F64: c_is_used = ((const double *)beta)[0] != 0; break;
    case ORC_C32: c_is_used = ((const float *)beta)[0] != 0 || ((const float *)beta)[1] != 0; break;
    case ORC_C64: c_is_used = ((const double *)beta)[0] != 0 || ((const double *)beta)[1] != 0; break;
    default: return ORC_ERR_NOT_SUPPORTED;
    }
    int rc = orc_prepare(A, B, C, D, c_is_used, &L);
    if (rc != ORC_OK) return rc;
    if (want)
        for (int64_t e = 0; e < n_want; ++e)
            if (want[e] < 0 || want[e] >= L.sizeD) return ORC_ERR_INVALID_ARGUMENT;
    if (!c_is_used) C = NULL;

#define ORC_CALL(F, T) F(&L, A, B, C, D, (const T *)alpha, (const T *)beta, n_want, want, (T *)out_val, out_scale)
    switch (dtype) {
    case ORC_F32: if (native_acc) ORC_CALL(loops_f32_native, float); else ORC_CALL(loops_f32_wide, float); break;
    case ORC_F64: if (native_acc) ORC_CALL(loops_f64_native, double); else ORC_CALL(loops_f64_wide, double); break;
    case ORC_C32: if (native_acc) ORC_CALL(loops_c32_native, float); else ORC_CALL(loops_c32_wide, float); break;
    case ORC_C64: if (native_acc) ORC_CALL(loops_c64_native, double); else ORC_CALL(loops_c64_wide, double); break;
    }
#undef ORC_CALL
    return ORC_OK;
}

/*
 * Mixed element types (Sec. "Challenge: Datatypes": the reference implementation lets every tensor
 * have its own type).  Same definition, same loop order; every operand is read through its own type
 * (a real element is the complex number with zero imaginary part), products and sums are formed in
 * long double, and the result is rounded once to D's type.  D must be complex when any of A, B, C is;
 * alpha and beta are given as two doubles each (re, im; the imaginary part must be 0 when D is real).
 * Written as one plain function with a reader per element instead of one loop nest per type
 * combination: slower, easier to check.
 */
static void orc_read(int dtype, const void *base, int64_t off, long double *re, long double *im)
{
    switch (dtype) {
    case ORC_F32: *re = ((const float *)base)[off]; *im = 0; break;
    case ORC_F64: *re = ((const double *)base)[off]; *im = 0; break;
    case ORC_C32: *re = ((const float *)base)[2 * off]; *im = ((const float *)base)[2 * off + 1]; break;
    default: *re = ((const double *)base)[2 * off]; *im = ((const double *)base)[2 * off + 1]; break;
    }
}

static void orc_write(int dtype, void *base, int64_t off, long double re, long double im)
{
    switch (dtype) {
    case ORC_F32: ((float *)base)[off] = (float)re; break;
    case ORC_F64: ((double *)base)[off] = (double)re; break;
    case ORC_C32: ((float *)base)[2 * off] = (float)re; ((float *)base)[2 * off + 1] = (float)im; break;
    default: ((double *)base)[2 * off] = (double)re; ((double *)base)[2 * off + 1] = (double)im; break;
    }
}

static int orc_is_complex(int dtype) { return dtype == ORC_C32 || dtype == ORC_C64; }

int orc_contract_mixed(int dtypeA, int dtypeB, int dtypeC, int dtypeD, const orc_tensor *A, const orc_tensor *B,
                       const orc_tensor *C, const orc_tensor *D, const double *alpha, const double *beta,
                       int64_t n_want, const int64_t *want, void *out_val, double *out_scale)
{
    orc_loops L;
    if (!alpha || !beta || !D) return ORC_ERR_INVALID_ARGUMENT;
    if (want && !out_val) return ORC_ERR_INVALID_ARGUMENT;
    const int types[4] = {dtypeA, dtypeB, dtypeC, dtypeD};
    for (int i = 0; i < 4; ++i)
        if (types[i] < ORC_F32 || types[i] > ORC_C64) return ORC_ERR_NOT_SUPPORTED;
    const int c_is_used = beta[0] != 0 || beta[1] != 0;
    if (!orc_is_complex(dtypeD)) {
        if (orc_is_complex(dtypeA) || orc_is_complex(dtypeB) || (c_is_used && orc_is_complex(dtypeC))) return ORC_ERR_NOT_SUPPORTED;
        if (alpha[1] != 0 || beta[1] != 0) return ORC_ERR_NOT_SUPPORTED;
    }
    int rc = orc_prepare(A, B, C, D, c_is_used, &L);
    if (rc != ORC_OK) return rc;
    if (want)
        for (int64_t e = 0; e < n_want; ++e)
            if (want[e] < 0 || want[e] >= L.sizeD) return ORC_ERR_INVALID_ARGUMENT;
    if (!c_is_used) C = NULL;
    const long double al_r = alpha[0], al_i = alpha[1], be_r = beta[0], be_i = beta[1];
    const int use_ab = (al_r != 0 || al_i != 0);
    const long double abs_al = sqrtl(al_r * al_r + al_i * al_i), abs_be = sqrtl(be_r * be_r + be_i * be_i);
    const long double sgnA = A->conj ? -1 : 1, sgnB = B->conj ? -1 : 1, sgnC = (C && C->conj) ? -1 : 1;
    const int64_t total = want ? n_want : L.sizeD;
    const int out_type = dtypeD;
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < total; ++e) {
        int64_t lin = want ? want[e] : e;
        int64_t offA = 0, offB = 0, offD = 0;
        for (int k = 0; k < L.nD; ++k) { /* first label of D fastest */
            int64_t i = lin % L.d[k].extent;
            lin /= L.d[k].extent;
            offA += i * L.d[k].sA;
            offB += i * L.d[k].sB;
            offD += i * L.d[k].sD;
        }
        long double acc_r = 0, acc_i = 0, absacc = 0;
        if (use_ab) {
            int64_t idx[ORC_MAX_LABELS];
            int64_t oa = offA, ob = offB;
            for (int k = 0; k < L.nS; ++k) idx[k] = 0;
            for (int64_t s = 0; s < L.sizeS; ++s) {
                long double ar, ai, br, bi;
                orc_read(dtypeA, A->data, oa, &ar, &ai);
                orc_read(dtypeB, B->data, ob, &br, &bi);
                ai *= sgnA;
                bi *= sgnB;
                acc_r += ar * br - ai * bi;
                acc_i += ar * bi + ai * br;
                absacc += sqrtl(ar * ar + ai * ai) * sqrtl(br * br + bi * bi);
                for (int k = 0; k < L.nS; ++k) { /* odometer over the summed labels, first fastest */
                    oa += L.s[k].sA;
                    ob += L.s[k].sB;
                    if (++idx[k] < L.s[k].extent) break;
                    oa -= idx[k] * L.s[k].sA;
                    ob -= idx[k] * L.s[k].sB;
                    idx[k] = 0;
                }
            }
        }
        long double d_r = al_r * acc_r - al_i * acc_i;
        long double d_i = al_r * acc_i + al_i * acc_r;
        long double sc = abs_al * absacc;
        if (C) {
            long double cr, ci;
            orc_read(dtypeC, C->data, offD, &cr, &ci);
            ci *= sgnC;
            d_r += be_r * cr - be_i * ci;
            d_i += be_r * ci + be_i * cr;
            sc += abs_be * sqrtl(cr * cr + ci * ci);
        }
        if (want) orc_write(out_type, out_val, e, d_r, d_i);
        else orc_write(out_type, D->data, offD, d_r, d_i);
        if (out_scale) out_scale[e] = (double)sc;
    }
    return ORC_OK;
}

/* Width of the wide accumulator's significand, so a test can see what "wide" meant here. */
int orc_long_double_mant_dig(void) { return __LDBL_MANT_DIG__; }

/* Threads the parallel loop uses (reported beside the timed baseline). */
#ifdef _OPENMP
#include <omp.h>
int orc_num_threads(void) { return omp_get_max_threads(); }
#else
int orc_num_threads(void) { return 1; }
#endif
