/*
 * CPU oracle for the binary / unary tensor operation
 *
 *     C := alpha * op(A) + beta * op(B)
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow evaluation of the paper's definition used to check the
 * GPU library; it shares no code with it and nothing in the product path may call it.
 *
 * What it follows in the paper (Sec. "Unary and Binary Operations"): B and C carry the same
 * labels; the labels of A and C split into H (in both), I_A (only in A) and I_B (only in B / C).
 * Labels only in A are summed over and labels only in B / C repeat A along them, so for every
 * multi-index over C's labels
 *         C[.] = alpha * sum_{I_A} op(A)[.] + beta * op(B)[.]
 * with A independent of the I_B indices.  Unary scaling B := alpha A is the case beta = 0; a
 * label repeated inside A addresses (semi-)diagonal elements: it acts as one mode whose stride is
 * the sum of the strides of its occurrences (Note 6).  Multi-indices advance like an odometer
 * whose first position is fastest; an element lives at base + sum_k index_k * stride_k.
 *
 * Readings where the paper is silent (kept identical to the library's):
 *   - op(X) is the element-wise complex conjugate when the flag is set.
 *   - beta == 0: B is never read (may be NULL); alpha == 0: A is never read.
 *   - B has C's rank, extents and label order; its strides are its own (B is an input like A).
 *   - a label repeated inside C is not supported; C's elements must not alias (same sufficient
 *     rule as for D of the contraction).
 *
 * Accumulation: one accumulator per element of C, wider than the element type (long double for
 * 64-bit parts, double for 32-bit parts) unless `native_acc`.  Beside every value it returns
 *     scale = |alpha| * sum |a| + |beta| * |b|.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORE_MAX_RANK 32
#define ORE_MAX_LABELS 64

enum { ORE_F32 = 0, ORE_F64 = 1, ORE_C32 = 2, ORE_C64 = 3 };
enum {
    ORE_OK = 0,
    ORE_ERR_INVALID_ARGUMENT = 1,
    ORE_ERR_INVALID_EXTENT = 2,
    ORE_ERR_EXTENT_MISMATCH = 3,
    ORE_ERR_B_C_MISMATCH = 4,
    ORE_ERR_C_ALIASING = 5,
    ORE_ERR_NOT_SUPPORTED = 7
};

typedef struct {
    int32_t rank;
    const int64_t *extent;
    const int64_t *stride; /* in elements, signed */
    const int64_t *label;
    int32_t conj;
    void *data; /* address of logical element (0,...,0) */
} ore_tensor;

typedef struct {
    int64_t label, extent, sA, sB, sC;
} ore_mode;

typedef struct {
    int nC, nS;
    ore_mode c[ORE_MAX_LABELS]; /* C's labels in C's order */
    ore_mode s[ORE_MAX_LABELS]; /* labels only in A: summed */
    int64_t sizeC, sizeS;
} ore_loops;

static int cmp_abs(const void *x, const void *y)
{
    const int64_t *a = (const int64_t *)x, *b = (const int64_t *)y;
    int64_t sa = a[0] < 0 ? -a[0] : a[0], sb = b[0] < 0 ? -b[0] : b[0];
    return (sa > sb) - (sa < sb);
}

static int ore_prepare(const ore_tensor *A, const ore_tensor *B, const ore_tensor *C, int b_is_used, ore_loops *L)
{
    if (!A || !C) return ORE_ERR_INVALID_ARGUMENT;
    const ore_tensor *T[2] = {A, C};
    for (int t = 0; t < 2; ++t) {
        if (T[t]->rank < 0 || T[t]->rank > ORE_MAX_RANK) return ORE_ERR_INVALID_ARGUMENT;
        if (T[t]->rank > 0 && (!T[t]->extent || !T[t]->stride || !T[t]->label)) return ORE_ERR_INVALID_ARGUMENT;
        for (int i = 0; i < T[t]->rank; ++i)
            if (T[t]->extent[i] < 1) return ORE_ERR_INVALID_EXTENT;
    }
    for (int i = 0; i < C->rank; ++i)
        for (int j = 0; j < i; ++j)
            if (C->label[i] == C->label[j]) return ORE_ERR_NOT_SUPPORTED;
    if (b_is_used) {
        if (!B || B->rank != C->rank) return ORE_ERR_B_C_MISMATCH;
        for (int i = 0; i < C->rank; ++i)
            if (B->extent[i] != C->extent[i] || B->label[i] != C->label[i]) return ORE_ERR_B_C_MISMATCH;
    }
    /* C's elements are distinct */
    {
        int64_t se[ORE_MAX_RANK][2];
        int n = 0;
        for (int i = 0; i < C->rank; ++i)
            if (C->extent[i] > 1) {
                if (C->stride[i] == 0) return ORE_ERR_C_ALIASING;
                se[n][0] = C->stride[i];
                se[n][1] = C->extent[i];
                ++n;
            }
        qsort(se, (size_t)n, sizeof se[0], cmp_abs);
        int64_t span = 0;
        for (int k = 0; k < n; ++k) {
            int64_t s = se[k][0] < 0 ? -se[k][0] : se[k][0];
            if (s < 1 + span) return ORE_ERR_C_ALIASING;
            span += s * (se[k][1] - 1);
        }
    }
    L->nC = L->nS = 0;
    L->sizeC = L->sizeS = 1;
    for (int i = 0; i < C->rank; ++i) {
        ore_mode *m = &L->c[L->nC++];
        m->label = C->label[i];
        m->extent = C->extent[i];
        m->sC = C->stride[i];
        m->sB = b_is_used ? B->stride[i] : 0;
        m->sA = 0; /* stays 0 for a label of I_B: A is broadcast along it */
        L->sizeC *= m->extent;
    }
    for (int i = 0; i < A->rank; ++i) {
        int k;
        for (k = 0; k < L->nC; ++k)
            if (L->c[k].label == A->label[i]) break;
        if (k < L->nC) { /* label of H */
            if (L->c[k].extent != A->extent[i]) return ORE_ERR_EXTENT_MISMATCH;
            L->c[k].sA += A->stride[i]; /* repeated occurrences add up */
            continue;
        }
        for (k = 0; k < L->nS; ++k)
            if (L->s[k].label == A->label[i]) break;
        if (k == L->nS) { /* first occurrence of a label of I_A */
            if (L->nS == ORE_MAX_LABELS) return ORE_ERR_INVALID_ARGUMENT;
            memset(&L->s[k], 0, sizeof L->s[k]);
            L->s[k].label = A->label[i];
            L->s[k].extent = A->extent[i];
            L->sizeS *= A->extent[i];
            ++L->nS;
        } else if (L->s[k].extent != A->extent[i]) {
            return ORE_ERR_EXTENT_MISMATCH;
        }
        L->s[k].sA += A->stride[i];
    }
    return ORE_OK;
}

#define ORE_DEFINE_LOOPS(NAME, T, ACC, NCOMP, SQRT, FABS)                                        \
    static void NAME(const ore_loops *L, const ore_tensor *A, const ore_tensor *B, const ore_tensor *C, \
                     const T *alpha, const T *beta, int64_t n_want, const int64_t *want,         \
                     T *out_val, double *out_scale)                                              \
    {                                                                                            \
        const T *pa = (const T *)A->data;                                                        \
        const T *pb = B ? (const T *)B->data : NULL;                                             \
        T *pc = (T *)C->data;                                                                    \
        const ACC al_r = alpha[0], al_i = (NCOMP == 2) ? alpha[NCOMP - 1] : (ACC)0;              \
        const ACC be_r = beta[0], be_i = (NCOMP == 2) ? beta[NCOMP - 1] : (ACC)0;                \
        const int use_a = (al_r != 0 || al_i != 0);                                              \
        const int use_b = (be_r != 0 || be_i != 0);                                              \
        const ACC abs_al = SQRT(al_r * al_r + al_i * al_i);                                      \
        const ACC abs_be = SQRT(be_r * be_r + be_i * be_i);                                      \
        const ACC sgnA = A->conj ? (ACC)-1 : (ACC)1;                                             \
        const ACC sgnB = (B && B->conj) ? (ACC)-1 : (ACC)1;                                      \
        const int64_t total = want ? n_want : L->sizeC;                                          \
        _Pragma("omp parallel for schedule(static)")                                             \
        for (int64_t e = 0; e < total; ++e) {                                                    \
            int64_t lin = want ? want[e] : e;                                                    \
            int64_t offA = 0, offB = 0, offC = 0;                                                \
            for (int k = 0; k < L->nC; ++k) { /* first label of C fastest */                     \
                int64_t i = lin % L->c[k].extent;                                                \
                lin /= L->c[k].extent;                                                           \
                offA += i * L->c[k].sA;                                                          \
                offB += i * L->c[k].sB;                                                          \
                offC += i * L->c[k].sC;                                                          \
            }                                                                                    \
            ACC acc_r = 0, acc_i = 0, absacc = 0;                                                \
            if (use_a) {                                                                         \
                int64_t idx[ORE_MAX_LABELS];                                                     \
                int64_t oa = offA;                                                               \
                for (int k = 0; k < L->nS; ++k) idx[k] = 0;                                      \
                for (int64_t s = 0; s < L->sizeS; ++s) {                                         \
                    const ACC ar = pa[NCOMP * oa];                                               \
                    const ACC ai = (NCOMP == 2) ? sgnA * (ACC)pa[NCOMP * oa + (NCOMP - 1)] : 0;  \
                    acc_r += ar;                                                                 \
                    acc_i += ai;                                                                 \
                    absacc += (NCOMP == 2) ? SQRT(ar * ar + ai * ai) : FABS(ar);                 \
                    for (int k = 0; k < L->nS; ++k) { /* odometer over I_A, first fastest */     \
                        oa += L->s[k].sA;                                                        \
                        if (++idx[k] < L->s[k].extent) break;                                    \
                        oa -= idx[k] * L->s[k].sA;                                               \
                        idx[k] = 0;                                                              \
                    }                                                                            \
                }                                                                                \
            }                                                                                    \
            ACC c_r = al_r * acc_r - al_i * acc_i;                                               \
            ACC c_i = al_r * acc_i + al_i * acc_r;                                               \
            ACC sc = abs_al * absacc;                                                            \
            if (use_b) {                                                                         \
                const ACC br = pb[NCOMP * offB];                                                 \
                const ACC bi = (NCOMP == 2) ? sgnB * (ACC)pb[NCOMP * offB + (NCOMP - 1)] : 0;    \
                c_r += be_r * br - be_i * bi;                                                    \
                c_i += be_r * bi + be_i * br;                                                    \
                sc += abs_be * SQRT(br * br + bi * bi);                                          \
            }                                                                                    \
            if (want) {                                                                          \
                out_val[NCOMP * e] = (T)c_r;                                                     \
                if (NCOMP == 2) out_val[NCOMP * e + (NCOMP - 1)] = (T)c_i;                       \
            } else {                                                                             \
                pc[NCOMP * offC] = (T)c_r;                                                       \
                if (NCOMP == 2) pc[NCOMP * offC + (NCOMP - 1)] = (T)c_i;                         \
            }                                                                                    \
            if (out_scale) out_scale[e] = (double)sc;                                            \
        }                                                                                        \
    }

ORE_DEFINE_LOOPS(ew_f32_wide, float, double, 1, sqrt, fabs)
ORE_DEFINE_LOOPS(ew_f32_native, float, float, 1, sqrtf, fabsf)
ORE_DEFINE_LOOPS(ew_f64_wide, double, long double, 1, sqrtl, fabsl)
ORE_DEFINE_LOOPS(ew_f64_native, double, double, 1, sqrt, fabs)
ORE_DEFINE_LOOPS(ew_c32_wide, float, double, 2, sqrt, fabs)
ORE_DEFINE_LOOPS(ew_c32_native, float, float, 2, sqrtf, fabsf)
ORE_DEFINE_LOOPS(ew_c64_wide, double, long double, 2, sqrtl, fabsl)
ORE_DEFINE_LOOPS(ew_c64_native, double, double, 2, sqrt, fabs)

/*
 * Entry point; arguments as for the contraction oracle: `want` NULL evaluates all of C in place
 * through C's strides, otherwise only the listed column-major linear indices over C's labels
 * (values to out_val, C untouched); out_scale is NULL or one double per evaluated element.
 * When B shares C's memory (in place) every element is read before it is written.
 */
int ore_elementwise(int dtype, const ore_tensor *A, const ore_tensor *B, const ore_tensor *C,
                    const void *alpha, const void *beta, int native_acc, int64_t n_want,
                    const int64_t *want, void *out_val, double *out_scale)
{
    ore_loops L;
    int b_is_used;
    if (!alpha || !beta || !C) return ORE_ERR_INVALID_ARGUMENT;
    if (want && !out_val) return ORE_ERR_INVALID_ARGUMENT;
    switch (dtype) {
    case ORE_F32: b_is_used = ((const float *)beta)[0] != 0; break;
    case ORE_F64: b_is_used = ((const double *)beta)[0] != 0; break;
    case ORE_C32: b_is_used = ((const float *)beta)[0] != 0 || ((const float *)beta)[1] != 0; break;
    case ORE_C64: b_is_used = ((const double *)beta)[0] != 0 || ((const double *)beta)[1] != 0; break;
    default: return ORE_ERR_NOT_SUPPORTED;
    }
    int rc = ore_prepare(A, B, C, b_is_used, &L);
    if (rc != ORE_OK) return rc;
    if (want)
        for (int64_t e = 0; e < n_want; ++e)
            if (want[e] < 0 || want[e] >= L.sizeC) return ORE_ERR_INVALID_ARGUMENT;
    if (!b_is_used) B = NULL;
#define ORE_CALL(F, T) F(&L, A, B, C, (const T *)alpha, (const T *)beta, n_want, want, (T *)out_val, out_scale)
    switch (dtype) {
    case ORE_F32: if (native_acc) ORE_CALL(ew_f32_native, float); else ORE_CALL(ew_f32_wide, float); break;
    case ORE_F64: if (native_acc) ORE_CALL(ew_f64_native, double); else ORE_CALL(ew_f64_wide, double); break;
    case ORE_C32: if (native_acc) ORE_CALL(ew_c32_native, float); else ORE_CALL(ew_c32_wide, float); break;
    case ORE_C64: if (native_acc) ORE_CALL(ew_c64_native, double); else ORE_CALL(ew_c64_wide, double); break;
    }
#undef ORE_CALL
    return ORE_OK;
}
