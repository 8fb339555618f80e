/*
 * CPU ORACLE -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT PATH.
 *
 * A plain, slow, step-by-step restatement of the fault-injected mixed-precision
 * GEMM and of the exponent-only checks, written from the paper's text:
 *
 *   - operand formats FP16 (1/5/10), BF16 (1/8/7), TF32 (1/8/10 in a 32-bit
 *     word), multiplied in low precision and accumulated in FP32
 *     (Section II-A, Section II-B "D = A x B + C", Section IV-C);
 *   - the fault: bit flips XORed into one multiplication result and carried
 *     into the running sum by the "write-back" of Eq. 1-2 (Section III-E),
 *     plus the operand / accumulator / output-element sites of the problem
 *     statement (same XOR, other places);
 *   - BoundCheck, RangeCheck-max and RangeCheck-flip (Section VI-A, Table III,
 *     and their bit-level forms in Section VI-C).
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file. It shares no code, header, table or constant with the CUDA path.
 *
 * Arithmetic: every element is accumulated as
 *     acc = +0 (or the addend c_ij);  for k = 0..K-1:  acc = fl32(acc + fl32(a_ik * b_kj))
 * in IEEE binary32, round-to-nearest-even, no fused multiply-add (build with
 * -ffp-contract=off). There is no blocking of the k loop and no reordering of
 * the additions of one element; the only loop interchange is across
 * independent output elements.
 *
 * Pins (tests/test_oracle_*.py): Table III values, the FP16 subnormal example
 * of Section V-B, exhaustive exponent sweeps of the three checks against
 * their Section VI-C bit-level forms, closed forms for bit flips, exact integer
 * GEMMs, linearity of operand faults, Eq. 1-2 exactness, brute-force flag
 * bitmaps; the addend form against a GEMM cut in two along k, exact integers
 * and a per-element Python loop; the write-back form of operand trials against
 * the recompute on exact integers and within two roundings elsewhere; the
 * 16-bit output rounding against library conversions, all ties and both
 * range ends. No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_FP16 = 0, ORC_BF16 = 1, ORC_TF32 = 2 };
enum { ORC_A = 0, ORC_B = 1, ORC_ACC = 2, ORC_OUT = 3, ORC_TERM = 4 };
enum { ORC_T_NONE = 0, ORC_T_BOUND = 1, ORC_T_RMAX = 2, ORC_T_RFLIP = 3 };
#define ORC_CORRECT 16

typedef struct {
    uint32_t kind, row, col, k, xor_mask, trial, pad0, pad1;
} orc_site;

typedef struct {
    uint32_t before_bits, after_bits, final_bits, status; /* status: 1 applied, 2 skipped (invalid) */
} orc_site_log;

typedef struct {
    uint32_t status;         /* bit0 changed, bit1 detected, bit2 corrected, bit8 invalid site */
    uint32_t kind;
    uint32_t primary_index;  /* OUT/ACC/TERM: i*N+j; A: i*K+k; B: j*K+k */
    uint32_t before_bits;
    uint32_t after_bits;
    uint32_t final_bits;
    uint32_t n_affected;
    uint32_t n_detected;
    uint64_t idx_hash;
    uint32_t first_detected;
    float max_abs_dev;
} orc_trial_record;

/* ------------------------------------------------------------------ bit views */

static inline uint32_t f2u(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static inline float u2f(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

uint32_t orc_f32_bits(float f) { return f2u(f); }
float orc_bits_f32(uint32_t u) { return u2f(u); }

/* Section II-A: widen a storage word to the FP32 word of the same value. */
uint32_t orc_widen_bits(int dtype, uint32_t s)
{
    if (dtype == ORC_BF16) return (s & 0xFFFFu) << 16;      /* same exponent width as FP32 */
    if (dtype == ORC_TF32) return s & 0xFFFFE000u;          /* 19 significant bits, low 13 ignored */
    /* FP16: 1 sign, 5 exponent (bias 15), 10 mantissa */
    uint32_t sign = (s & 0x8000u) << 16;
    uint32_t e = (s >> 10) & 0x1Fu;
    uint32_t m = s & 0x3FFu;
    if (e == 0x1Fu) return sign | 0x7F800000u | (m << 13);  /* Inf / NaN */
    if (e == 0) {
        /* zero or subnormal: m * 2^-24 (scale 2^-14 with a 10-bit fraction) */
        float v = ldexpf((float)m, -24);
        return sign | f2u(v);
    }
    return sign | ((e + 112u) << 23) | (m << 13);           /* rebias 15 -> 127 */
}

float orc_widen(int dtype, uint32_t s) { return u2f(orc_widen_bits(dtype, s)); }

/* XOR a fault mask into an operand's storage word. Mask bit b addresses storage
 * bit b of a 16-bit format; for TF32 bit b (0..18) addresses FP32 bit b+13. */
uint32_t orc_flip_operand(int dtype, uint32_t s, uint32_t mask)
{
    if (dtype == ORC_TF32) return (s & 0xFFFFE000u) ^ ((mask & 0x7FFFFu) << 13);
    return (s & 0xFFFFu) ^ (mask & 0xFFFFu);
}

/* ------------------------------------------------------------------ checks */

/* BoundCheck (Section VI-A): exponent MSB set together with any of the next
 * three exponent bits ("1eeexxxx" with some e = 1). */
int orc_boundcheck_detect(uint32_t bits)
{
    uint32_t E = (bits >> 23) & 0xFFu;
    return ((E & 0x80u) != 0) && ((E & 0x70u) != 0);
}

/* correction: clear the three e bits, keep sign, the x bits and the mantissa */
uint32_t orc_boundcheck_correct(uint32_t bits)
{
    if (!orc_boundcheck_detect(bits)) return bits;
    return bits & ~(0x70u << 23);
}

/* RangeCheck (Section VI-A): exponent of a product is at most e1 + e2 + 1.
 * With biased fields E = e + 127 this is E_m <= E1 + E2 - 126. */
int orc_rangecheck_bound(uint32_t a_bits, uint32_t b_bits)
{
    int E1 = (int)((a_bits >> 23) & 0xFFu);
    int E2 = (int)((b_bits >> 23) & 0xFFu);
    int bound = E1 + E2 - 126;
    if (bound < 0) bound = 0;
    if (bound > 255) bound = 255;
    return bound;
}

int orc_rangecheck_detect(uint32_t p_bits, int bound)
{
    return (int)((p_bits >> 23) & 0xFFu) > bound;
}

/* RangeCheck-max: replace the faulty exponent by the bound */
uint32_t orc_rangecheck_max(uint32_t p_bits, int bound)
{
    if (!orc_rangecheck_detect(p_bits, bound)) return p_bits;
    return (p_bits & 0x807FFFFFu) | ((uint32_t)bound << 23);
}

/* RangeCheck-flip: clear the 1s of the faulty exponent one at a time starting
 * from its rightmost bit, stop as soon as it is <= bound */
uint32_t orc_rangecheck_flip(uint32_t p_bits, int bound)
{
    if (!orc_rangecheck_detect(p_bits, bound)) return p_bits;
    uint32_t E = (p_bits >> 23) & 0xFFu;
    for (int b = 0; b < 8 && (int)E > bound; ++b)
        if (E & (1u << b)) E &= ~(1u << b);
    return (p_bits & 0x807FFFFFu) | (E << 23);
}

/* the check applied to a faulty product (TERM sites); *det reports detection */
static uint32_t product_check(int detect_mode, uint32_t p_err, uint32_t a_bits, uint32_t b_bits, int *det)
{
    int tech = detect_mode & 3;
    int corr = (detect_mode & ORC_CORRECT) != 0;
    *det = 0;
    if (tech == ORC_T_BOUND) {
        *det = orc_boundcheck_detect(p_err);
        return (corr && *det) ? orc_boundcheck_correct(p_err) : p_err;
    }
    if (tech == ORC_T_RMAX || tech == ORC_T_RFLIP) {
        int bound = orc_rangecheck_bound(a_bits, b_bits);
        *det = orc_rangecheck_detect(p_err, bound);
        if (corr && *det)
            return tech == ORC_T_RMAX ? orc_rangecheck_max(p_err, bound) : orc_rangecheck_flip(p_err, bound);
    }
    return p_err;
}

/* ------------------------------------------------------------------ one output element */

uint32_t orc_round_output(int out_fmt, uint32_t bits);      /* defined with the 16-bit output further down */

/*
 * An FP32 word rounded to the operand format `dtype`, to nearest with ties to even, as that format's storage word
 * (16 bits for FP16 and BF16; for TF32 the FP32 word with its low 13 bits zero). Used by the alternative reading of
 * the paper's fault in which the product lives in the operand format when its bits are flipped.
 */
uint32_t orc_round_to_operand(int dtype, uint32_t bits)
{
    if (dtype == ORC_FP16) return orc_round_output(0, bits);
    if (dtype == ORC_BF16) return orc_round_output(1, bits);
    uint32_t E = (bits >> 23) & 0xFFu;
    if (E == 0xFFu) return (bits & 0xFFFFE000u) | ((bits & 0x7FFFFFu) ? 0x00400000u : 0u);   /* Inf stays, NaN stays NaN */
    uint32_t keep = bits >> 13, rest = bits & 0x1FFFu;
    if (rest > 0x1000u || (rest == 0x1000u && (keep & 1u))) keep += 1u;     /* may carry into the exponent, up to Inf */
    return keep << 13;
}

#define ORC_TERM_IN_FORMAT 128

static inline uint32_t term_boundary(uint32_t k, int kstep, int K)
{
    uint32_t kb = (k / (uint32_t)kstep + 1u) * (uint32_t)kstep;
    return kb > (uint32_t)K ? (uint32_t)K : kb;
}

/*
 * The definition: one dot product in sequential k order with the ACC and TERM
 * sites of this element applied at their boundaries, in table order.
 * a[K], b[K]: widened operands (operand faults already applied).
 * idx[n_idx]: indices into sites[] of this element's ACC/TERM sites, ascending.
 * acc0: what the running sum starts from (+0, or the addend c_ij of D = A x B + C, Section II-B).
 */
static float element_with_sites(int dtype, const float *a, const float *b, int K, int kstep, int detect_mode,
                                const orc_site *sites, const int *idx, int n_idx, orc_site_log *log, float acc0)
{
    float acc = acc0;
    for (int k = 0; k < K; ++k) {
        float p = a[k] * b[k];
        acc = acc + p;
        uint32_t done = (uint32_t)k + 1u;       /* k elements accumulated so far */
        for (int t = 0; t < n_idx; ++t) {
            const orc_site *s = &sites[idx[t]];
            if (s->kind == ORC_ACC && s->k == done) {
                uint32_t before = f2u(acc);
                uint32_t after = before ^ s->xor_mask;
                acc = u2f(after);
                if (log) { log[idx[t]].before_bits = before; log[idx[t]].after_bits = after;
                           log[idx[t]].final_bits = after; log[idx[t]].status = 1; }
            } else if (s->kind == ORC_TERM && term_boundary(s->k, kstep, K) == done) {
                /* Eq. 1-2: remove the clean product, add the faulty one */
                float re2 = a[s->k] * b[s->k];
                uint32_t before = f2u(re2);
                uint32_t after = before ^ s->xor_mask;
                uint32_t p_err = after;
                if (detect_mode & ORC_TERM_IN_FORMAT) {
                    /* alternative reading: the multiplication's result is held in the operand format (the paper's own
                     * example of a flipped zero is a 16-bit pattern, Section V-B). re_2 is the product rounded to that
                     * format, the mask addresses that format's storage bits like an operand site's, and Eq. 1-2 are
                     * applied with this re_2 and its flipped version widened back to FP32. */
                    before = orc_round_to_operand(dtype, f2u(re2));
                    after = orc_flip_operand(dtype, before, s->xor_mask);
                    re2 = orc_widen(dtype, before);
                    p_err = orc_widen_bits(dtype, after);
                }
                int det;
                uint32_t fin = product_check(detect_mode, p_err, f2u(a[s->k]), f2u(b[s->k]), &det);
                float rep = acc - re2;          /* Eq. 1 */
                acc = rep + u2f(fin);           /* Eq. 2 */
                if (log) { log[idx[t]].before_bits = before; log[idx[t]].after_bits = after;
                           log[idx[t]].final_bits = fin; log[idx[t]].status = 1 | (det ? 4u : 0u); }
            }
        }
    }
    return acc;
}

static float element_clean(const float *a, const float *b, int K)
{
    float acc = 0.0f;
    for (int k = 0; k < K; ++k) {
        float p = a[k] * b[k];
        acc = acc + p;
    }
    return acc;
}

/* ------------------------------------------------------------------ helpers */

static int site_valid(const orc_site *s, int dtype, int M, int N, int K)
{
    (void)dtype;
    switch (s->kind) {
    case ORC_A:    return s->row < (uint32_t)M && s->k < (uint32_t)K;
    case ORC_B:    return s->col < (uint32_t)N && s->k < (uint32_t)K;
    case ORC_ACC:  return s->row < (uint32_t)M && s->col < (uint32_t)N && s->k >= 1 && s->k <= (uint32_t)K;
    case ORC_OUT:  return s->row < (uint32_t)M && s->col < (uint32_t)N;
    case ORC_TERM: return s->row < (uint32_t)M && s->col < (uint32_t)N && s->k < (uint32_t)K;
    default:       return 0;
    }
}

static inline uint32_t load_storage(int dtype, const void *p, size_t idx)
{
    return dtype == ORC_TF32 ? ((const uint32_t *)p)[idx] : (uint32_t)((const uint16_t *)p)[idx];
}

static float *widen_matrix(int dtype, const void *src, size_t rows, size_t cols)
{
    float *dst = (float *)malloc(sizeof(float) * rows * cols);
    if (!dst) return NULL;
#pragma omp parallel for schedule(static)
    for (long long r = 0; r < (long long)rows; ++r)
        for (size_t c = 0; c < cols; ++c)
            dst[(size_t)r * cols + c] = orc_widen(dtype, load_storage(dtype, src, (size_t)r * cols + c));
    return dst;
}

static const uint64_t HASH_MUL = 0x9E3779B97F4A7C15ull;

#define ORC_OUTPUT_RANGE 64

/*
 * Largest FP32 exponent field in each row of a rows x K operand matrix (for the output-level
 * range check below). Zero rows give 0, Inf/NaN give 255.
 */
void orc_operand_exponents(int dtype, int rows, int K, const void *X, uint32_t *out)
{
    for (int r = 0; r < rows; ++r) {
        uint32_t e = 0;
        for (int k = 0; k < K; ++k) {
            uint32_t f = (orc_widen_bits(dtype, load_storage(dtype, X, (size_t)r * K + k)) >> 23) & 0xFFu;
            if (f > e) e = f;
        }
        out[r] = e;
    }
}

/*
 * Output-level range bound (an extension of the product bound of Section VI-A to a dot product):
 * every |a_ik| < 2^(eA+1) and |b_kj| < 2^(eB+1) with eA, eB the largest exponents of row i of A and of
 * column j of B, so |C_ij| < K * 2^(eA+eB+2) <= 2^(eA+eB+2+ceil(log2 K)), i.e. the exponent of C_ij is at
 * most eA + eB + 1 + ceil(log2 K). With biased fields: E <= EA + EB - 126 + ceil(log2 K), clamped to 0..255.
 */
int orc_output_range_bound(uint32_t EA, uint32_t EB, int K)
{
    int L = 0;
    while ((1 << L) < K) ++L;
    int b = (int)EA + (int)EB - 126 + L;
    if (b < 0) b = 0;
    if (b > 255) b = 255;
    return b;
}

/* output-element check: returns final bits, sets *det. BoundCheck for technique 1; for the RangeCheck
 * techniques only when an output bound is given (bound >= 0: ORC_OUTPUT_RANGE was requested). */
static uint32_t output_check(int detect_mode, uint32_t bits, int bound, int *det)
{
    int tech = detect_mode & 3;
    *det = 0;
    if (tech == ORC_T_BOUND) {
        *det = orc_boundcheck_detect(bits);
        if (*det && (detect_mode & ORC_CORRECT)) return orc_boundcheck_correct(bits);
        return bits;
    }
    if ((tech == ORC_T_RMAX || tech == ORC_T_RFLIP) && bound >= 0) {
        *det = orc_rangecheck_detect(bits, bound);
        if (*det && (detect_mode & ORC_CORRECT))
            return tech == ORC_T_RMAX ? orc_rangecheck_max(bits, bound) : orc_rangecheck_flip(bits, bound);
    }
    return bits;
}

/* ------------------------------------------------------------------ full GEMM (the definition) */

/*
 * C = A x B (+ addend) with every site of the table applied (full recompute), then the
 * output check. A: M x K, Bt: N x K (B stored K-major), C: M x N, FP32.
 * addend (M x N FP32, or NULL): the C of D = A x B + C (Section II-B). On the paper's platform it is
 * the accumulator the products are added to, so here every running sum starts from addend[i,j]
 * instead of +0 and then takes the K products in k order as before.
 * hdr[16]: [0] status, [1] n_detected, [2] n_corrected, [3] sites applied,
 * [4] sites skipped. log[n_faults]. bitmap[M * ceil(N/32)]: bit j%32 of word
 * i*ceil(N/32) + j/32 set iff element (i,j) was detected.
 * Returns 0, or -1 on allocation failure.
 */
static int gemm_impl(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *addend, float *C,
                     const orc_site *sites, int n_faults, int detect_mode, int kstep,
                     uint32_t *hdr, orc_site_log *log, uint32_t *bitmap)
{
    size_t wpr = ((size_t)N + 31) / 32;
    if (hdr) memset(hdr, 0, 16 * sizeof(uint32_t));
    if (log) memset(log, 0, sizeof(orc_site_log) * (size_t)n_faults);
    if (bitmap) memset(bitmap, 0, sizeof(uint32_t) * wpr * (size_t)M);

    float *Af = widen_matrix(dtype, A, (size_t)M, (size_t)K);
    float *Bf = widen_matrix(dtype, Bt, (size_t)N, (size_t)K);
    float *BfT = (float *)malloc(sizeof(float) * (size_t)K * (size_t)N);
    if (!Af || !Bf || !BfT) { free(Af); free(Bf); free(BfT); return -1; }

    /* output-level range check: exponent maxima of the CLEAN operands (a faulty operand must not widen its own bound) */
    uint32_t *EA = NULL, *EB = NULL;
    int range_out = (detect_mode & ORC_OUTPUT_RANGE) && ((detect_mode & 3) == ORC_T_RMAX || (detect_mode & 3) == ORC_T_RFLIP);
    if (range_out) {
        EA = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)M);
        EB = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)N);
        orc_operand_exponents(dtype, M, K, A, EA);
        orc_operand_exponents(dtype, N, K, Bt, EB);
    }
#define OUT_BOUND(i, j) (range_out ? orc_output_range_bound(EA[i], EB[j], K) : -1)

    uint32_t applied = 0, skipped = 0;
    /* step 3, operand sites: flip the storage word, the faulty value serves the whole row/column */
    for (int t = 0; t < n_faults; ++t) {
        const orc_site *s = &sites[t];
        if (!site_valid(s, dtype, M, N, K)) { skipped++; if (log) log[t].status = 2; continue; }
        applied++;
        if (s->kind == ORC_A || s->kind == ORC_B) {
            float *dst = s->kind == ORC_A ? &Af[(size_t)s->row * K + s->k] : &Bf[(size_t)s->col * K + s->k];
            const void *src = s->kind == ORC_A ? A : Bt;
            size_t pos = s->kind == ORC_A ? (size_t)s->row * K + s->k : (size_t)s->col * K + s->k;
            uint32_t before = load_storage(dtype, src, pos), after;
            if (dtype == ORC_TF32) before &= 0xFFFFE000u;
            /* earlier sites on the same storage word compose, in table order */
            for (int q = 0; q < t; ++q) {
                const orc_site *e = &sites[q];
                if (e->kind == s->kind && e->k == s->k && site_valid(e, dtype, M, N, K) &&
                    (s->kind == ORC_A ? e->row == s->row : e->col == s->col))
                    before = orc_flip_operand(dtype, before, e->xor_mask);
            }
            after = orc_flip_operand(dtype, before, s->xor_mask);
            *dst = orc_widen(dtype, after);
            if (log) { log[t].before_bits = before; log[t].after_bits = after; log[t].final_bits = after; log[t].status = 1; }
        }
    }
    for (int k = 0; k < K; ++k)
        for (int j = 0; j < N; ++j)
            BfT[(size_t)k * N + j] = Bf[(size_t)j * K + k];

    /* step 2 on every element (rows are independent; each element's k order is sequential) */
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < M; ++i) {
        float *c = &C[(size_t)i * N];
        for (int j = 0; j < N; ++j) c[j] = addend ? addend[(size_t)i * N + j] : 0.0f;
        for (int k = 0; k < K; ++k) {
            float a = Af[(size_t)i * K + k];
            const float *b = &BfT[(size_t)k * N];
            for (int j = 0; j < N; ++j) {
                float p = a * b[j];
                c[j] = c[j] + p;
            }
        }
    }

    /* elements that carry ACC / TERM sites: redo them with the sites active */
    int *idx = (int *)malloc(sizeof(int) * (size_t)(n_faults > 0 ? n_faults : 1));
    char *done = (char *)calloc((size_t)(n_faults > 0 ? n_faults : 1), 1);
    for (int t = 0; t < n_faults; ++t) {
        const orc_site *s = &sites[t];
        if (done[t] || !(s->kind == ORC_ACC || s->kind == ORC_TERM) || !site_valid(s, dtype, M, N, K)) continue;
        int n_idx = 0;
        for (int q = t; q < n_faults; ++q) {
            const orc_site *e = &sites[q];
            if ((e->kind == ORC_ACC || e->kind == ORC_TERM) && e->row == s->row && e->col == s->col &&
                site_valid(e, dtype, M, N, K)) { idx[n_idx++] = q; done[q] = 1; }
        }
        C[(size_t)s->row * N + s->col] =
            element_with_sites(dtype, &Af[(size_t)s->row * K], &Bf[(size_t)s->col * K], K, kstep, detect_mode,
                               sites, idx, n_idx, log,
                               addend ? addend[(size_t)s->row * N + s->col] : 0.0f);
    }
    free(idx); free(done);

    /* output sites, table order */
    for (int t = 0; t < n_faults; ++t) {
        const orc_site *s = &sites[t];
        if (s->kind != ORC_OUT || !site_valid(s, dtype, M, N, K)) continue;
        float *c = &C[(size_t)s->row * N + s->col];
        uint32_t before = f2u(*c), after = before ^ s->xor_mask;
        int det;
        *c = u2f(after);
        if (log) { log[t].before_bits = before; log[t].after_bits = after;
                   log[t].final_bits = output_check(detect_mode, after, OUT_BOUND(s->row, s->col), &det); log[t].status = 1; }
    }
    /* a later OUT site on the same element changes what the earlier one finally became */
    if (log)
        for (int t = 0; t < n_faults; ++t) {
            const orc_site *s = &sites[t];
            if (s->kind != ORC_OUT || log[t].status != 1) continue;
            int det;
            log[t].final_bits = output_check(detect_mode, f2u(C[(size_t)s->row * N + s->col]), OUT_BOUND(s->row, s->col), &det);
        }

    /* step 4 on every output element */
    uint32_t n_det = 0;
    if ((detect_mode & 3) == ORC_T_BOUND || range_out) {
        for (int i = 0; i < M; ++i)
            for (int j = 0; j < N; ++j) {
                int det;
                uint32_t fin = output_check(detect_mode, f2u(C[(size_t)i * N + j]), OUT_BOUND(i, j), &det);
                if (det) {
                    n_det++;
                    if (bitmap) bitmap[(size_t)i * wpr + (size_t)j / 32] |= 1u << (j % 32);
                    C[(size_t)i * N + j] = u2f(fin);
                }
            }
    }
    if (hdr) {
        hdr[1] = n_det;
        hdr[2] = (detect_mode & ORC_CORRECT) ? n_det : 0;
        hdr[3] = applied;
        hdr[4] = skipped;
        if (skipped) hdr[0] |= 1u;
    }
    free(Af); free(Bf); free(BfT); free(EA); free(EB);
#undef OUT_BOUND
    return 0;
}

int orc_gemm(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C,
             const orc_site *sites, int n_faults, int detect_mode, int kstep,
             uint32_t *hdr, orc_site_log *log, uint32_t *bitmap)
{
    return gemm_impl(dtype, M, N, K, A, Bt, NULL, C, sites, n_faults, detect_mode, kstep, hdr, log, bitmap);
}

/* D = A x B + C_in (Section II-B); C_in and D are M x N FP32 and must not overlap. */
int orc_gemm_addend(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_in, float *D,
                    const orc_site *sites, int n_faults, int detect_mode, int kstep,
                    uint32_t *hdr, orc_site_log *log, uint32_t *bitmap)
{
    return gemm_impl(dtype, M, N, K, A, Bt, C_in, D, sites, n_faults, detect_mode, kstep, hdr, log, bitmap);
}

/* ------------------------------------------------------------------ 16-bit output */

enum { ORC_OUT_FP16 = 0, ORC_OUT_BF16 = 1 };      /* (orc_round_to_operand above relies on these two values) */

/*
 * Round an FP32 word to the nearest value of a 16-bit format, ties to even (the models of
 * Section IV-B run "16" / "bf16" end to end: the FP32 result D of D = A x B + C, Section II-B,
 * goes back to the 16-bit format before the next layer reads it).
 * Written from the formats' definitions (Section II-A): FP16 1/5/10, bias 15, subnormals below
 * 2^-14, largest finite value 65504; BF16 1/8/7 = the upper half of an FP32 word.
 * A NaN stays a (quiet) NaN; which payload it carries is not specified here.
 */
uint32_t orc_round_output(int out_fmt, uint32_t bits)
{
    uint32_t sign = (bits >> 16) & 0x8000u;
    uint32_t E = (bits >> 23) & 0xFFu;
    uint32_t m = bits & 0x7FFFFFu;
    if (out_fmt == ORC_OUT_BF16) {
        if (E == 0xFFu && m != 0) return sign | 0x7FC0u;
        uint32_t keep = bits >> 16, rest = bits & 0xFFFFu;             /* 16 bits dropped */
        if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;   /* carries into the exponent; Inf at the top */
        return keep & 0xFFFFu;
    }
    /* FP16 */
    if (E == 0xFFu) return sign | (m ? 0x7E00u : 0x7C00u);
    float x = fabsf(u2f(bits));
    if (x >= 65520.0f) return sign | 0x7C00u;          /* halfway between 65504 and 2^16 ties to the even one: infinity */
    if (x < 6.103515625e-05f) {                          /* below 2^-14: multiples of 2^-24; the scaling is exact */
        float q = nearbyintf(x * 16777216.0f);           /* round-to-nearest-even is the default rounding mode */
        return sign | (uint32_t)q;                       /* 1024 = the smallest normal number, as it should be */
    }
    uint32_t keep = m >> 13, rest = m & 0x1FFFu;         /* 13 mantissa bits dropped */
    uint32_t h = ((E - 112u) << 10) + keep;              /* rebias 127 -> 15 */
    if (rest > 0x1000u || (rest == 0x1000u && (keep & 1u))) h += 1u;
    return sign | h;
}

/*
 * The fault-injected GEMM with a 16-bit result: everything as orc_gemm / orc_gemm_addend (sites,
 * checks, flags, counts and log all on the FP32 values), then every FP32 element is rounded once.
 */
int orc_gemm_out16(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_in, int out_fmt,
                   uint16_t *D16, const orc_site *sites, int n_faults, int detect_mode, int kstep,
                   uint32_t *hdr, orc_site_log *log, uint32_t *bitmap)
{
    float *D = (float *)malloc(sizeof(float) * (size_t)M * (size_t)N);
    if (!D) return -1;
    int rc = gemm_impl(dtype, M, N, K, A, Bt, C_in, D, sites, n_faults, detect_mode, kstep, hdr, log, bitmap);
    if (rc == 0)
        for (size_t e = 0; e < (size_t)M * (size_t)N; ++e) D16[e] = (uint16_t)orc_round_output(out_fmt, f2u(D[e]));
    free(D);
    return rc;
}

/* ------------------------------------------------------------------ single trials (incremental mode) */

typedef struct {
    uint32_t n_aff, n_det, first;
    uint64_t hash;
    float maxdev;
    int changed;
} trial_acc;

static void trial_account(trial_acc *t, int detect_mode, float value, float clean, uint32_t lin, uint32_t *final_bits)
{
    int det;
    uint32_t fin = output_check(detect_mode, f2u(value), -1, &det);   /* campaigns have no output-level range check */
    t->n_aff++;
    if (det) {
        t->n_det++;
        t->hash += ((uint64_t)lin + 1ull) * HASH_MUL;
        if (lin < t->first) t->first = lin;
    }
    if (fin != f2u(clean)) t->changed = 1;
    float dev = fabsf(u2f(fin) - clean);
    if (dev != dev) dev = INFINITY;             /* NaN deviation counts as unbounded */
    if (dev > t->maxdev) t->maxdev = dev;
    if (final_bits) *final_bits = fin;
}

/*
 * Raw (unchecked) values of the output elements an operand site reaches: row s->row of C for an
 * A site (N values), column s->col for a B site (M values).
 *   form 0: the definition -- every affected element is accumulated again in k order with the
 *           faulty operand in place of the clean one;
 *   form 1: the write-back of Eq. 1-2 (Section III-E) applied to the FINISHED clean sum c:
 *           rep = fl32(c - fl32(x*y)), then c' = fl32(rep + fl32(x'*y)), with x the clean operand,
 *           x' the faulty one and y the other factor of the term. This is how a faulty term enters
 *           a sum that has already been accumulated; it differs from form 0 only by the roundings
 *           of the two steps.
 * Af, Bf: widened operands. Returns the number of values written.
 */
static int operand_trial_values(int dtype, int M, int N, int K, const void *A, const void *Bt,
                                const float *Af, const float *Bf, const float *C_clean,
                                const orc_site *s, int form, float *out)
{
    int isA = s->kind == ORC_A;
    size_t pos = isA ? (size_t)s->row * K + s->k : (size_t)s->col * K + s->k;
    uint32_t before = load_storage(dtype, isA ? A : Bt, pos);
    if (dtype == ORC_TF32) before &= 0xFFFFE000u;
    uint32_t after = orc_flip_operand(dtype, before, s->xor_mask);
    float x = orc_widen(dtype, before), xf = orc_widen(dtype, after);
    int n_other = isA ? N : M;
    if (form == 0) {
        float *vec = (float *)malloc(sizeof(float) * (size_t)K);
        memcpy(vec, isA ? &Af[(size_t)s->row * K] : &Bf[(size_t)s->col * K], sizeof(float) * (size_t)K);
        vec[s->k] = xf;
        for (int o = 0; o < n_other; ++o)
            out[o] = isA ? element_clean(vec, &Bf[(size_t)o * K], K) : element_clean(&Af[(size_t)o * K], vec, K);
        free(vec);
    } else {
        for (int o = 0; o < n_other; ++o) {
            float y = isA ? Bf[(size_t)o * K + s->k] : Af[(size_t)o * K + s->k];
            float c = isA ? C_clean[(size_t)s->row * N + o] : C_clean[(size_t)o * N + s->col];
            float re2 = x * y;          /* the clean term */
            float re_err = xf * y;      /* the faulty term */
            float rep = c - re2;        /* Eq. 1 */
            out[o] = rep + re_err;      /* Eq. 2 */
        }
    }
    return n_other;
}

int orc_operand_trial_values(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_clean,
                             const orc_site *s, int form, float *out)
{
    if (!(s->kind == ORC_A || s->kind == ORC_B) || !site_valid(s, dtype, M, N, K)) return -1;
    float *Af = widen_matrix(dtype, A, (size_t)M, (size_t)K);
    float *Bf = widen_matrix(dtype, Bt, (size_t)N, (size_t)K);
    if (!Af || !Bf) { free(Af); free(Bf); return -1; }
    int n = operand_trial_values(dtype, M, N, K, A, Bt, Af, Bf, C_clean, s, form, out);
    free(Af); free(Bf);
    return n;
}

/*
 * One record per trial, each trial = one site applied alone to the clean GEMM.
 * Only the affected output elements are recomputed (an A site: row i, a B site:
 * column j, others: one element), each by the same sequential loop as orc_gemm.
 * C_clean: the fault-free, unchecked output of orc_gemm (detect_mode 0).
 * operand_form: how an operand trial reaches its row / column, see operand_trial_values
 * (0 = recompute, the definition; 1 = Eq. 1-2 on the finished sums of C_clean).
 */
int orc_campaign_form(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_clean,
                      const orc_site *sites, int n_trials, int detect_mode, int kstep, int operand_form,
                      orc_trial_record *rec)
{
    float *Af = widen_matrix(dtype, A, (size_t)M, (size_t)K);
    float *Bf = widen_matrix(dtype, Bt, (size_t)N, (size_t)K);
    if (!Af || !Bf) { free(Af); free(Bf); return -1; }

#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < n_trials; ++t) {
        const orc_site *s = &sites[t];
        orc_trial_record *r = &rec[t];
        memset(r, 0, sizeof(*r));
        r->kind = s->kind;
        r->first_detected = 0xFFFFFFFFu;
        if (!site_valid(s, dtype, M, N, K)) { r->status = 1u << 8; continue; }
        trial_acc ta = {0, 0, 0xFFFFFFFFu, 0ull, 0.0f, 0};
        if (s->kind == ORC_OUT) {
            uint32_t lin = s->row * (uint32_t)N + s->col;
            uint32_t before = f2u(C_clean[lin]);
            uint32_t after = before ^ s->xor_mask;
            r->primary_index = lin; r->before_bits = before; r->after_bits = after;
            trial_account(&ta, detect_mode, u2f(after), C_clean[lin], lin, &r->final_bits);
        } else if (s->kind == ORC_ACC || s->kind == ORC_TERM) {
            uint32_t lin = s->row * (uint32_t)N + s->col;
            orc_site_log lg; int idx0 = 0;
            orc_site one = *s;
            float v = element_with_sites(dtype, &Af[(size_t)s->row * K], &Bf[(size_t)s->col * K], K, kstep,
                                         detect_mode, &one, &idx0, 1, &lg, 0.0f);
            r->primary_index = lin; r->before_bits = lg.before_bits; r->after_bits = lg.after_bits;
            trial_account(&ta, detect_mode, v, C_clean[lin], lin, &r->final_bits);
        } else {
            int isA = s->kind == ORC_A;
            size_t pos = isA ? (size_t)s->row * K + s->k : (size_t)s->col * K + s->k;
            uint32_t before = load_storage(dtype, isA ? A : Bt, pos);
            if (dtype == ORC_TF32) before &= 0xFFFFE000u;
            uint32_t after = orc_flip_operand(dtype, before, s->xor_mask);
            r->primary_index = (uint32_t)pos; r->before_bits = before; r->after_bits = after; r->final_bits = after;
            int n_other = isA ? N : M;
            float *vals = (float *)malloc(sizeof(float) * (size_t)n_other);
            operand_trial_values(dtype, M, N, K, A, Bt, Af, Bf, C_clean, s, operand_form, vals);
            for (int o = 0; o < n_other; ++o) {
                uint32_t lin = isA ? s->row * (uint32_t)N + (uint32_t)o : (uint32_t)o * (uint32_t)N + s->col;
                trial_account(&ta, detect_mode, vals[o], C_clean[lin], lin, NULL);
            }
            free(vals);
        }
        r->n_affected = ta.n_aff; r->n_detected = ta.n_det; r->idx_hash = ta.hash;
        r->first_detected = ta.first; r->max_abs_dev = ta.maxdev;
        r->status = (ta.changed ? 1u : 0u) | (ta.n_det ? 2u : 0u) |
                    ((ta.n_det && (detect_mode & ORC_CORRECT) && (detect_mode & 3) == ORC_T_BOUND) ? 4u : 0u);
    }
    free(Af); free(Bf);
    return 0;
}

int orc_campaign(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_clean,
                 const orc_site *sites, int n_trials, int detect_mode, int kstep, orc_trial_record *rec)
{
    return orc_campaign_form(dtype, M, N, K, A, Bt, C_clean, sites, n_trials, detect_mode, kstep, 0, rec);
}

/* ------------------------------------------------------------------ sampled outputs at any size */

/*
 * Clean C[i,j] for n sampled (i,j) pairs straight from the storage matrices,
 * with the operand XORs of (optional) A/B sites applied, and (|A||B|)_ij in
 * double for tolerances. No matrix is widened as a whole.
 * start (or NULL): start[t] is what sample t's running sum begins with, the addend c_ij of
 * D = A x B + C (Section II-B); |start[t]| joins out_absprod[t].
 */
static int sample_impl(int dtype, int K, const void *A, const void *Bt,
                       const orc_site *sites, int n_faults, const float *start,
                       const uint32_t *si, const uint32_t *sj, int n, float *out_c, double *out_absprod)
{
#pragma omp parallel for schedule(dynamic, 16)
    for (int t = 0; t < n; ++t) {
        uint32_t i = si[t], j = sj[t];
        float acc = start ? start[t] : 0.0f;
        double ap = start ? fabs((double)start[t]) : 0.0;
        for (int k = 0; k < K; ++k) {
            uint32_t sa = load_storage(dtype, A, (size_t)i * K + k);
            uint32_t sb = load_storage(dtype, Bt, (size_t)j * K + k);
            for (int q = 0; q < n_faults; ++q) {
                const orc_site *s = &sites[q];
                if (s->kind == ORC_A && s->row == i && s->k == (uint32_t)k) sa = orc_flip_operand(dtype, sa, s->xor_mask);
                if (s->kind == ORC_B && s->col == j && s->k == (uint32_t)k) sb = orc_flip_operand(dtype, sb, s->xor_mask);
            }
            float a = orc_widen(dtype, sa), b = orc_widen(dtype, sb);
            float p = a * b;
            acc = acc + p;
            ap += fabs((double)a) * fabs((double)b);
        }
        out_c[t] = acc;
        if (out_absprod) out_absprod[t] = ap;
    }
    return 0;
}

int orc_sample(int dtype, int M, int N, int K, const void *A, const void *Bt,
               const orc_site *sites, int n_faults,
               const uint32_t *si, const uint32_t *sj, int n, float *out_c, double *out_absprod)
{
    (void)M; (void)N;
    return sample_impl(dtype, K, A, Bt, sites, n_faults, NULL, si, sj, n, out_c, out_absprod);
}

int orc_sample_addend(int dtype, int M, int N, int K, const void *A, const void *Bt,
                      const orc_site *sites, int n_faults, const float *start,
                      const uint32_t *si, const uint32_t *sj, int n, float *out_c, double *out_absprod)
{
    (void)M; (void)N;
    return sample_impl(dtype, K, A, Bt, sites, n_faults, start, si, sj, n, out_c, out_absprod);
}

/* (|A||B|) for all elements, double precision; used only for tolerances at small sizes */
int orc_absprod(int dtype, int M, int N, int K, const void *A, const void *Bt, double *out)
{
    float *Af = widen_matrix(dtype, A, (size_t)M, (size_t)K);
    float *Bf = widen_matrix(dtype, Bt, (size_t)N, (size_t)K);
    if (!Af || !Bf) { free(Af); free(Bf); return -1; }
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i)
        for (int j = 0; j < N; ++j) {
            double s = 0.0;
            for (int k = 0; k < K; ++k)
                s += fabs((double)Af[(size_t)i * K + k]) * fabs((double)Bf[(size_t)j * K + k]);
            out[(size_t)i * N + j] = s;
        }
    free(Af); free(Bf);
    return 0;
}

/* ------------------------------------------------------------------ deviation summary */

/*
 * Section V-B: share of trials with zero difference (Table II) and the spread of the
 * non-zero differences, binned by the FP32 exponent field of the trial's largest
 * |final - clean|. out[0..5]: trials, invalid, zero-diff, detected, corrected, non-finite;
 * out[6..10]: trials per site kind; out[11..15]: zero-diff trials per kind;
 * out[16..271]: histogram over the exponent field (NaN counted with the infinities).
 */
void orc_summary(const orc_trial_record *rec, int n, uint32_t *out)
{
    memset(out, 0, sizeof(uint32_t) * 272);
    out[0] = (uint32_t)n;
    for (int t = 0; t < n; ++t) {
        const orc_trial_record *r = &rec[t];
        if (r->status & (1u << 8)) { out[1]++; continue; }
        int zero = (r->status & 1u) == 0;
        if (zero) out[2]++;
        if (r->status & 2u) out[3]++;
        if (r->status & 4u) out[4]++;
        if (r->kind < 5) { out[6 + r->kind]++; if (zero) out[11 + r->kind]++; }
        float d = r->max_abs_dev;
        if (d != d || isinf(d)) { out[5]++; out[16 + 255]++; continue; }
        if (d == 0.0f) continue;
        out[16 + ((f2u(d) >> 23) & 0xFFu)]++;
    }
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
