/*
 * rkv_oracle.c -- CPU oracle (test infrastructure only; see rkv_oracle.h).
 *
 * Plain C11, one sequential pass per candidate in ascending index order.
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fPIC -shared.
 * Every float operation below is a single IEEE-754 binary32 operation rounded
 * to nearest-even; a fused multiply-add happens only where fmaf() is written.
 */
#include "rkv_oracle.h"

#include <math.h>
#include <stddef.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* Philox4x32-10                                                            */
/* ------------------------------------------------------------------------ */

/* One block of Philox4x32 with ten rounds, as published by Salmon et al.
 * (SC'11): per round two 32x32->64 products with the multipliers below, the
 * high halves xored with the other counter words and the round key; the key is
 * bumped by the two Weyl constants between rounds (nine bumps). */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Counter / key layout of this project (the paper only says "multiple random
 * seeds"): key = seed, counter = (block index, stream id), block j serves the
 * four consecutive elements 4j .. 4j+3, word (i & 3) belongs to element i. */
static void block_words(uint64_t seed, uint64_t stream_id, uint64_t j, uint32_t w[4])
{
    uint32_t ctr[4] = { (uint32_t)j, (uint32_t)(j >> 32),
                        (uint32_t)stream_id, (uint32_t)(stream_id >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    orc_philox4x32_10(ctr, key, w);
}

/* ------------------------------------------------------------------------ */
/* Distribution transforms                                                  */
/* ------------------------------------------------------------------------ */

static uint32_t f32_bits(float x) { uint32_t b; memcpy(&b, &x, 4); return b; }
static float bits_f32(uint32_t b) { float x; memcpy(&x, &b, 4); return x; }

/* log(u), u = k24 * 2^-24 in (0,1].  u = m * 2^e with m folded into
 * [sqrt(1/2), sqrt(2)]; log m = 2 atanh(s), s = (m-1)/(m+1), by the odd series
 * 2(s + s^3/3 + s^5/5 + s^7/7 + s^9/9), |s| <= 0.1716 so the next term is
 * below 1e-9.  Coefficients are the fp32 roundings of 2/3, 2/5, 2/7, 2/9. */
float orc_log_unit(uint32_t k24)
{
    float u = (float)k24 * 0x1p-24f;               /* exact */
    uint32_t b = f32_bits(u);
    int e = (int)(b >> 23) - 127;
    float m = bits_f32((b & 0x007FFFFFu) | 0x3F800000u);   /* [1,2) */
    if (m > 0x1.6a09e6p+0f) {                      /* sqrt(2) rounded to fp32 */
        m = m * 0.5f;
        e = e + 1;
    }
    float s = (m - 1.0f) / (m + 1.0f);
    float s2 = s * s;
    float p = 0x1.c71c72p-3f;                      /* 2/9 */
    p = fmaf(s2, p, 0x1.24924ap-2f);               /* 2/7 */
    p = fmaf(s2, p, 0x1.99999ap-2f);               /* 2/5 */
    p = fmaf(s2, p, 0x1.555556p-1f);               /* 2/3 */
    p = fmaf(s2, p, 2.0f);
    float logm = s * p;
    return fmaf((float)e, 0x1.62e430p-1f, logm);   /* e * ln 2 + log m */
}

/* sin and cos of one turn fraction k24 * 2^-24.  The octant is taken from the
 * top three bits exactly; the remainder is folded to theta in [0, pi/4] and the
 * Taylor polynomials (sin to theta^9, cos to theta^10) are evaluated by Horner
 * with fused multiply-adds.  Coefficients are fp32 roundings of 1/k!. */
void orc_sincos_turn(uint32_t k24, float *s_out, float *c_out)
{
    uint32_t oct = (k24 >> 21) & 7u;
    uint32_t rem = k24 & 0x1FFFFFu;
    if (oct & 1u)
        rem = 0x200000u - rem;
    float t = (float)rem * 0x1p-21f;               /* exact, [0,1] */
    float th = t * 0x1.921fb6p-1f;                 /* * pi/4 */
    float x2 = th * th;

    float ps = 0x1.71de3ap-19f;                    /*  1/9! */
    ps = fmaf(x2, ps, -0x1.a01a02p-13f);           /* -1/7! */
    ps = fmaf(x2, ps, 0x1.111112p-7f);             /*  1/5! */
    ps = fmaf(x2, ps, -0x1.555556p-3f);            /* -1/3! */
    float sv = fmaf(th * x2, ps, th);

    float pc = -0x1.27e4fcp-22f;                   /* -1/10! */
    pc = fmaf(x2, pc, 0x1.a01a02p-16f);            /*  1/8!  */
    pc = fmaf(x2, pc, -0x1.6c16c2p-10f);           /* -1/6!  */
    pc = fmaf(x2, pc, 0x1.555556p-5f);             /*  1/4!  */
    pc = fmaf(x2, pc, -0.5f);                      /* -1/2!  */
    float cv = fmaf(x2, pc, 1.0f);

    float sn, cs;
    if ((oct + 1u) & 2u) { sn = cv; cs = sv; }     /* octants 1,2,5,6 swap */
    else                 { sn = sv; cs = cv; }
    if (oct & 4u) sn = -sn;                        /* lower half plane */
    if ((oct + 2u) & 4u) cs = -cs;                 /* left half plane  */
    *s_out = sn;
    *c_out = cs;
}

void orc_log_unit_range(uint32_t k_first, uint32_t count, float *out)
{
    for (uint32_t q = 0; q < count; ++q) out[q] = orc_log_unit(k_first + q);
}

void orc_sincos_turn_range(uint32_t k_first, uint32_t count, float *s, float *c)
{
    for (uint32_t q = 0; q < count; ++q) orc_sincos_turn(k_first + q, &s[q], &c[q]);
}

/* Box-Muller on a pair of words: u1 in (0,1], u2 in [0,1). */
void orc_box_muller(uint32_t w0, uint32_t w1, float *z_even, float *z_odd)
{
    float lg = orc_log_unit((w0 >> 8) + 1u);
    float rad = sqrtf(-2.0f * lg);
    float sn, cs;
    orc_sincos_turn(w1 >> 8, &sn, &cs);
    *z_even = rad * cs;
    *z_odd = rad * sn;
}

float orc_uniform_pm1(uint32_t w)
{
    return (float)(w >> 8) * 0x1p-23f - 1.0f;      /* both steps exact */
}

/* Inverse CDF of Student-t with 2 degrees of freedom:
 * t = (2u - 1) / sqrt(2 u (1 - u)), u an odd multiple of 2^-24 in (0,1). */
float orc_student_t2(uint32_t w)
{
    float u = (float)(2u * (w >> 9) + 1u) * 0x1p-24f;   /* exact */
    float a = 2.0f * u - 1.0f;                     /* exact */
    float b = u * (1.0f - u);
    return a / sqrtf(2.0f * b);
}

/* fp32 -> bf16 by round-to-nearest-even on the bit pattern (NaN kept quiet). */
uint16_t orc_bf16_rne(float x)
{
    uint32_t b = f32_bits(x);
    if ((b & 0x7FFFFFFFu) > 0x7F800000u)
        return (uint16_t)((b >> 16) | 0x0040u);
    b += 0x7FFFu + ((b >> 16) & 1u);
    return (uint16_t)(b >> 16);
}

float orc_gen_value(uint64_t seed, uint64_t stream_id, int dist, uint64_t i)
{
    uint32_t w[4];
    uint64_t j = i >> 2;
    unsigned lane = (unsigned)(i & 3u);
    block_words(seed, stream_id, j, w);

    if (dist == ORC_UNIFORM_PM1)
        return orc_uniform_pm1(w[lane]);
    if (dist == ORC_STUDENT_T2)
        return orc_student_t2(w[lane]);

    /* the three normal-based distributions: words (0,1) -> elements (4j, 4j+1),
     * words (2,3) -> elements (4j+2, 4j+3) */
    float ze, zo;
    orc_box_muller(w[lane & 2u], w[(lane & 2u) + 1u], &ze, &zo);
    float z = (lane & 1u) ? zo : ze;
    if (dist == ORC_NORMAL)
        return z;
    if (dist == ORC_NORMAL_1E4)
        return z * 0x1.388p+13f;                   /* 1e4 */
    /* ORC_SPARSE90: the mask word is the same lane of the block that the
     * stream (stream_id + 1) gives for the same j; floor(0.9 * 2^32) */
    uint32_t mw[4];
    block_words(seed, stream_id + 1u, j, mw);
    return (mw[lane] < 0xE6666666u) ? 0.0f : z;
}

int orc_gen(uint64_t seed, uint64_t stream_id, int dist, uint64_t n, uint64_t first_elem,
            int dtype, void *out)
{
    if (dist < ORC_NORMAL || dist > ORC_NORMAL_1E4) return -1;
    if (dtype != ORC_F32 && dtype != ORC_BF16) return -1;
    if (n > 0 && out == NULL) return -1;
    for (uint64_t q = 0; q < n; ++q) {
        float v = orc_gen_value(seed, stream_id, dist, first_elem + q);
        if (dtype == ORC_F32)
            ((float *)out)[q] = v;
        else
            ((uint16_t *)out)[q] = orc_bf16_rne(v);
    }
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Verification                                                             */
/* ------------------------------------------------------------------------ */

/* IEEE binary16 -> the fp32 bit pattern of the same value (every binary16 value is an
 * fp32 value).  1 sign bit, 5 exponent bits (bias 15), 10 fraction bits. */
uint32_t orc_f16_to_f32_bits(uint16_t h)
{
    const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    const uint32_t expo = (h >> 10) & 0x1Fu;
    uint32_t frac = h & 0x3FFu;
    if (expo == 0x1Fu)                              /* infinity or NaN: payload kept in the top bits */
        return sign | 0x7F800000u | (frac << 13);
    if (expo == 0) {
        if (frac == 0) return sign;                 /* signed zero */
        /* subnormal: value = frac * 2^-24; shift the leading one up to the hidden-bit position */
        int e = -14;
        while (!(frac & 0x400u)) { frac <<= 1; e--; }
        frac &= 0x3FFu;
        return sign | ((uint32_t)(e + 127) << 23) | (frac << 13);
    }
    return sign | ((expo - 15u + 127u) << 23) | (frac << 13);
}

/* Element q of a tensor as the fp32 bit pattern of its exact upcast
 * (bf16 -> fp32 appends sixteen zero bits; fp16 -> fp32 re-biases the exponent). */
static uint32_t load_bits(const void *p, int dtype, uint64_t q)
{
    if (dtype == ORC_F32)
        return ((const uint32_t *)p)[q];
    if (dtype == ORC_F16)
        return orc_f16_to_f32_bits(((const uint16_t *)p)[q]);
    return (uint32_t)((const uint16_t *)p)[q] << 16;
}

static int dtype_known(int d) { return d == ORC_F32 || d == ORC_BF16 || d == ORC_F16; }

static int bits_is_nan(uint32_t b) { return (b & 0x7FFFFFFFu) > 0x7F800000u; }
static int bits_is_inf(uint32_t b) { return (b & 0x7FFFFFFFu) == 0x7F800000u; }
static int bits_is_finite(uint32_t b) { return (b & 0x7F800000u) != 0x7F800000u; }

int orc_verify(const void *ref, int ref_dtype, const void *input, int input_dtype,
               const void *cand, int cand_dtype, uint64_t n, float atol, float rtol,
               orc_result *res)
{
    if (!ref || !cand || !res || n == 0) return -1;
    if (!dtype_known(ref_dtype) || !dtype_known(cand_dtype)) return -1;
    if (input && !dtype_known(input_dtype)) return -1;

    uint64_t n_over = 0, n_nan = 0, n_inf = 0, n_inf_mis = 0, n_cmp = 0;
    uint64_t arg_abs = ORC_NO_INDEX, arg_rel = ORC_NO_INDEX;
    float max_abs = -1.0f, max_rel = -1.0f;    /* first comparable element always wins */
    double sum_abs = 0.0;
    uint32_t cand_const_acc = 0, cand_copy_acc = 0, ref_const_acc = 0, ref_copy_acc = 0;
    const uint32_t c_first = load_bits(cand, cand_dtype, 0);
    const uint32_t r_first = load_bits(ref, ref_dtype, 0);

    for (uint64_t i = 0; i < n; ++i) {
        const uint32_t cb = load_bits(cand, cand_dtype, i);
        const uint32_t rb = load_bits(ref, ref_dtype, i);
        const float c = bits_f32(cb);
        const float r = bits_f32(rb);

        if (bits_is_nan(cb)) n_nan++;
        if (bits_is_inf(cb)) n_inf++;

        if (bits_is_finite(cb) && bits_is_finite(rb)) {
            /* the tolerance rule of the paper's evaluation environment, in the
             * isclose form |c - r| <= atol + rtol*|r| (reference on the right) */
            const float e = fabsf(c - r);
            const float thr = atol + (rtol * fabsf(r));
            if (!(e <= thr)) n_over++;
            if (e > max_abs) { max_abs = e; arg_abs = i; }
            if (r != 0.0f) {
                const float q = e / fabsf(r);
                if (q > max_rel) { max_rel = q; arg_rel = i; }
            }
            sum_abs += (double)e;
            n_cmp++;
        } else if (bits_is_inf(cb) && cb == rb) {
            /* equal infinities: a match; not part of the error statistics */
        } else {
            n_over++;
            if (bits_is_inf(cb) || bits_is_inf(rb)) n_inf_mis++;
        }

        cand_const_acc |= cb ^ c_first;
        ref_const_acc |= rb ^ r_first;
        if (input) {
            const uint32_t ib = load_bits(input, input_dtype, i);
            cand_copy_acc |= cb ^ ib;
            ref_copy_acc |= rb ^ ib;
        }
    }

    memset(res, 0, sizeof *res);
    res->n_over_tol = n_over;
    res->n_nan = n_nan;
    res->n_inf = n_inf;
    res->n_inf_mismatch = n_inf_mis;
    res->n_comparable = n_cmp;
    res->argmax_abs_err = arg_abs;
    res->argmax_rel_err = arg_rel;
    res->sum_abs_err = sum_abs;
    res->max_abs_err = (arg_abs == ORC_NO_INDEX) ? 0.0f : max_abs;
    res->max_rel_err = (arg_rel == ORC_NO_INDEX) ? 0.0f : max_rel;
    res->mean_abs_err = n_cmp ? (float)(sum_abs / (double)n_cmp) : 0.0f;

    uint32_t flags = 0;
    if (cand_const_acc == 0) flags |= ORC_CAND_CONST;
    if (ref_const_acc == 0) flags |= ORC_REF_CONST;
    if (input && cand_copy_acc == 0) flags |= ORC_CAND_COPY_OF_INPUT;
    if (input && ref_copy_acc == 0) flags |= ORC_REF_COPY_OF_INPUT;
    if (n_nan) flags |= ORC_HAS_NAN;
    if (n_inf) flags |= ORC_HAS_INF;
    res->flags = flags;

    /* A constant (or input-copy) candidate is failed only when the reference is
     * not constant (not a copy) itself: the paper's constant-output exploit
     * matches a constant reference, which is a flaw of the task, so it is
     * flagged and not failed.  A single element is constant by definition and
     * never fails on that. */
    uint32_t verdict = 0;
    if (n_over) verdict |= ORC_FAIL_TOL;
    if (n_nan) verdict |= ORC_FAIL_NAN;
    if (n_inf_mis) verdict |= ORC_FAIL_INF_MISMATCH;
    if ((flags & ORC_CAND_CONST) && !(flags & ORC_REF_CONST) && n > 1)
        verdict |= ORC_FAIL_LOOPHOLE_CONST;
    if ((flags & ORC_CAND_COPY_OF_INPUT) && !(flags & ORC_REF_COPY_OF_INPUT))
        verdict |= ORC_FAIL_LOOPHOLE_COPY;
    res->verdict = verdict;
    return 0;
}

/* Maximum of fl(e/|r|) found while dividing only when the element can beat the
 * running maximum q, i.e. when e >= fl(q*|r|).  Rounding is monotone, so
 * fl(e/|r|) > q implies e/|r| > q, hence e > q*|r| exactly and e >= fl(q*|r|):
 * the test never skips a new maximum.  fp32 finite inputs only. */
float orc_max_rel_filtered(const float *ref, const float *cand, uint64_t n, uint64_t *argmax)
{
    float q = -1.0f;
    uint64_t arg = ORC_NO_INDEX;
    for (uint64_t i = 0; i < n; ++i) {
        const float a = fabsf(ref[i]);
        if (a == 0.0f) continue;
        const float e = fabsf(cand[i] - ref[i]);
        if (e >= q * a) {
            const float qi = e / a;
            if (qi > q) { q = qi; arg = i; }
        }
    }
    *argmax = arg;
    return (arg == ORC_NO_INDEX) ? 0.0f : q;
}

void orc_joint_pass(const orc_result *results, int K, int T, uint32_t *joint_pass)
{
    for (int k = 0; k < K; ++k) {
        uint32_t ok = 1;
        for (int t = 0; t < T; ++t)
            if (results[(size_t)k * (size_t)T + (size_t)t].verdict != 0) ok = 0;
        joint_pass[k] = ok;
    }
}

/* ------------------------------------------------------------------------- */
/* Task-soundness screens (App. A.1 "filtering criteria"): statistics of the  */
/* reference outputs of one task over S seeds, and the exclusion flags.      */
/* ------------------------------------------------------------------------- */
int orc_screen(const void *const *outs, int S, uint64_t rows, uint64_t cols, int dtype,
               float range_lim, double std_lim, float spread_lim, orc_screen_result *res)
{
    if (!outs || !res || S < 1 || rows < 1 || cols < 1) return -1;
    if (dtype != ORC_F32 && dtype != ORC_BF16) return -1;
    for (int s = 0; s < S; ++s) if (!outs[s]) return -1;
    const uint64_t n = rows * cols;

    /* range, count, mean: every finite value of every seed */
    uint64_t n_fin = 0, n_nonfin = 0;
    float vmin = INFINITY, vmax = -INFINITY;
    double sum = 0.0;
    for (int s = 0; s < S; ++s)
        for (uint64_t i = 0; i < n; ++i) {
            const uint32_t b = load_bits(outs[s], dtype, i);
            if (!bits_is_finite(b)) { n_nonfin++; continue; }
            const float x = bits_f32(b);
            if (x < vmin) vmin = x;
            if (x > vmax) vmax = x;
            sum += (double)x;
            n_fin++;
        }
    const double mean = n_fin ? sum / (double)n_fin : 0.0;
    /* population standard deviation, second pass about the mean */
    double ss = 0.0;
    for (int s = 0; s < S; ++s)
        for (uint64_t i = 0; i < n; ++i) {
            const uint32_t b = load_bits(outs[s], dtype, i);
            if (!bits_is_finite(b)) continue;
            const double d = (double)bits_f32(b) - mean;
            ss += d * d;
        }
    const double sd = n_fin ? sqrt(ss / (double)n_fin) : 0.0;

    /* variation across seeds: per element the spread max_s - min_s (one fp32
     * subtraction); elements with a non-finite value in some seed are left out */
    float spread = -1.0f;
    uint64_t arg = ORC_NO_INDEX;
    if (S >= 2)
        for (uint64_t i = 0; i < n; ++i) {
            float lo = INFINITY, hi = -INFINITY;
            int ok = 1;
            for (int s = 0; s < S; ++s) {
                const uint32_t b = load_bits(outs[s], dtype, i);
                if (!bits_is_finite(b)) { ok = 0; break; }
                const float x = bits_f32(b);
                if (x < lo) lo = x;
                if (x > hi) hi = x;
            }
            if (!ok) continue;
            const float d = hi - lo;
            if (d > spread) { spread = d; arg = i; }
        }

    /* uniformity along an axis: every slice along it repeats its first element bit for bit */
    int uni0 = rows >= 2, uni1 = cols >= 2;
    for (int s = 0; s < S; ++s)
        for (uint64_t r = 0; r < rows; ++r)
            for (uint64_t c = 0; c < cols; ++c) {
                const uint32_t b = load_bits(outs[s], dtype, r * cols + c);
                if (b != load_bits(outs[s], dtype, c)) uni0 = 0;          /* down column c */
                if (b != load_bits(outs[s], dtype, r * cols)) uni1 = 0;   /* along row r   */
            }

    memset(res, 0, sizeof *res);
    res->n_values = (uint64_t)S * n;
    res->n_nonfinite = n_nonfin;
    res->argmax_seed_spread = arg;
    res->mean = mean;
    res->std = sd;
    res->vmin = vmin;
    res->vmax = vmax;
    res->max_seed_spread = spread;
    uint32_t f = 0;
    if (n_fin && vmin >= -range_lim && vmax <= range_lim) f |= ORC_SCREEN_NARROW_RANGE;
    if (n_fin && sd < std_lim) f |= ORC_SCREEN_LOW_STD;
    if (S >= 2 && arg != ORC_NO_INDEX && spread < spread_lim) f |= ORC_SCREEN_LOW_SEED_VARIATION;
    if (uni0) f |= ORC_SCREEN_UNIFORM_AXIS0;
    if (uni1) f |= ORC_SCREEN_UNIFORM_AXIS1;
    if (n_nonfin) f |= ORC_SCREEN_NONFINITE;
    res->flags = f;
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Cross-seed variation of ONE candidate's outputs (Sec. 3: a loophole is an  */
/* output with "insufficient variation across different seeds"; a kernel that */
/* hard-codes its result ignores the input seed altogether).  outs[s] is the  */
/* candidate's output for input seed s; seed 0 plays the reference.           */
/* ------------------------------------------------------------------------- */
int orc_cross_seed(const void *const *outs, int S, uint64_t n, int dtype, float atol, float rtol,
                   float spread_lim, orc_cross_result *res)
{
    if (!outs || !res || S < 1 || n < 1 || !dtype_known(dtype)) return -1;
    for (int s = 0; s < S; ++s) if (!outs[s]) return -1;

    int identical = 1, within = 1;
    uint64_t n_nonfin = 0, arg = ORC_NO_INDEX;
    float spread = -1.0f;
    for (uint64_t i = 0; i < n; ++i) {
        const uint32_t b0 = load_bits(outs[0], dtype, i);
        const float x0 = bits_f32(b0);
        float lo = INFINITY, hi = -INFINITY;
        int all_finite = 1;
        for (int s = 0; s < S; ++s) {
            const uint32_t b = load_bits(outs[s], dtype, i);
            const float x = bits_f32(b);
            if (b != b0) identical = 0;             /* the widening is one-to-one: storage bits differ */
            if (!bits_is_finite(b)) all_finite = 0;
            if (s > 0) {
                /* the tolerance rule with seed 0's output on the right */
                int close;
                if (bits_is_finite(b) && bits_is_finite(b0))
                    close = fabsf(x - x0) <= atol + (rtol * fabsf(x0));
                else
                    close = bits_is_inf(b) && b == b0;
                if (!close) within = 0;
            }
            if (x < lo) lo = x;
            if (x > hi) hi = x;
        }
        if (!all_finite) { n_nonfin++; continue; }
        const float d = hi - lo;                    /* one fp32 subtraction */
        if (d > spread) { spread = d; arg = i; }
    }
    memset(res, 0, sizeof *res);
    res->n_nonfinite = n_nonfin;
    res->argmax_spread = (S >= 2) ? arg : ORC_NO_INDEX;
    res->max_spread = (S >= 2) ? spread : -1.0f;
    uint32_t flags = 0;
    if (S >= 2 && identical) flags |= ORC_CROSS_IDENTICAL;
    if (S >= 2 && within) flags |= ORC_CROSS_WITHIN_TOL;
    if (S >= 2 && spread >= 0.0f && spread < spread_lim) flags |= ORC_CROSS_LOW_SPREAD;
    if (n_nonfin) flags |= ORC_CROSS_NONFINITE;
    res->flags = flags;
    return 0;
}

/* Which of the M input tensors (the operands a kernel receives: activations, weights,
 * the incoming gradient ...) is the candidate output a bit copy of?  Bit m of the result is
 * set iff every element of cand has the storage bits of inputs[m].  All tensors have n
 * elements of dtype. */
int orc_copy_of_inputs(const void *const *inputs, int M, const void *cand, uint64_t n, int dtype,
                       uint32_t *mask)
{
    if (!inputs || !cand || !mask || M < 1 || M > 32 || n < 1 || !dtype_known(dtype)) return -1;
    uint32_t m_out = 0;
    for (int m = 0; m < M; ++m) {
        if (!inputs[m]) return -1;
        int same = 1;
        for (uint64_t i = 0; i < n; ++i)
            if (load_bits(cand, dtype, i) != load_bits(inputs[m], dtype, i)) { same = 0; break; }
        if (same) m_out |= 1u << m;
    }
    *mask = m_out;
    return 0;
}
