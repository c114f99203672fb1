/*
 * CPU oracle for emulated 1/e/m floating-point training arithmetic.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow reference the CUDA library is
 * checked against.  It shares no code, header, table or helper with the CUDA path, and only
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * What it follows (arXiv 2103.15940):
 *   - Definition III.1, Eq. (1): a value is x = M * 2^(E-p+1) with E_min <= E <= E_max and an
 *     integer significand M; normal numbers have |x| >= 2^E_min, all others are denormal with
 *     E = E_min.
 *   - Definition III.2: a format is 1/e/m/d with e exponent bits, m stored mantissa bits, and
 *     "d" (denormals kept) or "n" (denormals flushed to zero).
 *   - Table I: bias 2^(e-1)-1 gives E_min = 1-bias, E_max = bias, smallest denormal
 *     2^(E_min-m).  The all-ones stored exponent field is reserved for inf/NaN and the
 *     all-zero field for zero/denormals (Section III's list of special encodings, read the
 *     IEEE way so that Table I's E_max stays the largest finite exponent).
 *   - Section IV-A: roundfp rounds each element to the nearest representable value
 *     (ties go to the even significand, the IEEE default), with e <= 8 and m <= 23.
 *   - Section II: loss scaling multiplies the tensors by a factor before they are rounded.
 *   - Section III-B: FMACS, a32 = round(a32 + x16*y16): exact products, wide accumulation.
 *     The contraction is order dependent in fp32, so the oracle gives the exact result
 *     (fp64 accumulation of exact products) together with sum |a||b| for the error bound.
 *   - Section III-B, FMAC, a16 = round(a16 + x16*y16), and Algorithm 1 (FMAC-8): the exact value
 *     of a + x*y is formed in integers and rounded once; the master accumulator adds in fp32.
 *   - Section IV-A: FMAC-8 also names a convolution whose sums are accumulated as in
 *     Algorithm 1; the order in which a convolution's reduction is walked is a reading, stated
 *     where oracle_conv_fmac8 is defined.
 *   - Section IV-A's layer formula Y = R(R(W^T X) + R(B)): exact sum of the two rounded
 *     terms, rounded once more.
 *   - Section V: "denormal fraction" of each tensor is the logged statistic.
 *
 * Every number here is handled as an integer significand times a power of two.
 *
 * Pins: tests/test_oracle_*.py (all "not gpu").  FTZ-mode variants and formats other than
 * 1/5/10, 1/8/7, 1/6/9 and 1/8/23 are pinned only by the brute-force invariants
 * ("parity unpinned" beyond those).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------ */
/* Format constants (Table I).                                                                  */
/* ------------------------------------------------------------------------------------------ */
int oracle_bias(int e) { return (1 << (e - 1)) - 1; }
int oracle_emax(int e) { return oracle_bias(e); }
int oracle_emin(int e) { return 1 - oracle_bias(e); }
/* exponents of two of the smallest normal / smallest denormal */
int oracle_min_normal_log2(int e) { return oracle_emin(e); }
int oracle_min_denormal_log2(int e, int m) { return oracle_emin(e) - m; }
/* largest normal = (2 - 2^-m) * 2^Emax, returned as a double (exact) */
double oracle_max_normal(int e, int m) { return ldexp(2.0 - ldexp(1.0, -m), oracle_emax(e)); }

/* ------------------------------------------------------------------------------------------ */
/* A finite nonnegative magnitude as  sig * 2^exp2  (sig a 64-bit integer).                     */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    uint64_t sig;
    int exp2;
} mag_t;

/* classes of an fp32 word */
enum { CLS_ZERO = 0, CLS_FINITE = 1, CLS_INF = 2, CLS_NAN = 3 };

/* Decode an fp32 bit pattern: sign, class, and for finite nonzero values sig*2^exp2 exactly. */
static int decode_f32(uint32_t u, int *sign, mag_t *mg) {
    uint32_t E = (u >> 23) & 0xFFu, f = u & 0x7FFFFFu;
    *sign = (int)(u >> 31);
    mg->sig = 0;
    mg->exp2 = 0;
    if (E == 255) return f ? CLS_NAN : CLS_INF;
    if (E == 0) {
        if (f == 0) return CLS_ZERO;
        mg->sig = f; /* fp32 denormal: f * 2^-149 */
        mg->exp2 = -149;
        return CLS_FINITE;
    }
    mg->sig = (uint64_t)f | 0x800000u; /* (2^23 + f) * 2^(E-150) */
    mg->exp2 = (int)E - 150;
    return CLS_FINITE;
}

static int floor_log2_u64(uint64_t v) { /* v > 0 */
    int b = -1;
    while (v) {
        v >>= 1;
        ++b;
    }
    return b;
}

/*
 * Round the exact magnitude sig*2^exp2 (sig > 0) to the nearest value of format (e, m) with
 * denormals, ties to even.  Result: Q * 2^g, where g is the exponent of the unit in the last
 * place that applies at this magnitude: g = max(floor(log2 v), E_min) - m.  Q may come out as
 * 2^(m+1) (carry into the next binade) or 0 (rounded to zero).  *is_inf is set when the rounded
 * value reaches 2^(E_max+1), i.e. exceeds the largest normal.
 */
static mag_t round_to_format(mag_t v, int e, int m, int *is_inf) {
    int emin = oracle_emin(e), emax = oracle_emax(e);
    int lg = floor_log2_u64(v.sig) + v.exp2;       /* floor(log2 value) */
    int g = (lg > emin ? lg : emin) - m;           /* quantum exponent */
    int r = g - v.exp2;                            /* bits to drop (may be <= 0: exact) */
    mag_t q;
    q.exp2 = g;
    *is_inf = 0;
    if (r <= 0) {
        q.sig = v.sig << (-r); /* already on the grid; callers keep sig small enough */
    } else if (r >= 64) {
        q.sig = 0; /* value is below a quarter of the quantum */
    } else {
        uint64_t keep = v.sig >> r;
        uint64_t rem = v.sig & (((uint64_t)1 << r) - 1);
        uint64_t half = (uint64_t)1 << (r - 1);
        if (rem > half || (rem == half && (keep & 1))) keep += 1;
        q.sig = keep;
    }
    if (q.sig != 0) {
        int top = floor_log2_u64(q.sig) + q.exp2;
        if (top > emax) *is_inf = 1;
    }
    return q;
}

/* Encode a finite magnitude Q*2^g (already a value of format (8,23) or coarser) as fp32 bits. */
static uint32_t encode_f32_mag(mag_t q) {
    if (q.sig == 0) return 0;
    int top = floor_log2_u64(q.sig);
    int lg = top + q.exp2;
    if (lg < -126) { /* fp32 denormal: multiple of 2^-149 */
        int sh = q.exp2 + 149;
        uint64_t f = sh >= 0 ? (q.sig << sh) : (q.sig >> (-sh));
        return (uint32_t)f;
    }
    uint64_t s24 = top >= 23 ? (q.sig >> (top - 23)) : (q.sig << (23 - top));
    return ((uint32_t)(lg + 127) << 23) | (uint32_t)(s24 & 0x7FFFFFu);
}

/* ------------------------------------------------------------------------------------------ */
/* Loss scale (Section II): y = fl32(x * S), IEEE single multiply, RNE, denormals honoured.     */
/* ------------------------------------------------------------------------------------------ */
uint32_t oracle_scale_bits(uint32_t xbits, uint32_t sbits) {
    int sx, ss;
    mag_t mx, ms;
    int cx = decode_f32(xbits, &sx, &mx), cs = decode_f32(sbits, &ss, &ms);
    uint32_t sign = (uint32_t)(sx ^ ss) << 31;
    if (cx == CLS_NAN || cs == CLS_NAN) return sign | 0x7FC00000u;
    if ((cx == CLS_INF && cs == CLS_ZERO) || (cx == CLS_ZERO && cs == CLS_INF)) return 0x7FC00000u;
    if (cx == CLS_INF || cs == CLS_INF) return sign | 0x7F800000u;
    if (cx == CLS_ZERO || cs == CLS_ZERO) return sign;
    mag_t p;
    p.sig = mx.sig * ms.sig; /* < 2^48, exact */
    p.exp2 = mx.exp2 + ms.exp2;
    int inf;
    mag_t q = round_to_format(p, 8, 23, &inf);
    if (inf) return sign | 0x7F800000u;
    return sign | encode_f32_mag(q);
}

/* ------------------------------------------------------------------------------------------ */
/* Quantize one fp32 word to 1/e/m (Section IV-A roundfp), result kept in an fp32 container.    */
/* *was_denormal: the rounded value, before any flush, is a nonzero denormal of the format.     */
/* ------------------------------------------------------------------------------------------ */
uint32_t oracle_quantize_bits(uint32_t ybits, int e, int m, int keep_denormals, int *was_denormal) {
    int s;
    mag_t v;
    int cls = decode_f32(ybits, &s, &v);
    uint32_t sign = (uint32_t)s << 31;
    if (was_denormal) *was_denormal = 0;
    if (cls == CLS_NAN) return sign | 0x7FC00000u;
    if (cls == CLS_INF) return sign | 0x7F800000u;
    if (cls == CLS_ZERO) return sign;
    int inf;
    mag_t q = round_to_format(v, e, m, &inf);
    if (inf) return sign | 0x7F800000u;
    if (q.sig == 0) return sign;
    /* below 2^E_min  <=>  Q < 2^m at the denormal quantum */
    int is_den = (floor_log2_u64(q.sig) + q.exp2) < oracle_emin(e);
    if (was_denormal) *was_denormal = is_den;
    if (is_den && !keep_denormals) return sign; /* flushed formats: denormals become zero */
    return sign | encode_f32_mag(q);
}

/* ------------------------------------------------------------------------------------------ */
/* Packed (1+e+m)-bit encodings: sign | stored exponent | mantissa (used for brute force).      */
/* ------------------------------------------------------------------------------------------ */
/* Value of a packed code as fp32 bits (Eq. (1) plus the special encodings). */
uint32_t oracle_decode_code(uint32_t code, int e, int m) {
    uint32_t sign = (code >> (e + m)) & 1u;
    uint32_t E = (code >> m) & ((1u << e) - 1u);
    uint32_t f = code & ((1u << m) - 1u);
    uint32_t sb = sign << 31;
    if (E == (1u << e) - 1u) return f ? (sb | 0x7FC00000u) : (sb | 0x7F800000u);
    mag_t q;
    if (E == 0) {
        q.sig = f;
        q.exp2 = oracle_emin(e) - m;
    } else {
        q.sig = ((uint64_t)1 << m) | f;
        q.exp2 = (int)E - oracle_bias(e) - m;
    }
    return sb | encode_f32_mag(q);
}

/* Packed code of an fp32 word that already holds a value of format (e, m). */
uint32_t oracle_encode_code(uint32_t qbits, int e, int m) {
    int s;
    mag_t v;
    int cls = decode_f32(qbits, &s, &v);
    uint32_t sb = (uint32_t)s << (e + m);
    uint32_t top = ((1u << e) - 1u) << m;
    if (cls == CLS_NAN) return sb | top | (1u << (m - 1));
    if (cls == CLS_INF) return sb | top;
    if (cls == CLS_ZERO) return sb;
    int lg = floor_log2_u64(v.sig) + v.exp2;
    int emin = oracle_emin(e);
    if (lg < emin) { /* denormal: mantissa = value / 2^(emin-m) */
        int sh = v.exp2 - (emin - m);
        uint64_t f = sh >= 0 ? (v.sig << sh) : (v.sig >> (-sh));
        return sb | (uint32_t)f;
    }
    int sh = v.exp2 - (lg - m);
    uint64_t sig = sh >= 0 ? (v.sig << sh) : (v.sig >> (-sh));
    return sb | ((uint32_t)(lg + oracle_bias(e)) << m) | (uint32_t)(sig & (((uint64_t)1 << m) - 1));
}

/* ------------------------------------------------------------------------------------------ */
/* Statistics record: 256 histogram bins followed by 8 counters (all 64-bit).                   */
/* ------------------------------------------------------------------------------------------ */
enum {
    ST_TOTAL = 256, ST_ZERO_IN, ST_DENORMAL, ST_UNDERFLOW, ST_OVERFLOW, ST_NAN, ST_INF_IN, ST_RESERVED,
    ST_WORDS
};

/* Stored exponent field of a quantized value: 0 zero/denormal, 1..2^e-2 normal, 2^e-1 inf/NaN. */
static int exponent_code(uint32_t qbits, int e) {
    int s;
    mag_t v;
    int cls = decode_f32(qbits, &s, &v);
    if (cls == CLS_NAN || cls == CLS_INF) return (1 << e) - 1;
    if (cls == CLS_ZERO) return 0;
    int lg = floor_log2_u64(v.sig) + v.exp2;
    if (lg < oracle_emin(e)) return 0;
    return lg + oracle_bias(e);
}

/*
 * Quantize n elements (after the loss-scale multiply) and count, one element at a time.
 * q may be NULL (statistics only); stats may be NULL.  stats[] is ADDED to (caller zeroes).
 */
void oracle_quantize_stats(const uint32_t *x, uint32_t *q, size_t n, int e, int m, int keep_denormals,
                           uint32_t scale_bits, uint64_t *stats) {
    for (size_t i = 0; i < n; ++i) {
        uint32_t xb = x[i];
        uint32_t yb = (scale_bits == 0x3F800000u) ? xb : oracle_scale_bits(xb, scale_bits);
        int was_den;
        uint32_t qb = oracle_quantize_bits(yb, e, m, keep_denormals, &was_den);
        if (q) q[i] = qb;
        if (!stats) continue;
        int sx;
        mag_t mx;
        int cx = decode_f32(xb, &sx, &mx);
        int q_zero = (qb & 0x7FFFFFFFu) == 0;
        int q_inf = (qb & 0x7FFFFFFFu) == 0x7F800000u;
        stats[exponent_code(qb, e)] += 1;
        stats[ST_TOTAL] += 1;
        if (cx == CLS_ZERO) stats[ST_ZERO_IN] += 1;
        if (cx == CLS_NAN) stats[ST_NAN] += 1;
        if (cx == CLS_INF) stats[ST_INF_IN] += 1;
        if (was_den) stats[ST_DENORMAL] += 1;
        if (cx == CLS_FINITE && q_zero) stats[ST_UNDERFLOW] += 1;
        if ((cx == CLS_FINITE || cx == CLS_ZERO) && q_inf) stats[ST_OVERFLOW] += 1;
    }
}

/*
 * The same over `threads` host threads: the tensor is cut into that many contiguous pieces, each
 * piece is handled by oracle_quantize_stats with a record of its own, and the records are summed
 * at the end (elements are independent and counts add).  For timing the oracle on all cores.
 */
void oracle_quantize_stats_threads(const uint32_t *x, uint32_t *q, size_t n, int e, int m, int keep_denormals,
                                   uint32_t scale_bits, uint64_t *stats, int threads) {
    if (threads < 1) threads = 1;
#pragma omp parallel for schedule(static) num_threads(threads)
    for (int t = 0; t < threads; ++t) {
        size_t lo = n / (size_t)threads * (size_t)t, hi = (t == threads - 1) ? n : n / (size_t)threads * (size_t)(t + 1);
        uint64_t local[ST_WORDS];
        memset(local, 0, sizeof local);
        oracle_quantize_stats(x + lo, q ? q + lo : NULL, hi - lo, e, m, keep_denormals, scale_bits,
                              stats ? local : NULL);
        if (stats) {
#pragma omp critical
            for (int w = 0; w < ST_WORDS; ++w) stats[w] += local[w];
        }
    }
}

/* ------------------------------------------------------------------------------------------ */
/* 16-bit storage (Section II: activations and gradients are kept in half precision, halving     */
/* storage and bandwidth): a tensor is rounded as oracle_quantize_stats does and each value is    */
/* stored as its packed code, sign | stored exponent | mantissa (1 + e + m <= 16 bits, in the     */
/* low bits of a 16-bit word); unpacking returns the fp32 containers.                             */
/* ------------------------------------------------------------------------------------------ */
void oracle_quantize_stats_pack16(const uint32_t *x, uint16_t *codes, size_t n, int e, int m, int keep_denormals,
                                  uint32_t scale_bits, uint64_t *stats) {
    for (size_t i = 0; i < n; ++i) {
        uint32_t q;
        oracle_quantize_stats(&x[i], &q, 1, e, m, keep_denormals, scale_bits, stats);
        codes[i] = (uint16_t)oracle_encode_code(q, e, m);
    }
}

void oracle_unpack16(const uint16_t *codes, uint32_t *q, size_t n, int e, int m) {
    for (size_t i = 0; i < n; ++i) q[i] = oracle_decode_code(codes[i], e, m);
}

/* ------------------------------------------------------------------------------------------ */
/* Exact signed sums, rounded once.                                                             */
/*                                                                                              */
/* Both FMAC (Section III-B: a16 = round(a16 + x16*y16), one rounding of the exact value) and   */
/* the layer formula of Section IV-A, Y = R(R(W^T X) + R(B)), need the exact sum of two finite  */
/* numbers rounded once to a format.  A number is sign, sig * 2^exp2.                           */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    int cls;  /* CLS_ZERO, CLS_FINITE, CLS_INF, CLS_NAN */
    int sign; /* 1 = negative */
    mag_t mg; /* for CLS_FINITE */
} num_t;

static num_t num_from_f32(uint32_t u) {
    num_t r;
    r.cls = decode_f32(u, &r.sign, &r.mg);
    return r;
}

static mag_t strip_zeros(mag_t v) {
    while (v.sig != 0 && (v.sig & 1u) == 0) {
        v.sig >>= 1;
        v.exp2 += 1;
    }
    return v;
}

/*
 * Exact a + b for finite nonzero a, b whose significands, trailing zeros removed, are at most
 * 24 bits wide.  The result is returned as sign and magnitude such that ROUNDING it to any
 * format with m <= 23 (or comparing it with zero) gives what the exact sum would give:
 * when the two numbers are within 38 binary places of each other the sum is formed exactly in
 * 64-bit integers; when they are further apart the smaller one lies more than 14 places below
 * the last bit of the larger, it cannot reach any grid point or halfway point of the result's
 * neighbourhood, and it is replaced by one unit 38 places below the larger one's last bit,
 * which lies strictly on the same side of all those points.
 * Returns CLS_ZERO for an exact cancellation.
 */
static int exact_sum(int sa, mag_t a, int sb, mag_t b, int *sign, mag_t *out) {
    a = strip_zeros(a);
    b = strip_zeros(b);
    int ta = floor_log2_u64(a.sig) + a.exp2, tb = floor_log2_u64(b.sig) + b.exp2;
    if (tb > ta) { /* make a the one that reaches higher */
        mag_t tm = a; a = b; b = tm;
        int ts = sa; sa = sb; sb = ts;
        int tt = ta; ta = tb; tb = tt;
    }
    int lo = a.exp2 < b.exp2 ? a.exp2 : b.exp2;
    uint64_t A, B;
    if (ta - lo <= 61) {
        A = a.sig << (a.exp2 - lo);
        B = b.sig << (b.exp2 - lo);
    } else { /* b far below a: only its presence and sign matter */
        A = a.sig << 38;
        B = 1;
        lo = a.exp2 - 38;
    }
    out->exp2 = lo;
    if (sa == sb) {
        out->sig = A + B;
        *sign = sa;
        return CLS_FINITE;
    }
    if (A == B) {
        out->sig = 0;
        *sign = 0;
        return CLS_ZERO;
    }
    if (A > B) {
        out->sig = A - B;
        *sign = sa;
    } else {
        out->sig = B - A;
        *sign = sb;
    }
    return CLS_FINITE;
}

/* IEEE rules for a sum whose operands are not both finite and nonzero; returns 1 if *r is set. */
static int special_sum(num_t a, num_t b, num_t *r) {
    r->mg.sig = 0;
    r->mg.exp2 = 0;
    if (a.cls == CLS_NAN || b.cls == CLS_NAN || (a.cls == CLS_INF && b.cls == CLS_INF && a.sign != b.sign)) {
        r->cls = CLS_NAN; /* the positive quiet NaN stands for every invalid or propagated NaN */
        r->sign = 0;
        return 1;
    }
    if (a.cls == CLS_INF) { *r = a; return 1; }
    if (b.cls == CLS_INF) { *r = b; return 1; }
    if (a.cls == CLS_ZERO && b.cls == CLS_ZERO) {
        r->cls = CLS_ZERO;
        r->sign = a.sign & b.sign; /* -0 only when both are -0 (round to nearest) */
        return 1;
    }
    if (a.cls == CLS_ZERO) { *r = b; return 1; }
    if (b.cls == CLS_ZERO) { *r = a; return 1; }
    return 0;
}

/* a + b, exact in the sense of exact_sum */
static num_t num_add(num_t a, num_t b) {
    num_t r;
    if (special_sum(a, b, &r)) return r;
    r.cls = exact_sum(a.sign, a.mg, b.sign, b.mg, &r.sign, &r.mg);
    return r;
}

/* exact product */
static num_t num_mul(num_t x, num_t y) {
    num_t r;
    r.sign = x.sign ^ y.sign;
    r.mg.sig = 0;
    r.mg.exp2 = 0;
    if (x.cls == CLS_NAN || y.cls == CLS_NAN || (x.cls == CLS_INF && y.cls == CLS_ZERO) ||
        (x.cls == CLS_ZERO && y.cls == CLS_INF)) {
        r.cls = CLS_NAN;
        r.sign = 0;
    } else if (x.cls == CLS_INF || y.cls == CLS_INF) {
        r.cls = CLS_INF;
    } else if (x.cls == CLS_ZERO || y.cls == CLS_ZERO) {
        r.cls = CLS_ZERO;
    } else {
        r.cls = CLS_FINITE;
        r.mg.sig = x.mg.sig * y.mg.sig; /* < 2^48 */
        r.mg.exp2 = x.mg.exp2 + y.mg.exp2;
    }
    return r;
}

/*
 * Round a number to format (e, m): fp32 container bits.  Same rules as oracle_quantize_bits
 * (overflow to inf, sign kept on zeros, flush after rounding when denormals are off).
 */
static uint32_t num_round_bits(num_t v, int e, int m, int keep_denormals, int *was_denormal) {
    uint32_t sign = (uint32_t)v.sign << 31;
    if (was_denormal) *was_denormal = 0;
    if (v.cls == CLS_NAN) return sign | 0x7FC00000u;
    if (v.cls == CLS_INF) return sign | 0x7F800000u;
    if (v.cls == CLS_ZERO) return sign;
    int inf;
    mag_t q = round_to_format(v.mg, e, m, &inf);
    if (inf) return sign | 0x7F800000u;
    if (q.sig == 0) return sign;
    int is_den = (floor_log2_u64(q.sig) + q.exp2) < oracle_emin(e);
    if (was_denormal) *was_denormal = is_den;
    if (is_den && !keep_denormals) return sign;
    return sign | encode_f32_mag(q);
}

/* round(a + b) to (e, m) for two fp32 words (their trailing-zero-free significands fit 24 bits). */
uint32_t oracle_add_round_bits(uint32_t abits, uint32_t bbits, int e, int m, int keep_denormals) {
    return num_round_bits(num_add(num_from_f32(abits), num_from_f32(bbits)), e, m, keep_denormals, NULL);
}

/*
 * FMAC (Section III-B): round(a + x*y) to (e, m) with ONE rounding of the exact value.
 * x and y must hold values with at most 12 significant bits each (any format with m <= 11),
 * so that the product's significand fits 24 bits.
 */
uint32_t oracle_fmac_bits(uint32_t abits, uint32_t xbits, uint32_t ybits, int e, int m, int keep_denormals) {
    num_t p = num_mul(num_from_f32(xbits), num_from_f32(ybits));
    if (p.cls == CLS_FINITE) p.mg = strip_zeros(p.mg);
    return num_round_bits(num_add(num_from_f32(abits), p), e, m, keep_denormals, NULL);
}

/*
 * Layer output of Section IV-A's worked example, Y = R(R(acc) + R(B)): acc is the matrix
 * product (rows x cols, leading dimension ld_acc), bias has one entry per column.  Both are
 * multiplied by the loss scale and rounded as oracle_quantize_stats does, added exactly and
 * rounded once more.  Statistics describe the OUTPUT tensor, with the exact sum in the role of
 * the input: n_zero_in counts sums that are zero, n_underflow nonzero sums that end as zero,
 * n_overflow finite sums that end as inf, n_inf_in / n_nan infinite / NaN sums.
 * bias may be NULL (then Y = R(acc), statistics as in oracle_quantize_stats).
 * stats[] is ADDED to; out may be NULL.
 */
void oracle_bias_quantize_stats(const uint32_t *acc, int64_t rows, int64_t cols, int64_t ld_acc,
                                const uint32_t *bias, uint32_t *out, int64_t ld_out, int e, int m,
                                int keep_denormals, uint32_t scale_bits, uint64_t *stats) {
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            uint32_t xb = acc[i * ld_acc + j];
            uint32_t yb = (scale_bits == 0x3F800000u) ? xb : oracle_scale_bits(xb, scale_bits);
            num_t s;
            if (bias) {
                uint32_t ra = oracle_quantize_bits(yb, e, m, keep_denormals, NULL);
                uint32_t bb = (scale_bits == 0x3F800000u) ? bias[j] : oracle_scale_bits(bias[j], scale_bits);
                uint32_t rb = oracle_quantize_bits(bb, e, m, keep_denormals, NULL);
                s = num_add(num_from_f32(ra), num_from_f32(rb));
            } else {
                s = num_from_f32(yb);
                if (s.cls == CLS_NAN) s.sign = (int)(xb >> 31);
            }
            int was_den;
            uint32_t qb = num_round_bits(s, e, m, keep_denormals, &was_den);
            if (out) out[i * ld_out + j] = qb;
            if (!stats) continue;
            int q_zero = (qb & 0x7FFFFFFFu) == 0;
            int q_inf = (qb & 0x7FFFFFFFu) == 0x7F800000u;
            int in_cls = s.cls;
            if (!bias) { /* as oracle_quantize_stats: classes of the unscaled input */
                int sx;
                mag_t mx;
                in_cls = decode_f32(xb, &sx, &mx);
            }
            stats[exponent_code(qb, e)] += 1;
            stats[ST_TOTAL] += 1;
            if (in_cls == CLS_ZERO) stats[ST_ZERO_IN] += 1;
            if (in_cls == CLS_NAN) stats[ST_NAN] += 1;
            if (in_cls == CLS_INF) stats[ST_INF_IN] += 1;
            if (was_den) stats[ST_DENORMAL] += 1;
            if (in_cls == CLS_FINITE && q_zero) stats[ST_UNDERFLOW] += 1;
            if ((in_cls == CLS_FINITE || in_cls == CLS_ZERO) && q_inf) stats[ST_OVERFLOW] += 1;
        }
}

/* ------------------------------------------------------------------------------------------ */
/* Dynamic loss scaling (Sections II and V use it; the paper cites the method and gives no        */
/* algorithm).  Rule taken: after a step whose gradient tensors held any overflow, infinity or    */
/* NaN the step is skipped, the scale is multiplied by `backoff` (not below min_scale) and the    */
/* count of clean steps restarts; otherwise the count grows, and when it reaches growth_interval   */
/* the scale is multiplied by `growth` (not above max_scale) and the count restarts.               */
/* The products are fp32 multiplications.                                                          */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    float scale, growth, backoff, min_scale, max_scale;
    int32_t growth_interval, clean_steps, skip, reserved;
    uint64_t n_steps, n_skipped;
} dls_t;

void oracle_dls_update(dls_t *st, const uint64_t *stats, int64_t n_records) {
    uint64_t bad = 0;
    for (int64_t r = 0; r < n_records; ++r) {
        const uint64_t *rec = stats + r * ST_WORDS;
        bad += rec[ST_OVERFLOW] + rec[ST_NAN] + rec[ST_INF_IN];
    }
    st->n_steps += 1;
    if (bad != 0) {
        float s = st->scale * st->backoff;
        st->scale = s < st->min_scale ? st->min_scale : s;
        st->clean_steps = 0;
        st->skip = 1;
        st->n_skipped += 1;
    } else {
        st->skip = 0;
        st->clean_steps += 1;
        if (st->clean_steps >= st->growth_interval) {
            float s = st->scale * st->growth;
            st->scale = s > st->max_scale ? st->max_scale : s;
            st->clean_steps = 0;
        }
    }
}

/* ------------------------------------------------------------------------------------------ */
/* Contractions (Section III-B, FMACS): exact products summed in fp64 in plain k order, with    */
/* t = sum |a||b| beside each output for the accumulation-error bound.                          */
/* Matrices are fp32, row-major with a leading dimension; trans != 0 reads the stored matrix    */
/* transposed, so op(A) is M x K and op(B) is K x N.                                            */
/* ------------------------------------------------------------------------------------------ */
static double elemA(const float *A, int64_t lda, int transA, int64_t i, int64_t k) {
    return transA ? (double)A[k * lda + i] : (double)A[i * lda + k];
}
static double elemB(const float *B, int64_t ldb, int transB, int64_t k, int64_t j) {
    return transB ? (double)B[j * ldb + k] : (double)B[k * ldb + j];
}

static void dot_ab(const float *A, int64_t lda, int transA, const float *B, int64_t ldb, int transB,
                   int64_t K, int64_t i, int64_t j, double *c, double *t) {
    double acc = 0.0, abs_acc = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        double a = elemA(A, lda, transA, i, k), b = elemB(B, ldb, transB, k, j);
        acc += a * b;
        abs_acc += fabs(a) * fabs(b);
    }
    *c = acc;
    if (t) *t = abs_acc;
}

/* Full output: C and T are M x N fp64, dense row-major.  T may be NULL. */
void oracle_gemm(const float *A, int64_t lda, int transA, const float *B, int64_t ldb, int transB,
                 int64_t M, int64_t N, int64_t K, double *C, double *T) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j)
            dot_ab(A, lda, transA, B, ldb, transB, K, i, j, &C[i * N + j], T ? &T[i * N + j] : NULL);
}

/* Sampled outputs: c[s], t[s] for the pairs (ii[s], jj[s]). */
void oracle_gemm_sampled(const float *A, int64_t lda, int transA, const float *B, int64_t ldb, int transB,
                         int64_t K, const int64_t *ii, const int64_t *jj, int64_t nsamp, double *c,
                         double *t) {
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsamp; ++s)
        dot_ab(A, lda, transA, B, ldb, transB, K, ii[s], jj[s], &c[s], t ? &t[s] : NULL);
}

/* ------------------------------------------------------------------------------------------ */
/* FMAC-8 (Algorithm 1).  A dot product is cut, from its start, into runs of `group` consecutive  */
/* terms (8 in the paper; the last run may be shorter).  Each run is summed by fused multiply-    */
/* accumulates into an accumulator of the 16-bit format that starts at zero, every FMAC rounding   */
/* its exact a + x*y once to the format; the finished run sum is then added, in fp32 arithmetic,  */
/* to a single-precision total that also starts at zero.  The total is rounded to the format at   */
/* the end.  An empty dot product gives R(+0).                                                     */
/* ------------------------------------------------------------------------------------------ */
static uint32_t f32_add_bits(uint32_t a, uint32_t b) { return oracle_add_round_bits(a, b, 8, 23, 1); }

static uint32_t word_of(float v) {
    uint32_t w;
    memcpy(&w, &v, 4);
    return w;
}

static uint32_t fmac8_dot(const float *A, int64_t lda, int transA, const float *B, int64_t ldb, int transB,
                          int64_t K, int64_t i, int64_t j, int e, int m, int keep_denormals, int group,
                          uint32_t *total_out) {
    uint32_t total = 0; /* fp32 word of +0 */
    for (int64_t first = 0; first < K; first += group) {
        const int64_t end = first + group < K ? first + group : K;
        uint32_t run_sum = 0; /* format value +0, kept as its fp32 word */
        for (int64_t k = first; k < end; ++k) {
            const float x = transA ? A[k * lda + i] : A[i * lda + k];
            const float y = transB ? B[j * ldb + k] : B[k * ldb + j];
            run_sum = oracle_fmac_bits(run_sum, word_of(x), word_of(y), e, m, keep_denormals);
        }
        total = f32_add_bits(total, run_sum);
    }
    if (total_out) *total_out = total; /* the single-precision total before the final rounding */
    return oracle_quantize_bits(total, e, m, keep_denormals, NULL);
}

/* C (M x N, dense row-major fp32 words) = FMAC-8 product of op(A) (M x K) and op(B) (K x N).   */
/* group is the number of consecutive FMACs (8 in the paper).  master (may be NULL) receives     */
/* the master accumulators before the final rounding.                                           */
void oracle_fmac8_gemm(const float *A, int64_t lda, int transA, const float *B, int64_t ldb, int transB,
                       int64_t M, int64_t N, int64_t K, int e, int m, int keep_denormals, int group,
                       uint32_t *C, uint32_t *master) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j)
            C[i * N + j] = fmac8_dot(A, lda, transA, B, ldb, transB, K, i, j, e, m, keep_denormals, group,
                                     master ? &master[i * N + j] : NULL);
}

void oracle_fmac8_gemm_sampled(const float *A, int64_t lda, int transA, const float *B, int64_t ldb, int transB,
                               int64_t K, int e, int m, int keep_denormals, int group, const int64_t *ii,
                               const int64_t *jj, int64_t nsamp, uint32_t *c) {
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsamp; ++s)
        c[s] = fmac8_dot(A, lda, transA, B, ldb, transB, K, ii[s], jj[s], e, m, keep_denormals, group, NULL);
}

/* ------------------------------------------------------------------------------------------ */
/* Convolution layers (Section V: the matrix multiplies at the core of convolution layers),     */
/* written as the direct definition on NCHW tensors: unit stride, zero padding, cross-          */
/* correlation as deep-learning frameworks define it.                                            */
/*   X [n][ci][h][w],  W [co][ci][r][s],  Y [n][co][oh][ow],  oh = h + 2*pad_h - r + 1.          */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    int64_t n, ci, h, w, co, r, s, pad_h, pad_w;
} conv_t;

static int64_t conv_oh(const conv_t *g) { return g->h + 2 * g->pad_h - g->r + 1; }
static int64_t conv_ow(const conv_t *g) { return g->w + 2 * g->pad_w - g->s + 1; }

/* forward: Y[n,co,oh,ow] = sum_{ci,r,s} X[n,ci,oh+r-pad,ow+s-pad] * W[co,ci,r,s] */
static void conv_fwd_one(const conv_t *g, const float *X, const float *Wt, int64_t n, int64_t co,
                         int64_t oh, int64_t ow, double *c, double *t) {
    double acc = 0.0, abs_acc = 0.0;
    for (int64_t ci = 0; ci < g->ci; ++ci)
        for (int64_t r = 0; r < g->r; ++r)
            for (int64_t s = 0; s < g->s; ++s) {
                int64_t ih = oh + r - g->pad_h, iw = ow + s - g->pad_w;
                if (ih < 0 || ih >= g->h || iw < 0 || iw >= g->w) continue;
                double a = X[((n * g->ci + ci) * g->h + ih) * g->w + iw];
                double b = Wt[((co * g->ci + ci) * g->r + r) * g->s + s];
                acc += a * b;
                abs_acc += fabs(a) * fabs(b);
            }
    *c = acc;
    if (t) *t = abs_acc;
}

/* data gradient: dX[n,ci,ih,iw] = sum_{co,r,s} dY[n,co,ih-r+pad,iw-s+pad] * W[co,ci,r,s] */
static void conv_dgrad_one(const conv_t *g, const float *dY, const float *Wt, int64_t n, int64_t ci,
                           int64_t ih, int64_t iw, double *c, double *t) {
    int64_t OH = conv_oh(g), OW = conv_ow(g);
    double acc = 0.0, abs_acc = 0.0;
    for (int64_t co = 0; co < g->co; ++co)
        for (int64_t r = 0; r < g->r; ++r)
            for (int64_t s = 0; s < g->s; ++s) {
                int64_t oh = ih - r + g->pad_h, ow = iw - s + g->pad_w;
                if (oh < 0 || oh >= OH || ow < 0 || ow >= OW) continue;
                double a = dY[((n * g->co + co) * OH + oh) * OW + ow];
                double b = Wt[((co * g->ci + ci) * g->r + r) * g->s + s];
                acc += a * b;
                abs_acc += fabs(a) * fabs(b);
            }
    *c = acc;
    if (t) *t = abs_acc;
}

/* filter gradient: dW[co,ci,r,s] = sum_{n,oh,ow} dY[n,co,oh,ow] * X[n,ci,oh+r-pad,ow+s-pad] */
static void conv_wgrad_one(const conv_t *g, const float *dY, const float *X, int64_t co, int64_t ci,
                           int64_t r, int64_t s, double *c, double *t) {
    int64_t OH = conv_oh(g), OW = conv_ow(g);
    double acc = 0.0, abs_acc = 0.0;
    for (int64_t n = 0; n < g->n; ++n)
        for (int64_t oh = 0; oh < OH; ++oh)
            for (int64_t ow = 0; ow < OW; ++ow) {
                int64_t ih = oh + r - g->pad_h, iw = ow + s - g->pad_w;
                if (ih < 0 || ih >= g->h || iw < 0 || iw >= g->w) continue;
                double a = dY[((n * g->co + co) * OH + oh) * OW + ow];
                double b = X[((n * g->ci + ci) * g->h + ih) * g->w + iw];
                acc += a * b;
                abs_acc += fabs(a) * fabs(b);
            }
    *c = acc;
    if (t) *t = abs_acc;
}

/*
 * which: 0 forward (output index space [n][co][oh][ow]), 1 data gradient ([n][ci][h][w]),
 * 2 filter gradient ([co][ci][r][s]).  P and Q are the two operands in the order of the
 * formulas above: (X, W), (dY, W), (dY, X).  idx holds flat indices into the output tensor;
 * idx == NULL means all outputs 0..count-1.
 */
void oracle_conv(int which, const int64_t *geom, const float *P, const float *Q, const int64_t *idx,
                 int64_t count, double *c, double *t) {
    conv_t g;
    g.n = geom[0]; g.ci = geom[1]; g.h = geom[2]; g.w = geom[3]; g.co = geom[4];
    g.r = geom[5]; g.s = geom[6]; g.pad_h = geom[7]; g.pad_w = geom[8];
    int64_t OH = conv_oh(&g), OW = conv_ow(&g);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < count; ++k) {
        int64_t f = idx ? idx[k] : k;
        double *tk = t ? &t[k] : NULL;
        if (which == 0) {
            int64_t ow = f % OW, oh = (f / OW) % OH, co = (f / (OW * OH)) % g.co, n = f / (OW * OH * g.co);
            conv_fwd_one(&g, P, Q, n, co, oh, ow, &c[k], tk);
        } else if (which == 1) {
            int64_t iw = f % g.w, ih = (f / g.w) % g.h, ci = (f / (g.w * g.h)) % g.ci, n = f / (g.w * g.h * g.ci);
            conv_dgrad_one(&g, P, Q, n, ci, ih, iw, &c[k], tk);
        } else {
            int64_t s = f % g.s, r = (f / g.s) % g.r, ci = (f / (g.s * g.r)) % g.ci, co = f / (g.s * g.r * g.ci);
            conv_wgrad_one(&g, P, Q, co, ci, r, s, &c[k], tk);
        }
    }
}

/* ------------------------------------------------------------------------------------------ */
/* FMAC-8 for convolution layers.  Section IV-A counts as FMAC-8 "a matrix multiplication or    */
/* convolution" whose sums are accumulated as in Algorithm 1: runs of `group` fused multiply-    */
/* accumulates in the 16-bit format, each run's sum added in fp32 to a single-precision total,   */
/* one rounding of the total at the end.  The paper does not say in which order a convolution's  */
/* reduction index is walked; the reading taken here (the order of an unfolded, channels-last   */
/* operand matrix):                                                                              */
/*   forward          filter taps row by row (r, then s), within a tap the input channels        */
/*   data gradient    filter taps row by row (r, then s), within a tap the output channels       */
/*   filter gradient  images, within an image the output rows, within a row the output pixels    */
/* A term whose input position lies in the zero padding is a term with a zero factor: it keeps   */
/* its place in its run (an FMAC with a zero factor leaves the accumulator as it is).            */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    uint32_t total;   /* fp32 word of the single-precision total */
    uint32_t run_sum; /* the 16-bit accumulator, as the fp32 word of its value */
    int in_run, group, e, m, keep;
} fmac8_state;

static void fmac8_begin(fmac8_state *st, int e, int m, int keep, int group) {
    st->total = 0; st->run_sum = 0; st->in_run = 0;
    st->group = group; st->e = e; st->m = m; st->keep = keep;
}
static void fmac8_term(fmac8_state *st, float x, float y) {
    st->run_sum = oracle_fmac_bits(st->run_sum, word_of(x), word_of(y), st->e, st->m, st->keep);
    if (++st->in_run == st->group) {
        st->total = f32_add_bits(st->total, st->run_sum);
        st->run_sum = 0;
        st->in_run = 0;
    }
}
static uint32_t fmac8_end(fmac8_state *st, uint32_t *total_out) {
    if (st->in_run > 0) st->total = f32_add_bits(st->total, st->run_sum);
    if (total_out) *total_out = st->total; /* the single-precision total before the final rounding */
    return oracle_quantize_bits(st->total, st->e, st->m, st->keep, NULL);
}

static uint32_t conv_fmac8_fwd_one(const conv_t *g, const float *X, const float *Wt, int64_t n, int64_t co,
                                   int64_t oh, int64_t ow, int e, int m, int keep, int group, uint32_t *total_out) {
    fmac8_state st;
    fmac8_begin(&st, e, m, keep, group);
    for (int64_t r = 0; r < g->r; ++r)
        for (int64_t s = 0; s < g->s; ++s)
            for (int64_t ci = 0; ci < g->ci; ++ci) {
                int64_t ih = oh + r - g->pad_h, iw = ow + s - g->pad_w;
                int inside = ih >= 0 && ih < g->h && iw >= 0 && iw < g->w;
                float x = inside ? X[((n * g->ci + ci) * g->h + ih) * g->w + iw] : 0.0f;
                fmac8_term(&st, x, Wt[((co * g->ci + ci) * g->r + r) * g->s + s]);
            }
    return fmac8_end(&st, total_out);
}

static uint32_t conv_fmac8_dgrad_one(const conv_t *g, const float *dY, const float *Wt, int64_t n, int64_t ci,
                                     int64_t ih, int64_t iw, int e, int m, int keep, int group, uint32_t *total_out) {
    int64_t OH = conv_oh(g), OW = conv_ow(g);
    fmac8_state st;
    fmac8_begin(&st, e, m, keep, group);
    for (int64_t r = 0; r < g->r; ++r)
        for (int64_t s = 0; s < g->s; ++s)
            for (int64_t co = 0; co < g->co; ++co) {
                int64_t oh = ih - r + g->pad_h, ow = iw - s + g->pad_w;
                int inside = oh >= 0 && oh < OH && ow >= 0 && ow < OW;
                float x = inside ? dY[((n * g->co + co) * OH + oh) * OW + ow] : 0.0f;
                fmac8_term(&st, x, Wt[((co * g->ci + ci) * g->r + r) * g->s + s]);
            }
    return fmac8_end(&st, total_out);
}

static uint32_t conv_fmac8_wgrad_one(const conv_t *g, const float *dY, const float *X, int64_t co, int64_t ci,
                                     int64_t r, int64_t s, int e, int m, int keep, int group, uint32_t *total_out) {
    int64_t OH = conv_oh(g), OW = conv_ow(g);
    fmac8_state st;
    fmac8_begin(&st, e, m, keep, group);
    for (int64_t n = 0; n < g->n; ++n)
        for (int64_t oh = 0; oh < OH; ++oh)
            for (int64_t ow = 0; ow < OW; ++ow) {
                int64_t ih = oh + r - g->pad_h, iw = ow + s - g->pad_w;
                int inside = ih >= 0 && ih < g->h && iw >= 0 && iw < g->w;
                float y = inside ? X[((n * g->ci + ci) * g->h + ih) * g->w + iw] : 0.0f;
                fmac8_term(&st, dY[((n * g->co + co) * OH + oh) * OW + ow], y);
            }
    return fmac8_end(&st, total_out);
}

/* Same index conventions as oracle_conv; out receives the fp32 words of the rounded results and     */
/* master (may be NULL) those of the single-precision totals before the final rounding.              */
void oracle_conv_fmac8(int which, const int64_t *geom, const float *P, const float *Q, int e, int m,
                       int keep_denormals, int group, const int64_t *idx, int64_t count, uint32_t *out,
                       uint32_t *master) {
    conv_t g;
    g.n = geom[0]; g.ci = geom[1]; g.h = geom[2]; g.w = geom[3]; g.co = geom[4];
    g.r = geom[5]; g.s = geom[6]; g.pad_h = geom[7]; g.pad_w = geom[8];
    int64_t OH = conv_oh(&g), OW = conv_ow(&g);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < count; ++k) {
        int64_t f = idx ? idx[k] : k;
        if (which == 0) {
            int64_t ow = f % OW, oh = (f / OW) % OH, co = (f / (OW * OH)) % g.co, n = f / (OW * OH * g.co);
            out[k] = conv_fmac8_fwd_one(&g, P, Q, n, co, oh, ow, e, m, keep_denormals, group, master ? &master[k] : NULL);
        } else if (which == 1) {
            int64_t iw = f % g.w, ih = (f / g.w) % g.h, ci = (f / (g.w * g.h)) % g.ci, n = f / (g.w * g.h * g.ci);
            out[k] = conv_fmac8_dgrad_one(&g, P, Q, n, ci, ih, iw, e, m, keep_denormals, group, master ? &master[k] : NULL);
        } else {
            int64_t s = f % g.s, r = (f / g.s) % g.r, ci = (f / (g.s * g.r)) % g.ci, co = f / (g.s * g.r * g.ci);
            out[k] = conv_fmac8_wgrad_one(&g, P, Q, co, ci, r, s, e, m, keep_denormals, group, master ? &master[k] : NULL);
        }
    }
}
