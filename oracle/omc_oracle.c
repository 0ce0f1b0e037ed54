/*
 * CPU oracle for Online Model Compression (OMC, arXiv 2205.03494).
 *
 * TEST INFRASTRUCTURE ONLY.  A plain, slow, scalar restatement of what the method computes,
 * written from the paper's text.  It shares no code with the CUDA library and must never be on a
 * product path: only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Everything here is value arithmetic (frexp / ldexp / nearbyint / fmaf, exact summation); there
 * are no bit tricks except where a NaN payload has to be placed, which no value operation can do.
 * Compile with -O2 -ffp-contract=off so that no multiply-add is fused behind the source's back.
 *
 * What follows the paper and what is a reading of it (the paper is silent on the encoding details):
 *   Sec. 2.2  floating-point quantisation SxEyMz: fewer exponent and mantissa bits than FP32.
 *             Reading: IEEE-754 interchange parametrisation (bias 2^(E-1)-1, gradual underflow,
 *             top exponent field = Inf/NaN) -- the one rule for which S1E8M23 is FP32 and S1E5M10
 *             is FP16, the two formats the paper names by their IEEE names (Sec. 2.2, Sec. 3.4).
 *             Rounding: to nearest, ties to even.
 *   Sec. 2.3  per-variable transformation: Vbar = s*Vtilde + b with (s, b) the least-squares
 *             minimiser of ||s*Vtilde + b*1 - V||_2; degenerate case s = 1; fp64 compute, fp32
 *             storage.  The closed forms printed in Sec. 2.3 are misprinted (they do not satisfy
 *             the normal equations of the minimisation stated beside them: a lossless code would
 *             not give s = 1, b = 0); the forms used here are the normal-equation solution.
 *   Sec. 2.1  update path: decompress, apply the gradient, compress again, discard.
 *   Sec. 2.4 / 2.5 / 3.1  weight matrices only; a random subset (fraction p) of them.
 *
 * Functions with no pin in the paper beyond their definition are marked "parity unpinned" below.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------ */
/* Format helpers (Sec. 2.2; notation SxEyMz from Sec. 3.1).  Only S = 1 exists in the paper.   */

static int fmt_bias(int E) { return (1 << (E - 1)) - 1; }
static int fmt_emin(int E) { return 1 - fmt_bias(E); }
static int fmt_emax(int E) { return fmt_bias(E); }

int orc_format_ok(int E, int M) { return E >= 2 && E <= 8 && M >= 0 && M <= 23; }

static uint32_t f32_bits(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }
static float bits_f32(uint32_t u) { float x; memcpy(&x, &u, 4); return x; }

/*
 * Sec. 2.2: decode one B-bit code (sign | exponent field | mantissa field) to its value.
 * Every SxEyMz value with E <= 8, M <= 23 is an FP32 value, so the returned float is exact.
 * NaN: the M mantissa bits go to the top of the FP32 mantissa (payload kept).
 */
float orc_decode(uint32_t code, int E, int M)
{
    const uint32_t sigma = (code >> (E + M)) & 1u;
    const uint32_t f = (code >> M) & ((1u << E) - 1u);
    const uint32_t m = code & ((1u << M) - 1u);
    const uint32_t fmax = (1u << E) - 1u;
    double mag;
    if (f == fmax) {
        if (m == 0) return sigma ? -INFINITY : INFINITY;
        return bits_f32((sigma << 31) | 0x7F800000u | (m << (23 - M)));
    }
    if (f == 0)
        mag = ldexp((double)m, fmt_emin(E) - M);                       /* zero / subnormal */
    else
        mag = ldexp(1.0 + ldexp((double)m, -M), (int)f - fmt_bias(E)); /* normal           */
    return sigma ? -(float)mag : (float)mag;
}

/*
 * Sec. 2.2: quantise one FP32 value to the nearest SxEyMz value (ties to even), gradual
 * underflow, overflow to infinity; returns the code.  Tie rule and specials are a reading of the
 * paper ("parity unpinned" by the paper except at S1E8M23 and S1E5M10, which it names).
 */
uint32_t orc_encode(float x, int E, int M)
{
    const uint32_t sigma = signbit(x) ? 1u : 0u;
    const uint32_t fmax = (1u << E) - 1u;
    const uint32_t sign_field = sigma << (E + M);
    const int emin = fmt_emin(E), emax = fmt_emax(E), bias = fmt_bias(E);

    if (isnan(x)) {
        if (M == 0) return sign_field | (fmax << M);          /* no NaN exists: infinity     */
        uint32_t m = (f32_bits(x) & 0x7FFFFFu) >> (23 - M);   /* top M bits of the payload   */
        if (m == 0) m = 1u << (M - 1);
        return sign_field | (fmax << M) | m;
    }
    if (isinf(x)) return sign_field | (fmax << M);
    const double a = fabs((double)x);
    if (a == 0.0) return sign_field;

    int ex;
    (void)frexp(a, &ex);                  /* a = fr * 2^ex, fr in [0.5, 1)  =>  floor(log2 a) = ex-1 */
    const int e = ex - 1;
    const int eq = e > emin ? e : emin;   /* binade whose spacing applies (subnormals share emin)    */
    const double q = ldexp(1.0, eq - M);  /* spacing of representable values around a                */
    const double k = nearbyint(a / q);    /* a/q is exact; default rounding mode = ties to even      */
    const double r = k * q;               /* exact: the rounded magnitude                            */

    if (r >= ldexp(1.0, emax + 1)) return sign_field | (fmax << M);
    if (r < ldexp(1.0, emin)) return sign_field | (uint32_t)k;          /* exponent field 0 */
    int ex2;
    (void)frexp(r, &ex2);                 /* rounding may have carried into the next binade */
    const int e2 = ex2 - 1;
    const uint32_t f = (uint32_t)(e2 + bias);
    const uint32_t m = (uint32_t)ldexp(ldexp(r, -e2) - 1.0, M);
    return sign_field | (f << M) | m;
}

void orc_decode_array(const uint32_t *codes, uint64_t n, int E, int M, float *out)
{
    for (uint64_t k = 0; k < n; ++k) out[k] = orc_decode(codes[k], E, M);
}

void orc_encode_array(const float *x, uint64_t n, int E, int M, uint32_t *codes)
{
    for (uint64_t k = 0; k < n; ++k) codes[k] = orc_encode(x[k], E, M);
}

/* ------------------------------------------------------------------------------------------ */
/*
 * Fixed-point variant.  Sec. 2.2 remarks that fixed-point (or other) formats can be used in place
 * of the floating-point one and says nothing more, so everything here is a reading ("parity
 * unpinned" by the paper): S1IxFy = one sign bit, x integer bits, y fraction bits, B = 1 + x + y;
 * a code is the B-bit two's complement of an integer k in [-2^(x+y), 2^(x+y) - 1] and stands for
 * k * 2^-y.  The scale is fixed by the format, not by the data: a scale taken from the data (a
 * maximum) would need a pass over the updated values before the first code could be written,
 * which the one-pass update of Sec. 2.1 has no room for; adapting to the variable is what the
 * per-variable transformation of Sec. 2.3 does afterwards, as for the floating-point codes.
 * Encoding: k = x * 2^y rounded to the nearest integer, ties to even, then clamped to the range
 * (saturation: there is no infinity); NaN has no code either and becomes 0.
 * x + y <= 23, so that every value is an FP32 value.
 */
int orc_fixed_format_ok(int I, int F) { return I >= 0 && I <= 8 && F >= 0 && I + F >= 1 && I + F <= 23; }

float orc_decode_fixed(uint32_t code, int I, int F)
{
    const int B = 1 + I + F;
    int64_t k = (int64_t)(code & ((1u << B) - 1u));
    if (k >= ((int64_t)1 << (B - 1))) k -= ((int64_t)1 << B);      /* two's complement */
    return (float)ldexp((double)k, -F);
}

uint32_t orc_encode_fixed(float x, int I, int F)
{
    const int B = 1 + I + F;
    const uint32_t mask = (1u << B) - 1u;
    if (isnan(x)) return 0u;
    const double lo = -ldexp(1.0, I + F), hi = ldexp(1.0, I + F) - 1.0;
    double k = nearbyint(ldexp((double)x, F));   /* exact scaling; default rounding mode = ties to even */
    if (k < lo) k = lo;
    if (k > hi) k = hi;
    return (uint32_t)(int64_t)k & mask;
}

/* The two codecs behind one switch: fixed != 0 reads (E, M) as (integer bits, fraction bits). */
static uint32_t enc_any(float x, int fixed, int E, int M)
{
    return fixed ? orc_encode_fixed(x, E, M) : orc_encode(x, E, M);
}
static float dec_any(uint32_t c, int fixed, int E, int M)
{
    return fixed ? orc_decode_fixed(c, E, M) : orc_decode(c, E, M);
}

void orc_decode_fixed_array(const uint32_t *codes, uint64_t n, int I, int F, float *out)
{
    for (uint64_t k = 0; k < n; ++k) out[k] = orc_decode_fixed(codes[k], I, F);
}

void orc_encode_fixed_array(const float *x, uint64_t n, int I, int F, uint32_t *codes)
{
    for (uint64_t k = 0; k < n; ++k) codes[k] = orc_encode_fixed(x[k], I, F);
}

/* ------------------------------------------------------------------------------------------ */
/* Bit packing.  The paper stores "B-bit codes"; the layout is this library's (paper silent):    */
/* little-endian bit stream, code k in bits [k*B, (k+1)*B), bit j of the stream = bit (j mod 8)  */
/* of byte (j div 8); the stream is zero-padded to a multiple of 16 bytes.                       */

uint64_t orc_packed_bytes(uint64_t n, int B)
{
    const uint64_t raw = (n * (uint64_t)B + 7u) / 8u;
    return (raw + 15u) / 16u * 16u;
}

void orc_pack(const uint32_t *codes, uint64_t n, int B, uint8_t *out)
{
    memset(out, 0, orc_packed_bytes(n, B));
    for (uint64_t k = 0; k < n; ++k)
        for (int j = 0; j < B; ++j) {
            const uint64_t pos = k * (uint64_t)B + (uint64_t)j;
            if ((codes[k] >> j) & 1u) out[pos >> 3] |= (uint8_t)(1u << (pos & 7u));
        }
}

uint32_t orc_unpack_one(const uint8_t *in, uint64_t k, int B)
{
    uint32_t c = 0;
    for (int j = 0; j < B; ++j) {
        const uint64_t pos = k * (uint64_t)B + (uint64_t)j;
        c |= (uint32_t)((in[pos >> 3] >> (pos & 7u)) & 1u) << j;
    }
    return c;
}

void orc_unpack(const uint8_t *in, uint64_t n, int B, uint32_t *codes)
{
    for (uint64_t k = 0; k < n; ++k) codes[k] = orc_unpack_one(in, k, B);
}

/* ------------------------------------------------------------------------------------------ */
/* Exact summation of doubles: a fixed-point accumulator wide enough for every finite double    */
/* (bit 0 has weight 2^-1074), so the sum is independent of order; rounded once at the end       */
/* (to nearest, ties to even).  Sec. 2.3 asks for 64-bit precision; the order of summation is    */
/* unstated, and the exact sum is the one result every order approximates.                       */

#define ACC_LIMBS 68 /* 68 * 32 = 2176 bits >= 1074 + 1024 + 64 guard bits */

typedef struct {
    int64_t limb[ACC_LIMBS]; /* base-2^32 digits, carries deferred */
    uint32_t pending;        /* additions since the last carry pass */
    int pos_inf, neg_inf, nan;
} exact_acc;

static void acc_init(exact_acc *a) { memset(a, 0, sizeof *a); }

static void acc_carry(exact_acc *a)
{
    int64_t carry = 0;
    for (int i = 0; i < ACC_LIMBS; ++i) {
        int64_t v = a->limb[i] + carry;
        carry = v >> 32;                 /* floor division: digits end in [0, 2^32) */
        a->limb[i] = v - carry * 4294967296LL;
    }
    /* the top limb keeps the sign: fold the final carry back (cannot overflow by sizing) */
    a->limb[ACC_LIMBS - 1] += carry * 4294967296LL;
    a->pending = 0;
}

static void acc_add(exact_acc *a, double x)
{
    if (isnan(x)) { a->nan = 1; return; }
    if (isinf(x)) { if (x > 0) a->pos_inf = 1; else a->neg_inf = 1; return; }
    if (x == 0.0) return;
    int ex;
    const double fr = frexp(fabs(x), &ex);               /* |x| = fr * 2^ex              */
    uint64_t mant = (uint64_t)ldexp(fr, 53);             /* 53-bit integer, exact        */
    int pos = ex - 53 + 1074;                            /* weight of mant's bit 0       */
    if (pos < 0) { mant >>= -pos; pos = 0; }             /* subnormal: low bits are zero */
    const int li = pos / 32, sh = pos % 32;
    const unsigned __int128 wide = (unsigned __int128)mant << sh;   /* <= 85 bits */
    const int64_t d0 = (int64_t)(uint32_t)wide;
    const int64_t d1 = (int64_t)(uint32_t)(wide >> 32);
    const int64_t d2 = (int64_t)(uint32_t)(wide >> 64);
    if (x > 0) { a->limb[li] += d0; a->limb[li + 1] += d1; a->limb[li + 2] += d2; }
    else       { a->limb[li] -= d0; a->limb[li + 1] -= d1; a->limb[li + 2] -= d2; }
    if (++a->pending >= (1u << 30)) acc_carry(a);
}

static double acc_round(exact_acc *a)
{
    if (a->nan || (a->pos_inf && a->neg_inf)) return NAN;
    if (a->pos_inf) return INFINITY;
    if (a->neg_inf) return -INFINITY;
    acc_carry(a);
    int negative = a->limb[ACC_LIMBS - 1] < 0;
    if (negative) {                       /* negate the whole number */
        for (int i = 0; i < ACC_LIMBS; ++i) a->limb[i] = -a->limb[i];
        acc_carry(a);
    }
    int top = ACC_LIMBS - 1;
    while (top >= 0 && a->limb[top] == 0) --top;
    if (top < 0) return 0.0;
    int msb = 31;
    while (!((a->limb[top] >> msb) & 1)) --msb;
    const int p = top * 32 + msb;         /* index of the leading one */
#define ACC_BIT(i) ((int)((a->limb[(i) / 32] >> ((i) % 32)) & 1))
    uint64_t mant = 0;
    const int lo = p - 52;                /* lowest bit kept (may be negative: then exact) */
    for (int i = p; i >= lo && i >= 0; --i) mant = (mant << 1) | (uint64_t)ACC_BIT(i);
    int shift = lo;
    if (lo <= 0) {
        shift = 0;                        /* fewer than 53 bits: nothing to round */
    } else {
        const int round_bit = ACC_BIT(lo - 1);
        int sticky = 0;
        for (int i = lo - 2; i >= 0 && !sticky; --i) sticky = ACC_BIT(i);
        if (round_bit && (sticky || (mant & 1u))) ++mant;
    }
#undef ACC_BIT
    const double mag = ldexp((double)mant, shift - 1074);
    return negative ? -mag : mag;
}

/* Order-independent, correctly rounded sum of n doubles (exported so a test can pin it). */
double orc_exact_sum(const double *x, uint64_t n)
{
    exact_acc a;
    acc_init(&a);
    for (uint64_t k = 0; k < n; ++k) acc_add(&a, x[k]);
    return acc_round(&a);
}

/* ------------------------------------------------------------------------------------------ */
/*
 * Sec. 2.3: per-variable transformation fit.  (s, b) = argmin || s*Vt + b*1 - V ||_2, i.e.
 *     s = (n*Sum(V*Vt) - Sum(V)*Sum(Vt)) / (n*Sum(Vt^2) - Sum(Vt)^2),   b = (Sum(V) - s*Sum(Vt)) / n
 * computed in fp64 from exact sums, stored as fp32.  Degenerate case (Sec. 2.3: denominator 0,
 * all elements the same): s = 1; detected exactly as "all Vt equal" and also taken when the
 * computed denominator is 0 or not finite.  b always follows from its formula with the fp64 s.
 * out4, if given, receives the four sums (Sum V, Sum Vt, Sum V*Vt, Sum Vt^2).
 */
void orc_fit(const float *V, const float *Vt, uint64_t n, int pvt, float *s_out, float *b_out,
             double *out4)
{
    if (!pvt) { *s_out = 1.0f; *b_out = 0.0f; return; }
    exact_acc ax, ay, axy, ayy;
    acc_init(&ax); acc_init(&ay); acc_init(&axy); acc_init(&ayy);
    int all_equal = 1;
    for (uint64_t k = 0; k < n; ++k) {
        const double v = (double)V[k], t = (double)Vt[k];
        acc_add(&ax, v);
        acc_add(&ay, t);
        acc_add(&axy, v * t);     /* 24-bit x 24-bit significands: exact in double */
        acc_add(&ayy, t * t);
        if (!(Vt[k] == Vt[0])) all_equal = 0;
    }
    const double Sx = acc_round(&ax), Sy = acc_round(&ay);
    const double Sxy = acc_round(&axy), Syy = acc_round(&ayy);
    if (out4) { out4[0] = Sx; out4[1] = Sy; out4[2] = Sxy; out4[3] = Syy; }
    const double nn = (double)n;
    const double num = nn * Sxy - Sx * Sy;
    const double den = nn * Syy - Sy * Sy;
    double s64;
    if (all_equal || den == 0.0 || !isfinite(den))
        s64 = 1.0;
    else
        s64 = num / den;
    *s_out = (float)s64;
    *b_out = (float)((Sx - s64 * Sy) / nn);
}

/* ------------------------------------------------------------------------------------------ */
/* Whole-variable operations (Sec. 2.1, Fig. 1).                                                */

/* Initial compression of one variable: quantise V itself, fit (s, b) against it, pack.
 * fixed != 0: the fixed-point codec with (E, M) = (integer bits, fraction bits). */
void orc_compress_var_fx(const float *V, uint64_t n, int fixed, int E, int M, int pvt, uint8_t *packed,
                         float *s_out, float *b_out)
{
    const int B = 1 + E + M;
    uint32_t *codes = (uint32_t *)malloc(n * sizeof(uint32_t));
    float *Vt = (float *)malloc(n * sizeof(float));
    for (uint64_t k = 0; k < n; ++k) {
        codes[k] = enc_any(V[k], fixed, E, M);
        Vt[k] = dec_any(codes[k], fixed, E, M);
    }
    orc_fit(V, Vt, n, pvt, s_out, b_out, NULL);
    orc_pack(codes, n, B, packed);
    free(codes);
    free(Vt);
}

void orc_compress_var(const float *V, uint64_t n, int E, int M, int pvt, uint8_t *packed,
                      float *s_out, float *b_out)
{
    orc_compress_var_fx(V, n, 0, E, M, pvt, packed, s_out, b_out);
}

/* Forward path: Vbar_k = s*Vt_k + b, one correctly rounded fp32 fused multiply-add per element
 * (the rounding of this fp32 operation is a reading: the paper gives only the formula). */
void orc_decompress_var_fx(const uint8_t *packed, uint64_t n, int fixed, int E, int M, float s, float b,
                           float *out)
{
    const int B = 1 + E + M;
    for (uint64_t k = 0; k < n; ++k)
        out[k] = fmaf(s, dec_any(orc_unpack_one(packed, k, B), fixed, E, M), b);
}

void orc_decompress_var(const uint8_t *packed, uint64_t n, int E, int M, float s, float b,
                        float *out)
{
    orc_decompress_var_fx(packed, n, 0, E, M, s, b, out);
}

/*
 * Backward path: decompress, W = Vbar - lr*g (one fp32 fused multiply-add), compress W, discard.
 * A NaN produced by the arithmetic has no payload fixed by IEEE-754; it is replaced by the
 * positive all-ones NaN so that the code written back is defined.  w_out (optional) receives W.
 */
void orc_update_recompress_var_fx(uint8_t *packed, uint64_t n, int fixed, int E, int M, int pvt, float *s_io,
                                  float *b_io, const float *g, float lr, float *w_out)
{
    float *W = (float *)malloc(n * sizeof(float));
    orc_decompress_var_fx(packed, n, fixed, E, M, *s_io, *b_io, W);
    for (uint64_t k = 0; k < n; ++k) {
        float w = fmaf(-lr, g[k], W[k]);
        if (isnan(w)) w = bits_f32(0x7FFFFFFFu);
        W[k] = w;
    }
    orc_compress_var_fx(W, n, fixed, E, M, pvt, packed, s_io, b_io);
    if (w_out) memcpy(w_out, W, n * sizeof(float));
    free(W);
}

void orc_update_recompress_var(uint8_t *packed, uint64_t n, int E, int M, int pvt, float *s_io,
                               float *b_io, const float *g, float lr, float *w_out)
{
    orc_update_recompress_var_fx(packed, n, 0, E, M, pvt, s_io, b_io, g, lr, w_out);
}

/* Variables that stay in FP32 (Sec. 2.4): plain SGD step in place. */
void orc_sgd_var(float *v, const float *g, uint64_t n, float lr)
{
    for (uint64_t k = 0; k < n; ++k) v[k] = fmaf(-lr, g[k], v[k]);
}

/*
 * Server side (Sec. 1: the clients' trained models are sent back and aggregated; Sec. 2.5: each
 * client compresses its own subset, so for one parameter some clients deliver decompressed values
 * and others full-precision ones).  The paper says only "aggregated"; the reading here is the
 * plain mean in FP32: x[0][e] + x[1][e] + ... in client order, every addition rounded to FP32,
 * then one correctly rounded division by K ("parity unpinned" by the paper beyond "mean").
 * x[k] = client k's values of the variable (already decompressed where it held codes).
 */
void orc_aggregate_var(const float *const *x, uint32_t K, uint64_t n, float *out)
{
    for (uint64_t e = 0; e < n; ++e) {
        float acc = x[0][e];
        for (uint32_t k = 1; k < K; ++k) acc = acc + x[k][e];
        out[e] = acc / (float)K;
    }
}

/*
 * The same mean taken in two stages, for clients spread over several servers or GPUs: each holder
 * adds up its own clients (client order, FP32, no division), the holders' sums are added in holder
 * order, and the total is divided once by the number of all clients.  With one holder this is
 * orc_aggregate_var.  (A reading like the mean itself; across holders the order of the additions
 * is whatever the transport does, so a real run is only bounded by, not equal to, this order.)
 */
void orc_sum_var(const float *const *x, uint32_t K, uint64_t n, float *out)
{
    for (uint64_t e = 0; e < n; ++e) {
        float acc = x[0][e];
        for (uint32_t k = 1; k < K; ++k) acc = acc + x[k][e];
        out[e] = acc;
    }
}

void orc_divide_var(const float *x, uint64_t n, uint32_t K, float *out)
{
    for (uint64_t e = 0; e < n; ++e) out[e] = x[e] / (float)K;
}

/* ------------------------------------------------------------------------------------------ */
/* Selection (Sec. 2.4, 2.5, 3.1) and size accounting (Tables 1 and 2).                         */

static uint64_t splitmix64_next(uint64_t *state)
{
    uint64_t z = (*state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

uint64_t orc_splitmix64(uint64_t seed, uint32_t nth) /* the nth (0-based) output for a seed */
{
    uint64_t st = seed, z = 0;
    for (uint32_t i = 0; i <= nth; ++i) z = splitmix64_next(&st);
    return z;
}

/*
 * Sec. 3.1: the selection varies "from round to round and from client to client", so every
 * (round, client) pair needs a selection seed of its own, derived from one seed for the whole job.
 * The rule is this library's (the paper says only that the selections vary): the seed of
 * (round, client) is output number round * 2^32 + client, counted from 0, of the SplitMix64 stream
 * seeded with `base`.  The generator's state is a counter (it advances by a fixed odd constant per
 * output), so output number k is the output function applied to base + (k + 1) * constant: no
 * stepping through the stream is needed.
 */
uint64_t orc_plan_seed(uint64_t base, uint32_t round, uint32_t client)
{
    const uint64_t k = ((uint64_t)round << 32) | (uint64_t)client;
    uint64_t z = base + (k + 1u) * 0x9E3779B97F4A7C15ull;      /* the state after k + 1 steps */
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/*
 * Which variables are quantised.  eligible[i] != 0 marks the weight matrices (Sec. 2.4);
 * k = floor(p*W + 1/2) of the W eligible ones are chosen at random (Sec. 2.5, Sec. 3.1): the
 * eligible indices in ascending order are shuffled by Fisher-Yates (i from W-1 down to 1,
 * j = next() mod (i+1), swap) driven by SplitMix64(seed), and the first k are taken.  The
 * generator and the shuffle order are this library's choice (the paper says only "randomly").
 */
void orc_select(const uint8_t *eligible, uint32_t nvars, double fraction, uint64_t seed,
                uint8_t *selected)
{
    uint32_t *perm = (uint32_t *)malloc((nvars ? nvars : 1) * sizeof(uint32_t));
    uint32_t W = 0;
    for (uint32_t i = 0; i < nvars; ++i) {
        selected[i] = 0;
        if (eligible[i]) perm[W++] = i;
    }
    uint64_t st = seed;
    for (uint32_t i = W; i-- > 1;) {
        const uint32_t j = (uint32_t)(splitmix64_next(&st) % (uint64_t)(i + 1));
        const uint32_t t = perm[i]; perm[i] = perm[j]; perm[j] = t;
    }
    uint32_t k = (uint32_t)floor(fraction * (double)W + 0.5);
    if (k > W) k = W;
    for (uint32_t i = 0; i < k; ++i) selected[perm[i]] = 1;
    free(perm);
}

/* Stored size of a model: B-bit codes plus (s, b) for quantised variables, FP32 for the rest. */
uint64_t orc_model_bytes(const uint64_t *numel, const uint8_t *selected, uint32_t nvars, int B)
{
    uint64_t bytes = 0;
    for (uint32_t i = 0; i < nvars; ++i)
        bytes += selected[i] ? (numel[i] * (uint64_t)B + 7u) / 8u + 8u : 4u * numel[i];
    return bytes;
}
