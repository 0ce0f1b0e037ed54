// SxEyMz codec arithmetic for the device side (Sec. 2.2 of the OMC paper; notation of Sec. 3.1).
//
// A code is sign<<(E+M) | exponent_field<<M | mantissa_field with the IEEE-754 interchange
// parametrisation: bias 2^(E-1)-1, exponent field 0 = zero/subnormal, all ones = Inf/NaN.
// Encoding rounds to nearest, ties to even, with gradual underflow and overflow to infinity.
//
// Each operation has a "fast" form that is exact for every finite in-range input and an "exact"
// form that also handles Inf/NaN/overflow; callers test once per group of elements whether the
// exact form is needed (it almost never is) instead of paying for it per element.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace omc {

template <int E_, int M_>
struct Fmt {
    static_assert(E_ >= 2 && E_ <= 8 && M_ >= 0 && M_ <= 23, "format outside the accepted family");
    static constexpr bool FIXED = false;
    static constexpr int E = E_, M = M_, B = 1 + E_ + M_;
    static constexpr int BIAS = (1 << (E_ - 1)) - 1;
    static constexpr int EMIN = 1 - BIAS, EMAX = BIAS;
    static constexpr int SH = 23 - M_;                                   // fp32 mantissa bits dropped
    static constexpr uint32_t CODE_MASK = (B == 32) ? 0xFFFFFFFFu : ((1u << (B % 32)) - 1u);
    static constexpr uint32_t MAG_MASK = (1u << (E_ + M_)) - 1u;         // exponent + mantissa fields
    static constexpr uint32_t INF_MAG = ((1u << E_) - 1u) << M_;         // magnitude code of infinity
    static constexpr uint32_t SIGN_BIT = 1u << (E_ + M_);
    // fp32 bit pattern of 2^k
    __host__ __device__ static constexpr uint32_t pow2_bits(int k) { return (uint32_t)(k + 127) << 23; }
    // Smallest FP32 magnitude that rounds to infinity: 2^EMAX * (2 - 2^-(M+1)) (a tie, which goes
    // to the even side = infinity); with M == 23 that is not an FP32 value and 2^(EMAX+1) is.
    __host__ __device__ static constexpr uint32_t ovf_bits()
    {
        if (E_ == 8) return 0x7F800000u;
        if (M_ == 23) return pow2_bits(EMAX + 1);
        return pow2_bits(EMAX) | (((1u << (M_ + 1)) - 1u) << (M_ == 23 ? 0 : 22 - M_));
    }
    static constexpr uint32_t OVF_BITS = ovf_bits();
};

// The fixed-point variant (Sec. 2.2 names fixed-point formats as an alternative without defining
// one): S1IxFy, a B = 1 + x + y bit two's-complement integer k standing for k * 2^-y, rounded to
// nearest even, saturating at both ends (there is no infinity), NaN -> 0.  E and M carry x and y
// so that the layout code (B bits per code, LU elements per lane) needs no second set of names.
// The fast forms below need every |k| <= 2^22 (x + y <= 22): the FP32 adder does the rounding to
// an integer (adding 1.5 * 2^23 leaves k in the low mantissa bits, as a two's complement), and a
// code with its sign bit flipped is an unsigned offset that drops straight into a mantissa.
template <int I_, int F_>
struct FixFmt {
    static_assert(I_ >= 0 && I_ <= 8 && F_ >= 0 && I_ + F_ >= 1 && I_ + F_ <= 22, "fixed-point format outside the compiled family");
    static constexpr bool FIXED = true;
    static constexpr int E = I_, M = F_, B = 1 + I_ + F_;
    static constexpr int SH = 0;
    static constexpr uint32_t CODE_MASK = (1u << B) - 1u;
    static constexpr uint32_t SIGN_BIT = 1u << (I_ + F_);
    static constexpr uint32_t MAG_MASK = SIGN_BIT - 1u, INF_MAG = 0xFFFFFFFFu, OVF_BITS = 0x7F800000u;
    static constexpr float SCALE = (float)(1u << F_), INV_SCALE = 1.f / (float)(1u << F_);
    static constexpr float LO = -(float)(1u << (I_ + F_)), HI = (float)((1u << (I_ + F_)) - 1u);
    static constexpr float MAGIC = 12582912.f;                    // 1.5 * 2^23
    static constexpr float OFFSET = 8388608.f + (float)(1u << (I_ + F_));   // 2^23 + 2^(B-1)
};

// Formats with E = 5 and M <= 10 are FP16 with the low mantissa bits dropped: code << (10-M) is
// an IEEE half, so the hardware half conversions do the exponent work (specials included).
template <class F>
struct HalfPath {
    static constexpr bool value = (!F::FIXED && F::E == 5 && F::M <= 10);
};

// Formats whose codes, below the top of the range, are those of a hardware narrow-float type
// (e5m2, e4m3 and the 6-bit e2m3, each held in one byte by the conversion instructions).
template <class F>
struct Fp8Path {
    static constexpr bool value =
        !F::FIXED && ((F::E == 5 && F::M == 2) || (F::E == 4 && F::M == 3) || (F::E == 2 && F::M == 3));
};

__device__ __forceinline__ uint32_t f2u(float x) { return __float_as_uint(x); }
__device__ __forceinline__ float u2f(uint32_t u) { return __uint_as_float(u); }

// ---------------------------------------------------------------------------------------------
// decode

// Exact for every code whose exponent field is not all ones.
template <class F>
__device__ __forceinline__ float decode_fast(uint32_t c)
{
    if constexpr (F::FIXED) {
        // 2^23 + (k + 2^(B-1)) as a float, then (that - 2^23 - 2^(B-1)) * 2^-y in one exact operation
        const float f = u2f(c ^ (F::SIGN_BIT | 0x4B000000u));
        return __fmaf_rn(f, F::INV_SCALE, -F::OFFSET * F::INV_SCALE);
    } else if constexpr (F::E == 8) {
        return u2f(c << F::SH);      // S1E8Mz is FP32 with the low mantissa bits dropped
    } else if constexpr (HalfPath<F>::value) {
        return __half2float(__ushort_as_half((unsigned short)(c << (10 - F::M))));   // exact, all codes
    } else {
        // Put the fields where FP32 keeps them: the result has the code's exponent field as its
        // own (subnormal codes become FP32 subnormals), so one exact multiplication by
        // 2^(127-BIAS) rebiases normal and subnormal codes alike.
        const uint32_t mag = (c & F::MAG_MASK) << F::SH;
        const float v = __fmul_rn(u2f(mag), u2f(F::pow2_bits(127 - F::BIAS)));
        return u2f(f2u(v) | ((c >> (F::E + F::M)) << 31));
    }
}

template <class F>
__device__ __forceinline__ bool code_is_special(uint32_t c)
{
    if constexpr (F::FIXED || F::E == 8 || HalfPath<F>::value) return false;   // decode_fast is already exact
    return (c & F::MAG_MASK) >= F::INF_MAG;
}

// Every code, Inf and NaN included (NaN: mantissa field kept in the top bits of the payload).
template <class F>
__device__ __forceinline__ float decode_exact(uint32_t c)
{
    if constexpr (!F::FIXED && F::E < 8 && !HalfPath<F>::value) {
        if ((c & F::MAG_MASK) >= F::INF_MAG) {
            const uint32_t m = c & ((1u << F::M) - 1u);
            return u2f(((c >> (F::E + F::M)) << 31) | 0x7F800000u | (m << F::SH));
        }
    }
    return decode_fast<F>(c);
}

// ---------------------------------------------------------------------------------------------
// encode: returns the code and the decoded value Q^-1(Q(w)) (needed by the Sec. 2.3 fit).

// Exact iff !needs_exact_encode(w).
template <class F>
__device__ __forceinline__ uint32_t encode_fast(float w, float &vt)
{
    const uint32_t u = f2u(w);
    if constexpr (F::FIXED) {
        // clamp (the bounds are integers, so clamping before the rounding is clamping after it),
        // round to an integer with the adder, read k off the mantissa
        const float t = fminf(fmaxf(__fmul_rn(w, F::SCALE), F::LO), F::HI);
        const float r = __fadd_rn(t, F::MAGIC);
        vt = __fmaf_rn(r, F::INV_SCALE, -F::MAGIC * F::INV_SCALE);     // (r - MAGIC) * 2^-y, exact
        return f2u(r) & F::CODE_MASK;
    } else if constexpr (F::M == 23 && F::E == 8) {
        vt = w;
        return u;
    } else if constexpr (HalfPath<F>::value && F::M == 10) {
        // FP16 itself: the hardware conversion rounds to nearest even, underflows gradually,
        // overflows to infinity and turns any NaN into 0x7FFF.
        const __half h = __float2half_rn(w);
        vt = __half2float(h);
        return (uint32_t)__half_as_ushort(h);
    } else if constexpr (F::E == 8) {
        // Only mantissa bits are dropped: round the FP32 pattern as an integer (a carry out of
        // the mantissa moves into the exponent, up to infinity, exactly as it should).
        const uint32_t a = u & 0x7FFFFFFFu;
        const uint32_t lsb = (a >> F::SH) & 1u;
        const uint32_t mag = (a + ((1u << (F::SH - 1)) - 1u) + lsb) >> F::SH;
        const uint32_t c = mag | ((u >> 31) << (F::E + F::M));
        vt = u2f(c << F::SH);
        return c;
    } else {
        // Let the FP32 adder do the rounding: adding 2^(e_q+23-M), e_q = max(exponent, EMIN),
        // leaves exactly the bits above the target spacing 2^(e_q-M), rounded to nearest even.
        if constexpr (F::M <= 22 && !HalfPath<F>::value) {
            // The constant as 2^e_q (with w's sign) times 2^(23-M): the product is exact, so the two
            // fused multiply-adds round exactly what the addition and the subtraction would, on
            // the signed value.  A negative w that rounds to zero gives +0 here; the sums and
            // the equality test do not tell the zeros apart, and the code takes its sign from w.
            const uint32_t m = max(u & 0x7F800000u, F::pow2_bits(F::EMIN));
            const float ms = u2f(m | (u & 0x80000000u));
            constexpr float K = (float)(1u << F::SH);
            vt = __fmaf_rn(ms, -K, __fmaf_rn(ms, K, w));
            // vt is a value of the format: rebias its magnitude exactly, read the fields off the pattern
            const float t = __fmul_rn(fabsf(vt), u2f(F::pow2_bits(F::BIAS - 127)));
            return (f2u(t) >> F::SH) | ((u >> (31 - F::E - F::M)) & F::SIGN_BIT);
        }
        const float a = fabsf(w);
        float r;
        if constexpr (F::M <= 22) {
            const float x2 = __fmul_rn(a, u2f(F::pow2_bits(F::SH)));
            const uint32_t eb = max(f2u(x2) & 0x7F800000u, F::pow2_bits(F::EMIN + F::SH));
            const float magic = u2f(eb);
            r = __fsub_rn(__fadd_rn(a, magic), magic);
        } else {
            // M == 23: normal-range values are kept as they are, only the subnormal range rounds
            const float magic = u2f(F::pow2_bits(F::EMIN));
            const float rs = __fsub_rn(__fadd_rn(a, magic), magic);
            r = (f2u(a) >= F::pow2_bits(F::EMIN)) ? a : rs;
        }
        vt = u2f(f2u(r) | (u & 0x80000000u));
        if constexpr (HalfPath<F>::value) {
            // r is an FP16 value with zero low mantissa bits: the half conversion is exact
            return (uint32_t)__half_as_ushort(__float2half_rn(vt)) >> (10 - F::M);
        } else {
            // r is a value of the format: rebias exactly and read the fields off the FP32 pattern.
            const float t = __fmul_rn(r, u2f(F::pow2_bits(F::BIAS - 127)));
            return (f2u(t) >> F::SH) | ((u >> 31) << (F::E + F::M));
        }
    }
}

// Two elements at once.  On the half path the two conversions to FP16 share one packed
// instruction (the single-value conversion runs on a unit with a quarter of the throughput).
template <class F>
__device__ __forceinline__ void encode_fast2(float w0, float w1, uint32_t &c0, uint32_t &c1, float &vt0,
                                             float &vt1)
{
    if constexpr (HalfPath<F>::value && F::M == 10) {
        const __half2 h = __floats2half2_rn(w0, w1);     // low half = w0
        const uint32_t x = *reinterpret_cast<const uint32_t *>(&h);
        c0 = x & 0xFFFFu;
        c1 = x >> 16;
        vt0 = __low2float(h);
        vt1 = __high2float(h);
    } else if constexpr (HalfPath<F>::value && F::M <= 9) {
        const uint32_t u0 = f2u(w0), u1 = f2u(w1);
        const float a0 = fabsf(w0), a1 = fabsf(w1);
        const float x0 = __fmul_rn(a0, u2f(F::pow2_bits(F::SH))), x1 = __fmul_rn(a1, u2f(F::pow2_bits(F::SH)));
        const float m0 = u2f(max(f2u(x0) & 0x7F800000u, F::pow2_bits(F::EMIN + F::SH)));
        const float m1 = u2f(max(f2u(x1) & 0x7F800000u, F::pow2_bits(F::EMIN + F::SH)));
        const float r0 = __fsub_rn(__fadd_rn(a0, m0), m0), r1 = __fsub_rn(__fadd_rn(a1, m1), m1);
        vt0 = u2f(f2u(r0) | (u0 & 0x80000000u));
        vt1 = u2f(f2u(r1) | (u1 & 0x80000000u));
        const __half2 h = __floats2half2_rn(vt0, vt1);   // exact: both are FP16 values
        const uint32_t x = *reinterpret_cast<const uint32_t *>(&h);
        c0 = (x & 0xFFFFu) >> (10 - F::M);
        c1 = x >> (26 - F::M);
    } else {
        c0 = encode_fast<F>(w0, vt0);
        c1 = encode_fast<F>(w1, vt1);
    }
}

// True when encode_fast would be wrong: NaN, and for E < 8 infinity and finite values that round
// to infinity.  KEEP_PAYLOAD = false means the caller accepts the positive all-ones NaN code for
// any NaN input, which is what the FP16 hardware conversion produces by itself.
template <class F, bool KEEP_PAYLOAD>
__device__ __forceinline__ bool needs_exact_encode(float w)
{
    const uint32_t a = f2u(w) & 0x7FFFFFFFu;
    if constexpr (F::FIXED) return a > 0x7F800000u;          // NaN only: everything else saturates
    if constexpr (HalfPath<F>::value && F::M == 10) return KEEP_PAYLOAD ? (a > 0x7F800000u) : false;
    if constexpr (F::E == 8) return a > 0x7F800000u;
    return a >= F::OVF_BITS;
}

// The same two tests for four elements at once, on values instead of bit patterns: one maximum
// of magnitudes (a NaN among them wins) and one comparison replace four integer comparisons.
__device__ __forceinline__ float absmax4(float a, float b, float c, float d)
{
    float r;
    asm("{\n\t.reg .f32 t0, t1, t2, t3;\n\t"
        "abs.f32 t0, %1;\n\tabs.f32 t1, %2;\n\tabs.f32 t2, %3;\n\tabs.f32 t3, %4;\n\t"
        "max.NaN.f32 t2, t2, t3;\n\t"
        "max.NaN.f32 %0, t0, t1, t2;\n\t}"
        : "=f"(r) : "f"(a), "f"(b), "f"(c), "f"(d));
    return r;
}

// dec = decode_fast of four codes: a code with an all-ones exponent field decodes to a magnitude
// of at least 2^(EMAX+1), every other code to less.
template <class F>
__device__ __forceinline__ bool any_code_special4(const float (&dec)[4])
{
    if constexpr (F::FIXED || F::E == 8 || HalfPath<F>::value) return false;
    else return absmax4(dec[0], dec[1], dec[2], dec[3]) >= u2f(F::pow2_bits(F::EMAX + 1));
}

template <class F, bool KEEP_PAYLOAD>
__device__ __forceinline__ bool any_needs_exact_encode4(const float (&w)[4])
{
    if constexpr (HalfPath<F>::value && F::M == 10 && !KEEP_PAYLOAD) return false;
    else {
        const float m = absmax4(w[0], w[1], w[2], w[3]);
        if constexpr (F::FIXED || (HalfPath<F>::value && F::M == 10) || F::E == 8) return m != m;      // NaN only
        else return !(m < u2f(F::OVF_BITS));                                               // overflow, Inf, NaN
    }
}

// NaN -> sign, all-ones exponent, top M payload bits (a quiet bit is forced if those are zero;
// with M == 0 there is no NaN code and infinity is written).
template <class F>
__device__ __forceinline__ uint32_t encode_exact(float w, float &vt)
{
    const uint32_t u = f2u(w);
    const uint32_t a = u & 0x7FFFFFFFu;
    if constexpr (F::FIXED) {
        if (a > 0x7F800000u) {      // NaN has no code: it becomes 0
            vt = 0.f;
            return 0u;
        }
        return encode_fast<F>(w, vt);
    }
    const uint32_t sign = (u >> 31) << (F::E + F::M);
    if (a > 0x7F800000u) {
        uint32_t c;
        if constexpr (F::M == 0) {
            c = sign | F::INF_MAG;
        } else {
            uint32_t m = (u & 0x7FFFFFu) >> F::SH;
            if (m == 0) m = 1u << (F::M - 1);
            c = sign | F::INF_MAG | m;
        }
        vt = decode_exact<F>(c);
        return c;
    }
    if constexpr (F::E < 8) {
        if (a >= F::OVF_BITS) {
            vt = u2f(0x7F800000u | (u & 0x80000000u));
            return sign | F::INF_MAG;
        }
    }
    return encode_fast<F>(w, vt);
}

// ---------------------------------------------------------------------------------------------
// Codes inside a run of 32-bit words (little-endian bit stream, code i at bits [i*B, (i+1)*B)).
// With i a compile-time constant after unrolling, every shift below is an immediate.

// The code at bit position `pos` of the words (pos = i*B for code i of an array that starts at code 0).
template <class F, int NW>
__device__ __forceinline__ uint32_t get_code_at(const uint32_t (&w)[NW], int pos)
{
    const int wi = pos >> 5, sh = pos & 31;
    uint32_t c;
    if (sh + F::B <= 32)
        c = w[wi] >> sh;
    else
        c = __funnelshift_r(w[wi], w[(wi + 1 < NW) ? wi + 1 : wi], sh);
    return c & F::CODE_MASK;
}

// The code at bit position `pos` with its fields where FP32 keeps them, before the rebias
// multiplication: decode_fast(code) = placed * 2^(127-BIAS) exactly.  A code with an all-ones
// exponent field gives a magnitude of at least u2f(INF_MAG << SH), every other code less.
template <class F, int NW>
__device__ __forceinline__ float placed_at(const uint32_t (&w)[NW], int pos)
{
    static_assert(!F::FIXED && F::E < 8 && !HalfPath<F>::value, "generic path");
    const int wi = pos >> 5, sh = pos & 31;
    uint32_t t;      // the code in the top B bits
    if (sh + F::B <= 32)
        t = w[wi] << (32 - sh - F::B);
    else
        t = __funnelshift_r(w[wi], w[(wi + 1 < NW) ? wi + 1 : wi], sh + F::B - 32);
    // an arithmetic shift keeps the sign at bit 31; the copies of it that follow are masked away
    return u2f((uint32_t)((int32_t)t >> (8 - F::E)) & (0x80000000u | (F::MAG_MASK << F::SH)));
}

// decode_fast of the code at bit position `pos`, without isolating the code first: one shift
// puts the code's sign at bit 31 (whatever follows the code stays in the low bits), a second one
// and a mask put exponent and mantissa where FP32 keeps them, and the sign is merged after the
// rebias multiplication.  Formats on the generic path only (E < 8, not the FP16 family).
template <class F, int NW>
__device__ __forceinline__ float decode_fast_at(const uint32_t (&w)[NW], int pos)
{
    return __fmul_rn(placed_at<F, NW>(w, pos), u2f(F::pow2_bits(127 - F::BIAS)));
}

template <class F, int NW>
__device__ __forceinline__ void put_code_at(uint32_t (&w)[NW], int pos, uint32_t c)
{
    // the fields are disjoint, so adding is OR-ing, and a shift-and-add is one instruction
    const int wi = pos >> 5, sh = pos & 31;
    w[wi] += c << sh;
    if (sh + F::B > 32) w[(wi + 1 < NW) ? wi + 1 : wi] += c >> (32 - sh);
}

}  // namespace omc
