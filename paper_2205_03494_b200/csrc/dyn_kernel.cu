// Fallback kernels for SxEyMz formats that have no compiled specialisation: the format is a
// run-time argument, every element takes the careful (all-cases) arithmetic, and each lane works
// through 32 consecutive elements with a streaming bit reader / writer straight on global memory.
// Same results, layouts, tile partition and fit as the specialised kernels; an order of magnitude
// slower, which is the price of covering all of 2 <= E <= 8, 0 <= M <= 23 without 168 builds.
#include <cmath>

#include "kernels.cuh"

namespace omc {

struct DynFmt {
    int fixed;               // the fixed-point variant S1IxFy: E = x, M = y
    float scale, inv_scale, lo, hi;      // 2^y, 2^-y, -2^(x+y), 2^(x+y) - 1
    int E, M, B, SH;
    uint32_t mag_mask, inf_mag, ovf_bits, min_normal_bits, clamp_bits;
    float up, down, xs;      // 2^(127-BIAS), 2^(BIAS-127), 2^SH
};

static DynFmt make_dyn(int E, int M, int fixed)
{
    DynFmt f{};
    f.E = E; f.M = M; f.B = 1 + E + M; f.SH = 23 - M;
    f.fixed = fixed;
    if (fixed) {
        f.scale = std::ldexp(1.f, M);
        f.inv_scale = std::ldexp(1.f, -M);
        f.lo = -std::ldexp(1.f, E + M);
        f.hi = std::ldexp(1.f, E + M) - 1.f;
        return f;
    }
    const int bias = (1 << (E - 1)) - 1, emin = 1 - bias, emax = bias;
    auto p2 = [](int k) { return (uint32_t)(k + 127) << 23; };
    auto asf = [](uint32_t u) { float x; memcpy(&x, &u, 4); return x; };
    f.mag_mask = (1u << (E + M)) - 1u;
    f.inf_mag = ((1u << E) - 1u) << M;
    if (E == 8) f.ovf_bits = 0x7F800000u;
    else if (M == 23) f.ovf_bits = p2(emax + 1);
    else f.ovf_bits = p2(emax) | (((1u << (M + 1)) - 1u) << (22 - M));
    f.min_normal_bits = (E == 8) ? 0x00800000u : p2(emin);
    f.clamp_bits = (E == 8) ? 0u : p2(emin + f.SH);      // exponent pattern of 2^(EMIN+SH)
    f.up = (E == 8) ? 1.f : asf(p2(127 - bias));
    f.down = (E == 8) ? 1.f : asf(p2(bias - 127));
    f.xs = asf(p2(f.SH));
    return f;
}

__device__ __forceinline__ float dyn_decode(const DynFmt &f, uint32_t c)
{
    if (f.fixed) {      // two's complement, k * 2^-y
        const int k = (int)(c << (32 - f.B)) >> (32 - f.B);
        return __fmul_rn((float)k, f.inv_scale);
    }
    if (f.E == 8) return u2f(c << f.SH);
    const uint32_t mag = c & f.mag_mask;
    const uint32_t sign = (c >> (f.E + f.M)) << 31;
    if (mag >= f.inf_mag) return u2f(sign | 0x7F800000u | ((c & ((1u << f.M) - 1u)) << f.SH));
    return u2f(f2u(__fmul_rn(u2f(mag << f.SH), f.up)) | sign);
}

// Round to nearest even with gradual underflow, overflow to infinity, NaN payload kept.
__device__ __forceinline__ uint32_t dyn_encode(const DynFmt &f, float w, float &vt)
{
    const uint32_t u = f2u(w), a = u & 0x7FFFFFFFu;
    if (f.fixed) {      // nearest integer multiple of 2^-y, ties to even, saturating; NaN -> 0
        if (a > 0x7F800000u) { vt = 0.f; return 0u; }
        const int k = __float2int_rn(fminf(fmaxf(__fmul_rn(w, f.scale), f.lo), f.hi));
        vt = __fmul_rn((float)k, f.inv_scale);
        return (uint32_t)k & ((1u << f.B) - 1u);
    }
    const uint32_t sign = (u >> 31) << (f.E + f.M);
    if (a > 0x7F800000u) {
        uint32_t c = sign | f.inf_mag;
        if (f.M > 0) {
            uint32_t m = (u & 0x7FFFFFu) >> f.SH;
            if (m == 0) m = 1u << (f.M - 1);
            c |= m;
        }
        vt = dyn_decode(f, c);
        return c;
    }
    if (f.E == 8) {
        if (f.M == 23) { vt = w; return u; }
        const uint32_t lsb = (a >> f.SH) & 1u;
        const uint32_t c = ((a + ((1u << (f.SH - 1)) - 1u) + lsb) >> f.SH) | sign;
        vt = u2f(c << f.SH);
        return c;
    }
    if (a >= f.ovf_bits) {
        vt = u2f(0x7F800000u | (u & 0x80000000u));
        return sign | f.inf_mag;
    }
    const float af = u2f(a);
    float r;
    if (f.M <= 22) {     // the FP32 adder rounds at the target spacing 2^(max(e, EMIN) - M)
        const uint32_t eb = max(f2u(__fmul_rn(af, f.xs)) & 0x7F800000u, f.clamp_bits);
        r = __fsub_rn(__fadd_rn(af, u2f(eb)), u2f(eb));
    } else {             // M == 23: only the subnormal range of the format rounds
        const float magic = u2f(f.min_normal_bits);
        r = (a >= f.min_normal_bits) ? af : __fsub_rn(__fadd_rn(af, magic), magic);
    }
    vt = u2f(f2u(r) | (u & 0x80000000u));
    return (f2u(__fmul_rn(r, f.down)) >> f.SH) | sign;
}

template <int MODE, bool WOUT>
__global__ void __launch_bounds__(THREADS) omc_dyn_kernel(const KParams p, const DynFmt f)
{
    const int lane = threadIdx.x & 31;
    const uint32_t warp = blockIdx.x * WARPS_PER_CTA + (threadIdx.x >> 5);
    if (warp >= p.nwarps) return;
    const uint32_t code_mask = f.B == 32 ? 0xFFFFFFFFu : ((1u << f.B) - 1u);
    for (uint32_t run = warp; run < p.nruns; run += p.nwarps) {
        uint64_t t, tend;
        run_tile_range(p, run, t, tend);
        uint32_t v = run_first_var(p, run, t);
        while (t < tend) {
            const VarDev var = p.vars[v];
            const uint32_t local = (uint32_t)(t - var.tile_start);
            const uint64_t left = tend - t;
            const uint32_t cnt = (uint32_t)((uint64_t)(var.ntiles - local) < left ? (var.ntiles - local) : left);
            if (var.quantised) {
                float s = 1.f, b = 0.f;
                if (MODE != COMPRESS) { s = __ldcg(p.sb + 2 * var.sb_slot); b = __ldcg(p.sb + 2 * var.sb_slot + 1); }
                Acc acc;
                acc.reset();
                uint32_t *const cw = reinterpret_cast<uint32_t *>(p.packed + var.store_off);
                const uint64_t nwords = var.packed_bytes / 4;
                for (uint32_t i = 0; i < cnt; ++i) {
                    // this lane's 32 elements of the tile and the B words that hold exactly their codes
                    const uint64_t e0 = (uint64_t)(local + i) * TILE + (uint64_t)lane * 32;
                    const uint64_t w0 = e0 / 32 * f.B;
                    const int valid = e0 >= var.n ? 0 : (var.n - e0 < 32 ? (int)(var.n - e0) : 32);
                    uint64_t rbuf = 0, wbuf = 0;      // bit reader / writer over consecutive words
                    int rfill = 0, wfill = 0;
                    uint64_t rw = w0, ww = w0;
                    uint32_t ref = 0u, diff = 0u;
                    for (int k = 0; k < valid; ++k) {
                        float w;
                        if (MODE != COMPRESS) {
                            if (rfill < f.B) { rbuf |= (uint64_t)cw[rw++] << rfill; rfill += 32; }
                            const uint32_t c = (uint32_t)rbuf & code_mask;
                            rbuf >>= f.B; rfill -= f.B;
                            const float vbar = __fmaf_rn(s, dyn_decode(f, c), b);
                            w = vbar;
                            if (MODE == UPDATE) {
                                w = __fmaf_rn(p.neg_lr, p.fin[var.full_off + e0 + k], vbar);
                                if (w != w) w = u2f(0x7FFFFFFFu);     // arithmetic NaNs get one pattern
                            }
                        } else {
                            w = p.fin[var.full_off + e0 + k];
                        }
                        if (MODE != DECOMPRESS) {
                            float vt;
                            const uint32_t c = dyn_encode(f, w, vt);
                            acc.add(w, vt);
                            if (k == 0) ref = f2u(vt); else diff |= f2u(vt) ^ ref;
                            wbuf |= (uint64_t)c << wfill; wfill += f.B;
                            if (wfill >= 32) { cw[ww++] = (uint32_t)wbuf; wbuf >>= 32; wfill -= 32; }
                        }
                        if (MODE == DECOMPRESS || WOUT) p.fout[var.full_off + e0 + k] = w;
                    }
                    if (MODE != DECOMPRESS) {
                        if (valid > 0) { acc.band &= ref & ~diff; acc.bor |= ref | diff; }
                        if (wfill > 0) { cw[ww++] = (uint32_t)wbuf; }
                        // words of this lane's share that hold no code any more: zero padding
                        for (; ww < w0 + (uint64_t)f.B && ww < nwords; ++ww) cw[ww] = 0u;
                    }
                }
                if (MODE != DECOMPRESS) {
                    if (p.pvt) {
                        flush_and_maybe_finalise(p.slots + var.slot_base, run - var.first_run, var.nslots,
                                                 p.tickets + var.sb_slot, cnt, var.ntiles, var.n, 0x7FFFFFFFu,
                                                 p.sb + 2 * var.sb_slot, acc, lane);
                    } else if (MODE == COMPRESS && local == 0 && lane == 0) {
                        p.sb[2 * var.sb_slot] = 1.f;
                        p.sb[2 * var.sb_slot + 1] = 0.f;
                    }
                }
            } else {
                resid_tiles<MODE, WOUT>(p.resid + var.store_off, (MODE != DECOMPRESS) ? p.fin + var.full_off : nullptr,
                                        ((MODE == DECOMPRESS) || WOUT) ? p.fout + var.full_off : nullptr, var.n, local,
                                        cnt, p.neg_lr, lane);
            }
            t += cnt;
            ++v;
        }
    }
}

template <int MODE, bool WOUT>
static void launch_dyn(const KParams &p, int grid, void *stream)
{
    omc_dyn_kernel<MODE, WOUT><<<grid, THREADS, 0, static_cast<cudaStream_t>(stream)>>>(p, make_dyn((int)p.dyn_e, (int)p.dyn_m, (int)p.dyn_fixed));
}

extern const FmtOps ops_dynamic = {-1, -1, -1, WARPS_PER_CTA, CTAS_PER_SM, launch_dyn<COMPRESS, false>, launch_dyn<DECOMPRESS, false>,
                                   launch_dyn<UPDATE, false>, launch_dyn<UPDATE, true>, nullptr, nullptr, nullptr};

}  // namespace omc
