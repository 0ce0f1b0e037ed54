// The three OMC kernels (compress, decompress, fused update-recompress) as one warp-tiled
// template.  Work is a flat list of 1024-element tiles over all variables; the tiles are divided
// into contiguous runs, one per warp, so that ragged variable lists load-balance and a warp keeps
// the fit's running sums in registers across the tiles of a variable.  Per (variable, warp) one
// partial-sum record goes to the workspace; the warp that completes a variable's last tile adds the
// records in a fixed order and finalises (s, b) -- deterministic, no floating-point atomics, and
// nothing ever waits on another warp.
#pragma once
#include "codec.cuh"
#include "omc_internal.h"

namespace omc {

enum Mode { COMPRESS = 0, DECOMPRESS = 1, UPDATE = 2 };

// How many consecutive elements one lane takes per step: the smallest run whose codes fill
// whole 32-bit words.
template <class F>
struct Unit {
    static constexpr int LU = (F::B % 8 == 0) ? 4 : (F::B % 4 == 0) ? 8 : (F::B % 2 == 0) ? 16 : 32;
    static constexpr int NWORDS = LU * F::B / 32;
    static constexpr int STEP = 32 * LU;          // elements per warp step
    static constexpr int STEPS = TILE / STEP;     // steps per tile
    static constexpr int K = STEPS < 4 ? STEPS : 4;   // steps whose loads are issued together
};

struct Acc {
    double sx, sy, sxy, syy;
    float mn, mx;
    __device__ __forceinline__ void reset()
    {
        sx = sy = sxy = syy = 0.0;
        mn = __int_as_float(0x7F800000);
        mx = __int_as_float(0xFF800000);
    }
    // Sec. 2.3: the sums are taken in fp64; the two products are exact there (24-bit factors).
    __device__ __forceinline__ void add(float w, float vt)
    {
        const double dw = (double)w, dv = (double)vt;
        sx += dw;
        sy += dv;
        sxy = fma(dw, dv, sxy);
        syy = fma(dv, dv, syy);
        mn = fminf(mn, vt);
        mx = fmaxf(mx, vt);
    }
    __device__ __forceinline__ void merge(const Acc &o)
    {
        sx += o.sx; sy += o.sy; sxy += o.sxy; syy += o.syy;
        mn = fminf(mn, o.mn); mx = fmaxf(mx, o.mx);
    }
    __device__ __forceinline__ void warp_reduce()
    {
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            Acc o;
            o.sx = __shfl_xor_sync(0xFFFFFFFFu, sx, d);
            o.sy = __shfl_xor_sync(0xFFFFFFFFu, sy, d);
            o.sxy = __shfl_xor_sync(0xFFFFFFFFu, sxy, d);
            o.syy = __shfl_xor_sync(0xFFFFFFFFu, syy, d);
            o.mn = __shfl_xor_sync(0xFFFFFFFFu, mn, d);
            o.mx = __shfl_xor_sync(0xFFFFFFFFu, mx, d);
            merge(o);
        }
    }
};

// Sec. 2.3 closed form from the four sums (normal equations of min ||s*Vt + b - V||), fp64 with
// every operation rounded separately, stored as FP32.  Degenerate case: s = 1.
__device__ __forceinline__ void fit_from_sums(const Acc &a, uint64_t n, float &s, float &b)
{
    const double nn = (double)n;
    const double num = __dsub_rn(__dmul_rn(nn, a.sxy), __dmul_rn(a.sx, a.sy));
    const double den = __dsub_rn(__dmul_rn(nn, a.syy), __dmul_rn(a.sy, a.sy));
    const bool degenerate = (a.mn == a.mx) || den == 0.0 || !isfinite(den);
    const double s64 = degenerate ? 1.0 : __ddiv_rn(num, den);
    s = __double2float_rn(s64);
    b = __double2float_rn(__ddiv_rn(__dsub_rn(a.sx, __dmul_rn(s64, a.sy)), nn));
}

// Called by a whole warp after it finished `cnt` tiles of a variable.  `slots` are the variable's
// partial-sum records, `my_slot` this warp's record among them, `ticket` the variable's count of
// finished tiles.  Out of line and with scalar arguments only: it runs once per (variable, warp).
static __device__ __noinline__ void flush_and_maybe_finalise(Partial *slots, uint32_t my_slot,
                                                             uint32_t nslots, uint32_t *ticket,
                                                             uint32_t cnt, uint32_t ntiles, uint64_t n,
                                                             float *sb, Acc acc, int lane)
{
    acc.warp_reduce();
    uint32_t last = 0;
    if (lane == 0) {
        Partial q;
        q.sx = acc.sx; q.sy = acc.sy; q.sxy = acc.sxy; q.syy = acc.syy;
        q.mn = acc.mn; q.mx = acc.mx; q.pad[0] = q.pad[1] = 0.f;
        slots[my_slot] = q;
        __threadfence();
        const uint32_t old = atomicAdd(ticket, cnt);
        last = (old + cnt == ntiles);
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    __threadfence();
    Acc tot;
    tot.reset();
    for (uint32_t i = lane; i < nslots; i += 32) {
        const double2 a = __ldcg(reinterpret_cast<const double2 *>(slots + i));
        const double2 c = __ldcg(reinterpret_cast<const double2 *>(slots + i) + 1);
        const float2 m = __ldcg(reinterpret_cast<const float2 *>(slots + i) + 4);
        Acc o;
        o.sx = a.x; o.sy = a.y; o.sxy = c.x; o.syy = c.y; o.mn = m.x; o.mx = m.y;
        tot.merge(o);
    }
    tot.warp_reduce();
    if (lane == 0) {
        float s, b;
        fit_from_sums(tot, n, s, b);
        sb[0] = s;
        sb[1] = b;
        *ticket = 0;      // leave the workspace clean for the next launch
    }
}

template <int N>
__device__ __forceinline__ void load_words(uint32_t (&w)[N], const uint32_t *p)
{
    if constexpr (N == 1) {
        w[0] = *p;
    } else if constexpr (N == 2) {
        const uint2 v = *reinterpret_cast<const uint2 *>(p);
        w[0] = v.x; w[1] = v.y;
    } else if constexpr (N % 4 == 0) {
#pragma unroll
        for (int i = 0; i < N / 4; ++i) {
            const uint4 v = reinterpret_cast<const uint4 *>(p)[i];
            w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) w[i] = p[i];
    }
}

template <int N>
__device__ __forceinline__ void store_words(const uint32_t (&w)[N], uint32_t *p)
{
    if constexpr (N == 1) {
        *p = w[0];
    } else if constexpr (N == 2) {
        *reinterpret_cast<uint2 *>(p) = make_uint2(w[0], w[1]);
    } else if constexpr (N % 4 == 0) {
#pragma unroll
        for (int i = 0; i < N / 4; ++i)
            reinterpret_cast<uint4 *>(p)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) p[i] = w[i];
    }
}

// One tile of a quantised variable.  `n_rem` = elements of the variable from the tile's start on
// (>= TILE for a full tile); `w_rem` = 32-bit words of its code stream from the tile's start on.
template <class F, int MODE, bool WOUT, bool TAIL>
__device__ __forceinline__ void tile_quantised(uint32_t *__restrict__ cw, const float *__restrict__ fin,
                                               float *__restrict__ fout, uint64_t n_rem,
                                               uint64_t w_rem, float s, float b, float neg_lr,
                                               Acc &acc, int lane)
{
    using U = Unit<F>;
    constexpr int LU = U::LU, NW = U::NWORDS, K = U::K;
    constexpr bool HAS_FIN = (MODE != DECOMPRESS);
    constexpr bool HAS_CIN = (MODE != COMPRESS);
    constexpr bool HAS_FOUT = (MODE == DECOMPRESS) || WOUT;
    const uint64_t n_pad = (n_rem + 3) & ~3ull;       // floats that exist in the full layout

#pragma unroll 1
    for (int s0 = 0; s0 < U::STEPS; s0 += K) {
        if (TAIL && (uint64_t)s0 * U::STEP >= n_rem) break;
        uint32_t win[K][NW];
        float4 fv[K][LU / 4];
        // ---- all loads of K steps first: the codes are updated in place, so the compiler could
        //      not move a later step's loads above an earlier step's stores by itself
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const uint32_t unit = (uint32_t)(s0 + k) * 32u + (uint32_t)lane;
            const uint64_t e0 = (uint64_t)unit * LU;
            if constexpr (HAS_CIN) {
                if (!TAIL) {
                    load_words<NW>(win[k], cw + (size_t)unit * NW);
                } else {
#pragma unroll
                    for (int j = 0; j < NW; ++j)
                        win[k][j] = ((uint64_t)unit * NW + j < w_rem) ? cw[(size_t)unit * NW + j] : 0u;
                }
            }
            if constexpr (HAS_FIN) {
#pragma unroll
                for (int j = 0; j < LU / 4; ++j) {
                    if (!TAIL || e0 + 4 * j < n_pad)
                        fv[k][j] = __ldcs(reinterpret_cast<const float4 *>(fin + e0) + j);
                    else
                        fv[k][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
        // ---- compute and store
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const uint32_t unit = (uint32_t)(s0 + k) * 32u + (uint32_t)lane;
            const uint64_t e0 = (uint64_t)unit * LU;
            uint32_t wout[NW];
#pragma unroll
            for (int j = 0; j < NW; ++j) wout[j] = 0u;
#pragma unroll
            for (int g = 0; g < LU / 4; ++g) {
                const float fin4[4] = {fv[k][g].x, fv[k][g].y, fv[k][g].z, fv[k][g].w};
                uint32_t cin[4], cout[4];
                float w[4], vt[4];
                bool bad = false;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if constexpr (HAS_CIN) {
                        cin[j] = get_code<F, NW>(win[k], 4 * g + j);
                        bad |= code_is_special<F>(cin[j]);
                        const float vbar = __fmaf_rn(s, decode_fast<F>(cin[j]), b);
                        w[j] = (MODE == UPDATE) ? __fmaf_rn(neg_lr, fin4[j], vbar) : vbar;
                    } else {
                        w[j] = fin4[j];
                    }
                    if constexpr (MODE != DECOMPRESS) {
                        bad |= needs_exact_encode<F>(w[j]);
                        cout[j] = encode_fast<F>(w[j], vt[j]);
                    }
                }
                if (bad) {   // Inf / NaN / overflow somewhere in these four: redo them carefully
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if constexpr (HAS_CIN) {
                            const float vbar = __fmaf_rn(s, decode_exact<F>(cin[j]), b);
                            w[j] = (MODE == UPDATE) ? __fmaf_rn(neg_lr, fin4[j], vbar) : vbar;
                            // a NaN made by the arithmetic gets one fixed pattern
                            if (MODE == UPDATE && w[j] != w[j]) w[j] = u2f(0x7FFFFFFFu);
                        }
                        if constexpr (MODE != DECOMPRESS) cout[j] = encode_exact<F>(w[j], vt[j]);
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool valid = !TAIL || (e0 + 4 * g + j < n_rem);
                    if constexpr (MODE != DECOMPRESS) {
                        if (valid) {
                            acc.add(w[j], vt[j]);
                            put_code<F, NW>(wout, 4 * g + j, cout[j]);
                        }
                    }
                    if (TAIL && !valid) w[j] = 0.f;
                }
                if constexpr (HAS_FOUT) {
                    if (!TAIL || e0 + 4 * g < n_pad)
                        reinterpret_cast<float4 *>(fout + e0)[g] = make_float4(w[0], w[1], w[2], w[3]);
                }
            }
            if constexpr (MODE != DECOMPRESS) {
                if (!TAIL) {
                    store_words<NW>(wout, cw + (size_t)unit * NW);
                } else {
#pragma unroll
                    for (int j = 0; j < NW; ++j)
                        if ((uint64_t)unit * NW + j < w_rem) cw[(size_t)unit * NW + j] = wout[j];
                }
            }
        }
    }
}

// The ragged last tile of a variable: rare, kept out of line so that it costs the main loop no
// registers.
template <class F, int MODE, bool WOUT>
__device__ __noinline__ Acc tile_quantised_tail(uint32_t *cw, const float *fin, float *fout, uint64_t n_rem,
                                                uint64_t w_rem, float s, float b, float neg_lr, Acc acc,
                                                int lane)
{
    tile_quantised<F, MODE, WOUT, true>(cw, fin, fout, n_rem, w_rem, s, b, neg_lr, acc, lane);
    return acc;
}

// One tile of a variable that stays FP32 (Sec. 2.4): copy in / copy out / plain SGD step.
template <int MODE, bool WOUT>
__device__ __forceinline__ void tile_resid(float *__restrict__ r, const float *__restrict__ fin,
                                           float *__restrict__ fout, uint64_t n_rem, float neg_lr,
                                           int lane)
{
    const uint64_t n4 = ((n_rem < (uint64_t)TILE ? n_rem : (uint64_t)TILE) + 3) / 4;   // float4s
    float4 a[TILE / 128], g[TILE / 128];
#pragma unroll
    for (int j = 0; j < TILE / 128; ++j) {
        const uint32_t i = j * 32 + lane;
        if (i < n4) {
            if constexpr (MODE != COMPRESS) a[j] = reinterpret_cast<const float4 *>(r)[i];
            if constexpr (MODE != DECOMPRESS) g[j] = __ldcs(reinterpret_cast<const float4 *>(fin) + i);
        }
    }
#pragma unroll
    for (int j = 0; j < TILE / 128; ++j) {
        const uint32_t i = j * 32 + lane;
        if (i < n4) {
            if constexpr (MODE == COMPRESS) {
                reinterpret_cast<float4 *>(r)[i] = g[j];
            } else if constexpr (MODE == DECOMPRESS) {
                reinterpret_cast<float4 *>(fout)[i] = a[j];
            } else {
                float4 w;
                w.x = __fmaf_rn(neg_lr, g[j].x, a[j].x);
                w.y = __fmaf_rn(neg_lr, g[j].y, a[j].y);
                w.z = __fmaf_rn(neg_lr, g[j].z, a[j].z);
                w.w = __fmaf_rn(neg_lr, g[j].w, a[j].w);
                reinterpret_cast<float4 *>(r)[i] = w;
                if constexpr (WOUT) reinterpret_cast<float4 *>(fout)[i] = w;
            }
        }
    }
}

template <class F, int MODE, bool WOUT>
__global__ void __launch_bounds__(THREADS, CTAS_PER_SM) omc_kernel(const KParams p)
{
    const int lane = threadIdx.x & 31;
    const uint32_t warp = blockIdx.x * WARPS_PER_CTA + (threadIdx.x >> 5);
    if (warp >= p.nwarps) return;
    uint64_t t = p.tile_begin + (uint64_t)warp * p.tile_count / p.nwarps;
    const uint64_t tend = p.tile_begin + (uint64_t)(warp + 1) * p.tile_count / p.nwarps;
    // variable that holds tile t
    uint32_t lo = p.var_begin, hi = p.var_end;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (__ldg(&p.vars[mid].tile_start) <= t) lo = mid; else hi = mid;
    }
    uint32_t v = lo;
    while (t < tend) {
        VarDev var;
        {
            const VarDev *src = p.vars + v;
            const ulonglong2 a = __ldg(reinterpret_cast<const ulonglong2 *>(src));
            const ulonglong2 c = __ldg(reinterpret_cast<const ulonglong2 *>(src) + 1);
            const uint4 d = __ldg(reinterpret_cast<const uint4 *>(src) + 2);
            const uint4 e = __ldg(reinterpret_cast<const uint4 *>(src) + 3);
            var.n = a.x; var.full_off = a.y; var.store_off = c.x; var.packed_bytes = c.y;
            var.tile_start = ((uint64_t)d.y << 32) | d.x;
            var.ntiles = d.z; var.quantised = d.w;
            var.sb_slot = e.x; var.slot_base = e.y; var.first_warp = e.z; var.nslots = e.w;
        }
        const uint32_t local = (uint32_t)(t - var.tile_start);
        const uint64_t left = tend - t;
        const uint32_t cnt = (uint32_t)((uint64_t)(var.ntiles - local) < left ? (var.ntiles - local) : left);
        if (var.quantised) {
            float s = 1.f, b = 0.f;
            if constexpr (MODE != COMPRESS) {
                s = __ldcg(p.sb + 2 * var.sb_slot);
                b = __ldcg(p.sb + 2 * var.sb_slot + 1);
            }
            Acc acc;
            acc.reset();
            uint32_t *cw_var = reinterpret_cast<uint32_t *>(p.packed + var.store_off);
            for (uint32_t i = 0; i < cnt; ++i) {
                const uint64_t e0 = (uint64_t)(local + i) * TILE;
                const uint64_t w0 = e0 / 32 * F::B;              // first word of the tile's codes
                uint32_t *cw = cw_var + w0;
                const float *fin = (MODE != DECOMPRESS) ? p.fin + var.full_off + e0 : nullptr;
                float *fout = ((MODE == DECOMPRESS) || WOUT) ? p.fout + var.full_off + e0 : nullptr;
                const uint64_t n_rem = var.n - e0;
                if (n_rem >= (uint64_t)TILE)
                    tile_quantised<F, MODE, WOUT, false>(cw, fin, fout, n_rem, 0, s, b, p.neg_lr, acc, lane);
                else
                    acc = tile_quantised_tail<F, MODE, WOUT>(cw, fin, fout, n_rem, var.packed_bytes / 4 - w0,
                                                             s, b, p.neg_lr, acc, lane);
            }
            if constexpr (MODE != DECOMPRESS) {
                if (p.pvt) {
                    flush_and_maybe_finalise(p.slots + var.slot_base, warp - var.first_warp, var.nslots,
                                             p.tickets + var.sb_slot, cnt, var.ntiles, var.n,
                                             p.sb + 2 * var.sb_slot, acc, lane);
                } else if (MODE == COMPRESS && local == 0 && lane == 0) {
                    p.sb[2 * var.sb_slot] = 1.f;
                    p.sb[2 * var.sb_slot + 1] = 0.f;
                }
            }
        } else {
            for (uint32_t i = 0; i < cnt; ++i) {
                const uint64_t e0 = (uint64_t)(local + i) * TILE;
                tile_resid<MODE, WOUT>(p.resid + var.store_off + e0,
                                       (MODE != DECOMPRESS) ? p.fin + var.full_off + e0 : nullptr,
                                       ((MODE == DECOMPRESS) || WOUT) ? p.fout + var.full_off + e0 : nullptr,
                                       var.n - e0, p.neg_lr, lane);
            }
        }
        t += cnt;
        ++v;
    }
}

template <class F, int MODE, bool WOUT>
void launch(const KParams &p, int grid, void *stream)
{
    omc_kernel<F, MODE, WOUT><<<grid, THREADS, 0, static_cast<cudaStream_t>(stream)>>>(p);
}

#define OMC_DEFINE_FORMAT(E_, M_)                                                               \
    extern const FmtOps ops_E##E_##M##M_ = {E_, M_, launch<Fmt<E_, M_>, COMPRESS, false>,       \
                                            launch<Fmt<E_, M_>, DECOMPRESS, false>,             \
                                            launch<Fmt<E_, M_>, UPDATE, false>,                 \
                                            launch<Fmt<E_, M_>, UPDATE, true>};

}  // namespace omc
