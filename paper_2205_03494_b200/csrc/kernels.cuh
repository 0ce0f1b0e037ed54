// The three OMC kernels (compress, decompress, fused update-recompress) as one warp-tiled
// template.
//
// Work is a flat list of 1024-element tiles over all variables; the tiles are divided into
// contiguous runs and warp w takes runs w, w + nwarps, ...  The kernels that fit (s, b) get one
// run per warp, of equal estimated cost, so that ragged variable lists load-balance and a warp
// keeps the fit's running sums in registers across the tiles of a variable; the decoder, which
// keeps no sums, gets short runs of equal length, so that the warps running at the same time
// work on neighbouring memory.  Every warp is its own
// producer/consumer pipeline: lane 0 streams the next granule (a tile or half a tile: packed codes
// and FP32 operand) into one of the warp's shared-memory stages with 1-D TMA bulk copies that
// complete on an mbarrier while the warp computes on the current stage; results go to an output
// buffer and leave through a bulk store.  There is no block-wide barrier anywhere.  Ragged ends of
// variables and FP32-only variables take a plain path with predicated vector loads and stores.
//
// Per (variable, run) one partial-sum record goes to the workspace; the warp that completes a
// variable's last tile adds the records in a fixed order and finalises (s, b): deterministic, no
// floating-point atomics, and no warp ever waits for another.  The only waits are on the warp's
// own copies; they are bounded, and a wait that runs out sets the plan's status word and ends
// the warp.
#pragma once
#include <type_traits>

#include "codec.cuh"
#include "omc_internal.h"

namespace omc {

enum Mode { COMPRESS = 0, DECOMPRESS = 1, UPDATE = 2 };

// Input stages per warp (granules fetched ahead = stages - 1), per kind of kernel: two for each
// (three and four were measured: no gain for the decoder, slower for the others, fewer CTAs fit).
constexpr int MAX_STAGES = 4;               // mbarriers reserved per warp
constexpr int stages_for(int /*mode*/) { return 2; }
constexpr uint32_t WAIT_LIMIT = 1u << 24;   // polls of one mbarrier before giving up

// How many consecutive elements one lane takes per step: the smallest run whose codes fill
// whole 32-bit words.
template <class F>
struct Unit {
    static constexpr int LU = (F::B % 8 == 0) ? 4 : (F::B % 4 == 0) ? 8 : (F::B % 2 == 0) ? 16 : 32;
    static constexpr int NWORDS = LU * F::B / 32;
    static constexpr int STEP = 32 * LU;          // elements per warp step
    // Pipeline granule: the elements one pair of bulk copies brings in and one bulk store takes out.
    // 16-bit codes run best with half-tile granules and two output buffers (measured); the narrower
    // codes, which spend more instructions per byte, with whole tiles and one buffer.
    static constexpr int SUB_DEFAULT = (F::B == 16) ? 512 : TILE;
    static constexpr int SUB = SUB_DEFAULT > STEP ? SUB_DEFAULT : STEP;
    static constexpr int SUB_STEPS = SUB / STEP;
    static constexpr int OUTBUFS = SUB < TILE ? 2 : 1;
    static_assert(TILE % SUB == 0 && (OUTBUFS == 1 || OUTBUFS == 2), "");
    static_assert(LU != 32 || SUB == STEP, "row layout: one 32-element row per lane and granule");
};

// Shared-memory budget of one warp: NSTAGES input stages and OUTBUFS output buffers of one granule.
template <class F, int MODE, bool WOUT>
struct Smem {
    static constexpr int SUB = Unit<F>::SUB;
    static constexpr int OUTBUFS = Unit<F>::OUTBUFS;
    static constexpr bool ROWS = (Unit<F>::LU == 32);   // a lane reads and writes FP32 data as one 128-byte row
    static constexpr int CB = SUB * F::B / 8;     // bytes of one granule's codes
    static constexpr int FB = SUB * 4;            // bytes of one granule's FP32 data
    static constexpr int IN_C = (MODE != COMPRESS) ? CB : 0;
    static constexpr int IN_F = (MODE != DECOMPRESS) ? FB : 0;
    static constexpr int STAGE = IN_C + IN_F;
    static constexpr int TX_BYTES = STAGE;        // what the stage's copies bring in
    static constexpr int NSTAGES = stages_for(MODE);
    static_assert(NSTAGES >= 2 && NSTAGES <= MAX_STAGES, "");
    static constexpr int DIST = NSTAGES - 1;      // granules fetched ahead
    // Row layout, fused round: a lane rewrites its own code words behind its reads, so the new codes
    // take the place of the old ones in the stage and are stored from there.
    static constexpr bool CODES_IN_PLACE = ROWS && MODE == UPDATE;
    static constexpr int OUT_C = (MODE != DECOMPRESS && !CODES_IN_PLACE) ? CB : 0;
    static constexpr int OUT_F = (MODE == DECOMPRESS || WOUT) ? FB : 0;
    static constexpr int OUT = OUT_C + OUT_F;
    static constexpr int PER_WARP = NSTAGES * STAGE + OUTBUFS * OUT;
    static_assert(!ROWS || (STAGE % 128 == 0 && OUT % 128 == 0 && CB % 128 == 0), "row layout: FP32 granules stay 128-byte aligned");
    static constexpr int WARPS = (MODE == DECOMPRESS) ? WARPS_PER_CTA : fit_warps_per_cta(F::B, F::FIXED);
    static constexpr int BAR_PAD = (8 * MAX_STAGES * WARPS + 127) / 128 * 128;   // the mbarriers
    static constexpr int TOTAL = BAR_PAD + WARPS * PER_WARP;
    static_assert(STAGE % 16 == 0 && CB % 16 == 0, "bulk copies move multiples of 16 bytes");
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers: mbarrier and 1-D bulk copies (TMA without a tensor map)

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// Running sums of the Sec. 2.3 fit.

struct Acc {
    double sx, sy, sxy, syy;   // Sum W, Sum Vt, Sum W*Vt, Sum Vt^2
    uint32_t band, bor;        // AND / OR of ValuePattern(Vt): all Vt equal <=> band == bor
    __device__ __forceinline__ void reset()
    {
        sx = sy = sxy = syy = 0.0;
        band = 0xFFFFFFFFu;
        bor = 0u;
    }
    // Sec. 2.3: the sums are taken in fp64; the two products are exact there (24-bit factors).
    __device__ __forceinline__ void add(float w, float vt)
    {
        const double dw = (double)w, dv = (double)vt;
        sx += dw;
        sy += dv;
        sxy = fma(dw, dv, sxy);
        syy = fma(dv, dv, syy);
    }
    // the same with Vt already in fp64 (converted straight from its FP16 pattern)
    __device__ __forceinline__ void add_d(float w, double dv)
    {
        const double dw = (double)w;
        sx += dw;
        sy += dv;
        sxy = fma(dw, dv, sxy);
        syy = fma(dv, dv, syy);
    }
    __device__ __forceinline__ void merge(const Acc &o)
    {
        sx += o.sx; sy += o.sy; sxy += o.sxy; syy += o.syy;
        band &= o.band; bor |= o.bor;
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
            o.band = __shfl_xor_sync(0xFFFFFFFFu, band, d);
            o.bor = __shfl_xor_sync(0xFFFFFFFFu, bor, d);
            merge(o);
        }
    }
};

// Sec. 2.3 closed form from the four sums (normal equations of min ||s*Vt + b - V||), fp64 with
// every operation rounded separately, stored as FP32.  Degenerate case (all Vt equal, which
// includes zeros of mixed sign; or a zero / non-finite denominator): s = 1.
__device__ __forceinline__ void fit_from_sums(const Acc &a, uint64_t n, uint32_t magnitude_mask, float &s,
                                              float &b)
{
    const double nn = (double)n;
    const double num = __dsub_rn(__dmul_rn(nn, a.sxy), __dmul_rn(a.sx, a.sy));
    const double den = __dsub_rn(__dmul_rn(nn, a.syy), __dmul_rn(a.sy, a.sy));
    const bool all_equal = (a.band == a.bor) || ((a.bor & magnitude_mask) == 0u);
    const bool degenerate = all_equal || den == 0.0 || !isfinite(den);
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
                                                             uint32_t magnitude_mask, float *sb, Acc acc,
                                                             int lane)
{
    acc.warp_reduce();
    if (nslots == 1) {      // the variable is this warp's alone: nothing to hand over
        if (lane == 0) {
            float s, b;
            fit_from_sums(acc, n, magnitude_mask, s, b);
            sb[0] = s;
            sb[1] = b;
        }
        return;
    }
    uint32_t last = 0;
    if (lane == 0) {
        Partial q;
        q.sx = acc.sx; q.sy = acc.sy; q.sxy = acc.sxy; q.syy = acc.syy;
        q.band = acc.band; q.bor = acc.bor; q.pad[0] = q.pad[1] = 0u;
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
        const uint2 m = __ldcg(reinterpret_cast<const uint2 *>(slots + i) + 4);
        Acc o;
        o.sx = a.x; o.sy = a.y; o.sxy = c.x; o.syy = c.y; o.band = m.x; o.bor = m.y;
        tot.merge(o);
    }
    tot.warp_reduce();
    if (lane == 0) {
        float s, b;
        fit_from_sums(tot, n, magnitude_mask, s, b);
        sb[0] = s;
        sb[1] = b;
        *ticket = 0;      // leave the workspace clean for the next launch
    }
}

// A 32-bit pattern that identifies the value Q^-1(code) up to the sign of zero; the fit only needs
// to know whether all of a variable's values are equal.  The narrow-float formats use the code in
// all four bytes (so that four codes can be compared per operation), the others the FP32 pattern.
template <class F>
struct WordPath {      // full units are handled a unit's code words at a time (compute_unit_b12)
    static constexpr bool value = (F::B == 12 && HalfPath<F>::value);
};
template <class F>
struct ValuePattern {
    static constexpr bool BY_CODE = Fp8Path<F>::value || WordPath<F>::value;
    static constexpr uint32_t MAGNITUDE_MASK = Fp8Path<F>::value ? F::MAG_MASK * 0x01010101u
                                               : WordPath<F>::value ? F::MAG_MASK : 0x7FFFFFFFu;
    __device__ static __forceinline__ uint32_t of(uint32_t code, float vt)
    {
        if constexpr (Fp8Path<F>::value) return code * 0x01010101u;
        if constexpr (WordPath<F>::value) return code;
        return f2u(vt);
    }
};

// Equality of all the codes a lane has produced in full units since reset(), kept on whole code
// words (every unit starts at a multiple of LU elements, so equal codes mean equal words from unit
// to unit): one logic operation per word instead of one per element.  fold() hands the result to
// the running sums' AND / OR trackers.
template <class F>
struct EqTracker {
    static constexpr bool USED = WordPath<F>::value;
    static constexpr int NW = USED ? Unit<F>::NWORDS : 1;
    uint32_t ref[NW], diff, seen;
    __device__ __forceinline__ void reset()
    {
        diff = 0u;
        seen = 0u;
#pragma unroll
        for (int j = 0; j < NW; ++j) ref[j] = 0u;
    }
    // `first`: this is the warp's first unit since reset().  A lane whose first unit took the careful
    // path instead keeps the reference 0 and reports "different" from then on, which is the truth:
    // that unit held an Inf or NaN code and the units that come here never do.
    __device__ __forceinline__ void unit(const uint32_t (&w)[NW], bool first)
    {
        if (first) {
#pragma unroll
            for (int j = 0; j < NW; ++j) ref[j] = w[j];
        }
#pragma unroll
        for (int j = 0; j < NW; ++j) diff |= w[j] ^ ref[j];
        seen = 1u;
    }
    __device__ __forceinline__ void fold(Acc &acc) const
    {
        if constexpr (USED) {
            if (!seen) return;
            // the reference unit itself: LU equal codes c give these words
            const uint32_t c = ref[0] & F::CODE_MASK;
            uint32_t d = diff;
#pragma unroll
            for (int j = 0; j < NW; ++j) {
                uint32_t e = 0u;
#pragma unroll
                for (int k = 0; k < Unit<F>::LU; ++k) {
                    const int pos = k * F::B - 32 * j;
                    if (pos > -F::B && pos < 32) e |= pos >= 0 ? c << pos : c >> -pos;
                }
                d |= e ^ ref[j];
            }
            const uint32_t all = d ? 0xFFFFFFFFu : 0u;
            acc.band &= c & ~all;
            acc.bor |= c | all;
        }
    }
};

// ---------------------------------------------------------------------------------------------
// Arithmetic of one lane's unit: LU consecutive elements held in registers.
//   win  : the unit's codes (read unless COMPRESS)       fv : the unit's FP32 operand (params / grads)
//   wout : the unit's new codes (written unless DECOMPRESS)  fo : FP32 result (decompressed value / W)
//   valid: number of leading elements that exist (LU except in a ragged tile)

// A loop whose index is a compile-time constant in every iteration (what "#pragma unroll" only
// asks for): bit positions inside the code stream must fold to immediates.
template <int I, int N>
struct StaticFor {
    template <class Fn>
    __device__ __forceinline__ static void run(Fn &&fn)
    {
        fn(std::integral_constant<int, I>{});
        StaticFor<I + 1, N>::run(fn);
    }
};
template <int N>
struct StaticFor<N, N> {
    template <class Fn>
    __device__ __forceinline__ static void run(Fn &&) {}
};

// Four consecutive elements (group g of the unit): codes from `win`, FP32 operand `fin4`; results
// into `wout` (codes), `w` (FP32 values), the running sums and the equality trackers ref / diff.
// `win` / `wout` hold the bits from position `bitbase` of the unit's code stream on (bitbase = 0
// when they hold the whole unit).
template <class F, int MODE, bool TAIL, int NWI, int NWO>
__device__ __forceinline__ void compute_group(const uint32_t (&win)[NWI], int g, const float (&fin4)[4],
                                              uint32_t (&wout)[NWO], float (&w)[4], float s, float b,
                                              float neg_lr, Acc &acc, uint32_t &ref, uint32_t &diff, int valid,
                                              int bitbase = 0)
{
    constexpr bool HAS_CIN = (MODE != COMPRESS);
    constexpr bool KEEP_PAYLOAD = (MODE == COMPRESS);    // UPDATE gives arithmetic NaNs one pattern
    constexpr bool GENERIC = !F::FIXED && F::E < 8 && !HalfPath<F>::value;   // codes are isolated only on the careful path
    uint32_t cin[4], cout[4];
    float vt[4];
    bool bad = false;
    if constexpr (HAS_CIN) {
        float dec[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if constexpr (GENERIC) {
                dec[j] = decode_fast_at<F, NWI>(win, (4 * g + j) * F::B - bitbase);
            } else {
                cin[j] = get_code_at<F, NWI>(win, (4 * g + j) * F::B - bitbase);
                dec[j] = decode_fast<F>(cin[j]);
            }
            const float vbar = __fmaf_rn(s, dec[j], b);
            w[j] = (MODE == UPDATE) ? __fmaf_rn(neg_lr, fin4[j], vbar) : vbar;
        }
        bad = any_code_special4<F>(dec);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j] = fin4[j];
    }
    if constexpr (MODE != DECOMPRESS) bad |= any_needs_exact_encode4<F, KEEP_PAYLOAD>(w);
    if constexpr (MODE != DECOMPRESS) {
        encode_fast2<F>(w[0], w[1], cout[0], cout[1], vt[0], vt[1]);
        encode_fast2<F>(w[2], w[3], cout[2], cout[3], vt[2], vt[3]);
    }
    if (bad) {   // Inf / NaN / overflow somewhere in these four: redo them carefully
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if constexpr (HAS_CIN) {
                if constexpr (GENERIC) cin[j] = get_code_at<F, NWI>(win, (4 * g + j) * F::B - bitbase);
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
        const bool ok = !TAIL || (4 * g + j < valid);
        if constexpr (MODE != DECOMPRESS) {
            if (ok) {
                acc.add(w[j], vt[j]);
                put_code_at<F, NWO>(wout, (4 * g + j) * F::B - bitbase, cout[j]);
                const uint32_t pat = ValuePattern<F>::of(cout[j], vt[j]);
                if (g == 0 && j == 0) ref = pat;             // element 0 exists whenever the unit does
                else diff |= pat ^ ref;
            }
        }
        if (TAIL && !ok) w[j] = 0.f;
    }
}

template <class F, int MODE, bool TAIL>
__device__ __forceinline__ void compute_unit(const uint32_t (&win)[Unit<F>::NWORDS], const float4 (&fv)[Unit<F>::LU / 4],
                                             uint32_t (&wout)[Unit<F>::NWORDS], float4 (&fo)[Unit<F>::LU / 4],
                                             float s, float b, float neg_lr, Acc &acc, int valid)
{
    constexpr int LU = Unit<F>::LU, NW = Unit<F>::NWORDS;
#pragma unroll
    for (int j = 0; j < NW; ++j) wout[j] = 0u;
    uint32_t ref = 0u, diff = 0u;
#pragma unroll
    for (int g = 0; g < LU / 4; ++g) {
        const float fin4[4] = {fv[g].x, fv[g].y, fv[g].z, fv[g].w};
        float w[4];
        compute_group<F, MODE, TAIL, NW, NW>(win, g, fin4, wout, w, s, b, neg_lr, acc, ref, diff, valid);
        fo[g] = make_float4(w[0], w[1], w[2], w[3]);
    }
    if constexpr (MODE != DECOMPRESS) {
        if (!TAIL || valid > 0) {
            acc.band &= ref & ~diff;
            acc.bor |= ref | diff;
        }
    }
}

// A full unit of 32 elements per lane (odd code widths) whose FP32 operand and FP32 result live in
// shared-memory rows: the operand is fetched four elements at a time right where it is used and
// the result is stored at once, so that a lane never holds 32 values in registers.
//
// Row layout of a granule of 1024 FP32 values (4 KB, 128-byte aligned): lane l owns values
// 32 l .. 32 l + 31, a 128-byte row, and its 16-byte chunk c sits at chunk c xor (l mod 8) of
// the row, so that the eight lanes of a quarter warp touch all 32 banks.  The bulk copies move
// dense granules; the warp swizzles them in place (eight 16-byte loads, eight stores per lane).
__device__ __forceinline__ void rows_swizzle_in_place(float *granule, int lane, bool to_rows)
{
    float4 *g4 = reinterpret_cast<float4 *>(granule);
    float4 v[8];
    // float4 number 32 i + lane of the dense granule is chunk lane mod 8 of row 4 i + lane / 8
    const int c = lane & 7;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + (lane >> 3);
        v[i] = g4[to_rows ? 32 * i + lane : r * 8 + (c ^ (r & 7))];
    }
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + (lane >> 3);
        g4[to_rows ? r * 8 + (c ^ (r & 7)) : 32 * i + lane] = v[i];
    }
    __syncwarp();
}

__device__ __forceinline__ uint32_t lds_volatile(uint32_t shared_addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(shared_addr));
    return v;
}

// Everything is streamed, four elements at a time: the code words and the operand are fetched
// right where they are used (volatile loads, so that the compiler does not hoist them all to the
// top), finished output words are stored at once, and a word shared by two groups is carried in
// one register.  `cin` / `cout` / `fin_row` / `fout_row` are this lane's slices in shared memory.
template <class F, int MODE, bool WOUT>
__device__ __forceinline__ void compute_unit_rows(const uint32_t *cin, const float *fin_granule, uint32_t *cout,
                                                  float *fout_granule, float s, float b, float neg_lr, Acc &acc, int lane)
{
    constexpr int LU = Unit<F>::LU, B = F::B;
    constexpr int GW = (4 * B + 31) / 32 + 1;      // words a group of four codes can touch
    uint32_t ref = 0u, diff = 0u, carry = 0u;
    const uint32_t cin_a = smem_addr(cin);                                 // shared-window addresses, once
    // chunk g of this lane's row: (row | swizzle) xor 16 g, the granule being 128-byte aligned
    const uint32_t row_sw = (uint32_t)lane * 128u + (((uint32_t)lane & 7u) << 4);
    const uint32_t fin_a = smem_addr(fin_granule) + row_sw, fout_a = smem_addr(fout_granule) + row_sw;
    StaticFor<0, LU / 4>::run([&](auto gi) {
        constexpr int g = decltype(gi)::value;
        constexpr int bit0 = 4 * g * B, f0 = bit0 >> 5, cnt = ((bit0 + 4 * B - 1) >> 5) - f0 + 1;
        constexpr bool ends_on_word = ((bit0 + 4 * B) & 31) == 0;
        uint32_t gw[GW], ow[GW];
#pragma unroll
        for (int q = 0; q < GW; ++q) {
            gw[q] = (MODE != COMPRESS && q < cnt) ? lds_volatile(cin_a + 4u * (f0 + q)) : 0u;
            ow[q] = 0u;
        }
        ow[0] = carry;
        float fin4[4] = {0.f, 0.f, 0.f, 0.f};
        if constexpr (MODE != DECOMPRESS) {
            float4 v;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                         : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(fin_a ^ (16u * g)));
            fin4[0] = v.x; fin4[1] = v.y; fin4[2] = v.z; fin4[3] = v.w;
        }
        float w[4];
        compute_group<F, MODE, false, GW, GW>(gw, g, fin4, ow, w, s, b, neg_lr, acc, ref, diff, LU, 32 * f0);
        if constexpr (MODE != DECOMPRESS) {
#pragma unroll
            for (int q = 0; q < GW; ++q)
                if (q < cnt - 1 || (q == cnt - 1 && ends_on_word)) cout[f0 + q] = ow[q];
            carry = ends_on_word ? 0u : ow[cnt - 1];
        }
        if constexpr (MODE == DECOMPRESS || WOUT)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};"
                         ::"r"(fout_a ^ (16u * g)), "f"(w[0]), "f"(w[1]), "f"(w[2]), "f"(w[3]) : "memory");
    });
    if constexpr (MODE != DECOMPRESS) {
        acc.band &= ref & ~diff;
        acc.bor |= ref | diff;
    }
}

// ---------------------------------------------------------------------------------------------
// Full units of the formats whose finite codes are the codes of a hardware narrow-float type
// (S1E5M2 = e5m2, S1E4M3 = e4m3 up to exponent field 14, S1E2M3 = e2m3 up to field 2).  The
// conversion instructions keep one code per byte and do the rounding (to nearest even, gradual
// underflow) and the unpacking two elements at a time; four codes travel in one register.  The
// hardware types differ from the paper's family at the top of the range only (saturation instead
// of infinity; e4m3 and e2m3 have finite values where the family has Inf/NaN), and every code that
// high, read or produced, sends the unit to compute_unit.

// Four codes, one per byte -> two pairs of FP16 patterns (exact).
template <class F>
__device__ __forceinline__ void fp8x4_halves(uint32_t cw, uint32_t &h01, uint32_t &h23)
{
    if constexpr (F::E == 5) {                   // a code is the top byte of its FP16 pattern
        h01 = __byte_perm(cw, 0u, 0x1404);
        h23 = __byte_perm(cw, 0u, 0x3424);
    } else if constexpr (F::E == 4) {
        asm("{\n\t.reg .b16 lo, hi;\n\t"
            "mov.b32 {lo, hi}, %2;\n\t"
            "cvt.rn.f16x2.e4m3x2 %0, lo;\n\t"
            "cvt.rn.f16x2.e4m3x2 %1, hi;\n\t}"
            : "=r"(h01), "=r"(h23) : "r"(cw));
    } else {
        asm("{\n\t.reg .b16 lo, hi;\n\t"
            "mov.b32 {lo, hi}, %2;\n\t"
            "cvt.rn.f16x2.e2m3x2 %0, lo;\n\t"
            "cvt.rn.f16x2.e2m3x2 %1, hi;\n\t}"
            : "=r"(h01), "=r"(h23) : "r"(cw));
    }
}

template <class F>
__device__ __forceinline__ void fp8x4_decode(uint32_t cw, float (&v)[4])
{
    uint32_t h01, h23;
    fp8x4_halves<F>(cw, h01, h23);
    const __half2 a = *reinterpret_cast<const __half2 *>(&h01), c = *reinterpret_cast<const __half2 *>(&h23);
    v[0] = __low2float(a); v[1] = __high2float(a);
    v[2] = __low2float(c); v[3] = __high2float(c);
}

// A pair of FP16 patterns -> two fp64 values, without the detour through FP32.
__device__ __forceinline__ void half2_to_doubles(uint32_t h2, double &lo, double &hi)
{
    asm("{\n\t.reg .b16 l, h;\n\t"
        "mov.b32 {l, h}, %2;\n\t"
        "cvt.f64.f16 %0, l;\n\t"
        "cvt.f64.f16 %1, h;\n\t}"
        : "=d"(lo), "=d"(hi) : "r"(h2));
}

// Four FP32 values -> four codes, one per byte (element 0 in the low byte).  Saturating: a
// magnitude beyond the type's largest finite value gives that value; a NaN gives the type's NaN,
// or, in e2m3, which has none, its largest value.
template <class F>
__device__ __forceinline__ uint32_t fp8x4_encode(const float (&w)[4])
{
    uint32_t cw;
    if constexpr (F::E == 5)
        asm("{\n\t.reg .b16 lo, hi;\n\t"
            "cvt.rn.satfinite.e5m2x2.f32 lo, %2, %1;\n\t"
            "cvt.rn.satfinite.e5m2x2.f32 hi, %4, %3;\n\t"
            "mov.b32 %0, {lo, hi};\n\t}"
            : "=r"(cw) : "f"(w[0]), "f"(w[1]), "f"(w[2]), "f"(w[3]));
    else if constexpr (F::E == 4)
        asm("{\n\t.reg .b16 lo, hi;\n\t"
            "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
            "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
            "mov.b32 %0, {lo, hi};\n\t}"
            : "=r"(cw) : "f"(w[0]), "f"(w[1]), "f"(w[2]), "f"(w[3]));
    else
        asm("{\n\t.reg .b16 lo, hi;\n\t"
            "cvt.rn.satfinite.e2m3x2.f32 lo, %2, %1;\n\t"
            "cvt.rn.satfinite.e2m3x2.f32 hi, %4, %3;\n\t"
            "mov.b32 %0, {lo, hi};\n\t}"
            : "=r"(cw) : "f"(w[0]), "f"(w[1]), "f"(w[2]), "f"(w[3]));
    return cw;
}

// Non-zero iff one of the four codes (one per byte) has a magnitude of at least TOP.
template <class F, uint32_t TOP>
__device__ __forceinline__ uint32_t fp8x4_any_at_least(uint32_t cw)
{
    return ((cw & (F::MAG_MASK * 0x01010101u)) + (0x80u - TOP) * 0x01010101u) & 0x80808080u;
}

// 6-bit codes: 24 bits of the packed stream <-> four codes, one per byte.
__device__ __forceinline__ uint32_t spread6(uint32_t t)
{
    return (t & 0x3Fu) | ((t << 2) & 0x3F00u) | ((t << 4) & 0x3F0000u) | ((t << 6) & 0x3F000000u);
}
__device__ __forceinline__ uint32_t gather6(uint32_t c)
{
    return (c & 0x3Fu) | ((c >> 2) & 0xFC0u) | ((c >> 4) & 0x3F000u) | ((c >> 6) & 0xFC0000u);
}

// Out-of-line compute_group for the rare group of four that holds a code from the top of the
// range: `g` is a run-time value here and everything lives behind pointers, so that the main path
// keeps its registers.  New codes are OR-ed into wout_p (as compute_group does).
template <class F, int MODE>
__device__ __noinline__ void compute_group_careful(const uint32_t *win_p, int g, float4 f4, uint32_t *wout_p,
                                                   float *w_p, float s, float b, float neg_lr, Acc *acc_p,
                                                   uint32_t *ref_p, uint32_t *diff_p)
{
    constexpr int NW = Unit<F>::NWORDS;
    uint32_t win[NW], wout[NW];
#pragma unroll
    for (int j = 0; j < NW; ++j) {
        win[j] = win_p[j];
        wout[j] = wout_p[j];
    }
    const float fin4[4] = {f4.x, f4.y, f4.z, f4.w};
    float w[4];
    Acc acc = *acc_p;
    uint32_t ref = *ref_p, diff = *diff_p;
    if (g == 0)     // compute_group takes element 0's pattern as the reference when g is 0
        compute_group<F, MODE, false, NW, NW>(win, 0, fin4, wout, w, s, b, neg_lr, acc, ref, diff, Unit<F>::LU);
    else
        compute_group<F, MODE, false, NW, NW>(win, g, fin4, wout, w, s, b, neg_lr, acc, ref, diff, Unit<F>::LU);
    *acc_p = acc;
    *ref_p = ref;
    *diff_p = diff;
#pragma unroll
    for (int j = 0; j < NW; ++j) wout_p[j] = wout[j];
#pragma unroll
    for (int j = 0; j < 4; ++j) w_p[j] = w[j];
}

template <class F, int MODE>
__device__ __forceinline__ void compute_unit_fp8(const uint32_t (&win)[Unit<F>::NWORDS],
                                                 const float4 (&fv)[Unit<F>::LU / 4],
                                                 uint32_t (&wout)[Unit<F>::NWORDS], float4 (&fo)[Unit<F>::LU / 4],
                                                 float s, float b, float neg_lr, Acc &acc)
{
    constexpr int LU = Unit<F>::LU, NW = Unit<F>::NWORDS, NG = LU / 4;
    static_assert((F::B == 8 && NG == 1) || (F::B == 6 && NG == 4 && NW == 3), "one byte or six bits per code");
    // Codes from here up are not handled by the hardware type as the format wants them: Inf/NaN
    // codes when read (e5m2 alone decodes them as such); when written, the largest finite code
    // too (saturation hides an overflow behind it) and with it every Inf/NaN.
    constexpr uint32_t TOP_IN = F::INF_MAG, TOP_OUT = F::INF_MAG - 1u;
    uint32_t cin[NG], cout[NG];
    if constexpr (MODE != COMPRESS) {
        if constexpr (F::B == 8) {
            cin[0] = win[0];
        } else {            // group g is bits [24 g, 24 g + 24) of the unit's three words
            cin[0] = spread6(win[0]);
            cin[1] = spread6(__funnelshift_r(win[0], win[1], 24));
            cin[2] = spread6(__funnelshift_r(win[1], win[2], 16));
            cin[3] = spread6(win[2] >> 8);
        }
    }
    uint32_t diff = 0u, ref = 0u;
    uint32_t wout_sp[NW];       // codes written by the careful path, already at their place in the stream
#pragma unroll
    for (int j = 0; j < NW; ++j) wout_sp[j] = 0u;
#pragma unroll
    for (int g = 0; g < NG; ++g) {
        float w[4];
        uint32_t special = 0u, vh01 = 0u, vh23 = 0u;
        if constexpr (MODE != COMPRESS) {
            float dec[4];
            fp8x4_decode<F>(cin[g], dec);
            if constexpr (F::E != 5) special = fp8x4_any_at_least<F, TOP_IN>(cin[g]);
            const float gr[4] = {fv[g].x, fv[g].y, fv[g].z, fv[g].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float vbar = __fmaf_rn(s, dec[j], b);
                w[j] = (MODE == UPDATE) ? __fmaf_rn(neg_lr, gr[j], vbar) : vbar;
            }
        } else {
            w[0] = fv[g].x; w[1] = fv[g].y; w[2] = fv[g].z; w[3] = fv[g].w;
        }
        if constexpr (MODE != DECOMPRESS) {
            cout[g] = fp8x4_encode<F>(w);
            special |= fp8x4_any_at_least<F, TOP_OUT>(cout[g]);
            fp8x4_halves<F>(cout[g], vh01, vh23);        // Q^-1 of the new codes, as FP16 patterns
        }
        if (special) {
            // on copies, so that only they (and not the registers of the main path) have addresses
            uint32_t win_c[NW];
            float w_c[4];
            Acc acc_c = acc;
            uint32_t ref_c = ref, diff_c = diff;
#pragma unroll
            for (int j = 0; j < NW; ++j) win_c[j] = (MODE != COMPRESS) ? win[j] : 0u;
            compute_group_careful<F, MODE>(win_c, g, fv[g], wout_sp, w_c, s, b, neg_lr, &acc_c, &ref_c, &diff_c);
            acc = acc_c;
            ref = ref_c;
            diff = diff_c;
#pragma unroll
            for (int j = 0; j < 4; ++j) w[j] = w_c[j];
            if constexpr (MODE != DECOMPRESS) cout[g] = 0u;
        } else if constexpr (MODE != DECOMPRESS) {
            double dv[4];
            half2_to_doubles(vh01, dv[0], dv[1]);
            half2_to_doubles(vh23, dv[2], dv[3]);
#pragma unroll
            for (int j = 0; j < 4; ++j) acc.add_d(w[j], dv[j]);
            if (g == 0) ref = __byte_perm(cout[0], 0u, 0x0000);     // element 0's code in all four bytes
            diff |= cout[g] ^ ref;
        }
        fo[g] = make_float4(w[0], w[1], w[2], w[3]);
    }
    if constexpr (MODE != DECOMPRESS) {
        acc.band &= ref & ~diff;
        acc.bor |= ref | diff;
        if constexpr (F::B == 8) {
            wout[0] = cout[0] | wout_sp[0];
        } else {
            const uint32_t t0 = gather6(cout[0]), t1 = gather6(cout[1]), t2 = gather6(cout[2]), t3 = gather6(cout[3]);
            wout[0] = t0 | (t1 << 24) | wout_sp[0];
            wout[1] = (t1 >> 8) | (t2 << 16) | wout_sp[1];
            wout[2] = (t2 >> 16) | (t3 << 8) | wout_sp[2];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Full units of S1E5M6: eight 12-bit codes in three words.  A code << 4 is an IEEE half, and the
// half-to-float conversion reads either half of a register, so a code is moved to bits 4..15 (or
// 20..31) of a register with one or two operations and everything above or beside it is ignored;
// new codes leave the packed conversion as pairs of halves and are squeezed into 24 bits per pair
// and byte-permuted into the three words.  A unit in which a value overflows (the fast rounding
// would keep it finite) is redone by compute_unit.

// A whole unit on the careful path, out of line, from and to the unit's places in shared memory, so
// that the main path keeps its registers and prepares nothing for it.
template <class F, int MODE, bool WOUT>
__device__ __noinline__ Acc compute_unit_careful(const uint32_t *cin, const float *fin, uint32_t *cout, float *fout,
                                                 float s, float b, float neg_lr, Acc acc)
{
    constexpr int LU = Unit<F>::LU, NW = Unit<F>::NWORDS;
    uint32_t win[NW], wout[NW];
    float4 fv[LU / 4], fo[LU / 4];
#pragma unroll
    for (int j = 0; j < NW; ++j) win[j] = (MODE != COMPRESS) ? cin[j] : 0u;
#pragma unroll
    for (int j = 0; j < LU / 4; ++j)
        fv[j] = (MODE != DECOMPRESS) ? reinterpret_cast<const float4 *>(fin)[j] : make_float4(0.f, 0.f, 0.f, 0.f);
    compute_unit<F, MODE, false>(win, fv, wout, fo, s, b, neg_lr, acc, LU);
    if constexpr (MODE != DECOMPRESS) {
#pragma unroll
        for (int j = 0; j < NW; ++j) cout[j] = wout[j];
    }
    if constexpr (MODE == DECOMPRESS || WOUT) {
#pragma unroll
        for (int j = 0; j < LU / 4; ++j) reinterpret_cast<float4 *>(fout)[j] = fo[j];
    }
    return acc;
}

__device__ __forceinline__ float half_lo(uint32_t r)
{
    return __low2float(*reinterpret_cast<const __half2 *>(&r));
}
__device__ __forceinline__ float half_hi(uint32_t r)
{
    return __high2float(*reinterpret_cast<const __half2 *>(&r));
}
__device__ __forceinline__ float max3_nan(float a, float b, float c)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Returns false, with nothing accumulated or produced, when the unit has to take the careful path.
template <class F, int MODE>
__device__ __forceinline__ bool compute_unit_b12(const uint32_t (&win)[3], const float4 (&fv)[2], uint32_t (&wout)[3],
                                                 float4 (&fo)[2], float s, float b, float neg_lr, Acc &acc,
                                                 EqTracker<F> &eq, bool first)
{
    static_assert(F::B == 12 && HalfPath<F>::value && Unit<F>::LU == 8, "S1E5M6");
    float w[8];
    if constexpr (MODE != COMPRESS) {
        const uint32_t w0 = win[0], w1 = win[1], w2 = win[2];
        float dec[8];
        dec[0] = half_lo(w0 << 4);                                   // code 0: bits 0..11
        dec[1] = half_lo((w0 >> 8) & 0xFFF0u);                       // code 1: bits 12..23
        dec[2] = half_lo(__funnelshift_r(w0, w1, 24) << 4);          // code 2: bits 24..35
        dec[3] = half_lo(w1 & 0xFFF0u);                              // code 3: bits 4..15 of word 1
        dec[4] = half_lo((w1 >> 12) & 0xFFF0u);                      // code 4: bits 16..27 of word 1
        dec[5] = half_lo(__funnelshift_r(w1, w2, 28) << 4);          // code 5: bits 28..39 of word 1
        dec[6] = half_lo((w2 >> 4) & 0xFFF0u);                       // code 6: bits 8..19 of word 2
        dec[7] = half_hi(w2 & 0xFFF00000u);                          // code 7: bits 20..31 of word 2
        const float g[8] = {fv[0].x, fv[0].y, fv[0].z, fv[0].w, fv[1].x, fv[1].y, fv[1].z, fv[1].w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float vbar = __fmaf_rn(s, dec[j], b);
            w[j] = (MODE == UPDATE) ? __fmaf_rn(neg_lr, g[j], vbar) : vbar;
        }
    } else {
        w[0] = fv[0].x; w[1] = fv[0].y; w[2] = fv[0].z; w[3] = fv[0].w;
        w[4] = fv[1].x; w[5] = fv[1].y; w[6] = fv[1].z; w[7] = fv[1].w;
    }
    fo[0] = make_float4(w[0], w[1], w[2], w[3]);
    fo[1] = make_float4(w[4], w[5], w[6], w[7]);
    if constexpr (MODE != DECOMPRESS) {
        // Inf, NaN or a value that rounds to infinity among the eight: the careful path
        const float m = max3_nan(max3_nan(fabsf(w[0]), fabsf(w[1]), fabsf(w[2])),
                                 max3_nan(fabsf(w[3]), fabsf(w[4]), fabsf(w[5])), max3_nan(fabsf(w[6]), fabsf(w[7]), 0.f));
        if (!(m < u2f(F::OVF_BITS))) return false;
        float vt[8];
        uint32_t pr[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            // The software rounding of encode_fast2 with the adder's constant 2^(max(e, EMIN) + 23 - M)
            // written as 2^max(e, EMIN) * 2^(23 - M): the product is exact, so each fused
            // multiply-add rounds exactly what the addition and the subtraction would.
            const float w0_ = w[2 * k], w1_ = w[2 * k + 1];
            const uint32_t u0 = f2u(w0_), u1 = f2u(w1_);
            const float m0 = u2f(max(u0 & 0x7F800000u, F::pow2_bits(F::EMIN)));
            const float m1 = u2f(max(u1 & 0x7F800000u, F::pow2_bits(F::EMIN)));
            constexpr float K = (float)(1u << F::SH);
            const float r0 = __fmaf_rn(m0, -K, __fmaf_rn(m0, K, fabsf(w0_)));
            const float r1 = __fmaf_rn(m1, -K, __fmaf_rn(m1, K, fabsf(w1_)));
            vt[2 * k] = u2f(f2u(r0) | (u0 & 0x80000000u));
            vt[2 * k + 1] = u2f(f2u(r1) | (u1 & 0x80000000u));
            const __half2 h = __floats2half2_rn(vt[2 * k], vt[2 * k + 1]);   // exact: both are FP16 values
            const uint32_t x = *reinterpret_cast<const uint32_t *>(&h);      // code 2k << 4 | code 2k+1 << 20
            // the pair as 24 bits: code 2k in bits 0..11, code 2k+1 in bits 12..23
            const uint32_t lo = x >> 4, hi = x >> 8;
            pr[k] = (lo & 0xFFFu) | (hi & ~0xFFFu);
        }
        wout[0] = __byte_perm(pr[0], pr[1], 0x4210);
        wout[1] = __byte_perm(pr[1], pr[2], 0x5421);
        wout[2] = __byte_perm(pr[2], pr[3], 0x6542);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc.add(w[j], vt[j]);
        eq.unit(wout, first);
    }
    return true;
}

// ---------------------------------------------------------------------------------------------
// Register <-> memory moves of a unit (global or shared: the address space is inferred).

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

// A full granule (SUB elements) whose inputs sit in the warp's shared-memory stage.
template <class F, int MODE, bool WOUT>
__device__ __forceinline__ void granule_from_smem(const uint32_t *s_cin, const float *s_fin, uint32_t *s_cout,
                                                  float *s_fout, float s, float b, float neg_lr, Acc &acc,
                                                  EqTracker<F> &eq, bool first_granule, int lane)
{
    using U = Unit<F>;
    constexpr int LU = U::LU, NW = U::NWORDS;
    if constexpr (LU == 32) {       // one unit per lane; FP32 data in swizzled 128-byte rows
        compute_unit_rows<F, MODE, WOUT>(s_cin + lane * NW, s_fin, s_cout + lane * NW, s_fout, s, b, neg_lr, acc, lane);
        return;
    }
    constexpr int G = (U::SUB_STEPS >= 2 && LU == 4) ? 2 : 1;   // steps whose operands are fetched together
    constexpr int UNROLL = (F::B == 8 || F::B == 12) ? 4 : 1;     // measured
#pragma unroll UNROLL
    for (int k0 = 0; k0 < U::SUB_STEPS; k0 += G) {
        uint32_t win[G][NW];
        float4 fv[G][LU / 4];
        // fetch first, so that the loads of both steps are in flight before the arithmetic starts
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int unit = (k0 + g) * 32 + lane;
            if constexpr (MODE != COMPRESS) load_words<NW>(win[g], s_cin + unit * NW);
            if constexpr (MODE != DECOMPRESS) {
#pragma unroll
                for (int j = 0; j < LU / 4; ++j) fv[g][j] = reinterpret_cast<const float4 *>(s_fin + unit * LU)[j];
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int unit = (k0 + g) * 32 + lane;
            uint32_t wout[NW];
            float4 fo[LU / 4];
            if constexpr (Fp8Path<F>::value)
                compute_unit_fp8<F, MODE>(win[g], fv[g], wout, fo, s, b, neg_lr, acc);
            else if constexpr (WordPath<F>::value) {
                if (!compute_unit_b12<F, MODE>(win[g], fv[g], wout, fo, s, b, neg_lr, acc, eq,
                                               first_granule && k0 + g == 0)) {
                    acc = compute_unit_careful<F, MODE, WOUT>(s_cin + unit * NW, s_fin + unit * LU, s_cout + unit * NW,
                                                              s_fout + unit * LU, s, b, neg_lr, acc);
                    continue;
                }
            } else
                compute_unit<F, MODE, false>(win[g], fv[g], wout, fo, s, b, neg_lr, acc, LU);
            if constexpr (MODE != DECOMPRESS) store_words<NW>(wout, s_cout + unit * NW);
            if constexpr (MODE == DECOMPRESS || WOUT) {
#pragma unroll
                for (int j = 0; j < LU / 4; ++j) reinterpret_cast<float4 *>(s_fout + unit * LU)[j] = fo[j];
            }
        }
    }
}

// The ragged end of a variable (fewer than SUB elements), straight from and to global memory
// with predicated accesses.  `n_rem` = elements left in the variable; `w_rem` = 32-bit words left
// in its padded code stream.  All loads are issued before the arithmetic starts, so that the warp
// waits for memory once and not once per step.  Out of line: it runs once per (variable, warp) at
// most and must cost the main loop no registers.
template <class F, int MODE, bool WOUT>
__device__ __noinline__ Acc tile_ragged(uint32_t *cw, const float *fin, float *fout, uint32_t n_rem,
                                        uint32_t w_rem, float s, float b, float neg_lr, Acc acc, int lane)
{
    using U = Unit<F>;
    constexpr int LU = U::LU, NW = U::NWORDS, NS = U::SUB_STEPS;
    static_assert(NS * (NW + LU) <= 64, "the ragged end is held in registers");
    const uint32_t n_pad = (n_rem + 3u) & ~3u;       // floats that exist in the full layout
    uint32_t win[NS][NW];
    float4 fv[NS][LU / 4];
#pragma unroll
    for (int k = 0; k < NS; ++k) {
        const uint32_t unit = (uint32_t)k * 32u + (uint32_t)lane;
        const uint32_t e0 = unit * LU;
        if constexpr (MODE != COMPRESS) {
#pragma unroll
            for (int j = 0; j < NW; ++j) win[k][j] = (unit * NW + j < w_rem) ? cw[unit * NW + j] : 0u;
        }
        if constexpr (MODE != DECOMPRESS) {
#pragma unroll
            for (int j = 0; j < LU / 4; ++j)
                fv[k][j] = (e0 + 4 * j < n_pad) ? reinterpret_cast<const float4 *>(fin + e0)[j]
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
#pragma unroll
    for (int k = 0; k < NS; ++k) {
        if ((uint32_t)k * U::STEP < n_rem) {         // the same for the whole warp
            const uint32_t unit = (uint32_t)k * 32u + (uint32_t)lane;
            const uint32_t e0 = unit * LU;
            uint32_t wout[NW];
            float4 fo[LU / 4];
            const int valid = e0 >= n_rem ? 0 : (n_rem - e0 < (uint32_t)LU ? (int)(n_rem - e0) : LU);
            compute_unit<F, MODE, true>(win[k], fv[k], wout, fo, s, b, neg_lr, acc, valid);
            if constexpr (MODE != DECOMPRESS) {
#pragma unroll
                for (int j = 0; j < NW; ++j)
                    if (unit * NW + j < w_rem) cw[unit * NW + j] = wout[j];
            }
            if constexpr (MODE == DECOMPRESS || WOUT) {
#pragma unroll
                for (int j = 0; j < LU / 4; ++j)
                    if (e0 + 4 * j < n_pad) reinterpret_cast<float4 *>(fout + e0)[j] = fo[j];
            }
        }
    }
    return acc;
}

// `cnt` consecutive tiles of a variable that stays FP32 (Sec. 2.4), from tile `local` on: copy in / copy out / plain SGD
// step.  Out of line: the values in flight take 32 to 64 registers per lane, which
// the kernels of the narrower codes, already at their register limit, can only afford in a frame of
// its own (inlined and tile by tile, the fused round of the 100M set with a tenth of the matrices
// in FP32 took 0.19 ms with 12-bit codes).
// AHEAD: chunks of 512 elements with the next chunk's loads in flight (best for the queue, where
// a warp does nothing else); otherwise whole tiles one after the other (best inside the runs).
template <int MODE, bool WOUT, bool AHEAD = false>
__device__ __noinline__ void resid_tiles(float *__restrict__ r, const float *__restrict__ fin, float *__restrict__ fout,
                                         uint64_t n, uint32_t local, uint32_t cnt, float neg_lr, int lane)
{
    constexpr int PER = AHEAD ? 4 : 8;             // 16-byte values per lane and chunk
    const uint64_t e_begin = (uint64_t)local * TILE;
    const uint64_t e_end = (uint64_t)(local + cnt) * TILE < n ? (uint64_t)(local + cnt) * TILE : n;
    const uint32_t n4 = (uint32_t)((e_end - e_begin + 3) / 4);          // at most cnt * 256
    float4 *const r4 = reinterpret_cast<float4 *>(r + e_begin);
    const float4 *const g4 = (MODE != DECOMPRESS) ? reinterpret_cast<const float4 *>(fin + e_begin) : nullptr;
    float4 *const o4 = (MODE == DECOMPRESS || WOUT) ? reinterpret_cast<float4 *>(fout + e_begin) : nullptr;
    float4 a[PER], g[PER], an[PER], gn[PER];
    auto load = [&](uint32_t base, float4 (&av)[PER], float4 (&gv)[PER]) {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const uint32_t i = base + j * 32 + lane;
            if (i < n4) {
                if constexpr (MODE != COMPRESS) av[j] = r4[i];
                if constexpr (MODE != DECOMPRESS) gv[j] = __ldcs(g4 + i);
            }
        }
    };
    if constexpr (AHEAD) load(0, a, g);
    for (uint32_t base = 0; base < n4; base += PER * 32) {
        if constexpr (AHEAD) {
            if (base + PER * 32 < n4) load(base + PER * 32, an, gn);
        } else {
            load(base, a, g);
        }
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const uint32_t i = base + j * 32 + lane;
            if (i < n4) {
                if constexpr (MODE == COMPRESS) {
                    r4[i] = g[j];
                } else if constexpr (MODE == DECOMPRESS) {
                    o4[i] = a[j];
                } else {
                    float4 w;
                    w.x = __fmaf_rn(neg_lr, g[j].x, a[j].x);
                    w.y = __fmaf_rn(neg_lr, g[j].y, a[j].y);
                    w.z = __fmaf_rn(neg_lr, g[j].z, a[j].z);
                    w.w = __fmaf_rn(neg_lr, g[j].w, a[j].w);
                    r4[i] = w;
                    if constexpr (WOUT) o4[i] = w;
                }
            }
        }
        if constexpr (AHEAD) {
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                a[j] = an[j];
                g[j] = gn[j];
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------

// The state of a warp's pipeline: its slice of shared memory, its mbarriers, how many granules it
// has moved so far (which fixes the stage, the barrier phase and the output buffer of the next
// one) and whether a wait ran out.
struct WarpPipe {
    uint8_t *wbase;
    uint32_t bar0;
    uint32_t k;
    uint32_t phases;      // bit i: the parity the next wait on mbarrier i looks for
    uint32_t wait_limit;  // polls of one mbarrier before giving up
    bool skip_loads;      // diagnostics: announce the loads, do not issue them
    bool failed;
};

__device__ __forceinline__ void pipe_init(WarpPipe &pipe, const KParams &p)
{
    pipe.k = 0;
    pipe.phases = 0u;
    pipe.wait_limit = p.wait_limit ? p.wait_limit : WAIT_LIMIT;
    pipe.skip_loads = p.skip_loads != 0u;
    pipe.failed = false;
}

// Elements [e_begin, e_end) of one quantised variable (e_begin on a tile boundary, e_end on a tile
// boundary or at the variable's end): whole granules through the warp's pipeline, the rest (only
// at the variable's end) through the predicated path.  `codes`, `fin`, `fout` point at the
// variable's first element in their arenas.
template <class F, int MODE, bool WOUT>
__device__ __forceinline__ void run_elements(WarpPipe &pipe, uint8_t *codes, const float *fin, float *fout,
                                             uint64_t e_begin, uint64_t e_end, uint64_t n, uint64_t packed_bytes,
                                             float s, float b, float neg_lr, Acc &acc, int lane)
{
    using SM = Smem<F, MODE, WOUT>;
    uint8_t *const wbase = pipe.wbase;
    uint8_t *const outs = wbase + SM::NSTAGES * SM::STAGE;
    const uint32_t bar0 = pipe.bar0;
    uint32_t k = pipe.k;
    bool failed = false;
    constexpr uint32_t SUB = Unit<F>::SUB;
    const uint32_t g0 = (uint32_t)(e_begin / SUB);                  // first granule
    const uint32_t ng = (uint32_t)((e_end - e_begin) / SUB);        // whole granules

    constexpr bool ROWS_IN = SM::ROWS && SM::IN_F > 0, ROWS_OUT = SM::ROWS && SM::OUT_F > 0;
    auto issue = [&](uint32_t g, uint32_t kk) {           // called by the whole warp
        const uint32_t st = kk % SM::NSTAGES;
        const uint32_t bar = bar0 + 8u * st;
        uint8_t *dst = wbase + st * SM::STAGE;
        if (lane == 0) {
            mbar_expect_tx(bar, (uint32_t)SM::TX_BYTES);
            if (!pipe.skip_loads) {
                if constexpr (SM::IN_C > 0)
                    bulk_load(smem_addr(dst), codes + (size_t)g * SM::CB, SM::CB, bar);
                if constexpr (SM::IN_F > 0)
                    bulk_load(smem_addr(dst + SM::IN_C), fin + (size_t)g * SUB, SM::FB, bar);
            }
        }
    };

    EqTracker<F> eq;
    eq.reset();
    for (uint32_t i = 0; i < (uint32_t)SM::DIST && i < ng; ++i) issue(g0 + i, k + i);
    for (uint32_t i = 0; i < ng; ++i, ++k) {
        const uint32_t g = g0 + i;
        if constexpr (SM::CODES_IN_PLACE) {
            if (lane == 0) bulk_wait_read0();      // the stage refilled next was stored from last round
            __syncwarp();
        }
        if (i + SM::DIST < ng) issue(g + SM::DIST, k + SM::DIST);   // its stage was consumed last round
        if (lane == 0 && !SM::CODES_IN_PLACE) {
            // the output buffer written next must have left with its last store
            if constexpr (SM::OUTBUFS == 2) bulk_wait_read1(); else bulk_wait_read0();
        }
        __syncwarp();
        // wait for this granule's bytes (bounded)
        const uint32_t st = k % SM::NSTAGES, bar = bar0 + 8u * st, parity = (pipe.phases >> st) & 1u;
        pipe.phases ^= 1u << st;
        uint32_t polls = 0;
        while (!__all_sync(0xFFFFFFFFu, mbar_try_wait(bar, parity))) {
            if (++polls > pipe.wait_limit) { failed = true; break; }
        }
        if (failed) break;
        uint8_t *stage = wbase + st * SM::STAGE;
        uint8_t *ob = outs + (k % SM::OUTBUFS) * SM::OUT;
        const float *fsrc = reinterpret_cast<const float *>(stage + SM::IN_C);
        float *fdst = reinterpret_cast<float *>(ob + SM::OUT_C);
        if constexpr (ROWS_IN) rows_swizzle_in_place(const_cast<float *>(fsrc), lane, true);
        uint8_t *cdst = SM::CODES_IN_PLACE ? stage : ob;
        granule_from_smem<F, MODE, WOUT>(reinterpret_cast<const uint32_t *>(stage), fsrc, reinterpret_cast<uint32_t *>(cdst),
                                         fdst, s, b, neg_lr, acc, eq, i == 0, lane);
        if constexpr (ROWS_OUT) {
            __syncwarp();
            rows_swizzle_in_place(fdst, lane, false);
        }
        fence_proxy_async();           // make the results visible to the bulk store
        __syncwarp();
        if (lane == 0) {
            if constexpr (MODE != DECOMPRESS)
                bulk_store(codes + (size_t)g * SM::CB, smem_addr(cdst), SM::CB);
            if constexpr (SM::OUT_F > 0)
                bulk_store(fout + (size_t)g * SUB, smem_addr(ob + SM::OUT_C), SM::FB);
            bulk_commit();
        }
    }
    if (failed) { pipe.k = k; pipe.failed = true; return; }
    if constexpr (MODE != DECOMPRESS) eq.fold(acc);
    const uint64_t e_rag = e_begin + (uint64_t)ng * SUB;
    if (e_rag < e_end) {     // the variable's ragged end
        const uint64_t w0 = e_rag / 32 * F::B;
        acc = tile_ragged<F, MODE, WOUT>(reinterpret_cast<uint32_t *>(codes) + w0,
                                         fin ? fin + e_rag : nullptr, fout ? fout + e_rag : nullptr,
                                         (uint32_t)(n - e_rag), (uint32_t)(packed_bytes / 4 - w0),
                                         s, b, neg_lr, acc, lane);
    }
    pipe.k = k;
}

// One table entry, through the read-only path with 16-byte loads (all lanes read the same entry).
__device__ __forceinline__ VarDev load_var(const VarDev *src)
{
    VarDev var;
    const ulonglong2 a = __ldg(reinterpret_cast<const ulonglong2 *>(src));
    const ulonglong2 c = __ldg(reinterpret_cast<const ulonglong2 *>(src) + 1);
    const uint4 d = __ldg(reinterpret_cast<const uint4 *>(src) + 2);
    const uint4 e = __ldg(reinterpret_cast<const uint4 *>(src) + 3);
    var.n = a.x; var.full_off = a.y; var.store_off = c.x; var.packed_bytes = c.y;
    var.tile_start = ((uint64_t)d.y << 32) | d.x;
    var.ntiles = d.z; var.quantised = d.w;
    var.sb_slot = e.x; var.slot_base = e.y; var.first_run = e.z; var.nslots = e.w;
    return var;
}

// The FP32 variables' tiles of a launch form one list, taken in chunks by whichever warp is through
// with its run of quantised tiles: FP32 tiles cost a warp more or less than tiles of codes
// depending on how many other warps move FP32 data at the same time, which no fixed division can
// know, and they need no sums, so any warp can take any of them.  queue[0] hands out chunks,
// queue[1] counts the warps that are through; the last of them clears both for the next launch.
constexpr uint32_t FP32_CHUNK_TILES = 4;

template <int MODE, bool WOUT>
__device__ __noinline__ void fp32_queue(const KParams &p, int lane)
{
    // the first three quarters of the list go out in chunks of FP32_CHUNK_TILES tiles, the rest tile
    // by tile, so that the warps finish within a tile of each other
    const uint64_t total = __ldg(p.fp32_tile_start + p.n_fp32);
    const uint64_t big = total * 3 / 4 / FP32_CHUNK_TILES;
    const uint64_t nchunks = big + (total - big * FP32_CHUNK_TILES);
    uint32_t next = 0;
    if (lane == 0) next = atomicAdd(p.queue, 1u);
    next = __shfl_sync(0xFFFFFFFFu, next, 0);
    while (next < nchunks) {
        const uint32_t c = next;
        if (lane == 0) next = atomicAdd(p.queue, 1u);       // the following chunk, asked for ahead of the work
        uint64_t t = c < big ? (uint64_t)c * FP32_CHUNK_TILES : big * FP32_CHUNK_TILES + (c - big);
        const uint64_t tend = c < big ? t + FP32_CHUNK_TILES : t + 1;
        uint32_t lo = 0, hi = p.n_fp32;                     // the FP32 variable that holds tile t
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (__ldg(p.fp32_tile_start + mid) <= t) lo = mid; else hi = mid;
        }
        while (t < tend) {
            const uint64_t first = __ldg(p.fp32_tile_start + lo), after = __ldg(p.fp32_tile_start + lo + 1);
            const VarDev var = load_var(p.vars + __ldg(p.fp32_var + lo));
            const uint32_t local = (uint32_t)(t - first);
            const uint32_t cnt = (uint32_t)((after < tend ? after : tend) - t);
            resid_tiles<MODE, WOUT, true>(p.resid + var.store_off, p.fin + var.full_off,
                                          WOUT ? p.fout + var.full_off : nullptr, var.n, local, cnt, p.neg_lr, lane);
            t += cnt;
            ++lo;
        }
        next = __shfl_sync(0xFFFFFFFFu, next, 0);
    }
    if (lane == 0) {
        __threadfence();
        if (atomicAdd(p.queue + 1, 1u) == p.nwarps - 1) {   // every warp has taken its last chunk number
            p.queue[0] = 0u;
            p.queue[1] = 0u;
        }
    }
}


// QUEUE (fused round only): the FP32 variables' tiles are taken from the queue (fp32_queue above)
// instead of the runs; a separate instantiation, because the call costs the kernels of
// all-quantised models 3 to 8 %.
template <class F, int MODE, bool WOUT, bool QUEUE = false>
__global__ void __launch_bounds__(32 * Smem<F, MODE, WOUT>::WARPS, MODE == DECOMPRESS ? DECOMPRESS_CTAS_PER_SM : CTAS_PER_SM)
omc_kernel(const KParams p)
{
    using SM = Smem<F, MODE, WOUT>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // read once (volatile): otherwise the compiler re-reads the special register all over the main
    // loop instead of keeping the lane number in a register
    int lane;
    asm volatile("mov.u32 %0, %%laneid;" : "=r"(lane));
    const int wid = threadIdx.x >> 5;
    const uint32_t warp = blockIdx.x * SM::WARPS + wid;
    if (warp >= p.nwarps) return;

    // this warp's slice of shared memory: the input stages, then the output buffers
    WarpPipe pipe;
    pipe.wbase = smem_raw + SM::BAR_PAD + wid * SM::PER_WARP;
    pipe.bar0 = smem_addr(smem_raw) + (uint32_t)wid * MAX_STAGES * 8u;
    pipe_init(pipe, p);
    const uint32_t bar0 = pipe.bar0;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < MAX_STAGES; ++i) mbar_init(bar0 + 8u * i, 1u);
        fence_mbar_init();
        fence_proxy_async();
    }
    __syncwarp();
    // Where the launch is the programmatic dependent of the kernel before it on the stream
    // (KParams::dependent), the launch and the set-up above overlap that kernel's last warps; nothing
    // of global memory is touched before it has completed.  The kernel after this one may be set up
    // the same way.  In an ordinary launch both instructions do nothing.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    for (uint32_t run = warp; run < p.nruns && !pipe.failed; run += p.nwarps) {
        uint64_t t, tend;
        run_tile_range(p, run, t, tend);
        uint32_t v = run_first_var(p, run, t);
        while (t < tend && !pipe.failed) {
            const VarDev var = load_var(p.vars + v);
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
                uint8_t *const codes = p.packed + var.store_off;
                const float *const fin = (MODE != DECOMPRESS) ? p.fin + var.full_off : nullptr;
                float *const fout = (MODE == DECOMPRESS || WOUT) ? p.fout + var.full_off : nullptr;
                const uint64_t e_begin = (uint64_t)local * TILE;
                const uint64_t e_end = (uint64_t)(local + cnt) * TILE < var.n ? (uint64_t)(local + cnt) * TILE : var.n;
                run_elements<F, MODE, WOUT>(pipe, codes, fin, fout, e_begin, e_end, var.n, var.packed_bytes, s, b,
                                            p.neg_lr, acc, lane);
                if (pipe.failed) break;
                if constexpr (MODE != DECOMPRESS) {
                    if (p.pvt) {
                        flush_and_maybe_finalise(p.slots + var.slot_base, run - var.first_run, var.nslots,
                                                 p.tickets + var.sb_slot, cnt, var.ntiles, var.n,
                                                 ValuePattern<F>::MAGNITUDE_MASK, p.sb + 2 * var.sb_slot, acc, lane);
                    } else if (MODE == COMPRESS && local == 0 && lane == 0) {
                        p.sb[2 * var.sb_slot] = 1.f;
                        p.sb[2 * var.sb_slot + 1] = 0.f;
                    }
                }
            } else if (!QUEUE) {
                resid_tiles<MODE, WOUT>(p.resid + var.store_off, (MODE != DECOMPRESS) ? p.fin + var.full_off : nullptr,
                                        ((MODE == DECOMPRESS) || WOUT) ? p.fout + var.full_off : nullptr, var.n, local,
                                        cnt, p.neg_lr, lane);
            }       // else: FP32 tiles are taken from the queue below
            t += cnt;
            ++v;
        }
    }
    if constexpr (QUEUE) {
        if (!pipe.failed) fp32_queue<MODE, WOUT>(p, lane);
    }
    if (pipe.failed && lane == 0) atomicExch(p.status, 1u);   // a bulk load never arrived
    bulk_wait_all();                                     // stores must finish before the CTA's memory goes
}

template <class F, int MODE, bool WOUT, bool QUEUE = false>
void launch(const KParams &p, int grid, void *stream)
{
    using SM = Smem<F, MODE, WOUT>;
    static bool configured[64] = {};    // once per device and instantiation
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaFuncSetAttribute(omc_kernel<F, MODE, WOUT, QUEUE>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL);
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    if (p.dependent) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(32 * SM::WARPS);
        cfg.dynamicSmemBytes = SM::TOTAL;
        cfg.stream = static_cast<cudaStream_t>(stream);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaLaunchKernelEx(&cfg, omc_kernel<F, MODE, WOUT, QUEUE>, p);
    } else {
        omc_kernel<F, MODE, WOUT, QUEUE><<<grid, 32 * SM::WARPS, SM::TOTAL, static_cast<cudaStream_t>(stream)>>>(p);
    }
}

// ---------------------------------------------------------------------------------------------
// Re-selection (Sec. 3.1: the quantised subset changes from round to round): the state of a model
// under one plan becomes its state under another plan of the same variables and format, in one
// launch over the destination plan's tile list.  Per variable: still quantised -> its codes and
// (s, b) are copied; still FP32 -> copied; released -> decompressed into the FP32 arena
// (fma(s, Vt, b)); newly selected -> quantised from its FP32 values with a fresh fit.  Most bytes
// are plain copies; the two converting cases use the predicated global-memory path.

// Shared memory of the transition kernel: a warp's slice must hold either converting pipeline.
template <class F>
struct TransitionSmem {
    using C = Smem<F, COMPRESS, false>;
    using D = Smem<F, DECOMPRESS, false>;
    static constexpr int PER_WARP = C::PER_WARP > D::PER_WARP ? C::PER_WARP : D::PER_WARP;
    static constexpr int WARPS = C::WARPS;
    static constexpr int TOTAL = C::BAR_PAD + WARPS * PER_WARP;
};

// 16-byte copy of `count` units by one warp, eight loads in flight per lane.
__device__ __forceinline__ void warp_copy16(uint4 *__restrict__ to, const uint4 *__restrict__ from, uint64_t count,
                                            int lane)
{
    uint64_t i = lane;
    for (; i + 7 * 32 < count; i += 8 * 32) {
        uint4 r[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) r[j] = __ldcs(from + i + j * 32);
#pragma unroll
        for (int j = 0; j < 8; ++j) to[i + j * 32] = r[j];
    }
    for (; i < count; i += 32) to[i] = __ldcs(from + i);
}

template <class F>
__global__ void __launch_bounds__(32 * TransitionSmem<F>::WARPS, CTAS_PER_SM) omc_transition_kernel(const KParams p)
{
    using TS = TransitionSmem<F>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int lane = threadIdx.x & 31;
    const int wid = threadIdx.x >> 5;
    const uint32_t warp = blockIdx.x * TS::WARPS + wid;
    if (warp >= p.nwarps) return;
    WarpPipe pipe;
    pipe.wbase = smem_raw + TS::C::BAR_PAD + wid * TS::PER_WARP;
    pipe.bar0 = smem_addr(smem_raw) + (uint32_t)wid * MAX_STAGES * 8u;
    pipe_init(pipe, p);
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < MAX_STAGES; ++i) mbar_init(pipe.bar0 + 8u * i, 1u);
        fence_mbar_init();
        fence_proxy_async();
    }
    __syncwarp();

    // This launch's own division (transition_division.cu) is written by the kernel before it on the
    // stream; launched as its programmatic dependent, this kernel may start while that one ends,
    // and waits here for its results.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t nruns = *reinterpret_cast<const volatile uint32_t *>(p.nruns_dev);
    for (uint32_t run = warp; run < nruns && !pipe.failed; run += p.nwarps) {
        uint64_t t, tend;
        run_tile_range(p, run, t, tend);
        uint32_t v = run_first_var(p, run, t);
        while (t < tend && !pipe.failed) {
            const VarDev var = load_var(p.vars + v);            // where the variable goes
            const VarDev src = load_var(p.vars_from + v);       // where it is now
            const uint32_t local = (uint32_t)(t - var.tile_start);
            const uint64_t left = tend - t;
            const uint32_t cnt = (uint32_t)((uint64_t)(var.ntiles - local) < left ? (var.ntiles - local) : left);
            const uint64_t e_begin = (uint64_t)local * TILE;
            const uint64_t e_end = (uint64_t)(local + cnt) * TILE < var.n ? (uint64_t)(local + cnt) * TILE : var.n;
            if (var.quantised && src.quantised) {
                // same codes, other place: this run's share of the padded stream
                const uint64_t b0 = e_begin / 8 * F::B;
                const uint64_t b1 = (uint64_t)(local + cnt) == var.ntiles ? var.packed_bytes : e_end / 8 * F::B;
                warp_copy16(reinterpret_cast<uint4 *>(p.packed + var.store_off + b0),
                            reinterpret_cast<const uint4 *>(p.packed_from + src.store_off + b0), (b1 - b0) / 16, lane);
                if (local == 0 && lane == 0) {
                    p.sb[2 * var.sb_slot] = p.sb_from[2 * src.sb_slot];
                    p.sb[2 * var.sb_slot + 1] = p.sb_from[2 * src.sb_slot + 1];
                }
            } else if (!var.quantised && !src.quantised) {
                warp_copy16(reinterpret_cast<uint4 *>(p.resid + var.store_off + e_begin),
                            reinterpret_cast<const uint4 *>(p.resid_from + src.store_off + e_begin),
                            (e_end - e_begin + 3) / 4, lane);
            } else if (src.quantised) {
                // released: decompress into the FP32 arena
                const float s = __ldcg(p.sb_from + 2 * src.sb_slot), b = __ldcg(p.sb_from + 2 * src.sb_slot + 1);
                Acc none;
                none.reset();
                run_elements<F, DECOMPRESS, false>(pipe, const_cast<uint8_t *>(p.packed_from) + src.store_off, nullptr,
                                                   p.resid + var.store_off, e_begin, e_end, var.n, src.packed_bytes,
                                                   s, b, 0.f, none, lane);
            } else {
                // newly selected: quantise the FP32 values, fit (s, b)
                Acc acc;
                acc.reset();
                run_elements<F, COMPRESS, false>(pipe, p.packed + var.store_off, p.resid_from + src.store_off, nullptr,
                                                 e_begin, e_end, var.n, var.packed_bytes, 1.f, 0.f, 0.f, acc, lane);
                if (pipe.failed) break;
                if (p.pvt) {
                    const uint4 tv = __ldg(reinterpret_cast<const uint4 *>(p.trans_vars) + v);   // first_run, nslots, slot_base
                    flush_and_maybe_finalise(p.slots + tv.z, run - tv.x, tv.y, p.tickets + var.sb_slot, cnt,
                                             var.ntiles, var.n, ValuePattern<F>::MAGNITUDE_MASK,
                                             p.sb + 2 * var.sb_slot, acc, lane);
                } else if (local == 0 && lane == 0) {
                    p.sb[2 * var.sb_slot] = 1.f;
                    p.sb[2 * var.sb_slot + 1] = 0.f;
                }
            }
            t += cnt;
            ++v;
        }
    }
    if (pipe.failed && lane == 0) atomicExch(p.status, 1u);
    bulk_wait_all();
}

template <class F>
void launch_transition(const KParams &p, int grid, void *stream)
{
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaFuncSetAttribute(omc_transition_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TransitionSmem<F>::TOTAL);
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(32 * TransitionSmem<F>::WARPS);
    cfg.dynamicSmemBytes = TransitionSmem<F>::TOTAL;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, omc_transition_kernel<F>, p);
}

// ---------------------------------------------------------------------------------------------
// Server-side aggregation (Sec. 1: the clients' models are transported back and aggregated;
// Sec. 2.5: each client quantises its own subset, so the server receives precise values of a
// parameter from the clients that kept it in FP32).  out = (x_0 + x_1 + ... + x_{K-1}) / K per
// element, FP32, clients added in index order, one rounded division at the end, where x_k is
// client k's decompressed value fma(s_k, Vt_k, b_k) or its FP32 value.  Without the division it is
// the sum, and the sum may start from what `out` holds: more clients than one launch takes are
// added batch after batch, in the same order of additions as in one pass.
//
// The tiles are cut into short runs of equal length, dealt out to the warps in turn.  Tile by tile a
// warp walks the clients in index order with the tile's 32 sums per lane in registers; the codes of
// the (tile, client) pairs ahead are already on their way into a ring of shared-memory slots, one
// bulk copy each, so that the bytes in flight do not depend on how many registers a lane has left.
// FP32 copies of a tile are read with plain vector loads when their turn comes, their lines asked
// for (an L2 prefetch) when the producer passes them.  Every element is read once per client and
// written once.  The waits are on the warp's own copies and bounded, as in the other kernels.

// What the tile loop needs to know about one client's copy of the current variable.
struct AggClientVar {
    uint64_t base;        // the variable's codes, or its FP32 values
    uint32_t last_bytes;  // how many bytes of codes its last tile has (padding included)
    uint32_t quantised;
    float s, b;
    float sk;             // s * 2^(127-BIAS) where agg_add can use it (folded != 0)
    uint32_t folded;
};

// Shared memory of one warp: a ring of slots, each one client's codes of one tile.
template <class F>
struct AggSmem {
    static constexpr int CB = TILE * F::B / 8;
    static constexpr int RING_BYTES = 8192;
    static constexpr int MAX_SLOTS = 8;         // mbarriers reserved per warp
    static constexpr int NSLOT = RING_BYTES / CB < 2 ? 2 : RING_BYTES / CB > MAX_SLOTS ? MAX_SLOTS : RING_BYTES / CB;
    static constexpr int PER_WARP = NSLOT * CB;
    static constexpr int BAR_PAD = (8 * MAX_SLOTS * WARPS_PER_CTA + 127) / 128 * 128;
    static constexpr int TOTAL = BAR_PAD + WARPS_PER_CTA * PER_WARP;
    static_assert(CB % 16 == 0, "bulk copies move multiples of 16 bytes");
};

// Formats whose codes the aggregation decodes by placing the fields (codec.cuh, placed_at).
template <class F>
struct PlacedPath {
    static constexpr bool value = !F::FIXED && F::E < 8 && !HalfPath<F>::value && !Fp8Path<F>::value;
};

// acc[j] (+)= fma(s, Vt_j, b) for the AL consecutive elements whose codes are the ANW words of
// `win`; FIRST: the sum starts with this client.
// PlacedPath formats: `sk` is s * 2^(127-BIAS).  Where that did not overflow (`folded`) it is exact,
// and as Vt = placed * 2^(127-BIAS) exactly, fma(sk, placed, b) rounds the same real number as
// fma(s, Vt, b): the rebias multiplication is never made.  A variable whose s is that large takes
// the path of the Inf/NaN codes, element by element, for all of its values.
template <class F, int AL, int ANW, bool FIRST>
__device__ __forceinline__ void agg_add(const uint32_t (&win)[ANW], float s, float sk, float b, bool folded, float *acc)
{
    float x[AL];
    if constexpr (Fp8Path<F>::value) {
        // four codes at a time through the narrow-float conversions; Inf/NaN codes redone
#pragma unroll
        for (int g = 0; g < AL / 4; ++g) {
            float dec[4];
            uint32_t c4;            // the group's codes, one per byte
            if constexpr (F::B == 8) c4 = win[g];
            else c4 = spread6(g == 0 ? win[0] : g == 1 ? __funnelshift_r(win[0], win[1], 24)
                              : g == 2 ? __funnelshift_r(win[1], win[2], 16) : win[2] >> 8);
            fp8x4_decode<F>(c4, dec);
            if (F::E != 5 && fp8x4_any_at_least<F, F::INF_MAG>(c4)) {
#pragma unroll
                for (int j = 0; j < 4; ++j) dec[j] = decode_exact<F>((c4 >> (8 * j)) & 0xFFu);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) x[4 * g + j] = __fmaf_rn(s, dec[j], b);
        }
    } else if constexpr (PlacedPath<F>::value) {
        // eight values at a time, tested together for Inf/NaN codes
        constexpr int G = AL >= 8 ? 8 : 4;
#pragma unroll
        for (int g = 0; g < AL / G; ++g) {
            float v[G];
#pragma unroll
            for (int j = 0; j < G; ++j) v[j] = placed_at<F, ANW>(win, (G * g + j) * F::B);
            float m = absmax4(v[0], v[1], v[2], v[3]);
            if constexpr (G == 8) m = fmaxf(m, absmax4(v[4], v[5], v[6], v[7]));
            if (m >= u2f(F::INF_MAG << F::SH) || !folded) {
#pragma unroll
                for (int j = 0; j < G; ++j)
                    x[G * g + j] = __fmaf_rn(s, decode_exact<F>(get_code_at<F, ANW>(win, (G * g + j) * F::B)), b);
            } else {
#pragma unroll
                for (int j = 0; j < G; ++j) x[G * g + j] = __fmaf_rn(sk, v[j], b);
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < AL; ++j) x[j] = __fmaf_rn(s, decode_exact<F>(get_code_at<F, ANW>(win, j * F::B)), b);
    }
#pragma unroll
    for (int j = 0; j < AL; ++j) acc[j] = FIRST ? x[j] : __fadd_rn(acc[j], x[j]);
}

// One client's codes of one tile, in a slot of the ring: each lane adds its 32 values to its sums.
template <class F, bool FIRST>
__device__ __forceinline__ void agg_tile_codes(const uint32_t *sw, float s, float sk, float b, bool folded,
                                               float (&acc)[32], int lane)
{
    using U = Unit<F>;
    // A lane takes AL consecutive elements at a time, at least four (one 16-byte store), NQ times per tile.
    constexpr int UF = U::LU < 4 ? 4 / U::LU : 1, AL = U::LU * UF, ANW = U::NWORDS * UF, NQ = 32 / AL;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        uint32_t win[ANW];
        const uint32_t *uw = sw + (q * 32 + lane) * ANW;
        if constexpr (ANW % 4 == 0) {
#pragma unroll
            for (int j = 0; j < ANW / 4; ++j) {
                const uint4 w4 = reinterpret_cast<const uint4 *>(uw)[j];
                win[4 * j] = w4.x; win[4 * j + 1] = w4.y; win[4 * j + 2] = w4.z; win[4 * j + 3] = w4.w;
            }
        } else if constexpr (ANW % 2 == 0) {
#pragma unroll
            for (int j = 0; j < ANW / 2; ++j) {
                const uint2 w2 = reinterpret_cast<const uint2 *>(uw)[j];
                win[2 * j] = w2.x; win[2 * j + 1] = w2.y;
            }
        } else {
#pragma unroll
            for (int j = 0; j < ANW; ++j) win[j] = uw[j];
        }
        agg_add<F, AL, ANW, FIRST>(win, s, sk, b, folded, acc + q * AL);
    }
}

// One client's FP32 values of one tile, element e of the tile at r[e]: the same elements per lane.
// WHOLE: the tile lies inside the variable; otherwise only the first `n_pad` floats exist.
template <class F, bool FIRST, bool WHOLE>
__device__ __forceinline__ void agg_tile_fp32(const float *r, uint32_t n_pad, float (&acc)[32], int lane)
{
    using U = Unit<F>;
    constexpr int UF = U::LU < 4 ? 4 / U::LU : 1, AL = U::LU * UF, NQ = 32 / AL;
    float4 f[8];
#pragma unroll
    for (int q = 0; q < NQ; ++q)
#pragma unroll
        for (int j = 0; j < AL / 4; ++j) {
            const uint32_t e = (uint32_t)(q * 32 + lane) * AL + 4 * j;
            f[q * (AL / 4) + j] = (WHOLE || e < n_pad) ? __ldcs(reinterpret_cast<const float4 *>(r + e))
                                                       : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        acc[4 * i] = FIRST ? f[i].x : __fadd_rn(acc[4 * i], f[i].x);
        acc[4 * i + 1] = FIRST ? f[i].y : __fadd_rn(acc[4 * i + 1], f[i].y);
        acc[4 * i + 2] = FIRST ? f[i].z : __fadd_rn(acc[4 * i + 2], f[i].z);
        acc[4 * i + 3] = FIRST ? f[i].w : __fadd_rn(acc[4 * i + 3], f[i].w);
    }
}

__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

template <class F>
__global__ void __launch_bounds__(THREADS, aggregate_ctas_per_sm(F::B)) omc_aggregate_kernel(const AggParams p)
{
    using U = Unit<F>;
    using AS = AggSmem<F>;
    constexpr int UF = U::LU < 4 ? 4 / U::LU : 1, AL = U::LU * UF, NQ = 32 / AL;
    constexpr uint32_t CB = AS::CB, NSLOT = AS::NSLOT;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ AggClientVar cv_all[WARPS_PER_CTA][MAX_CLIENTS];
    int lane;
    asm volatile("mov.u32 %0, %%laneid;" : "=r"(lane));
    const int wid = threadIdx.x >> 5;
    const uint32_t warp = blockIdx.x * WARPS_PER_CTA + wid;
    if (warp >= p.nwarps) return;
    uint8_t *const ring = smem_raw + AS::BAR_PAD + wid * AS::PER_WARP;
    const uint32_t bar0 = smem_addr(smem_raw) + (uint32_t)wid * AS::MAX_SLOTS * 8u;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < (int)NSLOT; ++i) mbar_init(bar0 + 8u * i, 1u);
        fence_mbar_init();
        fence_proxy_async();
    }
    __syncwarp();
    AggClientVar *cv = cv_all[wid];
    const uint32_t K = p.nclients;
    const uint32_t wait_limit = p.wait_limit ? p.wait_limit : WAIT_LIMIT;
    const bool skip_loads = p.skip_loads != 0u;
    uint32_t phases = 0u;            // bit i: the parity the next wait on slot i looks for
    uint32_t pslot = 0u, cslot = 0u; // the slot filled next, the slot read next
    uint32_t in_ring = 0u;           // copies issued and not yet consumed
    bool failed = false;
    // FP32 copies the producer has passed and the consumer has not yet read: at most FP32_AHEAD, so
    // that what is prefetched for all warps together stays a fraction of the L2
    constexpr uint32_t FP32_AHEAD = 3;
    uint32_t fp32_ahead = 0u;
    const float kf = (float)K;
    // Dividing by a power of two is a multiplication by its exact reciprocal: both are the correctly
    // rounded value of the same real number.
    const bool pow2 = (K & (K - 1)) == 0;
    const float kinv = 1.f / kf;
    const bool divide = p.divide != 0u, accumulate = p.accumulate != 0u;
    auto mean_of = [&](float a) { return !divide ? a : pow2 ? __fmul_rn(a, kinv) : __fdiv_rn(a, kf); };

    // Short runs of equal length, dealt out to the warps in turn: what a tile costs depends on how many
    // clients hold it in FP32, and a long stretch of costly tiles is shared by all warps this way.
    for (uint32_t run = warp; run < p.nruns && !failed; run += p.nwarps) {
        uint64_t t = (uint64_t)run * p.tile_count / p.nruns;
        const uint64_t tend = (uint64_t)(run + 1) * p.tile_count / p.nruns;
        uint32_t lo = 0, hi = p.nvars;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (__ldg(&p.vars[0][mid].tile_start) <= t) lo = mid; else hi = mid;
        }
        uint32_t v = lo;

        while (t < tend && !failed) {
            const VarDev var = load_var(p.vars[0] + v);
            __syncwarp();
            if ((uint32_t)lane < K) {
                const VarDev vk = load_var(p.vars[lane] + v);
                AggClientVar c;
                c.quantised = vk.quantised;
                c.last_bytes = vk.ntiles ? (uint32_t)(vk.packed_bytes - (uint64_t)(vk.ntiles - 1) * CB) : 0u;
                c.base = vk.quantised ? reinterpret_cast<uint64_t>(p.packed[lane] + vk.store_off)
                                      : reinterpret_cast<uint64_t>(p.resid[lane] + vk.store_off);
                c.s = vk.quantised ? __ldg(p.sb[lane] + 2 * vk.sb_slot) : 1.f;
                c.b = vk.quantised ? __ldg(p.sb[lane] + 2 * vk.sb_slot + 1) : 0.f;
                c.sk = c.s;
                c.folded = 0u;
                if constexpr (PlacedPath<F>::value) {
                    c.sk = __fmul_rn(c.s, u2f(F::pow2_bits(127 - F::BIAS)));
                    c.folded = fabsf(c.sk) < u2f(0x7F800000u) ? 1u : 0u;       // no overflow: the product is exact
                }
                cv[lane] = c;
            }
            __syncwarp();
            const uint32_t local = (uint32_t)(t - var.tile_start);
            const uint64_t left = tend - t;
            const uint32_t cnt = (uint32_t)((uint64_t)(var.ntiles - local) < left ? (var.ntiles - local) : left);

            // the producer's place in this variable's (tile, client) pairs
            uint32_t ptile = 0u, pk = 0u;
            auto fill = [&]() {                     // called by the whole warp
                while (ptile < cnt && in_ring < NSLOT && fp32_ahead < FP32_AHEAD) {
                    const AggClientVar c = cv[pk];
                    if (c.quantised) {
                        // packed sizes are multiples of 16 bytes, and so is what is left of one in its last tile
                        const uint64_t off = (uint64_t)(local + ptile) * CB;
                        const uint32_t bytes = local + ptile + 1 == var.ntiles ? c.last_bytes : CB;
                        if (lane == 0) {
                            const uint32_t bar = bar0 + 8u * pslot;
                            mbar_expect_tx(bar, bytes);
                            if (!skip_loads)
                                bulk_load(smem_addr(ring + pslot * CB), reinterpret_cast<const uint8_t *>(c.base) + off, bytes,
                                          bar);
                        }
                        pslot = pslot + 1 == NSLOT ? 0u : pslot + 1;
                        ++in_ring;
                    } else {
                        // an FP32 copy is read with plain loads when its turn comes: ask for its lines now
                        const uint64_t e = (uint64_t)(local + ptile) * TILE + (uint32_t)lane * 32u;
                        if (e < var.n) prefetch_l2(reinterpret_cast<const float *>(c.base) + e);
                        ++fp32_ahead;
                    }
                    if (++pk == K) { pk = 0u; ++ptile; }
                }
            };

            for (uint32_t ti = 0; ti < cnt && !failed; ++ti) {
                fill();
                const uint64_t e_tile = (uint64_t)(local + ti) * TILE;
                const bool whole = e_tile + TILE <= var.n;
                const uint32_t n_here = whole ? (uint32_t)TILE : (uint32_t)(var.n - e_tile);     // the tile's elements
                const uint32_t n_pad = (n_here + 3u) & ~3u;
                float acc[32];
                // client k's turn; false: the wait for its codes ran out
                auto client = [&](auto first, uint32_t k) -> bool {
                    constexpr bool FIRST = decltype(first)::value;
                    const AggClientVar c = cv[k];
                    if (c.quantised) {
                        const uint32_t bar = bar0 + 8u * cslot, parity = (phases >> cslot) & 1u;
                        phases ^= 1u << cslot;
                        uint32_t polls = 0;
                        while (!__all_sync(0xFFFFFFFFu, mbar_try_wait(bar, parity))) {
                            if (++polls > wait_limit) return false;
                        }
                        const uint32_t *sw = reinterpret_cast<const uint32_t *>(ring + cslot * CB);
                        if constexpr (PlacedPath<F>::value) agg_tile_codes<F, FIRST>(sw, c.s, c.sk, c.b, c.folded != 0u, acc, lane);
                        else agg_tile_codes<F, FIRST>(sw, c.s, c.s, c.b, true, acc, lane);
                        __syncwarp();               // every lane has read the slot: it may be filled again
                        cslot = cslot + 1 == NSLOT ? 0u : cslot + 1;
                        --in_ring;
                        fill();
                    } else {
                        const float *r = reinterpret_cast<const float *>(c.base) + e_tile;
                        if (whole) agg_tile_fp32<F, FIRST, true>(r, n_pad, acc, lane);
                        else agg_tile_fp32<F, FIRST, false>(r, n_pad, acc, lane);
                        --fp32_ahead;
                        fill();
                    }
                    return true;
                };
                float *o = p.out + var.full_off + e_tile;
                uint32_t k = 0;
                if (accumulate) {       // the sum so far, left in `out` by the call before
                    if (whole) agg_tile_fp32<F, true, true>(o, n_pad, acc, lane);
                    else agg_tile_fp32<F, true, false>(o, n_pad, acc, lane);
                } else {
                    failed = !client(std::true_type{}, 0u);
                    k = 1;
                }
                for (; k < K && !failed; ++k) failed = !client(std::false_type{}, k);
                if (failed) break;
#pragma unroll
                for (int q = 0; q < NQ; ++q)
#pragma unroll
                    for (int j = 0; j < AL / 4; ++j) {
                        const uint32_t e = (uint32_t)(q * 32 + lane) * AL + 4 * j;
                        const int i = q * AL + 4 * j;
                        float4 m = make_float4(mean_of(acc[i]), mean_of(acc[i + 1]), mean_of(acc[i + 2]), mean_of(acc[i + 3]));
                        if (whole) {
                            *reinterpret_cast<float4 *>(o + e) = m;
                        } else if (e < n_pad) {
                            if (e + 3 >= n_here) {          // the padding after the variable's last element: zeros
                                if (e + 1 >= n_here) m.y = 0.f;
                                if (e + 2 >= n_here) m.z = 0.f;
                                m.w = 0.f;
                            }
                            *reinterpret_cast<float4 *>(o + e) = m;
                        }
                    }
            }
            t += cnt;
            ++v;
        }
    }
    if (failed && lane == 0) atomicExch(p.status, 1u);       // a bulk load never arrived
}

template <class F>
void launch_aggregate(const AggParams &p, int grid, void *stream)
{
    static bool configured[64] = {};    // once per device and instantiation
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaFuncSetAttribute(omc_aggregate_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize, AggSmem<F>::TOTAL);
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    omc_aggregate_kernel<F><<<grid, THREADS, AggSmem<F>::TOTAL, static_cast<cudaStream_t>(stream)>>>(p);
}

#define OMC_DEFINE_FIXED_FORMAT(I_, F_)                                                         \
    extern const FmtOps ops_I##I_##F##F_ = {I_, F_, 1, fit_warps_per_cta(1 + I_ + F_, true),    \
                                            aggregate_ctas_per_sm(1 + I_ + F_),                 \
                                            launch<FixFmt<I_, F_>, COMPRESS, false>,            \
                                            launch<FixFmt<I_, F_>, DECOMPRESS, false>,          \
                                            launch<FixFmt<I_, F_>, UPDATE, false>,              \
                                            launch<FixFmt<I_, F_>, UPDATE, true>,               \
                                            launch<FixFmt<I_, F_>, UPDATE, false, true>,        \
                                            launch_transition<FixFmt<I_, F_>>,                  \
                                            launch_aggregate<FixFmt<I_, F_>>};

#define OMC_DEFINE_FORMAT(E_, M_)                                                               \
    extern const FmtOps ops_E##E_##M##M_ = {E_, M_, 0, fit_warps_per_cta(1 + E_ + M_, false),   \
                                            aggregate_ctas_per_sm(1 + E_ + M_),                 \
                                            launch<Fmt<E_, M_>, COMPRESS, false>,               \
                                            launch<Fmt<E_, M_>, DECOMPRESS, false>,             \
                                            launch<Fmt<E_, M_>, UPDATE, false>,                 \
                                            launch<Fmt<E_, M_>, UPDATE, true>,                  \
                                            launch<Fmt<E_, M_>, UPDATE, false, true>,           \
                                            launch_transition<Fmt<E_, M_>>,                     \
                                            launch_aggregate<Fmt<E_, M_>>};

}  // namespace omc
