// omc_matmul: the forward path of Fig. 1 with the decompression fused into the consumer.
//
// A layer's weight matrix W (N x K, K contiguous) is held as S1E5Mz codes; code << (10 - z) is an
// IEEE half bit pattern, and the transformed weight is Wbar = s*Wt + b (Sec. 2.3), so
//     Y = X * Wbar^T = s * (X * Wt^T) + b * rowsum(X).
// The codes therefore go straight from the packed arena into shared memory and from there into the
// 5th-generation tensor cores as the B operand: the transient FP32 copy of the weights that
// omc_decompress would write, and a GEMM would read back, never exists.
//
// One persistent CTA per SM walks over 128 x 256 tiles of Y.  Warp 0 (one thread) runs the TMA
// pipeline over K (64 columns per stage), warp 1 (one thread) issues tcgen05.mma (128x256x16, FP16
// inputs, FP32 accumulator in tensor memory) and commits each stage back to the producer, warps 2-5
// read finished accumulators with tcgen05.ld and apply the epilogue above.  Tensor memory holds two
// accumulators (2 x 256 columns), so the epilogue of one tile runs under the MMAs of the next.
//   S1E5M10: the codes are halves already; TMA puts them into the 128-byte-swizzled operand tile.
//   S1E5M6 / S1E5M2: the tile's packed bytes arrive through a byte-typed tensor map, and eight more
//   warps expand them (byte permutes and shifts only) into the swizzled operand tile.
//   Products of at least 256 rows and columns run on pairs of SMs instead (matmul_pair_kernel below).
// Every wait is bounded; a wait that runs out sets the plan's status word, and the tensor memory is
// released on every path.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "omc_internal.h"

namespace omc {
int note_cuda(cudaError_t e);
}

constexpr int MATMUL_DECODER_THREADS = 512;      // sixteen decoder warps (measured against eight)

namespace {

constexpr int BM = 128, BK = 64;                 // CTA tile rows; BK halves = one 128-byte swizzle row
constexpr int BN_WIDE = 256, BN_SPLIT = 128;     // CTA tile columns: 256, or 128 for the two-term format
constexpr int UMMA_K = 16;                       // K of one tcgen05.mma with 16-bit inputs
constexpr int TILE_A_BYTES = BM * BK * 2;
constexpr int TMEM_COLS = 512;                   // two accumulators of 128 lanes x (up to) 256 FP32 columns
constexpr uint32_t WAIT_LIMIT = 1u << 20;        // polls of one mbarrier before giving up

// B = bits per code, E = exponent bits.  16: no decode stage, four stages of 48 KB.  12 / 8 / 6:
// three stages of 72 / 64 / 60 KB (X tile, operand tile, packed bytes of the tile) and sixteen
// decoder warps.  E = 5 codes are FP16 patterns with the low mantissa bits dropped; S1E4M3 and
// S1E2M3 codes go through the narrow-float conversion instructions.
// Odd code widths (11 and 13 bits: S1E3M7 of Table 2, S1E3M9 / S1E4M8 / S1E5M7 of Sec. 3.5.3): the
// 64 codes of a tile row are 8 B bytes, so every other K block starts 8 bytes off the 16-byte
// grid that a bulk tensor copy has to start on.  The copy then starts at the boundary below and
// is 8 bytes wider (BOX_BYTES), and the decoders index from the remainder; a row of the matrix
// must itself be a multiple of 16 bytes (K % 128 == 0).  Every value of these formats is an FP16
// value: E = 5 codes are FP16 patterns (code << 3), the others become FP16 patterns whose exponent
// field is too small by 15 - bias, which one exact packed multiplication by 2^(15 - bias) repairs
// for normal and subnormal codes alike; Inf / NaN codes are patched in afterwards.
// E = 0 stands for the fixed-point variant S1I0Fy with y = B - 1 (B = 8, 12, 16).
template <int B, int E>
struct Cfg {
    static_assert((E == 5 && (B == 16 || B == 12 || B == 8)) || (E == 4 && B == 8) || (E == 2 && B == 6) ||
                  (B == 13 && (E == 5 || E == 3 || E == 4)) || (B == 11 && E == 3) || (B == 19 && E == 4) ||
                  (E == 0 && (B == 8 || B == 12 || B == 16)), "");
    static constexpr bool FIXED = E == 0;        // S1I0Fy, y = B - 1: two's complement k, value k * 2^-y
    static constexpr bool DECODE = B != 16 || FIXED;
    static constexpr bool ODD = (B % 2) != 0;
    // S1E4M14 (Table 1) has 15 significant bits, four more than an FP16 value: a weight is split
    // exactly into hi + lo, both FP16 values (hi = the weight rounded to FP16, lo = the rest, at
    // most 5 significant bits and never below 2^-20), the tile has two operand tiles and every K
    // step two products into the same accumulator.  The tile is 128 columns wide then.
    // S1I0F15 has 15 significant bits as well: k = 64 hi + lo with -512 <= hi < 512 and 0 <= lo < 64,
    // the weight is hi * 2^-9 + lo * 2^-15, two FP16 values again.
    static constexpr bool SPLIT = (B == 19) || (FIXED && B == 16);
    static constexpr int BN = SPLIT ? BN_SPLIT : BN_WIDE;
    static constexpr int TILE_B_BYTES = BN * BK * 2;              // one operand tile
    static constexpr int OPERAND_BYTES = (SPLIT ? 2 : 1) * TILE_B_BYTES;
    static constexpr uint32_t IDESC = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    static constexpr int MAN = B - 1 - E;
    static constexpr int ROW_BYTES = BK * B / 8;                 // one tile row of codes
    static constexpr int BOX_BYTES = ODD ? (ROW_BYTES + 8 + 15) / 16 * 16 : ROW_BYTES;   // what one copy brings per row
    static constexpr int RAW_BYTES = DECODE ? BN * BOX_BYTES : 0;
    static constexpr int STAGE = TILE_A_BYTES + OPERAND_BYTES + RAW_BYTES;
    static constexpr int NSTAGES = !DECODE ? 4 : (3 * STAGE + 1280 <= 227 * 1024 ? 3 : 2);
    static constexpr int SMEM = NSTAGES * STAGE + 1024 /* alignment slack */ + 256 /* barriers, tmem slot */;
    static constexpr int DEC_THREADS = DECODE ? MATMUL_DECODER_THREADS : 0;
    static constexpr int THREADS = 192 + DEC_THREADS;
    static constexpr uint32_t TX_BYTES = TILE_A_BYTES + (DECODE ? RAW_BYTES : TILE_B_BYTES);
    static_assert(STAGE % 1024 == 0, "operand tiles stay 1024-byte aligned");
    static_assert(SMEM <= 227 * 1024, "one CTA per SM");
};

__device__ __forceinline__ uint32_t saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait for the phase with the given parity; false if it never completed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit)
{
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Shared-memory matrix descriptor of a K-major tile with 128-byte swizzle: rows of 128 bytes,
// groups of 8 rows 1024 bytes apart (stride byte offset), leading byte offset unused (1),
// descriptor version 1, layout type 2 (128-byte swizzle).  Addresses and offsets in 16-byte units.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_byte_addr)
{
    return (uint64_t)((smem_byte_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor (Cfg::IDESC): D = FP32 (bits 4-5 = 1), A = B = FP16 (0), both K-major, N/8 at bit 17,
// M/16 at bit 24.
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__global__ void rowsum_kernel(const __half *__restrict__ x, uint32_t M, uint32_t K, float *__restrict__ out)
{
    // the product that follows is launched as this kernel's programmatic dependent and may start at once;
    // its epilogue waits for this kernel before it reads the sums
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // one warp per row; fixed order (lane-strided partial sums, then a shuffle tree)
    const uint32_t row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= M) return;
    const int lane = threadIdx.x & 31;
    float acc = 0.f;
    for (uint32_t k = lane; k < K; k += 32) acc += __half2float(x[(size_t)row * K + k]);
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    if (lane == 0) out[row] = acc;
}

// Four codes of a narrow-float type, one per byte, as two FP16 pairs.  MAG_MASK / INF_MAG: the
// magnitude bits of a code and the magnitude of the family's infinity; the hardware type has
// finite values (or its own NaN) from there on, the family has Inf (INF_MAG) and NaNs (above),
// which are patched in afterwards (rare: a weight would have to be Inf or NaN).
template <int E>
__device__ __forceinline__ void narrow_to_halves(uint32_t c4, uint32_t &h01, uint32_t &h23)
{
    constexpr uint32_t MAG_MASK = E == 4 ? 0x7Fu : 0x1Fu, INF_MAG = E == 4 ? 0x78u : 0x18u;
    constexpr uint32_t SIGN_SHIFT = E == 4 ? 7u : 5u;
    if constexpr (E == 4)
        asm("{\n\t.reg .b16 lo, hi;\n\t"
            "mov.b32 {lo, hi}, %2;\n\t"
            "cvt.rn.f16x2.e4m3x2 %0, lo;\n\t"
            "cvt.rn.f16x2.e4m3x2 %1, hi;\n\t}"
            : "=r"(h01), "=r"(h23) : "r"(c4));
    else
        asm("{\n\t.reg .b16 lo, hi;\n\t"
            "mov.b32 {lo, hi}, %2;\n\t"
            "cvt.rn.f16x2.e2m3x2 %0, lo;\n\t"
            "cvt.rn.f16x2.e2m3x2 %1, hi;\n\t}"
            : "=r"(h01), "=r"(h23) : "r"(c4));
    if (((c4 & (MAG_MASK * 0x01010101u)) + (0x80u - INF_MAG) * 0x01010101u) & 0x80808080u) {
        uint32_t h[4] = {h01 & 0xFFFFu, h01 >> 16, h23 & 0xFFFFu, h23 >> 16};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t c = (c4 >> (8 * j)) & 0xFFu, mag = c & MAG_MASK;
            if (mag >= INF_MAG) h[j] = (((c >> SIGN_SHIFT) & 1u) << 15) | (mag == INF_MAG ? 0x7C00u : 0x7E00u);
        }
        h01 = h[0] | (h[1] << 16);
        h23 = h[2] | (h[3] << 16);
    }
}

// Fixed-point codes (two's complement k in B bits, value k * 2^-(B-1)) as FP16 values, without an
// integer-to-float conversion: flipping the sign bit gives k + 2^(B-1) >= 0; up to ten bits of a
// non-negative integer j dropped into the mantissa of 1024 make the FP16 value 1024 + j, and one
// fused multiply-add, exact because its result is an FP16 value, scales it and takes the offset off.
__device__ __forceinline__ uint32_t hfma2_bits(uint32_t a, float mul, float add)
{
    const __half2 r = __hfma2(*reinterpret_cast<const __half2 *>(&a), __float2half2_rn(mul), __float2half2_rn(add));
    return *reinterpret_cast<const uint32_t *>(&r);
}
// S1I0F7, four codes of one word: 1024 + (k + 128) = 1152 + k, times 2^-7, minus 9.
__device__ __forceinline__ void fixed8_to_halves(uint32_t c4, uint32_t &h01, uint32_t &h23)
{
    const uint32_t x = c4 ^ 0x80808080u;
    h01 = hfma2_bits(__byte_perm(x, 0x64646464u, 0x5140), 0.0078125f, -9.f);
    h23 = hfma2_bits(__byte_perm(x, 0x64646464u, 0x5342), 0.0078125f, -9.f);
}
// S1I0F11, two codes: `t` holds three bytes of the stream as (b0 b1 | b1 b2), so code 0 is the low
// 12 bits of the low half and code 1 the high 12 bits of the high half; one shift and a byte permute
// put both in the low 12 bits of their halves (what lies above is masked away below).
// j = k + 2048 = code xor 0x800 has twelve bits: the low ten go into one FP16 value (1024 + lo), the
// top two into another (1024 + 256 hi; the xor only touches bit 11 and is folded into the constant);
// then (1024 + 256 hi) 2^-9 - 3.5 = hi/2 - 1.5 and (1024 + lo) 2^-11 + that = (lo + 1024 hi) / 2048 - 1 = k / 2048.
__device__ __forceinline__ uint32_t fixed12_to_halves(uint32_t t)
{
    const uint32_t v = __byte_perm(t, t >> 4, 0x7610);
    const uint32_t lo = (v & 0x03FF03FFu) | 0x64006400u, hi = ((v >> 2) & 0x03000300u) ^ 0x66006600u;
    const __half2 c = __hfma2(*reinterpret_cast<const __half2 *>(&hi), __float2half2_rn(0.001953125f), __float2half2_rn(-3.5f));
    const __half2 r = __hfma2(*reinterpret_cast<const __half2 *>(&lo), __float2half2_rn(0.00048828125f), c);
    return *reinterpret_cast<const uint32_t *>(&r);
}
// S1I0F15, two codes of one word: j = k + 32768; the top ten bits give hi + 512, the low six lo.
// (1024 + hi + 512) 2^-9 - 3 = hi 2^-9;  (1024 + lo) 2^-15 - 2^-5 = lo 2^-15 (an FP16 subnormal below 2^-14).
__device__ __forceinline__ void fixed16_to_halves(uint32_t c2, uint32_t &hi, uint32_t &lo)
{
    const uint32_t x = c2 ^ 0x80008000u;
    hi = hfma2_bits(((x >> 6) & 0x03FF03FFu) | 0x64006400u, 0.001953125f, -3.f);
    lo = hfma2_bits((x & 0x003F003Fu) | 0x64006400u, 0.000030517578125f, -0.03125f);
}
// Eight S1I0F15 codes (16 bytes) -> eight FP16 pairs (hi, lo) with hi + lo = the weight exactly.
__device__ __forceinline__ void expand_chunk_split_fixed16(const uint8_t *raw, uint4 &hi4, uint4 &lo4)
{
    const uint4 w = *reinterpret_cast<const uint4 *>(raw);
    fixed16_to_halves(w.x, hi4.x, lo4.x);
    fixed16_to_halves(w.y, hi4.y, lo4.y);
    fixed16_to_halves(w.z, hi4.z, lo4.z);
    fixed16_to_halves(w.w, hi4.w, lo4.w);
}

// Eight codes (one 16-byte chunk of halves) from their B packed bytes.
template <int B, int E>
__device__ __forceinline__ uint4 expand_chunk(const uint8_t *raw)
{
    if constexpr (B == 8 && E == 0) {        // S1I0F7
        const uint2 w = *reinterpret_cast<const uint2 *>(raw);
        uint4 o;
        fixed8_to_halves(w.x, o.x, o.y);
        fixed8_to_halves(w.y, o.z, o.w);
        return o;
    } else if constexpr (B == 12 && E == 0) {    // S1I0F11: pair p is bytes 3p .. 3p+2
        const uint32_t *rw = reinterpret_cast<const uint32_t *>(raw);
        const uint32_t w0 = rw[0], w1 = rw[1], w2 = rw[2];
        const uint32_t t0 = __byte_perm(w0, 0u, 0x2110), t1 = __byte_perm(w0, w1, 0x5443);
        const uint32_t t2 = __byte_perm(w1, w2, 0x4332), t3 = __byte_perm(w2, 0u, 0x3221);
        return make_uint4(fixed12_to_halves(t0), fixed12_to_halves(t1), fixed12_to_halves(t2), fixed12_to_halves(t3));
    } else if constexpr (B == 8 && E == 5) {        // a code is the top byte of its half
        const uint2 w = *reinterpret_cast<const uint2 *>(raw);
        return make_uint4(__byte_perm(w.x, 0u, 0x1404), __byte_perm(w.x, 0u, 0x3424),
                          __byte_perm(w.y, 0u, 0x1404), __byte_perm(w.y, 0u, 0x3424));
    } else if constexpr (B == 8) {           // S1E4M3
        const uint2 w = *reinterpret_cast<const uint2 *>(raw);
        uint4 o;
        narrow_to_halves<E>(w.x, o.x, o.y);
        narrow_to_halves<E>(w.y, o.z, o.w);
        return o;
    } else if constexpr (B == 6) {           // S1E2M3: 48 bits, spread to one code per byte
        const uint16_t *r16 = reinterpret_cast<const uint16_t *>(raw);
        const uint32_t a = r16[0], m = r16[1], z = r16[2];
        const uint32_t lo24 = a | ((m & 0xFFu) << 16), hi24 = (m >> 8) | (z << 8);
        auto spread = [](uint32_t t) {
            return (t & 0x3Fu) | ((t << 2) & 0x3F00u) | ((t << 4) & 0x3F0000u) | ((t << 6) & 0x3F000000u);
        };
        uint4 o;
        narrow_to_halves<E>(spread(lo24), o.x, o.y);
        narrow_to_halves<E>(spread(hi24), o.z, o.w);
        return o;
    } else {                                 // 12-bit codes: pair p is bytes 3p .. 3p+2, half = code << 4
        const uint32_t *rw = reinterpret_cast<const uint32_t *>(raw);
        const uint32_t w0 = rw[0], w1 = rw[1], w2 = rw[2];
        const uint32_t t0 = __byte_perm(w0, 0u, 0x2110), t1 = __byte_perm(w0, w1, 0x5443);
        const uint32_t t2 = __byte_perm(w1, w2, 0x4332), t3 = __byte_perm(w2, 0u, 0x3221);
        return make_uint4(((t0 << 4) & 0x0000FFF0u) | (t0 & 0xFFF00000u), ((t1 << 4) & 0x0000FFF0u) | (t1 & 0xFFF00000u),
                          ((t2 << 4) & 0x0000FFF0u) | (t2 & 0xFFF00000u), ((t3 << 4) & 0x0000FFF0u) | (t3 & 0xFFF00000u));
    }
}

// Odd widths: the chunk's B bytes start at any byte; four aligned words hold them.  A code is taken
// with its sign at bit 31 (one shift, or a funnel shift where it straddles two words); one arithmetic
// shift then puts exponent and mantissa where FP16 keeps them, with copies of the sign above, and a
// mask keeps bit 15 of those and drops what follows the code: the low half of the pair from a shift
// by 21 - E, the high half from a shift by 5 - E, so the pair needs no further assembly.
template <int B, int E>
__device__ __forceinline__ uint4 expand_chunk_odd(const uint8_t *raw)
{
    constexpr int M = B - 1 - E;
    constexpr uint32_t MAG = (1u << (E + M)) - 1u, INF_MAG = ((1u << E) - 1u) << M;
    constexpr uint32_t HMASK = 0x8000u | (MAG << (10 - M));
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(raw);
    const uint32_t sh = (a & 3u) * 8u;
    uint32_t w0, w1, w2, w3;
    asm volatile("ld.shared.u32 %0, [%4];\n\tld.shared.u32 %1, [%4+4];\n\tld.shared.u32 %2, [%4+8];\n\tld.shared.u32 %3, [%4+12];"
                 : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(a & ~3u));
    uint32_t v[4] = {__funnelshift_r(w0, w1, sh), __funnelshift_r(w1, w2, sh), __funnelshift_r(w2, w3, sh), w3 >> sh};
    auto top = [&](int j) -> uint32_t {          // code j in the top B bits of the result
        const int pos = j * B, wi = pos >> 5, bs = pos & 31;
        return (bs + B <= 32) ? (v[wi] << (32 - bs - B)) : __funnelshift_r(v[wi], v[wi + 1 < 4 ? wi + 1 : wi], bs + B - 32);
    };
    uint32_t h[4];
    bool special = false;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const uint32_t lo = (uint32_t)((int32_t)top(2 * p) >> (21 - E)) & HMASK;
        uint32_t hp = ((uint32_t)((int32_t)top(2 * p + 1) >> (5 - E)) & (HMASK << 16)) | lo;
        if constexpr (E != 5) {
            // exponent field + (15 - bias): one exact multiplication, subnormal codes included; a code with
            // an all-ones exponent field then has a magnitude of at least 2^(2^E - 1 - bias), every other less
            constexpr int BIAS = (1 << (E - 1)) - 1;
            const __half2 r = __hmul2(*reinterpret_cast<const __half2 *>(&hp), __float2half2_rn((float)(1u << (15 - BIAS))));
            special |= !__hblt2(__habs2(r), __float2half2_rn((float)(1u << ((1 << E) - 1 - BIAS))));
            hp = *reinterpret_cast<const uint32_t *>(&r);
        }
        h[p] = hp;
    }
    if (E != 5 && special) {         // rare: a weight is Inf or NaN
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t c = top(j) >> (32 - B);
            const uint32_t mag = c & MAG;
            if (mag >= INF_MAG) {
                const uint32_t hb = ((c >> (E + M)) << 15) | (mag == INF_MAG ? 0x7C00u : 0x7E00u);
                h[j >> 1] = (j & 1) ? ((h[j >> 1] & 0x0000FFFFu) | (hb << 16)) : ((h[j >> 1] & 0xFFFF0000u) | hb);
            }
        }
    }
    return make_uint4(h[0], h[1], h[2], h[3]);
}

// S1E4M14: eight 19-bit codes (19 bytes from any byte) -> eight FP16 pairs (hi, lo) with
// hi + lo = the weight exactly.  The weight is built as an FP32 value first (fields in place by one
// arithmetic shift and a mask, as above, then one exact multiplication by 2^(127 - 7) that also
// normalises subnormal codes), hi is its FP16 rounding, lo the FP16 value of the exact FP32
// remainder.  Inf / NaN codes: hi = Inf / NaN, lo = 0.
__device__ __forceinline__ void expand_chunk_split(const uint8_t *raw, uint4 &hi4, uint4 &lo4)
{
    constexpr int B = 19, E = 4, M = 14;
    constexpr uint32_t MAG = (1u << (E + M)) - 1u, INF_MAG = ((1u << E) - 1u) << M;
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(raw);
    const uint32_t sh = (a & 3u) * 8u;
    uint32_t w[6];
    asm volatile("ld.shared.u32 %0, [%6];\n\tld.shared.u32 %1, [%6+4];\n\tld.shared.u32 %2, [%6+8];\n\t"
                 "ld.shared.u32 %3, [%6+12];\n\tld.shared.u32 %4, [%6+16];\n\tld.shared.u32 %5, [%6+20];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]) : "r"(a & ~3u));
    uint32_t v[5];
#pragma unroll
    for (int i = 0; i < 5; ++i) v[i] = __funnelshift_r(w[i], w[i + 1], sh);
    auto top = [&](int j) -> uint32_t {          // code j in the top 19 bits of the result
        const int pos = j * B, wi = pos >> 5, bs = pos & 31;
        return (bs + B <= 32) ? (v[wi] << (32 - bs - B)) : __funnelshift_r(v[wi], v[wi + 1 < 5 ? wi + 1 : wi], bs + B - 32);
    };
    uint32_t h[4], l[4];
    bool special = false;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        float val[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const uint32_t placed = (uint32_t)((int32_t)top(2 * p + q) >> (8 - E)) & (0x80000000u | (MAG << (23 - M)));
            val[q] = __fmul_rn(__uint_as_float(placed), __uint_as_float((uint32_t)(127 - 7 + 127) << 23));
        }
        special |= !(fmaxf(fabsf(val[0]), fabsf(val[1])) < 256.f);      // an all-ones exponent field: 2^8 or more
        // both roundings as packed conversions of the pair (the one-value conversion runs at a quarter of the rate)
        const __half2 hh = __floats2half2_rn(val[0], val[1]);
        const float2 hf = __half22float2(hh);
        const __half2 ll = __floats2half2_rn(__fsub_rn(val[0], hf.x), __fsub_rn(val[1], hf.y));
        h[p] = *reinterpret_cast<const uint32_t *>(&hh);
        l[p] = *reinterpret_cast<const uint32_t *>(&ll);
    }
    if (special) {          // rare: a weight is Inf or NaN
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t c = top(j) >> (32 - B);
            const uint32_t mag = c & MAG;
            if (mag >= INF_MAG) {
                const uint32_t hb = ((c >> (E + M)) << 15) | (mag == INF_MAG ? 0x7C00u : 0x7E00u);
                h[j >> 1] = (j & 1) ? ((h[j >> 1] & 0x0000FFFFu) | (hb << 16)) : ((h[j >> 1] & 0xFFFF0000u) | hb);
                l[j >> 1] &= (j & 1) ? 0x0000FFFFu : 0xFFFF0000u;
            }
        }
    }
    hi4 = make_uint4(h[0], h[1], h[2], h[3]);
    lo4 = make_uint4(l[0], l[1], l[2], l[3]);
}

template <int B, int E>
__global__ void __launch_bounds__(Cfg<B, E>::THREADS, 1)
matmul_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
              const float *__restrict__ sb, const float *__restrict__ rowsum, float *__restrict__ y,
              uint32_t M, uint32_t N, uint32_t K, uint32_t *status, uint32_t inject_polls)
{
    using C = Cfg<B, E>;
    constexpr int NS = C::NSTAGES;
    // diagnostics (omc_plan_inject_wait_timeout): the producer announces its loads without issuing
    // them and every wait gives up after inject_polls polls, with no copy in flight
    const uint32_t limit = inject_polls ? inject_polls : WAIT_LIMIT;
    const bool skip_loads = inject_polls != 0u;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (saddr(smem_raw) + 1023u) & ~1023u;      // tiles need 1024-byte alignment
    const uint32_t bars = base + NS * C::STAGE;     // full[NS], decoded[NS], empty[NS], acc_full[2], acc_empty[2], tmem slot
    auto full = [&](int s) { return bars + 8u * s; };
    auto decoded = [&](int s) { return bars + 8u * (NS + s); };
    auto empty = [&](int s) { return bars + 8u * (2 * NS + s); };
    auto acc_full = [&](int b) { return bars + 8u * (3 * NS + b); };
    auto acc_empty = [&](int b) { return bars + 8u * (3 * NS + 2 + b); };
    const uint32_t tmem_slot = bars + 8u * (3 * NS + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t nkb = K / BK;
    constexpr int BN = C::BN, TILE_B_BYTES = C::TILE_B_BYTES;
    const uint32_t tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN - 1) / BN, ntiles = tiles_m * tiles_n;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full(s), 1);
            mbar_init(decoded(s), C::DECODE ? C::DEC_THREADS : 1);
            mbar_init(empty(s), 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 128); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // one warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    bool ok = true;
    if (tid == 0) {
        // ---- producer: per K block the X tile and either the code tile (halves) or its packed bytes
        uint32_t it = 0;
        for (uint32_t t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
            const int tm = t % tiles_m, tn = t / tiles_m;
            for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % NS;
                if (it >= (uint32_t)NS) ok = mbar_wait(empty(s), ((it / NS) - 1) & 1u, limit);
                if (!ok) break;
                mbar_expect_tx(full(s), C::TX_BYTES);
                if (skip_loads) continue;
                const uint32_t a = base + s * C::STAGE;
                tma_load_2d(a, &map_x, (int)(kb * BK), tm * BM, full(s));
                if constexpr (C::DECODE)      // odd widths: from the 16-byte boundary at or below the K block's first byte
                    tma_load_2d(a + TILE_A_BYTES + C::OPERAND_BYTES, &map_w, (int)((kb * C::ROW_BYTES) & ~15u), tn * BN, full(s));
                else
                    tma_load_2d(a + TILE_A_BYTES, &map_w, (int)(kb * BK), tn * BN, full(s));
            }
        }
    } else if (tid == 32) {
        // ---- MMA issuer: accumulator lt mod 2; a stage goes back to the producer when its MMAs have read it
        uint32_t it = 0, lt = 0;
        for (uint32_t t = blockIdx.x; t < ntiles && ok; t += gridDim.x, ++lt) {
            const uint32_t buf = lt & 1u;
            if (lt >= 2) ok = mbar_wait(acc_empty(buf), ((lt >> 1) - 1) & 1u, limit);   // the epilogue has drained it
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t d = tmem_base + buf * (uint32_t)BN;
            for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % NS;
                ok = mbar_wait(full(s), (it / NS) & 1u, limit);
                if constexpr (C::DECODE) ok = ok && mbar_wait(decoded(s), (it / NS) & 1u, limit);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a = base + s * C::STAGE, b = a + TILE_A_BYTES;
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                    umma_f16(d, umma_desc(a + k * UMMA_K * 2), umma_desc(b + k * UMMA_K * 2), (kb | k) != 0, C::IDESC);
                    if constexpr (C::SPLIT)      // the low parts of the weights, into the same accumulator
                        umma_f16(d, umma_desc(a + k * UMMA_K * 2), umma_desc(b + TILE_B_BYTES + k * UMMA_K * 2), 1u, C::IDESC);
                }
                umma_commit(empty(s));
            }
            if (ok) umma_commit(acc_full(buf));     // complete once all MMAs issued so far have finished
        }
    } else if (warp >= 2 && warp < 6) {
        // ---- epilogue: tensor-memory lane quarter = warp mod 4; one thread = one row of the tile
        const int q = warp & 3;
        const float s = __ldg(sb), b = __ldg(sb + 1);
        asm volatile("griddepcontrol.wait;" ::: "memory");      // the row sums of X are complete and visible
        uint32_t lt = 0;
        for (uint32_t t = blockIdx.x; t < ntiles; t += gridDim.x, ++lt) {
            const int tm = t % tiles_m, tn = t / tiles_m;
            const uint32_t buf = lt & 1u;
            ok = mbar_wait(acc_full(buf), (lt >> 1) & 1u, limit);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t row = tm * BM + q * 32 + lane;
            const float bias = (row < M) ? b * __ldg(rowsum + row) : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * (uint32_t)BN + (uint32_t)c0;
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                      "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                      "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                      "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const uint32_t col = tn * BN + c0;
                if (row < M && col < N) {
                    float4 *dst = reinterpret_cast<float4 *>(y + (size_t)row * N + col);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        dst[j] = make_float4(__fmaf_rn(s, __uint_as_float(v[4 * j]), bias), __fmaf_rn(s, __uint_as_float(v[4 * j + 1]), bias),
                                             __fmaf_rn(s, __uint_as_float(v[4 * j + 2]), bias), __fmaf_rn(s, __uint_as_float(v[4 * j + 3]), bias));
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(acc_empty(buf));
        }
    } else if (warp >= 6) {
        if constexpr (C::DECODE) {
            // ---- decoders: a tile is 2048 chunks of 8 codes (16 bytes of halves); thread t takes chunks
            // t, t + 256, ...  Consecutive lanes read consecutive 8- or 12-byte groups (no bank conflicts)
            // and the eight lanes of a row write its eight swizzled chunks, one full 128-byte line.
            // full(s) of block it implies that the MMAs of block it - NS have released the operand tile.
            uint8_t *const base_ptr = smem_raw + (base - saddr(smem_raw));
            const int t = tid - 192;
            const int c = t & 7;
            uint32_t it = 0;
            for (uint32_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % NS;
                    ok = mbar_wait(full(s), (it / NS) & 1u, limit);
                    if (!ok) break;
                    uint8_t *stage = base_ptr + s * C::STAGE;
                    const uint8_t *raw = stage + TILE_A_BYTES + C::OPERAND_BYTES + t * B;      // 8 codes = B bytes
                    uint8_t *dst = stage + TILE_A_BYTES;
                    const uint32_t off = C::ODD ? ((kb * C::ROW_BYTES) & 15u) : 0u;      // where the K block starts in its copy
#pragma unroll
                    for (int i = 0; i < BN * 8 / C::DEC_THREADS; ++i) {
                        const int r = i * (C::DEC_THREADS / 8) + (t >> 3);
                        uint4 o;
                        if constexpr (C::SPLIT) {
                            uint4 lo;
                            if constexpr (C::FIXED)
                                expand_chunk_split_fixed16(stage + TILE_A_BYTES + C::OPERAND_BYTES + r * C::BOX_BYTES + c * B, o, lo);
                            else
                                expand_chunk_split(stage + TILE_A_BYTES + C::OPERAND_BYTES + r * C::BOX_BYTES + off + c * B, o, lo);
                            *reinterpret_cast<uint4 *>(dst + TILE_B_BYTES + r * 128 + ((c ^ (r & 7)) << 4)) = lo;
                        } else if constexpr (C::ODD)
                            o = expand_chunk_odd<B, E>(stage + TILE_A_BYTES + C::OPERAND_BYTES + r * C::BOX_BYTES + off + c * B);
                        else
                            o = expand_chunk<B, E>(raw + i * C::DEC_THREADS * B);
                        // 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r mod 8)
                        *reinterpret_cast<uint4 *>(dst + r * 128 + ((c ^ (r & 7)) << 4)) = o;
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // visible to the tensor cores
                    mbar_arrive(decoded(s));
                }
            }
        }
    }
    if (!ok) atomicExch(status, 2u);

    // ---- release the tensor memory on every path
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [rows x cols] halves, cols contiguous; boxes of box_rows rows x 64 columns, 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {BK, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The packed codes of an N x K matrix as bytes: [rows x row_bytes], boxes of 256 rows x box_bytes, no swizzle.
bool make_raw_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t row_bytes, uint32_t box_bytes, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {row_bytes, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {box_bytes, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---------------------------------------------------------------------------------------------
// The same product on pairs of SMs.  Two CTAs of a cluster share one 256 x 256 tile of Y: each holds its own
// 128 rows of X and its own 128 rows of the codes per K block (with S1E5M10 32 KB instead of the 48 KB
// of the one-SM kernel for the same number of products, and six stages instead of four), the leader's
// MMA thread issues tcgen05.mma.cta_group::2 (M = 256: the upper 128 rows accumulate in the
// leader's tensor memory, the lower in its peer's; the 256 columns of the B operand are read from
// both CTAs' shared memory), and each CTA's epilogue warps store their own 128 rows.
//   full(s)      lives in the leader: its producer announces the bytes of both CTAs; both producers'
//                copies complete on it (bulk tensor copies in their cta_group::2 form, which may
//                signal the barrier of the pair's other CTA; no multicast).
//   empty(s)     one in each CTA, for its producer: the MMA thread's commit reaches both.
//   acc_full(b)  one in each CTA, for its epilogue: the commit after a tile's last MMA reaches both.
//   acc_empty(b) lives in the leader, 256 arrivals: the epilogue threads of both CTAs.
// The barriers are initialised before a cluster-wide barrier and nothing of the peer is touched
// before it; a second one before the tensor memory is released keeps either CTA alive while the
// other may still signal it.  Every mbarrier wait is bounded; a wait that runs out ends that role's
// loop, so that both CTAs always reach the closing barrier.
// Formats that are decoded on the way in: each CTA's decoder warps expand its own 128 rows (half the
// decoding per SM of the one-SM kernel), from packed bytes that arrive on a barrier of its own
// (rawfull(s): an ordinary bulk tensor copy); the leader's decoders arrive on decoded(s) in the
// leader, and the peer's idle MMA thread waits for its own decoders and forwards one arrival across
// the pair, so that the leader's MMA thread sees both halves ready with two waits.
template <int B, int E>
struct PairCfg {
    using C1 = Cfg<B, E>;
    static constexpr bool DECODE = C1::DECODE, ODD = C1::ODD, SPLIT = C1::SPLIT, FIXED = C1::FIXED;
    static constexpr int HALF = 128;                                  // rows of the codes per CTA
    static constexpr int TILE_B_BYTES = HALF * BK * 2;                // one operand tile of this CTA
    static constexpr int OPERAND_BYTES = (SPLIT ? 2 : 1) * TILE_B_BYTES;
    static constexpr int ROW_BYTES = C1::ROW_BYTES, BOX_BYTES = C1::BOX_BYTES;
    static constexpr int RAW_BYTES = DECODE ? HALF * BOX_BYTES : 0;
    static constexpr int STAGE = TILE_A_BYTES + OPERAND_BYTES + RAW_BYTES;
    static constexpr int MAX_STAGES = 6;
    static constexpr int FIT = (227 * 1024 - 1280) / STAGE;
    static constexpr int NSTAGES = FIT < MAX_STAGES ? FIT : MAX_STAGES;
    static constexpr int SMEM = NSTAGES * STAGE + 1024 /* alignment slack */ + 256 /* barriers, tmem slot */;
    static constexpr int DEC_THREADS = DECODE ? MATMUL_DECODER_THREADS : 0;
    static constexpr int THREADS = 192 + DEC_THREADS;
    // what completes on the leader's full(s): the X tiles of both CTAs, and without decoding their operand tiles too
    static constexpr uint32_t FULL_TX = 2u * (TILE_A_BYTES + (DECODE ? 0 : TILE_B_BYTES));
    static constexpr uint32_t IDESC = (1u << 4) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
    static_assert(STAGE % 1024 == 0, "operand tiles stay 1024-byte aligned");
    static_assert(NSTAGES >= 2 && 8 * (4 * NSTAGES + 5) <= 256, "stages and their barriers fit");
};

__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// The shared::cluster address of the same location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Tile into this CTA's shared memory; the bytes complete on `bar`, a shared::cluster address in either CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
// Arrives, once the MMAs issued so far have finished, on the barrier at this address in both CTAs.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(both) : "memory");
}
// Arrival on a barrier of the pair's other CTA (or this one), in the plain form: a release of cluster
// scope on every arrival makes the forwarder of the decoders' completion the slowest link of the
// pipeline (measured: S1E5M2 0.51 ms against 0.27 ms), and what it would order is already ordered,
// since the operand bytes stay in the shared memory of the SM that wrote them, were handed to the
// asynchronous proxy there (fence.proxy.async by their writers, before their own arrival), and are
// read by that SM's half of the pair's MMA, which is issued only after this arrival was seen.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

template <int B, int E>
__global__ void __launch_bounds__(PairCfg<B, E>::THREADS, 1)
matmul_pair_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                   const float *__restrict__ sb, const float *__restrict__ rowsum, float *__restrict__ y,
                   uint32_t M, uint32_t N, uint32_t K, uint32_t *status, uint32_t inject_polls)
{
    using C = PairCfg<B, E>;
    constexpr int NS = C::NSTAGES, TILE_B_BYTES = C::TILE_B_BYTES;
    const uint32_t limit = inject_polls ? inject_polls : WAIT_LIMIT;
    const bool skip_loads = inject_polls != 0u;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (saddr(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + NS * C::STAGE;   // full[NS], rawfull[NS], decoded[NS], empty[NS], acc_full[2], acc_empty[2], tmem slot
    auto full = [&](int s) { return bars + 8u * s; };
    auto rawfull = [&](int s) { return bars + 8u * (NS + s); };
    auto decoded = [&](int s) { return bars + 8u * (2 * NS + s); };
    auto empty = [&](int s) { return bars + 8u * (3 * NS + s); };
    auto acc_full = [&](int b) { return bars + 8u * (4 * NS + b); };
    auto acc_empty = [&](int b) { return bars + 8u * (4 * NS + 2 + b); };
    const uint32_t tmem_slot = bars + 8u * (4 * NS + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_cta_rank();          // 0: the leader
    const uint32_t nkb = K / BK;
    const uint32_t tiles_m = (M + 255) / 256, tiles_n = (N + 255) / 256, ntiles = tiles_m * tiles_n;
    const uint32_t pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full(s), 1);
            mbar_init(rawfull(s), 1);
            // the leader's: its own decoders and the arrival its peer forwards
            mbar_init(decoded(s), C::DECODE ? C::DEC_THREADS + (rank == 0 ? 1 : 0) : 1);
            mbar_init(empty(s), 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 256); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs allocates the pair's tensor memory
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_barrier();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    bool ok = true;
    if (tid == 0) {
        // ---- producer of this CTA: its 128 rows of X and its 128 rows of the codes (halves, or their packed bytes) per K block
        uint32_t it = 0;
        for (uint32_t t = pair; t < ntiles && ok; t += npairs) {
            const int tm = t % tiles_m, tn = t / tiles_m;
            for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % NS;
                if (it >= (uint32_t)NS) ok = mbar_wait(empty(s), ((it / NS) - 1) & 1u, limit);
                if (!ok) break;
                if (rank == 0) mbar_expect_tx(full(s), C::FULL_TX);              // the bytes of both CTAs
                if constexpr (C::DECODE) mbar_expect_tx(rawfull(s), C::RAW_BYTES);
                if (skip_loads) continue;
                const uint32_t a = base + s * C::STAGE, lead_full = map_to_cta(full(s), 0u);
                tma_load_2d_pair(a, &map_x, (int)(kb * BK), tm * 256 + (int)rank * 128, lead_full);
                if constexpr (C::DECODE)      // odd widths: from the 16-byte boundary at or below the K block's first byte
                    tma_load_2d(a + TILE_A_BYTES + C::OPERAND_BYTES, &map_w, (int)((kb * C::ROW_BYTES) & ~15u),
                                tn * 256 + (int)rank * C::HALF, rawfull(s));
                else
                    tma_load_2d_pair(a + TILE_A_BYTES, &map_w, (int)(kb * BK), tn * 256 + (int)rank * C::HALF, lead_full);
            }
        }
    } else if (tid == 32 && rank == 0) {
        // ---- MMA issuer (leader only): accumulator lt mod 2 in both CTAs' tensor memory
        uint32_t it = 0, lt = 0;
        for (uint32_t t = pair; t < ntiles && ok; t += npairs, ++lt) {
            const uint32_t buf = lt & 1u;
            if (lt >= 2) ok = mbar_wait(acc_empty(buf), ((lt >> 1) - 1) & 1u, limit);   // both epilogues have drained it
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t d = tmem_base + buf * 256u;
            for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % NS;
                ok = mbar_wait(full(s), (it / NS) & 1u, limit);
                if constexpr (C::DECODE) ok = ok && mbar_wait(decoded(s), (it / NS) & 1u, limit);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a = base + s * C::STAGE, b = a + TILE_A_BYTES;
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                    umma_f16_pair(d, umma_desc(a + k * UMMA_K * 2), umma_desc(b + k * UMMA_K * 2), (kb | k) != 0, C::IDESC);
                    if constexpr (C::SPLIT)      // the low parts of the weights, into the same accumulator
                        umma_f16_pair(d, umma_desc(a + k * UMMA_K * 2), umma_desc(b + TILE_B_BYTES + k * UMMA_K * 2), 1u, C::IDESC);
                }
                umma_commit_pair(empty(s));          // the stage goes back to both producers
            }
            if (ok) umma_commit_pair(acc_full(buf));
        }
    } else if (tid == 32) {
        // ---- the peer's MMA thread has no products to issue: it tells the leader when its decoders are through
        if constexpr (C::DECODE) {
            uint32_t it = 0;
            for (uint32_t t = pair; t < ntiles && ok; t += npairs) {
                for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % NS;
                    ok = mbar_wait(decoded(s), (it / NS) & 1u, limit);
                    if (!ok) break;
                    mbar_arrive_cluster(map_to_cta(decoded(s), 0u));
                }
            }
        }
    } else if (warp >= 2 && warp < 6) {
        // ---- epilogue of this CTA: its 128 rows of the tile; tensor-memory lane quarter = warp mod 4
        const int q = warp & 3;
        const float s = __ldg(sb), b = __ldg(sb + 1);
        asm volatile("griddepcontrol.wait;" ::: "memory");      // the row sums of X are complete and visible
        uint32_t lt = 0;
        for (uint32_t t = pair; t < ntiles; t += npairs, ++lt) {
            const int tm = t % tiles_m, tn = t / tiles_m;
            const uint32_t buf = lt & 1u;
            ok = mbar_wait(acc_full(buf), (lt >> 1) & 1u, limit);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t row = tm * 256 + rank * 128 + q * 32 + lane;
            const float bias = (row < M) ? b * __ldg(rowsum + row) : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < 256; c0 += 32) {
                uint32_t v[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * 256u + (uint32_t)c0;
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                      "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                      "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                      "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const uint32_t col = tn * 256 + c0;
                if (row < M && col < N) {
                    float4 *dst = reinterpret_cast<float4 *>(y + (size_t)row * N + col);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        dst[j] = make_float4(__fmaf_rn(s, __uint_as_float(v[4 * j]), bias), __fmaf_rn(s, __uint_as_float(v[4 * j + 1]), bias),
                                             __fmaf_rn(s, __uint_as_float(v[4 * j + 2]), bias), __fmaf_rn(s, __uint_as_float(v[4 * j + 3]), bias));
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive_cluster(map_to_cta(acc_empty(buf), 0u));
        }
    } else if (warp >= 6) {
        if constexpr (C::DECODE) {
            // ---- decoders of this CTA: its 128 rows are 1024 chunks of 8 codes; thread t takes chunks t and t + 512.
            // rawfull(s) of block it implies that the MMAs of block it - NS have released the operand tile.
            uint8_t *const base_ptr = smem_raw + (base - saddr(smem_raw));
            const int t = tid - 192;
            const int c = t & 7;
            uint32_t it = 0;
            for (uint32_t tile = pair; tile < ntiles && ok; tile += npairs) {
                for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % NS;
                    ok = mbar_wait(rawfull(s), (it / NS) & 1u, limit);
                    if (!ok) break;
                    uint8_t *stage = base_ptr + s * C::STAGE;
                    const uint8_t *raw = stage + TILE_A_BYTES + C::OPERAND_BYTES + t * B;      // 8 codes = B bytes
                    uint8_t *dst = stage + TILE_A_BYTES;
                    const uint32_t off = C::ODD ? ((kb * C::ROW_BYTES) & 15u) : 0u;      // where the K block starts in its copy
#pragma unroll
                    for (int i = 0; i < C::HALF * 8 / C::DEC_THREADS; ++i) {
                        const int r = i * (C::DEC_THREADS / 8) + (t >> 3);
                        uint4 o;
                        if constexpr (C::SPLIT) {
                            uint4 lo;
                            if constexpr (C::FIXED)
                                expand_chunk_split_fixed16(stage + TILE_A_BYTES + C::OPERAND_BYTES + r * C::BOX_BYTES + c * B, o, lo);
                            else
                                expand_chunk_split(stage + TILE_A_BYTES + C::OPERAND_BYTES + r * C::BOX_BYTES + off + c * B, o, lo);
                            *reinterpret_cast<uint4 *>(dst + TILE_B_BYTES + r * 128 + ((c ^ (r & 7)) << 4)) = lo;
                        } else if constexpr (C::ODD)
                            o = expand_chunk_odd<B, E>(stage + TILE_A_BYTES + C::OPERAND_BYTES + r * C::BOX_BYTES + off + c * B);
                        else
                            o = expand_chunk<B, E>(raw + i * C::DEC_THREADS * B);
                        // 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r mod 8)
                        *reinterpret_cast<uint4 *>(dst + r * 128 + ((c ^ (r & 7)) << 4)) = o;
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // visible to the tensor cores
                    mbar_arrive(decoded(s));
                }
            }
        }
    }
    if (!ok) atomicExch(status, 2u);

    // ---- both CTAs are through with each other's barriers and tensor memory before either lets go
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_barrier();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
}

template <int B, int E>
int launch(const CUtensorMap &map_x, const void *codes, const float *sb, const float *rowsum, float *y,
           uint32_t M, uint32_t N, uint32_t K, uint32_t n_sm, uint32_t *status, uint32_t inject_polls, cudaStream_t st)
{
    using C = Cfg<B, E>;
    CUtensorMap map_w;
    constexpr int BN = C::BN;
    if (C::DECODE ? !make_raw_map(&map_w, codes, N, (uint64_t)K * B / 8, C::BOX_BYTES, BN) : !make_map(&map_w, codes, N, K, BN))
        return OMC_ERR_CUDA;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        int rc = omc::note_cuda(cudaFuncSetAttribute(matmul_kernel<B, E>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
        if (rc) return rc;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const uint32_t ntiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
    const uint32_t grid = ntiles < n_sm ? ntiles : n_sm;
    // the programmatic dependent of rowsum_kernel: set-up, copies and products overlap it
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return omc::note_cuda(cudaLaunchKernelEx(&cfg, matmul_kernel<B, E>, map_x, map_w, sb, rowsum, y, M, N, K, status, inject_polls));
}

// The kernel on pairs of SMs: clusters of two CTAs, one cluster per pair of SMs.
template <int B, int E>
int launch_pair(const CUtensorMap &map_x, const void *codes, const float *sb, const float *rowsum, float *y,
                uint32_t M, uint32_t N, uint32_t K, uint32_t n_sm, uint32_t *status, uint32_t inject_polls, cudaStream_t st)
{
    using C = PairCfg<B, E>;
    CUtensorMap map_w;
    if (C::DECODE ? !make_raw_map(&map_w, codes, N, (uint64_t)K * B / 8, C::BOX_BYTES, C::HALF) : !make_map(&map_w, codes, N, K, C::HALF))
        return OMC_ERR_CUDA;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        int rc = omc::note_cuda(cudaFuncSetAttribute(matmul_pair_kernel<B, E>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
        if (rc) return rc;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const uint32_t ntiles = ((M + 255) / 256) * ((N + 255) / 256);
    const uint32_t max_pairs = n_sm / 2 ? n_sm / 2 : 1;
    const uint32_t npairs = ntiles < max_pairs ? ntiles : max_pairs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * npairs);
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // the programmatic dependent of rowsum_kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return omc::note_cuda(cudaLaunchKernelEx(&cfg, matmul_pair_kernel<B, E>, map_x, map_w, sb, rowsum, y, M, N, K, status, inject_polls));
}

// A tile of the kernel on pairs of SMs is 256 x 256: smaller products stay on the one-SM kernel.
template <int B, int E>
int launch_either(const CUtensorMap &map_x, const void *codes, const float *sb, const float *rowsum, float *y,
                  uint32_t M, uint32_t N, uint32_t K, uint32_t n_sm, uint32_t *status, uint32_t inject_polls, cudaStream_t st)
{
    if (M >= 256 && N >= 256 && n_sm >= 2) return launch_pair<B, E>(map_x, codes, sb, rowsum, y, M, N, K, n_sm, status, inject_polls, st);
    return launch<B, E>(map_x, codes, sb, rowsum, y, M, N, K, n_sm, status, inject_polls, st);
}

}  // namespace

extern "C" int omc_matmul(const omc_plan_t *plan, uint32_t var, const uint8_t *packed, const float *sb,
                          const void *x_half, uint32_t M, uint32_t N, uint32_t K, float *y, float *rowsum_scratch,
                          void *stream)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    if (!plan->d_vars) return OMC_ERR_PLAN_MISMATCH;
    {   // the plan's tables and status word live on the device it was prepared on
        int dev = 0;
        const int rc = omc::note_cuda(cudaGetDevice(&dev));
        if (rc) return rc;
        if (dev != plan->device) return OMC_ERR_PLAN_MISMATCH;
    }
    if (!packed || !sb || !x_half || !y || !rowsum_scratch) return OMC_ERR_NULL_PTR;
    if (var >= plan->nvars || !plan->vars[var].quantised) return OMC_ERR_INVALID_ARG;
    const int exp = plan->fmt.exp_bits, man = plan->fmt.man_bits;
    const bool fixed = (plan->fmt.flags & OMC_FORMAT_FIXED_POINT) != 0;
    if (fixed && !(exp == 0 && (man == 7 || man == 11 || man == 15))) return OMC_ERR_BAD_FORMAT;   // S1I0F7 / F11 / F15
    const bool half_family = !fixed && exp == 5 && (man == 10 || man == 6 || man == 2);
    const bool narrow = !fixed && ((exp == 4 && man == 3) || (exp == 2 && man == 3));
    const bool split = !fixed && exp == 4 && man == 14;
    const bool odd = !fixed && ((exp == 5 && man == 7) || (exp == 3 && man == 7) || (exp == 3 && man == 9) ||
                               (exp == 4 && man == 8) || split);
    if (!fixed && !half_family && !narrow && !odd) return OMC_ERR_BAD_FORMAT;
    if (odd && K % 128 != 0) return OMC_ERR_INVALID_ARG;      // a row of 11- or 13-bit codes must be whole 16-byte units
    if (M == 0 || N == 0 || K == 0 || N % 128 != 0 || K % BK != 0 || (uint64_t)N * K != plan->vars[var].n)
        return OMC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(packed) | reinterpret_cast<uintptr_t>(x_half) | reinterpret_cast<uintptr_t>(y) |
         reinterpret_cast<uintptr_t>(sb)) & 15u)
        return OMC_ERR_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(rowsum_scratch) & 3u) return OMC_ERR_MISALIGNED;
    const omc::VarDev &v = plan->vars[var];
    CUtensorMap map_x;
    if (!make_map(&map_x, x_half, M, K, BM)) return OMC_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rowsum_kernel<<<(M + 7) / 8, 256, 0, st>>>(static_cast<const __half *>(x_half), M, K, rowsum_scratch);
    const uint8_t *codes = packed + v.store_off;
    const float *sbv = sb + 2 * v.sb_slot;
    const uint32_t n_sm = plan->n_sm ? plan->n_sm : 1;
    const uint32_t inject = plan->inject_polls;      // diagnostics: applies to this launch only
    plan->inject_polls = 0;
    if (fixed) {
        if (man == 7) return launch_either<8, 0>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
        if (man == 11) return launch_either<12, 0>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
        return launch_either<16, 0>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    }
    if (split) return launch_either<19, 4>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    if (odd) {
        if (exp == 5) return launch_either<13, 5>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
        if (exp == 4) return launch_either<13, 4>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
        if (man == 9) return launch_either<13, 3>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
        return launch_either<11, 3>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    }
    if (exp == 4) return launch_either<8, 4>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    if (exp == 2) return launch_either<6, 2>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    switch (man) {
    case 10: return launch_either<16, 5>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    case 6: return launch_either<12, 5>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    default: return launch_either<8, 5>(map_x, codes, sbv, rowsum_scratch, y, M, N, K, n_sm, plan->d_status, inject, st);
    }
}
