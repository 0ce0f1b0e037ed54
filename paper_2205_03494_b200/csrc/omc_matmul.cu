// omc_matmul: the forward path of Fig. 1 with the decompression fused into the consumer.
//
// A layer's weight matrix W (N x K, K contiguous) is held as S1E5M10 codes, which are IEEE half
// bit patterns; the transformed weight is Wbar = s*Wt + b (Sec. 2.3), so
//     Y = X * Wbar^T = s * (X * Wt^T) + b * rowsum(X).
// The codes therefore go straight from the packed arena into shared memory (TMA, 128-byte swizzle)
// and from there into the 5th-generation tensor cores as the B operand: the transient FP32 copy of
// the weights that omc_decompress would write, and a GEMM would read back, never exists.
//
// One CTA computes a 128 x 128 tile of Y: thread 0 runs a three-stage TMA pipeline over K (64
// columns per stage), thread 32 issues tcgen05.mma (128x128x16, FP16 inputs, FP32 accumulator in
// tensor memory) and commits each stage back to the producer, then all four warps read the
// accumulator with tcgen05.ld and apply the epilogue above.  Every wait is bounded; a wait that
// runs out sets the plan's status word, and the tensor memory is released on every path.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "omc_internal.h"

namespace omc {
int note_cuda(cudaError_t e);
}

namespace {

constexpr int BM = 128, BN = 128, BK = 64;       // CTA tile; BK halves = one 128-byte swizzle row
constexpr int STAGES = 3;                      // 3 x 32 KB per CTA: two CTAs fit one SM, so one computes while the other stores
constexpr int UMMA_K = 16;                       // K of one tcgen05.mma with 16-bit inputs
constexpr int TILE_A_BYTES = BM * BK * 2, TILE_B_BYTES = BN * BK * 2;
constexpr int STAGE_BYTES = TILE_A_BYTES + TILE_B_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers, tmem slot */;
constexpr int TMEM_COLS = 128;                   // 128 lanes x 128 FP32 columns
constexpr uint32_t WAIT_LIMIT = 1u << 20;   // polls of one mbarrier before giving up

__device__ __forceinline__ uint32_t saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false if it never completed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
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
// Instruction descriptor: D = FP32 (bits 4-5 = 1), A = B = FP16 (0), both K-major, N/8 at bit 17, M/16 at bit 24.
constexpr uint32_t IDESC = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(IDESC), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__global__ void rowsum_kernel(const __half *__restrict__ x, uint32_t M, uint32_t K, float *__restrict__ out)
{
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

__global__ void __launch_bounds__(128, 2)
matmul_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
              const float *__restrict__ sb, const float *__restrict__ rowsum, float *__restrict__ y,
              uint32_t M, uint32_t N, uint32_t K, uint32_t *status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (saddr(smem_raw) + 1023u) & ~1023u;      // tiles need 1024-byte alignment
    const uint32_t bars = base + STAGES * STAGE_BYTES;             // full[S], empty[S], accum, tmem slot
    auto full = [&](int s) { return bars + 8u * s; };
    auto empty = [&](int s) { return bars + 8u * (STAGES + s); };
    const uint32_t accum_bar = bars + 8u * (2 * STAGES);
    const uint32_t tmem_slot = bars + 8u * (2 * STAGES + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile_n = blockIdx.x, tile_m = blockIdx.y;
    const uint32_t nkb = K / BK;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        mbar_init(accum_bar, 1);
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
        // ---- producer: TMA loads of the X tile and the code tile of each K block
        for (uint32_t kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % STAGES;
            if (kb >= STAGES) ok = mbar_wait(empty(s), ((kb / STAGES) - 1) & 1u);
            if (!ok) break;
            mbar_expect_tx(full(s), STAGE_BYTES);
            const uint32_t a = base + s * STAGE_BYTES, b = a + TILE_A_BYTES;
            tma_load_2d(a, &map_x, (int)(kb * BK), tile_m * BM, full(s));
            tma_load_2d(b, &map_w, (int)(kb * BK), tile_n * BN, full(s));
        }
    } else if (tid == 32) {
        // ---- MMA issuer
        for (uint32_t kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % STAGES;
            ok = mbar_wait(full(s), (kb / STAGES) & 1u);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a = base + s * STAGE_BYTES, b = a + TILE_A_BYTES;
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
                umma_f16(tmem_base, umma_desc(a + k * UMMA_K * 2), umma_desc(b + k * UMMA_K * 2), (kb | k) != 0);
            umma_commit(empty(s));          // the stage is free once these MMAs have read it
        }
        if (ok) umma_commit(accum_bar);     // the accumulator is complete once all MMAs have finished
    }
    if (!ok) atomicExch(status, 2u);

    // ---- epilogue: every warp reads its 32 accumulator rows and writes s*acc + b*rowsum(x)
    __syncwarp();
    bool ready = mbar_wait(accum_bar, 0);
    ready = __all_sync(0xFFFFFFFFu, ready);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ready) {
        const float s = __ldg(sb), b = __ldg(sb + 1);
        const uint32_t row = tile_m * BM + warp * 32 + lane;
        const float bias = (row < M) ? b * __ldg(rowsum + row) : 0.f;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0;
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                  "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                  "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                  "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                : "r"(taddr));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (row < M) {
                float4 *dst = reinterpret_cast<float4 *>(y + (size_t)row * N + (size_t)tile_n * BN + c0);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    dst[j] = make_float4(__fmaf_rn(s, __uint_as_float(r[4 * j]), bias), __fmaf_rn(s, __uint_as_float(r[4 * j + 1]), bias),
                                         __fmaf_rn(s, __uint_as_float(r[4 * j + 2]), bias), __fmaf_rn(s, __uint_as_float(r[4 * j + 3]), bias));
            }
        }
    } else if (lane == 0) {
        atomicExch(status, 2u);
    }
    // ---- release the tensor memory on every path
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
}


// ---------------------------------------------------------------------------------------------
// The same product for the narrower E = 5 formats (S1E5M6: 12-bit codes, S1E5M2: 8-bit codes),
// where decompression is real work: code << (10 - M) is the IEEE half.  The packed codes of a
// 128 x 64 tile arrive by TMA as raw bytes; four warps expand them (byte permutes and shifts only)
// straight into the 128-byte-swizzled operand tile the tensor cores read; the FP32 or FP16 weights
// are never materialised anywhere else.  Warp 0: TMA producer, warp 1: MMA issuer and tensor-memory
// owner, warps 2-5: decoders, then the epilogue.

template <int B>
struct DecodeCfg {
    static constexpr int ROW_BYTES = BK * B / 8;                 // one tile row of codes: 64 or 96 bytes
    static constexpr int RAW_BYTES = BN * ROW_BYTES;
    static constexpr int STAGE = TILE_A_BYTES + TILE_B_BYTES + RAW_BYTES;
#ifndef OMC_MM_DECODE_STAGES
#define OMC_MM_DECODE_STAGES 2
#endif
#ifndef OMC_MM_DECODE_CTAS
#define OMC_MM_DECODE_CTAS 2
#endif
    static constexpr int NSTAGES = OMC_MM_DECODE_STAGES;
    static constexpr int SMEM = NSTAGES * STAGE + 1024 + 256;
    static_assert(STAGE % 1024 == 0, "operand tiles stay 1024-byte aligned");
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int B>
__global__ void __launch_bounds__(192, OMC_MM_DECODE_CTAS)
matmul_decode_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_raw,
                     const float *__restrict__ sb, const float *__restrict__ rowsum, float *__restrict__ y,
                     uint32_t M, uint32_t N, uint32_t K, uint32_t *status)
{
    using C = DecodeCfg<B>;
    constexpr int NS = C::NSTAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (saddr(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - saddr(smem_raw));
    const uint32_t bars = base + NS * C::STAGE;                  // full[NS], decoded[NS], empty[NS], accum, slot
    auto full = [&](int s) { return bars + 8u * s; };
    auto decoded = [&](int s) { return bars + 8u * (NS + s); };
    auto empty = [&](int s) { return bars + 8u * (2 * NS + s); };
    const uint32_t accum_bar = bars + 8u * (3 * NS);
    const uint32_t tmem_slot = bars + 8u * (3 * NS + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile_n = blockIdx.x, tile_m = blockIdx.y;
    const uint32_t nkb = K / BK;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full(s), 1); mbar_init(decoded(s), 128); mbar_init(empty(s), 1); }
        mbar_init(accum_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
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
        // ---- producer: X tile (swizzled) and the raw code bytes of the W tile
        for (uint32_t kb = 0; kb < nkb; ++kb) {
            const int s = kb % NS;
            if (kb >= (uint32_t)NS) ok = mbar_wait(empty(s), ((kb / NS) - 1) & 1u);
            if (!ok) break;
            mbar_expect_tx(full(s), TILE_A_BYTES + C::RAW_BYTES);
            const uint32_t a = base + s * C::STAGE;
            tma_load_2d(a, &map_x, (int)(kb * BK), tile_m * BM, full(s));
            tma_load_2d(a + TILE_A_BYTES + TILE_B_BYTES, &map_raw, (int)(kb * C::ROW_BYTES), tile_n * BN, full(s));
        }
    } else if (tid == 32) {
        // ---- MMA issuer: needs the X tile (full) and the expanded W tile (decoded)
        for (uint32_t kb = 0; kb < nkb; ++kb) {
            const int s = kb % NS;
            ok = mbar_wait(full(s), (kb / NS) & 1u) && mbar_wait(decoded(s), (kb / NS) & 1u);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a = base + s * C::STAGE, b = a + TILE_A_BYTES;
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
                umma_f16(tmem_base, umma_desc(a + k * UMMA_K * 2), umma_desc(b + k * UMMA_K * 2), (kb | k) != 0);
            umma_commit(empty(s));
        }
        if (ok) umma_commit(accum_bar);
    } else if (warp >= 2) {
        // ---- decoders: the tile is 1024 chunks of 8 codes (16 bytes of halves); thread t takes chunks
        // t, t + 128, ...  Consecutive lanes read consecutive 8- or 12-byte groups (no bank conflicts)
        // and the eight lanes of a row write its eight swizzled chunks, one full 128-byte line.
        const int t = tid - 64;
        const int c = t & 7;
        for (uint32_t kb = 0; kb < nkb; ++kb) {
            const int s = kb % NS;
            // the operand tile of this stage was last read by the MMAs of block kb - NS
            if (kb >= (uint32_t)NS) ok = mbar_wait(empty(s), ((kb / NS) - 1) & 1u);
            ok = ok && mbar_wait(full(s), (kb / NS) & 1u);
            if (!ok) break;
            uint8_t *stage = base_ptr + s * C::STAGE;
            const uint32_t *raw = reinterpret_cast<const uint32_t *>(stage + TILE_A_BYTES + TILE_B_BYTES) + t * (B / 4);
            uint8_t *dst = stage + TILE_A_BYTES;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = i * 16 + (t >> 3);
                uint4 o;
                if constexpr (B == 8) {              // a code is the top byte of its half
                    const uint2 w = *reinterpret_cast<const uint2 *>(raw + i * 128 * 2);
                    o = make_uint4(__byte_perm(w.x, 0u, 0x1404), __byte_perm(w.x, 0u, 0x3424),
                                   __byte_perm(w.y, 0u, 0x1404), __byte_perm(w.y, 0u, 0x3424));
                } else {                             // 12-bit codes: pair p is bytes 3p .. 3p+2, half = code << 4
                    const uint32_t w0 = raw[i * 128 * 3], w1 = raw[i * 128 * 3 + 1], w2 = raw[i * 128 * 3 + 2];
                    const uint32_t t0 = __byte_perm(w0, 0u, 0x2110), t1 = __byte_perm(w0, w1, 0x5443);
                    const uint32_t t2 = __byte_perm(w1, w2, 0x4332), t3 = __byte_perm(w2, 0u, 0x3221);
                    o = make_uint4(((t0 << 4) & 0x0000FFF0u) | (t0 & 0xFFF00000u), ((t1 << 4) & 0x0000FFF0u) | (t1 & 0xFFF00000u),
                                   ((t2 << 4) & 0x0000FFF0u) | (t2 & 0xFFF00000u), ((t3 << 4) & 0x0000FFF0u) | (t3 & 0xFFF00000u));
                }
                // 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r mod 8)
                *reinterpret_cast<uint4 *>(dst + r * 128 + ((c ^ (r & 7)) << 4)) = o;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // visible to the tensor cores
            mbar_arrive(decoded(s));
        }
    }
    if (!ok) atomicExch(status, 2u);

    // ---- epilogue by warps 2-5 (tensor-memory lane quarter = warp mod 4)
    __syncwarp();
    if (warp >= 2) {
        bool ready = mbar_wait(accum_bar, 0);
        ready = __all_sync(0xFFFFFFFFu, ready);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ready) {
            const int q = warp & 3;
            const float s = __ldg(sb), b = __ldg(sb + 1);
            const uint32_t row = tile_m * BM + q * 32 + lane;
            const float bias = (row < M) ? b * __ldg(rowsum + row) : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0;
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
                if (row < M) {
                    float4 *dst = reinterpret_cast<float4 *>(y + (size_t)row * N + (size_t)tile_n * BN + c0);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        dst[j] = make_float4(__fmaf_rn(s, __uint_as_float(v[4 * j]), bias), __fmaf_rn(s, __uint_as_float(v[4 * j + 1]), bias),
                                             __fmaf_rn(s, __uint_as_float(v[4 * j + 2]), bias), __fmaf_rn(s, __uint_as_float(v[4 * j + 3]), bias));
                }
            }
        } else if (lane == 0) {
            atomicExch(status, 2u);
        }
    }
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

// [rows x cols] halves, cols contiguous; boxes of 128 rows x 64 columns, 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t cols)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {BK, BM};
    const cuuint32_t elem[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The packed codes of an N x K matrix as bytes: [rows x row_bytes], boxes of 128 rows x box_bytes, no swizzle.
bool make_raw_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t row_bytes, uint32_t box_bytes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {row_bytes, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {box_bytes, BN};
    const cuuint32_t elem[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int B>
int launch_decode(const CUtensorMap &map_x, const void *codes, const float *sb, const float *rowsum, float *y,
                  uint32_t M, uint32_t N, uint32_t K, uint32_t *status, cudaStream_t st)
{
    using C = DecodeCfg<B>;
    CUtensorMap map_raw;
    if (!make_raw_map(&map_raw, codes, N, (uint64_t)K * B / 8, C::ROW_BYTES)) return OMC_ERR_CUDA;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        int rc = omc::note_cuda(cudaFuncSetAttribute(matmul_decode_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
        if (rc) return rc;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    dim3 grid(N / BN, (M + BM - 1) / BM);
    matmul_decode_kernel<B><<<grid, 192, C::SMEM, st>>>(map_x, map_raw, sb, rowsum, y, M, N, K, status);
    return omc::note_cuda(cudaGetLastError());
}

}  // namespace

extern "C" int omc_matmul(const omc_plan_t *plan, uint32_t var, const uint8_t *packed, const float *sb,
                          const void *x_half, uint32_t M, uint32_t N, uint32_t K, float *y, float *rowsum_scratch,
                          void *stream)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    if (!plan->d_vars) return OMC_ERR_PLAN_MISMATCH;
    if (!packed || !sb || !x_half || !y || !rowsum_scratch) return OMC_ERR_NULL_PTR;
    if (var >= plan->nvars || !plan->vars[var].quantised) return OMC_ERR_INVALID_ARG;
    const int man = plan->fmt.man_bits;
    if (plan->fmt.exp_bits != 5 || (man != 10 && man != 6 && man != 2)) return OMC_ERR_BAD_FORMAT;
    if (M == 0 || N == 0 || K == 0 || N % BN != 0 || K % BK != 0 || (uint64_t)N * K != plan->vars[var].n)
        return OMC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(packed) | reinterpret_cast<uintptr_t>(x_half) | reinterpret_cast<uintptr_t>(y)) & 15u)
        return OMC_ERR_MISALIGNED;
    const omc::VarDev &v = plan->vars[var];
    CUtensorMap map_x, map_w;
    if (!make_map(&map_x, x_half, M, K)) return OMC_ERR_CUDA;
    if (man != 10) {
        cudaStream_t st2 = static_cast<cudaStream_t>(stream);
        rowsum_kernel<<<(M + 7) / 8, 256, 0, st2>>>(static_cast<const __half *>(x_half), M, K, rowsum_scratch);
        return man == 6 ? launch_decode<12>(map_x, packed + v.store_off, sb + 2 * v.sb_slot, rowsum_scratch, y, M, N, K,
                                            plan->d_status, st2)
                        : launch_decode<8>(map_x, packed + v.store_off, sb + 2 * v.sb_slot, rowsum_scratch, y, M, N, K,
                                           plan->d_status, st2);
    }
    if (!make_map(&map_w, packed + v.store_off, N, K)) return OMC_ERR_CUDA;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        int rc = omc::note_cuda(cudaFuncSetAttribute(matmul_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        if (rc) return rc;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rowsum_kernel<<<(M + 7) / 8, 256, 0, st>>>(static_cast<const __half *>(x_half), M, K, rowsum_scratch);
    dim3 grid(N / BN, (M + BM - 1) / BM);
    matmul_kernel<<<grid, 128, SMEM_BYTES, st>>>(map_x, map_w, sb + 2 * v.sb_slot, rowsum_scratch, y, M, N, K,
                                                 plan->d_status);
    return omc::note_cuda(cudaGetLastError());
}
