// omc_compress_var_static: compression of one variable for callers that may not allocate.
//
// Everything omc_compress keeps in caller- or plan-owned device memory besides the inputs and
// outputs (the one-entry variable table, the ticket, the status word, the division of the tiles
// among warps and the per-warp partial-sum records of the fit) lives here in a fixed array inside
// the library's own device image.
#include <cuda_runtime.h>

#include <mutex>

#include "omc_internal.h"

namespace omc {
int note_cuda(cudaError_t e);
}

namespace {

constexpr uint32_t MAX_SLOTS = 4096;                     // runs, each of which leaves one record
constexpr size_t OFF_VAR = 0;                            // omc::VarDev, 64 bytes
constexpr size_t OFF_TICKET = 64;                        // uint32_t
constexpr size_t OFF_STATUS = 68;                        // uint32_t
constexpr size_t OFF_SLOTS = 256;                        // omc::Partial[MAX_SLOTS]
constexpr size_t OFF_RUN_START = OFF_SLOTS + sizeof(omc::Partial) * MAX_SLOTS;   // uint64_t[MAX_SLOTS + 1]
constexpr size_t OFF_RUN_VAR = OFF_RUN_START + sizeof(uint64_t) * (MAX_SLOTS + 1);    // uint32_t[MAX_SLOTS], all zero
constexpr size_t SCRATCH_BYTES = OFF_RUN_VAR + sizeof(uint32_t) * MAX_SLOTS;   // 246,024 bytes

// Held by every GPU that loads the library until the process exits.  In host code this name is
// only a handle for cudaGetSymbolAddress; it is never passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
struct DeviceScratch {
    std::once_flag once;
    int rc = OMC_OK;
    unsigned char *addr = nullptr;      // device address of the array on this device
    int sms = 0;
};
DeviceScratch g_dev[MAX_DEVICES];

// First use on the current device: look up where the array lives there (once per device, also
// when several host threads make their first call at the same time).
int scratch_for_current_device(unsigned char **out, int *sms)
{
    int dev = 0;
    int rc = omc::note_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    if (dev < 0 || dev >= MAX_DEVICES) return OMC_ERR_INVALID_ARG;
    DeviceScratch &d = g_dev[dev];
    std::call_once(d.once, [&d, dev]() {
        void *p = nullptr;
        d.rc = omc::note_cuda(cudaGetSymbolAddress(&p, g_static_scratch));
        if (d.rc) return;
        int n = 0;
        d.rc = omc::note_cuda(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        if (d.rc) return;
        d.sms = n;
        d.addr = static_cast<unsigned char *>(p);
    });
    if (d.rc) return d.rc;
    *out = d.addr;
    *sms = d.sms;
    return OMC_OK;
}

// What the call needs in the array before the compression kernel starts, written on the device
// (the host hands over nothing that lives in its own memory, only kernel arguments): the
// one-entry variable table, the cleared ticket and status word, and the division of the tiles into
// runs -- the rule of omc_plan's division for a single quantised variable, solved per run: a tile
// costs T, entering the variable V, and tile k belongs to run floor((V + T k) * nruns / total),
// so run r starts at the first tile k with V + T k >= ceil(r * total / nruns).
// numel <= 2^28 and nruns <= 4096 keep every product below 2^36.
__global__ void static_setup_kernel(unsigned char *scratch, uint64_t numel, uint64_t packed_bytes, uint32_t ntiles,
                                    uint32_t nruns)
{
    constexpr uint64_t TILE_COST = omc::COST_TILE, VAR_COST = omc::COST_VARIABLE;
    const uint64_t total = TILE_COST * ntiles + VAR_COST;
    auto run_of = [&](uint64_t cost) { return (uint32_t)(cost * nruns / total); };
    uint64_t *run_start = reinterpret_cast<uint64_t *>(scratch + OFF_RUN_START);
    uint32_t *run_var = reinterpret_cast<uint32_t *>(scratch + OFF_RUN_VAR);
    for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r <= nruns; r += gridDim.x * blockDim.x) {
        uint64_t k;
        if (r == nruns) {
            k = ntiles;
        } else {
            const uint64_t need = ((uint64_t)r * total + nruns - 1) / nruns;
            k = need <= VAR_COST ? 0 : (need - VAR_COST + TILE_COST - 1) / TILE_COST;
            if (k > ntiles) k = ntiles;
            run_var[r] = 0u;
        }
        run_start[r] = k;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        omc::VarDev v;
        v.n = numel;
        v.full_off = 0;
        v.store_off = 0;
        v.packed_bytes = packed_bytes;
        v.tile_start = 0;
        v.ntiles = ntiles;
        v.quantised = 1;
        v.sb_slot = 0;
        v.slot_base = 0;
        v.first_run = run_of(VAR_COST);
        v.nslots = run_of(VAR_COST + TILE_COST * (ntiles - 1)) - v.first_run + 1;
        *reinterpret_cast<omc::VarDev *>(scratch + OFF_VAR) = v;
        *reinterpret_cast<uint32_t *>(scratch + OFF_TICKET) = 0u;
        *reinterpret_cast<uint32_t *>(scratch + OFF_STATUS) = 0u;
    }
}

}  // namespace

extern "C" int omc_compress_var_static(const float *values, uint64_t numel, omc_format_t fmt, uint32_t flags,
                                       uint8_t *packed, float *sb, void *stream)
{
    if (!values || !packed || !sb) return OMC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(values) | reinterpret_cast<uintptr_t>(packed)) & 15u) return OMC_ERR_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(sb) & 7u) return OMC_ERR_MISALIGNED;
    if (flags & ~(uint32_t)OMC_PLAN_PVT) return OMC_ERR_INVALID_ARG;
    if (numel == 0) return OMC_ERR_INVALID_ARG;
    if (numel > OMC_STATIC_MAX_NUMEL) return OMC_ERR_TOO_LARGE;
    if (fmt.sign_bits != 1 || (fmt.flags & ~OMC_FORMAT_FIXED_POINT)) return OMC_ERR_BAD_FORMAT;
    const int fixed = (fmt.flags & OMC_FORMAT_FIXED_POINT) ? 1 : 0;
    if (fixed ? !omc::fixed_format_ok(fmt.exp_bits, fmt.man_bits)
              : (fmt.exp_bits < 2 || fmt.exp_bits > 8 || fmt.man_bits > 23))
        return OMC_ERR_BAD_FORMAT;
    const omc::FmtOps *ops = omc::find_ops(fmt.exp_bits, fmt.man_bits, fixed);
    if (!ops) return OMC_ERR_BAD_FORMAT;

    unsigned char *scratch = nullptr;
    int sms = 0;
    int rc = scratch_for_current_device(&scratch, &sms);
    if (rc) return rc;

    // one variable, one tile list, divided among the warps exactly as omc_plan divides a model
    const uint32_t B = 1u + fmt.exp_bits + fmt.man_bits;
    const uint64_t tiles = (numel + omc::TILE - 1) / omc::TILE;
    const uint64_t max_warps = (uint64_t)sms * omc::CTAS_PER_SM * ops->fit_warps;
    const uint32_t nwarps = (uint32_t)(tiles < max_warps ? tiles : max_warps);
    if (nwarps > MAX_SLOTS) return OMC_ERR_TOO_LARGE;
    const uint32_t nruns = nwarps;          // one run per warp, as in omc_compress
    const uint64_t packed_bytes = ((numel * B + 7) / 8 + 15) / 16 * 16;

    // The array keeps what the last call left.  A small kernel on `stream` rewrites the table entry
    // and the division and clears the ticket and the status word; the records are all rewritten by
    // the compression kernel before they are read.  Nothing is copied from host memory, so the call
    // leaves no pointer to the caller's stack or heap behind on the stream.
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    static_setup_kernel<<<(nruns + 1 + 255) / 256, 256, 0, st>>>(scratch, numel, packed_bytes, (uint32_t)tiles, nruns);
    rc = omc::note_cuda(cudaGetLastError());
    if (rc) return rc;

    omc::KParams p{};
    p.vars = reinterpret_cast<const omc::VarDev *>(scratch + OFF_VAR);
    p.var_begin = 0;
    p.var_end = 1;
    p.tile_begin = 0;
    p.tile_count = tiles;
    p.nwarps = nwarps;
    p.nruns = nruns;
    p.run_start = reinterpret_cast<const uint64_t *>(scratch + OFF_RUN_START);
    p.run_var = reinterpret_cast<const uint32_t *>(scratch + OFF_RUN_VAR);
    p.pvt = (flags & OMC_PLAN_PVT) ? 1u : 0u;
    p.dyn_e = fmt.exp_bits;
    p.dyn_m = fmt.man_bits;
    p.dyn_fixed = (uint32_t)fixed;
    p.packed = packed;
    p.resid = nullptr;
    p.sb = sb;
    p.fin = values;
    p.tickets = reinterpret_cast<uint32_t *>(scratch + OFF_TICKET);
    p.status = reinterpret_cast<uint32_t *>(scratch + OFF_STATUS);
    p.slots = reinterpret_cast<omc::Partial *>(scratch + OFF_SLOTS);
    ops->compress(p, (int)((nwarps + ops->fit_warps - 1) / ops->fit_warps), stream);
    return omc::note_cuda(cudaGetLastError());
}

extern "C" int omc_static_status(void *stream, uint32_t *host_status)
{
    if (!host_status) return OMC_ERR_NULL_PTR;
    unsigned char *scratch = nullptr;
    int sms = 0;
    int rc = scratch_for_current_device(&scratch, &sms);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = omc::note_cuda(cudaMemcpyAsync(host_status, scratch + OFF_STATUS, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    if (rc) return rc;
    return omc::note_cuda(cudaStreamSynchronize(st));
}
