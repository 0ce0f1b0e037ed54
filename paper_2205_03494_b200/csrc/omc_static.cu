// omc_compress_var_static: compression of one variable for callers that may not allocate.
//
// Everything omc_compress keeps in caller- or plan-owned device memory besides the inputs and
// outputs (the one-entry variable table, the ticket, the status word, the division of the tiles
// among warps and the per-warp partial-sum records of the fit) lives here in a fixed array inside
// the library's own device image.
#include <cuda_runtime.h>

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
unsigned char *g_scratch_addr[MAX_DEVICES] = {};         // device address of the array, per device
int g_sm_count[MAX_DEVICES] = {};

// First use on the current device: look up where the array lives there.
int scratch_for_current_device(unsigned char **out, int *sms)
{
    int dev = 0;
    int rc = omc::note_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    if (dev < 0 || dev >= MAX_DEVICES) return OMC_ERR_INVALID_ARG;
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        rc = omc::note_cuda(cudaGetSymbolAddress(&p, g_static_scratch));
        if (rc) return rc;
        int n = 0;
        rc = omc::note_cuda(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        if (rc) return rc;
        g_sm_count[dev] = n;
        g_scratch_addr[dev] = static_cast<unsigned char *>(p);
    }
    *out = g_scratch_addr[dev];
    *sms = g_sm_count[dev];
    return OMC_OK;
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
    if (fmt.sign_bits != 1 || fmt.exp_bits < 2 || fmt.exp_bits > 8 || fmt.man_bits > 23 || fmt.flags != 0)
        return OMC_ERR_BAD_FORMAT;
    const omc::FmtOps *ops = omc::find_ops(fmt.exp_bits, fmt.man_bits);
    if (!ops) return OMC_ERR_BAD_FORMAT;

    unsigned char *scratch = nullptr;
    int sms = 0;
    int rc = scratch_for_current_device(&scratch, &sms);
    if (rc) return rc;

    // one variable, one tile list, divided among the warps exactly as omc_plan divides a model
    const uint32_t B = 1u + fmt.exp_bits + fmt.man_bits;
    const uint64_t tiles = (numel + omc::TILE - 1) / omc::TILE;
    const uint64_t max_warps = (uint64_t)sms * omc::CTAS_PER_SM * omc::WARPS_PER_CTA;
    const uint32_t nwarps = (uint32_t)(tiles < max_warps ? tiles : max_warps);
    if (nwarps > MAX_SLOTS) return OMC_ERR_TOO_LARGE;
    const uint32_t nruns = nwarps;          // one run per warp, as in omc_compress

    omc::VarDev v{};
    v.n = numel;
    v.full_off = 0;
    v.store_off = 0;
    v.packed_bytes = ((numel * B + 7) / 8 + 15) / 16 * 16;
    v.tile_start = 0;
    v.ntiles = (uint32_t)tiles;
    v.quantised = 1;
    v.sb_slot = 0;
    v.slot_base = 0;
    uint64_t run_start[MAX_SLOTS + 1];         // host copy; the same division omc_plan makes
    uint32_t run_var[MAX_SLOTS];               // all zero: there is one variable
    omc::divide_tiles(&v, 1, nruns, run_start, run_var);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps what the last call left: the table entry and the division are rewritten, the
    // ticket and the status word are cleared; the records are all rewritten by the kernel before
    // they are read.  Both host buffers are pageable, so each copy has left them when it returns.
    rc = omc::note_cuda(cudaMemcpyAsync(scratch + OFF_VAR, &v, sizeof v, cudaMemcpyHostToDevice, st));
    if (rc) return rc;
    rc = omc::note_cuda(cudaMemcpyAsync(scratch + OFF_RUN_START, run_start, sizeof(uint64_t) * (nruns + 1),
                                        cudaMemcpyHostToDevice, st));
    if (rc) return rc;
    rc = omc::note_cuda(cudaMemcpyAsync(scratch + OFF_RUN_VAR, run_var, sizeof(uint32_t) * nruns,
                                        cudaMemcpyHostToDevice, st));
    if (rc) return rc;
    rc = omc::note_cuda(cudaMemsetAsync(scratch + OFF_TICKET, 0, 8, st));
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
    p.packed = packed;
    p.resid = nullptr;
    p.sb = sb;
    p.fin = values;
    p.tickets = reinterpret_cast<uint32_t *>(scratch + OFF_TICKET);
    p.status = reinterpret_cast<uint32_t *>(scratch + OFF_STATUS);
    p.slots = reinterpret_cast<omc::Partial *>(scratch + OFF_SLOTS);
    ops->compress(p, (int)((nwarps + omc::WARPS_PER_CTA - 1) / omc::WARPS_PER_CTA), stream);
    return omc::note_cuda(cudaGetLastError());
}
