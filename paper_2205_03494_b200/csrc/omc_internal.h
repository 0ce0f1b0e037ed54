// Internal declarations shared by the host-side plan code and the kernel launchers.
#pragma once
#include <stdint.h>

#include <vector>

#include "../../include/omc.h"

namespace omc {

// Launch shape (overridable at build time for tuning runs).
#ifndef OMC_WARPS_PER_CTA
#define OMC_WARPS_PER_CTA 8
#endif
#ifndef OMC_CTAS_PER_SM
#define OMC_CTAS_PER_SM 2
#endif

constexpr int TILE = 1024;         // elements per tile: the unit of work a warp takes
constexpr int WARPS_PER_CTA = OMC_WARPS_PER_CTA;
constexpr int THREADS = 32 * WARPS_PER_CTA;
constexpr int CTAS_PER_SM = OMC_CTAS_PER_SM;
#ifndef OMC_DECOMPRESS_CTAS_PER_SM
#define OMC_DECOMPRESS_CTAS_PER_SM 2
#endif
// The decompress kernel keeps no running sums and needs fewer registers: it may run more CTAs per SM
// (it divides its tiles at launch, so its grid is independent of the plan's partition).
constexpr int DECOMPRESS_CTAS_PER_SM = OMC_DECOMPRESS_CTAS_PER_SM;
constexpr int DEFAULT_SMS = 148;   // B200; used when no device can be queried at plan time

// One per variable, in the caller's order; lives in device memory after omc_plan_prepare.
struct VarDev {
    uint64_t n;             // elements
    uint64_t full_off;      // element offset in the full FP32 layout
    uint64_t store_off;     // quantised: byte offset in the packed arena; else element offset in resid
    uint64_t packed_bytes;  // quantised: padded byte size of the code stream; else 0
    uint64_t tile_start;    // index of the variable's first tile among all tiles of the plan
    uint32_t ntiles;
    uint32_t quantised;
    uint32_t sb_slot;       // index into sb[] and the ticket array
    uint32_t slot_base;     // first partial-sum slot of this variable in the workspace
    uint32_t first_warp;    // the warp (of the plan-wide partition) that owns the first tile
    uint32_t nslots;        // number of warps that own at least one tile of this variable
};
static_assert(sizeof(VarDev) == 64, "VarDev is laid out for 16-byte loads");

// Per-warp partial sums of the Sec. 2.3 fit, one slot per (variable, warp that touched it).
struct Partial {
    double sx, sy, sxy, syy;   // Sum W, Sum Vt, Sum W*Vt, Sum Vt^2
    uint32_t band, bor;        // AND / OR of the bit patterns of Vt (equal <=> all Vt equal)
    uint32_t pad[2];
};
static_assert(sizeof(Partial) == 48, "");

constexpr uint64_t WS_HEADER_BYTES = 256;

// Arguments of one kernel launch.
struct KParams {
    const VarDev *vars;
    uint32_t var_begin, var_end;   // variables covered by this launch
    uint64_t tile_begin;           // first tile covered
    uint64_t tile_count;           // number of tiles covered
    uint32_t nwarps;               // warps the tiles are divided among (<= tile_count)
    // Optional: nwarps + 1 tile indices, warp w owns tiles [warp_start[w], warp_start[w + 1]).
    // NULL: warp w owns [tile_begin + w * tile_count / nwarps, tile_begin + (w + 1) * tile_count / nwarps).
    const uint64_t *warp_start;
    uint32_t pvt;
    uint32_t dyn_e, dyn_m;         // the format, for the kernels that take it at run time
    uint8_t *packed;
    float *resid;
    float *sb;
    const float *fin;              // compress: params; update: grads (full layout)
    float *fout;                   // decompress: out; update: optional W (full layout)
    float neg_lr;
    Partial *slots;
    uint32_t *tickets;
    // plan-to-plan transition only: the source plan's table and state
    const VarDev *vars_from;
    const uint8_t *packed_from;
    const float *resid_from;
    const float *sb_from;
    uint32_t *status;              // the plan's device status word: set non-zero if a copy never arrived
};

// Arguments of the aggregation kernel: the states of up to MAX_CLIENTS replicas of one model.
constexpr int MAX_CLIENTS = 16;
struct AggParams {
    const VarDev *vars[MAX_CLIENTS];     // each replica's plan table (same variables, own selection)
    const uint8_t *packed[MAX_CLIENTS];
    const float *resid[MAX_CLIENTS];
    const float *sb[MAX_CLIENTS];
    uint32_t nclients;
    uint32_t nvars;
    uint64_t tile_count;
    uint32_t nwarps;
    float *out;                          // full layout
};

struct FmtOps {
    int E, M;
    void (*compress)(const KParams &, int grid, void *stream);
    void (*decompress)(const KParams &, int grid, void *stream);
    void (*update)(const KParams &, int grid, void *stream);     // W not stored
    void (*update_w)(const KParams &, int grid, void *stream);   // W stored to fout
    void (*transition)(const KParams &, int grid, void *stream); // plan-to-plan; NULL if unsupported
    void (*aggregate)(const AggParams &, int grid, void *stream); // mean of replicas; NULL if unsupported
};
const FmtOps *find_ops(int E, int M);

// Divides the tiles of vars[0 .. nvars) (n, quantised, tile_start and ntiles filled in) among
// nwarps warps: writes warp_start[0 .. nwarps] (warp w owns tiles [warp_start[w], warp_start[w+1]))
// and each variable's first_warp, nslots and slot_base; returns the number of partial-sum slots.
uint32_t divide_tiles(VarDev *vars, uint32_t nvars, uint32_t nwarps, uint64_t *warp_start);

// The tiles [t, tend) of warp `warp` under the launch's division of the work.
#ifdef __CUDACC__
__device__ __forceinline__ void warp_tile_range(const KParams &p, uint32_t warp, uint64_t &t, uint64_t &tend)
{
    if (p.warp_start) {
        t = __ldg(p.warp_start + warp);
        tend = __ldg(p.warp_start + warp + 1);
    } else {
        t = p.tile_begin + (uint64_t)warp * p.tile_count / p.nwarps;
        tend = p.tile_begin + (uint64_t)(warp + 1) * p.tile_count / p.nwarps;
    }
}
#endif

}  // namespace omc

struct omc_plan {
    omc_format_t fmt;
    uint32_t flags;
    uint32_t nvars, nq;
    std::vector<omc::VarDev> vars;
    std::vector<uint64_t> resid_off;   // per variable (valid iff !quantised)
    uint64_t full_elems, resid_elems, packed_bytes, closed_form_bytes;
    uint64_t ntiles;                   // all tiles
    uint32_t n_sm, n_cta, nwarps;      // launch geometry the partition was made for
    uint32_t nslots;
    uint64_t ws_tickets_off, ws_slots_off, ws_bytes;
    const omc::FmtOps *ops;
    // device side
    std::vector<uint64_t> warp_start;  // nwarps + 1 entries: the cost-balanced division of the tiles
    omc::VarDev *d_vars;               // one allocation: the variable table, the status word, warp_start
    uint32_t *d_status;
    uint64_t *d_warp_start;
    int device;                        // device the tables live on, -1 before prepare
};
