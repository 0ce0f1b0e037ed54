// Internal declarations shared by the host-side plan code and the kernel launchers.
#pragma once
#include <stdint.h>

#include <vector>

#include "../../include/omc.h"

namespace omc {

// Launch shape (measured best on B200 among 4 / 8 / 16 warps and 1 to 4 CTAs per SM).
constexpr int TILE = 1024;         // elements per tile: the unit of work a warp takes
constexpr int WARPS_PER_CTA = 8;
constexpr int THREADS = 32 * WARPS_PER_CTA;
// Warps per CTA of the kernels that fit (s, b) (compress, fused round, transition).  Eight warps
// leave a thread 128 registers; the 12- and 19-bit kernels, which need more to keep several
// elements' arithmetic in flight, run faster with six warps and up to 168 registers (measured:
// S1E5M6 on the 1.6-billion set 3-5 % per clock, S1E4M14 5 %, Q11 4 %; the 16- and 8-bit kernels lose 2-3 %,
// the 11- and 13-bit ones gain a per cent and a half, which their compress kernel would lose again).
constexpr int fit_warps_per_cta(int code_bits, bool /*fixed_point*/)
{
    return (code_bits == 12 || code_bits == 19) ? 6 : WARPS_PER_CTA;
}
constexpr int CTAS_PER_SM = 2;
// CTAs per SM of the aggregation: with 8-bit codes it gets by on the 80 registers that three leave it
// (nine words spilled, outside the tile loop; measured 11-14 % faster than two); with any other
// width it spills inside the loop (up to 29 % slower).
constexpr int aggregate_ctas_per_sm(int code_bits) { return code_bits == 8 ? 3 : CTAS_PER_SM; }
// The decompress kernel divides its tiles at launch, so its grid is independent of the plan's division.
constexpr int DECOMPRESS_CTAS_PER_SM = 2;
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
    uint32_t first_run;     // the run (of the plan-wide division) that holds the first tile
    uint32_t nslots;        // number of runs that hold at least one tile of this variable
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

// Estimated cost of a warp's work in the division of the tiles, in sixteenths of the time of one
// tile of codes (measured on B200 with the fused round): a tile of codes, a tile of FP32 values,
// and what entering a quantised variable costs on top (pipeline restart, ragged end, hand-over of
// the fit's sums).
constexpr uint64_t COST_TILE = 16, COST_FP32_TILE = 16, COST_VARIABLE = 48;

struct TransitionVar;

// Arguments of one kernel launch.
struct KParams {
    const VarDev *vars;
    uint32_t var_begin, var_end;   // variables covered by this launch
    uint64_t tile_begin;           // first tile covered
    uint64_t tile_count;           // number of tiles covered
    uint32_t nwarps;               // warps launched (<= tile_count)
    // The tiles are divided into nruns contiguous runs; warp w takes runs w, w + nwarps, ... so that
    // the warps running at the same time work on neighbouring memory.
    // run_start: nruns + 1 tile indices, run r = tiles [run_start[r], run_start[r + 1]); if NULL, run r =
    // tiles [tile_begin + r * tile_count / nruns, tile_begin + (r + 1) * tile_count / nruns).
    // run_var[r] = the variable that holds the run's first tile; if NULL, the kernel searches for it.
    uint32_t nruns;
    const uint64_t *run_start;
    const uint32_t *run_var;
    uint32_t pvt;
    uint32_t dyn_e, dyn_m;         // the format, for the kernels that take it at run time
    uint32_t dyn_fixed;            // ... and whether it is the fixed-point variant (then integer / fraction bits)
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
    // FP32 variables in omc_update_recompress (where they are a real share of the work): their tiles
    // are not processed with the runs but as one list that the warps take chunks from as they finish
    // their runs (a counter in the workspace header).  fp32_tile_start: n_fp32 + 1 entries, the tiles before each FP32 variable
    // among the FP32 variables' tiles; fp32_var: the variables' indices.  NULL: none.
    const uint64_t *fp32_tile_start;
    const uint32_t *fp32_var;
    uint32_t n_fp32;
    uint32_t *queue;                   // [0] next chunk, [1] warps that are through
    const TransitionVar *trans_vars;   // the launch's own record numbering
    const uint32_t *nruns_dev;         // the launch's run count (replaces nruns)
    uint32_t *status;              // the plan's device status word: set non-zero if a copy never arrived
    // Diagnostics (omc_plan_inject_wait_timeout): polls of one mbarrier before a warp gives up (0 = the
    // default), and whether the warps announce their bulk loads to the mbarrier without issuing them,
    // so that the waits run out with nothing in flight.
    uint32_t wait_limit;
    uint32_t skip_loads;
    // Host side: launch as the programmatic dependent of the kernel before it on the stream.  On for
    // the fused round and compress (measured on the 100M set: 1.5-2.6 % per round in a row of rounds,
    // nothing lost on the larger sets) and for omc_decompress of a part of the model (17 block-wise
    // calls 12.3 -> 10.7 us each); off for whole-model decompress calls in a row, which lose with
    // 8-bit codes (0.0845 -> 0.0926 ms: the CTAs of a dependent launch take their SMs in the order
    // in which the kernel before it leaves them).
    uint32_t dependent;
};

// omc_transition's own division of the work, made on the device before each launch.
struct TransitionVar {          // for a variable that gets a fresh fit: its partial-sum records
    uint32_t first_run, nslots, slot_base, pad;
};
struct TransitionTables {       // device memory owned by the destination plan
    uint64_t *before;           // nvars: estimated cost of all variables before this one
    uint64_t *last;             // nvars: estimated cost of everything before this variable's last tile
    TransitionVar *vars;        // nvars
    uint64_t *run_start;        // max_runs + 1
    uint32_t *run_var;          // max_runs
    uint32_t *nruns;            // 1: how many runs this launch has
};
struct TransitionCosts {        // per tile, in sixteenths of a tile that is quantised and fitted
    uint32_t copy_codes, copy_fp32, convert, fit_entry, max_tile;
};
void launch_transition_division(const VarDev *to, const VarDev *from, uint32_t nvars, uint64_t ntiles,
                                uint32_t max_runs, const TransitionCosts &c, const TransitionTables &out,
                                void *stream);

// Arguments of the aggregation kernel: the states of up to MAX_CLIENTS replicas of one model.
constexpr int MAX_CLIENTS = 16;
struct AggParams {
    const VarDev *vars[MAX_CLIENTS];     // each replica's plan table (same variables, own selection)
    const uint8_t *packed[MAX_CLIENTS];
    const float *resid[MAX_CLIENTS];
    const float *sb[MAX_CLIENTS];
    uint32_t nclients;
    uint32_t divide;                     // 1: out = sum / nclients; 0: out = the sum itself (first stage of a mean across GPUs)
    uint32_t accumulate;                 // 1: the sum starts from what `out` holds (clients beyond the first MAX_CLIENTS)
    uint32_t nvars;
    uint64_t tile_count;
    uint32_t nwarps;
    uint32_t nruns;                      // equal runs of tiles, run r to warp r mod nwarps
    float *out;                          // full layout
    uint32_t *status;                    // set to 1 by a warp whose wait for a bulk copy ran out
    uint32_t wait_limit;                 // polls of one mbarrier before giving up; 0: the default
    uint32_t skip_loads;                 // diagnostics: announce the bulk loads, do not issue them
};

struct FmtOps {
    int E, M;          // fixed != 0: integer bits and fraction bits of S1IxFy
    int fixed;
    int fit_warps;     // warps per CTA of compress / update / transition (the decoder and the aggregation use WARPS_PER_CTA)
    int agg_ctas;      // CTAs per SM of the aggregation
    void (*compress)(const KParams &, int grid, void *stream);
    void (*decompress)(const KParams &, int grid, void *stream);
    void (*update)(const KParams &, int grid, void *stream);     // W not stored
    void (*update_w)(const KParams &, int grid, void *stream);   // W stored to fout
    void (*update_q)(const KParams &, int grid, void *stream);   // FP32 variables' tiles from the queue; NULL if unsupported
    void (*transition)(const KParams &, int grid, void *stream); // plan-to-plan; NULL if unsupported
    void (*aggregate)(const AggParams &, int grid, void *stream); // mean of replicas; NULL if unsupported
};
const FmtOps *find_ops(int E, int M, int fixed);
// Limits of the fixed-point variant S1IxFy (every value k * 2^-y must be an FP32 value).
inline bool fixed_format_ok(int I, int F) { return I >= 0 && I <= 8 && F >= 0 && I + F >= 1 && I + F <= 23; }

// Divides the tiles of vars[0 .. nvars) (n, quantised, tile_start and ntiles filled in) into nruns
// contiguous runs of about equal estimated cost: writes run_start[0 .. nruns], run_var[0 .. nruns)
// and each variable's first_run, nslots and slot_base; returns the number of partial-sum slots.
uint32_t divide_tiles(VarDev *vars, uint32_t nvars, uint32_t nruns, uint64_t *run_start, uint32_t *run_var);
// How many runs of about tiles_per_run tiles a launch of nwarps warps over `tiles` tiles is cut
// into: a multiple of nwarps, at most max_runs (but at least nwarps).
uint32_t runs_for(uint64_t tiles, uint32_t nwarps, uint32_t tiles_per_run, uint32_t max_runs);
// The decoder's runs, in tiles (measured on B200 with 8-, 12- and 16-bit codes: best at about four
// pipeline granules per run; one-tile runs are slower than none at all).
constexpr uint32_t decode_tiles_per_run(uint32_t code_bits) { return code_bits >= 16 ? 4u : 2u; }
constexpr uint32_t DECODE_MAX_RUNS = 1u << 22;
// The aggregation's runs, in tiles: about 64 (tile, client) pairs each.
constexpr uint32_t aggregate_tiles_per_run(uint32_t nclients)
{
    return nclients >= 16 ? 4u : nclients <= 2 ? 32u : 64u / nclients;
}

#ifdef __CUDACC__
// The tiles [t, tend) of run `run`.
__device__ __forceinline__ void run_tile_range(const KParams &p, uint32_t run, uint64_t &t, uint64_t &tend)
{
    if (p.run_start) {
        t = __ldg(p.run_start + run);
        tend = __ldg(p.run_start + run + 1);
    } else {
        // tile_count < 2^40 and nruns <= 2^22: the products fit 64 bits
        t = p.tile_begin + (uint64_t)run * p.tile_count / p.nruns;
        tend = p.tile_begin + (uint64_t)(run + 1) * p.tile_count / p.nruns;
    }
}
// The variable that holds tile t, the first tile of run `run`.
__device__ __forceinline__ uint32_t run_first_var(const KParams &p, uint32_t run, uint64_t t)
{
    if (p.run_var) return __ldg(p.run_var + run);
    uint32_t lo = p.var_begin, hi = p.var_end;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (__ldg(&p.vars[mid].tile_start) <= t) lo = mid; else hi = mid;
    }
    return lo;
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
    uint32_t n_sm, n_cta, nwarps;      // launch geometry the division was made for
    uint32_t nruns;
    uint32_t dec_nwarps, dec_nruns;    // the decoder's launch: equal runs, dealt out in turn
    uint32_t dec_tiles_per_run;
    uint32_t nslots;
    uint64_t ws_tickets_off, ws_slots_off, ws_bytes;
    const omc::FmtOps *ops;
    // device side
    std::vector<uint64_t> run_start;   // nruns + 1 entries: the cost-balanced division of the tiles
    std::vector<uint32_t> run_var;     // nruns entries: the variable each run starts in
    std::vector<uint32_t> dec_run_var; // dec_nruns entries: the same for the decoder's runs
    std::vector<uint64_t> fp32_tile_start;   // n_fp32 + 1: tiles before each FP32 variable among the FP32 tiles
    std::vector<uint32_t> fp32_var;          // n_fp32: their indices
    omc::VarDev *d_vars;               // one allocation: the variable table, the status word, the two run tables
    uint32_t *d_status;
    uint64_t *d_run_start;
    uint32_t *d_run_var;
    uint32_t *d_dec_run_var;
    uint64_t *d_fp32_tile_start;
    uint32_t *d_fp32_var;
    omc::TransitionTables d_trans;     // omc_transition's tables (this plan as the destination)
    mutable uint32_t inject_polls;     // omc_plan_inject_wait_timeout: applies to the next launch, then 0
    int device;                        // device the tables live on, -1 before prepare
};
