// Host side of libomc: the plan (which variables are compressed, where everything lives, how the
// tiles are divided among warps) and the C-ABI entry points that need no kernel.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "omc_internal.h"

using omc::VarDev;

static thread_local int g_last_cuda_error = 0;

namespace omc {
int note_cuda(cudaError_t e)
{
    if (e == cudaSuccess) return OMC_OK;
    g_last_cuda_error = (int)e;
    (void)cudaGetLastError();
    return OMC_ERR_CUDA;
}
}  // namespace omc

extern "C" const char *omc_strerror(int status)
{
    switch (status) {
        case OMC_OK: return "ok";
        case OMC_ERR_INVALID_ARG: return "invalid argument";
        case OMC_ERR_BAD_FORMAT: return "format outside S1EyMz with 2<=y<=8, 0<=z<=23";
        case OMC_ERR_NULL_PTR: return "required pointer is NULL";
        case OMC_ERR_MISALIGNED: return "device pointer is not 16-byte aligned";
        case OMC_ERR_PLAN_MISMATCH: return "plan not prepared, or not usable for this call";
        case OMC_ERR_CUDA: return "CUDA runtime error (see omc_last_cuda_error)";
        case OMC_ERR_NO_MEMORY: return "out of host memory";
        case OMC_ERR_TOO_LARGE: return "size beyond the fixed capacity of the allocation-free entry point";
        default: return "unknown status";
    }
}

extern "C" int omc_last_cuda_error(void) { return g_last_cuda_error; }

// SplitMix64 (Steele, Lea, Flood 2014): the generator that drives the subset draw.
static uint64_t splitmix64(uint64_t &state)
{
    uint64_t z = (state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// The k-th output (k = round * 2^32 + client) of the stream seeded with base_seed: SplitMix64
// keeps a counter as its state, so the stream can be entered anywhere.
extern "C" uint64_t omc_plan_seed(uint64_t base_seed, uint32_t round, uint32_t client)
{
    uint64_t state = base_seed + ((((uint64_t)round << 32) | client) * 0x9E3779B97F4A7C15ull);
    return splitmix64(state);
}

static uint64_t round_up(uint64_t x, uint64_t m) { return (x + m - 1) / m * m; }

static uint32_t query_sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
        (void)cudaGetLastError();
        return omc::DEFAULT_SMS;
    }
    return (uint32_t)sms;
}

// Division of the tiles into contiguous runs of equal estimated cost.  A run pays for a tile and,
// on top, for every quantised variable it enters (pipeline restart, ragged end, hand-over of the
// fit's sums).  A tile goes to run floor(cost before it * nruns / total cost): monotone in the tile
// index, and inside a variable consecutive tiles' runs differ by at most one, so the runs
// first_run .. first_run + nslots - 1 of a variable all hold one of its tiles.
uint32_t omc::divide_tiles(VarDev *vars, uint32_t nvars, uint32_t nruns, uint64_t *run_start, uint32_t *run_var)
{
    const uint64_t NR = nruns;
    auto var_cost = [](const VarDev &v) {
        return v.quantised ? omc::COST_TILE * v.ntiles + omc::COST_VARIABLE
                           : omc::COST_FP32_TILE * v.ntiles;
    };
    uint64_t total_cost = 0, tiles = 0;
    for (uint32_t i = 0; i < nvars; ++i) {
        total_cost += var_cost(vars[i]);
        tiles += vars[i].ntiles;
    }
    // 128-bit products: the cost of 2^40-element variables times the run count overflows 64 bits
    auto run_of = [&](uint64_t cost) { return (uint32_t)(((unsigned __int128)cost * NR) / total_cost); };
    run_start[0] = 0;
    run_var[0] = 0;
    uint32_t slots = 0, r = 0;
    uint64_t before = 0;
    for (uint32_t i = 0; i < nvars; ++i) {
        VarDev &v = vars[i];
        const uint64_t per_tile = v.quantised ? omc::COST_TILE : omc::COST_FP32_TILE;
        const uint64_t c = before + (v.quantised ? omc::COST_VARIABLE : 0);     // cost before tile 0 of v
        v.first_run = run_of(c);
        // the tiles of v at which the run changes, solved for instead of walking every tile
        uint64_t k = 0;
        while (k < v.ntiles) {
            const uint32_t own = run_of(c + per_tile * k);
            while (r < own) {
                run_start[++r] = v.tile_start + k;
                run_var[r] = i;
            }
            // smallest cost that belongs to the next run, and the first tile of v that reaches it
            const unsigned __int128 need = ((unsigned __int128)(own + 1) * total_cost + NR - 1) / NR;
            uint64_t k2 = (uint64_t)((need - c + per_tile - 1) / per_tile);
            if (k2 <= k) k2 = k + 1;
            k = k2 < v.ntiles ? k2 : v.ntiles;
        }
        v.nslots = run_of(c + per_tile * (v.ntiles - 1)) - v.first_run + 1;
        if (v.quantised) {
            v.slot_base = slots;
            slots += v.nslots;
        }
        before += var_cost(v);
    }
    while (r < NR) {
        run_start[++r] = tiles;
        if (r < NR) run_var[r] = nvars - 1;      // an empty run at the end
    }
    return slots;
}

// Runs of about tiles_per_run tiles, a whole number of them per warp (at least one, at most max_runs
// in all).
uint32_t omc::runs_for(uint64_t tiles, uint32_t nwarps, uint32_t tiles_per_run, uint32_t max_runs)
{
    const uint64_t per_round = (uint64_t)nwarps * tiles_per_run;
    uint64_t rounds = (tiles + per_round - 1) / per_round;
    if (rounds * nwarps > max_runs) rounds = max_runs / nwarps;
    if (rounds < 1) rounds = 1;
    return (uint32_t)(rounds * nwarps);
}

extern "C" int omc_plan(const omc_var_desc_t *vars, uint32_t nvars, omc_format_t fmt, double fraction,
                        uint64_t seed, const uint8_t *mask, uint32_t flags, omc_plan_t **out)
{
    if (!vars || !out) return OMC_ERR_NULL_PTR;
    *out = nullptr;
    if (nvars == 0) return OMC_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)OMC_PLAN_DEFAULT) return OMC_ERR_INVALID_ARG;
    if (fmt.sign_bits != 1 || (fmt.flags & ~OMC_FORMAT_FIXED_POINT)) return OMC_ERR_BAD_FORMAT;
    const int fixed = (fmt.flags & OMC_FORMAT_FIXED_POINT) ? 1 : 0;
    if (fixed ? !omc::fixed_format_ok(fmt.exp_bits, fmt.man_bits)
              : (fmt.exp_bits < 2 || fmt.exp_bits > 8 || fmt.man_bits > 23))
        return OMC_ERR_BAD_FORMAT;
    const omc::FmtOps *ops = omc::find_ops(fmt.exp_bits, fmt.man_bits, fixed);
    if (!ops) return OMC_ERR_BAD_FORMAT;
    if (!mask && !(fraction > 0.0 && fraction <= 1.0)) return OMC_ERR_INVALID_ARG;
    for (uint32_t i = 0; i < nvars; ++i)
        if (vars[i].numel == 0 || vars[i].kind > OMC_KIND_OTHER || vars[i].reserved != 0 ||
            vars[i].numel > (1ull << 40))
            return OMC_ERR_INVALID_ARG;

    omc_plan_t *pl = new (std::nothrow) omc_plan_t();
    if (!pl) return OMC_ERR_NO_MEMORY;
    try {
        pl->fmt = fmt;
        pl->flags = flags;
        pl->nvars = nvars;
        pl->ops = ops;
        pl->d_vars = nullptr;
        pl->d_status = nullptr;
        pl->inject_polls = 0;
        pl->d_run_start = nullptr;
        pl->d_run_var = nullptr;
        pl->d_dec_run_var = nullptr;
        pl->d_fp32_tile_start = nullptr;
        pl->d_fp32_var = nullptr;
        pl->d_trans = omc::TransitionTables{};
        pl->device = -1;
        const uint32_t B = 1u + fmt.exp_bits + fmt.man_bits;

        // ---- selection (Sec. 2.4, 2.5, 3.1)
        std::vector<uint8_t> sel(nvars, 0);
        std::vector<uint32_t> eligible;
        for (uint32_t i = 0; i < nvars; ++i)
            if (!(flags & OMC_PLAN_WEIGHTS_ONLY) || vars[i].kind == OMC_KIND_WEIGHT_MATRIX)
                eligible.push_back(i);
        if (mask) {
            for (uint32_t i = 0; i < nvars; ++i) sel[i] = mask[i] ? 1 : 0;
            std::vector<uint8_t> ok(nvars, 0);
            for (uint32_t i : eligible) ok[i] = 1;
            for (uint32_t i = 0; i < nvars; ++i)
                if (sel[i] && !ok[i]) { delete pl; return OMC_ERR_INVALID_ARG; }
        } else {
            const uint32_t W = (uint32_t)eligible.size();
            uint64_t st = seed;
            for (uint32_t i = W; i-- > 1;) {
                const uint32_t j = (uint32_t)(splitmix64(st) % (uint64_t)(i + 1));
                std::swap(eligible[i], eligible[j]);
            }
            uint32_t k = (uint32_t)std::floor(fraction * (double)W + 0.5);
            if (k > W) k = W;
            for (uint32_t i = 0; i < k; ++i) sel[eligible[i]] = 1;
        }

        // ---- layouts
        pl->vars.resize(nvars);
        pl->resid_off.assign(nvars, 0);
        uint64_t full = 0, resid = 0, packed = 0, tiles = 0, closed = 0;
        uint32_t nq = 0;
        for (uint32_t i = 0; i < nvars; ++i) {
            VarDev &v = pl->vars[i];
            std::memset(&v, 0, sizeof v);
            v.n = vars[i].numel;
            v.full_off = full;
            full += round_up(v.n, 4);
            v.quantised = sel[i];
            if (sel[i]) {
                v.store_off = packed;
                v.packed_bytes = round_up((v.n * B + 7) / 8, 16);
                packed += v.packed_bytes;
                v.sb_slot = nq++;
                closed += (v.n * B + 7) / 8 + 8;
            } else {
                v.store_off = resid;
                pl->resid_off[i] = resid;
                resid += round_up(v.n, 4);
                closed += 4 * v.n;
            }
            v.tile_start = tiles;
            v.ntiles = (uint32_t)((v.n + omc::TILE - 1) / omc::TILE);
            tiles += v.ntiles;
        }
        pl->nq = nq;
        pl->full_elems = full;
        pl->resid_elems = resid;
        pl->packed_bytes = packed;
        pl->closed_form_bytes = closed;
        pl->ntiles = tiles;

        // ---- division of the tiles among warps
        pl->n_sm = query_sm_count();
        pl->n_cta = pl->n_sm * omc::CTAS_PER_SM;
        const uint64_t max_warps = (uint64_t)pl->n_cta * ops->fit_warps;      // the fitting kernels' launch
        pl->nwarps = (uint32_t)(tiles < max_warps ? tiles : max_warps);
        // Kernels that fit (s, b) take one run per warp: a run ends with a hand-over of the sums,
        // which costs more than working side by side with the other warps gains.
        pl->nruns = pl->nwarps;
        pl->run_start.assign((size_t)pl->nruns + 1, 0);
        pl->run_var.assign((size_t)pl->nruns, 0);
        const uint32_t slots = omc::divide_tiles(pl->vars.data(), nvars, pl->nruns, pl->run_start.data(),
                                                 pl->run_var.data());
        pl->nslots = slots;

        // ---- the FP32 variables' tiles as one list (taken in chunks by whichever warp is free)
        pl->fp32_tile_start.assign(1, 0);
        for (uint32_t i = 0; i < nvars; ++i)
            if (!pl->vars[i].quantised) {
                pl->fp32_var.push_back(i);
                pl->fp32_tile_start.push_back(pl->fp32_tile_start.back() + pl->vars[i].ntiles);
            }

        // ---- the decoder's own division (it keeps no sums): short runs of equal length, dealt out
        // to the warps in turn, so that the warps of a launch sweep through memory side by side
        const uint64_t max_dec_warps = (uint64_t)pl->n_sm * omc::DECOMPRESS_CTAS_PER_SM * omc::WARPS_PER_CTA;
        pl->dec_nwarps = (uint32_t)(tiles < max_dec_warps ? tiles : max_dec_warps);
        pl->dec_tiles_per_run = omc::decode_tiles_per_run(B);
        pl->dec_nruns = omc::runs_for(tiles, pl->dec_nwarps, pl->dec_tiles_per_run, omc::DECODE_MAX_RUNS);
        pl->dec_run_var.assign(pl->dec_nruns, 0);
        for (uint32_t r = 0, i = 0; r < pl->dec_nruns; ++r) {
            const uint64_t t = (uint64_t)(((unsigned __int128)r * tiles) / pl->dec_nruns);   // the run's first tile
            while (i + 1 < nvars && pl->vars[i + 1].tile_start <= t) ++i;
            pl->dec_run_var[r] = i;
        }
        pl->ws_tickets_off = omc::WS_HEADER_BYTES;
        pl->ws_slots_off = round_up(pl->ws_tickets_off + 4ull * (nq ? nq : 1), 256);
        // omc_transition numbers the records anew for each launch: at most one per run and one more
        // per variable that is fitted
        const uint64_t slots_cap = std::max<uint64_t>(slots ? slots : 1, (uint64_t)pl->nwarps + nq);
        pl->ws_bytes = round_up(pl->ws_slots_off + sizeof(omc::Partial) * slots_cap, 256);
    } catch (const std::bad_alloc &) {
        delete pl;
        return OMC_ERR_NO_MEMORY;
    }
    *out = pl;
    return OMC_OK;
}

extern "C" int omc_plan_destroy(omc_plan_t *plan)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    int rc = OMC_OK;
    if (plan->d_vars) {
        int cur = 0;
        (void)cudaGetDevice(&cur);
        if (plan->device >= 0 && plan->device != cur) (void)cudaSetDevice(plan->device);
        rc = omc::note_cuda(cudaFree(plan->d_vars));
        if (plan->device >= 0 && plan->device != cur) (void)cudaSetDevice(cur);
    }
    delete plan;
    return rc;
}

extern "C" int omc_plan_sizes(const omc_plan_t *plan, uint64_t *full_elems, uint64_t *resid_elems,
                              uint64_t *packed_bytes, uint32_t *n_quantised, uint64_t *workspace_bytes,
                              uint64_t *closed_form_bytes)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    if (full_elems) *full_elems = plan->full_elems;
    if (resid_elems) *resid_elems = plan->resid_elems;
    if (packed_bytes) *packed_bytes = plan->packed_bytes;
    if (n_quantised) *n_quantised = plan->nq;
    if (workspace_bytes) *workspace_bytes = plan->ws_bytes;
    if (closed_form_bytes) *closed_form_bytes = plan->closed_form_bytes;
    return OMC_OK;
}

extern "C" int omc_plan_division(const omc_plan_t *plan, uint32_t *n_warps, uint32_t *n_runs, uint64_t *n_tiles,
                                 const uint64_t **run_start)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    if (n_warps) *n_warps = plan->nwarps;
    if (n_runs) *n_runs = plan->nruns;
    if (n_tiles) *n_tiles = plan->ntiles;
    if (run_start) *run_start = plan->run_start.data();
    return OMC_OK;
}

extern "C" int omc_plan_var(const omc_plan_t *plan, uint32_t i, int *quantised, uint64_t *full_off_elems,
                            uint64_t *resid_off_elems, uint64_t *packed_off_bytes, uint64_t *packed_bytes,
                            uint32_t *sb_slot)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    if (i >= plan->nvars) return OMC_ERR_INVALID_ARG;
    const VarDev &v = plan->vars[i];
    if (quantised) *quantised = (int)v.quantised;
    if (full_off_elems) *full_off_elems = v.full_off;
    if (resid_off_elems) *resid_off_elems = v.quantised ? 0 : v.store_off;
    if (packed_off_bytes) *packed_off_bytes = v.quantised ? v.store_off : 0;
    if (packed_bytes) *packed_bytes = v.packed_bytes;
    if (sb_slot) *sb_slot = v.quantised ? v.sb_slot : 0;
    return OMC_OK;
}
