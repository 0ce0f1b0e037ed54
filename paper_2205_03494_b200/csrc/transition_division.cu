// Division of the work of one omc_transition launch, made on the device just before it.
//
// What a tile of a variable costs in a transition depends on both plans (codes copied, FP32 values
// copied, codes expanded, values quantised and fitted), so neither plan's own division balances
// it.  One thread block walks the two variable tables, adds up the estimated costs, cuts the tile
// list into runs of equal cost (the rule omc_plan uses: a tile goes to run
// floor(cost before it * runs / total cost)) and numbers the partial-sum records of the
// variables that get a fresh fit.  Everything stays on the stream: no host copy, no wait.
// A few blocks share the runs and the last one numbers the records; each of them adds up the costs
// for itself (the tables they write that way hold the same values).
#include <cuda_runtime.h>

#include "omc_internal.h"

namespace omc {

namespace {

constexpr int DIV_THREADS = 1024;
constexpr uint32_t LAST_IN_SMEM = 4096;      // variables whose costs a block keeps in shared memory

struct VarCost {
    uint64_t per_tile, entry;
    bool fitted;
};

__device__ __forceinline__ VarCost cost_of(const VarDev *to, const VarDev *from, uint32_t i, const TransitionCosts &c)
{
    const bool qt = to[i].quantised != 0, qf = from[i].quantised != 0;
    VarCost r;
    r.fitted = qt && !qf;
    r.per_tile = (qt && qf) ? c.copy_codes : (!qt && !qf) ? c.copy_fp32 : c.convert;
    r.entry = r.fitted ? c.fit_entry : 0;
    return r;
}

// Exclusive prefix sum over the block's values; returns this thread's prefix, `total` to all.
__device__ __forceinline__ uint64_t block_exclusive_scan(uint64_t x, uint64_t *warp_sums, uint64_t &total)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint64_t incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += y;
    }
    if (lane == 31) warp_sums[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        uint64_t w = lane < DIV_THREADS / 32 ? warp_sums[lane] : 0, wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, wi, d);
            if (lane >= d) wi += y;
        }
        warp_sums[lane] = wi - w;                   // exclusive prefix of the warps' sums
        if (lane == 31) warp_sums[32] = wi;         // the block's total
    }
    __syncthreads();
    const uint64_t r = warp_sums[wid] + incl - x;
    total = warp_sums[32];
    __syncthreads();                                // warp_sums is reused by the next call
    return r;
}

__global__ void __launch_bounds__(DIV_THREADS) transition_division_kernel(const VarDev *to, const VarDev *from,
                                                                          uint32_t nvars, uint64_t ntiles,
                                                                          uint32_t max_runs, TransitionCosts c,
                                                                          TransitionTables out)
{
    __shared__ uint64_t warp_sums[33];
    __shared__ uint64_t s_total;
    __shared__ uint32_t s_nruns;
    __shared__ uint64_t s_last[LAST_IN_SMEM];      // out.last for the searches below, if it fits
    const uint32_t tid = threadIdx.x;
    const bool cached = nvars <= LAST_IN_SMEM;
    // omc_transition's main kernel may be scheduled now; it waits for this grid's results itself
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- cost before each variable
    uint64_t carry = 0;
    for (uint32_t base = 0; base < nvars; base += DIV_THREADS) {
        const uint32_t i = base + tid;
        uint64_t x = 0;
        if (i < nvars) {
            const VarCost vc = cost_of(to, from, i, c);
            x = vc.entry + vc.per_tile * to[i].ntiles;
        }
        uint64_t chunk;
        const uint64_t pre = block_exclusive_scan(x, warp_sums, chunk);
        if (i < nvars) {
            const VarCost vc = cost_of(to, from, i, c);
            out.before[i] = carry + pre;
            const uint64_t last = carry + pre + vc.entry + vc.per_tile * (to[i].ntiles - 1);   // cost before its last tile
            out.last[i] = last;
            if (cached) s_last[i] = last;
        }
        carry += chunk;
    }
    if (tid == 0) {
        // runs no shorter than the dearest tile, so that consecutive tiles of a variable lie in the
        // same run or in neighbouring ones
        uint64_t nr = carry / c.max_tile;
        if (nr > max_runs) nr = max_runs;
        if (nr < 1) nr = 1;
        s_total = carry;
        s_nruns = (uint32_t)nr;
        if (blockIdx.x == 0) *out.nruns = (uint32_t)nr;
    }
    __syncthreads();
    const uint64_t total = s_total;
    const uint32_t nruns = s_nruns;
    // cost * nruns / total and its ceiling; 64-bit arithmetic when the product fits (it does unless
    // the model has more than 2^40 tiles), which spares two long software divisions per thread
    const bool small = total < (1ull << 50) && nruns < (1u << 14);
    auto run_of = [&](uint64_t cost) {
        return small ? (uint32_t)(cost * nruns / total) : (uint32_t)(((unsigned __int128)cost * nruns) / total);
    };
    auto first_cost_of_run = [&](uint32_t r) {
        return small ? ((uint64_t)r * total + nruns - 1) / nruns
                     : (uint64_t)(((unsigned __int128)r * total + nruns - 1) / nruns);
    };
    auto last_cbt = [&](uint32_t i) { return cached ? s_last[i] : out.last[i]; };

    // ---- where each run starts: the first tile whose cost-before reaches ceil(r * total / nruns)
    const uint32_t run_blocks = gridDim.x - 1;        // the last block numbers the records instead
    for (uint32_t r = blockIdx.x * DIV_THREADS + tid; blockIdx.x < run_blocks && r <= nruns;
         r += run_blocks * DIV_THREADS) {
        if (r == nruns) {
            out.run_start[r] = ntiles;
            continue;
        }
        const uint64_t target = first_cost_of_run(r);
        uint32_t lo = 0, hi = nvars;                 // smallest i with last_cbt(i) >= target, or nvars
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (last_cbt(mid) >= target) hi = mid; else lo = mid + 1;
        }
        if (lo == nvars) {                           // an empty run at the end
            out.run_start[r] = ntiles;
            out.run_var[r] = nvars - 1;
        } else {
            const VarCost vc = cost_of(to, from, lo, c);
            const uint64_t first = out.before[lo] + vc.entry;
            const uint64_t k = target <= first ? 0 : (target - first + vc.per_tile - 1) / vc.per_tile;
            out.run_start[r] = to[lo].tile_start + k;
            out.run_var[r] = lo;
        }
    }

    // ---- partial-sum records of the variables that get a fresh fit
    if (blockIdx.x != run_blocks) return;
    uint32_t slot_carry = 0;
    for (uint32_t base = 0; base < nvars; base += DIV_THREADS) {
        const uint32_t i = base + tid;
        uint32_t first = 0, n = 0;
        if (i < nvars) {
            const VarCost vc = cost_of(to, from, i, c);
            if (vc.fitted) {
                first = run_of(out.before[i] + vc.entry);
                n = run_of(last_cbt(i)) - first + 1;
            }
        }
        uint64_t chunk;
        const uint64_t pre = block_exclusive_scan(n, warp_sums, chunk);
        if (i < nvars) {
            TransitionVar tv;
            tv.first_run = first;
            tv.nslots = n;
            tv.slot_base = slot_carry + (uint32_t)pre;
            tv.pad = 0;
            out.vars[i] = tv;
        }
        slot_carry += (uint32_t)chunk;
    }
}

}  // namespace

void launch_transition_division(const VarDev *to, const VarDev *from, uint32_t nvars, uint64_t ntiles,
                                uint32_t max_runs, const TransitionCosts &c, const TransitionTables &out,
                                void *stream)
{
    uint32_t grid = (max_runs + DIV_THREADS) / DIV_THREADS;      // one thread per run, within reason
    if (grid > 32) grid = 32;
    grid += 1;                                                   // and one block for the records
    transition_division_kernel<<<grid, DIV_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(to, from, nvars, ntiles,
                                                                                          max_runs, c, out);
}

}  // namespace omc
