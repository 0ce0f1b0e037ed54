// Device-side C-ABI entry points: argument checks, launch geometry, dispatch on the format.
#include <cuda_runtime.h>

#include <algorithm>

#include "omc_internal.h"

namespace omc {
int note_cuda(cudaError_t e);

#define OMC_DECLARE_FORMAT(E_, M_) extern const FmtOps ops_E##E_##M##M_;
#define OMC_FORMAT_LIST(X)                                                                      \
    X(5, 2) X(4, 3) X(5, 6) X(5, 10) /* benchmark configurations                              */ \
    X(4, 14) X(3, 7) X(2, 3)         /* Tables 1 and 2 of the paper                           */ \
    X(3, 9) X(4, 8) X(5, 7)          /* the 13-bit formats of Sec. 3.5.3                      */ \
    X(8, 7) X(8, 23)                 /* bfloat16 and FP32 itself                              */
OMC_FORMAT_LIST(OMC_DECLARE_FORMAT)
// the fixed-point variant (Sec. 2.2): Q7, Q11 and Q15, the widths of the benchmark configurations
#define OMC_DECLARE_FIXED_FORMAT(I_, F_) extern const FmtOps ops_I##I_##F##F_;
#define OMC_FIXED_FORMAT_LIST(X) X(0, 7) X(0, 11) X(0, 15)
OMC_FIXED_FORMAT_LIST(OMC_DECLARE_FIXED_FORMAT)
extern const FmtOps ops_dynamic;   // any other format of either family, at run time

const FmtOps *find_ops(int E, int M, int fixed)
{
#define OMC_ADDR(E_, M_) &ops_E##E_##M##M_,
#define OMC_FIXED_ADDR(I_, F_) &ops_I##I_##F##F_,
    static const FmtOps *const table[] = {OMC_FORMAT_LIST(OMC_ADDR) OMC_FIXED_FORMAT_LIST(OMC_FIXED_ADDR)};
    for (const FmtOps *o : table)
        if (o->E == E && o->M == M && o->fixed == (fixed ? 1 : 0)) return o;
    if (fixed) return fixed_format_ok(E, M) ? &ops_dynamic : nullptr;
    if (E >= 2 && E <= 8 && M >= 0 && M <= 23) return &ops_dynamic;
    return nullptr;
}
}  // namespace omc

using omc::KParams;

// omc_transition's cost model (sixteenths of a tile; swept on B200, flat around these values): an
// FP32 tile copied, and the fixed part of a tile converted.
constexpr uint32_t TCOST_COPY = 16, TCOST_CONVERT = 12;

static bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

extern "C" int omc_plan_prepare(omc_plan_t *plan, void *workspace, void *stream)
{
    if (!plan || !workspace) return OMC_ERR_NULL_PTR;
    if (misaligned(workspace)) return OMC_ERR_MISALIGNED;
    int dev = 0;
    int rc = omc::note_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    if (plan->d_vars && plan->device != dev) return OMC_ERR_PLAN_MISMATCH;
    if (!plan->d_vars) {
        const size_t bytes = sizeof(omc::VarDev) * (size_t)plan->nvars;
        const size_t rs_bytes = sizeof(uint64_t) * plan->run_start.size();
        const size_t rv_bytes = sizeof(uint32_t) * plan->run_var.size();
        const size_t dv_bytes = sizeof(uint32_t) * plan->dec_run_var.size();
        // omc_transition's tables (filled on the device before each launch)
        const size_t nv = plan->nvars, nw = plan->nwarps;
        const size_t tables = (bytes + 16 + rs_bytes + rv_bytes + dv_bytes + 15) / 16 * 16;
        const size_t nf = plan->fp32_var.size();
        const size_t tr_bytes = 16 * nv + 8 * (nw + 1) + sizeof(omc::TransitionVar) * nv + 4 * nw + 16 +
                                8 * (nf + 1) + 4 * nf + 16;
        rc = omc::note_cuda(cudaMalloc(reinterpret_cast<void **>(&plan->d_vars), tables + tr_bytes));
        if (rc) { plan->d_vars = nullptr; return rc; }
        char *const base = reinterpret_cast<char *>(plan->d_vars);
        rc = omc::note_cuda(cudaMemcpy(base, plan->vars.data(), bytes, cudaMemcpyHostToDevice));
        if (!rc) rc = omc::note_cuda(cudaMemset(base + bytes, 0, 16));
        if (!rc) rc = omc::note_cuda(cudaMemcpy(base + bytes + 16, plan->run_start.data(), rs_bytes, cudaMemcpyHostToDevice));
        if (!rc) rc = omc::note_cuda(cudaMemcpy(base + bytes + 16 + rs_bytes, plan->run_var.data(), rv_bytes, cudaMemcpyHostToDevice));
        if (!rc) rc = omc::note_cuda(cudaMemcpy(base + bytes + 16 + rs_bytes + rv_bytes, plan->dec_run_var.data(), dv_bytes, cudaMemcpyHostToDevice));
        if (rc) { (void)cudaFree(plan->d_vars); plan->d_vars = nullptr; return rc; }
        plan->d_status = reinterpret_cast<uint32_t *>(base + bytes);
        plan->d_run_start = reinterpret_cast<uint64_t *>(base + bytes + 16);
        plan->d_run_var = reinterpret_cast<uint32_t *>(base + bytes + 16 + rs_bytes);
        plan->d_dec_run_var = reinterpret_cast<uint32_t *>(base + bytes + 16 + rs_bytes + rv_bytes);
        char *tr = base + tables;                    // 16-byte entries first, then 8-byte ones, then 4-byte ones
        plan->d_trans.vars = reinterpret_cast<omc::TransitionVar *>(tr);
        plan->d_trans.before = reinterpret_cast<uint64_t *>(tr + sizeof(omc::TransitionVar) * nv);
        plan->d_trans.last = plan->d_trans.before + nv;
        plan->d_trans.run_start = plan->d_trans.last + nv;
        plan->d_trans.run_var = reinterpret_cast<uint32_t *>(plan->d_trans.run_start + nw + 1);
        plan->d_trans.nruns = plan->d_trans.run_var + nw;
        // the FP32 variables' tile list, behind the transition tables (8-byte aligned)
        char *fl = reinterpret_cast<char *>(plan->d_trans.run_var) + (4 * nw + 4 + 7) / 8 * 8;
        plan->d_fp32_tile_start = reinterpret_cast<uint64_t *>(fl);
        plan->d_fp32_var = reinterpret_cast<uint32_t *>(fl + 8 * (nf + 1));
        rc = omc::note_cuda(cudaMemcpy(plan->d_fp32_tile_start, plan->fp32_tile_start.data(), 8 * (nf + 1), cudaMemcpyHostToDevice));
        if (!rc && nf) rc = omc::note_cuda(cudaMemcpy(plan->d_fp32_var, plan->fp32_var.data(), 4 * nf, cudaMemcpyHostToDevice));
        if (rc) { (void)cudaFree(plan->d_vars); plan->d_vars = nullptr; return rc; }
        plan->device = dev;
    }
    // a repeated call also clears the status word (after a kernel gave up, the workspace's counters
    // are left mid-count and the caller prepares again)
    rc = omc::note_cuda(cudaMemsetAsync(plan->d_status, 0, sizeof(uint32_t), static_cast<cudaStream_t>(stream)));
    if (rc) return rc;
    return omc::note_cuda(cudaMemsetAsync(workspace, 0, plan->ws_bytes, static_cast<cudaStream_t>(stream)));
}

static int check_ready(const omc_plan_t *plan)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    if (!plan->d_vars) return OMC_ERR_PLAN_MISMATCH;
    int dev = 0;
    int rc = omc::note_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    return dev == plan->device ? OMC_OK : OMC_ERR_PLAN_MISMATCH;
}

// The diagnostic of omc_plan_inject_wait_timeout applies to one launch.
static void take_injection(const omc_plan_t *plan, KParams &p)
{
    p.wait_limit = plan->inject_polls;
    p.skip_loads = plan->inject_polls ? 1u : 0u;
    plan->inject_polls = 0;
}

static KParams whole_model(const omc_plan_t *plan, void *workspace)
{
    KParams p{};
    take_injection(plan, p);
    p.dependent = 1u;
    p.vars = plan->d_vars;
    p.var_begin = 0;
    p.var_end = plan->nvars;
    p.tile_begin = 0;
    p.tile_count = plan->ntiles;
    p.nwarps = plan->nwarps;
    p.nruns = plan->nruns;
    p.run_start = plan->d_run_start;
    p.run_var = plan->d_run_var;
    p.pvt = (plan->flags & OMC_PLAN_PVT) ? 1u : 0u;
    p.dyn_e = plan->fmt.exp_bits;
    p.dyn_m = plan->fmt.man_bits;
    p.dyn_fixed = plan->fmt.flags & OMC_FORMAT_FIXED_POINT;
    p.status = plan->d_status;
    p.queue = static_cast<uint32_t *>(workspace);       // the workspace header
    p.tickets = reinterpret_cast<uint32_t *>(static_cast<char *>(workspace) + plan->ws_tickets_off);
    p.slots = reinterpret_cast<omc::Partial *>(static_cast<char *>(workspace) + plan->ws_slots_off);
    return p;
}

// Whether the fused round takes the FP32 variables' tiles from the queue: the format has such a
// kernel and the FP32 tiles are a real share of the work.  Measured on the 100M set, against FP32
// tiles inside the runs: 8 to 28 % faster from a tenth of the matrices in FP32 on (S1E4M14 at a
// tenth: 0.232 -> 0.167 ms), except with S1E5M10, whose kernel already moves 6.3 TB/s at a tenth
// (the queue is 4 % slower there) and gains 8 % at a half: hence a quarter of the tiles as its
// threshold and a fiftieth for the other formats (a few small vectors are cheaper inside the runs
// than one more round trip to the counter for every warp).
static bool use_fp32_queue(const omc_plan_t *plan, KParams &p)
{
    if (!plan->ops->update_q || plan->fp32_var.empty()) return false;
    const bool fp16 = plan->fmt.exp_bits == 5 && plan->fmt.man_bits == 10;
    if (plan->fp32_tile_start.back() * (fp16 ? 4 : 50) < plan->ntiles) return false;
    p.fp32_tile_start = plan->d_fp32_tile_start;
    p.fp32_var = plan->d_fp32_var;
    p.n_fp32 = (uint32_t)plan->fp32_var.size();
    return true;
}

static int grid_for(uint32_t nwarps, int warps_per_cta = omc::WARPS_PER_CTA)
{
    return (int)((nwarps + warps_per_cta - 1) / warps_per_cta);
}

extern "C" int omc_compress(const omc_plan_t *plan, const float *params, uint8_t *packed, float *resid,
                            float *sb, void *workspace, void *stream)
{
    int rc = check_ready(plan);
    if (rc) return rc;
    if (!params || !workspace) return OMC_ERR_NULL_PTR;
    if (plan->nq && (!packed || !sb)) return OMC_ERR_NULL_PTR;
    if (plan->resid_elems && !resid) return OMC_ERR_NULL_PTR;
    if (misaligned(params) || misaligned(packed) || misaligned(resid) || misaligned(sb) || misaligned(workspace))
        return OMC_ERR_MISALIGNED;
    KParams p = whole_model(plan, workspace);
    p.packed = packed; p.resid = resid; p.sb = sb; p.fin = params;
    plan->ops->compress(p, grid_for(p.nwarps, plan->ops->fit_warps), stream);
    return omc::note_cuda(cudaGetLastError());
}

extern "C" int omc_decompress(const omc_plan_t *plan, const uint8_t *packed, const float *resid,
                              const float *sb, uint32_t first_var, uint32_t n_vars, float *out, void *stream)
{
    int rc = check_ready(plan);
    if (rc) return rc;
    if (n_vars == 0 || first_var >= plan->nvars || n_vars > plan->nvars - first_var) return OMC_ERR_INVALID_ARG;
    if (!out) return OMC_ERR_NULL_PTR;
    bool any_q = false, any_r = false;
    for (uint32_t i = first_var; i < first_var + n_vars; ++i)
        (plan->vars[i].quantised ? any_q : any_r) = true;
    if (any_q && (!packed || !sb)) return OMC_ERR_NULL_PTR;
    if (any_r && !resid) return OMC_ERR_NULL_PTR;
    if (misaligned(packed) || misaligned(resid) || misaligned(sb) || misaligned(out)) return OMC_ERR_MISALIGNED;
    KParams p{};
    take_injection(plan, p);
    p.dependent = n_vars != plan->nvars ? 1u : 0u;
    p.vars = plan->d_vars;
    p.var_begin = first_var;
    p.var_end = first_var + n_vars;
    p.tile_begin = plan->vars[first_var].tile_start;
    const omc::VarDev &lastv = plan->vars[first_var + n_vars - 1];
    p.tile_count = lastv.tile_start + lastv.ntiles - p.tile_begin;
    const uint64_t max_warps = (uint64_t)plan->n_sm * omc::DECOMPRESS_CTAS_PER_SM * omc::WARPS_PER_CTA;
    p.nwarps = (uint32_t)(p.tile_count < max_warps ? p.tile_count : max_warps);
    // short runs of equal length, dealt out to the warps in turn
    if (n_vars == plan->nvars) {      // the whole model: the plan knows where each run starts
        p.nwarps = plan->dec_nwarps;
        p.nruns = plan->dec_nruns;
        p.run_var = plan->d_dec_run_var;
    } else {
        p.nruns = omc::runs_for(p.tile_count, p.nwarps, plan->dec_tiles_per_run, omc::DECODE_MAX_RUNS);
    }
    p.pvt = (plan->flags & OMC_PLAN_PVT) ? 1u : 0u;
    p.dyn_e = plan->fmt.exp_bits;
    p.dyn_m = plan->fmt.man_bits;
    p.dyn_fixed = plan->fmt.flags & OMC_FORMAT_FIXED_POINT;
    p.status = plan->d_status;
    p.packed = const_cast<uint8_t *>(packed);
    p.resid = const_cast<float *>(resid);
    p.sb = const_cast<float *>(sb);
    p.fout = out;
    plan->ops->decompress(p, grid_for(p.nwarps), stream);
    return omc::note_cuda(cudaGetLastError());
}

extern "C" int omc_update_recompress(const omc_plan_t *plan, uint8_t *packed, float *resid, float *sb,
                                     const float *grads, float lr, float *debug_w_out, void *workspace,
                                     void *stream)
{
    int rc = check_ready(plan);
    if (rc) return rc;
    if (!grads || !workspace) return OMC_ERR_NULL_PTR;
    if (plan->nq && (!packed || !sb)) return OMC_ERR_NULL_PTR;
    if (plan->resid_elems && !resid) return OMC_ERR_NULL_PTR;
    if (misaligned(grads) || misaligned(packed) || misaligned(resid) || misaligned(sb) ||
        misaligned(workspace) || misaligned(debug_w_out))
        return OMC_ERR_MISALIGNED;
    KParams p = whole_model(plan, workspace);
    p.packed = packed; p.resid = resid; p.sb = sb; p.fin = grads; p.fout = debug_w_out;
    p.neg_lr = -lr;
    if (debug_w_out)
        plan->ops->update_w(p, grid_for(p.nwarps, plan->ops->fit_warps), stream);
    else if (use_fp32_queue(plan, p))
        plan->ops->update_q(p, grid_for(p.nwarps, plan->ops->fit_warps), stream);
    else
        plan->ops->update(p, grid_for(p.nwarps, plan->ops->fit_warps), stream);
    return omc::note_cuda(cudaGetLastError());
}

extern "C" int omc_update_recompress_host(const omc_plan_t *plan, uint8_t *packed, float *resid, float *sb,
                                          const float *host_grads, float lr, float *grads_staging,
                                          float *host_sb_out, void *workspace, void *stream)
{
    int rc = check_ready(plan);
    if (rc) return rc;
    if (!host_grads || !grads_staging) return OMC_ERR_NULL_PTR;
    if (misaligned(grads_staging)) return OMC_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = omc::note_cuda(cudaMemcpyAsync(grads_staging, host_grads, sizeof(float) * plan->full_elems,
                                        cudaMemcpyHostToDevice, st));
    if (rc) return rc;
    rc = omc_update_recompress(plan, packed, resid, sb, grads_staging, lr, nullptr, workspace, stream);
    if (rc) return rc;
    if (host_sb_out && plan->nq) {
        rc = omc::note_cuda(cudaMemcpyAsync(host_sb_out, sb, sizeof(float) * 2 * plan->nq,
                                            cudaMemcpyDeviceToHost, st));
        if (rc) return rc;
    }
    return omc::note_cuda(cudaStreamSynchronize(st));
}

extern "C" int omc_plan_status(const omc_plan_t *plan, void *stream, uint32_t *host_status)
{
    int rc = check_ready(plan);
    if (rc) return rc;
    if (!host_status) return OMC_ERR_NULL_PTR;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = omc::note_cuda(cudaMemcpyAsync(host_status, plan->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    if (rc) return rc;
    return omc::note_cuda(cudaStreamSynchronize(st));
}

extern "C" int omc_plan_inject_wait_timeout(omc_plan_t *plan, uint32_t polls)
{
    if (!plan) return OMC_ERR_NULL_PTR;
    if (polls == 0 || polls > (1u << 24)) return OMC_ERR_INVALID_ARG;
    plan->inject_polls = polls;
    return OMC_OK;
}

extern "C" int omc_transition(const omc_plan_t *from, const omc_plan_t *to, const uint8_t *packed_from,
                              const float *resid_from, const float *sb_from, uint8_t *packed_to,
                              float *resid_to, float *sb_to, void *workspace_to, void *stream)
{
    int rc = check_ready(from);
    if (rc) return rc;
    rc = check_ready(to);
    if (rc) return rc;
    if (from->nvars != to->nvars || from->fmt.exp_bits != to->fmt.exp_bits || from->fmt.man_bits != to->fmt.man_bits ||
        from->fmt.flags != to->fmt.flags)
        return OMC_ERR_PLAN_MISMATCH;
    for (uint32_t i = 0; i < to->nvars; ++i)
        if (from->vars[i].n != to->vars[i].n) return OMC_ERR_PLAN_MISMATCH;
    if (!to->ops->transition) return OMC_ERR_BAD_FORMAT;
    if (!workspace_to) return OMC_ERR_NULL_PTR;
    if (from->nq && (!packed_from || !sb_from)) return OMC_ERR_NULL_PTR;
    if (from->resid_elems && !resid_from) return OMC_ERR_NULL_PTR;
    if (to->nq && (!packed_to || !sb_to)) return OMC_ERR_NULL_PTR;
    if (to->resid_elems && !resid_to) return OMC_ERR_NULL_PTR;
    if (misaligned(packed_from) || misaligned(resid_from) || misaligned(sb_from) || misaligned(packed_to) ||
        misaligned(resid_to) || misaligned(sb_to) || misaligned(workspace_to))
        return OMC_ERR_MISALIGNED;
    // The launch's own division of the work, by what each tile costs given both plans: copying codes
    // moves B/4 bytes per element, copying FP32 values 8, converting 4 + B/8 plus the arithmetic; a
    // variable that is fitted costs three tiles more (as in omc_plan).
    const uint32_t B = 1u + to->fmt.exp_bits + to->fmt.man_bits;
    omc::TransitionCosts costs;
    costs.copy_codes = (B + 1) / 2 * TCOST_COPY / 16;
    costs.copy_fp32 = TCOST_COPY;
    costs.convert = TCOST_CONVERT + B / 4;
    costs.fit_entry = 48;
    if (costs.copy_codes < 1) costs.copy_codes = 1;
    costs.max_tile = std::max(std::max(costs.copy_codes, costs.copy_fp32), costs.convert);
    omc::launch_transition_division(to->d_vars, from->d_vars, to->nvars, to->ntiles, to->nwarps, costs, to->d_trans,
                                    stream);
    KParams p = whole_model(to, workspace_to);
    p.packed = packed_to; p.resid = resid_to; p.sb = sb_to;
    p.vars_from = from->d_vars;
    p.packed_from = packed_from; p.resid_from = resid_from; p.sb_from = sb_from;
    p.run_start = to->d_trans.run_start;
    p.run_var = to->d_trans.run_var;
    p.trans_vars = to->d_trans.vars;
    p.nruns_dev = to->d_trans.nruns;
    to->ops->transition(p, grid_for(p.nwarps, to->ops->fit_warps), stream);
    return omc::note_cuda(cudaGetLastError());
}

static int aggregate_impl(const omc_plan_t *const *plans, uint32_t n_clients, const uint8_t *const *packed,
                          const float *const *resid, const float *const *sb, float *out, uint32_t divide,
                          uint32_t accumulate, void *stream)
{
    if (!plans || !packed || !resid || !sb || !out) return OMC_ERR_NULL_PTR;
    if (n_clients == 0 || n_clients > (uint32_t)omc::MAX_CLIENTS) return OMC_ERR_INVALID_ARG;
    if (misaligned(out)) return OMC_ERR_MISALIGNED;
    omc::AggParams p{};
    const omc_plan_t *first = plans[0];
    for (uint32_t k = 0; k < n_clients; ++k) {
        const omc_plan_t *pl = plans[k];
        int rc = check_ready(pl);
        if (rc) return rc;
        if (pl->nvars != first->nvars || pl->fmt.exp_bits != first->fmt.exp_bits ||
            pl->fmt.man_bits != first->fmt.man_bits || pl->fmt.flags != first->fmt.flags)
            return OMC_ERR_PLAN_MISMATCH;
        for (uint32_t i = 0; i < pl->nvars; ++i)
            if (pl->vars[i].n != first->vars[i].n) return OMC_ERR_PLAN_MISMATCH;
        if (pl->nq && (!packed[k] || !sb[k])) return OMC_ERR_NULL_PTR;
        if (pl->resid_elems && !resid[k]) return OMC_ERR_NULL_PTR;
        if (misaligned(packed[k]) || misaligned(resid[k]) || misaligned(sb[k])) return OMC_ERR_MISALIGNED;
        p.vars[k] = pl->d_vars;
        p.packed[k] = packed[k];
        p.resid[k] = resid[k];
        p.sb[k] = sb[k];
    }
    if (!first->ops->aggregate) return OMC_ERR_BAD_FORMAT;
    p.nclients = n_clients;
    p.divide = divide;
    p.accumulate = accumulate;
    p.nvars = first->nvars;
    p.tile_count = first->ntiles;
    const uint64_t max_warps = (uint64_t)first->n_sm * first->ops->agg_ctas * omc::WARPS_PER_CTA;
    p.nwarps = (uint32_t)(p.tile_count < max_warps ? p.tile_count : max_warps);
    p.nruns = omc::runs_for(p.tile_count, p.nwarps, omc::aggregate_tiles_per_run(n_clients), omc::DECODE_MAX_RUNS);
    p.out = out;
    p.status = first->d_status;
    p.wait_limit = first->inject_polls;       // the diagnostic of omc_plan_inject_wait_timeout, for one launch
    p.skip_loads = first->inject_polls ? 1u : 0u;
    first->inject_polls = 0;
    first->ops->aggregate(p, grid_for(p.nwarps), stream);
    return omc::note_cuda(cudaGetLastError());
}

extern "C" int omc_aggregate(const omc_plan_t *const *plans, uint32_t n_clients, const uint8_t *const *packed,
                             const float *const *resid, const float *const *sb, float *out, void *stream)
{
    return aggregate_impl(plans, n_clients, packed, resid, sb, out, 1u, 0u, stream);
}

extern "C" int omc_aggregate_sum(const omc_plan_t *const *plans, uint32_t n_clients, const uint8_t *const *packed,
                                 const float *const *resid, const float *const *sb, float *out, void *stream)
{
    return aggregate_impl(plans, n_clients, packed, resid, sb, out, 0u, 0u, stream);
}

extern "C" int omc_aggregate_add(const omc_plan_t *const *plans, uint32_t n_clients, const uint8_t *const *packed,
                                 const float *const *resid, const float *const *sb, float *out, void *stream)
{
    return aggregate_impl(plans, n_clients, packed, resid, sb, out, 0u, 1u, stream);
}

namespace {
// out[e] = out[e] / divisor, one correctly rounded FP32 division per element (a multiplication by
// the exact reciprocal when the divisor is a power of two: the same real number, rounded once).
__global__ void divide_kernel(float4 *__restrict__ x, uint64_t n4, float divisor, int pow2)
{
    const float inv = 1.f / divisor;
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n4; i += (uint64_t)gridDim.x * blockDim.x) {
        float4 v = x[i];
        if (pow2) {
            v.x = __fmul_rn(v.x, inv); v.y = __fmul_rn(v.y, inv); v.z = __fmul_rn(v.z, inv); v.w = __fmul_rn(v.w, inv);
        } else {
            v.x = __fdiv_rn(v.x, divisor); v.y = __fdiv_rn(v.y, divisor);
            v.z = __fdiv_rn(v.z, divisor); v.w = __fdiv_rn(v.w, divisor);
        }
        x[i] = v;
    }
}
}  // namespace

extern "C" int omc_divide(const omc_plan_t *plan, float *values, uint32_t divisor, void *stream)
{
    int rc = check_ready(plan);
    if (rc) return rc;
    if (!values) return OMC_ERR_NULL_PTR;
    if (misaligned(values)) return OMC_ERR_MISALIGNED;
    if (divisor == 0 || divisor > (1u << 24)) return OMC_ERR_INVALID_ARG;       // exact as an FP32 value
    const uint64_t n4 = (plan->full_elems + 3) / 4;
    const uint64_t want = (n4 + 255) / 256;
    const uint64_t cap = (uint64_t)plan->n_sm * 8;
    const unsigned grid = (unsigned)(want < cap ? (want ? want : 1) : cap);
    divide_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(reinterpret_cast<float4 *>(values), n4,
                                                                        (float)divisor, (divisor & (divisor - 1)) == 0);
    return omc::note_cuda(cudaGetLastError());
}
