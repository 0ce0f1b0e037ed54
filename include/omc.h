/*
 * libomc -- Online Model Compression (arXiv 2205.03494) parameter store for one NVIDIA B200.
 *
 * Model parameters live in a reduced-bit-width floating-point format (Sec. 2.2) with a
 * per-variable linear transformation (Sec. 2.3); they are decompressed on the fly into a transient
 * FP32 copy for the forward pass and, in the backward pass, decompressed, updated with the gradient
 * and compressed again without the FP32 value ever being stored (Sec. 2.1, Fig. 1).  Only weight
 * matrices are quantised (Sec. 2.4), and only a chosen subset of them (Sec. 2.5, Sec. 3.1).
 *
 * Conventions
 *   - Every function returns OMC_OK (0) or a negative omc_status.  Nothing throws, aborts or traps.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA device memory owned by
 *     the caller, 16-byte aligned, valid until the work queued on `stream` has finished.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Device calls only
 *     enqueue work; they do not synchronise.  Apart from omc_plan_prepare they allocate nothing.
 *     Work queued on one stream runs in stream order.  The library's kernels allow the launch of
 *     a programmatic dependent early (griddepcontrol.launch_dependents) and wait for the kernel
 *     before them themselves; a kernel of the caller's that is launched with programmatic stream
 *     serialization right after a library call must, like any such kernel, call
 *     cudaGridDependencySynchronize() before it reads what that call wrote.
 *   - Non-finite values are data, never errors: they propagate as IEEE-754 prescribes.
 *   - A plan is not thread-safe; distinct plans are independent.
 *
 * Memory layouts (all fixed by the plan; query them with omc_plan_sizes / omc_plan_var)
 *   full   : FP32 arena holding every variable, variable i at element offset full_off[i]; every
 *            offset is a multiple of 4 elements, the gap after a variable is padding that the
 *            library may read and overwrite but never interprets.  Gradients and decompressed output use it.
 *   resid  : FP32 arena with only the variables that stay in FP32, same alignment rule.
 *   packed : byte arena with the codes of the quantised variables.  Variable i occupies
 *            packed_bytes[i] = roundup16(ceil(numel*B/8)) bytes at packed_off[i]; inside it code k
 *            occupies bits [k*B, (k+1)*B) of a little-endian bit stream (bit j of the stream is
 *            bit j%8 of byte j/8); the bits after the last code are zero.  A code is
 *            sign<<(E+M) | exponent_field<<M | mantissa_field.
 *   sb     : float[2 * n_quantised]; sb[2*slot] = s and sb[2*slot+1] = b of Sec. 2.3.
 */
#ifndef OMC_H_
#define OMC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* SxEyMz of Sec. 3.1: x sign, y exponent, z mantissa bits.  Accepted: sign_bits == 1,
 * 2 <= exp_bits <= 8, 0 <= man_bits <= 23 (so 3 <= B <= 32).  S1E8M23 is FP32, S1E5M10 is FP16
 * (Sec. 2.2, Sec. 3.4); the family is the IEEE-754 interchange parametrisation (bias
 * 2^(E-1)-1, gradual underflow, top exponent field = Inf/NaN), rounding to nearest, ties to even.
 * `flags` is 0 for these.
 *
 * flags == OMC_FORMAT_FIXED_POINT selects the fixed-point variant that Sec. 2.2 mentions as an
 * alternative without defining it; the definition here is this library's.  S1IxFy: exp_bits = x
 * integer bits (0 .. 8), man_bits = y fraction bits, 1 <= x + y <= 23, B = 1 + x + y.  A code is
 * the B-bit two's complement of an integer k in [-2^(x+y), 2^(x+y) - 1] and stands for k * 2^-y.
 * Encoding rounds value * 2^y to the nearest integer, ties to even, and saturates at both ends
 * (there is no infinity; +-Inf saturate too); NaN has no code and becomes 0.  The scale is fixed
 * by the format and not taken from the data (that would cost the one-pass update a second pass);
 * the per-variable transformation of Sec. 2.3 adapts to the variable as it does for the
 * floating-point codes.  Layouts, packing and every call are the same.  Q7, Q11 and Q15 (x = 0)
 * have compiled kernels (omc_matmul accepts these three); the other formats run on the slower
 * kernels that take the format at run time. */
typedef struct {
    uint8_t sign_bits, exp_bits, man_bits, flags;
} omc_format_t;
#define OMC_FORMAT_FIXED_POINT 1u

/* What a variable is (Sec. 2.4): only weight matrices are ever quantised. */
enum { OMC_KIND_WEIGHT_MATRIX = 0, OMC_KIND_BIAS = 1, OMC_KIND_NORM = 2, OMC_KIND_OTHER = 3 };

typedef struct {
    uint64_t numel;    /* number of FP32 elements, 1 .. 2^40 */
    uint32_t kind;     /* OMC_KIND_* */
    uint32_t reserved; /* 0 */
} omc_var_desc_t;

typedef struct omc_plan omc_plan_t; /* opaque, owned by the library */

/* Plan flags: the switches of the paper's ablation (Table 4). */
#define OMC_PLAN_PVT 1u          /* fit and apply the per-variable transformation (Sec. 2.3)   */
#define OMC_PLAN_WEIGHTS_ONLY 2u /* only OMC_KIND_WEIGHT_MATRIX is eligible (Sec. 2.4)         */
#define OMC_PLAN_DEFAULT (OMC_PLAN_PVT | OMC_PLAN_WEIGHTS_ONLY)

typedef enum {
    OMC_OK = 0,
    OMC_ERR_INVALID_ARG = -1,   /* a size, index, fraction or flag is out of range             */
    OMC_ERR_BAD_FORMAT = -2,    /* omc_format_t outside the accepted family                    */
    OMC_ERR_NULL_PTR = -3,      /* a required pointer is NULL                                  */
    OMC_ERR_MISALIGNED = -4,    /* a device pointer is not 16-byte aligned                     */
    OMC_ERR_PLAN_MISMATCH = -5, /* the plan was not prepared, or not for this call             */
    OMC_ERR_CUDA = -6,          /* a CUDA runtime call failed (see omc_last_cuda_error)        */
    OMC_ERR_NO_MEMORY = -7,     /* host allocation failed                                      */
    OMC_ERR_TOO_LARGE = -8      /* beyond the fixed capacity of omc_compress_var_static        */
} omc_status;

const char *omc_strerror(int status);
/* cudaError_t of the most recent failing runtime call on the calling thread (0 if none). */
int omc_last_cuda_error(void);

/*
 * omc_plan -- decide which variables are compressed and lay out the arenas (host only; touches no
 * device memory and needs no GPU).
 *   Sec. 2.4: with OMC_PLAN_WEIGHTS_ONLY only weight matrices are eligible; biases and
 *   normalisation parameters stay FP32.  Sec. 2.5 / Sec. 3.1: a fraction of the eligible
 *   variables is quantised, chosen at random (the paper's default is 0.9 and a new draw per round
 *   and per client: make one plan per draw).
 *   vars[nvars]  host; the model's variables in the order the arenas will hold them.
 *   fraction     in (0, 1]: k = floor(fraction * W + 1/2) of the W eligible variables.
 *   seed         used iff mask == NULL: the eligible indices, ascending, are shuffled by
 *                Fisher-Yates (i = W-1 .. 1, j = next() mod (i+1)) driven by SplitMix64(seed); the
 *                first k are quantised.
 *   mask         optional host array of nvars bytes; non-zero = quantise variable i.  Overrides
 *                fraction and seed; a marked variable that is not eligible is an error.
 *   flags        OMC_PLAN_* bits.
 *   out          receives the plan; release it with omc_plan_destroy.
 */
int omc_plan(const omc_var_desc_t *vars, uint32_t nvars, omc_format_t fmt, double fraction,
             uint64_t seed, const uint8_t *mask, uint32_t flags, omc_plan_t **out);
int omc_plan_destroy(omc_plan_t *plan); /* also frees the plan's device tables, if any */

/*
 * omc_plan_seed -- one seed per (round, client) from one seed for the whole job (host only).
 * Sec. 3.1 varies the selection from round to round and from client to client; the paper does
 * not say how the draws are seeded, so the rule is this library's: the seed of (round, client) is
 * output number round * 2^32 + client (counted from 0) of the SplitMix64 stream seeded with
 * base_seed.  Pass the result to omc_plan as `seed`.  The generator's state is a counter, so the
 * call costs the same for every (round, client).  base_seed = 0, round = 0 gives the generator's
 * published check values for client = 0, 1, 2, ...
 */
uint64_t omc_plan_seed(uint64_t base_seed, uint32_t round, uint32_t client);

/*
 * Sizes the caller must allocate (any output pointer may be NULL).
 *   closed_form_bytes: the stored size of the model as the paper counts it (Tables 1 and 2):
 *   sum over quantised variables of ceil(numel*B/8) + 8, plus 4*numel for the others.
 */
int omc_plan_sizes(const omc_plan_t *plan, uint64_t *full_elems, uint64_t *resid_elems,
                   uint64_t *packed_bytes, uint32_t *n_quantised, uint64_t *workspace_bytes,
                   uint64_t *closed_form_bytes);
/* Where variable i lives.  resid_off_elems is meaningful iff !quantised; packed_* and sb_slot iff
 * quantised. */
int omc_plan_var(const omc_plan_t *plan, uint32_t i, int *quantised, uint64_t *full_off_elems,
                 uint64_t *resid_off_elems, uint64_t *packed_off_bytes, uint64_t *packed_bytes,
                 uint32_t *sb_slot);

/*
 * omc_plan_division -- how the plan divides the work of one launch (host only).
 * The model's variables are cut into tiles of 1024 elements, numbered in variable order (a
 * variable's last tile may be short), and the tiles into *n_runs contiguous runs of about equal
 * estimated cost: run r = tiles [run_start[r], run_start[r + 1]).  Warp w of omc_compress and
 * omc_update_recompress takes runs w, w + *n_warps, ... (one run per warp as the plans are made
 * today: *n_runs == *n_warps), so that a warp adds up a variable's elements in its registers.
 * *run_start points at *n_runs + 1 non-decreasing entries owned by the plan (valid until
 * omc_plan_destroy), the first 0 and the last *n_tiles; *n_runs is a multiple of *n_warps.  Any
 * output pointer may be NULL.  Sec. 2.3's sums are taken per variable whatever the division; it
 * only decides which warp adds which elements, and so the order of the fp64 additions.
 * (omc_decompress keeps no sums and deals out short runs of equal length to its warps instead;
 * omc_transition makes a division of its own for each call.)
 */
int omc_plan_division(const omc_plan_t *plan, uint32_t *n_warps, uint32_t *n_runs, uint64_t *n_tiles,
                      const uint64_t **run_start);

/*
 * omc_plan_prepare -- copy the plan's tables to the current device (the one allocation the
 * library makes; synchronous) and clear `workspace` (device, workspace_bytes) on `stream`.
 * Must precede the first device call with this plan; the workspace then stays valid from call
 * to call (each kernel leaves it cleared) as long as calls using it do not overlap on the GPU.
 * Calling it again re-clears the workspace and the plan's status word (the way back to a usable
 * state after omc_plan_status reported a kernel that gave up).
 */
int omc_plan_prepare(omc_plan_t *plan, void *workspace, void *stream);

/*
 * omc_plan_status -- waits for `stream`, then reports the plan's device status word in
 * *host_status (host): 0 = every kernel launched with this plan so far ran to completion;
 * non-zero = a kernel gave up waiting for one of its own asynchronous copies (its outputs are
 * then incomplete; the context stays usable).  The kernels never wait for each other, so this
 * is not expected to happen; the bounded wait exists so that a fault cannot hang the GPU.
 */
int omc_plan_status(const omc_plan_t *plan, void *stream, uint32_t *host_status);

/*
 * omc_plan_inject_wait_timeout -- diagnostics for the bounded waits (the paper has no counterpart).
 * The next kernel launched with this plan (omc_compress, omc_decompress, omc_update_recompress,
 * omc_transition with the plan as destination, omc_aggregate, omc_aggregate_sum and
 * omc_aggregate_add with the plan first in the list, omc_matmul) announces its asynchronous loads to
 * their barriers without issuing them and gives up each wait after `polls` polls (1 .. 2^24):
 * every wait runs out with no copy in flight, the kernel sets the status word and returns, its
 * outputs are garbage.  Afterwards omc_plan_status reports non-zero; call omc_plan_prepare again
 * (it clears the status word and the workspace, whose counters the kernel left mid-count) before
 * the next real call.  Host only; applies to one launch.  For tests of the give-up path: nothing
 * faults, hangs or reads out of bounds.
 */
int omc_plan_inject_wait_timeout(omc_plan_t *plan, uint32_t polls);

/*
 * omc_compress -- initial compression of a full-precision model (Sec. 2.2, 2.3).
 * For each quantised variable V: codes = Q(V); Vt = Q^-1(codes); (s, b) = argmin ||s*Vt+b-V||_2
 * from fp64 sums, stored FP32 (s = 1 when all Vt are equal or the denominator is 0 / not finite;
 * s = 1, b = 0 without OMC_PLAN_PVT).  Other variables are copied to the resid arena.
 *   params  device, full layout, read only.     packed, resid, sb  device, written.
 */
int omc_compress(const omc_plan_t *plan, const float *params, uint8_t *packed, float *resid,
                 float *sb, void *workspace, void *stream);

/*
 * omc_decompress -- forward path of Fig. 1: the transient FP32 copy of variables
 * [first_var, first_var + n_vars), written at their offsets in `out` (device, full layout):
 * Vbar_k = fma(s, Vt_k, b) for quantised variables (one rounding), a copy for the others.
 */
int omc_decompress(const omc_plan_t *plan, const uint8_t *packed, const float *resid,
                   const float *sb, uint32_t first_var, uint32_t n_vars, float *out, void *stream);

/*
 * omc_update_recompress -- backward path of Fig. 1 in one launch: per element
 * W = fma(-lr, g, fma(s, Vt, b)), re-quantised at once; (s, b) refitted per variable from fp64
 * sums over (W, Q^-1 Q(W)); FP32 variables take W = fma(-lr, g, V) in place.  W itself is never
 * stored, unless debug_w_out (device, full layout, may be NULL) asks for it.
 *   packed, resid, sb  device, updated in place.    grads  device, full layout, read only.
 * A NaN produced by the arithmetic is encoded as the positive NaN with all mantissa bits set.
 */
int omc_update_recompress(const omc_plan_t *plan, uint8_t *packed, float *resid, float *sb,
                          const float *grads, float lr, float *debug_w_out, void *workspace,
                          void *stream);

/*
 * omc_update_recompress_host -- the same round (Sec. 2.1) for a caller whose gradients arrive in
 * host memory: copies host_grads (host, full layout, pinned for full speed) into grads_staging
 * (device, full layout), runs omc_update_recompress, copies the refitted (s, b) array back into
 * host_sb_out (host, 2*n_quantised floats, may be NULL) and waits for `stream` before returning.
 */
int omc_update_recompress_host(const omc_plan_t *plan, uint8_t *packed, float *resid, float *sb,
                               const float *host_grads, float lr, float *grads_staging,
                               float *host_sb_out, void *workspace, void *stream);

/*
 * omc_transition -- re-selection (Sec. 2.5, Sec. 3.1: the quantised subset of weight matrices
 * changes from round to round and from client to client).  Takes a model's state under plan `from`
 * to its state under plan `to` in one call (a small kernel that divides the work by what each
 * variable needs, given both plans, and the kernel that does it; `to`'s device tables are
 * rewritten by the first, so calls with the same `to` must not overlap on the GPU).  Both plans
 * must be prepared on the current device
 * and describe the same variables (count, sizes) in the same format, else OMC_ERR_PLAN_MISMATCH.
 * Per variable: quantised in both -> codes and (s, b) copied; FP32 in both -> copied; quantised only
 * in `from` -> decompressed into resid_to (fma(s, Vt, b)); quantised only in `to` -> quantised from
 * its FP32 values with a fresh (s, b) fit, exactly as omc_compress would.
 *   *_from  device, state under `from`, read only.     *_to  device, state under `to`, written.
 *   workspace_to  device, `to`'s workspace (prepared).  The two states must not overlap.
 * Formats without a compiled specialisation return OMC_ERR_BAD_FORMAT.
 */
int omc_transition(const omc_plan_t *from, const omc_plan_t *to, const uint8_t *packed_from,
                   const float *resid_from, const float *sb_from, uint8_t *packed_to, float *resid_to,
                   float *sb_to, void *workspace_to, void *stream);

/*
 * omc_aggregate -- server-side aggregation of client replicas (Sec. 1: the trained client models
 * are transported back, in compressed form, and aggregated; Sec. 2.5: each client quantises its
 * own subset, so for every parameter some clients deliver full-precision values).
 * out[e] = (x_0[e] + x_1[e] + ... + x_{K-1}[e]) / K in FP32, the clients added in index order and
 * one correctly rounded division at the end, where x_k[e] is client k's decompressed value
 * fma(s_k, Vt_k, b_k) if k quantised the variable and its FP32 value otherwise.
 *   plans[K]   host array: each client's prepared plan (same variables and format, own selection).
 *   packed[K], resid[K], sb[K]   host arrays of device pointers: each client's state, read only.
 *   out        device, full layout, written (the padding after each variable with zeros).
 *   1 <= K <= 16 (else OMC_ERR_INVALID_ARG).
 * The kernel streams the codes through shared memory with bounded waits like the other calls; one
 * that runs out sets the status word of plans[0] (omc_plan_status).
 * Formats without a compiled specialisation return OMC_ERR_BAD_FORMAT.
 */
int omc_aggregate(const omc_plan_t *const *plans, uint32_t n_clients, const uint8_t *const *packed,
                  const float *const *resid, const float *const *sb, float *out, void *stream);

/*
 * omc_aggregate_sum / omc_divide -- the same aggregation (Sec. 1, Sec. 2.5) when the clients'
 * models sit on several GPUs.  Each GPU adds up its own clients with omc_aggregate_sum
 * (out[e] = x_0[e] + ... + x_{K-1}[e], FP32, its clients in index order, no division; arguments
 * as for omc_aggregate), the per-GPU sums are added across GPUs by the caller's collective (one
 * all-reduce over `out`, which every GPU owns a full copy of: this library hands no memory of
 * another GPU to any kernel), and omc_divide turns the total into the mean: values[e] /= divisor,
 * one correctly rounded FP32 division, over a buffer in the plan's full layout (1 <= divisor <=
 * 2^24: the total number of clients).  The order in which a collective adds the per-GPU sums is
 * not defined, so with three or more GPUs the result can differ from omc_aggregate over all
 * clients in the last bits: by at most (K - 1) * 2^-24 * sum_k |x_k[e]| / K for K clients.
 */
int omc_aggregate_sum(const omc_plan_t *const *plans, uint32_t n_clients, const uint8_t *const *packed,
                      const float *const *resid, const float *const *sb, float *out, void *stream);
int omc_divide(const omc_plan_t *plan, float *values, uint32_t divisor, void *stream);

/*
 * omc_aggregate_add -- more clients than one call takes (a round of the paper's experiments has
 * more than 16, Sec. 3.1): out[e] = out[e] + x_0[e] + ... + x_{K-1}[e], FP32, starting from what
 * `out` holds and adding this call's clients in index order (arguments as for omc_aggregate_sum;
 * `out` is read and written; the padding after each variable is written with zeros).
 * omc_aggregate_sum over the first batch of clients, omc_aggregate_add over each further batch
 * and omc_divide by the number of all clients make exactly the additions, in exactly the order,
 * of one omc_aggregate over all of them: the result is the same bit for bit.
 */
int omc_aggregate_add(const omc_plan_t *const *plans, uint32_t n_clients, const uint8_t *const *packed,
                      const float *const *resid, const float *const *sb, float *out, void *stream);

/*
 * omc_matmul -- forward path of Fig. 1 with the decompression fused into the consumer (Sec. 2.1:
 * a layer's parameters are decompressed only when the layer needs them; here they never exist in
 * FP32 at all).  For variable `var` of the plan, read as an N x K matrix W (K contiguous):
 *     Y = X * Wbar^T,  Wbar = s*Wt + b (Sec. 2.3),  computed as  s * (X * Wt^T) + b * rowsum(X)
 * with X and the codes as FP16 operands of the tensor cores and FP32 accumulation (the paper
 * leaves the precision of the layer arithmetic open: full precision or a format the hardware supports).
 *   S1E5M10 (the codes are IEEE halves and feed the tensor cores as they are); S1E5M6, S1E5M2,
 *   S1E4M3 and S1E2M3 (every value of these formats is an FP16 value: the codes are expanded to
 *   halves inside the kernel, on the way into the operand tile; Inf and NaN codes included); other
 *   S1E3M7 (Table 2), S1E3M9, S1E4M8 and S1E5M7 (Sec. 3.5.3) the same way, with K % 128 == 0 (a row
 *   of 11-, 13- or 19-bit codes must be whole 16-byte units for the bulk tensor copies); S1E4M14
 *   (Table 1) has 15 significant bits, more than FP16 holds, so each weight enters as two FP16
 *   terms whose sum is the weight exactly and every K step makes two products into the same FP32
 *   accumulator.  Of the fixed-point variant S1I0F7 and S1I0F11 (every value is an FP16 value)
 *   and S1I0F15 (two FP16 terms per weight, like S1E4M14).  Other formats return
 *   OMC_ERR_BAD_FORMAT; for those, omc_decompress the variable and multiply.
 *   var must be quantised and N*K == its numel; N % 128 == 0, K % 64 == 0 (else OMC_ERR_INVALID_ARG).
 *   packed, sb      device, the model state (read only).
 *   x_half          device, M x K IEEE halves, K contiguous, 16-byte aligned.
 *   y               device, M x N floats, written.       rowsum_scratch  device, M floats, written.
 */
int omc_matmul(const omc_plan_t *plan, uint32_t var, const uint8_t *packed, const float *sb, const void *x_half,
               uint32_t M, uint32_t N, uint32_t K, float *y, float *rowsum_scratch, void *stream);

/*
 * omc_compress_var_static -- compress ONE variable without a plan, a workspace or any allocation.
 * (The paper has no counterpart: this is a convenience of this library, not part of the method.)
 *
 * For code that must not allocate device memory when it needs a variable compressed: a callback
 * running while another framework owns the device's memory pool, a real-time or
 * fragmentation-sensitive service whose buffers are all reserved at start-up, or a plug-in that is
 * handed its input and output buffers and nothing else.  Such a caller cannot use omc_compress,
 * because omc_plan_prepare allocates the plan's device table and the caller would have to provide a
 * workspace.  Here the table entry, the ticket, the status word, the division of the work into
 * runs and the per-run partial sums of the Sec. 2.3 fit live in a fixed 246,024-byte array inside
 * the library's device image (every GPU that loads the library carries it until the process ends).
 * The function calls no cudaMalloc, cudaFree or other allocating routine; the result is
 * bit-identical to omc_compress on a one-variable plan.
 *
 *   values  device, numel floats (readable up to the next multiple of 4), 16-byte aligned.
 *   numel   1 .. OMC_STATIC_MAX_NUMEL; anything larger returns OMC_ERR_TOO_LARGE and does nothing.
 *   fmt     as for omc_plan.      flags   0 or OMC_PLAN_PVT (without it s = 1, b = 0 are written).
 *   packed  device, roundup16(ceil(numel*B/8)) bytes, 16-byte aligned; written, padding zeroed.
 *   sb      device, 2 floats (s, b), 8-byte aligned; written.
 *
 * The first call on a device looks up the array's address on that device (with that device
 * current; safe when several host threads make it at once); make that first call outside any
 * stream capture.  All calls share the one array, which keeps the previous call's contents: each
 * call queues a small kernel on `stream` that rewrites the table entry and the division and clears
 * the counters, then the compression kernel (two launches, no copies from host memory), so
 * back-to-back calls on one stream are fine, but two calls whose work overlaps on the same GPU
 * (different streams or host threads) race on the array and give wrong results.  Asynchronous like
 * the other device calls.
 */
#define OMC_STATIC_MAX_NUMEL (1ull << 28)
int omc_compress_var_static(const float *values, uint64_t numel, omc_format_t fmt, uint32_t flags,
                            uint8_t *packed, float *sb, void *stream);
/*
 * omc_static_status -- the status word of omc_compress_var_static on the current device (it lives
 * in the same fixed array, so no plan can report it; the paper has no counterpart either).  Waits
 * for `stream`, then writes to *host_status (host) 0 if the most recent call's kernel ran to
 * completion, non-zero if it gave up waiting for one of its own copies (its outputs are then
 * incomplete).  Each call of omc_compress_var_static clears the word, so ask before the next one.
 * Allocates nothing.
 */
int omc_static_status(void *stream, uint32_t *host_status);

#ifdef __cplusplus
}
#endif
#endif /* OMC_H_ */
