/*
 * nb_linear: dense bf16 linear layers, forward and backward, for NVIDIA B200 (sm_100a).
 *
 * The calls below are the part of a GPT-2 124M training step that takes most of its
 * time: the QKV, attention-output, MLP fc (+GELU), MLP projection and tied lm_head
 * products, forward and backward (paper: Results/Speed, the stage table, the row of
 * the matrix products; layer shapes in Method/Model and Figure 1). The library
 * follows the paper's description of a C ABI that bindings in any language compose
 * from, with return codes that tell a malformed request from a failed execution
 * (paper: The stack under test).
 *
 * Conventions for every call
 *  - Every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned,
 *    row-major and dense. The library never frees or keeps caller memory.
 *  - Activations, weights, biases and activation gradients are bf16. Weight and bias
 *    gradients are fp32 (paper: Method/Optimisation and precision). Products are
 *    accumulated in fp32 on the tensor cores; each bf16 result is rounded once,
 *    round-to-nearest-even.
 *  - Shapes: inp [BT, C], weight [OC, C], bias [OC], out / dout [BT, OC]
 *    ([BT, OC/2] for SwiGLU), pre_act [BT, OC], dinp [BT, C], dweight [OC, C],
 *    dbias [OC]. C and OC must be multiples of 8 (OC/2 a multiple of 8 for SwiGLU);
 *    BT is arbitrary. Dimensions must be below 2^31 and BT*OC, BT*C below 2^40.
 *  - Calls are asynchronous on a CUDA stream: the `_ex` forms take it as an argument
 *    (a cudaStream_t passed as void*), the short forms use the stream last given to
 *    nb_set_stream on the calling thread (default: the legacy default stream).
 *  - Return value: NB_OK or an NB_ERR_* code; nb_last_error() gives the text for the
 *    calling thread. NB_ERR_INVALID_ARG and NB_ERR_UNSUPPORTED are malformed requests
 *    and launch nothing. NB_ERR_CUDA is a driver / launch failure. NB_ERR_TIMEOUT is
 *    reported by nb_check_status when a kernel gave up on a bounded wait.
 *  - The library keeps a grow-only device workspace, a 64-byte device status word per
 *    device and a host-side cache of TMA descriptors. Two kinds of call use the
 *    workspace: backward calls that apply this layer's own activation derivative
 *    (act != NB_ACT_NONE: dz is formed there) and nb_lm_head_ce_forward (its softmax
 *    partials). There is ONE workspace per device, so such calls must be ordered with
 *    respect to each other: issue them on one stream, or order the streams with
 *    events; two of them running at the same time overwrite each other's data. Growing
 *    the workspace synchronises the device and frees the old one, which is not allowed
 *    while a stream is being captured into a CUDA graph: size it first with
 *    nb_workspace_reserve (a call that would have to grow it during a capture returns
 *    NB_ERR_UNSUPPORTED and launches nothing).
 */
#ifndef NB_LINEAR_H
#define NB_LINEAR_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NB_OK 0
#define NB_ERR_INVALID_ARG 1 /* null / misaligned pointer, negative size, bad enum */
#define NB_ERR_UNSUPPORTED 2 /* shape outside the constraints above */
#define NB_ERR_CUDA 3        /* CUDA driver or launch failure */
#define NB_ERR_TIMEOUT 4     /* a device-side bounded wait expired */

#define NB_ACT_NONE 0
#define NB_ACT_GELU 1   /* tanh form: 0.5 z (1 + tanh(sqrt(2/pi)(z + 0.044715 z^3))) */
#define NB_ACT_SWIGLU 2 /* weight rows [0,H) gate, [H,2H) up; out = silu(gate) * up */

#define NB_DTYPE_F32 0
#define NB_DTYPE_BF16 1

/* Library version as major*10000 + minor*100 + patch. */
int nb_version(void);

/* Text of the last error on the calling thread ("" if none). Never NULL. */
const char *nb_last_error(void);

/* Stream used by the short-form calls on this thread (a cudaStream_t; NULL = default). */
int nb_set_stream(void *stream);
void *nb_get_stream(void);

/*
 * Number of bf16 elements the `out` argument of nb_linear_forward must hold:
 * BT*OC for NB_ACT_NONE; BT*OC (activated plane) + BT*OC (pre-activation plane) for
 * NB_ACT_GELU; BT*OC/2 + BT*OC for NB_ACT_SWIGLU. Returns -1 on a bad argument.
 */
int64_t nb_linear_out_elems(int64_t BT, int64_t OC, int act);

/*
 * Forward: z = inp . weight^T (+ bias); out = act(z).
 * (paper: Figure 1, the MLP box of a block and the head box: the head is tied to the
 * token embedding and has no bias)
 *
 *   out     [out] act == NONE : [BT, OC] bf16.
 *                 act != NONE : two planes back to back, the activated result first
 *                 ([BT, OC], or [BT, OC/2] for SwiGLU) and then the pre-activation z
 *                 [BT, OC], which backward needs. Size: nb_linear_out_elems().
 *   inp     [in]  [BT, C] bf16
 *   weight  [in]  [OC, C] bf16
 *   bias    [in]  [OC] bf16 or NULL
 *   act           NB_ACT_*
 * BT == 0 is accepted and does nothing.
 */
int nb_linear_forward(void *out, const void *inp, const void *weight, const void *bias,
                      int64_t BT, int64_t C, int64_t OC, int act);

/*
 * Forward with the pre-activation plane and the stream given explicitly.
 * pre_act: [BT, OC] bf16, required and written when act != NONE, ignored for
 * act == NONE. nb_linear_forward wraps this call.
 */
int nb_linear_forward_ex(void *out, void *pre_act, const void *inp, const void *weight,
                         const void *bias, int64_t BT, int64_t C, int64_t OC, int act,
                         void *stream);

/*
 * Backward of one layer (paper: Method/Optimisation and precision for the fp32
 * gradients; Method/Batch geometry for accumulation over micro-steps).
 *
 *   dz      = dout                      when pre_act == NULL
 *           = dout * gelu'(pre_act)     when pre_act != NULL (this layer's own
 *                                       pre-activation [BT, OC]; tanh-GELU)
 *   dinp    [out] [BT, C] bf16  = dz . weight              always overwritten
 *   dweight [i/o] [OC, C] fp32 (+)= dz^T . inp
 *   dbias   [i/o] [OC]    fp32 (+)= column sums of dz
 *   accumulate    0: dweight and dbias are overwritten (they need not be zeroed);
 *                 non-zero: the new gradient is added to what they hold.
 * Any of dinp, dweight, dbias may be NULL; that product is skipped (frozen weights).
 * inp may be NULL when dweight is NULL; weight may be NULL when dinp is NULL.
 * BT == 0: dinp untouched, dweight/dbias zeroed when accumulate == 0.
 *
 * When pre_act != NULL, dz is first written to the library's device workspace
 * (BT*OC bf16, allocated on first need with cudaMalloc and kept). When both dweight
 * and dbias are requested, the bias gradient is summed inside the wgrad kernel from the
 * dz tiles it already holds in shared memory. Summation order of dweight/dbias across
 * row blocks is not fixed (split-K reduce-adds, atomics), so results may differ in the
 * last bits between runs.
 */
int nb_linear_backward(void *dinp, void *dweight, void *dbias, const void *dout,
                       const void *inp, const void *weight, const void *pre_act, int64_t BT,
                       int64_t C, int64_t OC, int accumulate);

/*
 * Backward, general form.
 *   act           activation of THIS layer, applied through pre_act (required when
 *                 act != NONE): GELU as above; SWIGLU with dout [BT, OC/2] and
 *                 pre_act [BT, OC] = [gate | up]:
 *                   dz[:, j]     = dout[:, j] * up_j * silu'(gate_j)
 *                   dz[:, H + j] = dout[:, j] * silu(gate_j)
 *   inp_pre_act   NULL, or [BT, C] bf16: the pre-activation of the GELU layer that
 *                 produced `inp`. Then dinp = (dz . weight) * gelu'(inp_pre_act), i.e.
 *                 the dz of that producer, applied in the dgrad epilogue in fp32
 *                 before the single rounding to bf16 (the activation backward the
 *                 paper's stack launches as a separate kernel, fused here).
 *   dweight_dtype NB_DTYPE_F32 (the paper's arrangement). NB_DTYPE_BF16 is accepted
 *                 only with accumulate == 0.
 *   stream        cudaStream_t as void*.
 */
int nb_linear_backward_ex(void *dinp, void *dweight, void *dbias, const void *dout,
                          const void *inp, const void *weight, const void *pre_act,
                          const void *inp_pre_act, int64_t BT, int64_t C, int64_t OC, int act,
                          int accumulate, int dweight_dtype, void *stream);

/*
 * Stand-alone column reduction: dbias[o] (+)= sum over rows of dout[m, o].
 * dout [BT, OC] bf16, dbias [OC] fp32, OC a multiple of 8. Uses the stream of
 * nb_set_stream. (The bias gradient of every biased layer; paper: Method/Model lists
 * the biased linears through the parameter count.)
 */
int nb_reduce_dbias(void *dbias, const void *dout, int64_t BT, int64_t OC, int accumulate);

/*
 * Head with fused cross-entropy statistics (paper: Figure 1, the loss box: the loss covers only
 * the real vocabulary, the padding takes no part in it and receives no gradient, and it is
 * computed in 32-bit; Results/Speed lists the cross-entropy forward and backward as separate
 * kernels next to the head's GEMMs).
 *
 * nb_lm_head_ce_forward: logits = inp . weight^T (bf16, [BT, Vp], stored as by nb_linear_forward),
 * and, in the same pass, from the stored (rounded) logits of the first V columns:
 *     lse[i]  = log sum_{j < V} exp(logits[i, j])          fp32 [BT]
 *     loss[i] = lse[i] - logits[i, targets[i]]             fp32 [BT]
 * The GEMM epilogue keeps per-row (max, sum of exp) per column tile; a small second kernel
 * combines them, so the logits are never re-read for the softmax normaliser. targets: int32
 * [BT] on the device, each in [0, V); an out-of-range target yields NaN in loss[i]. Vp and C
 * multiples of 8, 0 < V <= Vp. Uses the library workspace (BT * 2*ceil(Vp/256) * 8 bytes).
 *
 * nb_ce_backward: dlogits[i, j] = gscale * (exp(logits[i, j] - lse[i]) - [j == targets[i]]) for
 * j < V and 0 for j >= V, bf16 [BT, Vp]; dlogits may be the logits buffer itself (in place). Its
 * result is the `dout` of nb_linear_backward for the head. gscale is the upstream gradient of
 * every row's loss (1/BT for a mean over the micro-batch, times 1/accumulation steps).
 */
int nb_lm_head_ce_forward(void *logits, void *loss, void *lse, const void *inp, const void *weight,
                          const void *targets, int64_t BT, int64_t C, int64_t Vp, int64_t V,
                          void *stream);
int nb_ce_backward(void *dlogits, const void *logits, const void *lse, const void *targets,
                   float gscale, int64_t BT, int64_t Vp, int64_t V, void *stream);

/*
 * Low-rank adapter beside a frozen linear layer (paper: Method/The clinical stage: rank-16
 * adapters with rank-stabilised scaling on the projections of Qwen3-0.6B, base weights frozen).
 *
 * nb_lora_linear_forward:
 *     t   = bf16( scale * inp . lora_a^T )                      [BT, r]   lora_a [r, C]
 *     out = inp . weight^T (+ bias) + t . lora_b^T              [BT, OC]  lora_b [OC, r]
 * The second line is ONE GEMM: the r columns of t and lora_b are appended to the K range of the
 * base product, so the adapter costs one extra k-block in the accumulator, no extra pass over out.
 * t is an output (bf16, kept for backward). scale is alpha / sqrt(r) (rank-stabilised) or
 * alpha / r; r a multiple of 8 in [8, 64].
 *
 * nb_lora_linear_backward (weight frozen: no dweight):
 *     u       = bf16( scale * dout . lora_b )                   [BT, r]   caller-provided scratch
 *     dinp    = dout . weight + u . lora_a                      [BT, C]   one GEMM, K extended by r
 *     dlora_b (+)= dout^T . t                                   [OC, r]   fp32
 *     dlora_a (+)= u^T . inp                                    [r, C]    fp32
 * dinp, dlora_a, dlora_b may be NULL (skipped); accumulate as in nb_linear_backward. t and u are
 * rounded to bf16 once each (they are tensor-core operands); everything else follows the
 * conventions at the top of this file. When dlora_b is asked for, u and dlora_b come out of one
 * kernel that reads dout once (both products are bound by that read); when dlora_a is asked for
 * as well, the same launch also reads inp once and forms dlora_a. Both gradients are summed by
 * reduce-adds of per-row-panel partial sums, in no fixed order.
 *
 * Projections that share an input and are laid out as one layer (a qkv or a gate_up projection:
 * weights stacked by rows) can use these two calls as they are, with r = the sum of the members'
 * ranks (<= 64): lora_a = the members' A matrices stacked by rows, lora_b [sum of OC, r] = their B
 * matrices as diagonal blocks and zeros elsewhere. Every member's columns of out, its rows of
 * dlora_a and its diagonal block of dlora_b then equal what the member alone would give, dinp is
 * the sum of the members' input gradients, and the other blocks of dlora_b hold values that belong
 * to no parameter.
 */
int nb_lora_linear_forward(void *out, void *t, const void *inp, const void *weight, const void *bias,
                           const void *lora_a, const void *lora_b, float scale, int64_t BT,
                           int64_t C, int64_t OC, int64_t r, void *stream);
int nb_lora_linear_backward(void *dinp, void *dlora_a, void *dlora_b, void *u, const void *dout,
                            const void *inp, const void *weight, const void *lora_a,
                            const void *lora_b, const void *t, float scale, int64_t BT, int64_t C,
                            int64_t OC, int64_t r, int accumulate, void *stream);

/*
 * Adapters that share an input, stacked (paper: Method/The clinical stage: the query, key and value
 * projections of a layer read the same activations, and so do the gate and up projections; each of
 * the seven projections has its own rank-16 adapter). Stacking the A matrices of such a group row
 * by row gives one rank-R product for the whole group instead of one skinny product per adapter,
 * and the input is read once:
 *
 *   nb_lora_down_stacked:            t_stack = bf16( scale * inp . a_stack^T )   [BT, R]
 *                                    a_stack [R, C] = the groups' A matrices one after the other
 *   nb_lora_linear_forward_stacked:  out = inp . weight^T (+ bias) + t_stack[:, off:off+r] . lora_b^T
 *                                    (one GEMM, as in nb_lora_linear_forward; t_stack is an input)
 *   nb_lora_linear_backward_stacked: u_stack[:, off:off+r] = bf16( scale * dout . lora_b )
 *                                    dinp    = dout . weight + u_stack[:, off:off+r] . lora_a
 *                                    dlora_b (+)= dout^T . t_stack[:, off:off+r]       [OC, r] fp32
 *                                    (lora_a [r, C] is this adapter's rows of a_stack; dinp and dlora_b
 *                                    may be NULL; the gradient of A is NOT formed here)
 *   nb_lora_da_stacked:              da_stack (+)= u_stack^T . inp                    [R, C] fp32
 *                                    once per group, after the backward calls of all its members have
 *                                    filled their columns of u_stack; rows [off, off+r) are that
 *                                    adapter's dlora_a
 *
 * r and off are multiples of 8, off + r <= R <= 64, R a multiple of 8. Column slices of t_stack and
 * u_stack are addressed in place (row stride R); columns outside a slice are neither read into a
 * product nor written. Every result equals what the unstacked calls give for that adapter; rounding
 * points and all other conventions are those of nb_lora_linear_forward / _backward.
 */
int nb_lora_down_stacked(void *t_stack, const void *inp, const void *a_stack, float scale, int64_t BT,
                         int64_t C, int64_t R, void *stream);
int nb_lora_linear_forward_stacked(void *out, const void *inp, const void *weight, const void *bias,
                                   const void *t_stack, const void *lora_b, int64_t BT, int64_t C,
                                   int64_t OC, int64_t r, int64_t R, int64_t off, void *stream);
int nb_lora_linear_backward_stacked(void *dinp, void *dlora_b, void *u_stack, const void *dout,
                                    const void *weight, const void *lora_a, const void *lora_b,
                                    const void *t_stack, float scale, int64_t BT, int64_t C, int64_t OC,
                                    int64_t r, int64_t R, int64_t off, int accumulate, void *stream);
int nb_lora_da_stacked(void *da_stack, const void *u_stack, const void *inp, int64_t BT, int64_t C,
                       int64_t R, int accumulate, void *stream);

/*
 * Master-weight cast: dst[i] = bf16(src[i]), round to nearest even, for n elements.
 * (paper: Method/Optimisation and precision keeps fp32 master weights and bf16 compute copies;
 * Results/Speed, the table of levers: the cast is done once per optimizer step and reused by
 * every micro-step.) src fp32 and dst bf16 are device pointers, 16-byte aligned; n >= 0.
 * Infinities are kept, values beyond the largest finite bf16 round to infinity, NaN stays NaN.
 */
int nb_cast_f32_to_bf16(void *dst, const void *src, int64_t n, void *stream);

/*
 * Bias gradient of a GELU layer without any allocation (the paper has no counterpart; this
 * exists for callers that must not allocate device memory):
 *
 *     dbias[o] (+)= sum over rows m of  dout[m, o] * gelu'(pre_act[m, o])
 *
 * It computes what nb_linear_backward_ex computes for `dbias` when it is given `pre_act`
 * and NB_ACT_GELU, but where that call keeps dz = dout * gelu'(pre_act) in a workspace it
 * obtains with cudaMalloc, this one keeps dz in a fixed array compiled into the library
 * image (NB_NOALLOC_MAX_ELEMS bf16 elements, 8 MiB, resident on every GPU that loads the
 * library until the process exits). Who needs it: code that runs where cudaMalloc is
 * forbidden or unsafe, for example between other libraries' timing-critical sections, in
 * processes whose device memory is fully handed to another allocator, or inside a service
 * that promised its host a fixed footprint.
 *
 *   dbias   [i/o] [OC] fp32, device, 16-byte aligned; overwritten when accumulate == 0
 *   dout    [in]  [BT, OC] bf16, device, 16-byte aligned
 *   pre_act [in]  [BT, OC] bf16, device, 16-byte aligned
 *   stream        cudaStream_t as void*
 * Limits and errors: OC a multiple of 8; BT*OC must not exceed NB_NOALLOC_MAX_ELEMS,
 * otherwise NB_ERR_UNSUPPORTED with a message naming the limit (nothing is launched).
 * The call uses no cudaMalloc / cudaFree and no allocating library routine. The first call
 * on each device looks up the device address of the built-in array (one
 * cudaGetSymbolAddress, with that device current); make that first call before starting any
 * stream capture.
 * The array is shared by every call on the device and keeps what the last call wrote. Each
 * call overwrites the part it uses before reading it, so nothing has to start at zero; but
 * two calls whose kernels may overlap on the GPU (different streams, no ordering between
 * them) race on it and must be serialised by the caller.
 */
#define NB_NOALLOC_MAX_ELEMS 4194304
int nb_gelu_dbias_noalloc(void *dbias, const void *dout, const void *pre_act, int64_t BT,
                          int64_t OC, int accumulate, void *stream);

/*
 * Make sure the workspace holds at least `bytes` (so later calls do not allocate), or
 * release everything the library holds on the current device (workspace, status word,
 * descriptor cache) with nb_release.
 */
int nb_workspace_reserve(int64_t bytes);
int nb_release(void);

/*
 * Synchronise the current device and report whether any kernel since the last check
 * gave up on a bounded wait (NB_ERR_TIMEOUT, detail in nb_last_error) or a CUDA error is
 * pending (NB_ERR_CUDA). Clears the device status word.
 */
int nb_check_status(void);

/*
 * Number of kernels this library has launched from the calling process since it was
 * loaded (memsets issued through the CUDA runtime are not counted).
 */
int64_t nb_kernel_launches(void);

/*
 * Host-only view of how a wgrad of shape dweight[M, N] = sum over K rows is cut into work units
 * (no device is touched): out[0] = row tiles, out[1] = column tiles, out[2] = split-K factor,
 * out[3] = 64-row k-blocks per split, out[4] = k-blocks in total. `tile_m` is 128 or 256 (CTA
 * pair), `slots` the number of tiles resident at once (SMs, or SM pairs). Unit u covers k-blocks
 * [s*out[3], min((s+1)*out[3], out[4])) of tile t, with s = u / (out[0]*out[1]), t = u % (...).
 */
int nb_debug_split_plan(int64_t M, int64_t N, int64_t K, int slots, int tile_m, int *out);

/*
 * Host-only view of how nb_linear_backward_ex schedules a layer whose dinp and fp32 dweight are
 * both requested (BT > 128): one persistent launch whose CTA pairs each walk a list of work units,
 * 256 x 256 tiles of dinp over all of K = OC and 256 x 256 tiles of dweight over ranges of 64-row
 * k-blocks of K = BT (paper: Results/Speed, stage table, the GEMM row: this is its backward half
 * for one layer). No device is touched. `pairs` is the number of CTA pairs (SM count / 2),
 * `gelu_grad` whether the producer's GELU derivative is applied in the dinp epilogue (it makes
 * those units dearer in the balance). out[0..7] = dinp row tiles, dinp column tiles, k-blocks of
 * a dinp tile, dweight row tiles, dweight column tiles, k-blocks of K = BT, k-blocks per dweight
 * chunk, whole rounds. Then one record of six ints per unit in execution order of each pair:
 * (pair, is_dweight, row tile, column tile, first k-block, end k-block). Returns the number of
 * records, or minus an NB_ERR_* code (buffer too small, shape the schedule does not cover).
 */
int nb_debug_layer_bwd_plan(int64_t BT, int64_t C, int64_t OC, int pairs, int gelu_grad, int *out,
                            int64_t cap);

/*
 * Self-test of the bounded-wait mechanism: launches a one-block kernel that waits, for
 * at most `limit_us` microseconds, on a barrier nothing ever signals, then returns
 * normally after recording the expiry. nb_check_status() afterwards reports
 * NB_ERR_TIMEOUT; the context stays usable.
 */
int nb_debug_wait_timeout(int64_t limit_us);

/*
 * Self-test of the GEMM kernel's own time-out exit (paper: The stack under test asks of the
 * surface that a failed execution is told apart from a malformed request; this is how the
 * former is exercised without a fault): a one-tile, one-CTA forward product
 * out[128, 256] = inp[128, 256] . weight[256, 256]^T in which the producer warp stops after two
 * of the four k-blocks. The MMA issuer's bounded wait for the third stage runs out after
 * `limit_us` microseconds (100 .. 1000000), it records the event in the device status word, the
 * other roles see the abort flag, and every thread leaves through the kernel's common exit
 * (wait for copies in flight, free tensor memory). `out` is left unwritten. Afterwards
 * nb_check_status() reports NB_ERR_TIMEOUT naming wait 300 + stage; the context stays usable.
 * All three pointers are device pointers, 16-byte aligned, bf16, dense row-major.
 */
int nb_debug_gemm_timeout(void *out, const void *inp, const void *weight, int64_t limit_us);

#ifdef __cplusplus
}
#endif
#endif /* NB_LINEAR_H */
