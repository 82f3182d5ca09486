/*
 * dig_gla.h -- C ABI of the B200 (sm_100a) library for the hot path of DiG's token mixer
 * (arxiv 2405.18428): gated linear attention over 2-D patch grids in four scan orders,
 * forward and backward, plus the 3x3 depthwise convolution of the SREM module.
 *
 * Conventions shared by every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned, dense,
 *     with no aliasing between inputs and outputs.  `tau_per_head` and every size are host
 *     values.  `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - Token tensors are [B][L][H][d], L = grid_h*grid_w, canonical token index y*grid_w + x
 *     (the row-major flattening of the patch grid, i.e. the (B, T, D) sequence of Algorithm 1
 *     split into H heads).  Results are written at canonical positions for every direction.
 *   - Calls only enqueue work on the given stream; they do not synchronise and allocate no
 *     device memory.  Scratch memory is a caller-provided workspace (dig_gla_fwd_static alone
 *     keeps its scratch in an array of the library image).
 *   - Errors are return codes.  Arguments are validated on the host before any launch; after a
 *     non-zero return the outputs are unspecified.  Nothing traps, aborts or prints.
 */
#ifndef DIG_GLA_H_
#define DIG_GLA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DIG_OK = 0,
    DIG_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, non-positive size, bad enum */
    DIG_ERR_UNSUPPORTED = 2,   /* valid request outside what the kernels cover */
    DIG_ERR_WORKSPACE = 3,     /* workspace missing or smaller than dig_gla_workspace_bytes */
    DIG_ERR_CUDA = 4,          /* a CUDA runtime call failed (launch, attribute, ...) */
    DIG_ERR_TIMEOUT = 5,       /* a bounded device-side wait gave up (see dig_last_device_status) */
    DIG_ERR_SCRATCH_LIMIT = 6, /* dig_gla_fwd_static: the problem needs more than its built-in scratch */
    DIG_ERR_RANGE = 7          /* gates decay faster than the kernels can represent (see dig_gla_fwd, dig_last_device_status) */
} dig_status;

/* Storage type of q, k, v, out, d_out, dq, dk, dv, x, y, w, bias.  Gates are always fp32.
 *   DIG_F32          fp32 storage, fp32 FMA arithmetic.
 *   DIG_BF16         bf16 storage in and out; products on the tensor cores with operands
 *                    carried at 11 significant bits (fp16 tiles in the tcgen05 kernels, tf32 in
 *                    the warp-level ones) and fp32 accumulation; outputs rounded to nearest-even
 *                    bf16.
 *   DIG_BF16_F32OUT  as DIG_BF16 but out / dq / dk / dv are stored as fp32 (the unrounded
 *                    accumulators).  DIG_BF16 results equal these rounded to bf16, bit for bit. */
typedef enum { DIG_F32 = 0, DIG_BF16 = 1, DIG_BF16_F32OUT = 2 } dig_dtype;

/* Scan order of the token grid (Algorithm 1 / Algorithm 4: the orders reached by alternating
 * "flip" and "transpose" of the reshaped token matrix block by block). */
typedef enum { DIG_ROW_FWD = 0, DIG_ROW_REV = 1, DIG_COL_FWD = 2, DIG_COL_REV = 3 } dig_dir;

/* Which kernel family serves a call.  AUTO picks the tcgen05 tensor-core kernels (TENSOR) when they
 * cover the request (bf16 storage, d_k = d_v = 64 or 72, any chunk size), else the warp-level
 * tensor-core kernels (MMA: bf16 storage, any supported head and chunk size that fits shared
 * memory), else the fp32-FMA kernels (fp32 storage, whose products must be fp32-accurate).  Forcing
 * a family that does not cover the request returns DIG_ERR_UNSUPPORTED.  Process-wide; meant for
 * tests and benchmarks. */
typedef enum { DIG_IMPL_AUTO = 0, DIG_IMPL_FMA = 1, DIG_IMPL_TENSOR = 2, DIG_IMPL_MMA = 3 } dig_impl;
dig_status dig_set_impl(int impl);
/* The family the next call with these parameters would use (DIG_IMPL_FMA, _TENSOR or _MMA),
 * or a negative dig_status if no family covers it. */
int dig_gla_query_impl(int d_k, int d_v, int chunk, int dtype, int backward);

/* Bytes of workspace dig_gla_fwd (backward = 0) or dig_gla_bwd (backward = 1) needs.
 * Returns 0 for invalid arguments. */
size_t dig_gla_workspace_bytes(int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk,
                               int dtype, int backward);

/* Gate transform (Eq. gate_gla, key-channel gate alpha = sigmoid(x)^(1/tau)) in log space:
 *   gate[b,l,h,c] = log(alpha) = logsigmoid(g[b,l,h,c]) / tau_per_head[h]
 * g: [B][L][H][d_k] in `dtype` storage (bf16 for both DIG_BF16 variants); tau_per_head: HOST array
 * of H positive floats; gate: fp32 [B][L][H][d_k]. */
dig_status dig_gate_logsigmoid(const void *g, const float *tau_per_head, float *gate,
                               int B, int L, int H, int d_k, int dtype, void *cuda_stream);

/* Gated linear attention, forward (Eq. attn_gla with the value-channel gate fixed to 1):
 *   S_t = diag(exp(gate_t)) S_{t-1} + k_t^T v_t,  S before the first token = 0,
 *   out_t = q_t S_t,
 * t running over the grid in `direction`, independently per (batch, head).  Evaluated chunk by
 * chunk (Section 3.5: chunks of `chunk` tokens worked in on-chip memory); the result does not
 * depend on `chunk` beyond rounding.  No 1/sqrt(d) scaling and no normaliser are applied.
 *   q, k, gate: [B][L][H][d_k]; v, out: [B][L][H][d_v]; gate is log(alpha) <= 0, fp32.
 *   d_k, d_v: multiples of 8, 8..128; chunk in {16, 32, 64, 128}; L need not be a multiple of chunk.
 * The tcgen05 kernels work on 64-token tiles whatever `chunk` is: a shorter chunk is worked as sub-chunks
 * of a tile, a longer one as 64 (dig_gla_query_impl tells which family serves a request).
 * Range of the gates.  The in-chunk decay is formed as exp(+-cumulative gate).  The tcgen05 kernels keep
 * the decayed operands in fp16 around the centre of a (sub-)chunk: where the gates of a 64-token tile sum
 * to more than 15.9 in magnitude (any channel) the tile is worked in sub-chunks of 32, 16 or 8 tokens, so
 * results stay exact for any decay up to 15.9 per 8 consecutive scan positions (log alpha about -2 per
 * token).  Beyond that the call still completes with finite values, which are not the result, and
 * dig_last_device_status reports DIG_ERR_RANGE.  The other families form exp(+-sum) in fp32 / tf32: there
 * the magnitude of the gate summed over one chunk must stay below 80; beyond it results may overflow.
 * Sigmoid gates with temperature >= 1 are inside both ranges with a wide margin. */
dig_status dig_gla_fwd(const void *q, const void *k, const void *v, const float *gate, void *out,
                       int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk,
                       int direction, int dtype, void *workspace, size_t workspace_bytes,
                       void *cuda_stream);

/* Forward GLA without any allocation (the paper has no counterpart; this is a packaging variant
 * of dig_gla_fwd, same arguments minus the workspace, same results bit for bit).
 *
 * Who it is for: callers that cannot obtain device memory at call time -- a host application that
 * owns every byte of the GPU and hands plugins only their inputs and outputs, a latency-critical
 * loop in which cudaMalloc's implicit synchronisation is unacceptable, a process whose memory
 * budget was fixed at start-up.  For them the segment states and decay factors that dig_gla_fwd keeps
 * in the caller's workspace live in a device array of DIG_GLA_STATIC_SCRATCH_BYTES that is part of
 * the library image.  A device holds that array from the moment the CUDA runtime loads this part of
 * the library on it until the process exits: with lazy module loading (the default since CUDA 12)
 * that moment is the first dig_gla_fwd_static call on the device, whose address look-up triggers the
 * load and may take a while or fail with DIG_ERR_CUDA; with CUDA_MODULE_LOADING=EAGER it is context
 * creation.  Make that first call at start-up, outside any stream capture and outside the loop that
 * must not stall; every later call allocates and frees nothing, on the host side of CUDA or through
 * torch.
 *
 * Limit: requests for which dig_gla_workspace_bytes(..., backward = 0) exceeds
 * DIG_GLA_STATIC_SCRATCH_BYTES return DIG_ERR_SCRATCH_LIMIT before anything is launched (16 MiB
 * covers e.g. B*H = 48 sequences of 1024 tokens at d_k = d_v = 64, chunk 64).
 *
 * All calls on a device share the one array: it keeps whatever the previous call left there (the
 * kernels overwrite every entry they read, so nothing needs clearing), and two calls whose kernels
 * overlap on the GPU -- different streams, or different host threads -- race on it.  Serialise them
 * on one stream. */
#define DIG_GLA_STATIC_SCRATCH_BYTES ((size_t)16 << 20)
dig_status dig_gla_fwd_static(const void *q, const void *k, const void *v, const float *gate,
                              void *out, int B, int H, int grid_h, int grid_w, int d_k, int d_v,
                              int chunk, int direction, int dtype, void *cuda_stream);

/* Gated linear attention, backward: gradients of <d_out, out> with respect to q, k, v and gate
 * (reverse-mode derivative of Eq. attn_gla; the paper trains through the operator but does not
 * print it).  Nothing is saved by the forward call: chunk states are recomputed here.
 *   d_out: [B][L][H][d_v]; dq, dk: [B][L][H][d_k]; dv: [B][L][H][d_v]; dgate: fp32 [B][L][H][d_k].
 * The fp32-FMA and warp-level families cover chunk <= 64 here (shared memory); chunk = 128 is served by
 * the tcgen05 family only (bf16 storage, d_k = d_v = 64 or 72, 64-token tiles). */
dig_status dig_gla_bwd(const void *q, const void *k, const void *v, const float *gate,
                       const void *d_out, void *dq, void *dk, void *dv, float *dgate,
                       int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk,
                       int direction, int dtype, void *workspace, size_t workspace_bytes,
                       void *cuda_stream);

/* SREM depthwise convolution (Algorithm 1: DWConv2d(reshape2d(z)), 3x3, stride 1, zero padding 1,
 * cross-correlation, one filter per channel):
 *   y = conv3x3(z2d, w) + bias, where z2d is the token matrix of a residual stream that is
 *   currently laid out in scan order `direction`.
 * x and y are nevertheless addressed canonically, [B][grid_h*grid_w][D]; the re-orientation is
 * folded into the filter taps (reverse orders rotate the filter by 180 degrees, column orders
 * transpose it), so no permuted copy is made.
 *   w: [3][3][D]; bias: [D] or NULL; D a multiple of 8.  fp32 accumulation.
 * For DIG_BF16_F32OUT y is fp32, x / w / bias are bf16. */
dig_status dig_srem_dwconv(const void *x, const void *w, const void *bias, void *y,
                           int B, int grid_h, int grid_w, int D, int direction, int dtype,
                           void *cuda_stream);

/* Reverse mode of dig_srem_dwconv (the paper trains through the SREM module; the derivative is not
 * printed there): given dy = dL/dy, computes dx = dL/dx, dw = dL/dw and, if dbias is not NULL,
 * dbias = dL/dbias of  y = conv3x3(z2d, w) + bias  in the same scan-order convention.
 *   x, dy, dx: [B][grid_h*grid_w][D] canonical order (dx in the output storage type of `dtype`);
 *   w: [3][3][D] in the storage type; dw: fp32 [3][3][D]; dbias: fp32 [D] or NULL.
 * dx is the forward stencil run on dy in the opposite scan sense; dw and dbias are reductions over
 * all pixels, summed in a fixed order (bit-identical from run to run).  Needs a workspace of
 * dig_srem_dwconv_bwd_workspace_bytes (0 for invalid sizes) for per-slab partial sums. */
size_t dig_srem_dwconv_bwd_workspace_bytes(int B, int grid_h, int grid_w, int D);
dig_status dig_srem_dwconv_bwd(const void *x, const void *w, const void *dy, void *dx, float *dw, float *dbias,
                               int B, int grid_h, int grid_w, int D, int direction, int dtype, void *workspace,
                               size_t workspace_bytes, void *cuda_stream);

/* Output gate of the GLA layer (Eq. attn_gla, the line that forms Y_t before the projection W_O):
 *     z = Swish(r) (.) LN(o),   Swish(r) = r * sigmoid(r),
 * per row of d_v values; `rows` = B * L * H rows of the [B][L][H][d_v] tensors o (the output of
 * dig_gla_fwd), r (the gate pre-activation X W_r + b_r) and z, in the storage types of `dtype`.
 * The paper does not fix LN further; here it normalises each (token, head) row over its d_v values
 * (biased variance, `eps` added under the root) and applies an optional affine part shared by all
 * heads: ln_w, ln_b are fp32 [d_v] device arrays or NULL (weight 1 / bias 0).
 * d_v: a multiple of 8, at most 128.  fp32 arithmetic. */
dig_status dig_gla_outgate_fwd(const void *o, const void *r, const float *ln_w, const float *ln_b, void *z,
                               long long rows, int d_v, float eps, int dtype, void *cuda_stream);

/* Reverse mode of dig_gla_outgate_fwd (not printed in the paper): from dz = dL/dz computes d_o and d_r
 * (output storage type of `dtype`) and, where the pointer is not NULL, dln_w and dln_b (fp32 [d_v]; the
 * gradients at weight 1 / bias 0 where ln_w / ln_b is NULL), summed over all rows in a fixed order.
 * The workspace (dig_gla_outgate_bwd_workspace_bytes; 0 for invalid sizes) holds per-CTA partial sums
 * and is needed only when dln_w or dln_b is requested. */
size_t dig_gla_outgate_bwd_workspace_bytes(long long rows, int d_v);
dig_status dig_gla_outgate_bwd(const void *o, const void *r, const float *ln_w, const float *ln_b, const void *dz,
                               void *d_o, void *d_r, float *dln_w, float *dln_b, long long rows, int d_v, float eps,
                               int dtype, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* dig_gla_fwd / dig_gla_bwd with the state of the recurrence as an argument (the paper always starts
 * from S = 0 and drops the final state; these are what a caller needs to cut a long sequence into
 * pieces or to shard it over devices: run the pieces in scan order and chain them through the state).
 * All state tensors are fp32 [B][H][d_k][d_v] row-major device arrays; each may be NULL.
 *   s_in   state before the first token in scan order (NULL = 0)
 *   s_out  receives the state after the last token (NULL = not wanted)
 *   ds_out gradient of the loss with respect to s_out (NULL = 0)
 *   ds_in  receives the gradient with respect to s_in (NULL = not wanted)
 * dig_gla_bwd_state returns the gradients of  <d_out, out> + <ds_out, s_out>.  Workspace sizes are
 * those of dig_gla_fwd / dig_gla_bwd.  The states are kept in fp32 across the whole sequence; the
 * kernels that consume them round them to tf32 per chunk exactly as without these arguments. */
dig_status dig_gla_fwd_state(const void *q, const void *k, const void *v, const float *gate, const float *s_in,
                             void *out, float *s_out, int B, int H, int grid_h, int grid_w, int d_k, int d_v,
                             int chunk, int direction, int dtype, void *workspace, size_t workspace_bytes,
                             void *cuda_stream);
dig_status dig_gla_bwd_state(const void *q, const void *k, const void *v, const float *gate, const void *d_out,
                             const float *s_in, const float *ds_out, void *dq, void *dk, void *dv, float *dgate,
                             float *ds_in, int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk,
                             int direction, int dtype, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* dig_gla_fwd followed by the output gate of the layer, z = Swish(r) * LN(out) (dig_gla_outgate_fwd),
 * in one call.  r: gate pre-activation [B][L][H][d_v] in the input storage type of `dtype`; ln_w, ln_b:
 * fp32 [d_v] or NULL; z: [B][L][H][d_v] in the output storage type; `out` may be NULL when only z is
 * wanted (z then serves as the intermediate buffer).  LN sees `out` as it is stored (rounded to bf16 for
 * DIG_BF16).  The two steps run one after the other on the stream.  Workspace as for dig_gla_fwd. */
dig_status dig_gla_fwd_outgate(const void *q, const void *k, const void *v, const float *gate, const void *r,
                               const float *ln_w, const float *ln_b, float eps, void *out, void *z, int B, int H,
                               int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Gated linear attention with the paper's full gate G_t = alpha_t^T beta_t (Eq. gate_gla): the state
 * also decays along the value channels,
 *   S_t = diag(exp(gate_t)) S_{t-1} diag(exp(bgate_t)) + k_t^T v_t,   out_t = q_t S_t,
 * bgate = log(beta) <= 0, fp32 [B][L][H][d_v]; everything else as in dig_gla_fwd / dig_gla_bwd.
 * dig_gla_bwd_beta returns dbgate (fp32 [B][L][H][d_v]) beside the other gradients.
 * Served by the warp-level tensor-core kernels, for every dtype: with bf16 storage the operands are rounded
 * to tf32 (results within 2e-2 of RMS like dig_gla_fwd), with DIG_F32 every operand is split into two tf32
 * parts and the products are exact to about 2^-21 (results within 1e-4 of RMS, the fp32 bound).  Any
 * supported head and chunk size that fits shared memory.  The workspace is larger than that of
 * dig_gla_fwd / dig_gla_bwd: dig_gla_beta_workspace_bytes (0 for invalid or unsupported sizes).  The same
 * bound of 80 on the magnitude of a gate summed over one chunk applies to bgate. */
size_t dig_gla_beta_workspace_bytes(int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int dtype,
                                    int backward);
dig_status dig_gla_fwd_beta(const void *q, const void *k, const void *v, const float *gate, const float *bgate, void *out,
                            int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);
dig_status dig_gla_bwd_beta(const void *q, const void *k, const void *v, const float *gate, const float *bgate,
                            const void *d_out, void *dq, void *dk, void *dv, float *dgate, float *dbgate,
                            int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Several scan orders at once (Algorithm 2, bidirectional scanning: GLA(z) + flip(GLA(flip(z))); Algorithm 3,
 * 4-directional scanning: the row and column orders, forward and flipped, summed):
 *     out = sum over the directions d in direction_mask of dig_gla_fwd(..., direction = d),
 * bit d of direction_mask (1 .. 15) selecting dig_dir d, all orders reading the same q, k, v and gate and
 * writing canonical positions.  dig_gla_bwd_multi returns the gradients of <d_out, out> (the sums of the
 * single-order gradients).  The orders run one after the other on the stream; each adds its fp32 results
 * to the same buffers (caller's for DIG_BF16_F32OUT, workspace for DIG_BF16), so the sum is formed in fp32
 * and rounded to bf16 once.  Served by the tcgen05 kernels only (bf16 storage, d_k = d_v = 64 or 72; else
 * DIG_ERR_UNSUPPORTED); workspace from dig_gla_multi_workspace_bytes (0 for invalid or unsupported sizes).
 * Tensors, sizes and the gate range are those of dig_gla_fwd / dig_gla_bwd. */
size_t dig_gla_multi_workspace_bytes(int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int dtype,
                                     int backward);
dig_status dig_gla_fwd_multi(const void *q, const void *k, const void *v, const float *gate, void *out, int B, int H,
                             int grid_h, int grid_w, int d_k, int d_v, int chunk, unsigned direction_mask, int dtype,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);
dig_status dig_gla_bwd_multi(const void *q, const void *k, const void *v, const float *gate, const void *d_out,
                             void *dq, void *dk, void *dv, float *dgate, int B, int H, int grid_h, int grid_w, int d_k,
                             int d_v, int chunk, unsigned direction_mask, int dtype, void *workspace,
                             size_t workspace_bytes, void *cuda_stream);

/* Synchronises `cuda_stream`, then returns and clears the status recorded by device code on the
 * current device since the last query: DIG_ERR_TIMEOUT if a bounded wait inside a kernel expired,
 * else DIG_ERR_RANGE if some gates decayed faster than the tcgen05 kernels represent (see dig_gla_fwd),
 * DIG_ERR_CUDA if the synchronisation itself failed, DIG_OK otherwise.  The status is one word per
 * device, shared by all streams and host threads: with several streams in flight the query tells that
 * one of the calls since the last query had the condition, not which.  dig_set_impl is process-wide too. */
dig_status dig_last_device_status(void *cuda_stream);

/* Self-test of the bounded waits (the paper has no counterpart): launches one small kernel whose only
 * wait can never be satisfied and gives up after limit_us microseconds (1 .. 100000), exactly as the
 * production kernels' waits do after 0.25 s.  Afterwards dig_last_device_status returns DIG_ERR_TIMEOUT
 * once; the device and the context stay usable. */
dig_status dig_selftest_wait_timeout(unsigned limit_us, void *cuda_stream);

const char *dig_status_string(int status);

/* Per-kernel timing aid for benchmarks (the paper has no counterpart).  While enabled, every kernel
 * the library launches is bracketed by two CUDA events on the launching stream (a pool of 32768
 * pairs; launches beyond it are counted but not timed).  dig_profile_enable(1) clears the counters
 * and starts recording, dig_profile_enable(0) stops.  dig_profile_read synchronises the recorded
 * events and returns, for kernel number `index` (0 .. dig_profile_kernels()-1), its name (copied
 * into `name`, NUL-terminated, at most name_bytes), the number of launches recorded and their
 * summed device time in milliseconds.  Not thread-safe; meant for one benchmarking thread. */
dig_status dig_profile_enable(int on);
int dig_profile_kernels(void);
dig_status dig_profile_read(int index, char *name, int name_bytes, int *launches, float *total_ms);

#ifdef __cplusplus
}
#endif
#endif /* DIG_GLA_H_ */
