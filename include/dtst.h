/*
 * dtst.h — C ABI of the truncated spectral layer (single-GPU hot path of the
 * Distributed Truncated Spectral Transform, DTST).
 *
 * The layer is  y = I( M( F(x), W ) )  with
 *   F  forward partial DFT: only the retained modes S = S_0 x ... x S_{d-1} of a
 *      real field are computed, one dimension at a time, by contracting with the
 *      per-dimension basis (B_j)_{s,n} = exp(-2 pi i s (off_j + n) / N_j)
 *      (Eq. 5, Eq. 6, Eq. 18; order of Algorithm 1 line 2);
 *   M  per-mode complex channel mixing (Eq. 12);
 *   I  inverse partial DFT back to the real grid (Eq. 14, B^{-1} = B^H / N),
 *      with Hermitian doubling on the one-sided last dimension;
 *   and the adjoint of each step for the backward pass (Section "Backward Pass").
 *
 * Retained set (Section "Background and Motivation"): dims 0..d-2 keep the DFT
 * indices [0..k_j-1] followed by [N_j-k_j..N_j-1] (K_j = 2 k_j entries, ascending
 * index); the last dim, the rfft dimension of the real input, keeps [0..k_{d-1}-1]
 * (K_{d-1} = k_{d-1}).  M = prod K_j modes, flattened row-major.
 *
 * General rules for every call
 *   - All data pointers are DEVICE pointers owned by the caller, contiguous
 *     row-major with the last grid dimension fastest, 16-byte aligned.
 *   - Complex values are interleaved (re, im) float pairs (float2 == complex64).
 *   - `stream` is a cudaStream_t passed as void*; NULL means the default stream.
 *   - Compute calls are asynchronous on `stream`, allocate nothing, and do not
 *     synchronise.  Outputs are overwritten in full.
 *   - Every function returns a dtst_status; nothing throws or aborts.  On error
 *     no kernel has been launched unless the code is DTST_ERR_CUDA.
 *   - A plan may be used from one host thread at a time.  Calls on the same
 *     plan must be stream-ordered with respect to each other because they share
 *     the plan's workspace.
 */
#ifndef DTST_H_
#define DTST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dtst_plan dtst_plan;   /* opaque; created and destroyed by the caller */
typedef int dtst_status;

enum {
  DTST_OK = 0,
  DTST_ERR_INVALID_ARG = -1,     /* null/misaligned pointer, bad shape, bad option          */
  DTST_ERR_UNSUPPORTED = -2,     /* valid request this build cannot serve                   */
  DTST_ERR_ALLOC = -3,           /* host allocation failed                                  */
  DTST_ERR_CUDA = -4,            /* a CUDA runtime call or launch failed                    */
  DTST_ERR_WORKSPACE = -5,       /* workspace missing or smaller than workspace_bytes       */
  DTST_ERR_DEVICE_TIMEOUT = -6,  /* a bounded device-side wait gave up (see dtst_plan_status) */
  DTST_ERR_STATIC_LIMIT = -7     /* dtst_forward_static: the plan needs more than DTST_STATIC_SCRATCH_BYTES */
};

#define DTST_MAX_DIMS 6

/* Kernel families selectable with dtst_plan_set_kernel_path. */
enum {
  DTST_PATH_AUTO = 0,      /* fused streaming kernels where the shape allows, else generic */
  DTST_PATH_GENERIC = 1,   /* one generic contraction kernel per dimension                 */
  DTST_PATH_ROW = 2        /* reported only: streaming kernel on the contiguous dimension (any extent up to 512,
                              odd ones included, and multiples of 8 up to 16384; up to 32 one-sided modes; with the
                              dimension in front of it inside
                              the same kernel where its extent is a multiple of 16 - 32 for extents up to 64 - and at
                              most 256), folded kernels on the others (shapes without a two-dimension tensor-map kernel) */
};

/*
 * Create a plan for a grid that lives entirely on the current device.
 *   d        number of transformed dimensions, 1..DTST_MAX_DIMS
 *   N[d]     grid extents (host array), N[d-1] contiguous in memory
 *   kmax[d]  retained modes per dimension (host array): 1 <= k_j, 2 k_j <= N_j for
 *            j < d-1, and k_{d-1} <= N_{d-1}/2 + 1
 *   B, C_in, C_out  batch and channel counts (>= 1)
 * The plan records the current CUDA device; every compute call must be made with that
 * device current, else it returns DTST_ERR_INVALID_ARG without launching anything.
 * Errors: DTST_ERR_INVALID_ARG for any violated bound, DTST_ERR_ALLOC.
 */
dtst_status dtst_plan_create(dtst_plan** out, int d, const int64_t N[], const int32_t kmax[],
                             int B, int C_in, int C_out);

/*
 * Create a plan for one rank's block of a distributed grid (Eq. 18): the block
 * has extents N_local[j] and starts at global index offset[j] along each
 * dimension; the basis carries the global phase exp(-2 pi i s (offset_j + n)/N_j).
 * dtst_forward then yields this rank's PARTIAL spectrum (Eq. 6), which the caller
 * sums over ranks (Eq. 7); dtst_inverse reconstructs only this rank's block.
 * Requires 0 <= offset[j], offset[j] + N_local[j] <= N_global[j].
 */
dtst_status dtst_plan_create_local(dtst_plan** out, int d, const int64_t N_global[],
                                   const int64_t N_local[], const int64_t offset[],
                                   const int32_t kmax[], int B, int C_in, int C_out);

/*
 * The DTST primitive as Section "Distributed Truncated Spectral Transforms" states it: a COMPLEX d-dimensional
 * tensor and the two-sided retained set S_j = [0..k_j-1, N_j-k_j..N_j-1] on EVERY dimension, the last one included
 * (K_j = 2 k_j for all j, 2 k_j <= N_j).  Arguments as dtst_plan_create_local; N_local and offset may both be NULL
 * for a grid that lives entirely on this device.  Such a plan is used with dtst_forward_complex,
 * dtst_spectral_mul (unchanged), dtst_inverse_complex and dtst_backward_complex; the real-field entry points
 * return DTST_ERR_INVALID_ARG for it.  Virtual shards and per-rank blocks work as for real plans.  The contiguous
 * dimension of a complex plan has no streaming kernel (those read real grids and rely on the rfft fold), so it is
 * contracted LAST, on the most reduced tensor, and expanded first; the grid itself is streamed by the folded and
 * slab kernels of the other dimensions.
 *   F: Xhat[b,c,m] = sum_n x[b,c,n] prod_j exp(-2 pi i s_j(m) (off_j + n_j) / N_j)        (Eq. 5-6, Eq. 18)
 *   I: y[b,o,n]    = (1/prod N) sum_m Yhat[b,o,m] prod_j exp(+2 pi i s_j(m) (off_j + n_j) / N_j)   (Eq. 14)
 *      - no Hermitian doubling: nothing is implied by symmetry;
 *   B: G_Y = F(grad_y) / prod N,  G_X and grad_W as in dtst_backward,  grad_x = sum_m G_X[m] e^{+i theta_m n}
 *      (complex), gradients in the convention dL/dRe + i dL/dIm.
 *   x, y, grad_y, grad_x: [B, C, n_0..n_{d-1}] complex64; spectra [B, C, K_0..K_{d-1}] complex64.
 */
dtst_status dtst_plan_create_complex(dtst_plan** out, int d, const int64_t N_global[], const int64_t N_local[],
                                     const int64_t offset[], const int32_t kmax[], int B, int C_in, int C_out);
dtst_status dtst_forward_complex(dtst_plan* plan, const void* x, void* Xhat, void* stream);
dtst_status dtst_inverse_complex(dtst_plan* plan, const void* Yhat, void* y, void* stream);
dtst_status dtst_backward_complex(dtst_plan* plan, const void* grad_y, const void* Xhat_saved, const void* W,
                                  void* grad_x, void* grad_W, void* stream);

/*
 * Virtual shards: split the (local) grid into P slabs along dim 0, compute each
 * slab's partial spectrum with its global phase offset and sum the P partials on
 * the device in ascending slab order (Eq. 6-7 without a collective).  The inverse
 * and the adjoints expand slab by slab with the same offsets.  P must divide the
 * local extent of dim 0; P = 1 (default) turns the mode off.  Changes
 * workspace_bytes: query it again afterwards.
 */
dtst_status dtst_plan_set_virtual_shards(dtst_plan* plan, int P);

/* Choose the kernel family (DTST_PATH_*).  Changes workspace_bytes. */
dtst_status dtst_plan_set_kernel_path(dtst_plan* plan, int path);

/* Reports which family the plan's calls will actually run: DTST_PATH_AUTO when the fused
 * two-dimension streaming kernels serve this shape, DTST_PATH_ROW when the one-dimension streaming
 * kernels do, else DTST_PATH_GENERIC. */
dtst_status dtst_plan_kernel_path(const dtst_plan* plan, int* path);

/*
 * Contraction order (Section "cuBLAS vs cuFFT", paragraph on dimension ordering: the result does not depend on
 * the order, the work does - contracting the most compressing dimension first shrinks the tensor soonest).
 * The grid-side kernel always takes the contiguous dimension (and, on the fused path, the one in front of it);
 * `order` lists the remaining candidates, the dimensions 0..d-2 (n = d-1 entries, a permutation), in the order
 * the forward-type transforms contract them; the inverse-type transforms expand in the reverse order.  On the
 * fused path the position of dimension d-2 in the list is ignored.  Default: d-2, d-3, .., 0 (Algorithm 1
 * line 2).  With virtual shards dimension 0 must come last (the slab partial spectra are summed after the last
 * stage), else DTST_ERR_INVALID_ARG.  Changes workspace_bytes: query it again.
 * dtst_plan_tune_contraction_order picks the order by ascending K_j / n_j (local extent), dimension 0 last if it
 * carries virtual shards, and reports the bytes the stages behind the grid-side kernel move per forward-type
 * transform before and after (either pointer may be NULL).
 */
dtst_status dtst_plan_set_contraction_order(dtst_plan* plan, const int32_t order[], int n);
dtst_status dtst_plan_get_contraction_order(const dtst_plan* plan, int32_t order[]);
dtst_status dtst_plan_tune_contraction_order(dtst_plan* plan, double* bytes_before, double* bytes_after);

/*
 * "Fast path or fail".  Shapes outside the streaming kernels' reach (odd extents, a contiguous extent that is not
 * a multiple of 32, k outside {4, 8, 12, 16} on a middle dimension, offsets on the contiguous dimension) are
 * served by a generic kernel that is several times slower.  With required != 0 this call returns
 * DTST_ERR_UNSUPPORTED if ANY stage of the plan's forward- or inverse-type transforms would take that kernel,
 * and otherwise DTST_OK, after which the compute calls of this plan return DTST_ERR_UNSUPPORTED (launching
 * nothing) should a later option change (virtual shards, kernel path) make a stage fall back.  required = 0
 * lifts the requirement.  dtst_plan_kernel_path tells which family serves the grid-side stage.
 */
dtst_status dtst_plan_require_fast_path(dtst_plan* plan, int required);

/*
 * Optional variant of the inverse-type stage (dtst_inverse and the last stage of dtst_backward) for plans on
 * the fused streaming path with d >= 3: the expansion of dimension d-3 (B^H along it, Eq. 14) runs INSIDE the
 * kernel that writes the grid, on one extra warp per CTA that stays a few columns ahead of the warps expanding
 * the last two dimensions, through a ring of `ring_columns` columns that is consumed from L2; the separate
 * launch for that dimension and its full-size intermediate in HBM disappear.  Same arithmetic, same bits.
 * Off by default (ring_columns = 0): measured on the largest benchmark shape it shortens an isolated inverse
 * call by 6 % (ring of 48-64 columns) but a whole step not at all - the single helper warp is the pipeline's
 * bottleneck under the power cap - and it slows small grids down.  Returns DTST_ERR_UNSUPPORTED (and stays off)
 * when the plan's shape has no such kernel.  Call it before querying workspace_bytes.
 */
dtst_status dtst_plan_set_column_expansion(dtst_plan* plan, int ring_columns);

/*
 * Forward-type transforms (dtst_forward and the first stage of dtst_backward) of plans on the fused streaming path
 * whose shape has such a kernel contract the dimension d-3 INSIDE the kernel that streams the grid (columns of
 * planes batched in shared memory, the column's accumulator in tensor-core fragments): the reduced tensor of the
 * plane stage never reaches HBM and one launch disappears.  Same tolerance against the float64 statement.
 *   mode  0 (default): whenever the kernel exists for the shape, dimension d-3 is whole on this device, first in
 *                      the contraction order, and the plan has enough columns (batch x channels x leading extents)
 *                      to keep every SM busy in the last round;
 *   mode  1: whenever the kernel exists (small problems: for tests);   mode -1: never.
 */
dtst_status dtst_plan_set_column_contraction(dtst_plan* plan, int mode);

/*
 * Arithmetic of the tensor-core stages of the kernels for contiguous extents that are no multiple of 32 or longer than
 * 256 points and for middle dimensions of any extent and mode count (the paper's own layer, time axis 30, runs on
 * them; they are bound by their arithmetic, not by HBM):
 *   DTST_ARITH_TF32X3  (default) every product as three TF32 products of hi/lo operand parts with fp32
 *                      accumulation: rel-L2 of each output tensor against the float64 statement <= 1e-5
 *                      (measured 1e-6..2e-6);
 *   DTST_ARITH_TF32    one TF32 product per term (operands rounded to 11 significant bits, fp32 accumulation):
 *                      rel-L2 <= 2e-3 (measured 2e-4..6e-4), a third of the tensor-core work.
 * The other kernels (tensor-map plane and row kernels, double-folded middle kernels, mixing) are bound by HBM with
 * the compensated arithmetic in place and are not affected.
 */
enum { DTST_ARITH_TF32X3 = 0, DTST_ARITH_TF32 = 1 };
dtst_status dtst_plan_set_arithmetic(dtst_plan* plan, int mode);

dtst_status dtst_plan_destroy(dtst_plan* plan);

/* M = number of retained modes; K[d] (host, may be NULL) = entries kept per dim. */
dtst_status dtst_plan_num_modes(const dtst_plan* plan, int64_t* M, int64_t K[]);

/* The retained DFT indices of dimension `dim`, ascending: writes K[dim] int64
 * values to the HOST array idx.  Bit-exact contract: [0..k-1, N-k..N-1] for
 * dim < d-1, [0..k-1] for dim = d-1. */
dtst_status dtst_plan_mode_indices(const dtst_plan* plan, int dim, int64_t* idx);

/* Scratch the compute calls need, in bytes (device memory, 256-byte aligned). */
dtst_status dtst_plan_workspace_bytes(const dtst_plan* plan, size_t* bytes);

/* Hand the plan a caller-owned device buffer of at least workspace_bytes; it must
 * stay valid while compute calls of this plan are in flight.  The plan never
 * frees it.  Errors: DTST_ERR_INVALID_ARG (null / not 256-byte aligned),
 * DTST_ERR_WORKSPACE (too small). */
dtst_status dtst_plan_set_workspace(dtst_plan* plan, void* dev_ptr, size_t bytes);

/*
 * F — forward partial DFT (Eq. 5-6, Eq. 18).
 *   x    [B, C_in, n_0..n_{d-1}] float32 (device, read once)
 *   Xhat [B, C_in, K_0..K_{d-1}] complex64 (device, written)
 *   Xhat[b,c,m] = sum_n x[b,c,n] prod_j exp(-2 pi i s_j(m) (off_j + n_j) / N_j)
 */
dtst_status dtst_forward(dtst_plan* plan, const float* x, void* Xhat, void* stream);

/*
 * M — per-mode channel mixing (Eq. 12):
 *   Yhat[b,o,m] = sum_i Xhat[b,i,m] * W[i,o,m]
 *   Xhat [B, C_in, M], W [C_in, C_out, M], Yhat [B, C_out, M], all complex64.
 * Yhat must not alias Xhat or W.
 */
dtst_status dtst_spectral_mul(dtst_plan* plan, const void* Xhat, const void* W, void* Yhat,
                              void* stream);

/*
 * I — inverse partial DFT with Hermitian doubling (Eq. 14):
 *   y[b,o,n] = (1/prod N) sum_m c(m) Re( Yhat[b,o,m] prod_j exp(+2 pi i s_j(m) (off_j+n_j)/N_j) )
 *   c(m) = 1 if the last-dim frequency f is 0 or Nyquist (2f = N_{d-1}), else 2.
 *   Yhat [B, C_out, M] complex64 (read), y [B, C_out, n_0..n_{d-1}] float32 (written once).
 */
dtst_status dtst_inverse(dtst_plan* plan, const void* Yhat, float* y, void* stream);

/*
 * B — backward pass of y = I(M(F(x), W)) for upstream gradient grad_y
 * (Section "Backward Pass": every step is linear, so each is replaced by its adjoint):
 *   G_Y  = (c / prod N) * F(grad_y)
 *   G_X[b,i,m]     = sum_o G_Y[b,o,m] * conj(W[i,o,m])
 *   grad_W[i,o,m]  = sum_b conj(Xhat_saved[b,i,m]) * G_Y[b,o,m]
 *   grad_x[b,i,n]  = Re sum_m G_X[b,i,m] prod_j exp(+2 pi i s_j(m) (off_j+n_j)/N_j)
 * Complex gradients follow the convention dL/dRe + i dL/dIm.
 *   grad_y [B, C_out, n...] float32; Xhat_saved = dtst_forward's output; W as above;
 *   grad_x [B, C_in, n...] float32 and grad_W [C_in, C_out, M] complex64 are ASSIGNED
 *   (not accumulated); either may be NULL to skip it (not both).  Xhat_saved is read only
 *   for grad_W and may be NULL when grad_W is NULL.
 */
dtst_status dtst_backward(dtst_plan* plan, const float* grad_y, const void* Xhat_saved,
                          const void* W, float* grad_x, void* grad_W, void* stream);

/*
 * The whole block around the layer (Section "Block Structure"; Algorithm 1 lines 1 and 8; Eq. 1):
 *   z   = W_bypass x + I(M(F(x), W))        z[b,o,n] = sum_i W_bypass[o,i] x[b,i,n] + y[b,o,n]
 *   out = GELU(z) = z Phi(z)                 (exact erf form; the paper names GELU and no bias)
 *   x [B, C_in, n...] float32; W [C_in, C_out, M] complex64 (the spectral weights of dtst_spectral_mul);
 *   W_bypass [C_out, C_in] float32, row-major (the point-wise linear operator, a 1x1 convolution's weight);
 *   out [B, C_out, n...] float32 (written); Xhat_saved [B, C_in, M] complex64 (written: F(x), needed by
 *   the backward pass); z_saved [B, C_out, n...] float32, the pre-activation, written when not NULL (pass NULL
 *   for inference).  out and z_saved must not alias x or each other.
 * The mixed spectrum lives in the plan's workspace.  Needs grid points per (b, c) % 4 == 0 (always true, the
 * contiguous extent is a multiple of 4) and C_in + C_out <= 64, else DTST_ERR_UNSUPPORTED.
 */
dtst_status dtst_block_forward(dtst_plan* plan, const float* x, const void* W, const float* W_bypass,
                               float* out, void* Xhat_saved, float* z_saved, void* stream);

/*
 * Which kernel forms the bypass product W_bypass x inside dtst_block_forward:
 *   DTST_BLOCK_EPILOGUE_FFMA    exact fp32 multiply-adds, any channel count;
 *   DTST_BLOCK_EPILOGUE_TENSOR  the tensor cores (tcgen05.mma kind::tf32 with the accumulator in tensor memory,
 *                               three TF32 products per fp32 product): C_in in {8, 16, 32}, C_out in {16, 32},
 *                               plans on the streaming kernel family; DTST_ERR_UNSUPPORTED otherwise;
 *   DTST_BLOCK_EPILOGUE_AUTO    (default) the faster of the two as measured on B200: the FFMA kernel, at every
 *                               channel count the tensor-core kernel exists for.
 * Both meet the same tolerance against the float64 statement of the block.
 */
enum { DTST_BLOCK_EPILOGUE_AUTO = 0, DTST_BLOCK_EPILOGUE_FFMA = 1, DTST_BLOCK_EPILOGUE_TENSOR = 2 };
dtst_status dtst_plan_set_block_epilogue(dtst_plan* plan, int mode);

/*
 * Backward pass of the block for upstream gradient grad_out = dL/d out (Section "Backward Pass": the linear
 * steps are replaced by their adjoints; the activation by its derivative):
 *   g_z            = grad_out * GELU'(z_saved),   GELU'(z) = Phi(z) + z phi(z)
 *   grad_W_bypass[o,i] = sum_{b,n} g_z[b,o,n] x[b,i,n]
 *   (grad_x, grad_W)   = dtst_backward(g_z, ...);   grad_x += W_bypass^T g_z
 *   scratch [B, C_out, n...] float32: caller-owned, overwritten with g_z (it may be grad_out itself when the
 *   caller no longer needs grad_out); it must not alias x, z_saved or grad_x.
 *   grad_x [B, C_in, n...], grad_W [C_in, C_out, M] complex64, grad_W_bypass [C_out, C_in] are ASSIGNED; any of
 *   them may be NULL to skip it (not all three).  Xhat_saved is read for grad_W only.
 * The sum over grid points for grad_W_bypass runs in a fixed order (per-CTA partial sums in the workspace,
 * added in ascending CTA order): repeated calls give the same bits.
 */
dtst_status dtst_block_backward(dtst_plan* plan, const float* grad_out, const float* x, const float* z_saved,
                                const void* Xhat_saved, const void* W, const float* W_bypass, float* scratch,
                                float* grad_x, void* grad_W, float* grad_W_bypass, void* stream);

/*
 * Point-wise linear layers: the lifting network P and the projection network Q around the blocks of an FNO
 * (Section "Background and Motivation", Eq. 1: "lifted ... via a pointwise network P ... projected ... via a
 * pointwise network Q"; taken here as one linear map each, with an optional bias).  No plan is involved.
 *   out[b,o,p] = sum_i W[o,i] x[b,i,p] + bias[o]
 *   x [B, C_in, points], out [B, C_out, points] float32 (device, 16-byte aligned, points % 4 == 0, out != x);
 *   W [C_out, C_in] row-major; bias [C_out] or NULL.
 * Backward for upstream gradient grad_out [B, C_out, points]:
 *   grad_x[b,i,p] = sum_o W[o,i] grad_out[b,o,p]   (assigned)
 *   grad_W[o,i]   = sum_{b,p} grad_out[b,o,p] x[b,i,p],   grad_bias[o] = sum_{b,p} grad_out[b,o,p]
 * any of the three may be NULL (not all).  The two sums over points run in a fixed order through `scratch`
 * (device, dtst_pointwise_linear_scratch_bytes; DTST_ERR_WORKSPACE if missing or too small): same bits on every
 * run.  Needs C_in + C_out <= 64 for the backward pass, else DTST_ERR_UNSUPPORTED.
 */
dtst_status dtst_pointwise_linear(int B, int C_in, int C_out, int64_t points, const float* x, const float* W,
                                  const float* bias, float* out, void* stream);
dtst_status dtst_pointwise_linear_scratch_bytes(int C_in, int C_out, size_t* bytes);
dtst_status dtst_pointwise_linear_backward(int B, int C_in, int C_out, int64_t points, const float* grad_out,
                                           const float* x, const float* W, float* grad_x, float* grad_W,
                                           float* grad_bias, void* scratch, size_t scratch_bytes, void* stream);

/*
 * The same steps one by one, for a caller that runs the layer across several ranks (Algorithm 1: each
 * rank owns a slab of the grid and an equal, contiguous share S_p of the flattened modes, Eq. 12) and
 * exchanges spectra between the steps with its own collectives:
 *   forward:  dtst_forward on the slab (plan from dtst_plan_create_local)  -> partial spectrum
 *             all-reduce(sum) over ranks (Eq. 7)                           -> Xhat, full [B, C_in, M]
 *             dtst_spectral_mul_modes on [m0, m0 + count)                  -> Yhat chunk [B, C_out, count]
 *             all-gather of the chunks                                     -> Yhat, full
 *             dtst_inverse on the slab                                     -> y on the slab
 *   backward: dtst_backward_spectrum (partial G_Y), all-reduce, dtst_backward_mix_modes on the rank's
 *             modes (grad_W shard stays local: no all-reduce of weight gradients), all-gather of the
 *             G_X chunks, dtst_backward_input on the slab.
 * Layouts: full spectra [B, C, M]; W_shard, grad_W_shard [C_in, C_out, count]; chunks [B, C, count];
 * all complex64, device, 16-byte aligned.  0 <= m0, count >= 1, m0 + count <= M, else
 * DTST_ERR_INVALID_ARG.  Outputs are assigned.  dtst_backward_mix_modes: GX_chunk or grad_W_shard may be
 * NULL to skip it (not both); Xhat_saved is only read for grad_W_shard.
 */
dtst_status dtst_spectral_mul_modes(dtst_plan* plan, const void* Xhat, const void* W_shard,
                                    void* Yhat_chunk, int64_t m0, int64_t count, void* stream);
/* G_Y = (c / prod N_global) * F(grad_y) of this plan's block: [B, C_out, M] (the adjoint of dtst_inverse). */
dtst_status dtst_backward_spectrum(dtst_plan* plan, const float* grad_y, void* GY, void* stream);
dtst_status dtst_backward_mix_modes(dtst_plan* plan, const void* GY, const void* Xhat_saved,
                                    const void* W_shard, void* GX_chunk, void* grad_W_shard,
                                    int64_t m0, int64_t count, void* stream);
/* grad_x = Re sum_m G_X[m] e^{+i theta_m n} on this plan's block: no doubling, no 1 / prod N
 * (the adjoint of dtst_forward).  GX [B, C_in, M]. */
dtst_status dtst_backward_input(dtst_plan* plan, const void* GX, float* grad_x, void* stream);

/*
 * The whole step for callers whose activations live in HOST memory.  One step = F, M, I (Eq. 5-14) and B
 * (Section "Backward Pass") on inputs x and grad_y that are copied in from the host and results y, grad_x and
 * grad_W that are copied back, inside the call's work:
 *   dtst_plan_host_io_bytes   device staging the step needs (x, grad_y, y, grad_x, two spectra, grad_W);
 *   dtst_plan_enable_host_io  hands that staging over (device pointer, 256-byte aligned, caller-owned) and creates
 *                             the three internal streams (copy-in, compute, copy-out) and their events - the only
 *                             allocation; NULL switches the facility off and releases them;
 *   dtst_step_host            enqueues one step and returns at once: hx [B, C_in, n...], hgy [B, C_out, n...] host
 *                             (read), dW [C_in, C_out, M] complex64 DEVICE (the layer's parameter), hy, hgx, hgW
 *                             host (written).  Transfers overlap the kernels and each other, also across
 *                             consecutive steps (a step's copy-in runs under the previous step's backward pass).
 *                             Use page-locked host buffers: pageable ones make the copies synchronous.  The host
 *                             buffers of a step must stay untouched until dtst_host_io_wait has returned.
 *   dtst_host_io_wait         blocks until the outputs of every enqueued step are in host memory.
 * The plan needs its workspace as for the device-pointer calls.  Real plans only.
 */
dtst_status dtst_plan_host_io_bytes(const dtst_plan* plan, size_t* bytes);
dtst_status dtst_plan_enable_host_io(dtst_plan* plan, void* dev_staging, size_t bytes);
dtst_status dtst_step_host(dtst_plan* plan, const float* hx, const float* hgy, const void* dW, float* hy,
                           float* hgx, void* hgW);
dtst_status dtst_host_io_wait(dtst_plan* plan);

/*
 * The forward partial DFT without any caller-provided or allocated scratch.
 * (The paper has no counterpart to this call; it exists for integration reasons.)
 *
 * Who needs it: code that is not allowed to allocate device memory at the point
 * where it calls the transform and has no workspace to hand over either - for
 * example a plug-in running inside a host application that owns the whole
 * memory pool, a real-time loop that forbids allocator calls after start-up, or
 * a process whose device memory has been fully pre-committed by another
 * framework.  For those callers dtst_forward is unusable, because its
 * intermediates live in the workspace given to dtst_plan_set_workspace.
 *
 * This variant computes exactly what dtst_forward's generic path computes
 * (same kernels, same order, same virtual-shard handling), but keeps the
 * intermediates in one fixed array of DTST_STATIC_SCRATCH_BYTES that is part of
 * the library image.  Consequences the caller must know:
 *   - Every GPU that loads this library holds those bytes until the process exits.
 *   - The plan needs no workspace for this call.  If its intermediates (two
 *     stage buffers plus, with virtual shards, P partial spectra) exceed
 *     DTST_STATIC_SCRATCH_BYTES the call launches nothing and returns
 *     DTST_ERR_STATIC_LIMIT; use a smaller batch/channel count per call or
 *     dtst_forward with a workspace.
 *   - The call itself calls no cudaMalloc/cudaFree and no allocating library
 *     routine.  The FIRST call on each device looks up the array's device
 *     address (once per device, with that device current); make that first call
 *     during start-up, before any stream capture.
 *   - All calls, from all plans and streams, share the one array, which keeps
 *     whatever the previous call left in it.  Nothing in it has to start at
 *     zero: each intermediate is written in full before it is read.  Two calls
 *     that overlap in time on the GPU (different streams, or different host
 *     threads) race on it and corrupt each other's results: serialise them.
 * Arguments and result as for dtst_forward.
 */
#define DTST_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
dtst_status dtst_forward_static(dtst_plan* plan, const float* x, void* Xhat, void* stream);

/* Synchronises `stream` and reports the plan's device-side status word:
 * DTST_OK, or DTST_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel gave up
 * (the kernel then exited normally and its output is undefined).  Clears the word. */
dtst_status dtst_plan_status(dtst_plan* plan, void* stream);

/*
 * Diagnostic for the failure-reporting path, not for production use.  Every device-side wait in
 * the streaming kernels is bounded: when its poll budget runs out the kernel raises the plan's
 * status word and returns normally (no trap, no hang).  This call makes that happen on purpose:
 * from now on the forward plane kernel's producer stops feeding its shared-memory ring after
 * `withhold_after_fills` slot fills and the waits give up after `poll_limit` polls (1..65536, so
 * that the run ends within milliseconds); the call's output is then undefined and
 * dtst_plan_status reports DTST_ERR_DEVICE_TIMEOUT once.  withhold_after_fills < 0 restores
 * normal operation.  Only plans on the fused streaming path are affected (dtst_plan_kernel_path
 * == DTST_PATH_AUTO).
 */
dtst_status dtst_plan_debug_ring_fault(dtst_plan* plan, int64_t withhold_after_fills, uint32_t poll_limit);

/* Number of kernel launches the plan's compute calls have issued so far. */
dtst_status dtst_plan_launch_count(const dtst_plan* plan, int64_t* launches);

/*
 * Optional per-kernel timing for benchmarks.  When enabled, the compute calls
 * bracket selected kernels with CUDA events on the call's stream; nothing is
 * synchronised until the query.  `capacity` = launches recorded per kind before
 * recording stops (events are created here, never inside a compute call);
 * capacity 0 disables timing and frees the events.
 * Kinds: the kernel that streams the real grid in (forward-type, used by F and by
 * the first stage of B), the kernel that streams the real grid out (inverse-type,
 * used by I and by the last stage of B), the mixing kernel, the mixing adjoint.
 */
enum {
  DTST_KERNEL_GRID_READ = 0,
  DTST_KERNEL_GRID_WRITE = 1,
  DTST_KERNEL_MIX = 2,
  DTST_KERNEL_MIX_ADJOINT = 3,
  DTST_KERNEL_BLOCK_EPILOGUE = 4,   /* dtst_block_forward: bypass product + add + GELU                 */
  DTST_KERNEL_GELU_BACKWARD = 5,    /* dtst_block_backward: g_z = grad_out * GELU'(z)                   */
  DTST_KERNEL_BYPASS_BACKWARD = 6,  /* dtst_block_backward: grad_x += W_bypass^T g_z, grad_W_bypass      */
  DTST_KERNEL_KINDS = 7
};
dtst_status dtst_plan_enable_kernel_timing(dtst_plan* plan, int capacity);

/* Synchronises the device, then reports for `kind` the number of recorded launches and
 * the sum of their durations in milliseconds, and resets that kind's record. */
dtst_status dtst_plan_kernel_timing(dtst_plan* plan, int kind, int64_t* launches, double* total_ms);

/* After a call returned DTST_ERR_CUDA: the CUDA runtime's error code and its text for the
 * failing runtime call or launch of this plan (0 / "no error" otherwise).  The string is static. */
dtst_status dtst_plan_last_cuda_error(const dtst_plan* plan, int* code, const char** text);

/*
 * Diagnostics read once from the environment (for A/B measurements; not for production use):
 *   DTST_NO_PDL=1            launch every kernel without the programmatic-dependent-launch attribute
 *   DTST_NO_COLFUSE=1        forward-type transforms: contract the third dimension in a launch of its own instead of
 *                            inside the kernel that streams the grid (shapes for which that kernel exists)
 *   DTST_NO_PLANEG=1         contiguous extents that are no multiple of 32: contract / expand the dimension in front in a
 *                            launch of its own instead of inside the row kernel
 */
const char* dtst_status_string(dtst_status s);

/* Library version as major*10000 + minor*100 + patch. */
int dtst_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DTST_H_ */
