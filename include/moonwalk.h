/*
 * moonwalk.h -- C ABI of the B200 (sm_100a) Moonwalk gradient library.
 *
 * Moonwalk (mixed mode, Section 4.1 of the paper) computes the parameter gradients of a
 * sequential network x_i = f_i(x_{i-1}; theta_i) with scalar loss J in three phases:
 *   Phase I   forward pass that keeps only the residuals the input-cotangent path needs
 *             (one sign bit per activation, Section "Residual Impact");
 *   Phase II  reverse pass for the input cotangent h_0 = dJ/dx_0 only; on the way it writes
 *             cotangent checkpoints (Section 4.1, "gradient checkpointing in Phase II") and
 *             the fragments of non-submersive layers (Section 5.1);
 *   Phase III forward sweep (Algorithm 1): per layer recompute x_i, carry the cotangent with
 *             h_i = vijp(f_i, x_{i-1}, h_{i-1}) (Eq. "h_i") and form g_i = vjp(f_i, theta_i, h_i)
 *             (Eq. "g_i").
 *
 * Conventions
 *   - Layer i: z = linear_i(x_{i-1}), x_i = phi(z).  No bias.  Dense weights are row-major
 *     [n_out][n_in], z = x W^T.  Convolutions follow Lemma 1: channel-last activations
 *     [B][H][W][C], kernel w[kh][kw][c_in][c_out], x'[i',c'] = sum w[j,c,c'] x[s i'+j-p, c],
 *     zero padding.  The head (MW_HEAD_LINEAR) is a dense layer on the flattened activation,
 *     allowed only as the last layer; it needs no vijp.
 *   - "positive" means z > 0 strictly; 0, -0.0 and NaN take the negative branch.
 *   - Every device buffer is allocated and owned by the caller.  The library allocates no
 *     device memory: all per-step state lives in the caller's `workspace`.
 *   - Calls enqueue work on `stream` and return without synchronising, unless stated.
 *     Argument errors are returned synchronously.  Device-side conditions (a bounded wait that
 *     ran out, an inverse that did not converge) are recorded in a status word inside the
 *     workspace and read back by mw_last_device_status().
 *   - Nothing aborts, throws or prints.
 */
#ifndef MOONWALK_H_
#define MOONWALK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mw_net mw_net; /* opaque, host side; owns no device memory */

typedef enum {
  MW_OK = 0,
  MW_ERR_INVALID_ARG = 1,    /* null pointer, bad enum, inconsistent sizes               */
  MW_ERR_UNSUPPORTED = 2,    /* layer / size combination the library has no kernel for  */
  MW_ERR_WORKSPACE = 3,      /* workspace null, misaligned (256 B) or too small          */
  MW_ERR_STATE = 4,          /* sweep called without a matching mw_input_cotangent       */
  MW_ERR_NOT_SUBMERSIVE = 5, /* a layer's Jacobian could not be inverted to tolerance    */
  MW_ERR_TIMEOUT = 6,        /* a bounded device-side wait expired                       */
  MW_ERR_CUDA = 7            /* a CUDA runtime / driver call failed                      */
} mw_status;

/* MW_CONV1D: a convolution along one dimension, [W positions][C channels] per sample (H = 1),
 * kernel w[k][c_in][c_out]; its reverse pass is undone with fragmental checkpoints (Section 5.1). */
typedef enum { MW_DENSE = 0, MW_CONV2D = 1, MW_HEAD_LINEAR = 2, MW_CONV1D = 3 } mw_kind;
typedef enum { MW_ACT_NONE = 0, MW_ACT_LEAKY_RELU = 1, MW_ACT_RELU = 2 } mw_act;

/* Storage / arithmetic:
 *   MW_F64          x, W, targets, g0, dW double; arithmetic double (CUDA cores).
 *   MW_F32          x, W, targets, g0, dW float; products accurate to fp32 (tensor cores with
 *                   operands split into bf16 terms, fp32 accumulate; or CUDA-core FMA).
 *   MW_BF16_F32ACC  x, W bf16; targets, g0, dW float; activations between layers bf16; the
 *                   cotangent chain (h, W^-1), fragments and checkpoints fp32-accurate.    */
typedef enum { MW_F64 = 0, MW_F32 = 1, MW_BF16_F32ACC = 2 } mw_prec;

/* MW_LOSS_HALF_SSE   J = 0.5 * sum (y-t)^2 over all B*n entries; target = [B][n] floats.
 * MW_LOSS_MSE_MEAN   J = mean (y-t)^2 over all B*n entries.
 * MW_LOSS_XENT_MEAN  J = mean over the batch of -log softmax(y_b)[label_b]; target = int32[B]. */
typedef enum { MW_LOSS_HALF_SSE = 0, MW_LOSS_MSE_MEAN = 1, MW_LOSS_XENT_MEAN = 2 } mw_loss;

typedef enum { MW_BACKEND_AUTO = 0, MW_BACKEND_SIMT = 1, MW_BACKEND_TENSOR = 2 } mw_backend;

typedef struct {
  int32_t kind;          /* mw_kind */
  int32_t act;           /* mw_act  */
  double slope;          /* leaky-ReLU negative slope (ignored otherwise)                 */
  int32_t n_in, n_out;   /* dense / head: features in and out (dense must be square)      */
  int32_t H, W, C_in, C_out, k, stride, pad; /* conv: input H x W x C_in, kernel k x k    */
} mw_layer_desc;

typedef struct {
  int32_t prec;            /* mw_prec */
  int32_t loss;            /* mw_loss */
  int32_t reseed_every;    /* K: Phase II keeps the full cotangent h_l for every l that is a
                              multiple of K (0 < l < L) and Phase III restarts its recursion
                              from it.  0 = never: the literal Algorithm 1.                 */
  int32_t conv_vijp_iters; /* fixed-point updates of the stride-1 convolution vijp          */
  int32_t backend;         /* mw_backend; AUTO = tensor cores when the sizes allow          */
  int32_t inverse_iters;   /* Newton-Schulz steps for W^-1 (0 = default for the precision)  */
  int32_t resident_inverse;/* 1: mw_input_cotangent computes every layer's W^-1 (and split
                              operands) once and keeps them in the workspace; 0: the sweep
                              builds them layer by layer in a transient slot (lean memory) */
  int32_t warm_inverse;    /* 1 (dense nets on the tensor cores with resident_inverse = 1): the
                              workspace keeps every W^-1 from one mw_input_cotangent to the next,
                              and a call on the same workspace REFRESHES them with the last step
                              of the Newton-Schulz schedule instead of computing them from
                              scratch.  For loops whose steps move the weights very little
                              (fine tuning, small learning rates): the kept inverse X must
                              still satisfy ||I - W X||_F <= 5e-4 (MW_F32) / 4e-3 (bf16) for
                              the new W -- roughly ||delta W||_F below that -- which the call
                              checks per layer (MW_ERR_NOT_SUBMERSIVE through
                              mw_last_device_status; after that report the next call starts
                              from scratch again).  The workspace must be left alone between
                              steps.  0: every call computes the inverses from scratch.        */
  int32_t frag_block;      /* MW_CONV1D nets: Phase II keeps the output cotangent of every
                              convolution at the first k - 1 positions of each block of this
                              many positions (2..64, dividing W); Phase III rebuilds the rest  */
  int32_t lu_param;        /* 1: every dense layer is parameterised by the triangular factors of
                              its weight, the paper's constrained-layer idea (Section "Constrained
                              Convolutions") carried to dense layers: params[l] ([n][n]) holds L
                              strictly below the diagonal (unit diagonal implied) and U on and
                              above it, the layer's weight is W = L U, and gradients come back in
                              the same layout (dJ/dL below, dJ/dU on and above the diagonal).
                              W^-1 = U^-1 L^-1 is then built from the factors by block
                              substitution, exactly: no Newton-Schulz iteration, no convergence
                              domain; a zero on the diagonal of U is the only failure
                              (MW_ERR_NOT_SUBMERSIVE).  Tensor-core backend, MW_F32, widths that
                              are multiples of 128, resident_inverse = 1, warm_inverse = 0;
                              mw_forward_sweep_apply is not available.  0: params[l] is W.      */
} mw_net_opts;

/* Build a host-side description.  `batch` is fixed per net.
 * Dense layers must be invertible (the vijp of Section 3.1 is g_z = h W^-1).  The CUDA-core
 * backend inverts with pivoted elimination (widths up to 64) and accepts any invertible W.  The
 * tensor-core backend iterates X <- X + X (I - W X) from X_0 = (n / ||W||_F^2) W^T in a fixed
 * number of steps: it converges while sigma_max(W)^2 < 2 mean(sigma_i^2) and reaches working
 * precision in its default schedule when ||I - W X_0|| is about 0.15 or less, i.e. for weights
 * near a multiple of an orthogonal matrix (mw_net_opts.inverse_iters adds steps).  Outside that
 * domain the layer is reported per step as MW_ERR_NOT_SUBMERSIVE, never answered silently
 * (mw_net_opts.lu_param parameterises the layers so that the inverse is exact instead).
 * Returns MW_ERR_UNSUPPORTED for
 * shapes outside: dense layers square; convolutions with C_in = C_out, either stride 1 with
 * k = 2*pad+1 (same size), or every layer of the net meeting Lemma 1 (i) with stride 2 (the
 * paper's submersive CNN: MW_F32 or MW_BF16_F32ACC, 64 or 128 channels, k - 1 - pad < 2, even image sizes, a
 * loss on the last feature map; conditions (ii) and (iii) on the anchor tap w[pad][pad] are
 * checked on the device every step: MW_ERR_NOT_SUBMERSIVE); MW_CONV1D nets: every layer k = 3,
 * stride 1, padding 1, the same W (a multiple of 128) and C (64..256, a multiple of 64), MW_F32 or
 * MW_BF16_F32ACC,
 * tap 0 lower triangular in (c_in, c_out) with a non-zero diagonal (checked on the device);
 * head only as the last layer; all layers of one net share `prec`. */
mw_status mw_net_create(const mw_layer_desc* layers, int32_t n_layers, int32_t batch,
                        const mw_net_opts* opts, mw_net** out);
void mw_net_destroy(mw_net* net);

/* Bytes of workspace (256-byte aligned device memory) needed by the Moonwalk calls and by
 * mw_backprop_reference.  `residual_bytes` (may be NULL) receives the part of each that must
 * survive between the phases: [0] Moonwalk (sign bits + fragments + cotangent checkpoints),
 * [1] backprop (stored activations + sign bits). */
mw_status mw_workspace_bytes(const mw_net* net, size_t* moonwalk_bytes, size_t* backprop_bytes,
                             size_t residual_bytes[2]);

/* Phases I and II (Section 4.1): g0 = dJ/dx_0.
 *   params       host array of n_layers DEVICE pointers to the weights (read-only).
 *   x            device, [B][n_0] (or NHWC), storage type of `prec`.
 *   loss_target  device, see mw_loss.
 *   g0_out       device, [B][n_0], double (MW_F64) or float.  May be NULL for a net of strided
 *                submersive convolutions: the vijp of such a layer (Lemma 1) reads the input
 *                cotangent at the pixels (s*y, s*x) only, so only those are then computed
 *                (one ninth of the first layer's TransposeConv for k = 3) and kept in the
 *                workspace; call mw_forward_sweep with g0 = NULL.
 *   loss_out     device pointer to one double receiving J, or NULL.
 * Also fills the workspace with the residual stores the sweep consumes. */
mw_status mw_input_cotangent(mw_net* net, const void* const* params, const void* x,
                             const void* loss_target, void* g0_out, double* loss_out,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Phase III with the last line of Algorithm 1 ("apply g_i to theta_i") fused into the weight vjp:
 * params_out[l] = params[l] - lr * g_l for every layer, written by the epilogue of the product that
 * forms g_l, so that no gradient buffer exists (gradients need not coexist, Section 4.3).
 * params_out[l] (device, float, shaped like the weight) may be params[l] itself: the products of
 * the sweep read the term planes Phase I made of the weights, never params again (with
 * resident_inverse = 0 layer l's weight is read just before its own update).  A NULL entry skips
 * that layer.  In nets whose convolutions are constrained to a triangular tap (Lemma 1 (ii);
 * Section 5.1 for MW_CONV1D) the entries that the constraint fixes at zero are not parameters
 * (Section "Constrained Convolutions") and stay zero.  MW_F32 nets on the tensor-core backend;
 * otherwise MW_ERR_UNSUPPORTED.  Other arguments, requirements and errors as for
 * mw_forward_sweep. */
mw_status mw_forward_sweep_apply(mw_net* net, const void* const* params, const void* x,
                                 const void* g0, double lr, void* const* params_out,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* Phase III (Algorithm 1): all parameter gradients from x and g0.
 *   dW_out  host array of n_layers DEVICE pointers, each shaped like its weight, double
 *           (MW_F64) or float; overwritten.  A NULL entry skips storing that layer's gradient
 *           (gradients need not coexist, Section 4.3 last paragraph but one).
 *   g0      the result of mw_input_cotangent; NULL where that call allows g0_out = NULL: the sweep
 *           then starts from the part of g0 that call left in the workspace.
 * Requires the workspace last written by mw_input_cotangent on the same net, with the same x,
 * unchanged since (MW_ERR_STATE where that can be told). */
mw_status mw_forward_sweep(mw_net* net, const void* const* params, const void* x, const void* g0,
                           void* const* dW_out, void* workspace, size_t workspace_bytes,
                           void* stream);

/* Gradient buckets for data-parallel training (Algorithm 1 produces the gradients front to back, so
 * the all-reduce of the first layers can run while the sweep works on the later ones).  After this
 * call every mw_forward_sweep on `net` records events[b] (CUDA events of the caller, n_events =
 * ceil(n_layers / layers_per_bucket)) on its stream as soon as the work that completes dW of the
 * layers [b * layers_per_bucket, (b + 1) * layers_per_bucket) is enqueued; a consumer stream that
 * waits for events[b] may then reduce those gradients.  Dense nets on the tensor cores signal the
 * buckets as they go (one launch per bucket); other nets record all events at the end of the
 * call.  layers_per_bucket = 0 turns the feature off.  The events stay the caller's. */
mw_status mw_sweep_bucket_events(mw_net* net, int32_t layers_per_bucket, void* const* events,
                                 int32_t n_events);

/* Plain reverse mode ("Backprop", Appendix "Complexity Analysis" item 1): forward storing every
 * layer input, backward with both vjps.  Same kernels, for the memory and runtime comparison. */
mw_status mw_backprop_reference(mw_net* net, const void* const* params, const void* x,
                                const void* loss_target, void* const* dW_out, double* loss_out,
                                void* workspace, size_t workspace_bytes, void* stream);

/* Canonical copy of layer `layer`'s sign bits to HOST memory: uint32 words [rows][ceil(n/32)],
 * rows = B (dense) or B*H*W (conv), bit (j & 31) of word (j >> 5) = (z_j > 0).  Synchronises
 * the stream.  `rows_out`/`words_per_row_out` may be NULL. */
mw_status mw_export_masks(const mw_net* net, const void* workspace, int32_t layer,
                          uint32_t* host_words, size_t host_words_capacity, int32_t* rows_out,
                          int32_t* words_per_row_out, void* stream);

/* Synchronise `stream`, then return the first device-side error recorded in the workspace
 * (MW_OK if none) and clear it.  `detail` (may be NULL) receives kernel-specific words. */
mw_status mw_last_device_status(const mw_net* net, void* workspace, void* stream,
                                uint32_t detail[4]);

const char* mw_status_string(mw_status s);

/* ---- stand-alone forms of the residual-store and elementwise kernels ------------------- */

/* Sign-bit pack (Section "Residual Impact"): words[r][w] bit b = (z[r][32 w + b] > 0).
 * z: device [rows][cols], dtype 0 = double, 1 = float, 2 = bf16; cols need not be a multiple of
 * 32 (padding bits are zero).  words: device uint32 [rows][ceil(cols/32)]. */
mw_status mw_pack_sign_bits(const void* z, int32_t dtype, int64_t rows, int32_t cols,
                            uint32_t* words, void* stream);

/* ReLU fragment store (Section 5.1 applied to ReLU): for every row r, the output-cotangent
 * values at dead units (mask bit 0), in increasing column order, are written from
 * vals[off[r]]; cnt[r] = number of dead units, off = exclusive prefix sum of cnt over rows.
 * h: device float [rows][cols]; words: sign bits as above; cnt, off: device uint32[rows];
 * vals: device float, capacity >= rows*cols.  total_out (device uint32, may be NULL) = sum cnt.
 * scratch: device, >= 4*(rows+1024) bytes. */
mw_status mw_relu_fragment_compact(const float* h, const uint32_t* words, int64_t rows,
                                   int32_t cols, uint32_t* cnt, uint32_t* off, float* vals,
                                   uint32_t* total_out, void* scratch, size_t scratch_bytes,
                                   void* stream);

/* Activation vijp (Eq. "h_i" restricted to phi): h_out = g_z (bit 1) or g_z / slope (bit 0) for
 * leaky-ReLU; for ReLU (act = MW_ACT_RELU) live units take g_z and dead units pop
 * vals[off[r] + rank], and gz_out (may be NULL) receives g_z with exact zeros at dead units. */
mw_status mw_activation_vijp(const float* gz, const uint32_t* words, int64_t rows, int32_t cols,
                             int32_t act, float slope, const uint32_t* off, const float* vals,
                             float* h_out, float* gz_out, void* stream);

/* Tensor-core product used by every dense step, exposed for unit parity tests:
 *   D[M][N] (float, row-major) = A * B with A given as [M][K] (a_mn = 0) or [K][M] (a_mn = 1)
 *   and B given as [N][K] (b_mn = 0) or [K][N] (b_mn = 1), all row-major float in device
 *   memory.  terms = 1, 2 or 3: each operand is split into that many bf16 terms and the
 *   1, 3 or 6 leading cross products are accumulated in fp32 (terms = 3 is fp32-accurate).
 *   scratch: device, >= 6*(M*K + N*K) bytes + 1024.  M, N, K multiples of 64. */
mw_status mw_gemm_split_bf16(const float* A, int32_t a_mn, const float* B, int32_t b_mn, float* D,
                             int32_t M, int32_t N, int32_t K, int32_t terms, void* scratch,
                             size_t scratch_bytes, void* stream);

/* The three convolution steps of a stride-1, same-size, 64-channel layer on the tensor cores,
 * exposed for unit parity tests (Lemma 1; Eq. "conv-vjp"; Eq. "g_i"):
 *   op 0  forward        out[b,i',c'] = sum_{j,c} w[j,c,c'] a[b,i'+j-p,c]      a = x, b = w
 *   op 1  TransposeConv  out[b,i,c]   = sum_{j,c'} w[j,c,c'] a[b,i+p-j,c']     a = h', b = w
 *   op 2  weight vjp     out[j,c,c']  = sum_{b,i'} a[b,i'+j-p,c] b[b,i',c']    a = x, b = g_z
 * Pixel arrays are channel-last float [images][H][W][64], kernels float [k][k][64][64], p = k/2,
 * zero padding; all device memory.  terms as in mw_gemm_split_bf16.  Sizes: 128 % W == 0 (64 % W
 * == 0 for op 2), H*W % 128 == 0, k odd.  scratch: device, 256-byte aligned, >= 1024 + 8*terms*
 * (elements of a + elements of b) bytes (+ 256 * k*k*16 KiB for op 2).  Synchronises `stream`. */
mw_status mw_conv2d_split_bf16(int32_t op, const float* a, const float* b, float* out,
                               int32_t images, int32_t H, int32_t W, int32_t k, int32_t terms,
                               void* scratch, size_t scratch_bytes, void* stream);

/* The same three steps for a k x k convolution with C channels in and out (C a multiple of 64),
 * stride s and zero padding p (Lemma 1's general form; Section "Fully Parallel Submersive 2D CNN"
 * uses k = 3, s = 2, p = 1, C = 128): Ho = (H + 2p - k)/s + 1, Wo likewise,
 *   op 0  out[images][Ho][Wo][C] = sum_{j,c} w[j,c,c'] a[b, s i' + j - p, c]      a = x [images][H][W][C], b = w
 *   op 1  out[images][H][W][C]   = sum_{j,c'} w[j,c,c'] hbar'[b, i + p - j, c']   a = h' [images][Ho][Wo][C], b = w;
 *         hbar' is h' dilated by s (Eq. "conv-vjp").  s = 1 (k = 2p + 1), or s = 2 with H = 2 Ho, W = 2 Wo.
 *   op 2  out[k][k][C][C]        = sum_{b,i'} a[b, s i' + j - p, c] b[b, i', c']   a = x, b = g_z [images][Ho][Wo][C]
 * A tile of 128 consecutive product pixels (64 for op 2) must be part of an image row, whole rows
 * of one image, or whole images (widths and heights that are powers of two up to 256 qualify);
 * images*Ho*Wo % 64 == 0 for op 2.  Otherwise MW_ERR_UNSUPPORTED.  scratch: device, 256-byte
 * aligned, >= 1024 + 8*terms*(elements of a + elements of b) + (op 2: 1024 * k*k*C*C) bytes.
 * Synchronises `stream`. */
mw_status mw_conv2d_strided_split_bf16(int32_t op, const float* a, const float* b, float* out,
                                       int32_t images, int32_t H, int32_t W, int32_t C, int32_t k,
                                       int32_t stride, int32_t pad, int32_t terms, void* scratch,
                                       size_t scratch_bytes, void* stream);

/* The same product as mw_gemm_split_bf16 for callers that have no scratch buffer to lend and
 * cannot allocate one when they call: code that runs inside a host framework whose memory pool
 * owns the whole device (a direct cudaMalloc there fails or stalls every stream), and services
 * with a fixed memory plan that forbid allocation after start-up.  (The paper has no counterpart;
 * this is a convenience of the library.)
 *   A, B, D, M, N, K, terms, a_mn, b_mn: exactly as in mw_gemm_split_bf16; the caller still owns
 *   the inputs and the output.
 * The scratch (status block + bf16 term planes of A and B) lives in an array built into the
 * library, MW_GEMM_STATIC_SCRATCH_BYTES per GPU, held by every GPU that loads the library until
 * the process exits.  Sizes that need more, 256 + 2*terms*(M*K + N*K) bytes (+ padding), are
 * rejected with MW_ERR_WORKSPACE before any GPU work.  The call itself allocates nothing on host
 * or device and frees nothing.
 * The first call on a device looks up the array's device address (with that device current); make
 * that first call before any stream capture begins.
 * All calls on one GPU share the array, which keeps the previous call's contents; the entry point
 * clears the part that must start at zero.  Two calls whose GPU work overlaps (different streams,
 * or threads) race on it: serialise them.  Synchronises `stream` before returning. */
#define MW_GEMM_STATIC_SCRATCH_BYTES (16u << 20)
mw_status mw_gemm_split_bf16_static(const float* A, int32_t a_mn, const float* B, int32_t b_mn,
                                    float* D, int32_t M, int32_t N, int32_t K, int32_t terms,
                                    void* stream);

/* ---- whole step from host buffers, and measurement hooks --------------------------------- */

/* One Moonwalk gradient step (Algorithm 1 with Phases I-II in front) whose per-step inputs
 * arrive in HOST memory: copies x and the loss target to the caller's device staging buffers
 * (x_dev, target_dev), runs mw_input_cotangent and mw_forward_sweep, copies the loss back to
 * loss_host and synchronises the stream.  params, dW_out, g0_dev, loss_dev, workspace: device,
 * as in the calls above.  Use pinned host memory for asynchronous copies. */
mw_status mw_gradient_step_host(mw_net* net, const void* const* params, const void* x_host,
                                size_t x_bytes, const void* target_host, size_t target_bytes,
                                void* x_dev, void* target_dev, void* g0_dev, void* const* dW_out,
                                double* loss_dev, double* loss_host, void* workspace,
                                size_t workspace_bytes, void* stream);

/* Number of kernel launches this library has enqueued since it was loaded (host-side count;
 * the paper has no counterpart: bookkeeping for benchmarks). */
int64_t mw_launch_count(void);

/* Between mw_profile_begin() and mw_profile_end() every launch of the tensor-core product
 * kernel is bracketed by CUDA events on its stream.  mw_profile_end() waits for them and
 * returns the summed kernel time, the number of launches, the algorithmic flops (2*M*N*K per
 * product) and the flops the tensor cores executed (times the number of term pairs).  Not
 * thread-safe; meant for benchmarks (the paper has no counterpart). */
void mw_profile_begin(void);
mw_status mw_profile_end(double* total_ms, int64_t* launches, double* flops, double* mma_flops);

/* Self-test of the bounded device-side waits (failure detection): launches one small product that
 * depends on something no product of its launch ever completes, with every wait of that launch
 * bounded by limit_ms (1..1000) instead of the usual 2 s.  The waiting lane must give up, record
 * MW_ERR_TIMEOUT and unwind the CTA (other roles leave, tensor memory is released) so that the
 * kernel ends and the context stays usable.  *timed_out_status receives the status the launch
 * recorded (MW_ERR_TIMEOUT when the path works); the return value is that of the host calls.
 * scratch: device, 256-byte aligned, >= 256 KiB; the status block inside it is cleared again.
 * Synchronises `stream`.  (The paper has no counterpart.) */
mw_status mw_selftest_bounded_wait(void* scratch, size_t scratch_bytes, uint32_t limit_ms,
                                   int32_t* timed_out_status, void* stream);

/* The tensor-core product kernel has two forms: one CTA per 128-row tile, and a pair of CTAs (a
 * cluster of two SMs, tcgen05 cta_group::2) per 256-row tile that stage half of the B tile each.
 * Launches whose products all qualify (operands of at most two bf16 terms, M a multiple of 256,
 * N of 128) use the pair form.  enable = 0 turns it off for the launches that follow, 1 (the
 * default) turns it back on; returns the previous setting.  Process-wide; for comparisons and
 * tests (the paper has no counterpart). */
int32_t mw_set_pair_mode(int32_t enable);

/* Pair form, operands of two bf16 terms: with enable = 1 (the default) the three kept cross
 * products of a tile accumulate in one block of 256 accumulator columns (full-width tensor-core
 * instructions); with 0 the leading product and the two first-order products have blocks of
 * their own, added in the epilogue (tiles of 128 columns).  Returns the previous setting.
 * Process-wide; for comparisons and tests (the paper has no counterpart). */
int32_t mw_set_merge_orders(int32_t enable);

/* Whole phases run as one launch whose products wait for one another, which needs every CTA
 * resident: such launches carry the cooperative-launch attribute (enable = 1, the default).  A
 * profiler that cannot replay a cooperative launch of clusters can have it left out (0); the grid
 * never exceeds what the device holds at once, so on an otherwise idle GPU nothing changes.
 * Returns the previous setting.  Process-wide (the paper has no counterpart). */
int32_t mw_set_cooperative_launch(int32_t enable);

/* Epilogues of the product kernel hand outputs that are plain [M][N] arrays to the copy engine
 * (staged in shared memory, cp.async.bulk.tensor stores; enable = 1, the default) or write them
 * with per-lane 16-byte stores (0), as scattered outputs always are.  Returns the previous
 * setting.  Process-wide; for comparisons and tests (the paper has no counterpart). */
int32_t mw_set_bulk_epilogue(int32_t enable);

/* Dense nets with resident inverses run the forward sweep (Algorithm 1) as chains: per block of
 * batch rows, layer l's recompute and vijp wait only for the same rows of layer l - 1, all inside
 * one launch (enable = 1, the default): on CTA pairs with row blocks of 256 when a layer has at
 * least 32 such tiles per product, else on single CTAs with row blocks of 128.  2: CTA pairs
 * whenever the sizes allow.  0: one launch per layer instead.  Returns the previous setting.
 * Process-wide; read when a net's sweep is first built (a net keeps the form it
 * started with); for comparisons and tests (the paper has no counterpart). */
int32_t mw_set_sweep_chains(int32_t enable);

#ifdef __cplusplus
}
#endif
#endif /* MOONWALK_H_ */
