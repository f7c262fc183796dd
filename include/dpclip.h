/*
 * dpclip.h -- C ABI of libdpclip: per-example gradient clipping for DP-SGD on
 * one B200 (sm_100a), after Lee & Kifer, "Scaling up Differentially Private
 * Deep Learning with Fast Per-Example Gradient Clipping".
 *
 * Problem statement (paper, Sec. "algorithm": per layer the method needs only
 * the gradient w.r.t. the pre-activations and the layer's input):
 *
 *   layer l, example i:  A_i   in R^{T x d_in}    layer input rows
 *                        Zb_i  in R^{T x d_out}   dLoss_i/dZ rows, as given (no hidden 1/tau)
 *     T = 1 dense layer (Algorithm 2), T = H'W' im2col patches for a convolution
 *     (Algorithm 3), T = sequence length for recurrent/LSTM layers (Algorithm 4)
 *     and attention projections (Sec. "Multi-head attention").
 *   per-example gradient  G_i  = sum_t zb_{i,t} (outer) a_{i,t}   (d_out x d_in)
 *                         gb_i = sum_t zb_{i,t}                    (bias)
 *   norm    n_i = sqrt( sum_l ||G_{i,l}||_F^2 + ||gb_{i,l}||^2 )   (text after Eq. "weighted_loss")
 *   factor  c_i = min(1, C / n_i)                                  (Eq. "per_example_weight")
 *   release sum_i c_i G_i (+ bias)  + N(0, sigma^2 C^2)            (Algorithm 1, last line, as a SUM)
 *
 * The library never writes a per-example gradient or a Gram matrix to global
 * memory.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the parameter comment says "host".
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *     Calls only enqueue work; they never synchronise the stream.
 *   - The caller owns every buffer, including the workspace.  The library
 *     allocates no device memory, and no result depends on an earlier call.
 *     What the process keeps between calls is bookkeeping only: an atomic
 *     launch counter (dpclip_launch_count), the path-switch mask read once
 *     from the environment (dpclip_reload_path_switches), per-device kernel
 *     attributes set at a kernel's first launch, and the device address of
 *     dpclip_clipped_grad_noalloc's fixed array.  Entry points may be called
 *     from several host threads.  A
 *     workspace holds scratch (partial tiles) and, in its header, a status
 *     word, the grid-barrier counter of the one-launch T = 1 step and the
 *     item counter of the Gram kernel for T = 256 (both return to zero by
 *     themselves when a launch completes): calls that may run at the same
 *     time (different streams) need workspaces of their own; calls ordered
 *     on one stream can share one.
 *   - Layout: A is B x T x d_in with row stride `lda` ELEMENTS (>= d_in), rows
 *     of one example contiguous (example i starts at row i*T); Zbar likewise
 *     with `ldz`.  Outputs are fp32; gW is d_out x d_in row-major with row
 *     stride `ldg` (>= d_in), the layout of a dense weight [out, in] or of a
 *     convolution weight flattened to [c_out, c_in*k*k].
 *   - Return value: DPCLIP_OK or a negative dpclip_status.  Argument errors
 *     are detected on the host before anything is launched.  A device-side
 *     bounded wait that ran out sets a status word in the workspace header
 *     (see dpclip_read_status); the kernel then exits, it never traps.
 *   - NaN/Inf inputs propagate; nothing is screened.
 */
#ifndef DPCLIP_H_
#define DPCLIP_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { DPCLIP_F32 = 0, DPCLIP_BF16 = 1 } dpclip_dtype;

/* How a layer's squared norms are computed.  AUTO picks T1 when T == 1 and
 * otherwise the cheaper exact form by flop count, restricted to the forms the
 * shape and alignment allow. */
typedef enum {
    DPCLIP_AUTO = 0,
    DPCLIP_T1 = 1,           /* ||a||^2 ||zb||^2, Goodfellow's closed form (Sec. "Fully-connected Layers") */
    DPCLIP_GRAM = 2,         /* sum_{t,s} (a_t.a_s)(zb_t.zb_s): Gram tiles on the tensor cores (bf16)        */
    DPCLIP_MATERIALIZE = 3,  /* ||Zb_i^T A_i||_F^2 with the tile held on chip, Frobenius sum in the epilogue   */
    DPCLIP_SIMT = 4          /* MATERIALIZE on the fp32 ALUs (any dtype, any alignment)                        */
} dpclip_method;

typedef enum {
    DPCLIP_OK = 0,
    DPCLIP_ERR_INVALID_ARG = -1,      /* null pointer, non-positive size, stride < width          */
    DPCLIP_ERR_UNSUPPORTED = -2,      /* method not available for this dtype / shape / alignment   */
    DPCLIP_ERR_MISALIGNED = -3,       /* pointer not aligned to its element size                   */
    DPCLIP_ERR_WORKSPACE = -4,        /* workspace NULL or smaller than dpclip_workspace_bytes()   */
    DPCLIP_ERR_CUDA = -5,             /* a CUDA runtime/driver call or a launch failed              */
    DPCLIP_ERR_TIMEOUT = -6,          /* (device status) a bounded wait inside a kernel ran out     */
    DPCLIP_ERR_RANGE = -7             /* (device status, -DDPCLIP_DEBUG builds only) an index left its
                                         buffer; the access was skipped, the kernel went on          */
} dpclip_status;

/* Squared per-example gradient norm of ONE layer, for every example:
 *   sq_layer[i] = || sum_t zb_{i,t} (outer) a_{i,t} ||_F^2  (+ || sum_t zb_{i,t} ||^2 if has_bias).
 * T = 1 is Goodfellow's closed form; T > 1 follows Algorithms 3-4 (the sum
 * over t is taken BEFORE the norm) without storing G_i.
 *   A, Zbar   inputs as described above, dtype `dtype` (bf16 = raw 16-bit payload)
 *   sq_layer  [B] fp32, OVERWRITTEN (row l of the caller's [L][B] array)
 *   workspace >= dpclip_workspace_bytes(...) bytes, 256-byte aligned; its first
 *             256 bytes are the status header (see dpclip_workspace_init).
 * Errors: INVALID_ARG for B, T, d_in or d_out <= 0, lda < d_in, ldz < d_out or
 * null pointers; UNSUPPORTED when `method` cannot run this dtype/shape (e.g.
 * T1 with T > 1, GRAM with fp32 inputs or rows not a multiple of 16 bytes). */
int dpclip_layer_sqnorms(const void* A, long lda, const void* Zbar, long ldz,
                         int B, int T, int d_in, int d_out,
                         dpclip_dtype dtype, int has_bias, dpclip_method method,
                         float* sq_layer, void* workspace, size_t workspace_bytes, void* stream);

/* Cross-layer accumulate and clip factors (the norm of the whole per-example gradient is the root of
 * the sum of the per-layer squared norms: text after Eq. "weighted_loss"; the factor is Eq.
 * "per_example_weight", nu_i = min(1, c / ||g_i||), equal to the clip_c definition of Sec. "Preliminaries"):
 *   norms[i] = sqrt(sum_l sq_layers[l*ld_sq + i]),  clip[i] = 1 if norms[i] <= C else C / norms[i].
 * The stored factor is exactly 1.0f for an unclipped example (including a zero
 * norm).  norms and n_clipped may be NULL; n_clipped[0] receives the number
 * of examples with clip < 1.  Errors: INVALID_ARG for L, B <= 0, C <= 0 or
 * ld_sq < B. */
int dpclip_factors(const float* sq_layers, int L, long ld_sq, int B, float C,
                   float* clip, float* norms, int* n_clipped, void* stream);

/* Clipped sum of ONE layer (the weight-gradient product of Algorithm 1's
 * reweighted backward pass, with the per-example weight applied while the
 * operand is loaded):
 *   gW[o][k] = sum_i clip[i] sum_t zb_{i,t}[o] a_{i,t}[k],   gb[o] = sum_i clip[i] sum_t zb_{i,t}[o].
 *   clip  [B] fp32, or NULL for all ones (the plain batch gradient Zbar^T A)
 *   gW    d_out x d_in fp32, row stride ldg, OVERWRITTEN;  gb [d_out] or NULL, OVERWRITTEN
 * bf16 layers whose rows are 16-byte multiples take the tensor-core path: rows
 * are split over CTAs, partial tiles go to the workspace and are added in a
 * fixed order (bit-reproducible).  Other layers take the fp32-ALU path, which
 * combines row slices with fp32 atomic adds (low-order bits may vary). */
int dpclip_clipped_grad(const void* A, long lda, const void* Zbar, long ldz,
                        int B, int T, int d_in, int d_out, dpclip_dtype dtype,
                        const float* clip, float* gW, long ldg, float* gb,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Element-wise parameter layers h = gamma (.) hbar + beta (Sec. "LayerNorm Layers" and its
 * Algorithm, G = Z (.) H): per example the gradients are
 *   ggamma_i = sum_t zb_{i,t} (.) hbar_{i,t}   and   gbeta_i = sum_t zb_{i,t},
 * the sum over the T positions that share gamma and beta being taken before the norm.
 *   Hbar, Zbar  device, [B*T][ld] row-major, dtype `dtype`: the NORMALISED layer input and the
 *               back-propagated signal of the layer output (the caller normalises; the library
 *               never sees mean or variance)
 *   sq_layer    [B] fp32, OVERWRITTEN with ||ggamma_i||^2 (+ ||gbeta_i||^2 when has_shift): one
 *               more row of the [L][B] array that dpclip_factors sums
 *   clip        [B] or NULL (all ones)
 *   g_scale     [d] fp32, OVERWRITTEN with sum_i clip[i] ggamma_i
 *   g_shift     [d] fp32 or NULL, OVERWRITTEN with sum_i clip[i] gbeta_i
 * Noise is added with dpclip_add_noise on g_scale / g_shift.  No workspace; partial sums of a
 * column are combined with fp32 atomics, so the last bits depend on the order of arrival.
 * Errors as for dpclip_layer_sqnorms. */
int dpclip_elementwise_sqnorms(const void* Hbar, long ldh, const void* Zbar, long ldz,
                               int B, int T, int d, dpclip_dtype dtype, int has_shift,
                               float* sq_layer, void* stream);
int dpclip_elementwise_clipped_grad(const void* Hbar, long ldh, const void* Zbar, long ldz,
                                    int B, int T, int d, dpclip_dtype dtype,
                                    const float* clip, float* g_scale, float* g_shift, void* stream);

/* Gaussian mechanism: g[j] += sigma * C * xi_j for j in [0, n), xi_j ~ N(0,1).
 * The paper names no generator.  This library uses Philox4x32-10 with key =
 * (seed lo, seed hi) and counter = (q lo, q hi, stream_id lo, stream_id hi),
 * q = j / 4; word w of the block maps to u = fma(float(w), 2^-32, 2^-33) in
 * (0,1]; Box-Muller on words (0,1) gives elements 4q (cos) and 4q+1 (sin),
 * words (2,3) give 4q+2 and 4q+3.  The result depends only on (seed,
 * stream_id, j): no generator state is kept, and a (seed, stream_id) pair must
 * not be reused for two tensors.  n == 0 is a no-op.  Errors: INVALID_ARG for
 * a null g with n > 0 or negative sigma or C.
 * Limitation: the draws are an fp32 approximation of N(0,1), not exact Gaussians.  u lies on a 2^-32
 * grid with minimum 2^-33, so |xi| <= sqrt(2 ln 2^33) = 6.76 and every draw is one of finitely many
 * values; the device's log2 / sqrt / sin / cos approximations put each draw within 1e-5 (absolute, in
 * units of sigma * C) of the value the same u gives in double precision.  The privacy analysis of
 * Algorithm 1 assumes exact Gaussians; the known floating-point caveat of the Gaussian mechanism applies
 * and is not addressed here.
 * Releasing a step: a bounded wait inside a kernel that ran out (DPCLIP_ERR_TIMEOUT in the workspace
 * header) leaves that step's outputs undefined while the enqueueing call has long returned DPCLIP_OK, so
 * check dpclip_read_status() before anything computed by a step leaves the process. */
int dpclip_add_noise(float* g, size_t n, float sigma, float C,
                     unsigned long long seed, unsigned long long stream_id, void* stream);

/* Clipped sum and noise of ONE layer in one call: dpclip_clipped_grad followed by
 * dpclip_add_noise on gW (stream stream_id_w) and on gb (stream stream_id_b),
 * with the noise folded into the last pass over the output where the layer's
 * kernel has one (Algorithm 1, last line: the noised clipped sum is what is
 * released).  gW has dense rows (row stride d_in).  Same results as the two
 * separate calls, bit for bit. */
int dpclip_clipped_grad_noise(const void* A, long lda, const void* Zbar, long ldz,
                              int B, int T, int d_in, int d_out, dpclip_dtype dtype,
                              const float* clip, float* gW, float* gb,
                              float sigma, float C, unsigned long long seed,
                              unsigned long long stream_id_w, unsigned long long stream_id_b,
                              void* workspace, size_t workspace_bytes, void* stream);

/* dpclip_clipped_grad for callers that cannot supply a workspace.  (The paper
 * has no counterpart: this is an interface variant, not a step of the method.)
 *
 * Who needs it: code that cannot obtain device memory at the point of the call
 * -- a plug-in inside an application that owns all GPU memory, a server whose
 * pool is fixed at start-up, or a caller already inside a region where device
 * allocation is not allowed.  The scratch the split-row clipped sum needs is a
 * fixed 16 MB array inside the library image instead; every GPU that loads the
 * library holds it until the process exits.
 *
 * Same arguments, results and tolerances as dpclip_clipped_grad, minus the
 * workspace.  Limits and rules:
 *   - the output, padded to 256 x 256 tiles, must be at most
 *     dpclip_noalloc_max_output_bytes() (8 MB, e.g. 1024 x 2048 fp32);
 *     larger layers return DPCLIP_ERR_WORKSPACE and nothing is launched.  The
 *     row split over SMs is clamped to what the array holds (one partial tile
 *     per output tile and one per run of rows): small outputs run as wide as
 *     dpclip_clipped_grad, an output at the limit on a fifth of the SMs;
 *   - no device memory is allocated or freed by this call, on any path;
 *   - the first call on each device looks up the array's device address (that
 *     device must be current); make that first call outside any stream capture;
 *   - all calls share the one array: two calls whose kernels may overlap on
 *     the GPU (different streams, no ordering between them) race on it;
 *   - a bounded-wait timeout inside the kernel is recorded in the array's
 *     header, which this call clears at its start; there is no read-back
 *     entry for it. */
int dpclip_clipped_grad_noalloc(const void* A, long lda, const void* Zbar, long ldz,
                                int B, int T, int d_in, int d_out, dpclip_dtype dtype,
                                const float* clip, float* gW, long ldg, float* gb, void* stream);
size_t dpclip_noalloc_max_output_bytes(void);

/* One layer of a whole step. */
typedef struct {
    const void* A;  long lda;       /* B x T x d_in  */
    const void* Zbar; long ldz;     /* B x T x d_out */
    int T, d_in, d_out;
    int has_bias;
    int method;                     /* dpclip_method for the norm */
    float* gW; long ldg;            /* d_out x d_in, overwritten with the noised clipped sum */
    float* gb;                      /* [d_out] or NULL when has_bias == 0 */
} dpclip_layer;

/* The whole path over L layers on one stream: per-layer squared norms ->
 * factors -> per-layer clipped sums -> noise on every released coordinate
 * (weights of layer l use noise stream stream_id0 + 2l, its bias + 2l + 1).
 *   layers     host array of L descriptors whose pointers are device pointers
 *   sq_layers  [L][B] fp32 scratch/outputs, clip [B], norms [B] or NULL
 *   workspace  >= the largest dpclip_workspace_bytes() over the layers
 * Output rows must be dense (ldg == d_in; UNSUPPORTED otherwise) because the
 * noise is indexed by the element's position in the dense tensor.
 * A model whose layers all have T = 1 runs as ONE cooperative launch when its
 * input rows are 16-byte multiples (4 fp32 / 8 bf16 elements; the zb rows of
 * a layer with at most 16 outputs excepted): norms, a grid-wide barrier with a
 * bounded wait, factors, clipped sums on the tensor cores, noise; else as two
 * launches; other models run layer by layer, their T = 1 layers together. */
int dpclip_step(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                float C, float sigma, unsigned long long seed, unsigned long long stream_id0,
                float* sq_layers, float* clip, float* norms,
                void* workspace, size_t workspace_bytes, void* stream);

/* dpclip_step with the launches of a stage spread over several streams INSIDE the library (Algorithm 1
 * fixes only the order norms -> factors -> clipped sums; within the norm stage and within the clipped-sum
 * stage the layers are independent, so one layer's kernel can start on the SMs another layer's kernel has
 * already left).  Same arguments and results as dpclip_step, bit for bit, except:
 *   streams     host array of n_streams (1..8) distinct cudaStream_t.  streams[0] is the caller's stream:
 *               the step waits for nothing but what is already enqueued there, and when the call returns
 *               everything the step enqueued, on any stream, is ordered before whatever the caller enqueues
 *               on streams[0] next.  The other streams are used only between the library's own fork
 *               (event record on streams[0] + waits) and join (event records + waits on streams[0]); they
 *               must not be capturing or busy with work that conflicts with the step's buffers.
 *   workspaces  host array of n_streams distinct device buffers of `workspace_bytes` each (the size
 *               dpclip_step wants), each initialised once with dpclip_workspace_init; launches on different
 *               streams overlap, so they cannot share scratch.  Check every one with dpclip_read_status.
 * The call creates and destroys a few CUDA events (no device memory).  It may be recorded into a CUDA
 * graph by capturing streams[0]: the fork and join become graph dependencies, and the benchmark's step is
 * exactly one such call.  n_streams == 1 is dpclip_step.  All-T=1 models take the one-launch step on
 * streams[0] whatever n_streams is.  Errors as dpclip_step; INVALID_ARG for n_streams outside 1..8 or
 * repeated streams / workspaces. */
int dpclip_step_streams(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                        float C, float sigma, unsigned long long seed, unsigned long long stream_id0,
                        float* sq_layers, float* clip, float* norms,
                        int n_streams, void* const* streams /* host */, void* const* workspaces /* host */,
                        size_t workspace_bytes);

/* Convolution layers given by their INPUT feature map (implicit im2col).  Algorithm 3 unfolds the input into
 * the patch matrix (kh * kw copies of every pixel) and reshapes dL/dZ to [tau, c_out, T]; here element
 * (row (i, t), column (c, ky, kx)) of that matrix is read straight from
 *   X[i][c][y' * stride - pad + ky][x' * stride - pad + kx]   (zero outside the map), t = y' * W' + x',
 * so the unfolded copy never exists, and dL/dZ can be passed as it comes out of back-propagation.
 *   X       device, [B][C][H][W] contiguous, dtype `dtype`
 *   Zbar    device, [B][T][d_out] (z_channel_major = 0) or [B][d_out][T] (= 1, i.e. [B][c_out][H'][W']),
 *           T = H' * W', H' = (H + 2 pad - kh) / stride + 1, likewise W'
 *   sq_layer, clip, gW, gb  as for dpclip_layer_sqnorms / dpclip_clipped_grad; gW is [d_out][C*kh*kw] with
 *           columns ordered (c, ky, kx), c slowest: a convolution weight [c_out][c_in][kh][kw] flattened
 * Square or rectangular kernels, any stride and zero padding; dilation 1.  fp32 layers with dL/dZ as
 * [B][T][d_out] (rows 16-byte multiples) above 2^25 multiply-adds run on the tensor cores (error-
 * compensated tf32, the patch rows gathered by the warps that prepare the operand planes) and need a
 * workspace of dpclip_workspace_bytes(B, T, C*kh*kw, d_out, ...) bytes.  bf16 layers (dL/dZ in either
 * layout) also run on the tensor cores when the stride is 1, the output width is 8, 16, 32 or 64, T is a
 * multiple of 64, d_out a multiple of 8 and at most 128, a feature map (C*H*W) at most 32 KB and a multiple of
 * 16 bytes, X and Zbar 16-byte aligned, and a workspace is given (its header for the norms; the partial tiles
 * for the clipped sum): the feature map of an example is copied to shared memory once and the patch tiles are
 * built there.  Everything else, and any call with workspace == NULL, runs on fp32-ALU tiles (64 x 64) and
 * combines the partial sums of split rows with fp32 atomics.  Noise is added with dpclip_add_noise.  Errors as for dpclip_layer_sqnorms. */
typedef struct { int C, H, W, kh, kw, stride, pad; } dpclip_conv;
int dpclip_conv_sqnorms(const void* X, const void* Zbar, int z_channel_major, int B, const dpclip_conv* geom,
                        int d_out, dpclip_dtype dtype, int has_bias, float* sq_layer,
                        void* workspace, size_t workspace_bytes, void* stream);
int dpclip_conv_clipped_grad(const void* X, const void* Zbar, int z_channel_major, int B, const dpclip_conv* geom,
                             int d_out, dpclip_dtype dtype, const float* clip, float* gW, long ldg, float* gb,
                             void* workspace, size_t workspace_bytes, void* stream);
/* Workspace for the two calls above: dpclip_workspace_bytes() of the layer's patch-matrix shape, plus, for
 * fp32 layers with dL/dZ channel-major that are large enough for the tensor cores, B*T*d_out*4 bytes for a
 * [B][T][d_out] copy of dL/dZ (written by a transpose kernel at the start of each call; with less workspace
 * the call still works and reads dL/dZ in place on the fp32-ALU kernel). */
size_t dpclip_conv_workspace_bytes(int B, const dpclip_conv* geom, int d_out, dpclip_dtype dtype, int z_channel_major);

/* Per-layer clipping: every layer's per-example gradient is clipped to its own threshold C_layer[l] (for
 * instance C / sqrt(L), so that the concatenated gradient stays within C), the variant that per-layer norms
 * make possible (Sec. "Related Work", per-layer clipping).  The stages of dpclip_step with a factor vector per
 * layer: squared norms of every layer -> factors of layer l from row l alone, against C_layer[l] -> clipped sums,
 * layer l with its own factors -> noise N(0, sigma^2 * sum_l C_layer[l]^2) on every coordinate (the
 * sensitivity of the concatenated clipped gradient), streams stream_id0 + 2l / + 2l + 1 as in dpclip_step.
 * The launches several layers share under global clipping (Gram norms; the clipped sums of wide bf16 layers)
 * are shared here too.
 *   C_layer       host [L], each > 0
 *   sq_layers     [L][B], clip_layers [L][B] (row l = layer l's factors), norms_layers [L][B] or NULL
 * workspace >= dpclip_step_workspace_bytes().  Errors as for dpclip_step. */
int dpclip_step_per_layer(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                          const float* C_layer /* host */, float sigma,
                          unsigned long long seed, unsigned long long stream_id0,
                          float* sq_layers, float* clip_layers, float* norms_layers,
                          void* workspace, size_t workspace_bytes, void* stream);

/* The whole path over a model whose layers are not all dense products: Algorithm 1 with the per-layer
 * gradients of Sec. "Fully-connected", "Convolutional" and "LayerNorm" layers in one call.
 *   kind DPCLIP_KIND_DENSE       `layer` as in dpclip_step.
 *   kind DPCLIP_KIND_ELEMENTWISE gain/shift of a normalisation layer: layer.A = hbar [B][T][d] (lda),
 *                                layer.Zbar = dL/dh [B][T][d] (ldz), d_in = d_out = d, has_bias = the layer
 *                                has a shift, gW = the gain's gradient [d], gb = the shift's [d]; ldg, method
 *                                unused.
 *   kind DPCLIP_KIND_CONV        convolution given by its input feature map: layer.A = X [B][C][H][W] dense,
 *                                layer.Zbar = dL/dZ ([B][Ho*Wo][d_out], or [B][d_out][Ho*Wo] when
 *                                z_channel_major), `conv` the geometry, gW [d_out][C*kh*kw] with ldg =
 *                                C*kh*kw, gb [d_out]; lda, ldz, T, d_in, method unused.
 * Row l of sq_layers [L][B] and the noise streams stream_id0 + 2l (gW) and + 2l + 1 (gb) belong to layer l
 * whatever its kind; factors and norms are over all L layers.  Dense layers take the same launches as in
 * dpclip_step (a model of dense layers only IS dpclip_step); the other kinds run through their per-layer
 * entry points followed by dpclip_add_noise.  workspace >= dpclip_model_workspace_bytes().  L <= 256.
 * Errors as for the per-layer entry points; INVALID_ARG for an unknown kind or d_in != d_out in an
 * element-wise layer; UNSUPPORTED for padded output rows. */
typedef enum { DPCLIP_KIND_DENSE = 0, DPCLIP_KIND_ELEMENTWISE = 1, DPCLIP_KIND_CONV = 2 } dpclip_layer_kind;
typedef struct {
    int kind;                       /* dpclip_layer_kind */
    dpclip_layer layer;
    dpclip_conv conv;               /* kind CONV */
    int z_channel_major;            /* kind CONV */
} dpclip_model_layer;
int dpclip_model_step(const dpclip_model_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                      float C, float sigma, unsigned long long seed, unsigned long long stream_id0,
                      float* sq_layers, float* clip, float* norms,
                      void* workspace, size_t workspace_bytes, void* stream);
size_t dpclip_model_workspace_bytes(const dpclip_model_layer* layers /* host */, int L, int B, dpclip_dtype dtype);
/* dpclip_model_step over several streams: streams, workspaces and rules as for dpclip_step_streams, every
 * workspace of dpclip_model_workspace_bytes() bytes. */
int dpclip_model_step_streams(const dpclip_model_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                              float C, float sigma, unsigned long long seed, unsigned long long stream_id0,
                              float* sq_layers, float* clip, float* norms,
                              int n_streams, void* const* streams /* host */, void* const* workspaces /* host */,
                              size_t workspace_bytes);

/* Parameter updates with the noise folded in (one pass over the parameters instead of a noise pass and
 * an optimiser pass).  gsum is the PRE-noise clipped sum of one tensor (run the step with sigma = 0);
 * the noisy mean gradient is g[j] = (gsum[j] + sigma * C * xi_j) * inv_tau with xi as in dpclip_add_noise
 * for the same (seed, stream_id), inv_tau = 1 / batch size.
 *   dpclip_dp_sgd_step : theta -= lr * g                                  (Algorithm 1, last line)
 *   dpclip_dp_adam_step: m = beta1 m + (1 - beta1) g, v = beta2 v + (1 - beta2) g^2,
 *                        theta -= lr * (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps),
 *                        step counted from 1 (the private Adam of Sec. "Experiments": lr 0.001,
 *                        beta1 0.9, beta2 0.999 there).
 * theta, m, v [n] fp32 updated in place; gsum [n] fp32 read only.  Errors: INVALID_ARG (null pointer,
 * negative sigma or C, inv_tau <= 0, step < 1, beta outside [0, 1)), MISALIGNED. */
int dpclip_dp_sgd_step(float* theta, const float* gsum, size_t n, float inv_tau, float C, float sigma,
                       unsigned long long seed, unsigned long long stream_id, float lr, void* stream);
int dpclip_dp_adam_step(float* theta, float* m, float* v, const float* gsum, size_t n, float inv_tau,
                        float C, float sigma, unsigned long long seed, unsigned long long stream_id,
                        float lr, float beta1, float beta2, float eps, int step, void* stream);

/* Noise on every released tensor of a model in one launch: weights of layer l on noise stream
 * stream_id0 + 2l, its bias on + 2l + 1, exactly as dpclip_step numbers them (dense output rows
 * required).  For callers that add the noise after their own reduction over ranks.
 * sigma * C == 0 launches nothing. */
int dpclip_step_noise(const dpclip_layer* layers /* host */, int L, float C, float sigma,
                      unsigned long long seed, unsigned long long stream_id0, void* stream);

/* The T = 1 layers of a descriptor array taken together (layers with T > 1 are skipped): their
 * squared norms in one launch, written to THEIR rows of sq_layers [L][B]; and, given the factors
 * of the whole model, their clipped sums with the noise (streams stream_id0 + 2l, + 2l + 1 for
 * layer l of the array) in one tensor-core launch.  This is what dpclip_step does for the T = 1
 * layers of a mixed model; the two calls let a caller that spreads the layers of a model over
 * several streams do the same.  Input rows must be 16-byte multiples (the zb rows of a layer
 * with at most 16 outputs excepted), output rows dense, and at least one of the layers must have
 * more than 16 outputs: DPCLIP_ERR_UNSUPPORTED otherwise, and nothing is launched. */
int dpclip_t1_layers_supported(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype); /* 1 or 0 */
int dpclip_t1_layers_sqnorms(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                             float* sq_layers, void* stream);
int dpclip_t1_layers_clipped_grad_noise(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                                        const float* clip, float C, float sigma,
                                        unsigned long long seed, unsigned long long stream_id0,
                                        void* workspace, size_t workspace_bytes, void* stream);

/* The layers of a descriptor array whose norms go by the Gram identity (Section "Extension to
 * recurrent layers" and the attention section: sum over (t, s) of (a_t . a_s)(zb_t . zb_s)), taken
 * together: bf16 layers with T > 1 whose method is DPCLIP_GRAM, or DPCLIP_AUTO resolving to it,
 * and whose rows TMA can address, run in ONE launch per eight layers of a kind (the kinds:
 * T = 256; other T with at most two 128-row blocks per example; longer examples).  Their squared norms go to
 * THEIR rows of sq_layers [L][B].  taken (host, [L], may be NULL) is set to 1 for every layer
 * that was handled and to 0 for the others, which the caller passes to dpclip_layer_sqnorms as
 * before; fewer than two candidates, fp32 input or no workspace: nothing is launched and
 * nothing is taken.  With a small batch (one example per SM) a single layer's launch is a chain
 * of exposed latencies; a queue of items per CTA hides them.  The workspace is used for its
 * status header only. */
int dpclip_gram_layers_sqnorms(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype,
                               float* sq_layers, int* taken /* host, out */,
                               void* workspace, size_t workspace_bytes, void* stream);

/* Clipped sums with noise (Eq. 1 applied to the sum over examples of c_i Zbar_i^T A_i, Algorithm 1's
 * last two steps) of layers taken together: bf16 layers with T > 1, rows TMA can address, dense output
 * rows and d_in a multiple of 4.  Layers with ONE T and d_out wide enough for 512-row tiles (d_out >
 * 256 and little padding) share a launch whatever their shapes, up to eight at a time: their tiles'
 * work is cut into equal runs over all pairs of SMs (needs the workspace dpclip_step_workspace_bytes
 * reports).  Other layers share a launch when they have ONE shape (T, d_in, d_out) and would be short
 * on their own.  Each launch is followed by one reduce launch that adds the noise.  Results and noise streams are those of
 * dpclip_step: layer l of the array draws from streams stream_id0 + 2l (weights) and + 2l + 1
 * (bias).  taken (host, [L], required) is set to 1 for the layers that were handled; the caller
 * runs dpclip_clipped_grad_noise on the others.  Nothing qualifies: nothing is launched.  The
 * launches share `workspace` (one set of partial tiles for the whole group): run them on the
 * stream that owns it. */
int dpclip_same_shape_layers_clipped_grad_noise(const dpclip_layer* layers /* host */, int L, int B,
                                                dpclip_dtype dtype, const float* clip, float C, float sigma,
                                                unsigned long long seed, unsigned long long stream_id0,
                                                int* taken /* host, out */,
                                                void* workspace, size_t workspace_bytes, void* stream);

/* Same, for callers whose tensors live in HOST memory (pinned memory makes the
 * copies asynchronous).  `layers[l].A/Zbar/gW/gb` are HOST pointers with dense
 * rows (lda = d_in, ldz = d_out, ldg = d_in are required).  `arena` is a device
 * buffer of at least dpclip_step_host_arena_bytes() bytes that stages inputs,
 * outputs and the workspace.  host_clip [B] and host_norms [B] (either may be
 * NULL) receive the factors.  All copies and kernels are enqueued on `stream`;
 * the results are valid after the caller synchronises it.
 * Copies are merged when the host tensors of a direction are carved out of one
 * buffer in arena order, each on the next 256-byte boundary: inputs as
 * A_0, Zbar_0, A_1, Zbar_1, ... give ONE host-to-device copy; results as gW_0,
 * gb_0 (its d_out*4-byte slot is kept even without a bias), gW_1, ..., clip,
 * norms give ONE device-to-host copy.  Any other placement is copied tensor by
 * tensor. */
int dpclip_step_host(const dpclip_layer* layers /* host, host pointers inside */, int L, int B,
                     dpclip_dtype dtype, float C, float sigma,
                     unsigned long long seed, unsigned long long stream_id0,
                     float* host_clip, float* host_norms,
                     void* arena, size_t arena_bytes, void* stream);
size_t dpclip_step_host_arena_bytes(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype);

/* Bytes of workspace that dpclip_layer_sqnorms / dpclip_clipped_grad need for
 * this shape: the 256-byte status header, plus, for bf16 layers, room for one
 * fp32 partial tile per SM of the split-row clipped sum (about 39 MB).  Long
 * bf16 layers whose 256 x 256 output tiles do not fill one wave of SMs (64
 * tiles: 128 of 148) are cut into more, shorter row slices that do; the query
 * then reports one partial tile per slice (up to a few hundred MB).  A smaller
 * workspace of at least the 39 MB form is accepted: the layer then runs as one
 * wave. */
size_t dpclip_workspace_bytes(int B, int T, int d_in, int d_out, dpclip_dtype dtype, dpclip_method method);

/* Workspace for dpclip_step / dpclip_step_streams / dpclip_step_per_layer over these layers: the largest
 * per-layer need, and room for the launches several layers share (bf16 layers of one T whose d_out is wide
 * enough for 512-row tiles go into one clipped-sum launch: one fp32 partial tile of 512 x 256 per output tile
 * of all of them and one per pair of SMs).  With less (but at least the per-layer needs) the step still
 * runs, those layers in launches of their own. */
size_t dpclip_step_workspace_bytes(const dpclip_layer* layers /* host */, int L, int B, dpclip_dtype dtype);

/* Zero the 256-byte status header.  Call once after allocating a workspace. */
int dpclip_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Copy the device status word to *host_status (host pointer) and synchronise
 * `stream`.  0 means no kernel reported an anomaly since the header was
 * initialised. */
int dpclip_read_status(const void* workspace, int* host_status /* host */, void* stream);

/* Which form DPCLIP_AUTO resolves to for this layer (a dpclip_method). */
int dpclip_pick_method(int B, int T, int d_in, int d_out, long lda, long ldz, dpclip_dtype dtype);

/* Number of kernels this library has launched in this process (a host-side
 * counter for benchmarks and tests; cudaMemset calls are not counted). */
unsigned long long dpclip_launch_count(void);

/* Launch floor, for benchmarks: enqueue one EMPTY kernel with the launch shape of the one-launch T = 1 step
 * (grid CTAs of 18 warps, its dynamic shared memory; cooperative or plain).  The small all-T=1 workloads
 * (Sec. "Fully-connected Layers": MLPs at batch 32-128) have roofline times below any launch, so their
 * measured step time is reported next to this floor.  (No counterpart in the paper.)  grid in 1..148. */
int dpclip_null_launch(int cooperative, int grid, void* stream);

/* The DPCLIP_* environment switches that force a slower kernel form (for tests and measurements) are read
 * once, at the first call that needs them.  This re-reads them. */
void dpclip_reload_path_switches(void);

const char* dpclip_status_string(int status);
int dpclip_version(void);
/* 1 when the library was compiled with -DDPCLIP_DEBUG (range-checked accesses, see DPCLIP_ERR_RANGE). */
int dpclip_debug_build(void);

#ifdef __cplusplus
}
#endif
#endif /* DPCLIP_H_ */
