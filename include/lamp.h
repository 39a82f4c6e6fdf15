/*
 * lamp.h - C ABI of the B200 (sm_100a) 3-D U-Net convolution library.
 *
 * Scope: the dense 3-D convolutions of a large 3-D U-Net - forward, data
 * gradient and weight gradient - and the U-Net passes around them: one forward
 * pass, one forward+backward training step with a softmax-Dice loss, and
 * whole-volume versus sliding-window inference.  This is the per-device work
 * that the paper's model parallelism spreads over GPUs (Sec. 2.1, Eq. 1: each
 * partition's forward F_k is a chain of such layers, its backward B_k their
 * chain-rule derivative).  The network is the U-Net of Sec. 2.2 (Eq. 2).
 *
 * Conventions (all entry points):
 *  - Every data pointer is a DEVICE pointer unless the comment says "host".
 *    Descriptors (lamp_tensor_t, lamp_conv_desc_t, lamp_unet_spec_t) and the
 *    opaque lamp_unet_t are host objects, read during the call only.
 *  - The caller owns every buffer, including the workspace.  No entry point
 *    allocates or frees device memory.  Outputs are overwritten, never
 *    accumulated into, unless stated.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*; NULL
 *    is the default stream) and return without synchronising.  Errors that
 *    the host can detect return a status and launch nothing.  Conditions only
 *    the device can detect (a bounded wait that ran out) are recorded in a
 *    device-side status word read by lamp_get_async_status().
 *  - Activations are NDHWC, channel-contiguous.  A lamp_tensor_t describes a
 *    channel slice [c_offset, c_offset + c) of a buffer whose voxels are
 *    c_pitch elements apart, so a layer can write straight into its slice of a
 *    skip-concatenation buffer (Sec. 2.2: the skip s_i is a concatenation
 *    along the channel dimension).
 *  - Convolution is cross-correlation with zero padding.  Weights are bf16
 *    w[tap][c_out][c_in] with tap = (kd*k + kh)*k + kw for every variant;
 *    biases are fp32 [c_out].  Accumulation is fp32.  Weight and bias
 *    gradients are fp32.
 *  - Alignment: data pointers 16-byte aligned; for bf16 tensors c, c_pitch and
 *    c_offset are multiples of 8 except where a function says otherwise.
 */
#ifndef LAMP_H_
#define LAMP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LAMP_OK = 0,
    LAMP_ERR_INVALID_ARG = 1,     /* null pointer, negative size, inconsistent shapes            */
    LAMP_ERR_UNSUPPORTED = 2,     /* a combination this library has no kernel for                */
    LAMP_ERR_WORKSPACE = 3,       /* workspace missing, misaligned or smaller than required      */
    LAMP_ERR_CUDA = 4,            /* a CUDA runtime / driver call failed                         */
    LAMP_ERR_TIMEOUT = 5,         /* a bounded device-side wait ran out (see async status)       */
    LAMP_ERR_NOT_IMPLEMENTED = 6,
    LAMP_ERR_SCRATCH_LIMIT = 7    /* the problem needs more than the built-in static scratch     */
} lamp_status_t;

typedef enum { LAMP_BF16 = 0, LAMP_F32 = 1 } lamp_dtype_t;

/* A channel-slice view of an NDHWC device buffer.
 * ptr points at voxel (0,0,0,0), channel 0 of the underlying buffer; the view
 * covers channels [c_offset, c_offset + c) of each voxel; consecutive voxels
 * are c_pitch elements apart (c_pitch >= c_offset + c). */
typedef struct {
    void   *ptr;
    int32_t dtype;       /* lamp_dtype_t */
    int32_t n, d, h, w, c;
    int64_t c_pitch;
    int32_t c_offset;
} lamp_tensor_t;

/* Supported (ksize, stride, pad, transposed): (3,1,1,0) (3,2,1,0) (1,1,0,0) (2,2,0,1). */
typedef struct {
    int32_t c_in, c_out, ksize, stride, pad, transposed;
} lamp_conv_desc_t;

enum { LAMP_PASS_FWD = 0, LAMP_PASS_DGRAD = 1, LAMP_PASS_WGRAD = 2 };

/* ------------------------------------------------------------------------
 * Single-layer convolution passes (the layer functions f_i of Sec. 2.1 and
 * their derivatives).
 * ---------------------------------------------------------------------- */

/* Bytes of workspace with which the given pass runs fastest for input x (for LAMP_PASS_DGRAD,
 * x is the tensor that receives the gradient, i.e. the conv's input shape). */
size_t lamp_conv3d_workspace_bytes(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, int pass);

/* The smallest workspace the pass accepts (a smaller one gives LAMP_ERR_WORKSPACE).  The
 * two differ for forward and data-gradient passes over volumes so small that their tiles do
 * not fill the GPU (the deep levels of the U-Net): given the larger workspace the kernels
 * split the reduction over taps and input channels across several CTAs, keep fp32 partial
 * results there and add them in a fixed order; given less they run unsplit.  Both are
 * deterministic; they differ in the fp32 summation order only. */
size_t lamp_conv3d_workspace_min_bytes(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, int pass);

/* y[n,od,oh,ow,co] = bias[co] + sum_{tap,ci} x[n, od*s+kd-p, oh*s+kh-p, ow*s+kw-p, ci] * w[tap][co][ci]
 * (transposed: y[n, d*s+a, h*s+b, w*s+c, co] = bias[co] + sum_ci x[n,d,h,w,ci] * w[(a,b,c)][co][ci]).
 * x: bf16.  y: bf16 or fp32, extents must equal the conv's output extents.
 * bias: fp32 [c_out] or NULL.
 * stats: NULL, or fp64 [n][c_out][2]; the kernel ADDS, per (n, co), the sum and
 *   the sum of squares of the fp32 results (before any rounding to bf16) - the
 *   caller zeroes it.  These are the InstanceNorm statistics of the layer.
 * c_in may be any positive value (c_in == 1 is the network's first layer);
 * when x is not a multiple of 8 channels wide, c_pitch/c_offset need no alignment. */
lamp_status_t lamp_conv3d_fwd(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, const void *w,
                              const float *bias, lamp_tensor_t *y, double *stats,
                              void *ws, size_t ws_bytes, void *cuda_stream);

/* dx = gradient of lamp_conv3d_fwd with respect to x, given dy (bf16); dx bf16 or fp32,
 * its extents are the conv's input extents. */
lamp_status_t lamp_conv3d_dgrad(const lamp_conv_desc_t *desc, const lamp_tensor_t *dy, const void *w,
                                lamp_tensor_t *dx, void *ws, size_t ws_bytes, void *cuda_stream);

/* The same data gradient for callers that cannot allocate device memory when they call - e.g. a
 * layer running inside an engine that handed out all device memory at start-up, or a latency-
 * critical loop where cudaMalloc (it synchronises the device and can fail under memory pressure)
 * is ruled out - and so have no workspace to pass.  (The paper has no counterpart of this call:
 * it is a packaging variant of lamp_conv3d_dgrad, with the arithmetic and results of that call
 * given its smallest workspace.)
 * The scratch this pass needs, a transposed copy of the weights, sits in a fixed array of
 * LAMP_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library holds it
 * until the process exits.  The call itself allocates and frees nothing.
 *  - Limit: lamp_conv3d_workspace_min_bytes(desc, dx, LAMP_PASS_DGRAD) must not exceed
 *    LAMP_STATIC_SCRATCH_BYTES (27 * c_in * c_out * 2 bytes for the 3x3x3 s1 p1 conv, i.e. up to
 *    c_in * c_out = 77672, e.g. 256 x 256); otherwise LAMP_ERR_SCRATCH_LIMIT is returned and
 *    nothing is launched.  Variants that need no scratch are accepted at any size.
 *  - The first call on each device looks up the array's device address (with that device
 *    current) and keeps it; make that first call before starting any stream capture.  The kept
 *    address belongs to the device's primary context and is not looked up again: do not use this
 *    call after a cudaDeviceReset of a device on which it already ran.
 *  - All calls on a device share the one array, which keeps whatever the last call left in it.
 *    Nothing in it has to be zero beforehand (each call overwrites the part it reads), but two
 *    calls that overlap in time on the same GPU - different streams or threads - race on it:
 *    issue them on one stream, or order them yourself.
 * Arguments and errors are otherwise those of lamp_conv3d_dgrad. */
#define LAMP_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
lamp_status_t lamp_conv3d_dgrad_static_scratch(const lamp_conv_desc_t *desc, const lamp_tensor_t *dy, const void *w,
                                               lamp_tensor_t *dx, void *cuda_stream);

/* dw[tap][c_out][c_in] (fp32) = gradient with respect to w; dbias[c_out] (fp32, may be NULL)
 * = sum of dy over voxels.  x, dy bf16.  Both outputs are overwritten. */
lamp_status_t lamp_conv3d_wgrad(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, const lamp_tensor_t *dy,
                                float *dw, float *dbias, void *ws, size_t ws_bytes, void *cuda_stream);

/* ------------------------------------------------------------------------
 * Squeeze-and-excitation residual block: the SEU-Net variant of the network (Sec. 1 and Sec. 3 name a "3D SEU-Net"
 * after AnatomyNet; Tables 2, 3 and 5 report it; the paper does not define the block).  Reading: at the end of a
 * level's conv stack, with z = relu((y - mu) * rstd) of the level's LAST conv (y its stored raw output, mu_rstd as
 * written by lamp_instnorm_relu_fwd) and r = the output of the level's FIRST conv -> InstanceNorm -> ReLU,
 *     s[n,c] = mean over voxels of z,  h = relu(W1 s + b1),  e = sigmoid(W2 h + b2),  out = r + e[n,c] * z.
 * W1 fp32 [cr][c], b1 fp32 [cr], W2 fp32 [c][cr], b2 fp32 [c]; e, mean fp32 [n][c]; hidden fp32 [n][cr].
 * Tensors are bf16 with c a multiple of 8 (c <= 2048), channel slices allowed; z is never stored.
 * Forward:  lamp_se_squeeze (sums: fp64 [n][c], overwritten with sum_v z) -> lamp_se_excite -> lamp_se_apply_fwd
 *           (residual may be NULL: out = e * z).
 * Backward: lamp_se_bwd_reduce (de_sums: fp64 [n][c] = sum_v dout * z) -> lamp_se_excite_bwd (ds_over_v fp32 [n][c],
 *           and the gradients of W1, b1, W2, b2, summed over the samples) -> lamp_se_apply_bwd (dz = e * dout +
 *           ds_over_v, bf16: the incoming gradient of the last conv's lamp_instnorm_relu_bwd).  The residual branch's
 *           gradient is dout itself (the second gradient source of the first conv's lamp_instnorm_relu_bwd).
 * ---------------------------------------------------------------------- */
lamp_status_t lamp_se_squeeze(const lamp_tensor_t *y, const float *mu_rstd, double *sums, void *cuda_stream);
lamp_status_t lamp_se_excite(const double *sums, int64_t voxels_per_sample, int32_t n, int32_t c, int32_t cr,
                             const float *w1, const float *b1, const float *w2, const float *b2,
                             float *e, float *hidden, float *mean, void *cuda_stream);
lamp_status_t lamp_se_apply_fwd(const lamp_tensor_t *y, const float *mu_rstd, const float *e,
                                const lamp_tensor_t *residual, lamp_tensor_t *out, void *cuda_stream);
lamp_status_t lamp_se_bwd_reduce(const lamp_tensor_t *dout, const lamp_tensor_t *y, const float *mu_rstd,
                                 double *de_sums, void *cuda_stream);
lamp_status_t lamp_se_excite_bwd(const double *de_sums, int64_t voxels_per_sample, int32_t n, int32_t c, int32_t cr,
                                 const float *e, const float *hidden, const float *mean, const float *w1, const float *w2,
                                 float *ds_over_v, float *dw1, float *db1, float *dw2, float *db2, void *cuda_stream);
lamp_status_t lamp_se_apply_bwd(const lamp_tensor_t *dout, const float *e, const float *ds_over_v, lamp_tensor_t *dz,
                                void *cuda_stream);

/* ------------------------------------------------------------------------
 * Normalisation steps of a block.  No passage of the paper defines them (it gives the network's
 * topology only, Sec. 2.2); they are the steps between the convolutions of every block of this
 * library's U-Net and are exported so that each can be checked against the oracle on its own.
 * ---------------------------------------------------------------------- */

/* z = max(0, (y - mu) * rstd) per (n, c), mu = S1/V, rstd = (S2/V - mu^2 + eps)^-1/2 with
 * (S1, S2) = stats[n][c][0..1] (fp64, as accumulated by lamp_conv3d_fwd), V = d*h*w.
 * y bf16, z bf16 (may be a channel slice of a concat buffer).  mu_rstd: fp32 [n][c][2] scratch
 * that receives (mu, rstd) and is needed again by the backward call. */
lamp_status_t lamp_instnorm_relu_fwd(const lamp_tensor_t *y, const double *stats, float eps,
                                     float *mu_rstd, lamp_tensor_t *z, void *cuda_stream);

/* dy = rstd * (g - mean(g) - xhat * mean(g * xhat)),  g = (dz_a + dz_b) * [xhat > 0],
 * xhat = (y - mu) * rstd, means over d*h*w per (n, c).  dz_b may be NULL (the second
 * gradient source exists where a block output feeds both the next level and a skip).
 * sums: fp64 [n][c][2] scratch, zeroed by the call.  y, dz_*, dy bf16. */
lamp_status_t lamp_instnorm_relu_bwd(const lamp_tensor_t *dz_a, const lamp_tensor_t *dz_b,
                                     const lamp_tensor_t *y, const float *mu_rstd,
                                     double *sums, lamp_tensor_t *dy, void *cuda_stream);

/* ------------------------------------------------------------------------
 * U-Net (Sec. 2.2, Eq. 2; widths per Sec. 3).
 *   encoder level l: convs_per_level x [conv 3x3x3 s1 p1 -> InstanceNorm -> ReLU]; between
 *   levels a conv 3x3x3 s2 p1 -> InstanceNorm -> ReLU; decoder level l: transposed conv 2x2x2 s2
 *   (+bias), concat(skip, up), convs_per_level x [conv -> InstanceNorm -> ReLU]; head: conv 1x1x1
 *   to num_classes, softmax.  InstanceNorm: biased variance, eps = in_eps, no affine parameters.
 * Layer order (also parameter order): encoder levels top-down (convs, then the down conv),
 * decoder levels bottom-up (up conv, then convs), head.
 * ---------------------------------------------------------------------- */
typedef struct {
    int32_t levels;            /* 1..8                                     */
    int32_t channels[8];       /* width of each level, multiples of 8      */
    int32_t convs_per_level;   /* >= 1                                     */
    int32_t in_channels;       /* 1, or a multiple of 8                    */
    int32_t num_classes;       /* 2..16                                    */
    float   in_eps;
    int32_t se_ratio;          /* 0: plain U-Net.  > 0: SEU-Net variant - every level's conv stack ends in the squeeze-and-
                                  excitation residual step described above (hidden units = width / se_ratio, at least 1);
                                  needs convs_per_level >= 2 (the residual branch is the first conv's output)    */
} lamp_unet_spec_t;

typedef struct lamp_unet lamp_unet_t;          /* opaque, host-only plan */

lamp_status_t lamp_unet_create(const lamp_unet_spec_t *spec, lamp_unet_t **out);
/* SEU-Net variant: where the squeeze-and-excitation parameters of `layer` (a level's last conv) sit in the BIAS buffer
 * (fp32): from *se_off, W1 [cr][c], b1 [cr], W2 [c][cr], b2 [c] back to back, c = the layer's c_out, *cr hidden units;
 * their gradients sit at the same offsets of grad_b.  *cr = 0 for layers without the step. */
lamp_status_t lamp_unet_se_layout(const lamp_unet_t *net, int32_t layer, size_t *se_off, int32_t *cr);
void          lamp_unet_destroy(lamp_unet_t *net);
int32_t       lamp_unet_num_layers(const lamp_unet_t *net);
/* Elements of the flat bf16 weight buffer / of the flat fp32 bias buffer. */
size_t        lamp_unet_weight_count(const lamp_unet_t *net);
size_t        lamp_unet_bias_count(const lamp_unet_t *net);
/* Offsets (in elements) of layer `layer` inside the two flat buffers, and its conv descriptor. */
lamp_status_t lamp_unet_param_layout(const lamp_unet_t *net, int32_t layer, size_t *w_off, size_t *b_off,
                                     lamp_conv_desc_t *desc);

enum { LAMP_MODE_INFER = 0, LAMP_MODE_TRAIN = 1 };
size_t lamp_unet_workspace_bytes(const lamp_unet_t *net, int32_t n, int32_t d, int32_t h, int32_t w, int32_t mode);

/* Where a pass keeps one of its tensors inside the workspace, for inspection after the call
 * (no passage of the paper: exported so that tests can check every step of a pass on its own).
 * Training mode keeps every tensor listed; inference mode keeps LAMP_T_IN / LAMP_T_OUT only (the
 * raw conv output is a buffer shared by all layers there).  On success *offset is the byte offset
 * from the workspace base to the tensor's first element (the slice's first channel) and *out
 * describes it (ptr = NULL, c_offset = 0, c_pitch = distance between voxels).
 * LAMP_T_STATS is fp64 [n][c_out][2] (sum, sum of squares), LAMP_T_MU_RSTD fp32 [n][c_out][2],
 * LAMP_T_PROBS fp32 [n*d*h*w][num_classes] (present when the caller passed probs = NULL);
 * for these *out reports c = 2*c_out (or num_classes) per n.
 * Returns LAMP_ERR_UNSUPPORTED when the layer has no such tensor (e.g. LAMP_T_IN of layer 0, which
 * is the caller's buffer, or LAMP_T_Y of an up conv). */
enum {
    LAMP_T_IN = 0,       /* layer input (bf16)                                            */
    LAMP_T_Y = 1,        /* raw conv output before normalisation (bf16)                    */
    LAMP_T_OUT = 2,      /* layer output: normalised + ReLU, or the up conv's output (bf16)*/
    LAMP_T_STATS = 3,
    LAMP_T_MU_RSTD = 4,
    LAMP_T_DY = 5,       /* gradient w.r.t. the raw conv output (bf16)                     */
    LAMP_T_DIN = 6,      /* gradient w.r.t. the layer input (bf16)                         */
    LAMP_T_DOUT = 7,     /* gradient w.r.t. the layer output, main source (bf16)           */
    LAMP_T_DOUT2 = 8,    /* second source: the skip path's gradient, encoder block outputs */
    LAMP_T_PROBS = 9
};
lamp_status_t lamp_unet_tensor_layout(const lamp_unet_t *net, int32_t n, int32_t d, int32_t h, int32_t w, int32_t mode,
                                      int32_t layer, int32_t which, lamp_tensor_t *out, size_t *offset);

/* One forward pass.  x: bf16 [n,d,h,w,in_channels] (d,h,w divisible by 2^(levels-1)).
 * probs: fp32 [n*d*h*w][num_classes] softmax output, or NULL.  argmax: uint8 [n*d*h*w] class of
 * largest probability (lowest index on ties), or NULL.  Stored intermediates are bf16. */
lamp_status_t lamp_unet_forward(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                const lamp_tensor_t *x, float *probs, uint8_t *argmax,
                                void *ws, size_t ws_bytes, void *cuda_stream);

/* Layers [first_layer, last_layer) of the forward pass only: one partition F_k of the sequentialised network (Sec. 2.1,
 * Eq. 1; Sec. 2.2, Eq. 3).  The partition reads what earlier layers left in the workspace - the activation that enters
 * first_layer and, for every skip that crosses the cut, the kept encoder output e_{i,1} (LAMP_T_OUT of that encoder
 * layer, in inference mode) - and leaves its own outputs there; lamp_unet_tensor_layout says where each of them
 * lives, so a pipeline copies exactly those tensors from the previous partition's workspace (on another device: into
 * this device's own memory first) and calls this.  x must describe the network input in every partition (its shape
 * fixes the layout; its data is read only when first_layer = 0).  probs / argmax are written only by the partition
 * that contains the head.  Running the partitions of any cut one after the other on one workspace, or on several with
 * the boundary tensors copied, gives exactly lamp_unet_forward's result. */
lamp_status_t lamp_unet_forward_layers(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                       const lamp_tensor_t *x, int32_t first_layer, int32_t last_layer,
                                       float *probs, uint8_t *argmax, void *ws, size_t ws_bytes, void *cuda_stream);

/* One forward + backward pass with the softmax-Dice loss
 *   L = mean_n [ 1 - (1/K) sum_k (2 I_k + e)/(P_k + G_k + e) ],  I = sum p g, P = sum p, G = sum g, e = 1e-5.
 * labels: uint8 [n*d*h*w], values < num_classes.  loss: fp32 device scalar.
 * grad_w: fp32, laid out like the weight buffer; grad_b: fp32, like the bias buffer.
 * probs: fp32 [n*d*h*w][num_classes] or NULL (then taken from the workspace).
 * Streams: the weight gradients (and the per-step transposes of the weights the data gradients read) run on a
 * second stream owned by the handle, ordered against cuda_stream with events; that stream starts after all
 * work enqueued on cuda_stream before the call and is joined into cuda_stream before the call returns, so the
 * caller sees ordinary stream semantics.  The stream and its events are created by the first training step of a
 * handle on a device (no device memory is involved); that first call must therefore come before any stream
 * capture.  One handle must not run training steps from several host threads at once. */
lamp_status_t lamp_unet_train_step(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                   const lamp_tensor_t *x, const uint8_t *labels, float *loss,
                                   float *grad_w, float *grad_b, float *probs,
                                   void *ws, size_t ws_bytes, void *cuda_stream);

/* The same step for data-parallel training (Sec. 1: replicas that exchange gradients): the caller cuts grad_w into
 * n_buckets ranges [bucket_start[b], bucket_start[b+1]) (element offsets, ascending, bucket_start[0] = 0, the last
 * range ends at the weight count) and passes one CUDA event (a cudaEvent_t as void*) per bucket.  bucket_events[b] is
 * recorded as soon as every gradient of bucket b has been enqueued - the backward pass finishes the layers last to
 * first, so the buckets become final from the last to the first, the early ones long before the call's work ends -
 * and a stream that waits on the event may read (e.g. all-reduce) that range while the rest of the backward pass runs.
 * The events are recorded on a stream of the library; use them only with cudaStreamWaitEvent / cudaEventSynchronize.
 * grad_b, loss and probs are final when the work of the call on cuda_stream is.  Otherwise as lamp_unet_train_step. */
lamp_status_t lamp_unet_train_step_buckets(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                           const lamp_tensor_t *x, const uint8_t *labels, float *loss,
                                           float *grad_w, float *grad_b, float *probs,
                                           void *ws, size_t ws_bytes, void *cuda_stream,
                                           const int64_t *bucket_start /* host */, int32_t n_buckets,
                                           void *const *bucket_events /* host array */);

/* Sliding-window inference (Sec. 3: patches versus the whole image).  Patch origins per axis are
 * 0, s, 2s, ... with s = round(patch * (1 - overlap)) while the patch fits, plus one patch flush
 * with the border if needed; patches are ordered by origin (d, h, w), w fastest; each patch is a
 * separate network input (own InstanceNorm statistics).  Patch probabilities are blended with
 * weight 1 (window = 0) or a Gaussian (window = 1: sigma = patch/8 per axis, normalised to
 * maximum 1, floored at 1e-3): A[v,k] = sum_p w p / sum_p w.
 * volume: bf16 [1,d,h,w,in_channels].  probs_planar: fp32 [num_classes][d][h][w] or NULL.
 * argmax: uint8 [d*h*w].  sw_batch: patches per network pass (>= 1).
 * After the call the first n_patches*pd*ph*pw*num_classes floats of the workspace hold the
 * per-patch probabilities, fp32 [n_patches][pd*ph*pw][num_classes]. */
size_t lamp_sliding_window_workspace_bytes(const lamp_unet_t *net, int32_t d, int32_t h, int32_t w,
                                           const int32_t patch[3], float overlap, int32_t sw_batch);
lamp_status_t lamp_sliding_window_infer(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                        const lamp_tensor_t *volume, const int32_t patch[3], float overlap,
                                        int32_t sw_batch, int32_t window, float *probs_planar, uint8_t *argmax,
                                        void *ws, size_t ws_bytes, void *cuda_stream);

/* Sliding-window inference split over replicas by patch index (Sec. 1, data parallelism; Sec. 3, patches).
 * lamp_sliding_window_num_patches: patches of the grid (0 for invalid arguments).
 * lamp_sliding_window_partial runs patches first_patch .. first_patch + num_patches - 1 only and writes THEIR blend
 * un-normalised: sums_planar fp32 [num_classes][d][h][w] = sum_p w p, weight_sums fp32 [d][h][w] = sum_p w (zeros
 * where none of these patches covers a voxel); both 16-byte aligned.  Workspace as for lamp_sliding_window_infer.
 * The caller adds the buffers of all replicas (e.g. an all-reduce), then lamp_sliding_window_finish divides in place
 * (write_probs != 0) and / or takes the arg max (argmax may be NULL if write_probs).  With one replica holding all
 * patches the two calls give exactly what lamp_sliding_window_infer gives. */
int32_t lamp_sliding_window_num_patches(int32_t d, int32_t h, int32_t w, const int32_t patch[3], float overlap);
lamp_status_t lamp_sliding_window_partial(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                          const lamp_tensor_t *volume, const int32_t patch[3], float overlap,
                                          int32_t sw_batch, int32_t window, int32_t first_patch, int32_t num_patches,
                                          float *sums_planar, float *weight_sums, void *ws, size_t ws_bytes,
                                          void *cuda_stream);
lamp_status_t lamp_sliding_window_finish(float *sums_planar, const float *weight_sums, int32_t k, int64_t voxels,
                                         int32_t write_probs, uint8_t *argmax, void *cuda_stream);

/* Weighted overlap-add of per-patch probabilities on its own (the aggregation step of
 * lamp_sliding_window_infer, Sec. 3; no passage of its own: exported for testing).  patch_probs: fp32 [n_patches][pd*ph*pw][k], patches in the order
 * above for a d x h x w volume. */
lamp_status_t lamp_overlap_add(const float *patch_probs, int32_t k, int32_t d, int32_t h, int32_t w,
                               const int32_t patch[3], float overlap, int32_t window,
                               float *probs_planar, uint8_t *argmax, void *cuda_stream);

/* ------------------------------------------------------------------------
 * Parameter update (Sec. 3, training setup: RMSProp, learning rate 1e-3; the update is the
 * one of the lecture the paper cites, without momentum or centring).
 * ---------------------------------------------------------------------- */

/* For each of the n elements:  v = alpha * v + (1 - alpha) * g^2;  master -= lr * g / (sqrt(v) + eps);
 * param_bf16 = bf16(master) (round to nearest even).
 * grad, master, v: device fp32 [n] (v is the running mean of squared gradients, zero before the
 * first step); param_bf16: device bf16 [n], or NULL for parameters that are used in fp32 (biases).
 * master and v are updated in place.  n == 0 is a no-op.  Arithmetic in fp32.
 * The flat layouts of lamp_unet_param_layout fit: one call for the weights (with the bf16 copy
 * that the network calls read), one for the biases (param_bf16 = NULL, master = the bias vector). */
lamp_status_t lamp_rmsprop_step(int64_t n, const float *grad, float *master, float *v, void *param_bf16,
                                float lr, float alpha, float eps, void *cuda_stream);

/* Synchronises `cuda_stream`, then returns and clears the device-side status word
 * (LAMP_OK, or LAMP_ERR_TIMEOUT if a bounded wait inside a kernel ran out). */
lamp_status_t lamp_get_async_status(void *cuda_stream);
const char   *lamp_status_string(lamp_status_t s);
/* Self-test of the failure path every tensor-core kernel of this library shares: all device-side waits
 * (on TMA completions, on tensor-pipe completions) are bounded, and a wait that runs out records
 * LAMP_ERR_TIMEOUT and lets the kernel finish normally instead of hanging.  This call launches one
 * small kernel whose wait can never be satisfied (limit about 10 ms); afterwards
 * lamp_get_async_status() must return LAMP_ERR_TIMEOUT once and the context must remain usable. */
lamp_status_t lamp_selftest_wait_timeout(void *cuda_stream);
/* Library build identifier: "lamp-b200 <sm arch>". */
const char   *lamp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LAMP_H_ */
