// Shared device/host helpers of the library (not used by the CPU oracle).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/lamp.h"

namespace lamp {

typedef __nv_bfloat16 bf16;

// Device view of a lamp_tensor_t: pointer already advanced to the slice's first channel.
struct TView {
    void   *p;
    int32_t n, d, h, w, c;
    int64_t pitch;     // elements between voxels
    int32_t f32;       // 1: float elements, 0: bf16
};

static inline TView make_view(const lamp_tensor_t *t)
{
    TView v;
    const size_t es = t->dtype == LAMP_F32 ? 4 : 2;
    v.p = (char *)t->ptr + (size_t)t->c_offset * es;
    v.n = t->n; v.d = t->d; v.h = t->h; v.w = t->w; v.c = t->c;
    v.pitch = t->c_pitch;
    v.f32 = t->dtype == LAMP_F32;
    return v;
}

static inline int64_t voxels(const lamp_tensor_t *t) { return (int64_t)t->n * t->d * t->h * t->w; }

__device__ __forceinline__ float bf2f(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ bf16 f2bf(float v) { return __float2bfloat16_rn(v); }

// 8 bf16 values in one 16-byte word.
struct __align__(16) bf16x8 { bf16 v[8]; };

__device__ __forceinline__ void unpack8(const uint4 &u, float (&f)[8])
{
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i]     = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t *>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Device address of the status word (LAMP_OK or LAMP_ERR_TIMEOUT) on the current device
// (api.cu); NULL if it cannot be resolved.
int *status_word_ptr();

#define LAMP_CUDA_OK(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) return LAMP_ERR_CUDA;        \
    } while (0)

static inline lamp_status_t launch_status()
{
    return cudaGetLastError() == cudaSuccess ? LAMP_OK : LAMP_ERR_CUDA;
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// api.cu.  The driver's cuTensorMapEncodeTiled (a function of that signature with a small cache in front: the same
// arguments give the stored map), resolved once through the runtime (NULL if unavailable); declared as void* so that
// this header needs no driver types.
void *tensor_map_encoder();
// api.cu.  Number of SMs of the current device.
int sm_count();

// cudaFuncAttributeMaxDynamicSharedMemorySize is a per-device attribute of a kernel: a launcher keeps one of these
// per kernel instantiation and asks it before every launch; the attribute is set on the first launch on each device
// (bit i of `done` = device i; devices beyond 63 set it on every launch).  Safe to call from several host threads.
struct SmemAttrOnce {
    unsigned long long done = 0;
    template <typename K> lamp_status_t ensure(K kernel, int bytes)
    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return LAMP_ERR_CUDA;
        const unsigned long long bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
        if (bit && (__atomic_load_n(&done, __ATOMIC_ACQUIRE) & bit)) return LAMP_OK;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return LAMP_ERR_CUDA;
        if (bit) __atomic_fetch_or(&done, bit, __ATOMIC_RELEASE);
        return LAMP_OK;
    }
};

// Programmatic dependent launch.  A kernel launched through launch_pdl may be scheduled while the kernel in front
// of it on the stream is still running: its blocks set up shared memory, barriers and tensor memory, then stop at
// pdl_wait() until that kernel has completed and its writes are visible.  Rules every such kernel follows:
//   * every thread executes pdl_wait() before its first access to global memory and before any return, so that
//     the completion of this kernel implies the completion of all kernels in front of it;
//   * pdl_launch_dependents() (no memory semantics) is executed at the top, which lets the next kernel's blocks
//     take over SMs as this kernel's blocks retire.
// Kernels launched with <<<>>> keep the plain stream order on both sides.  `early` = false launches the kernel in
// plain stream order too: measured on one device, early scheduling gains ~4 % on chains of short kernels (the deep
// U-Net levels) and costs 1.5-2 % on launches that run for many waves (back-to-back C = 256 passes, the 512x512x128
// forward pass), so each launch site passes whether its launch is short.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline lamp_status_t launch_pdl(bool early, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                       cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = early ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) == cudaSuccess ? LAMP_OK : LAMP_ERR_CUDA;
}
#endif

// ---------------------------------------------------------------------------
// Internal launchers (one per kernel family); all enqueue on `st`.
// ---------------------------------------------------------------------------
struct ConvGeom {
    int32_t n, d, h, w;        // input extents (of x / dx)
    int32_t od, oh, ow;        // output extents (of y / dy)
    int32_t ci, co, k, s, p, transposed;
};

// conv_simt.cu
lamp_status_t simt_conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                            double *stats, cudaStream_t st);
lamp_status_t simt_conv_dgrad(const ConvGeom &g, const TView &dy, const bf16 *w, const TView &dx, cudaStream_t st);
size_t        simt_conv_wgrad_ws(const ConvGeom &g);
lamp_status_t simt_conv_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, float *db,
                              void *ws, size_t ws_bytes, cudaStream_t st);

// out[e] = sum_s part[s][e] in a fixed order; dbias[co] = sum_v dy[v][co] (ws: bias_grad_ws bytes)
lamp_status_t reduce_partials(const float *part, int64_t entries, int splits, float *out, cudaStream_t st);
// out[t][b][a] = sum_s in[s][t][a][b] (A, B multiples of 32, see transpose_sum_supported); bf16 form: one split
bool          transpose_sum_supported(int64_t taps, int A, int B);
lamp_status_t transpose_sum_f32(const float *in, int64_t taps, int A, int B, int splits, float *out, cudaStream_t st);
lamp_status_t transpose_bf16(const bf16 *in, int64_t taps, int A, int B, bf16 *out, cudaStream_t st);
size_t        bias_grad_ws(int64_t voxels, int co);
lamp_status_t bias_grad(const TView &dy, float *db, void *ws, cudaStream_t st);

// first layer (c_in = 1) on the tensor-core wgrad path: widen x to 32 channels, keep column 0 of the result
lamp_status_t pad_c1(const TView &x, bf16 *xpad, cudaStream_t st);
lamp_status_t take_c0(const float *dw32, float *dw, int n, cudaStream_t st);

// wgrad_umma.cu (tcgen05 weight gradient)
bool          umma_wgrad_supported(const ConvGeom &g, const TView &x, const TView &dy);
size_t        umma_wgrad_ws(const ConvGeom &g);
lamp_status_t umma_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, void *ws, size_t ws_bytes,
                         cudaStream_t st);

// wgrad_win.cu (tcgen05 weight gradient of the 3x3x3 s1 conv with the three kw taps on N; c_in < 256)
bool          win_wgrad_supported(const ConvGeom &g, const TView &x, const TView &dy);
size_t        win_wgrad_ws(const ConvGeom &g);
lamp_status_t win_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, void *ws, size_t ws_bytes,
                        cudaStream_t st);

// conv_umma.cu (tcgen05 implicit GEMM, voxels x channels form; see the file header for the kinds)
enum { UK_S1_FWD = 0, UK_S1_DGRAD = 1, UK_S2_FWD = 2, UK_S2_DGRAD = 3, UK_T_FWD = 4, UK_T_DGRAD = 5,
       UK_T_FWD_MERGED = 6 /* internal: chosen by umma_conv for UK_T_FWD when c_out % 32 == 0 and no statistics */ };
bool          umma_conv_supported(int kind, const ConvGeom &g, const TView &a, const TView &y);
// part / part_bytes: optional scratch of umma_splitk_ws bytes; with it a pass that has too few tiles to fill the
// GPU splits its K range over several CTAs (fp32 partial results, added in a fixed order by a second kernel)
lamp_status_t umma_conv(int kind, const ConvGeom &g, const TView &a, const bf16 *w, const float *bias, const TView &y,
                        double *stats, void *part, size_t part_bytes, cudaStream_t st);
size_t        umma_splitk_ws(int kind, const ConvGeom &g);
size_t        umma_dgrad_ws(const ConvGeom &g);
// head (1x1x1 conv + softmax + arg max + Dice sums) on the tensor cores; dice_sums must be zero on entry
bool          umma_head_supported(const TView &z, int K);
lamp_status_t umma_head(const TView &z, const bf16 *w, const float *b, int K, float *probs, uint8_t *argmax,
                        const uint8_t *labels, double *dice_sums, cudaStream_t st);
lamp_status_t umma_transpose_weights(const bf16 *w, bf16 *wt, int taps, int co, int ci, cudaStream_t st);

// conv_c1_umma.cu (tcgen05 first layer: c_in = 1, banded weight matrices along w)
bool          c1_umma_supported(const ConvGeom &g, const TView &x, const TView &y);
lamp_status_t c1_umma_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                          double *stats, cudaStream_t st);

// conv_t.cu (tcgen05 "weights x voxels" implicit GEMM over shared-memory-resident planes, c_out <= 128)
bool          ct_conv_fwd_supported(const ConvGeom &g, const TView &x, const TView &y);
lamp_status_t ct_conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                          double *stats, int mirror_taps, cudaStream_t st);

// conv_r.cu (tcgen05 "voxels x (kd, channels)" implicit GEMM with rotating accumulator slots, c_out = 64 or 32)
bool          cr_conv_fwd_supported(const ConvGeom &g, const TView &x, const TView &y);
lamp_status_t cr_conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                          double *stats, int mirror_taps, cudaStream_t st);

// elementwise.cu
// z = relu((y - mu) * rstd) with (mu, rstd) derived from the fp64 sums; also stores (mu, rstd) to mu_rstd
lamp_status_t k_instnorm_relu_fwd(const TView &y, const double *stats, float eps, float *mu_rstd, const TView &z,
                                  cudaStream_t st);
// sums: fp64 [n][c][2] scratch (cleared here unless sums_are_zero).  db != NULL: also db[c] = sum of the stored dy over
// voxels and samples, through db_acc (fp64 [c]) and the ticket counter db_count, both zero on entry.
lamp_status_t k_instnorm_relu_bwd(const TView &dza, const TView *dzb, const TView &y, const float *mu_rstd,
                                  double *sums, bool sums_are_zero, const TView &dy, double *db_acc, unsigned *db_count,
                                  float *db, cudaStream_t st);
lamp_status_t k_head_softmax(const TView &z, const bf16 *w, const float *b, int K, float *probs, uint8_t *argmax,
                             const uint8_t *labels, double *dice_sums, cudaStream_t st);
lamp_status_t k_dice_loss(const double *dice_sums, int N, int K, float *loss, cudaStream_t st);
size_t        head_bwd_ws(int64_t Vn, int n, int K, int C);
lamp_status_t k_head_bwd(const TView &z, const bf16 *w, int K, const float *probs, const uint8_t *labels,
                         const double *dice_sums, const TView &dz, float *dw, float *db, float *dlogits,
                         void *ws, size_t ws_bytes, cudaStream_t st);
lamp_status_t k_rmsprop(int64_t n, const float *g, float *w, float *v, bf16 *wb, float lr, float alpha, float eps,
                        cudaStream_t st);
lamp_status_t k_gather_patches(const TView &vol, const TView &patches, int first_patch, const int32_t nst[3],
                               const int32_t stride[3], cudaStream_t st);
// p_count < 0: all patches, normalised result (planar may be NULL) and arg max.  Otherwise pp holds the patches
// p_first .. p_first + p_count - 1 only; with wsum_out the un-normalised sums of those go to planar and their weight
// totals to wsum_out [d][h][w] (k_overlap_finish divides and takes the arg max once all shares have been added).
lamp_status_t k_overlap_add(const float *pp, int K, int D, int H, int W, const int32_t patch[3],
                            const int32_t nst[3], const int32_t stride[3], int window, float *planar,
                            uint8_t *argmax, cudaStream_t st, int p_first = 0, int p_count = -1, float *wsum_out = nullptr);
lamp_status_t k_overlap_finish(float *planar, const float *wsum, int K, int64_t V, int write_probs, uint8_t *argmax,
                               cudaStream_t st);

// se_block.cu: the squeeze-and-excitation residual block's steps for the U-Net executor (params: W1 [cr][c], b1 [cr],
// W2 [c][cr], b2 [c] back to back in fp32, dparams likewise), mu / rstd from the InstanceNorm sums, out = a + b
lamp_status_t k_mu_rstd(const double *stats, int64_t Vn, float eps, float *mr, int nc, cudaStream_t st);
lamp_status_t k_add2(const TView &a, const TView &b, const TView &out, cudaStream_t st);
lamp_status_t k_se_fwd(const TView &y, const float *mr, const float *params, int cr, double *sums, float *e, float *hid,
                       float *mean, const TView *res, const TView &out, cudaStream_t st);
lamp_status_t k_se_bwd(const TView &dout, const TView &y, const float *mr, const float *params, int cr, const float *e,
                       const float *hid, const float *mean, double *de, float *dsv, float *dparams, const TView &dz,
                       cudaStream_t st);

// api.cu: shape checks + kernel selection for one conv pass (used by the ABI and by the U-Net executor)
lamp_status_t conv_geom(const lamp_conv_desc_t *desc, const lamp_tensor_t *in, const lamp_tensor_t *out, ConvGeom *g);
size_t        conv_ws_bytes(const ConvGeom &g, int pass);       // scratch with which the pass runs fastest
size_t        conv_ws_min_bytes(const ConvGeom &g, int pass);   // smallest scratch the pass accepts
lamp_status_t conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                       double *stats, void *ws, size_t ws_bytes, cudaStream_t st);
lamp_status_t conv_dgrad(const ConvGeom &g, const TView &dy, const bf16 *w, const TView &dx, void *ws, size_t ws_bytes,
                         cudaStream_t st);
// the data gradient in two steps: the transposed weights written once (wt: conv_ws_min_bytes(g, LAMP_PASS_DGRAD)
// bytes), then any number of passes that read them (part: optional split-K scratch, see umma_conv)
lamp_status_t conv_dgrad_prepare(const ConvGeom &g, const TView &dy, const TView &dx, const bf16 *w, void *wt,
                                 size_t wt_bytes, cudaStream_t st);
lamp_status_t conv_dgrad_run(const ConvGeom &g, const TView &dy, const bf16 *w, const void *wt, const TView &dx,
                             void *part, size_t part_bytes, cudaStream_t st);
lamp_status_t conv_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, float *db, void *ws,
                         size_t ws_bytes, cudaStream_t st);

}  // namespace lamp
