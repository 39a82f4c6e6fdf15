// C ABI (include/lamp.h): argument checks, kernel selection, status word.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <mutex>
#include <string.h>
#include "common.cuh"
#include "umma_ptx.cuh"

namespace lamp {

__device__ int g_status_word = 0;

int *status_word_ptr()
{
    int *p = nullptr;
    if (cudaGetSymbolAddress((void **)&p, g_status_word) != cudaSuccess) return nullptr;
    return p;
}

// cuTensorMapEncodeTiled with a small cache in front.  A training step encodes two tensor maps per tensor-core launch
// (about 460 per step), always from the same few hundred argument sets: the encoded map depends on nothing but the
// arguments, so a hit returns the stored 128 bytes.  Direct-mapped, 1024 entries, one mutex (calls come from the host
// threads that enqueue work; an entry is compared in full before it is used).
namespace {

struct MapKey {
    uint64_t addr, gdim[5], gstride[4];
    uint32_t box[5], es[5], rank, dt, il, sw, l2, oob;
};
struct MapEntry { bool valid; MapKey key; CUtensorMap map; };
constexpr int MAP_CACHE_SLOTS = 1024;
MapEntry g_map_cache[MAP_CACHE_SLOTS];
std::mutex g_map_mutex;
PFN_cuTensorMapEncodeTiled_v12000 g_real_encode = nullptr;

CUresult CUDAAPI encode_tiled_cached(CUtensorMap *out, CUtensorMapDataType dt, cuuint32_t rank, void *addr, const cuuint64_t *gdim,
                                     const cuuint64_t *gstride, const cuuint32_t *box, const cuuint32_t *es,
                                     CUtensorMapInterleave il, CUtensorMapSwizzle sw, CUtensorMapL2promotion l2,
                                     CUtensorMapFloatOOBfill oob)
{
    if (rank < 1 || rank > 5) return g_real_encode(out, dt, rank, addr, gdim, gstride, box, es, il, sw, l2, oob);
    MapKey k;
    memset(&k, 0, sizeof(k));
    k.addr = (uint64_t)(uintptr_t)addr; k.rank = rank; k.dt = (uint32_t)dt; k.il = (uint32_t)il; k.sw = (uint32_t)sw;
    k.l2 = (uint32_t)l2; k.oob = (uint32_t)oob;
    for (cuuint32_t i = 0; i < rank; ++i) { k.gdim[i] = gdim[i]; k.box[i] = box[i]; k.es[i] = es[i]; }
    for (cuuint32_t i = 0; i + 1 < rank; ++i) k.gstride[i] = gstride[i];
    uint64_t h = 1469598103934665603ull;
    const unsigned char *b = (const unsigned char *)&k;
    for (size_t i = 0; i < sizeof(k); ++i) h = (h ^ b[i]) * 1099511628211ull;
    MapEntry &e = g_map_cache[h % MAP_CACHE_SLOTS];
    {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        if (e.valid && memcmp(&e.key, &k, sizeof(k)) == 0) { *out = e.map; return CUDA_SUCCESS; }
    }
    const CUresult r = g_real_encode(out, dt, rank, addr, gdim, gstride, box, es, il, sw, l2, oob);
    if (r == CUDA_SUCCESS) {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        e.key = k; e.map = *out; e.valid = true;
    }
    return r;
}

}  // namespace

void *tensor_map_encoder()
{
    // resolved once per process; the entry point does not depend on the device
    static void *fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            p = nullptr;
        g_real_encode = (PFN_cuTensorMapEncodeTiled_v12000)p;
        return p ? (void *)&encode_tiled_cached : nullptr;
    }();
    return fn;
}

int sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        sms <= 0)
        sms = 148;
    return sms;
}

static bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

static lamp_status_t check_tensor(const lamp_tensor_t *t, bool allow_f32, bool any_channels)
{
    if (!t || !t->ptr) return LAMP_ERR_INVALID_ARG;
    if (t->n < 0 || t->d < 0 || t->h < 0 || t->w < 0 || t->c <= 0 || t->c_offset < 0) return LAMP_ERR_INVALID_ARG;
    if (t->c_pitch < (int64_t)t->c_offset + t->c) return LAMP_ERR_INVALID_ARG;
    if (t->dtype != LAMP_BF16 && !(allow_f32 && t->dtype == LAMP_F32)) return LAMP_ERR_UNSUPPORTED;
    if (!aligned16(t->ptr)) return LAMP_ERR_INVALID_ARG;
    if (!any_channels && t->dtype == LAMP_BF16 && ((t->c & 7) || (t->c_pitch & 7) || (t->c_offset & 7)))
        return LAMP_ERR_UNSUPPORTED;
    if ((double)voxels(t) * (double)t->c_pitch * 4.0 > 1099511627776.0) return LAMP_ERR_UNSUPPORTED;   // 2^40 B
    return LAMP_OK;
}

// `in` has the conv's input extents, `out` its output extents (either may be NULL to skip the check).
lamp_status_t conv_geom(const lamp_conv_desc_t *d, const lamp_tensor_t *in, const lamp_tensor_t *out, ConvGeom *g)
{
    if (!d || !g) return LAMP_ERR_INVALID_ARG;
    if (d->c_in <= 0 || d->c_out <= 0) return LAMP_ERR_INVALID_ARG;
    const bool ok = (d->ksize == 3 && d->stride == 1 && d->pad == 1 && !d->transposed) ||
                    (d->ksize == 3 && d->stride == 2 && d->pad == 1 && !d->transposed) ||
                    (d->ksize == 1 && d->stride == 1 && d->pad == 0 && !d->transposed) ||
                    (d->ksize == 2 && d->stride == 2 && d->pad == 0 && d->transposed == 1);
    if (!ok) return LAMP_ERR_UNSUPPORTED;
    g->ci = d->c_in; g->co = d->c_out; g->k = d->ksize; g->s = d->stride; g->p = d->pad; g->transposed = d->transposed;
    const lamp_tensor_t *ref = in ? in : out;
    if (!ref) return LAMP_ERR_INVALID_ARG;
    if (in) {
        g->n = in->n; g->d = in->d; g->h = in->h; g->w = in->w;
        if (in->c != d->c_in) return LAMP_ERR_INVALID_ARG;
        if (d->transposed) { g->od = in->d * 2; g->oh = in->h * 2; g->ow = in->w * 2; }
        else {
            g->od = in->d ? (in->d + 2 * d->pad - d->ksize) / d->stride + 1 : 0;
            g->oh = in->h ? (in->h + 2 * d->pad - d->ksize) / d->stride + 1 : 0;
            g->ow = in->w ? (in->w + 2 * d->pad - d->ksize) / d->stride + 1 : 0;
        }
    }
    if (out) {
        if (out->c != d->c_out) return LAMP_ERR_INVALID_ARG;
        if (in) {
            if (out->n != g->n || out->d != g->od || out->h != g->oh || out->w != g->ow) return LAMP_ERR_INVALID_ARG;
        } else {
            return LAMP_ERR_INVALID_ARG;
        }
    }
    return LAMP_OK;
}

static int fwd_kind(const ConvGeom &g)
{
    if (g.transposed) return UK_T_FWD;
    if (g.k == 3 && g.s == 2) return UK_S2_FWD;
    if (g.k == 3 && g.s == 1) return UK_S1_FWD;
    return -1;
}

static int dgrad_kind(const ConvGeom &g)
{
    if (g.transposed) return UK_T_DGRAD;
    if (g.k == 3 && g.s == 2) return UK_S2_DGRAD;
    if (g.k == 3 && g.s == 1) return UK_S1_DGRAD;
    return -1;
}

static bool dgrad_on_tensor_cores(const ConvGeom &g)
{
    // channel counts only; the alignment of the real views is checked again at launch
    TView a{}, b{};
    a.pitch = 8; b.pitch = 8;
    const int kind = dgrad_kind(g);
    return kind >= 0 && umma_conv_supported(kind, g, a, b);
}

static size_t c1_padded_ws(const ConvGeom &g, size_t *xpad_bytes, size_t *dw32_bytes);

// scratch for fp32 partial results when the tensor-core "voxels x channels" kernel would take the pass
static size_t splitk_ws(const ConvGeom &g, int pass)
{
    TView a{}, b{};
    a.pitch = 8; b.pitch = 8;
    if (pass == LAMP_PASS_FWD) {
        a.d = g.d; a.h = g.h; a.w = g.w; a.c = g.ci;
        if (cr_conv_fwd_supported(g, a, b) || ct_conv_fwd_supported(g, a, b)) return 0;
        const int kind = fwd_kind(g);
        return kind >= 0 && umma_conv_supported(kind, g, a, b) ? umma_splitk_ws(kind, g) : 0;
    }
    const int kind = dgrad_kind(g);
    if (kind < 0 || !umma_conv_supported(kind, g, a, b)) return 0;
    if (kind == UK_S1_DGRAD) {
        ConvGeom t = g;
        t.ci = g.co; t.co = g.ci;
        a.d = g.d; a.h = g.h; a.w = g.w; a.c = g.co;
        if (cr_conv_fwd_supported(t, a, b) || ct_conv_fwd_supported(t, a, b)) return 0;
    }
    return umma_splitk_ws(kind, g);
}

size_t conv_ws_min_bytes(const ConvGeom &g, int pass)
{
    if (pass == LAMP_PASS_FWD) return 0;
    if (pass == LAMP_PASS_DGRAD) return dgrad_on_tensor_cores(g) ? umma_dgrad_ws(g) : 0;
    return conv_ws_bytes(g, pass);
}

size_t conv_ws_bytes(const ConvGeom &g, int pass)
{
    if (pass == LAMP_PASS_FWD) return splitk_ws(g, pass);
    if (pass == LAMP_PASS_DGRAD) return dgrad_on_tensor_cores(g) ? umma_dgrad_ws(g) + splitk_ws(g, pass) : 0;
    if (pass == LAMP_PASS_WGRAD) {
        size_t u = umma_wgrad_ws(g);             // 0 when the tensor-core kernels do not take this shape
        const size_t u2 = win_wgrad_ws(g);
        if (u2 > u) u = u2;
        const size_t tc = u ? u + bias_grad_ws((int64_t)g.n * g.od * g.oh * g.ow, g.co) : 0;
        size_t sm = simt_conv_wgrad_ws(g);
        size_t xb = 0, wb = 0;
        const size_t c1 = c1_padded_ws(g, &xb, &wb);
        if (c1 > sm) sm = c1;
        return tc > sm ? tc : sm;
    }
    return 0;
}

lamp_status_t conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                       double *stats, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (cr_conv_fwd_supported(g, x, y)) return cr_conv_fwd(g, x, w, bias, y, stats, 0, st);
    if (ct_conv_fwd_supported(g, x, y)) return ct_conv_fwd(g, x, w, bias, y, stats, 0, st);
    if (c1_umma_supported(g, x, y)) return c1_umma_fwd(g, x, w, bias, y, stats, st);
    const int kind = fwd_kind(g);
    if (kind >= 0 && umma_conv_supported(kind, g, x, y)) return umma_conv(kind, g, x, w, bias, y, stats, ws, ws_bytes, st);
    return simt_conv_fwd(g, x, w, bias, y, stats, st);
}

// Every tensor-core data gradient reads the weights as [tap][c_in][c_out]: conv_dgrad_prepare writes that form into
// wt (conv_ws_min_bytes(g, LAMP_PASS_DGRAD) bytes; nothing to do for passes that run on the CUDA cores),
// conv_dgrad_run takes it from there.  Callers that run many passes with the same weights prepare once.
static bool dgrad_reads_transposed(const ConvGeom &g, const TView &dy, const TView &dx)
{
    const int kind = dgrad_kind(g);
    return kind >= 0 && umma_conv_supported(kind, g, dy, dx);
}

lamp_status_t conv_dgrad_prepare(const ConvGeom &g, const TView &dy, const TView &dx, const bf16 *w, void *wt,
                                 size_t wt_bytes, cudaStream_t st)
{
    if (!dgrad_reads_transposed(g, dy, dx)) return LAMP_OK;
    if (!wt || wt_bytes < umma_dgrad_ws(g) || !aligned16(wt)) return LAMP_ERR_WORKSPACE;
    return umma_transpose_weights(w, (bf16 *)wt, g.k * g.k * g.k, g.co, g.ci, st);
}

lamp_status_t conv_dgrad_run(const ConvGeom &g, const TView &dy, const bf16 *w, const void *wt, const TView &dx,
                             void *part, size_t part_bytes, cudaStream_t st)
{
    if (!dgrad_reads_transposed(g, dy, dx)) return simt_conv_dgrad(g, dy, w, dx, st);
    if (!wt) return LAMP_ERR_WORKSPACE;
    const int kind = dgrad_kind(g);
    if (kind == UK_S1_DGRAD) {
        ConvGeom t = g;
        t.ci = g.co; t.co = g.ci;
        if (cr_conv_fwd_supported(t, dy, dx)) return cr_conv_fwd(t, dy, (const bf16 *)wt, nullptr, dx, nullptr, 1, st);
        if (ct_conv_fwd_supported(t, dy, dx)) return ct_conv_fwd(t, dy, (const bf16 *)wt, nullptr, dx, nullptr, 1, st);
    }
    return umma_conv(kind, g, dy, (const bf16 *)wt, nullptr, dx, nullptr, part, part_bytes, st);
}

lamp_status_t conv_dgrad(const ConvGeom &g, const TView &dy, const bf16 *w, const TView &dx, void *ws, size_t ws_bytes,
                         cudaStream_t st)
{
    if (!dgrad_reads_transposed(g, dy, dx)) return simt_conv_dgrad(g, dy, w, dx, st);
    const size_t need = umma_dgrad_ws(g);
    if (!ws || ws_bytes < need || !aligned16(ws)) return LAMP_ERR_WORKSPACE;
    const lamp_status_t s = conv_dgrad_prepare(g, dy, dx, w, ws, ws_bytes, st);
    if (s != LAMP_OK) return s;
    return conv_dgrad_run(g, dy, w, ws, dx, (char *)ws + need, ws_bytes - need, st);
}

// The one-channel first layer borrows the windowed tensor-core kernel: x is widened to 32 channels (zeros)
// in scratch, the 27 x c_out x 32 gradient is formed, and its first input-channel column is the answer.
static bool c1_padded_geom(const ConvGeom &g, ConvGeom *p)
{
    if (!(g.ci == 1 && g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed && (g.co == 32 || g.co == 64))) return false;
    *p = g;
    p->ci = 32;
    return win_wgrad_ws(*p) > 0;
}

static size_t c1_padded_ws(const ConvGeom &g, size_t *xpad_bytes, size_t *dw32_bytes)
{
    ConvGeom p;
    if (!c1_padded_geom(g, &p)) return 0;
    *xpad_bytes = align_up((size_t)g.n * g.d * g.h * g.w * 32 * sizeof(bf16), 256);
    *dw32_bytes = align_up((size_t)27 * g.co * 32 * sizeof(float), 256);
    return *xpad_bytes + *dw32_bytes + win_wgrad_ws(p) + bias_grad_ws((int64_t)g.n * g.od * g.oh * g.ow, g.co);
}

lamp_status_t conv_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, float *db, void *ws,
                         size_t ws_bytes, cudaStream_t st)
{
    {
        ConvGeom p;
        size_t xb = 0, wb = 0;
        const size_t need = c1_padded_ws(g, &xb, &wb);
        if (need && c1_padded_geom(g, &p) && dy.pitch % 8 == 0 && ((uintptr_t)dy.p & 15) == 0) {
            if (!ws || ws_bytes < need || !aligned16(ws)) return LAMP_ERR_WORKSPACE;
            char *base = (char *)ws;
            TView xp = x;
            xp.p = base; xp.c = 32; xp.pitch = 32;
            lamp_status_t s = pad_c1(x, (bf16 *)base, st);
            if (s != LAMP_OK) return s;
            const size_t u = win_wgrad_ws(p);
            s = win_wgrad(p, xp, dy, (float *)(base + xb), base + xb + wb, u, st);
            if (s != LAMP_OK) return s;
            s = take_c0((const float *)(base + xb), dw, 27 * g.co, st);
            if (s != LAMP_OK || !db) return s;
            return bias_grad(dy, db, base + xb + wb + u, st);
        }
    }
    if (win_wgrad_supported(g, x, dy)) {
        const size_t u = win_wgrad_ws(g);
        if (!ws || ws_bytes < u + (db ? bias_grad_ws((int64_t)g.n * g.od * g.oh * g.ow, g.co) : 0)) return LAMP_ERR_WORKSPACE;
        lamp_status_t s = win_wgrad(g, x, dy, dw, ws, u, st);
        if (s != LAMP_OK || !db) return s;
        return bias_grad(dy, db, (char *)ws + u, st);
    }
    if (umma_wgrad_supported(g, x, dy)) {
        const size_t u = umma_wgrad_ws(g);
        if (!ws || ws_bytes < u + (db ? bias_grad_ws((int64_t)g.n * g.od * g.oh * g.ow, g.co) : 0)) return LAMP_ERR_WORKSPACE;
        lamp_status_t s = umma_wgrad(g, x, dy, dw, ws, u, st);
        if (s != LAMP_OK || !db) return s;
        return bias_grad(dy, db, (char *)ws + u, st);
    }
    return simt_conv_wgrad(g, x, dy, dw, db, ws, ws_bytes, st);
}

}  // namespace lamp

using namespace lamp;

extern "C" {

size_t lamp_conv3d_workspace_bytes(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, int pass)
{
    ConvGeom g;
    if (!x || conv_geom(desc, x, nullptr, &g) != LAMP_OK) return 0;
    return conv_ws_bytes(g, pass);
}

size_t lamp_conv3d_workspace_min_bytes(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, int pass)
{
    ConvGeom g;
    if (!x || conv_geom(desc, x, nullptr, &g) != LAMP_OK) return 0;
    return conv_ws_min_bytes(g, pass);
}

lamp_status_t lamp_conv3d_fwd(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, const void *w,
                              const float *bias, lamp_tensor_t *y, double *stats,
                              void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!desc || !x || !w || !y) return LAMP_ERR_INVALID_ARG;
    lamp_status_t s;
    if ((s = check_tensor(x, false, true)) != LAMP_OK) return s;
    if ((s = check_tensor(y, true, true)) != LAMP_OK) return s;
    if (!aligned16(w)) return LAMP_ERR_INVALID_ARG;
    ConvGeom g;
    if ((s = conv_geom(desc, x, y, &g)) != LAMP_OK) return s;
    return conv_fwd(g, make_view(x), (const bf16 *)w, bias, make_view(y), stats, ws, ws_bytes, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_conv3d_dgrad(const lamp_conv_desc_t *desc, const lamp_tensor_t *dy, const void *w,
                                lamp_tensor_t *dx, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!desc || !dy || !w || !dx) return LAMP_ERR_INVALID_ARG;
    lamp_status_t s;
    if ((s = check_tensor(dy, false, true)) != LAMP_OK) return s;
    if ((s = check_tensor(dx, true, true)) != LAMP_OK) return s;
    if (!aligned16(w)) return LAMP_ERR_INVALID_ARG;
    ConvGeom g;
    if ((s = conv_geom(desc, dx, dy, &g)) != LAMP_OK) return s;
    return conv_dgrad(g, make_view(dy), (const bf16 *)w, make_view(dx), ws, ws_bytes, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_conv3d_wgrad(const lamp_conv_desc_t *desc, const lamp_tensor_t *x, const lamp_tensor_t *dy,
                                float *dw, float *dbias, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!desc || !x || !dy || !dw) return LAMP_ERR_INVALID_ARG;
    lamp_status_t s;
    if ((s = check_tensor(x, false, true)) != LAMP_OK) return s;
    if ((s = check_tensor(dy, false, true)) != LAMP_OK) return s;
    ConvGeom g;
    if ((s = conv_geom(desc, x, dy, &g)) != LAMP_OK) return s;
    if (conv_ws_bytes(g, LAMP_PASS_WGRAD) > 0 && (!ws || !aligned16(ws))) return LAMP_ERR_WORKSPACE;
    return conv_wgrad(g, make_view(x), make_view(dy), dw, dbias, ws, ws_bytes, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_instnorm_relu_fwd(const lamp_tensor_t *y, const double *stats, float eps,
                                     float *mu_rstd, lamp_tensor_t *z, void *cuda_stream)
{
    if (!y || !stats || !mu_rstd || !z) return LAMP_ERR_INVALID_ARG;
    lamp_status_t s;
    if ((s = check_tensor(y, false, false)) != LAMP_OK) return s;
    if ((s = check_tensor(z, false, false)) != LAMP_OK) return s;
    if (y->n != z->n || y->d != z->d || y->h != z->h || y->w != z->w || y->c != z->c) return LAMP_ERR_INVALID_ARG;
    return k_instnorm_relu_fwd(make_view(y), stats, eps, mu_rstd, make_view(z), (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_instnorm_relu_bwd(const lamp_tensor_t *dz_a, const lamp_tensor_t *dz_b,
                                     const lamp_tensor_t *y, const float *mu_rstd,
                                     double *sums, lamp_tensor_t *dy, void *cuda_stream)
{
    if (!dz_a || !y || !mu_rstd || !sums || !dy) return LAMP_ERR_INVALID_ARG;
    lamp_status_t s;
    const lamp_tensor_t *all[4] = {dz_a, dz_b, y, dy};
    for (int i = 0; i < 4; ++i) {
        if (!all[i]) continue;
        if ((s = check_tensor(all[i], false, false)) != LAMP_OK) return s;
        if (all[i]->n != y->n || all[i]->d != y->d || all[i]->h != y->h || all[i]->w != y->w || all[i]->c != y->c)
            return LAMP_ERR_INVALID_ARG;
    }
    TView vb{};
    if (dz_b) vb = make_view(dz_b);
    return k_instnorm_relu_bwd(make_view(dz_a), dz_b ? &vb : nullptr, make_view(y), mu_rstd, sums, false, make_view(dy),
                               nullptr, nullptr, nullptr, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_rmsprop_step(int64_t n, const float *grad, float *master, float *v, void *param_bf16,
                                float lr, float alpha, float eps, void *cuda_stream)
{
    if (n < 0) return LAMP_ERR_INVALID_ARG;
    if (n == 0) return LAMP_OK;
    if (!grad || !master || !v) return LAMP_ERR_INVALID_ARG;
    if (!(lr >= 0.f) || !(alpha >= 0.f && alpha <= 1.f) || !(eps >= 0.f)) return LAMP_ERR_INVALID_ARG;
    if ((((uintptr_t)grad | (uintptr_t)master | (uintptr_t)v) & 3) || ((uintptr_t)param_bf16 & 1)) return LAMP_ERR_INVALID_ARG;
    return k_rmsprop(n, grad, master, v, (bf16 *)param_bf16, lr, alpha, eps, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_get_async_status(void *cuda_stream)
{
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return LAMP_ERR_CUDA;
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_status_word, sizeof(int)) != cudaSuccess) return LAMP_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)) != cudaSuccess) return LAMP_ERR_CUDA;
    return (lamp_status_t)v;
}

const char *lamp_status_string(lamp_status_t s)
{
    switch (s) {
    case LAMP_OK: return "ok";
    case LAMP_ERR_INVALID_ARG: return "invalid argument";
    case LAMP_ERR_UNSUPPORTED: return "unsupported configuration";
    case LAMP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case LAMP_ERR_CUDA: return "CUDA call failed";
    case LAMP_ERR_TIMEOUT: return "device-side wait timed out";
    case LAMP_ERR_NOT_IMPLEMENTED: return "not implemented";
    case LAMP_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the library's built-in static array";
    }
    return "unknown status";
}

// One CTA waits, with the kernels' own bounded wait, on an mbarrier that nothing ever arrives on.
__global__ void wait_timeout_selftest_kernel(int *status, long long limit_clocks)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        ptx::mbar_init_fence();
    }
    __syncthreads();
    const bool ok = ptx::mbar_wait(ptx::smem_u32(&bar), 0, &abort_flag, limit_clocks);
    __syncthreads();
    if (threadIdx.x == 0 && !ok && status) atomicExch(status, (int)LAMP_ERR_TIMEOUT);
}

lamp_status_t lamp_selftest_wait_timeout(void *cuda_stream)
{
    int *st = status_word_ptr();
    if (!st) return LAMP_ERR_CUDA;
    wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(st, 20000000ll);      // about 10 ms
    return launch_status();
}

const char *lamp_version(void) { return "lamp-b200 sm_100a"; }

}  // extern "C"
