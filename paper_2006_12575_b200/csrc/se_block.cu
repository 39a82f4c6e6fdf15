// Squeeze-and-excitation residual block (the SEU-Net variant of the network: Sec. 1, Sec. 3, Tables 2, 3, 5), as
// steps around the conv -> InstanceNorm -> ReLU layers:
//
//   z = relu((y - mu) * rstd)  of the level's LAST conv (y: its stored raw output), r = output of its FIRST conv,
//   s[n,c] = mean_v z,   h = relu(W1 s + b1),   e = sigmoid(W2 h + b2),   out = r + e[n,c] * z.
//
// z itself is never stored: the squeeze pass reads y and forms the sums, the apply pass reads y again (and r) and
// writes out.  Both are HBM-bound passes with 16-byte accesses; the two small matrix products run in one block.
// Backward: de[n,c] = sum_v dout * z (one pass over dout and y), the excitation's backward in one block, then
// dz = e * dout + ds / V (one pass), which the InstanceNorm backward of the last conv takes as its incoming gradient;
// the residual branch receives dout unchanged (the second gradient source of the first conv's InstanceNorm backward).
#include "common.cuh"

namespace lamp {

namespace {

constexpr int SE_THREADS = 256;

// sums[n][c] += sum over this block's voxels of f(v, c): thread = (8-channel group, voxel lane)
// MODE 0: f = relu((y - mu) * rstd);  MODE 1: f = dout * relu((y - mu) * rstd)
template <int MODE>
__global__ void __launch_bounds__(SE_THREADS)
se_reduce_kernel(const bf16 *__restrict__ y, int64_t yp, const bf16 *__restrict__ g, int64_t gp,
                 const float *__restrict__ mu_rstd, double *__restrict__ sums, int64_t Vn, int C, int64_t v_per_block)
{
    extern __shared__ float red[];                 // [lanes][C]
    pdl_launch_dependents();
    pdl_wait();
    const int G = C >> 3, lanes = SE_THREADS / G;
    const int cg = threadIdx.x % G, vl = threadIdx.x / G;
    const int n = blockIdx.y;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    if (vl < lanes) {
        float mu[8], rs[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            mu[i] = mu_rstd[((int64_t)n * C + cg * 8 + i) * 2];
            rs[i] = mu_rstd[((int64_t)n * C + cg * 8 + i) * 2 + 1];
        }
        const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(Vn, v0 + v_per_block);
        for (int64_t v = v0 + vl; v < v1; v += lanes) {
            const int64_t vox = (int64_t)n * Vn + v;
            float fy[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(y + vox * yp) + cg), fy);
            if (MODE == 1) {
                float fg[8];
                unpack8(__ldg(reinterpret_cast<const uint4 *>(g + vox * gp) + cg), fg);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i] = fmaf(fg[i], fmaxf((fy[i] - mu[i]) * rs[i], 0.f), acc[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i] += fmaxf((fy[i] - mu[i]) * rs[i], 0.f);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) red[vl * C + cg * 8 + i] = acc[i];
    }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += SE_THREADS) {
        float a = 0.f;
        for (int l = 0; l < lanes; ++l) a += red[l * C + c];
        atomicAdd(sums + (int64_t)n * C + c, (double)a);
    }
}

// one block per sample: mean, hidden layer, excitation
__global__ void __launch_bounds__(SE_THREADS)
se_excite_kernel(const double *__restrict__ sums, double inv_v, int C, int Cr, const float *__restrict__ w1,
                 const float *__restrict__ b1, const float *__restrict__ w2, const float *__restrict__ b2,
                 float *__restrict__ e, float *__restrict__ hidden, float *__restrict__ mean)
{
    extern __shared__ float sm[];                  // mean [C], hidden [Cr]
    pdl_launch_dependents();
    pdl_wait();
    float *s = sm, *h = sm + C;
    const int n = blockIdx.x;
    for (int c = threadIdx.x; c < C; c += SE_THREADS) {
        s[c] = (float)(sums[(int64_t)n * C + c] * inv_v);
        mean[(int64_t)n * C + c] = s[c];
    }
    __syncthreads();
    for (int j = threadIdx.x; j < Cr; j += SE_THREADS) {
        float a = b1[j];
        for (int c = 0; c < C; ++c) a = fmaf(w1[(int64_t)j * C + c], s[c], a);
        h[j] = fmaxf(a, 0.f);
        hidden[(int64_t)n * Cr + j] = h[j];
    }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += SE_THREADS) {
        float a = b2[c];
        for (int j = 0; j < Cr; ++j) a = fmaf(w2[(int64_t)c * Cr + j], h[j], a);
        e[(int64_t)n * C + c] = 1.0f / (1.0f + expf(-a));
    }
}

// out = r + e * relu((y - mu) * rstd)    (r may be absent)
__global__ void __launch_bounds__(SE_THREADS)
se_apply_fwd_kernel(const bf16 *__restrict__ y, int64_t yp, const bf16 *__restrict__ r, int64_t rp,
                    const float *__restrict__ mu_rstd, const float *__restrict__ e, bf16 *__restrict__ out, int64_t op,
                    int64_t Vn, int C, int64_t total)
{
    pdl_launch_dependents();
    pdl_wait();
    const int G = C >> 3;
    const int64_t t = (int64_t)blockIdx.x * SE_THREADS + threadIdx.x;
    if (t >= total) return;
    const int cg = (int)(t % G);
    const int64_t vox = t / G;
    const int n = (int)(vox / Vn);
    float fy[8], fr[8], o[8];
    unpack8(__ldg(reinterpret_cast<const uint4 *>(y + vox * yp) + cg), fy);
    if (r) unpack8(__ldg(reinterpret_cast<const uint4 *>(r + vox * rp) + cg), fr);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t nc = (int64_t)n * C + cg * 8 + i;
        const float z = fmaxf((fy[i] - mu_rstd[nc * 2]) * mu_rstd[nc * 2 + 1], 0.f);
        o[i] = fmaf(e[nc], z, r ? fr[i] : 0.f);
    }
    reinterpret_cast<uint4 *>(out + vox * op)[cg] = pack8(o);
}

// dz = e * dout + ds_over_v
__global__ void __launch_bounds__(SE_THREADS)
se_apply_bwd_kernel(const bf16 *__restrict__ g, int64_t gp, const float *__restrict__ e, const float *__restrict__ dsv,
                    bf16 *__restrict__ dz, int64_t dp, int64_t Vn, int C, int64_t total)
{
    pdl_launch_dependents();
    pdl_wait();
    const int G = C >> 3;
    const int64_t t = (int64_t)blockIdx.x * SE_THREADS + threadIdx.x;
    if (t >= total) return;
    const int cg = (int)(t % G);
    const int64_t vox = t / G;
    const int n = (int)(vox / Vn);
    float fg[8], o[8];
    unpack8(__ldg(reinterpret_cast<const uint4 *>(g + vox * gp) + cg), fg);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t nc = (int64_t)n * C + cg * 8 + i;
        o[i] = fmaf(e[nc], fg[i], dsv[nc]);
    }
    reinterpret_cast<uint4 *>(dz + vox * dp)[cg] = pack8(o);
}

// One block: backward of the two small layers for all samples.
//   dt = de * e (1 - e);  dW2 = dt^T h;  db2 = sum_n dt;  dh = (dt W2) [h > 0];  dW1 = dh^T s;  db1 = sum_n dh;
//   ds_over_v = (dh W1) / V
__global__ void __launch_bounds__(SE_THREADS)
se_excite_bwd_kernel(const double *__restrict__ de_sums, double inv_v, int N, int C, int Cr, const float *__restrict__ e,
                     const float *__restrict__ hidden, const float *__restrict__ mean, const float *__restrict__ w1,
                     const float *__restrict__ w2, float *__restrict__ dsv, float *__restrict__ dw1, float *__restrict__ db1,
                     float *__restrict__ dw2, float *__restrict__ db2)
{
    extern __shared__ float sm[];                  // dt [N][C], dh [N][Cr]
    pdl_launch_dependents();
    pdl_wait();
    float *dt = sm, *dh = sm + (size_t)N * C;
    for (int i = threadIdx.x; i < N * C; i += SE_THREADS) dt[i] = (float)de_sums[i] * e[i] * (1.0f - e[i]);
    __syncthreads();
    for (int i = threadIdx.x; i < N * Cr; i += SE_THREADS) {
        const int n = i / Cr, j = i - n * Cr;
        float a = 0.f;
        for (int c = 0; c < C; ++c) a = fmaf(dt[n * C + c], w2[(int64_t)c * Cr + j], a);
        dh[i] = hidden[i] > 0.f ? a : 0.f;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < C * Cr; i += SE_THREADS) {
        const int c = i / Cr, j = i - c * Cr;
        float a2 = 0.f, a1 = 0.f;
        for (int n = 0; n < N; ++n) {
            a2 = fmaf(dt[n * C + c], hidden[n * Cr + j], a2);
            a1 = fmaf(dh[n * Cr + j], mean[n * C + c], a1);
        }
        dw2[(int64_t)c * Cr + j] = a2;
        dw1[(int64_t)j * C + c] = a1;
    }
    for (int c = threadIdx.x; c < C; c += SE_THREADS) {
        float a = 0.f;
        for (int n = 0; n < N; ++n) a += dt[n * C + c];
        db2[c] = a;
    }
    for (int j = threadIdx.x; j < Cr; j += SE_THREADS) {
        float a = 0.f;
        for (int n = 0; n < N; ++n) a += dh[n * Cr + j];
        db1[j] = a;
    }
    for (int i = threadIdx.x; i < N * C; i += SE_THREADS) {
        const int n = i / C, c = i - n * C;
        float a = 0.f;
        for (int j = 0; j < Cr; ++j) a = fmaf(dh[n * Cr + j], w1[(int64_t)j * C + c], a);
        dsv[i] = (float)((double)a * inv_v);
    }
}

// mu = S1 / V, rstd = (S2 / V - mu^2 + eps)^-1/2 from the fp64 sums, as the normalise kernel derives them
__global__ void __launch_bounds__(SE_THREADS)
mu_rstd_kernel(const double *__restrict__ stats, double inv_v, float eps, float *__restrict__ mr, int nc)
{
    pdl_launch_dependents();
    pdl_wait();
    const int i = blockIdx.x * SE_THREADS + threadIdx.x;
    if (i >= nc) return;
    const double m = stats[2 * i] * inv_v;
    double var = stats[2 * i + 1] * inv_v - m * m;
    if (var < 0.0) var = 0.0;
    mr[2 * i] = (float)m;
    mr[2 * i + 1] = __frsqrt_rn((float)var + eps);
}

// out = a + b (bf16, fp32 add)
__global__ void __launch_bounds__(SE_THREADS)
add2_kernel(const bf16 *__restrict__ a, int64_t ap, const bf16 *__restrict__ b, int64_t bp, bf16 *__restrict__ o, int64_t op,
            int C, int64_t total)
{
    pdl_launch_dependents();
    pdl_wait();
    const int G = C >> 3;
    const int64_t t = (int64_t)blockIdx.x * SE_THREADS + threadIdx.x;
    if (t >= total) return;
    const int cg = (int)(t % G);
    const int64_t vox = t / G;
    float fa[8], fb[8];
    unpack8(__ldg(reinterpret_cast<const uint4 *>(a + vox * ap) + cg), fa);
    unpack8(__ldg(reinterpret_cast<const uint4 *>(b + vox * bp) + cg), fb);
#pragma unroll
    for (int i = 0; i < 8; ++i) fa[i] += fb[i];
    reinterpret_cast<uint4 *>(o + vox * op)[cg] = pack8(fa);
}

bool se_tensor_ok(const lamp_tensor_t *t)
{
    return t && t->ptr && t->dtype == LAMP_BF16 && t->c > 0 && t->c % 8 == 0 && t->c_pitch % 8 == 0 && t->c_offset % 8 == 0 &&
           t->c_offset >= 0 && t->c_pitch >= (int64_t)t->c_offset + t->c && (((uintptr_t)t->ptr) & 15) == 0 && t->n >= 0 &&
           t->d >= 0 && t->h >= 0 && t->w >= 0 && t->c <= 2048;
}

bool same_shape(const lamp_tensor_t *a, const lamp_tensor_t *b)
{
    return a->n == b->n && a->d == b->d && a->h == b->h && a->w == b->w && a->c == b->c;
}

lamp_status_t se_reduce(int mode, const lamp_tensor_t *y, const lamp_tensor_t *g, const float *mu_rstd, double *sums, cudaStream_t st)
{
    const TView vy = make_view(y);
    const int64_t Vn = (int64_t)y->d * y->h * y->w;
    LAMP_CUDA_OK(cudaMemsetAsync(sums, 0, (size_t)y->n * y->c * sizeof(double), st));
    if (Vn == 0 || y->n == 0) return LAMP_OK;
    const int G = y->c / 8;
    if (G > SE_THREADS) return LAMP_ERR_UNSUPPORTED;
    const int lanes = SE_THREADS / G;
    int64_t blocks = (sm_count() * 8 + y->n - 1) / y->n;
    const int64_t max_blocks = (Vn + lanes * 16 - 1) / (lanes * 16);
    if (blocks > max_blocks) blocks = max_blocks;
    const int64_t vpb = (Vn + blocks - 1) / blocks;
    blocks = (Vn + vpb - 1) / vpb;
    const size_t smem = (size_t)lanes * y->c * sizeof(float);
    const dim3 grid((unsigned)blocks, y->n);
    if (mode == 0)
        (void)launch_pdl(false, se_reduce_kernel<0>, grid, dim3(SE_THREADS), smem, st, (const bf16 *)vy.p, vy.pitch, (const bf16 *)nullptr,
                         (int64_t)0, mu_rstd, sums, Vn, y->c, vpb);
    else {
        const TView vg = make_view(g);
        (void)launch_pdl(false, se_reduce_kernel<1>, grid, dim3(SE_THREADS), smem, st, (const bf16 *)vy.p, vy.pitch, (const bf16 *)vg.p,
                         vg.pitch, mu_rstd, sums, Vn, y->c, vpb);
    }
    return launch_status();
}

lamp_tensor_t as_tensor(const TView &v)
{
    lamp_tensor_t t;
    t.ptr = v.p; t.dtype = LAMP_BF16; t.n = v.n; t.d = v.d; t.h = v.h; t.w = v.w; t.c = v.c; t.c_pitch = v.pitch; t.c_offset = 0;
    return t;
}

}  // namespace

lamp_status_t k_mu_rstd(const double *stats, int64_t Vn, float eps, float *mr, int nc, cudaStream_t st)
{
    if (nc <= 0 || Vn <= 0) return LAMP_OK;
    (void)launch_pdl(true, mu_rstd_kernel, dim3((nc + SE_THREADS - 1) / SE_THREADS), dim3(SE_THREADS), (size_t)0, st, stats,
                     1.0 / (double)Vn, eps, mr, nc);
    return launch_status();
}

lamp_status_t k_add2(const TView &a, const TView &b, const TView &out, cudaStream_t st)
{
    const int64_t total = (int64_t)a.n * a.d * a.h * a.w * (a.c / 8);
    if (total == 0) return LAMP_OK;
    if (a.c % 8 || a.pitch % 8 || b.pitch % 8 || out.pitch % 8) return LAMP_ERR_UNSUPPORTED;
    (void)launch_pdl(false, add2_kernel, dim3((unsigned)((total + SE_THREADS - 1) / SE_THREADS)), dim3(SE_THREADS), (size_t)0, st,
                     (const bf16 *)a.p, a.pitch, (const bf16 *)b.p, b.pitch, (bf16 *)out.p, out.pitch, a.c, total);
    return launch_status();
}

// params: W1 [cr][c], b1 [cr], W2 [c][cr], b2 [c] back to back (fp32); dparams likewise
lamp_status_t k_se_fwd(const TView &y, const float *mr, const float *params, int cr, double *sums, float *e, float *hid,
                       float *mean, const TView *res, const TView &out, cudaStream_t st)
{
    const lamp_tensor_t ty = as_tensor(y), to = as_tensor(out);
    lamp_tensor_t tr{};
    if (res) tr = as_tensor(*res);
    const int c = y.c;
    const int64_t Vn = (int64_t)y.d * y.h * y.w;
    if (Vn == 0 || y.n == 0) return LAMP_OK;
    const float *w1 = params, *b1 = w1 + (size_t)cr * c, *w2 = b1 + cr, *b2 = w2 + (size_t)c * cr;
    lamp_status_t s = lamp_se_squeeze(&ty, mr, sums, st);
    if (s != LAMP_OK) return s;
    s = lamp_se_excite(sums, Vn, y.n, c, cr, w1, b1, w2, b2, e, hid, mean, st);
    if (s != LAMP_OK) return s;
    lamp_tensor_t tout = to;
    return lamp_se_apply_fwd(&ty, mr, e, res ? &tr : nullptr, &tout, st);
}

lamp_status_t k_se_bwd(const TView &dout, const TView &y, const float *mr, const float *params, int cr, const float *e,
                       const float *hid, const float *mean, double *de, float *dsv, float *dparams, const TView &dz,
                       cudaStream_t st)
{
    const lamp_tensor_t tg = as_tensor(dout), ty = as_tensor(y);
    lamp_tensor_t tz = as_tensor(dz);
    const int c = y.c;
    const int64_t Vn = (int64_t)y.d * y.h * y.w;
    if (Vn == 0 || y.n == 0) return LAMP_OK;
    const float *w1 = params, *w2 = params + (size_t)cr * c + cr;
    float *dw1 = dparams, *db1 = dw1 + (size_t)cr * c, *dw2 = db1 + cr, *db2 = dw2 + (size_t)c * cr;
    lamp_status_t s = lamp_se_bwd_reduce(&tg, &ty, mr, de, st);
    if (s != LAMP_OK) return s;
    s = lamp_se_excite_bwd(de, Vn, y.n, c, cr, e, hid, mean, w1, w2, dsv, dw1, db1, dw2, db2, st);
    if (s != LAMP_OK) return s;
    return lamp_se_apply_bwd(&tg, e, dsv, &tz, st);
}

}  // namespace lamp

using namespace lamp;

extern "C" {

lamp_status_t lamp_se_squeeze(const lamp_tensor_t *y, const float *mu_rstd, double *sums, void *cuda_stream)
{
    if (!se_tensor_ok(y) || !mu_rstd || !sums) return LAMP_ERR_INVALID_ARG;
    return se_reduce(0, y, nullptr, mu_rstd, sums, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_se_excite(const double *sums, int64_t voxels_per_sample, int32_t n, int32_t c, int32_t cr,
                             const float *w1, const float *b1, const float *w2, const float *b2,
                             float *e, float *hidden, float *mean, void *cuda_stream)
{
    if (!sums || !w1 || !b1 || !w2 || !b2 || !e || !hidden || !mean) return LAMP_ERR_INVALID_ARG;
    if (n < 0 || c <= 0 || cr <= 0 || voxels_per_sample <= 0) return LAMP_ERR_INVALID_ARG;
    if (c > 2048 || cr > 2048) return LAMP_ERR_UNSUPPORTED;
    if (n == 0) return LAMP_OK;
    (void)launch_pdl(true, se_excite_kernel, dim3(n), dim3(SE_THREADS), (size_t)(c + cr) * sizeof(float), (cudaStream_t)cuda_stream,
                     sums, 1.0 / (double)voxels_per_sample, (int)c, (int)cr, w1, b1, w2, b2, e, hidden, mean);
    return launch_status();
}

lamp_status_t lamp_se_apply_fwd(const lamp_tensor_t *y, const float *mu_rstd, const float *e,
                                const lamp_tensor_t *residual, lamp_tensor_t *out, void *cuda_stream)
{
    if (!se_tensor_ok(y) || !se_tensor_ok(out) || !mu_rstd || !e || !same_shape(y, out)) return LAMP_ERR_INVALID_ARG;
    if (residual && (!se_tensor_ok(residual) || !same_shape(y, residual))) return LAMP_ERR_INVALID_ARG;
    const int64_t Vn = (int64_t)y->d * y->h * y->w, total = (int64_t)y->n * Vn * (y->c / 8);
    if (total == 0) return LAMP_OK;
    const TView vy = make_view(y), vo = make_view(out);
    TView vr{};
    if (residual) vr = make_view(residual);
    (void)launch_pdl(false, se_apply_fwd_kernel, dim3((unsigned)((total + SE_THREADS - 1) / SE_THREADS)), dim3(SE_THREADS), (size_t)0,
                     (cudaStream_t)cuda_stream, (const bf16 *)vy.p, vy.pitch, residual ? (const bf16 *)vr.p : (const bf16 *)nullptr,
                     residual ? vr.pitch : (int64_t)0, mu_rstd, e, (bf16 *)vo.p, vo.pitch, Vn, (int)y->c, total);
    return launch_status();
}

lamp_status_t lamp_se_bwd_reduce(const lamp_tensor_t *dout, const lamp_tensor_t *y, const float *mu_rstd,
                                 double *de_sums, void *cuda_stream)
{
    if (!se_tensor_ok(y) || !se_tensor_ok(dout) || !same_shape(y, dout) || !mu_rstd || !de_sums) return LAMP_ERR_INVALID_ARG;
    return se_reduce(1, y, dout, mu_rstd, de_sums, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_se_excite_bwd(const double *de_sums, int64_t voxels_per_sample, int32_t n, int32_t c, int32_t cr,
                                 const float *e, const float *hidden, const float *mean, const float *w1, const float *w2,
                                 float *ds_over_v, float *dw1, float *db1, float *dw2, float *db2, void *cuda_stream)
{
    if (!de_sums || !e || !hidden || !mean || !w1 || !w2 || !ds_over_v || !dw1 || !db1 || !dw2 || !db2) return LAMP_ERR_INVALID_ARG;
    if (n <= 0 || c <= 0 || cr <= 0 || voxels_per_sample <= 0) return LAMP_ERR_INVALID_ARG;
    const size_t smem = (size_t)n * (c + cr) * sizeof(float);
    if (c > 2048 || cr > 2048 || smem > 48 * 1024) return LAMP_ERR_UNSUPPORTED;
    (void)launch_pdl(true, se_excite_bwd_kernel, dim3(1), dim3(SE_THREADS), smem, (cudaStream_t)cuda_stream, de_sums,
                     1.0 / (double)voxels_per_sample, (int)n, (int)c, (int)cr, e, hidden, mean, w1, w2, ds_over_v, dw1, db1, dw2, db2);
    return launch_status();
}

lamp_status_t lamp_se_apply_bwd(const lamp_tensor_t *dout, const float *e, const float *ds_over_v, lamp_tensor_t *dz,
                                void *cuda_stream)
{
    if (!se_tensor_ok(dout) || !se_tensor_ok(dz) || !same_shape(dout, dz) || !e || !ds_over_v) return LAMP_ERR_INVALID_ARG;
    const int64_t Vn = (int64_t)dout->d * dout->h * dout->w, total = (int64_t)dout->n * Vn * (dout->c / 8);
    if (total == 0) return LAMP_OK;
    const TView vg = make_view(dout), vd = make_view(dz);
    (void)launch_pdl(false, se_apply_bwd_kernel, dim3((unsigned)((total + SE_THREADS - 1) / SE_THREADS)), dim3(SE_THREADS), (size_t)0,
                     (cudaStream_t)cuda_stream, (const bf16 *)vg.p, vg.pitch, e, ds_over_v, (bf16 *)vd.p, vd.pitch, Vn, (int)dout->c, total);
    return launch_status();
}

}  // extern "C"
