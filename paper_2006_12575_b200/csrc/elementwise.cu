// HBM-bound kernels of the U-Net path: InstanceNorm statistics -> (mu, rstd), normalise + ReLU
// into a concat slice, its backward, the 1x1x1 head with softmax and Dice sums, the Dice
// gradient with the head's backward, patch gather and Gaussian-weighted overlap-add.
// All activation accesses are 16-byte vectors along the channel axis (bf16 x 8).
#include "common.cuh"

namespace lamp {

namespace {

// ------------------------------------------------------------------ InstanceNorm forward
// thread = (voxel row r of the block, group g of 8 channels); the per-channel constants stay in registers
// while the thread walks its voxels.  Every thread derives (mu, rstd) of its 8 channels from the fp64 sums - the
// mean and variance in fp64, the reciprocal square root as one correctly rounded fp32 operation - and the
// first block of each sample also stores them for the backward pass.
__global__ void __launch_bounds__(256)
instnorm_relu_fwd_kernel(const bf16 *__restrict__ y, int64_t yp, const double *__restrict__ stats, double inv_v, float eps,
                         float *__restrict__ mr, bf16 *__restrict__ z, int64_t zp, int64_t Vn, int C, int64_t v_per_block)
{
    const int G = C >> 3, RB = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    if (r >= RB) return;
    const int n = blockIdx.y;
    float mu[8], rs[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int64_t i = (int64_t)n * C + g * 8 + j;
        const double m = stats[2 * i] * inv_v;
        double var = stats[2 * i + 1] * inv_v - m * m;
        if (var < 0.0) var = 0.0;
        mu[j] = (float)m;
        rs[j] = __frsqrt_rn((float)var + eps);
        if (blockIdx.x == 0 && r == 0) { mr[2 * i] = mu[j]; mr[2 * i + 1] = rs[j]; }
    }
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(Vn, v0 + v_per_block);
#pragma unroll 4
    for (int64_t vv = v0 + r; vv < v1; vv += RB) {
        const int64_t v = (int64_t)n * Vn + vv;
        float f[8];
        unpack8(__ldg(reinterpret_cast<const uint4 *>(y + v * yp + g * 8)), f);
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] = fmaxf((f[j] - mu[j]) * rs[j], 0.f);
        *reinterpret_cast<uint4 *>(z + v * zp + g * 8) = pack8(f);
    }
}

// ------------------------------------------------------------------ InstanceNorm backward
// pass 1: per (n, c)  sum g  and  sum g * xhat,  g = (dza + dzb) * [xhat > 0]
__global__ void __launch_bounds__(256)
instnorm_bwd_sums_kernel(const bf16 *__restrict__ dza, int64_t ap, const bf16 *__restrict__ dzb, int64_t bp,
                         const bf16 *__restrict__ y, int64_t yp, const float *__restrict__ mr,
                         double *__restrict__ sums, int64_t Vn, int C, int64_t v_per_block)
{
    extern __shared__ float red[];          // [RB][G][16]
    const int G = C >> 3;
    const int RB = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    const int n = blockIdx.y;
    float s[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) s[j] = 0.f;
    if (r < RB) {
        float mu[8], rs[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            mu[j] = mr[((int64_t)n * C + g * 8 + j) * 2];
            rs[j] = mr[((int64_t)n * C + g * 8 + j) * 2 + 1];
        }
        const int64_t v0 = (int64_t)blockIdx.x * v_per_block;
        const int64_t v1 = min(Vn, v0 + v_per_block);
#pragma unroll 4
        for (int64_t vv = v0 + r; vv < v1; vv += RB) {
            const int64_t v = (int64_t)n * Vn + vv;
            float fy[8], fa[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(y + v * yp + g * 8)), fy);
            unpack8(__ldg(reinterpret_cast<const uint4 *>(dza + v * ap + g * 8)), fa);
            if (dzb) {
                float fb[8];
                unpack8(__ldg(reinterpret_cast<const uint4 *>(dzb + v * bp + g * 8)), fb);
#pragma unroll
                for (int j = 0; j < 8; ++j) fa[j] += fb[j];
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float xh = (fy[j] - mu[j]) * rs[j];
                const float gg = xh > 0.f ? fa[j] : 0.f;
                s[j] += gg;
                s[8 + j] = fmaf(gg, xh, s[8 + j]);
            }
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) red[(r * G + g) * 16 + j] = s[j];
    }
    __syncthreads();
    // thread t < G*16 sums column t over the RB rows
    for (int t = threadIdx.x; t < G * 16; t += 256) {
        double acc = 0.0;
        for (int rr = 0; rr < RB; ++rr) acc += red[rr * G * 16 + t];
        const int gg = t / 16, j = t % 16;
        const int c = gg * 8 + (j & 7);
        atomicAdd(&sums[((int64_t)n * C + c) * 2 + (j >> 3)], acc);
    }
}

// pass 2: dy = rstd * (g - m1 - xhat * m2); same thread layout as the forward kernel
__global__ void __launch_bounds__(256)
instnorm_bwd_apply_kernel(const bf16 *__restrict__ dza, int64_t ap, const bf16 *__restrict__ dzb, int64_t bp,
                          const bf16 *__restrict__ y, int64_t yp, const float *__restrict__ mr,
                          const double *__restrict__ sums, bf16 *__restrict__ dy, int64_t dp, int64_t Vn, int C,
                          int64_t v_per_block)
{
    const int G = C >> 3, RB = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    if (r >= RB) return;
    const int n = blockIdx.y;
    const float inv_v = 1.0f / (float)Vn;
    float mu[8], rs[8], m1[8], m2[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int64_t i = (int64_t)n * C + g * 8 + j;
        mu[j] = mr[2 * i];
        rs[j] = mr[2 * i + 1];
        m1[j] = (float)sums[2 * i] * inv_v;
        m2[j] = (float)sums[2 * i + 1] * inv_v;
    }
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(Vn, v0 + v_per_block);
#pragma unroll 2
    for (int64_t vv = v0 + r; vv < v1; vv += RB) {
        const int64_t v = (int64_t)n * Vn + vv;
        float fy[8], fa[8];
        unpack8(__ldg(reinterpret_cast<const uint4 *>(y + v * yp + g * 8)), fy);
        unpack8(__ldg(reinterpret_cast<const uint4 *>(dza + v * ap + g * 8)), fa);
        if (dzb) {
            float fb[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(dzb + v * bp + g * 8)), fb);
#pragma unroll
            for (int j = 0; j < 8; ++j) fa[j] += fb[j];
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float xh = (fy[j] - mu[j]) * rs[j];
            const float gg = xh > 0.f ? fa[j] : 0.f;
            fa[j] = rs[j] * (gg - m1[j] - xh * m2[j]);
        }
        *reinterpret_cast<uint4 *>(dy + v * dp + g * 8) = pack8(fa);
    }
}

// ------------------------------------------------------------------ head: 1x1x1 conv + softmax (+ Dice sums)
constexpr int KMAX = 16;

__global__ void __launch_bounds__(256)
head_softmax_kernel(const bf16 *__restrict__ z, int64_t zp, int C, const bf16 *__restrict__ w,
                    const float *__restrict__ b, int K, float *__restrict__ probs, uint8_t *__restrict__ amax,
                    const uint8_t *__restrict__ labels, double *__restrict__ dice, int64_t Vn, int64_t v_per_block)
{
    extern __shared__ float sm[];           // w as float [K][C], then bias [K], then reduce [3*KMAX]
    float *sw = sm, *sb = sm + K * C, *sred = sb + KMAX;
    for (int i = threadIdx.x; i < K * C; i += 256) sw[i] = bf2f(w[i]);
    if (threadIdx.x < KMAX) sb[threadIdx.x] = (threadIdx.x < K && b) ? b[threadIdx.x] : 0.f;
    if (threadIdx.x < 3 * KMAX) sred[threadIdx.x] = 0.f;
    __syncthreads();
    const int n = blockIdx.y;
    float sP[KMAX], sI[KMAX], sG[KMAX];
#pragma unroll
    for (int k = 0; k < KMAX; ++k) { sP[k] = 0.f; sI[k] = 0.f; sG[k] = 0.f; }
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(Vn, v0 + v_per_block);
    for (int64_t vv = v0 + threadIdx.x; vv < v1; vv += 256) {
        const int64_t v = (int64_t)n * Vn + vv;
        float l[KMAX];
#pragma unroll
        for (int k = 0; k < KMAX; ++k) l[k] = sb[k];
        for (int c0 = 0; c0 < C; c0 += 8) {
            float f[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(z + v * zp + c0)), f);
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                if (k < K) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) l[k] = fmaf(f[j], sw[k * C + c0 + j], l[k]);
                }
            }
        }
        float mx = l[0];
        int am = 0;
#pragma unroll
        for (int k = 1; k < KMAX; ++k) if (k < K && l[k] > mx) { mx = l[k]; am = k; }
        float sum = 0.f;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) if (k < K) { l[k] = expf(l[k] - mx); sum += l[k]; }
        const float inv = 1.0f / sum;
        const int lab = labels ? labels[v] : -1;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                const float p = l[k] * inv;
                if (probs) probs[v * K + k] = p;
                sP[k] += p;
                if (k == lab) { sI[k] += p; sG[k] += 1.f; }
            }
        }
        if (amax) amax[v] = (uint8_t)am;
    }
    if (dice) {
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                float a = sP[k], bb = sI[k], c = sG[k];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    a += __shfl_xor_sync(0xffffffffu, a, o);
                    bb += __shfl_xor_sync(0xffffffffu, bb, o);
                    c += __shfl_xor_sync(0xffffffffu, c, o);
                }
                if ((threadIdx.x & 31) == 0) {
                    atomicAdd(&sred[k * 3], bb);
                    atomicAdd(&sred[k * 3 + 1], a);
                    atomicAdd(&sred[k * 3 + 2], c);
                }
            }
        }
        __syncthreads();
        if (threadIdx.x < 3 * K) atomicAdd(&dice[(int64_t)n * K * 3 + threadIdx.x], (double)sred[threadIdx.x]);
    }
}

// dice[n][k][3] = (I, P, G)  ->  loss = mean_n (1 - mean_k (2I + e)/(P + G + e))
__global__ void dice_loss_kernel(const double *__restrict__ dice, int N, int K, float *__restrict__ loss)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const double eps = 1e-5;
    double L = 0.0;
    for (int n = 0; n < N; ++n) {
        double s = 0.0;
        for (int k = 0; k < K; ++k) {
            const double *q = dice + ((int64_t)n * K + k) * 3;
            s += (2.0 * q[0] + eps) / (q[1] + q[2] + eps);
        }
        L += 1.0 - s / K;
    }
    *loss = (float)(L / N);
}

// Head backward: dl = dL/dlogits from (probs, labels, Dice sums); dz = dl * W (bf16);
// dW[k][c] += sum_v dl[v,k] z[v,c]; db[k] += sum_v dl[v,k].   dW/db must be zero on entry.
__global__ void __launch_bounds__(256)
head_bwd_kernel(const bf16 *__restrict__ z, int64_t zp, int C, const bf16 *__restrict__ w, int K,
                const float *__restrict__ probs, const uint8_t *__restrict__ labels, const double *__restrict__ dice,
                int N, bf16 *__restrict__ dz, int64_t dzp, float *__restrict__ dw, float *__restrict__ db,
                float *__restrict__ dlog, int64_t Vn, int64_t v_per_block)
{
    extern __shared__ float sm[];
    // [K*C] weights, [2*KMAX] dice coefficients, [256*KMAX] dl tile, then bf16 z tile [256][C]
    float *sw = sm, *sa = sm + K * C, *sbq = sa + KMAX, *sdl = sbq + KMAX;
    bf16 *sz = reinterpret_cast<bf16 *>(sdl + 256 * KMAX);
    const int n = blockIdx.y;
    for (int i = threadIdx.x; i < K * C; i += 256) sw[i] = bf2f(w[i]);
    if (threadIdx.x < K) {
        const double eps = 1e-5;
        const double *q = dice + ((int64_t)n * K + threadIdx.x) * 3;
        const double den = q[1] + q[2] + eps;
        sa[threadIdx.x] = (float)(2.0 / (den * N * K));
        sbq[threadIdx.x] = (float)((2.0 * q[0] + eps) / (den * den * N * K));
    }
    __syncthreads();
    const int entries = K * (C + 1);                 // (k, c) for c < C, plus (k, C) = bias
    constexpr int EPT = 5;                           // entries per thread: K*(C+1) <= 16*65 = 1040 <= 256*5
    float acc[EPT];
#pragma unroll
    for (int j = 0; j < EPT; ++j) acc[j] = 0.f;
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(Vn, v0 + v_per_block);
    for (int64_t base = v0; base < v1; base += 256) {
        const int64_t vv = base + threadIdx.x;
        const bool live = vv < v1;
        const int64_t v = (int64_t)n * Vn + vv;
        float dl[KMAX];
        if (live) {
            const int lab = labels[v];
            float p[KMAX], dp[KMAX], dotp = 0.f;
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                if (k < K) {
                    p[k] = probs[v * K + k];
                    dp[k] = -((k == lab ? sa[k] : 0.f) - sbq[k]);
                    dotp = fmaf(p[k], dp[k], dotp);
                }
            }
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                dl[k] = (k < K) ? p[k] * (dp[k] - dotp) : 0.f;
                if (k < K && dlog) dlog[v * K + k] = dl[k];
            }
            for (int c0 = 0; c0 < C; c0 += 8) {
                float f[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] = 0.f;
#pragma unroll
                for (int k = 0; k < KMAX; ++k) {
                    if (k < K) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) f[j] = fmaf(dl[k], sw[k * C + c0 + j], f[j]);
                    }
                }
                *reinterpret_cast<uint4 *>(dz + v * dzp + c0) = pack8(f);
                *reinterpret_cast<uint4 *>(sz + (size_t)threadIdx.x * C + c0) =
                    __ldg(reinterpret_cast<const uint4 *>(z + v * zp + c0));
            }
        } else {
#pragma unroll
            for (int k = 0; k < KMAX; ++k) dl[k] = 0.f;
        }
#pragma unroll
        for (int k = 0; k < KMAX; ++k) sdl[threadIdx.x * KMAX + k] = dl[k];
        __syncthreads();
        const int nv = (int)((v1 - base) < 256 ? (v1 - base) : 256);
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const int e = threadIdx.x + j * 256;
            if (e < entries) {
                const int k = e / (C + 1), c = e % (C + 1);
                float a = acc[j];
                if (c < C) for (int t = 0; t < nv; ++t) a = fmaf(sdl[t * KMAX + k], bf2f(sz[(size_t)t * C + c]), a);
                else       for (int t = 0; t < nv; ++t) a += sdl[t * KMAX + k];
                acc[j] = a;
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
        const int e = threadIdx.x + j * 256;
        if (e < entries) {
            const int k = e / (C + 1), c = e % (C + 1);
            if (c < C) atomicAdd(&dw[k * C + c], acc[j]);
            else if (db) atomicAdd(&db[k], acc[j]);
        }
    }
}

// ------------------------------------------------------------------ sliding window
__device__ __forceinline__ int patch_origin(int i, int nst, int stride, int len, int patch)
{
    // origins 0, s, 2s, ...; the last one is flush with the border
    return i < nst - 1 ? i * stride : max(len - patch, 0);
}

// patches[b] = volume[origin(first + b) : + patch]   (hard borders)
__global__ void __launch_bounds__(256)
gather_patches_kernel(const bf16 *__restrict__ vol, int64_t vp, int D, int H, int W, int C,
                      bf16 *__restrict__ out, int64_t op, int B, int PD, int PH, int PW, int first,
                      int nd, int nh, int nw, int sd, int sh, int sw)
{
    const int64_t per = (int64_t)PD * PH * PW * C;
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= per * B) return;
    const int b = (int)(e / per);
    int64_t r = e % per;
    const int c = (int)(r % C); r /= C;
    const int pw = (int)(r % PW); r /= PW;
    const int ph = (int)(r % PH);
    const int pd = (int)(r / PH);
    const int pi = first + b;
    const int iw = pi % nw, ih = (pi / nw) % nh, id = pi / (nw * nh);
    const int d = patch_origin(id, nd, sd, D, PD) + pd;
    const int h = patch_origin(ih, nh, sh, H, PH) + ph;
    const int w = patch_origin(iw, nw, sw, W, PW) + pw;
    out[((((int64_t)b * PD + pd) * PH + ph) * PW + pw) * op + c] = vol[(((int64_t)d * H + h) * W + w) * vp + c];
}

// A[k][v] = sum_p w_p(v) p_p[v][k] / sum_p w_p(v) over the patches covering v, ascending patch
// index; argmax over k (lowest index on ties).  One thread per 4 voxels along W.
// KT > 0: the class count is a compile-time constant and, where every patch origin and extent along W is a
// multiple of 4 (aligned4), the 4 voxels x KT probabilities of a patch are read as KT 16-byte vectors.
template <int VEC, int KT>
__global__ void __launch_bounds__(256)
overlap_add_kernel(const float *__restrict__ pp, int Krt, int D, int H, int W, int PD, int PH, int PW,
                   int nd, int nh, int nw, int sd, int sh, int sw, int window, int aligned4,
                   float *__restrict__ planar, uint8_t *__restrict__ amax)
{
    const int K = KT > 0 ? KT : Krt;
    extern __shared__ float tab[];          // 1-D window factors: [PD] [PH] [PW], each normalised to max 1
    float *td = tab, *th = tab + PD, *tw = th + PH;
    for (int i = threadIdx.x; i < PD + PH + PW; i += 256) {
        int P, j;
        if (i < PD) { P = PD; j = i; } else if (i < PD + PH) { P = PH; j = i - PD; } else { P = PW; j = i - PD - PH; }
        float val = 1.f;
        if (window) {
            const float sig = 0.125f * P, cen = 0.5f * (P - 1);
            const float t = (j - cen) / sig;
            const float t0 = ((P & 1) ? 0.f : 0.5f) / sig;        // offset of the sample nearest the centre
            val = expf(-0.5f * t * t) / expf(-0.5f * t0 * t0);
        }
        tab[i] = val;
    }
    __syncthreads();
    const int WV = W / VEC;
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= (int64_t)D * H * WV) return;
    const int w0 = (int)(e % WV) * VEC;
    const int h = (int)((e / WV) % H);
    const int d = (int)(e / ((int64_t)WV * H));
    const int64_t PV = (int64_t)PD * PH * PW;
    float acc[VEC][KMAX], wsum[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        wsum[i] = 0.f;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) acc[i][k] = 0.f;
    }
    for (int id = 0; id < nd; ++id) {
        const int od = patch_origin(id, nd, sd, D, PD);
        if (d < od || d >= od + PD) continue;
        for (int ih = 0; ih < nh; ++ih) {
            const int oh = patch_origin(ih, nh, sh, H, PH);
            if (h < oh || h >= oh + PH) continue;
            for (int iw = 0; iw < nw; ++iw) {
                const int ow = patch_origin(iw, nw, sw, W, PW);
                if (w0 + VEC - 1 < ow || w0 >= ow + PW) continue;
                const int64_t pi = ((int64_t)id * nh + ih) * nw + iw;
                const float wdh = td[d - od] * th[h - oh];
                if (VEC == 4 && KT > 0 && aligned4) {
                    // origins and extents are multiples of 4: the four voxels lie inside the patch together
                    float wt[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        wt[i] = wdh * tw[w0 + i - ow];
                        if (window) wt[i] = fmaxf(wt[i], 1e-3f);
                        wsum[i] += wt[i];
                    }
                    const float4 *src4 = reinterpret_cast<const float4 *>(
                        pp + (pi * PV + ((int64_t)(d - od) * PH + (h - oh)) * PW + (w0 - ow)) * KT);
#pragma unroll
                    for (int j = 0; j < (KT > 0 ? KT : 1); ++j) {
                        const float4 q = __ldg(src4 + j);
                        const float qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                        for (int e2 = 0; e2 < 4; ++e2) {
                            constexpr int KD = KT > 0 ? KT : 1;
                            const int f = 4 * j + e2;
                            acc[(f / KD) % VEC][f % KD] = fmaf(wt[(f / KD) % VEC], qq[e2], acc[(f / KD) % VEC][f % KD]);
                        }
                    }
                    continue;
                }
#pragma unroll
                for (int i = 0; i < VEC; ++i) {
                    const int w = w0 + i;
                    if (w < ow || w >= ow + PW) continue;
                    float wt = wdh * tw[w - ow];
                    if (window) wt = fmaxf(wt, 1e-3f);
                    const float *src = pp + (pi * PV + ((int64_t)(d - od) * PH + (h - oh)) * PW + (w - ow)) * K;
#pragma unroll
                    for (int k = 0; k < KMAX; ++k) if (k < K) acc[i][k] = fmaf(wt, __ldg(src + k), acc[i][k]);
                    wsum[i] += wt;
                }
            }
        }
    }
    const int64_t v0 = ((int64_t)d * H + h) * W + w0;
    const int64_t plane = (int64_t)D * H * W;
    uint8_t am[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const float inv = 1.0f / wsum[i];
        float best = -1.f;
        am[i] = 0;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                acc[i][k] *= inv;
                if (acc[i][k] > best) { best = acc[i][k]; am[i] = (uint8_t)k; }
            }
        }
    }
    if (planar) {
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                if (VEC == 4) *reinterpret_cast<float4 *>(planar + k * plane + v0) = make_float4(acc[0][k], acc[1][k], acc[2][k], acc[3][k]);
                else          planar[k * plane + v0] = acc[0][k];
            }
        }
    }
    if (amax) {
        if (VEC == 4) *reinterpret_cast<uchar4 *>(amax + v0) = make_uchar4(am[0], am[1], am[2], am[3]);
        else          amax[v0] = am[0];
    }
}

}  // namespace

lamp_status_t k_instnorm_relu_fwd(const TView &y, const double *stats, float eps, float *mu_rstd, const TView &z,
                                  cudaStream_t st)
{
    const int64_t Vn = (int64_t)y.d * y.h * y.w;
    if (Vn == 0 || y.n == 0) return LAMP_OK;
    if (y.c / 8 > 256) return LAMP_ERR_UNSUPPORTED;
    const int64_t rb = 256 / (y.c / 8);
    int64_t vpb = (Vn / (148 * 16) + rb - 1) / rb * rb;
    if (vpb < rb * 8) vpb = rb * 8;
    dim3 grid((unsigned)((Vn + vpb - 1) / vpb), y.n);
    instnorm_relu_fwd_kernel<<<grid, 256, 0, st>>>((const bf16 *)y.p, y.pitch, stats, 1.0 / (double)Vn, eps, mu_rstd,
                                                   (bf16 *)z.p, z.pitch, Vn, y.c, vpb);
    return launch_status();
}

lamp_status_t k_instnorm_relu_bwd(const TView &dza, const TView *dzb, const TView &y, const float *mu_rstd,
                                  double *sums, const TView &dy, cudaStream_t st)
{
    const int64_t Vn = (int64_t)y.d * y.h * y.w;
    const int C = y.c, G = C / 8;
    if (G > 256) return LAMP_ERR_UNSUPPORTED;
    LAMP_CUDA_OK(cudaMemsetAsync(sums, 0, (size_t)y.n * C * 2 * sizeof(double), st));
    if (Vn == 0 || y.n == 0) return LAMP_OK;
    const int RB = 256 / G;
    int64_t blocks = (148 * 8 + y.n - 1) / y.n;
    const int64_t max_blocks = (Vn + RB - 1) / RB;
    if (blocks > max_blocks) blocks = max_blocks;
    const int64_t vpb = (Vn + blocks - 1) / blocks;
    blocks = (Vn + vpb - 1) / vpb;
    const size_t smem = (size_t)RB * G * 16 * sizeof(float);
    instnorm_bwd_sums_kernel<<<dim3((unsigned)blocks, y.n), 256, smem, st>>>(
        (const bf16 *)dza.p, dza.pitch, dzb ? (const bf16 *)dzb->p : nullptr, dzb ? dzb->pitch : 0,
        (const bf16 *)y.p, y.pitch, mu_rstd, sums, Vn, C, vpb);
    int64_t vpa = (Vn / (148 * 16) + RB - 1) / RB * RB;
    if (vpa < (int64_t)RB * 8) vpa = (int64_t)RB * 8;
    dim3 grid((unsigned)((Vn + vpa - 1) / vpa), y.n);
    instnorm_bwd_apply_kernel<<<grid, 256, 0, st>>>(
        (const bf16 *)dza.p, dza.pitch, dzb ? (const bf16 *)dzb->p : nullptr, dzb ? dzb->pitch : 0,
        (const bf16 *)y.p, y.pitch, mu_rstd, sums, (bf16 *)dy.p, dy.pitch, Vn, C, vpa);
    return launch_status();
}

static void head_grid(int64_t Vn, int n, int64_t &blocks, int64_t &vpb)
{
    blocks = (148 * 8 + n - 1) / n;
    const int64_t max_blocks = (Vn + 255) / 256;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    vpb = (Vn + blocks - 1) / blocks;
    vpb = (vpb + 255) / 256 * 256;
    blocks = (Vn + vpb - 1) / vpb;
}

lamp_status_t k_head_softmax(const TView &z, const bf16 *w, const float *b, int K, float *probs, uint8_t *argmax,
                             const uint8_t *labels, double *dice_sums, cudaStream_t st)
{
    const int64_t Vn = (int64_t)z.d * z.h * z.w;
    if (K > KMAX || K < 1) return LAMP_ERR_UNSUPPORTED;
    if (dice_sums) LAMP_CUDA_OK(cudaMemsetAsync(dice_sums, 0, (size_t)z.n * K * 3 * sizeof(double), st));
    if (Vn == 0 || z.n == 0) return LAMP_OK;
    int64_t blocks, vpb;
    head_grid(Vn, z.n, blocks, vpb);
    const size_t smem = ((size_t)K * z.c + KMAX + 3 * KMAX) * sizeof(float);
    head_softmax_kernel<<<dim3((unsigned)blocks, z.n), 256, smem, st>>>(
        (const bf16 *)z.p, z.pitch, z.c, w, b, K, probs, argmax, labels, dice_sums, Vn, vpb);
    return launch_status();
}

lamp_status_t k_dice_loss(const double *dice_sums, int N, int K, float *loss, cudaStream_t st)
{
    dice_loss_kernel<<<1, 32, 0, st>>>(dice_sums, N, K, loss);
    return launch_status();
}

lamp_status_t k_head_bwd(const TView &z, const bf16 *w, int K, const float *probs, const uint8_t *labels,
                         const double *dice_sums, const TView &dz, float *dw, float *db, float *dlogits,
                         cudaStream_t st)
{
    const int64_t Vn = (int64_t)z.d * z.h * z.w;
    const int C = z.c;
    if (K > KMAX || C > 64) return LAMP_ERR_UNSUPPORTED;
    LAMP_CUDA_OK(cudaMemsetAsync(dw, 0, (size_t)K * C * sizeof(float), st));
    if (db) LAMP_CUDA_OK(cudaMemsetAsync(db, 0, (size_t)K * sizeof(float), st));
    if (Vn == 0 || z.n == 0) return LAMP_OK;
    int64_t blocks, vpb;
    head_grid(Vn, z.n, blocks, vpb);
    const size_t smem = ((size_t)K * C + 2 * KMAX + 256 * KMAX) * sizeof(float) + (size_t)256 * C * sizeof(bf16);
    static bool attr_set = false;
    if (!attr_set) {
        LAMP_CUDA_OK(cudaFuncSetAttribute(head_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
        attr_set = true;
    }
    head_bwd_kernel<<<dim3((unsigned)blocks, z.n), 256, smem, st>>>(
        (const bf16 *)z.p, z.pitch, C, w, K, probs, labels, dice_sums, z.n, (bf16 *)dz.p, dz.pitch, dw, db,
        dlogits, Vn, vpb);
    return launch_status();
}

lamp_status_t k_gather_patches(const TView &vol, const TView &patches, int first_patch, const int32_t nst[3],
                               const int32_t stride[3], cudaStream_t st)
{
    const int64_t total = (int64_t)patches.n * patches.d * patches.h * patches.w * patches.c;
    if (total == 0) return LAMP_OK;
    gather_patches_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
        (const bf16 *)vol.p, vol.pitch, vol.d, vol.h, vol.w, vol.c, (bf16 *)patches.p, patches.pitch, patches.n,
        patches.d, patches.h, patches.w, first_patch, nst[0], nst[1], nst[2], stride[0], stride[1], stride[2]);
    return launch_status();
}

lamp_status_t k_overlap_add(const float *pp, int K, int D, int H, int W, const int32_t patch[3],
                            const int32_t nst[3], const int32_t stride[3], int window, float *planar,
                            uint8_t *argmax, cudaStream_t st)
{
    if (K > KMAX || K < 1) return LAMP_ERR_UNSUPPORTED;
    if ((int64_t)D * H * W == 0) return LAMP_OK;
    const size_t smem = (size_t)(patch[0] + patch[1] + patch[2]) * sizeof(float);
    const bool vec = (W % 4 == 0) && ((uintptr_t)planar % 16 == 0) && ((uintptr_t)argmax % 4 == 0);
    const int aligned4 = vec && patch[2] % 4 == 0 && (nst[2] == 1 || stride[2] % 4 == 0) && (W - patch[2]) % 4 == 0 &&
                         ((uintptr_t)pp % 16 == 0);
#define LAMP_OA(VECN, KTN)                                                                                              \
    overlap_add_kernel<VECN, KTN><<<(unsigned)((total + 255) / 256), 256, smem, st>>>(                                \
        pp, K, D, H, W, patch[0], patch[1], patch[2], nst[0], nst[1], nst[2], stride[0], stride[1], stride[2], window, \
        aligned4, planar, argmax)
    if (vec) {
        const int64_t total = (int64_t)D * H * (W / 4);
        switch (aligned4 ? K : 0) {
        case 2:  LAMP_OA(4, 2); break;
        case 3:  LAMP_OA(4, 3); break;
        case 4:  LAMP_OA(4, 4); break;
        case 5:  LAMP_OA(4, 5); break;
        case 8:  LAMP_OA(4, 8); break;
        case 10: LAMP_OA(4, 10); break;
        case 16: LAMP_OA(4, 16); break;
        default: LAMP_OA(4, 0); break;
        }
    } else {
        const int64_t total = (int64_t)D * H * W;
        LAMP_OA(1, 0);
    }
#undef LAMP_OA
    return launch_status();
}

}  // namespace lamp
