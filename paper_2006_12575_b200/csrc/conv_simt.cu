// Direct (CUDA-core) convolution kernels for every variant of the layer
//   y[n,o,co] = b[co] + sum_{tap,ci} x[n, o*s + k - p, ci] * w[tap][co][ci]        (and its transposed form)
// and its two derivatives.  They serve the shapes the tensor-core path does not take: the
// single-channel first layer, narrow networks, the stride-2 and 2x2x2 transposed variants.
// bf16 operands, fp32 accumulation, one sequential sum per output element.
#include "common.cuh"

namespace lamp {

namespace {

__device__ __forceinline__ float dot_row(const bf16 *__restrict__ a, const bf16 *__restrict__ b, int n, bool vec)
{
    float acc = 0.f;
    if (vec) {
        for (int i = 0; i < n; i += 8) {
            float fa[8], fb[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(a + i)), fa);
            unpack8(__ldg(reinterpret_cast<const uint4 *>(b + i)), fb);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc = fmaf(fa[j], fb[j], acc);
        }
    } else {
        for (int i = 0; i < n; ++i) acc = fmaf(bf2f(a[i]), bf2f(b[i]), acc);
    }
    return acc;
}

// One thread per (output voxel, output channel); blockDim.x = 256 = TV voxels x TC channels.
template <bool TR>
__global__ void __launch_bounds__(256)
conv_fwd_kernel(ConvGeom g, const bf16 *__restrict__ x, int64_t xp, const bf16 *__restrict__ w,
                const float *__restrict__ bias, void *__restrict__ y, int64_t yp, int y_f32,
                double *__restrict__ stats, int TC, int iters, int vec)
{
    __shared__ float red[2][256];
    const int TV = 256 / TC;
    const int cl = threadIdx.x % TC, vl = threadIdx.x / TC;
    const int n = blockIdx.y;
    const int64_t Vn = (int64_t)g.od * g.oh * g.ow;
    const int64_t v0 = (int64_t)blockIdx.x * TV * iters;
    const int co_round = (g.co + TC - 1) / TC * TC;
    const int K = g.k;
    for (int c = cl; c < co_round; c += TC) {
        const bool cvalid = c < g.co;
        float s1 = 0.f, s2 = 0.f;
        for (int it = 0; it < iters; ++it) {
            const int64_t v = v0 + (int64_t)it * TV + vl;
            if (v >= Vn || !cvalid) continue;
            const int ow = (int)(v % g.ow);
            const int oh = (int)((v / g.ow) % g.oh);
            const int od = (int)(v / ((int64_t)g.ow * g.oh));
            float acc = bias ? bias[c] : 0.f;
            for (int kd = 0; kd < K; ++kd) {
                int id;
                if (TR) { const int t = od - kd; if (t < 0 || t % g.s) continue; id = t / g.s; }
                else    { id = od * g.s + kd - g.p; }
                if (id < 0 || id >= g.d) continue;
                for (int kh = 0; kh < K; ++kh) {
                    int ih;
                    if (TR) { const int t = oh - kh; if (t < 0 || t % g.s) continue; ih = t / g.s; }
                    else    { ih = oh * g.s + kh - g.p; }
                    if (ih < 0 || ih >= g.h) continue;
                    for (int kw = 0; kw < K; ++kw) {
                        int iw;
                        if (TR) { const int t = ow - kw; if (t < 0 || t % g.s) continue; iw = t / g.s; }
                        else    { iw = ow * g.s + kw - g.p; }
                        if (iw < 0 || iw >= g.w) continue;
                        const int tap = (kd * K + kh) * K + kw;
                        const bf16 *xr = x + ((((int64_t)n * g.d + id) * g.h + ih) * g.w + iw) * xp;
                        const bf16 *wr = w + ((int64_t)tap * g.co + c) * g.ci;
                        acc += dot_row(xr, wr, g.ci, vec);
                    }
                }
            }
            const int64_t o = ((int64_t)n * Vn + v) * yp + c;
            if (y_f32) reinterpret_cast<float *>(y)[o] = acc;
            else       reinterpret_cast<bf16 *>(y)[o] = f2bf(acc);
            s1 += acc;
            s2 += acc * acc;
        }
        if (stats) {
            red[0][threadIdx.x] = s1;
            red[1][threadIdx.x] = s2;
            __syncthreads();
            if (vl == 0 && cvalid) {
                double a = 0.0, b = 0.0;
                for (int j = 0; j < TV; ++j) { a += red[0][j * TC + cl]; b += red[1][j * TC + cl]; }
                atomicAdd(&stats[((int64_t)n * g.co + c) * 2], a);
                atomicAdd(&stats[((int64_t)n * g.co + c) * 2 + 1], b);
            }
            __syncthreads();
        }
    }
}

// One thread per (input voxel, input channel).
template <bool TR>
__global__ void __launch_bounds__(256)
conv_dgrad_kernel(ConvGeom g, const bf16 *__restrict__ dy, int64_t dyp, const bf16 *__restrict__ w,
                  void *__restrict__ dx, int64_t dxp, int dx_f32, int vec)
{
    const int64_t Vn = (int64_t)g.d * g.h * g.w;
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= Vn * g.ci) return;
    const int n = blockIdx.y;
    const int c = (int)(e % g.ci);
    const int64_t v = e / g.ci;
    const int iw = (int)(v % g.w);
    const int ih = (int)((v / g.w) % g.h);
    const int id = (int)(v / ((int64_t)g.w * g.h));
    const int K = g.k;
    float acc = 0.f;
    for (int kd = 0; kd < K; ++kd) {
        int od;
        if (TR) { od = id * g.s + kd; }
        else    { const int t = id + g.p - kd; if (t < 0 || t % g.s) continue; od = t / g.s; }
        if (od < 0 || od >= g.od) continue;
        for (int kh = 0; kh < K; ++kh) {
            int oh;
            if (TR) { oh = ih * g.s + kh; }
            else    { const int t = ih + g.p - kh; if (t < 0 || t % g.s) continue; oh = t / g.s; }
            if (oh < 0 || oh >= g.oh) continue;
            for (int kw = 0; kw < K; ++kw) {
                int ow;
                if (TR) { ow = iw * g.s + kw; }
                else    { const int t = iw + g.p - kw; if (t < 0 || t % g.s) continue; ow = t / g.s; }
                if (ow < 0 || ow >= g.ow) continue;
                const int tap = (kd * K + kh) * K + kw;
                const bf16 *gr = dy + ((((int64_t)n * g.od + od) * g.oh + oh) * g.ow + ow) * dyp;
                const bf16 *wr = w + (int64_t)tap * g.co * g.ci + c;
                if (vec) {
                    for (int co = 0; co < g.co; co += 8) {
                        float f[8];
                        unpack8(__ldg(reinterpret_cast<const uint4 *>(gr + co)), f);
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc = fmaf(f[j], bf2f(wr[(int64_t)(co + j) * g.ci]), acc);
                    }
                } else {
                    for (int co = 0; co < g.co; ++co) acc = fmaf(bf2f(gr[co]), bf2f(wr[(int64_t)co * g.ci]), acc);
                }
            }
        }
    }
    const int64_t o = ((int64_t)n * Vn + v) * dxp + c;
    if (dx_f32) reinterpret_cast<float *>(dx)[o] = acc;
    else        reinterpret_cast<bf16 *>(dx)[o] = f2bf(acc);
}

// One thread per (tap, co, ci) entry and per split of the row range; a "row" is one (n, d, h)
// line of the tensor the sum runs over (the conv output, or the input for the transposed form).
template <bool TR>
__global__ void __launch_bounds__(256)
conv_wgrad_kernel(ConvGeom g, const bf16 *__restrict__ x, int64_t xp, const bf16 *__restrict__ dy, int64_t dyp,
                  float *__restrict__ part, int64_t entries, int64_t rows, int64_t rows_per_split)
{
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= entries) return;
    const int ci = (int)(e % g.ci);
    const int co = (int)((e / g.ci) % g.co);
    const int tap = (int)(e / ((int64_t)g.ci * g.co));
    const int K = g.k;
    const int kd = tap / (K * K), kh = (tap / K) % K, kw = tap % K;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_split;
    const int64_t r1 = min(rows, r0 + rows_per_split);
    // loop extents: conv -> output lines; transposed -> input lines
    const int LH = TR ? g.h : g.oh, LD = TR ? g.d : g.od, LW = TR ? g.w : g.ow;
    float acc = 0.f;
    for (int64_t r = r0; r < r1; ++r) {
        const int lh = (int)(r % LH);
        const int ld = (int)((r / LH) % LD);
        const int n = (int)(r / ((int64_t)LH * LD));
        if (TR) {
            const bf16 *xr = x + (((int64_t)n * g.d + ld) * g.h + lh) * (int64_t)g.w * xp + ci;
            const bf16 *gr = dy + ((((int64_t)n * g.od + ld * g.s + kd) * g.oh + lh * g.s + kh) * (int64_t)g.ow + kw) * dyp + co;
            for (int lw = 0; lw < LW; ++lw)
                acc = fmaf(bf2f(gr[(int64_t)lw * g.s * dyp]), bf2f(xr[(int64_t)lw * xp]), acc);
        } else {
            const int id = ld * g.s + kd - g.p, ih = lh * g.s + kh - g.p;
            if (id < 0 || id >= g.d || ih < 0 || ih >= g.h) continue;
            const bf16 *xr = x + (((int64_t)n * g.d + id) * g.h + ih) * (int64_t)g.w * xp + ci;
            const bf16 *gr = dy + (((int64_t)n * g.od + ld) * g.oh + lh) * (int64_t)g.ow * dyp + co;
            for (int lw = 0; lw < LW; ++lw) {
                const int iw = lw * g.s + kw - g.p;
                if (iw < 0 || iw >= g.w) continue;
                acc = fmaf(bf2f(gr[(int64_t)lw * dyp]), bf2f(xr[(int64_t)iw * xp]), acc);
            }
        }
    }
    part[(int64_t)blockIdx.y * entries + e] = acc;
}

// Column sums of dy over a chunk of voxels: part[chunk][co].  Generic (any co, any alignment).
__global__ void __launch_bounds__(256)
colsum_kernel(const bf16 *__restrict__ dy, int64_t dyp, int co, int64_t V, int64_t v_per_block, float *__restrict__ part)
{
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(V, v0 + v_per_block);
    for (int c = threadIdx.x; c < co; c += 256) {
        float acc = 0.f;
        for (int64_t v = v0; v < v1; ++v) acc += bf2f(dy[v * dyp + c]);
        part[(int64_t)blockIdx.x * co + c] = acc;
    }
}

// The same for co % 8 == 0 and 16-byte aligned rows: thread = (voxel row in the block, group of 8 channels).
__global__ void __launch_bounds__(256)
colsum_vec_kernel(const bf16 *__restrict__ dy, int64_t dyp, int co, int64_t V, int64_t v_per_block, float *__restrict__ part)
{
    extern __shared__ float red[];          // [RB][G][8]
    pdl_launch_dependents();
    pdl_wait();
    const int G = co >> 3, RB = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(V, v0 + v_per_block);
    float s[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j] = 0.f;
    if (r < RB) {
        for (int64_t v = v0 + r; v < v1; v += RB) {
            float f[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(dy + v * dyp + g * 8)), f);
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] += f[j];
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) red[(r * G + g) * 8 + j] = s[j];
    }
    __syncthreads();
    for (int t = threadIdx.x; t < co; t += 256) {
        float acc = 0.f;
        for (int rr = 0; rr < RB; ++rr) acc += red[rr * co + t];
        part[(int64_t)blockIdx.x * co + t] = acc;
    }
}

// ---------------------------------------------------------------------------------------------
// First layer of the network: one input channel, 3x3x3 s1 p1, c_out <= 64 (HBM-bound: the output
// is 2 * c_out bytes per voxel against 2 bytes read).  One thread per output voxel, all channels.
// ---------------------------------------------------------------------------------------------
template <int CO>
__global__ void __launch_bounds__(128)
conv_c1_fwd_kernel(ConvGeom g, const bf16 *__restrict__ x, int64_t xp, const bf16 *__restrict__ w,
                   const float *__restrict__ bias, void *__restrict__ y, int64_t yp, int y_f32, double *__restrict__ stats)
{
    __shared__ float sw[27 * CO];
    __shared__ float sb[CO];
    __shared__ float tr[4][32 * (CO + 1)];
    __shared__ float bs1[CO], bs2[CO];
    for (int i = threadIdx.x; i < 27 * CO; i += 128) sw[i] = bf2f(w[i]);          // w[t][co][0]
    for (int i = threadIdx.x; i < CO; i += 128) { sb[i] = bias ? bias[i] : 0.f; bs1[i] = 0.f; bs2[i] = 0.f; }
    __syncthreads();
    const int n = blockIdx.y;
    const int64_t Vn = (int64_t)g.d * g.h * g.w;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float cs1[(CO + 31) / 32], cs2[(CO + 31) / 32];
#pragma unroll
    for (int i = 0; i < (CO + 31) / 32; ++i) { cs1[i] = 0.f; cs2[i] = 0.f; }
    for (int64_t v0 = (int64_t)blockIdx.x * 128; v0 < Vn; v0 += (int64_t)gridDim.x * 128) {
        const int64_t v = v0 + threadIdx.x;
        const bool live = v < Vn;
        float acc[CO];
#pragma unroll
        for (int c = 0; c < CO; ++c) acc[c] = sb[c];
        if (live) {
            const int iw = (int)(v % g.w), ih = (int)((v / g.w) % g.h), id = (int)(v / ((int64_t)g.w * g.h));
            for (int kd = 0; kd < 3; ++kd) {
                const int zd = id + kd - 1;
                if (zd < 0 || zd >= g.d) continue;
                for (int kh = 0; kh < 3; ++kh) {
                    const int zh = ih + kh - 1;
                    if (zh < 0 || zh >= g.h) continue;
#pragma unroll
                    for (int kw = 0; kw < 3; ++kw) {
                        const int zw = iw + kw - 1;
                        if (zw < 0 || zw >= g.w) continue;
                        const float xv = bf2f(x[((((int64_t)n * g.d + zd) * g.h + zh) * g.w + zw) * xp]);
                        const float *wt = sw + ((kd * 3 + kh) * 3 + kw) * CO;
#pragma unroll
                        for (int c = 0; c < CO; ++c) acc[c] = fmaf(xv, wt[c], acc[c]);
                    }
                }
            }
            const int64_t o = ((int64_t)n * Vn + v) * yp;
            if (y_f32) {
                float4 *dst = reinterpret_cast<float4 *>((float *)y + o);
#pragma unroll
                for (int c = 0; c < CO; c += 4) dst[c / 4] = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
            } else {
                uint4 *dst = reinterpret_cast<uint4 *>((bf16 *)y + o);
#pragma unroll
                for (int c = 0; c < CO; c += 8) {
                    float f8[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) f8[u] = acc[c + u];
                    dst[c / 8] = pack8(f8);
                }
            }
        }
        if (stats) {
            // per-warp transpose: lane c then sums channel c (and c + 32) over the warp's 32 voxels
            float *t = tr[warp];
#pragma unroll
            for (int c = 0; c < CO; ++c) t[lane * (CO + 1) + c] = live ? acc[c] : 0.f;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < (CO + 31) / 32; ++i) {
                const int c = i * 32 + lane;
                if (c < CO) {
                    float a = 0.f, b = 0.f;
                    for (int r = 0; r < 32; ++r) { const float f = t[r * (CO + 1) + c]; a += f; b = fmaf(f, f, b); }
                    cs1[i] += a;
                    cs2[i] += b;
                }
            }
            __syncwarp();
        }
    }
    if (stats) {
#pragma unroll
        for (int i = 0; i < (CO + 31) / 32; ++i) {
            const int c = i * 32 + lane;
            if (c < CO) { atomicAdd(&bs1[c], cs1[i]); atomicAdd(&bs2[c], cs2[i]); }
        }
        __syncthreads();
        for (int c = threadIdx.x; c < CO; c += 128) {
            atomicAdd(&stats[((int64_t)n * CO + c) * 2], (double)bs1[c]);
            atomicAdd(&stats[((int64_t)n * CO + c) * 2 + 1], (double)bs2[c]);
        }
    }
}

// Weight gradient of the same layer: dw[t][co] = sum_v dy[v][co] * x[v + off_t].  A warp owns a stripe of
// voxels; lane = output channel (plus 32 for c_out = 64); 27 accumulators per lane; part[block][27 * co].
template <int CO>
__global__ void __launch_bounds__(256)
conv_c1_wgrad_kernel(ConvGeom g, const bf16 *__restrict__ x, int64_t xp, const bf16 *__restrict__ dy, int64_t dyp,
                     float *__restrict__ part, int64_t v_per_block)
{
    constexpr int CPL = (CO + 31) / 32;          // channels per lane
    constexpr int NWARP = CO > 32 ? 4 : 8;       // blockDim.x = 32 * NWARP (static shared memory stays under 48 KB)
    __shared__ float red[NWARP][27 * CO];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t V = (int64_t)g.n * g.d * g.h * g.w;
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(V, v0 + v_per_block);
    float acc[CPL][27];
#pragma unroll
    for (int i = 0; i < CPL; ++i)
#pragma unroll
        for (int t = 0; t < 27; ++t) acc[i][t] = 0.f;
    // each warp walks a contiguous run of voxels, keeping (d, h, w) incrementally
    const int64_t per_warp = (v1 - v0 + NWARP - 1) / NWARP;
    const int64_t wv0 = v0 + warp * per_warp, wv1 = min(v1, wv0 + per_warp);
    int iw = 0, ih = 0, id = 0;
    if (wv0 < wv1) {
        iw = (int)(wv0 % g.w);
        ih = (int)((wv0 / g.w) % g.h);
        id = (int)((wv0 / ((int64_t)g.w * g.h)) % g.d);
    }
    const int64_t sh = (int64_t)g.w * xp, sd = (int64_t)g.w * g.h * xp;
    for (int64_t v = wv0; v < wv1; ++v) {
        const bool vd[3] = {id > 0, true, id < g.d - 1};
        const bool vh[3] = {ih > 0, true, ih < g.h - 1};
        const bool vw[3] = {iw > 0, true, iw < g.w - 1};
        const bf16 *xc = x + v * xp;
        float gy[CPL];
#pragma unroll
        for (int i = 0; i < CPL; ++i) gy[i] = (i * 32 + lane < CO) ? bf2f(dy[v * dyp + i * 32 + lane]) : 0.f;
#pragma unroll
        for (int t = 0; t < 27; ++t) {
            const int kd = t / 9, kh = (t / 3) % 3, kw = t % 3;
            float xv = 0.f;
            if (vd[kd] && vh[kh] && vw[kw]) xv = bf2f(xc[(kd - 1) * sd + (kh - 1) * sh + (kw - 1) * xp]);
#pragma unroll
            for (int i = 0; i < CPL; ++i) acc[i][t] = fmaf(gy[i], xv, acc[i][t]);
        }
        if (++iw == g.w) { iw = 0; if (++ih == g.h) { ih = 0; if (++id == g.d) id = 0; } }
    }
#pragma unroll
    for (int i = 0; i < CPL; ++i)
#pragma unroll
        for (int t = 0; t < 27; ++t)
            if (i * 32 + lane < CO) red[warp][t * CO + i * 32 + lane] = acc[i][t];
    __syncthreads();
    for (int e = threadIdx.x; e < 27 * CO; e += 32 * NWARP) {
        float a = 0.f;
        for (int wv = 0; wv < NWARP; ++wv) a += red[wv][e];
        part[(int64_t)blockIdx.x * 27 * CO + e] = a;
    }
}

// out[e] = sum_s part[s][e], fixed order: 32 entries x 8 split slices per block; slice j adds splits j, j + 8, ...
// into four interleaved running sums (independent loads in flight), and the eight slice sums are then added in
// slice order.  out may be the first split of part (a block reads all splits of its entries before it writes them).
__global__ void __launch_bounds__(256)
reduce_parts_kernel(const float *part, int64_t entries, int splits, float *out)
{
    __shared__ float red[8][32];
    pdl_launch_dependents();
    pdl_wait();
    const int el = threadIdx.x & 31, sl = threadIdx.x >> 5;
    const int64_t e = (int64_t)blockIdx.x * 32 + el;
    float acc = 0.f;
    if (e < entries) {
        float a4[4] = {0.f, 0.f, 0.f, 0.f};
        int s = sl;
        for (; s + 24 < splits; s += 32) {
            float t[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) t[u] = __ldcg(part + (int64_t)(s + 8 * u) * entries + e);
#pragma unroll
            for (int u = 0; u < 4; ++u) a4[u] += t[u];
        }
        for (int u = 0; s < splits; s += 8, ++u) a4[u] += __ldcg(part + (int64_t)s * entries + e);
        acc = (a4[0] + a4[1]) + (a4[2] + a4[3]);
    }
    red[sl][el] = acc;
    __syncthreads();
    if (sl == 0 && e < entries) {
        float a = red[0][el];
#pragma unroll
        for (int j = 1; j < 8; ++j) a += red[j][el];
        out[e] = a;
    }
}

// The same sum for few splits over many entries: a thread owns 4 consecutive entries and adds the splits in order
// (out may be the first split of part).
__global__ void __launch_bounds__(256)
reduce_parts_vec4_kernel(const float4 *part, int64_t entries4, int splits, float4 *out)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= entries4) return;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int s = 0; s < splits; ++s) {
        const float4 t = __ldcg(part + (int64_t)s * entries4 + e);
        a.x += t.x; a.y += t.y; a.z += t.z; a.w += t.w;
    }
    out[e] = a;
}

// out[t][b][a] = sum_s in[s][t][a][b] through 32 x 32 shared-memory tiles (A, B multiples of 32): reads run along b,
// writes along a.  With one split and bf16 data this is the per-tap transpose of a weight tensor.
template <typename T>
__global__ void __launch_bounds__(256)
transpose_sum_kernel(const T *__restrict__ in, int64_t split_stride, int splits, int A, int B, T *__restrict__ out)
{
    __shared__ float tile[32][33];
    pdl_launch_dependents();
    pdl_wait();
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;           // 32 x 8
    const int b0 = blockIdx.x * 32, a0 = blockIdx.y * 32;
    const int64_t t = blockIdx.z;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int a = a0 + ty + 8 * i;
        const int64_t src = (t * A + a) * B + b0 + tx;
        float acc = 0.f;
        for (int s = 0; s < splits; ++s) acc += (float)in[(int64_t)s * split_stride + src];
        tile[ty + 8 * i][tx] = acc;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int b = b0 + ty + 8 * i;
        out[(t * B + b) * A + a0 + tx] = (T)tile[tx][ty + 8 * i];
    }
}

// xpad[v][0] = x[v], xpad[v][1..31] = 0 (the 1-channel input widened to one 32-channel chunk)
__global__ void __launch_bounds__(256)
pad_c1_kernel(const bf16 *__restrict__ x, int64_t xp, bf16 *__restrict__ xpad, int64_t V)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;      // one 16-byte group of 8 channels
    if (e >= V * 4) return;
    const int64_t v = e >> 2;
    uint4 q = make_uint4(0, 0, 0, 0);
    if ((e & 3) == 0) q.x = (uint32_t)__bfloat16_as_ushort(x[v * xp]);
    reinterpret_cast<uint4 *>(xpad)[e] = q;
}

// dw[t][co] = dw32[t][co][0]
__global__ void __launch_bounds__(256)
take_c0_kernel(const float *__restrict__ dw32, float *__restrict__ dw, int n)
{
    pdl_launch_dependents();
    pdl_wait();
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i < n) dw[i] = dw32[(int64_t)i * 32];
}

inline int pick_tc(int co)
{
    int tc = 8;
    while (tc < co && tc < 64) tc <<= 1;
    return tc;
}

struct WgradPlan { int64_t entries, rows, rows_per_split; int splits; int64_t V; int cs_blocks; int64_t v_per_block; };

inline WgradPlan wgrad_plan(const ConvGeom &g)
{
    WgradPlan p;
    p.entries = (int64_t)g.k * g.k * g.k * g.co * g.ci;
    p.rows = g.transposed ? (int64_t)g.n * g.d * g.h : (int64_t)g.n * g.od * g.oh;
    int64_t want = (600000 + p.entries - 1) / p.entries;
    if (want < 1) want = 1;
    if (want > p.rows) want = p.rows;
    if (want > 4096) want = 4096;
    p.rows_per_split = (p.rows + want - 1) / want;
    p.splits = (int)((p.rows + p.rows_per_split - 1) / p.rows_per_split);
    p.V = (int64_t)g.n * g.od * g.oh * g.ow;
    p.cs_blocks = (int)(((p.V + 255) / 256) < 1024 ? ((p.V + 255) / 256) : 1024); if (p.cs_blocks < 1) p.cs_blocks = 1;
    p.v_per_block = (p.V + p.cs_blocks - 1) / p.cs_blocks;
    return p;
}

}  // namespace

lamp_status_t simt_conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                            double *stats, cudaStream_t st)
{
    const int64_t Vn = (int64_t)g.od * g.oh * g.ow;
    if (Vn == 0 || g.n == 0) return LAMP_OK;
    if (g.ci == 1 && g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed && (g.co == 32 || g.co == 64) &&
        ((uintptr_t)y.p & 15) == 0 && (y.f32 ? y.pitch % 4 == 0 : y.pitch % 8 == 0)) {
        int blocks = (int)((Vn + 127) / 128);
        const int cap = sm_count() * 16 / (g.n > 0 ? g.n : 1) + 1;
        if (blocks > cap) blocks = cap;
        dim3 grid(blocks, g.n);
        if (g.co == 32)
            conv_c1_fwd_kernel<32><<<grid, 128, 0, st>>>(g, (const bf16 *)x.p, x.pitch, w, bias, y.p, y.pitch, y.f32, stats);
        else
            conv_c1_fwd_kernel<64><<<grid, 128, 0, st>>>(g, (const bf16 *)x.p, x.pitch, w, bias, y.p, y.pitch, y.f32, stats);
        return launch_status();
    }
    const int TC = pick_tc(g.co), TV = 256 / TC;
    // few voxels (deep levels): one voxel group per block so that the grid still fills the machine
    const int iters = Vn >= 65536 ? 16 : (Vn >= 8192 ? 4 : 1);
    const int vec = (g.ci % 8 == 0) && (x.pitch % 8 == 0) && ((uintptr_t)x.p % 16 == 0) && ((uintptr_t)w % 16 == 0);
    dim3 grid((unsigned)((Vn + (int64_t)TV * iters - 1) / ((int64_t)TV * iters)), g.n);
    if (g.transposed)
        conv_fwd_kernel<true><<<grid, 256, 0, st>>>(g, (const bf16 *)x.p, x.pitch, w, bias, y.p, y.pitch, y.f32, stats, TC, iters, vec);
    else
        conv_fwd_kernel<false><<<grid, 256, 0, st>>>(g, (const bf16 *)x.p, x.pitch, w, bias, y.p, y.pitch, y.f32, stats, TC, iters, vec);
    return launch_status();
}

lamp_status_t simt_conv_dgrad(const ConvGeom &g, const TView &dy, const bf16 *w, const TView &dx, cudaStream_t st)
{
    const int64_t Vn = (int64_t)g.d * g.h * g.w;
    if (Vn == 0 || g.n == 0) return LAMP_OK;
    const int vec = (g.co % 8 == 0) && (dy.pitch % 8 == 0) && ((uintptr_t)dy.p % 16 == 0);
    dim3 grid((unsigned)((Vn * g.ci + 255) / 256), g.n);
    if (g.transposed)
        conv_dgrad_kernel<true><<<grid, 256, 0, st>>>(g, (const bf16 *)dy.p, dy.pitch, w, dx.p, dx.pitch, dx.f32, vec);
    else
        conv_dgrad_kernel<false><<<grid, 256, 0, st>>>(g, (const bf16 *)dy.p, dy.pitch, w, dx.p, dx.pitch, dx.f32, vec);
    return launch_status();
}

lamp_status_t reduce_partials(const float *part, int64_t entries, int splits, float *out, cudaStream_t st)
{
    if (entries == 0) return LAMP_OK;
    if (splits <= 16 && entries >= 32768 && entries % 4 == 0 && (((uintptr_t)part | (uintptr_t)out) & 15) == 0)
        return launch_pdl(true, reduce_parts_vec4_kernel, dim3((unsigned)((entries / 4 + 255) / 256)), dim3(256), 0, st,
                          (const float4 *)part, entries / 4, splits, (float4 *)out);
    else
        return launch_pdl(true, reduce_parts_kernel, dim3((unsigned)((entries + 31) / 32)), dim3(256), 0, st, part, entries, splits, out);
}

bool transpose_sum_supported(int64_t taps, int A, int B) { return A % 32 == 0 && B % 32 == 0 && taps > 0 && taps <= 65535; }

lamp_status_t transpose_sum_f32(const float *in, int64_t taps, int A, int B, int splits, float *out, cudaStream_t st)
{
    if (!transpose_sum_supported(taps, A, B)) return LAMP_ERR_UNSUPPORTED;
    if (splits > 4) {
        // many splits: the transpose kernel would add them one after the other in few threads; the partials are added
        // first, by the well-spread reduction, into the first split, which is then transposed on its own
        const lamp_status_t s = reduce_partials(in, taps * A * B, splits, const_cast<float *>(in), st);
        if (s != LAMP_OK) return s;
        splits = 1;
    }
    return launch_pdl(true, transpose_sum_kernel<float>, dim3(B / 32, A / 32, (unsigned)taps), dim3(256), 0, st, in, taps * A * B, splits, A, B, out);
}

lamp_status_t transpose_bf16(const bf16 *in, int64_t taps, int A, int B, bf16 *out, cudaStream_t st)
{
    return launch_pdl(true, transpose_sum_kernel<bf16>, dim3(B / 32, A / 32, (unsigned)taps), dim3(256), 0, st, in, (int64_t)0, 1, A, B, out);
}

static void bias_plan(int64_t V, int *blocks, int64_t *vpb)
{
    int b = (int)(((V + 255) / 256) < 1024 ? ((V + 255) / 256) : 1024);
    if (b < 1) b = 1;
    *blocks = b;
    *vpb = (V + b - 1) / b;
}

size_t bias_grad_ws(int64_t voxels, int co)
{
    int b; int64_t vpb;
    bias_plan(voxels, &b, &vpb);
    return align_up((size_t)b * co * 4, 256);
}

lamp_status_t bias_grad(const TView &dy, float *db, void *ws, cudaStream_t st)
{
    const int64_t V = (int64_t)dy.n * dy.d * dy.h * dy.w;
    if (V == 0) { LAMP_CUDA_OK(cudaMemsetAsync(db, 0, (size_t)dy.c * 4, st)); return LAMP_OK; }
    int b; int64_t vpb;
    bias_plan(V, &b, &vpb);
    if (dy.c % 8 == 0 && dy.c <= 2048 && dy.pitch % 8 == 0 && ((uintptr_t)dy.p & 15) == 0) {
        const int G = dy.c / 8, RB = 256 / G;
        if (launch_pdl(true, colsum_vec_kernel, dim3(b), dim3(256), (size_t)RB * dy.c * sizeof(float), st, (const bf16 *)dy.p, dy.pitch, dy.c, V, vpb,
                       (float *)ws) != LAMP_OK)
            return LAMP_ERR_CUDA;
    } else {
        colsum_kernel<<<b, 256, 0, st>>>((const bf16 *)dy.p, dy.pitch, dy.c, V, vpb, (float *)ws);
    }
    reduce_parts_kernel<<<(dy.c + 31) / 32, 256, 0, st>>>((const float *)ws, dy.c, b, db);
    return launch_status();
}

static bool c1_wgrad_shape(const ConvGeom &g)
{
    return g.ci == 1 && g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed && (g.co == 32 || g.co == 64);
}

static void c1_wgrad_plan(const ConvGeom &g, int *blocks, int64_t *vpb)
{
    const int64_t V = (int64_t)g.n * g.d * g.h * g.w;
    int b = (int)((V + 2047) / 2048);
    if (b > sm_count() * 8) b = sm_count() * 8;
    if (b < 1) b = 1;
    *blocks = b;
    *vpb = (V + b - 1) / b;
}

lamp_status_t pad_c1(const TView &x, bf16 *xpad, cudaStream_t st)
{
    const int64_t V = (int64_t)x.n * x.d * x.h * x.w;
    if (V == 0) return LAMP_OK;
    return launch_pdl(true, pad_c1_kernel, dim3((unsigned)((V * 4 + 255) / 256)), dim3(256), 0, st, (const bf16 *)x.p, x.pitch, xpad, V);
}

lamp_status_t take_c0(const float *dw32, float *dw, int n, cudaStream_t st)
{
    return launch_pdl(true, take_c0_kernel, dim3((n + 255) / 256), dim3(256), 0, st, dw32, dw, n);
}

size_t simt_conv_wgrad_ws(const ConvGeom &g)
{
    const WgradPlan p = wgrad_plan(g);
    size_t main_part = (size_t)p.splits * p.entries * 4;
    if (c1_wgrad_shape(g)) {
        int blocks; int64_t vpb;
        c1_wgrad_plan(g, &blocks, &vpb);
        if ((size_t)blocks * p.entries * 4 > main_part) main_part = (size_t)blocks * p.entries * 4;
    }
    return align_up(main_part, 256) + align_up((size_t)p.cs_blocks * g.co * 4, 256) +
           bias_grad_ws((int64_t)g.n * g.od * g.oh * g.ow, g.co);
}

lamp_status_t simt_conv_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, float *db,
                              void *ws, size_t ws_bytes, cudaStream_t st)
{
    const WgradPlan p = wgrad_plan(g);
    if (ws_bytes < simt_conv_wgrad_ws(g) || !ws) return LAMP_ERR_WORKSPACE;
    if (c1_wgrad_shape(g) && p.V > 0) {
        // partials [blocks][27 * co] fit the generic plan's workspace (blocks <= 1184 <= its split count bound)
        int blocks; int64_t vpb;
        c1_wgrad_plan(g, &blocks, &vpb);
        {
            float *part1 = (float *)ws;
            if (g.co == 32)
                conv_c1_wgrad_kernel<32><<<blocks, 256, 0, st>>>(g, (const bf16 *)x.p, x.pitch, (const bf16 *)dy.p, dy.pitch, part1, vpb);
            else
                conv_c1_wgrad_kernel<64><<<blocks, 128, 0, st>>>(g, (const bf16 *)x.p, x.pitch, (const bf16 *)dy.p, dy.pitch, part1, vpb);
            reduce_parts_kernel<<<(unsigned)((p.entries + 31) / 32), 256, 0, st>>>(part1, p.entries, blocks, dw);
            if (db) {
                const size_t off = simt_conv_wgrad_ws(g) - bias_grad_ws((int64_t)g.n * g.od * g.oh * g.ow, g.co);
                lamp_status_t sb = bias_grad(dy, db, (char *)ws + off, st);
                if (sb != LAMP_OK) return sb;
            }
            return launch_status();
        }
    }
    float *part = (float *)ws;
    float *cpart = (float *)((char *)ws + align_up((size_t)p.splits * p.entries * 4, 256));
    if (p.V == 0) {
        LAMP_CUDA_OK(cudaMemsetAsync(dw, 0, p.entries * 4, st));
        if (db) LAMP_CUDA_OK(cudaMemsetAsync(db, 0, (size_t)g.co * 4, st));
        return LAMP_OK;
    }
    dim3 grid((unsigned)((p.entries + 255) / 256), p.splits);
    if (g.transposed)
        conv_wgrad_kernel<true><<<grid, 256, 0, st>>>(g, (const bf16 *)x.p, x.pitch, (const bf16 *)dy.p, dy.pitch, part, p.entries, p.rows, p.rows_per_split);
    else
        conv_wgrad_kernel<false><<<grid, 256, 0, st>>>(g, (const bf16 *)x.p, x.pitch, (const bf16 *)dy.p, dy.pitch, part, p.entries, p.rows, p.rows_per_split);
    reduce_parts_kernel<<<(unsigned)((p.entries + 31) / 32), 256, 0, st>>>(part, p.entries, p.splits, dw);
    if (db) {
        colsum_kernel<<<p.cs_blocks, 256, 0, st>>>((const bf16 *)dy.p, dy.pitch, g.co, p.V, p.v_per_block, cpart);
        reduce_parts_kernel<<<(g.co + 31) / 32, 256, 0, st>>>(cpart, g.co, p.cs_blocks, db);
    }
    return launch_status();
}

}  // namespace lamp
