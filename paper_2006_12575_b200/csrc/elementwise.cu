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
    pdl_launch_dependents();
    pdl_wait();
    const int G = C >> 3, RB = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    if (r >= RB) return;
    const int n = blockIdx.y;
    // blocks are numbered back to front: the convolution in front wrote y front to back, so the tensor's tail is what
    // the L2 cache still holds, and the head of z is what the next convolution finds there
    const int64_t v0 = (int64_t)(gridDim.x - 1 - blockIdx.x) * v_per_block, v1 = min(Vn, v0 + v_per_block);
    // the first voxels are requested before the per-channel constants: their latency overlaps the fp64 arithmetic
    constexpr int PF = 4;
    uint4 pre[PF];
#pragma unroll
    for (int k = 0; k < PF; ++k) {
        const int64_t vv = v0 + r + (int64_t)k * RB;
        pre[k] = vv < v1 ? __ldg(reinterpret_cast<const uint4 *>(y + ((int64_t)n * Vn + vv) * yp + g * 8)) : make_uint4(0, 0, 0, 0);
    }
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
    // groups of PF voxels: the next group's loads are issued before the current group is normalised and stored
    for (int64_t vb = v0 + r; vb < v1; vb += (int64_t)PF * RB) {
        uint4 cur[PF];
#pragma unroll
        for (int k = 0; k < PF; ++k) cur[k] = pre[k];
#pragma unroll
        for (int k = 0; k < PF; ++k) {
            const int64_t vv = vb + (int64_t)(PF + k) * RB;
            pre[k] = vv < v1 ? __ldg(reinterpret_cast<const uint4 *>(y + ((int64_t)n * Vn + vv) * yp + g * 8)) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int k = 0; k < PF; ++k) {
            const int64_t vv = vb + (int64_t)k * RB;
            if (vv < v1) {
                float f[8];
                unpack8(cur[k], f);
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] = fmaxf((f[j] - mu[j]) * rs[j], 0.f);
                *reinterpret_cast<uint4 *>(z + ((int64_t)n * Vn + vv) * zp + g * 8) = pack8(f);
            }
        }
    }
}

// ------------------------------------------------------------------ InstanceNorm backward
// pass 1: per (n, c)  sum g  and  sum g * xhat,  g = (dza + dzb) * [xhat > 0]
// HAS_B: a second gradient source exists.  PF voxels per thread are in flight while PF others are summed; without the
// second source twice as many fit in the same registers (the kernel is bound by the bytes it keeps in flight).
template <bool HAS_B, int PF>
__global__ void __launch_bounds__(256, 2)
instnorm_bwd_sums_kernel(const bf16 *__restrict__ dza, int64_t ap, const bf16 *__restrict__ dzb, int64_t bp,
                         const bf16 *__restrict__ y, int64_t yp, const float *__restrict__ mr,
                         double *__restrict__ sums, int64_t Vn, int C, int64_t v_per_block)
{
    pdl_launch_dependents();
    pdl_wait();
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
        // back to front (the tail of the gradient just written is still in L2); pass 2 then walks front to back
        // and finds the head of dz and y that this pass read last
        const int64_t v0 = (int64_t)(gridDim.x - 1 - blockIdx.x) * v_per_block;
        const int64_t v1 = min(Vn, v0 + v_per_block);
        // groups of PF voxels, the next group's loads in flight while the current one is summed; voxels past the end
        // arrive as zero gradients and add nothing
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        uint4 py[PF], pa[PF], pb[PF];
        auto fetch = [&](int64_t vv, uint4 &qy, uint4 &qa, uint4 &qb) {
            const bool in = vv < v1;
            const int64_t v = (int64_t)n * Vn + vv;
            qy = in ? __ldg(reinterpret_cast<const uint4 *>(y + v * yp + g * 8)) : zero4;
            qa = in ? __ldg(reinterpret_cast<const uint4 *>(dza + v * ap + g * 8)) : zero4;
            qb = (HAS_B && in) ? __ldg(reinterpret_cast<const uint4 *>(dzb + v * bp + g * 8)) : zero4;
        };
#pragma unroll
        for (int k = 0; k < PF; ++k) fetch(v0 + r + (int64_t)k * RB, py[k], pa[k], pb[k]);
        for (int64_t vb = v0 + r; vb < v1; vb += (int64_t)PF * RB) {
            uint4 cy[PF], ca[PF], cb[PF];
#pragma unroll
            for (int k = 0; k < PF; ++k) { cy[k] = py[k]; ca[k] = pa[k]; cb[k] = pb[k]; }
#pragma unroll
            for (int k = 0; k < PF; ++k) fetch(vb + (int64_t)(PF + k) * RB, py[k], pa[k], pb[k]);
#pragma unroll
            for (int k = 0; k < PF; ++k) {
                float fy[8], fa[8], fb[8];
                unpack8(cy[k], fy);
                unpack8(ca[k], fa);
                unpack8(cb[k], fb);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float xh = (fy[j] - mu[j]) * rs[j];
                    const float gg = xh > 0.f ? (HAS_B ? fa[j] + fb[j] : fa[j]) : 0.f;
                    s[j] += gg;
                    s[8 + j] = fmaf(gg, xh, s[8 + j]);
                }
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

// pass 2: dy = rstd * (g - m1 - xhat * m2); same thread layout as the forward kernel.
// With DB the kernel also forms the bias gradient of the conv in front, db[c] = sum over all voxels and samples of
// the dy values as stored (bf16): block sums go to db_acc (fp64 atomics, zero on entry) and the block that
// finishes last (ticket counter db_count, zero on entry) converts the totals to fp32.
template <bool DB, bool HAS_B, int PF>
__global__ void __launch_bounds__(256, 2)
instnorm_bwd_apply_kernel(const bf16 *__restrict__ dza, int64_t ap, const bf16 *__restrict__ dzb, int64_t bp,
                          const bf16 *__restrict__ y, int64_t yp, const float *__restrict__ mr,
                          const double *__restrict__ sums, bf16 *__restrict__ dy, int64_t dp, int64_t Vn, int C,
                          int64_t v_per_block, double *__restrict__ db_acc, unsigned *__restrict__ db_count,
                          float *__restrict__ db_out)
{
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ float cred[];          // DB: [RB][C] column sums of the block
    __shared__ int is_last;
    const int G = C >> 3, RB = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    const bool active = r < RB;
    const int n = blockIdx.y;
    const float inv_v = 1.0f / (float)Vn;
    float mu[8], rs[8], m1[8], m2[8], cs[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int64_t i = (int64_t)n * C + g * 8 + j;
        mu[j] = active ? mr[2 * i] : 0.f;
        rs[j] = active ? mr[2 * i + 1] : 0.f;
        m1[j] = active ? (float)sums[2 * i] * inv_v : 0.f;
        m2[j] = active ? (float)sums[2 * i + 1] * inv_v : 0.f;
        cs[j] = 0.f;
    }
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = active ? min(Vn, v0 + v_per_block) : v0;
    // groups of PF voxels, the next group's loads in flight while the current one is processed
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    uint4 py[PF], pa[PF], pb[PF];
    auto fetch = [&](int64_t vv, uint4 &qy, uint4 &qa, uint4 &qb) {
        const bool in = vv < v1;
        const int64_t v = (int64_t)n * Vn + vv;
        qy = in ? __ldg(reinterpret_cast<const uint4 *>(y + v * yp + g * 8)) : zero4;
        qa = in ? __ldg(reinterpret_cast<const uint4 *>(dza + v * ap + g * 8)) : zero4;
        qb = (HAS_B && in) ? __ldg(reinterpret_cast<const uint4 *>(dzb + v * bp + g * 8)) : zero4;
    };
#pragma unroll
    for (int k = 0; k < PF; ++k) fetch(v0 + r + (int64_t)k * RB, py[k], pa[k], pb[k]);
    for (int64_t vb = v0 + r; vb < v1; vb += (int64_t)PF * RB) {
        uint4 cy[PF], ca[PF], cb[PF];
#pragma unroll
        for (int k = 0; k < PF; ++k) { cy[k] = py[k]; ca[k] = pa[k]; cb[k] = pb[k]; }
#pragma unroll
        for (int k = 0; k < PF; ++k) fetch(vb + (int64_t)(PF + k) * RB, py[k], pa[k], pb[k]);
#pragma unroll
        for (int k = 0; k < PF; ++k) {
            const int64_t vv = vb + (int64_t)k * RB;
            if (vv >= v1) break;
            const int64_t v = (int64_t)n * Vn + vv;
            float fy[8], fa[8], fb[8];
            unpack8(cy[k], fy);
            unpack8(ca[k], fa);
            unpack8(cb[k], fb);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float xh = (fy[j] - mu[j]) * rs[j];
                const float gg = xh > 0.f ? (HAS_B ? fa[j] + fb[j] : fa[j]) : 0.f;
                fa[j] = rs[j] * (gg - m1[j] - xh * m2[j]);
            }
            const uint4 q = pack8(fa);
            *reinterpret_cast<uint4 *>(dy + v * dp + g * 8) = q;
            if (DB) {
                unpack8(q, fa);
#pragma unroll
                for (int j = 0; j < 8; ++j) cs[j] += fa[j];
            }
        }
    }
    if (!DB) return;
    if (active) {
#pragma unroll
        for (int j = 0; j < 8; ++j) cred[r * C + g * 8 + j] = cs[j];
    }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += 256) {
        float a = 0.f;
        for (int rr = 0; rr < RB; ++rr) a += cred[rr * C + c];
        atomicAdd(db_acc + c, (double)a);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned total = gridDim.x * gridDim.y;
        is_last = atomicAdd(db_count, 1u) == total - 1;
    }
    __syncthreads();
    if (is_last) {
        __threadfence();
        for (int c = threadIdx.x; c < C; c += 256) db_out[c] = (float)__ldcg(db_acc + c);
    }
}

// ------------------------------------------------------------------ head: 1x1x1 conv + softmax (+ Dice sums)
constexpr int KMAX = 16;

// KP = K rounded up to a multiple of 4 (rows k >= K of the weights are zero, their logits are masked).  A block walks
// tiles of 256 consecutive voxels, one voxel per thread; the probabilities of a tile leave through shared memory so
// that the [voxel][K] rows are written as one contiguous run.
template <int KP>
__global__ void __launch_bounds__(256)
head_softmax_kernel(const bf16 *__restrict__ z, int64_t zp, int C, const bf16 *__restrict__ w,
                    const float *__restrict__ b, int K, float *__restrict__ probs, uint8_t *__restrict__ amax,
                    const uint8_t *__restrict__ labels, double *__restrict__ dice, int64_t Vn, int64_t v_per_block)
{
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ __align__(16) float sm[];   // w as float [KP][C], bias [KP], reduce [3*KMAX], probability tile [256][K]
    float *sw = sm, *sb = sm + KP * C, *sred = sb + KP, *sp = sred + 3 * KMAX;
    for (int i = threadIdx.x; i < KP * C; i += 256) sw[i] = i < K * C ? bf2f(w[i]) : 0.f;
    if (threadIdx.x < KP) sb[threadIdx.x] = (threadIdx.x < K && b) ? b[threadIdx.x] : 0.f;
    if (threadIdx.x < 3 * KMAX) sred[threadIdx.x] = 0.f;
    __syncthreads();
    const int n = blockIdx.y;
    float sP[KP], sI[KP], sG[KP];
#pragma unroll
    for (int k = 0; k < KP; ++k) { sP[k] = 0.f; sI[k] = 0.f; sG[k] = 0.f; }
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(Vn, v0 + v_per_block);
    for (int64_t base = v0; base < v1; base += 256) {
        const int64_t vv = base + threadIdx.x;
        const bool live = vv < v1;
        const int64_t v = (int64_t)n * Vn + vv;
        if (live) {
            float l[KP];
#pragma unroll
            for (int k = 0; k < KP; ++k) l[k] = sb[k];
            const uint4 *zr = reinterpret_cast<const uint4 *>(z + v * zp);
            for (int c0 = 0; c0 < C; c0 += 32) {
                uint4 q[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) q[u] = (c0 + 8 * u < C) ? __ldg(zr + (c0 >> 3) + u) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (c0 + 8 * u < C) {
                        float f[8];
                        unpack8(q[u], f);
#pragma unroll
                        for (int k = 0; k < KP; ++k) {
                            const float4 wa = *reinterpret_cast<const float4 *>(sw + k * C + c0 + 8 * u);
                            const float4 wb = *reinterpret_cast<const float4 *>(sw + k * C + c0 + 8 * u + 4);
                            l[k] = fmaf(f[0], wa.x, l[k]); l[k] = fmaf(f[1], wa.y, l[k]);
                            l[k] = fmaf(f[2], wa.z, l[k]); l[k] = fmaf(f[3], wa.w, l[k]);
                            l[k] = fmaf(f[4], wb.x, l[k]); l[k] = fmaf(f[5], wb.y, l[k]);
                            l[k] = fmaf(f[6], wb.z, l[k]); l[k] = fmaf(f[7], wb.w, l[k]);
                        }
                    }
                }
            }
            float mx = l[0];
            int am = 0;
#pragma unroll
            for (int k = 1; k < KP; ++k) if (k < K && l[k] > mx) { mx = l[k]; am = k; }
            float sum = 0.f;
#pragma unroll
            for (int k = 0; k < KP; ++k) { l[k] = k < K ? expf(l[k] - mx) : 0.f; sum += l[k]; }
            const float inv = 1.0f / sum;
            const int lab = labels ? labels[v] : -1;
#pragma unroll
            for (int k = 0; k < KP; ++k) {
                const float p = l[k] * inv;
                if (k < K) sp[threadIdx.x * K + k] = p;
                sP[k] += p;
                if (k == lab) { sI[k] += p; sG[k] += 1.f; }
            }
            if (amax) amax[v] = (uint8_t)am;
        }
        if (probs) {
            __syncthreads();
            const int nv = (int)((v1 - base) < 256 ? (v1 - base) : 256);
            float *dst = probs + ((int64_t)n * Vn + base) * K;
            for (int i = threadIdx.x; i < nv * K; i += 256) dst[i] = sp[i];
            __syncthreads();
        }
    }
    if (dice) {
#pragma unroll
        for (int k = 0; k < KP; ++k) {
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
    pdl_launch_dependents();
    pdl_wait();
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
// dW[k][c] = sum_v dl[v,k] z[v,c]; db[k] = sum_v dl[v,k].
// A block walks tiles of 256 voxels.  Step 1, one voxel per thread: dl (kept in shared memory) and the dz row.
// Step 2, thread = (pair of channels, voxel lane): the outer products dl x z of the tile's voxels, accumulated in
// registers over all tiles.  At the end the voxel lanes are added in lane order and the block writes ITS sums to
// partW[block][K*C], partB[block][K]; a fixed-order reduction over the blocks follows (deterministic).
template <int KP>
__global__ void __launch_bounds__(256)
head_bwd_kernel(const bf16 *__restrict__ z, int64_t zp, int C, const bf16 *__restrict__ w, int K,
                const float *__restrict__ probs, const uint8_t *__restrict__ labels, const double *__restrict__ dice,
                int N, bf16 *__restrict__ dz, int64_t dzp, float *__restrict__ partW, float *__restrict__ partB,
                float *__restrict__ dlog, int64_t Vn, int64_t v_per_block)
{
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ __align__(16) float sm[];
    // [KP*C] weights, [KP] + [KP] dice coefficients, then the tile: dl [256][KP], probabilities [256][K], z [256][C] bf16
    float *sw = sm, *sa = sm + KP * C, *sbq = sa + KP, *sdl = sbq + KP, *sp = sdl + 256 * KP;
    bf16 *sz = reinterpret_cast<bf16 *>(sp + 256 * K);          // every offset so far is a multiple of 4 floats
    const int n = blockIdx.y;
    for (int i = threadIdx.x; i < KP * C; i += 256) sw[i] = i < K * C ? bf2f(w[i]) : 0.f;
    if (threadIdx.x < KP) {
        float a = 0.f, bq = 0.f;
        if (threadIdx.x < K) {
            const double eps = 1e-5;
            const double *q = dice + ((int64_t)n * K + threadIdx.x) * 3;
            const double den = q[1] + q[2] + eps;
            a = (float)(2.0 / (den * N * K));
            bq = (float)((2.0 * q[0] + eps) / (den * den * N * K));
        }
        sa[threadIdx.x] = a;
        sbq[threadIdx.x] = bq;
    }
    const int C8 = C >> 3, CP = C >> 1, VL = 256 / CP;
    const int cp = threadIdx.x % CP, vl = threadIdx.x / CP;
    float acc[KP][2], accb[KP];
#pragma unroll
    for (int k = 0; k < KP; ++k) { acc[k][0] = 0.f; acc[k][1] = 0.f; accb[k] = 0.f; }
    const int64_t v0 = (int64_t)blockIdx.x * v_per_block, v1 = min(Vn, v0 + v_per_block);
    for (int64_t base = v0; base < v1; base += 256) {
        const int nv = (int)((v1 - base) < 256 ? (v1 - base) : 256);
        const int64_t vb = (int64_t)n * Vn + base;
        __syncthreads();                                         // the previous tile has been consumed
        for (int i = threadIdx.x; i < nv * K; i += 256) sp[i] = __ldg(probs + vb * K + i);
        for (int i = threadIdx.x; i < 256 * C8; i += 256) {
            const int row = i / C8, col = i - row * C8;
            reinterpret_cast<uint4 *>(sz)[i] =
                row < nv ? __ldg(reinterpret_cast<const uint4 *>(z + (vb + row) * zp) + col) : make_uint4(0, 0, 0, 0);
        }
        __syncthreads();
        {
            float dl[KP];
            if (threadIdx.x < nv) {
                const int64_t v = vb + threadIdx.x;
                const int lab = labels[v];
                float p[KP], dp[KP], dotp = 0.f;
#pragma unroll
                for (int k = 0; k < KP; ++k) {
                    p[k] = k < K ? sp[threadIdx.x * K + k] : 0.f;
                    dp[k] = -((k == lab ? sa[k] : 0.f) - sbq[k]);
                    dotp = fmaf(p[k], dp[k], dotp);
                }
#pragma unroll
                for (int k = 0; k < KP; ++k) {
                    dl[k] = p[k] * (dp[k] - dotp);
                    if (k < K && dlog) dlog[v * K + k] = dl[k];
                }
                for (int c0 = 0; c0 < C; c0 += 8) {
                    float f[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) f[j] = 0.f;
#pragma unroll
                    for (int k = 0; k < KP; ++k) {
                        const float4 wa = *reinterpret_cast<const float4 *>(sw + k * C + c0);
                        const float4 wb = *reinterpret_cast<const float4 *>(sw + k * C + c0 + 4);
                        f[0] = fmaf(dl[k], wa.x, f[0]); f[1] = fmaf(dl[k], wa.y, f[1]);
                        f[2] = fmaf(dl[k], wa.z, f[2]); f[3] = fmaf(dl[k], wa.w, f[3]);
                        f[4] = fmaf(dl[k], wb.x, f[4]); f[5] = fmaf(dl[k], wb.y, f[5]);
                        f[6] = fmaf(dl[k], wb.z, f[6]); f[7] = fmaf(dl[k], wb.w, f[7]);
                    }
                    *reinterpret_cast<uint4 *>(dz + v * dzp + c0) = pack8(f);
                }
            } else {
#pragma unroll
                for (int k = 0; k < KP; ++k) dl[k] = 0.f;
            }
#pragma unroll
            for (int k4 = 0; k4 < KP / 4; ++k4)
                *reinterpret_cast<float4 *>(sdl + threadIdx.x * KP + 4 * k4) =
                    make_float4(dl[4 * k4], dl[4 * k4 + 1], dl[4 * k4 + 2], dl[4 * k4 + 3]);
        }
        __syncthreads();
        if (vl < VL) {
            for (int t = vl; t < 256; t += VL) {
                const __nv_bfloat162 zz = *reinterpret_cast<const __nv_bfloat162 *>(sz + t * C + 2 * cp);
                const float z0 = __low2float(zz), z1 = __high2float(zz);
#pragma unroll
                for (int k4 = 0; k4 < KP / 4; ++k4) {
                    const float4 d = *reinterpret_cast<const float4 *>(sdl + t * KP + 4 * k4);
                    const float dd[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        acc[4 * k4 + u][0] = fmaf(dd[u], z0, acc[4 * k4 + u][0]);
                        acc[4 * k4 + u][1] = fmaf(dd[u], z1, acc[4 * k4 + u][1]);
                        if (cp == 0) accb[4 * k4 + u] += dd[u];
                    }
                }
            }
        }
    }
    // block totals: red[vl][k][c] over the tile region of shared memory, then entry threads add the lanes in order
    __syncthreads();
    float *red = sdl, *redb = sdl + VL * KP * C;
    if (vl < VL) {
#pragma unroll
        for (int k = 0; k < KP; ++k) {
            red[(vl * KP + k) * C + 2 * cp] = acc[k][0];
            red[(vl * KP + k) * C + 2 * cp + 1] = acc[k][1];
            if (cp == 0) redb[vl * KP + k] = accb[k];
        }
    }
    __syncthreads();
    const int64_t blk = (int64_t)blockIdx.y * gridDim.x + blockIdx.x;
    for (int e = threadIdx.x; e < K * C; e += 256) {
        float a = 0.f;
        for (int r = 0; r < VL; ++r) a += red[r * KP * C + e];      // e = k * C + c
        partW[blk * K * C + e] = a;
    }
    if (threadIdx.x < K) {
        float a = 0.f;
        for (int r = 0; r < VL; ++r) a += redb[r * KP + threadIdx.x];
        partB[blk * K + threadIdx.x] = a;
    }
}

// ------------------------------------------------------------------ parameter update
// v = alpha v + (1 - alpha) g^2; w -= lr g / (sqrt(v) + eps); bf16 copy.  Four elements per thread when the
// pointers allow 16-byte accesses (22 bytes of traffic per element: HBM-bound).
__global__ void __launch_bounds__(256)
rmsprop_kernel(int64_t n, const float *__restrict__ g, float *__restrict__ w, float *__restrict__ v,
               bf16 *__restrict__ wb, float lr, float alpha, float eps, int vec)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    auto upd = [&](float gi, float &wi, float &vi) {
        vi = fmaf(alpha, vi, (1.0f - alpha) * gi * gi);
        wi -= lr * gi / (sqrtf(vi) + eps);
    };
    if (vec) {
        if (4 * i >= n) return;
        const float4 g4 = __ldg(reinterpret_cast<const float4 *>(g) + i);
        float4 w4 = reinterpret_cast<float4 *>(w)[i], v4 = reinterpret_cast<float4 *>(v)[i];
        upd(g4.x, w4.x, v4.x); upd(g4.y, w4.y, v4.y); upd(g4.z, w4.z, v4.z); upd(g4.w, w4.w, v4.w);
        reinterpret_cast<float4 *>(w)[i] = w4;
        reinterpret_cast<float4 *>(v)[i] = v4;
        if (wb) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(w4.x, w4.y), hi = __floats2bfloat162_rn(w4.z, w4.w);
            uint2 u;
            u.x = *reinterpret_cast<uint32_t *>(&lo);
            u.y = *reinterpret_cast<uint32_t *>(&hi);
            reinterpret_cast<uint2 *>(wb)[i] = u;
        }
    } else {
        if (i >= n) return;
        float wi = w[i], vi = v[i];
        upd(g[i], wi, vi);
        w[i] = wi; v[i] = vi;
        if (wb) wb[i] = f2bf(wi);
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
    pdl_launch_dependents();
    pdl_wait();
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
                   float *__restrict__ planar, uint8_t *__restrict__ amax, int p_first, int p_count,
                   float *__restrict__ wsum_out)
{
    pdl_launch_dependents();
    pdl_wait();
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
                // only patches p_first .. p_first + p_count - 1 take part (pp holds those, back to back)
                const int64_t pg = ((int64_t)id * nh + ih) * nw + iw;
                if (pg < p_first || pg >= (int64_t)p_first + p_count) continue;
                const int64_t pi = pg - p_first;
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
    if (wsum_out) {
        // partial result of a share of the patches: the weighted sums as they are and the weight totals; the
        // division and the arg max follow once the shares have been added (overlap_finish_kernel)
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                if (VEC == 4) *reinterpret_cast<float4 *>(planar + k * plane + v0) = make_float4(acc[0][k], acc[1][k], acc[2][k], acc[3][k]);
                else          planar[k * plane + v0] = acc[0][k];
            }
        }
        if (VEC == 4) *reinterpret_cast<float4 *>(wsum_out + v0) = make_float4(wsum[0], wsum[1], wsum[2], wsum[3]);
        else          wsum_out[v0] = wsum[0];
        return;
    }
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

// A[k][v] = acc[k][v] / wsum[v] in place (the same two operations as the one-pass kernel: reciprocal, multiply);
// arg max over k, lowest index on ties.
__global__ void __launch_bounds__(256)
overlap_finish_kernel(float *__restrict__ planar, const float *__restrict__ wsum, int K, int64_t V, int write_probs,
                      uint8_t *__restrict__ amax)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t v = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (v >= V) return;
    const float inv = 1.0f / wsum[v];
    float best = -1.f;
    int am = 0;
    for (int k = 0; k < K; ++k) {
        const float a = planar[k * V + v] * inv;
        if (write_probs) planar[k * V + v] = a;
        if (a > best) { best = a; am = k; }
    }
    if (amax) amax[v] = (uint8_t)am;
}

}  // namespace

// launches over at most this many elements count as short (see launch_pdl)
constexpr int64_t SHORT_ELEMS = (int64_t)32 << 20;

lamp_status_t k_instnorm_relu_fwd(const TView &y, const double *stats, float eps, float *mu_rstd, const TView &z,
                                  cudaStream_t st)
{
    const int64_t Vn = (int64_t)y.d * y.h * y.w;
    if (Vn == 0 || y.n == 0) return LAMP_OK;
    if (y.c / 8 > 256) return LAMP_ERR_UNSUPPORTED;
    const int64_t rb = 256 / (y.c / 8);
    int64_t vpb = (Vn / ((int64_t)sm_count() * 16) + rb - 1) / rb * rb;
    if (vpb < rb * 8) vpb = rb * 8;
    dim3 grid((unsigned)((Vn + vpb - 1) / vpb), y.n);
    (void)launch_pdl((int64_t)y.n * Vn * y.c <= SHORT_ELEMS, instnorm_relu_fwd_kernel, grid, dim3(256), (size_t)(0), st, (const bf16 *)y.p, y.pitch, stats, 1.0 / (double)Vn, eps, mu_rstd,
                                                   (bf16 *)z.p, z.pitch, Vn, y.c, vpb);
    return launch_status();
}

lamp_status_t k_instnorm_relu_bwd(const TView &dza, const TView *dzb, const TView &y, const float *mu_rstd,
                                  double *sums, bool sums_are_zero, const TView &dy, double *db_acc, unsigned *db_count,
                                  float *db, cudaStream_t st)
{
    const int64_t Vn = (int64_t)y.d * y.h * y.w;
    const int C = y.c, G = C / 8;
    if (G > 256) return LAMP_ERR_UNSUPPORTED;
    if (!sums_are_zero) LAMP_CUDA_OK(cudaMemsetAsync(sums, 0, (size_t)y.n * C * 2 * sizeof(double), st));
    if (Vn == 0 || y.n == 0) {
        if (db) LAMP_CUDA_OK(cudaMemsetAsync(db, 0, (size_t)C * sizeof(float), st));
        return LAMP_OK;
    }
    const int RB = 256 / G;
    // pass 1: at most 8 blocks per SM, and at least 16 voxels per thread: every block ends with 2 C fp64 atomics, which
    // dominate when a small tensor is cut into many blocks
    int64_t blocks = ((int64_t)sm_count() * 8 + y.n - 1) / y.n;
    const int64_t max_blocks = (Vn + RB * 16 - 1) / (RB * 16);
    if (blocks > max_blocks) blocks = max_blocks;
    const int64_t vpb = (Vn + blocks - 1) / blocks;
    blocks = (Vn + vpb - 1) / vpb;
    const size_t smem = (size_t)RB * G * 16 * sizeof(float);
    const bf16 *pa = (const bf16 *)dza.p, *pb = dzb ? (const bf16 *)dzb->p : nullptr, *py = (const bf16 *)y.p;
    const int64_t bpitch = dzb ? dzb->pitch : 0;
    const dim3 sgrid((unsigned)blocks, y.n);
    const bool early = (int64_t)y.n * Vn * C <= SHORT_ELEMS;
    if (pb)
        (void)launch_pdl(early, instnorm_bwd_sums_kernel<true, 2>, sgrid, dim3(256), smem, st, pa, dza.pitch, pb, bpitch, py, y.pitch,
                         mu_rstd, sums, Vn, C, vpb);
    else
        (void)launch_pdl(early, instnorm_bwd_sums_kernel<false, 4>, sgrid, dim3(256), smem, st, pa, dza.pitch, pb, bpitch, py, y.pitch,
                         mu_rstd, sums, Vn, C, vpb);
    int64_t vpa = (Vn / ((int64_t)sm_count() * 16) + RB - 1) / RB * RB;
    if (vpa < (int64_t)RB * 8) vpa = (int64_t)RB * 8;
    dim3 grid((unsigned)((Vn + vpa - 1) / vpa), y.n);
    const size_t dsmem = db ? (size_t)RB * C * sizeof(float) : 0;
    bf16 *pd = (bf16 *)dy.p;
#define LAMP_IN_APPLY(DBV, HB, PFV)                                                                                       \
    (void)launch_pdl(early, instnorm_bwd_apply_kernel<DBV, HB, PFV>, grid, dim3(256), dsmem, st, pa, dza.pitch, pb, bpitch, py,  \
                     y.pitch, mu_rstd, (const double *)sums, pd, dy.pitch, Vn, C, vpa, db_acc, db_count, db)
    if (db) { if (pb) LAMP_IN_APPLY(true, true, 2); else LAMP_IN_APPLY(true, false, 4); }
    else    { if (pb) LAMP_IN_APPLY(false, true, 2); else LAMP_IN_APPLY(false, false, 4); }
#undef LAMP_IN_APPLY
    return launch_status();
}

static void head_grid(int64_t Vn, int n, int64_t &blocks, int64_t &vpb)
{
    blocks = ((int64_t)sm_count() * 8 + n - 1) / n;
    const int64_t max_blocks = (Vn + 255) / 256;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    vpb = (Vn + blocks - 1) / blocks;
    vpb = (vpb + 255) / 256 * 256;
    blocks = (Vn + vpb - 1) / vpb;
}

static int head_kp(int K) { return (K + 3) / 4 * 4; }

lamp_status_t k_head_softmax(const TView &z, const bf16 *w, const float *b, int K, float *probs, uint8_t *argmax,
                             const uint8_t *labels, double *dice_sums, cudaStream_t st)
{
    const int64_t Vn = (int64_t)z.d * z.h * z.w;
    if (K > KMAX || K < 1 || z.c > 128 || z.c % 8) return LAMP_ERR_UNSUPPORTED;
    if (dice_sums) LAMP_CUDA_OK(cudaMemsetAsync(dice_sums, 0, (size_t)z.n * K * 3 * sizeof(double), st));
    if (Vn == 0 || z.n == 0) return LAMP_OK;
    if (umma_head_supported(z, K) && ((uintptr_t)w & 15) == 0) return umma_head(z, w, b, K, probs, argmax, labels, dice_sums, st);
    int64_t blocks, vpb;
    head_grid(Vn, z.n, blocks, vpb);
    const int KP = head_kp(K);
    const size_t smem = ((size_t)KP * z.c + KP + 3 * KMAX + 256 * K) * sizeof(float);
    const dim3 grid((unsigned)blocks, z.n);
#define LAMP_HEAD_FWD(kp)                                                                                         \
    (void)launch_pdl((int64_t)z.n * Vn <= SHORT_ELEMS / 32, head_softmax_kernel<kp>, grid, dim3(256), (size_t)(smem), st, (const bf16 *)z.p, z.pitch, z.c, w, b, K, probs, argmax, labels, \
                                                     dice_sums, Vn, vpb)
    switch (KP) {
    case 4:  LAMP_HEAD_FWD(4); break;
    case 8:  LAMP_HEAD_FWD(8); break;
    case 12: LAMP_HEAD_FWD(12); break;
    default: LAMP_HEAD_FWD(16); break;
    }
#undef LAMP_HEAD_FWD
    return launch_status();
}

lamp_status_t k_dice_loss(const double *dice_sums, int N, int K, float *loss, cudaStream_t st)
{
    (void)launch_pdl(true, dice_loss_kernel, dim3(1), dim3(32), (size_t)(0), st, dice_sums, N, K, loss);
    return launch_status();
}

size_t head_bwd_ws(int64_t Vn, int n, int K, int C)
{
    if (Vn <= 0 || n <= 0) return 0;
    int64_t blocks, vpb;
    head_grid(Vn, n, blocks, vpb);
    return align_up((size_t)blocks * n * K * C * sizeof(float), 256) + align_up((size_t)blocks * n * K * sizeof(float), 256);
}

template <int KP>
static lamp_status_t launch_head_bwd(const TView &z, const bf16 *w, int K, const float *probs, const uint8_t *labels,
                                     const double *dice_sums, const TView &dz, float *partW, float *partB, float *dlogits,
                                     int64_t Vn, int64_t blocks, int64_t vpb, cudaStream_t st)
{
    const int C = z.c;
    // the tile region (dl, probabilities, z) is reused for the end-of-block reduction [lanes][KP][C] + [lanes][KP]
    const size_t lanes = 256 / (C / 2);
    const size_t tile = (size_t)256 * KP + 256 * K + 128 * C, red = lanes * KP * C + lanes * KP;
    const size_t smem = ((size_t)KP * C + 2 * KP + (tile > red ? tile : red)) * sizeof(float);
    static SmemAttrOnce attr;
    { const lamp_status_t as = attr.ensure(head_bwd_kernel<KP>, (int)(128 * 1024)); if (as != LAMP_OK) return as; }
    (void)launch_pdl((int64_t)z.n * Vn <= SHORT_ELEMS / 32, head_bwd_kernel<KP>, dim3((unsigned)blocks, z.n), dim3(256), (size_t)(smem), st, 
        (const bf16 *)z.p, z.pitch, C, w, K, probs, labels, dice_sums, z.n, (bf16 *)dz.p, dz.pitch, partW, partB, dlogits,
        Vn, vpb);
    return launch_status();
}

// ws: head_bwd_ws bytes (per-block partial sums of dW and db)
lamp_status_t k_head_bwd(const TView &z, const bf16 *w, int K, const float *probs, const uint8_t *labels,
                         const double *dice_sums, const TView &dz, float *dw, float *db, float *dlogits,
                         void *ws, size_t ws_bytes, cudaStream_t st)
{
    const int64_t Vn = (int64_t)z.d * z.h * z.w;
    const int C = z.c;
    // the block's shared memory holds the weights, 256 voxels of z and the lane partials: 107 KB at C = 128, K = 16
    if (K > KMAX || C > 128 || C % 8) return LAMP_ERR_UNSUPPORTED;
    if (Vn == 0 || z.n == 0) {
        LAMP_CUDA_OK(cudaMemsetAsync(dw, 0, (size_t)K * C * sizeof(float), st));
        if (db) LAMP_CUDA_OK(cudaMemsetAsync(db, 0, (size_t)K * sizeof(float), st));
        return LAMP_OK;
    }
    if (!ws || ws_bytes < head_bwd_ws(Vn, z.n, K, C)) return LAMP_ERR_WORKSPACE;
    int64_t blocks, vpb;
    head_grid(Vn, z.n, blocks, vpb);
    float *partW = (float *)ws;
    float *partB = (float *)((char *)ws + align_up((size_t)blocks * z.n * K * C * sizeof(float), 256));
    lamp_status_t s;
    switch (head_kp(K)) {
    case 4:  s = launch_head_bwd<4>(z, w, K, probs, labels, dice_sums, dz, partW, partB, dlogits, Vn, blocks, vpb, st); break;
    case 8:  s = launch_head_bwd<8>(z, w, K, probs, labels, dice_sums, dz, partW, partB, dlogits, Vn, blocks, vpb, st); break;
    case 12: s = launch_head_bwd<12>(z, w, K, probs, labels, dice_sums, dz, partW, partB, dlogits, Vn, blocks, vpb, st); break;
    default: s = launch_head_bwd<16>(z, w, K, probs, labels, dice_sums, dz, partW, partB, dlogits, Vn, blocks, vpb, st); break;
    }
    if (s != LAMP_OK) return s;
    if ((s = reduce_partials(partW, (int64_t)K * C, (int)(blocks * z.n), dw, st)) != LAMP_OK) return s;
    return db ? reduce_partials(partB, K, (int)(blocks * z.n), db, st) : LAMP_OK;
}

lamp_status_t k_rmsprop(int64_t n, const float *g, float *w, float *v, bf16 *wb, float lr, float alpha, float eps,
                        cudaStream_t st)
{
    if (n == 0) return LAMP_OK;
    const bool vec = n % 4 == 0 && (((uintptr_t)g | (uintptr_t)w | (uintptr_t)v) & 15) == 0 && ((uintptr_t)wb & 7) == 0;
    const int64_t threads = vec ? n / 4 : n;
    (void)launch_pdl(n <= SHORT_ELEMS, rmsprop_kernel, dim3((unsigned)((threads + 255) / 256)), dim3(256), (size_t)(0), st, n, g, w, v, wb, lr, alpha, eps, vec ? 1 : 0);
    return launch_status();
}

lamp_status_t k_gather_patches(const TView &vol, const TView &patches, int first_patch, const int32_t nst[3],
                               const int32_t stride[3], cudaStream_t st)
{
    const int64_t total = (int64_t)patches.n * patches.d * patches.h * patches.w * patches.c;
    if (total == 0) return LAMP_OK;
    (void)launch_pdl(total <= SHORT_ELEMS, gather_patches_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), (size_t)(0), st, 
        (const bf16 *)vol.p, vol.pitch, vol.d, vol.h, vol.w, vol.c, (bf16 *)patches.p, patches.pitch, patches.n,
        patches.d, patches.h, patches.w, first_patch, nst[0], nst[1], nst[2], stride[0], stride[1], stride[2]);
    return launch_status();
}

lamp_status_t k_overlap_finish(float *planar, const float *wsum, int K, int64_t V, int write_probs, uint8_t *argmax,
                               cudaStream_t st)
{
    if (K > KMAX || K < 1) return LAMP_ERR_UNSUPPORTED;
    if (V == 0) return LAMP_OK;
    (void)launch_pdl(V <= SHORT_ELEMS / 32, overlap_finish_kernel, dim3((unsigned)((V + 255) / 256)), dim3(256), (size_t)0, st,
                     planar, wsum, K, V, write_probs, argmax);
    return launch_status();
}

lamp_status_t k_overlap_add(const float *pp, int K, int D, int H, int W, const int32_t patch[3],
                            const int32_t nst[3], const int32_t stride[3], int window, float *planar,
                            uint8_t *argmax, cudaStream_t st, int p_first, int p_count, float *wsum_out)
{
    if (K > KMAX || K < 1) return LAMP_ERR_UNSUPPORTED;
    if (p_count < 0) { p_first = 0; p_count = nst[0] * nst[1] * nst[2]; }
    if (wsum_out && !planar) return LAMP_ERR_INVALID_ARG;
    if ((int64_t)D * H * W == 0) return LAMP_OK;
    const size_t smem = (size_t)(patch[0] + patch[1] + patch[2]) * sizeof(float);
    const bool vec = (W % 4 == 0) && ((uintptr_t)planar % 16 == 0) && ((uintptr_t)argmax % 4 == 0) && ((uintptr_t)wsum_out % 16 == 0);
    const int aligned4 = vec && patch[2] % 4 == 0 && (nst[2] == 1 || stride[2] % 4 == 0) && (W - patch[2]) % 4 == 0 &&
                         ((uintptr_t)pp % 16 == 0);
#define LAMP_OA(VECN, KTN)                                                                                              \
    (void)launch_pdl(total <= SHORT_ELEMS / 32, overlap_add_kernel<VECN, KTN>, dim3((unsigned)((total + 255) / 256)), dim3(256), (size_t)(smem), st,                                 \
        pp, K, D, H, W, patch[0], patch[1], patch[2], nst[0], nst[1], nst[2], stride[0], stride[1], stride[2], window, \
        aligned4, planar, argmax, p_first, p_count, wsum_out)
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
