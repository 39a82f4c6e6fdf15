// 3x3x3 stride-1 pad-1 convolution, c_out in blocks of at most 128 channels: "weights x voxels"
// implicit GEMM with the activation planes resident in shared memory.
//
// Why this shape.  One tcgen05.mma (M = 128, K = 16, bf16) occupies the tensor pipe for N/2 cycles and a
// thread issues at most one every 60-100 cycles (measured): N = 256 keeps one issuing thread ahead of the pipe.  With output channels on N, a 64-channel layer
// would run at 42 % of it.  So here the OUTPUT CHANNELS are the M rows (A operand = weight tile
// [128 x 64], K-major) and 256 OUTPUT VOXELS are the N columns (B operand = an 8 (w) x 32 (h) window of
// an activation plane, K-major): D^T[co, voxel] += W[co, ci] * X[voxel + tap, ci].
//
//  * Activation planes.  For (input plane p, 64-channel chunk) one TMA load brings a halo box of
//    34 x 10 voxels (out-of-volume voxels zero-filled = the conv's zero padding) with 128-byte swizzled
//    rows.  The nine in-plane taps are shifted windows of that box: the shared-memory descriptor starts
//    (kh*10 + kw) rows in and steps 10 rows between 8-voxel groups.  The swizzle is a function of the
//    shared-memory address bits, so such a window reads exactly what TMA wrote.
//  * Narrow layers.  With c_out = 64 (32) the 128 rows hold the weights of 2 (4) CONSECUTIVE OUTPUT
//    PLANES: input plane p is tap kd = p - o + 1 of output plane o, so row block j carries the weights
//    of tap (kd = p - (o0 + j) + 1, kh, kw); where that kd falls outside 0..2 the TMA coordinate is out
//    of range and the block is zero-filled.  2 planes cost 4 input planes of MMAs instead of 2 x 3 at
//    half-empty M: 75 % (50 % for c_out = 32) of the full rate instead of 50 % (25 %).
//  * Accumulators: 128 lanes x 256 fp32 columns, two of them in TMEM, so the epilogue of one tile
//    overlaps the MMAs of the next.  The epilogue owns one output channel per thread: bias and the
//    InstanceNorm sums are per-thread scalars; a 32 x 32 shared-memory transpose per warp turns
//    TMEM rows into 64-byte (bf16) or 128-byte (fp32) channel runs per voxel for the NDHWC store.
//
//  * Stride 2 (ST = 2, the down-sampling conv).  Output voxel (h', w') reads input rows 2h' + kh - 1 and columns
//    2w' + kw - 1: per input plane FOUR parity boxes are loaded, each by one TMA box with element stride 2 along
//    w and h (9 x 33 voxels starting at (2 w0 - pw, 2 h0 - ph), pw / ph = 1 for the odd lattice).  Tap kw = 1 is a
//    window of the even-w box, kw = 0 and kw = 2 are the windows 0 and 1 voxels into the odd-w box (the same along
//    h), so every input voxel is fetched once per plane instead of once per tap.  Output plane o reads input
//    planes 2o - 1 .. 2o + 1: stacked block j carries tap kd = pi - 2j of input plane 2 o0 - 1 + pi (the weight box
//    walks kd with element stride 2).  Channels go in chunks of 32 so that two planes of four boxes fit.
//
// Warps: 0 = activation-plane TMA producer, 1 = MMA issuer (+ TMEM owner), 2 = weight-tile TMA
// producer, 3..6 = epilogue.  All waits are bounded (LAMP_ERR_TIMEOUT on expiry).
#include <cuda.h>
#include <cudaTypedefs.h>
#include "common.cuh"
#include "umma_ptx.cuh"

namespace lamp {

namespace {

using namespace ptx;

constexpr int CT_THREADS = 224;
constexpr int TW = 8, TH = 32;          // output window: 8 (w) x 32 (h) = 256 voxels = N
constexpr int HALO_W = TW + 2, HALO_H = TH + 2;
constexpr int MAX_NP = 4, MAX_NW = 8;

constexpr int S2_BOX_W = TW + 1, S2_BOX_H = TH + 1;      // voxels a stride-2 parity box delivers
constexpr int S2_SUB_BYTES = ((S2_BOX_W * S2_BOX_H * 64 + 1023) / 1024) * 1024;   // one parity box of 32 channels

struct CtParams {
    int32_t N, D, H, W;                 // extents of the OUTPUT tensor
    int32_t ID;                         // depth of the input tensor (= D for stride 1)
    int32_t nwt, nht, ngr, nct;         // tiles along w, h; plane groups; c_out blocks of 128
    int32_t chunks;                     // c_in / KC
    int32_t total_items;
    int32_t co, mirror, y_f32;
    int32_t np, nw;                     // ring depths: activation planes, weight tiles
    int32_t plane_bytes;                // 1024-aligned bytes of one plane box
    int64_t y_pitch;
    void   *y;
    const float *bias;
    double *stats;
    int    *status;
};

struct Item { int n, o0, h0, w0, ct; };

template <int S>
__device__ __forceinline__ Item decode_item(const CtParams &P, int item)
{
    Item it;
    it.ct = item % P.nct; item /= P.nct;
    it.w0 = (item % P.nwt) * TW; item /= P.nwt;
    it.h0 = (item % P.nht) * TH; item /= P.nht;
    it.o0 = (item % P.ngr) * S;
    it.n = item / P.ngr;
    return it;
}

// KC: channels per chunk (64: 128-byte swizzle, 32: 64-byte swizzle).  COB: output channels per plane
// inside the 128 rows (128, 64 or 32); S = 128 / COB output planes are stacked.
template <int KC, int COB, int ST>
__global__ void __launch_bounds__(CT_THREADS, 1)
conv3_t_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const CtParams P)
{
    constexpr int S = 128 / COB;
    constexpr int ROWB = KC * 2;
    constexpr uint32_t SWZ = KC == 64 ? 2u : 4u;
    static_assert(ST == 1 || KC == 32, "the stride-2 form works on 32-channel chunks");
    constexpr uint32_t S2_BOX_BYTES = S2_BOX_W * S2_BOX_H * ROWB;          // bytes one parity box delivers
    constexpr uint32_t PLANE_BOX_BYTES = ST == 1 ? HALO_W * HALO_H * ROWB : 4 * S2_BOX_BYTES;
    constexpr int NPL = ST == 1 ? S + 2 : 2 * S + 1;           // input planes an item of S output planes reads
    constexpr uint32_t W_BYTES = 128 * ROWB;                  // one tap's weight tile
    constexpr int TPS = (KC == 32 && ST == 1) ? 3 : 1;         // taps (one kh row) per weight stage: 32-channel chunks carry
                                                               // too little work per tap to pay a barrier round trip each
    constexpr uint32_t WST_BYTES = TPS * W_BYTES;
    constexpr uint32_t IDESC = make_idesc(256);
    // 32 -> 32 channels: all weights stay in shared memory.  Per in-plane tap the region [0 0 0 k0 k1 k2] of 32-row
    // blocks (kd = 0, 1, 2 after three zero blocks; three more zero blocks close the last region): the 128 stacked rows
    // of input plane pi are the four consecutive blocks that start at block pi (forward) or 5 - pi (mirrored taps).
    constexpr bool WRES = (KC == 32 && COB == 32 && ST == 1);
    constexpr uint32_t BLK_BYTES = 32 * ROWB;                  // one block of 32 output channels
    constexpr uint32_t WRES_TAP_BYTES = 6 * BLK_BYTES;
    constexpr uint32_t WRES_BYTES = 9 * WRES_TAP_BYTES + 3 * BLK_BYTES;

    extern __shared__ uint8_t smem_raw[];
    // aligned by offsetting the shared array itself, so that the compiler still sees shared-memory pointers
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *p_base = smem;
    uint8_t *w_base = p_base + (size_t)P.np * P.plane_bytes;
    float *epi = (float *)(w_base + (WRES ? (size_t)WRES_BYTES : (size_t)P.nw * WST_BYTES));
    uint64_t *bars = (uint64_t *)((uint8_t *)epi + 4 * 32 * 33 * 4);
    const uint32_t pfull0 = smem_u32(bars), pempty0 = smem_u32(bars + MAX_NP);
    const uint32_t wfull0 = smem_u32(bars + 2 * MAX_NP), wempty0 = smem_u32(bars + 2 * MAX_NP + MAX_NW);
    const uint32_t tfull0 = smem_u32(bars + 2 * MAX_NP + 2 * MAX_NW), tempty0 = tfull0 + 16;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * MAX_NP + 2 * MAX_NW + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_NP; ++s) { mbar_init(pfull0 + 8 * s, 1); mbar_init(pempty0 + 8 * s, 1); }
        for (int s = 0; s < MAX_NW; ++s) { mbar_init(wfull0 + 8 * s, 1); mbar_init(wempty0 + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(tfull0 + 8 * s, 1); mbar_init(tempty0 + 8 * s, 4); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    if (WRES) {
        // zero blocks of the resident weights (the kd blocks arrive by TMA below)
        for (uint32_t i = threadIdx.x; i < WRES_BYTES / 16; i += CT_THREADS) {
            const uint32_t off = i * 16, in_tap = off % WRES_TAP_BYTES;
            if (off >= 9 * WRES_TAP_BYTES || in_tap < 3 * BLK_BYTES) *reinterpret_cast<uint4 *>(w_base + off) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();
    }
    pdl_wait();                 // everything above touched shared and tensor memory only
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------------------- activation planes
            int ps = 0;
            uint32_t pph = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x) {
                const Item it = decode_item<S>(P, item);
                for (int pi = 0; pi < NPL && ok; ++pi) {
                    const int p = ST * it.o0 - 1 + pi;
                    if (p < 0 || p >= P.ID) continue;
                    for (int c = 0; c < P.chunks; ++c) {
                        if (!mbar_wait(pempty0 + 8 * ps, pph ^ 1, abort_flag)) { ok = false; break; }
                        mbar_expect_tx(pfull0 + 8 * ps, PLANE_BOX_BYTES);
                        const uint32_t dst = smem_u32(p_base + (size_t)ps * P.plane_bytes);
                        if (ST == 1) {
                            tma_load_5d(dst, &map_x, pfull0 + 8 * ps, c * KC, it.w0 - 1, it.h0 - 1, p, it.n);
                        } else {
                            // parity box (ph, pw): every second voxel from (2 h0 - ph, 2 w0 - pw)
#pragma unroll
                            for (int sb = 0; sb < 4; ++sb)
                                tma_load_5d(dst + sb * S2_SUB_BYTES, &map_x, pfull0 + 8 * ps, c * KC, 2 * it.w0 - (sb & 1),
                                            2 * it.h0 - (sb >> 1), p, it.n);
                        }
                        if (++ps == P.np) { ps = 0; pph ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 2) {
        if (lane == 0) {
            // ---------------------------------------------------------------- weight tiles
            int ws = 0;
            uint32_t wph = 0;
            bool ok = true;
            if (WRES) {
                // once: the three kd blocks of every in-plane tap (mirrored taps read tap 8 - t9)
                mbar_expect_tx(wfull0, 27 * BLK_BYTES);
                for (int t9 = 0; t9 < 9; ++t9)
                    tma_load_4d(smem_u32(w_base + t9 * WRES_TAP_BYTES + 3 * BLK_BYTES), &map_w, wfull0, 0, 0, 0, P.mirror ? 8 - t9 : t9);
            }
            for (int item = blockIdx.x; item < P.total_items && ok && !WRES; item += gridDim.x) {
                const Item it = decode_item<S>(P, item);
                for (int pi = 0; pi < NPL && ok; ++pi) {
                    const int p = ST * it.o0 - 1 + pi;
                    if (p < 0 || p >= P.ID) continue;
                    for (int c = 0; c < P.chunks && ok; ++c) {
                        for (int t9 = 0; t9 < 9; t9 += TPS) {
                            if (!mbar_wait(wempty0 + 8 * ws, wph ^ 1, abort_flag)) { ok = false; break; }
                            mbar_expect_tx(wfull0 + 8 * ws, WST_BYTES);
                            // one box fetches TPS taps x S stacked blocks: slot s, block b holds tap (kd, t9 + s) with
                            // kd = pi - (S - 1) + b (forward) or, with mirrored taps, the weight tap (2 - pi + b, 8 - t9 - (TPS - 1) + s);
                            // kd outside 0..2 is outside the tensor and arrives as zeros
                            const uint32_t dst = smem_u32(w_base + (size_t)ws * WST_BYTES);
                            // (stride 2: the box walks kd with element stride 2, block b holds kd = pi - 2 (S - 1) + 2 b)
                            if (P.mirror) tma_load_4d(dst, &map_w, wfull0 + 8 * ws, c * KC, it.ct * 128, 2 - pi, 8 - t9 - (TPS - 1));
                            else          tma_load_4d(dst, &map_w, wfull0 + 8 * ws, c * KC, it.ct * 128, pi - ST * (S - 1), t9);
                            if (++ws == P.nw) { ws = 0; wph ^= 1; }
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------------------------------------------------------- MMA issuer
            int ps = 0, ws = 0;
            uint32_t pph = 0, wph = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            if (WRES) { ok = mbar_wait(wfull0, 0, abort_flag); tc_fence_after(); }
            for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x) {
                const Item it = decode_item<S>(P, item);
                if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * 256;
                uint32_t accumulate = 0;
                for (int pi = 0; pi < NPL && ok; ++pi) {
                    const int p = ST * it.o0 - 1 + pi;
                    if (p < 0 || p >= P.ID) continue;
                    for (int c = 0; c < P.chunks && ok; ++c) {
                        if (!mbar_wait(pfull0 + 8 * ps, pph, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t plane = smem_u32(p_base + (size_t)ps * P.plane_bytes);
                        if (WRES) {
                            const uint32_t wwin = smem_u32(w_base) + (uint32_t)(P.mirror ? 5 - pi : pi) * BLK_BYTES;
#pragma unroll
                            for (int t9 = 0; t9 < 9; ++t9) {
                                const uint64_t da = make_desc(wwin + t9 * WRES_TAP_BYTES, 0, 8 * ROWB, SWZ);
                                const uint64_t db = make_desc(plane + ((t9 / 3) * HALO_W + t9 % 3) * ROWB, 0, HALO_W * ROWB, SWZ);
#pragma unroll
                                for (int k = 0; k < KC / 16; ++k) {
                                    umma_bf16(d_tmem, da + 2 * k, db + 2 * k, IDESC, accumulate);
                                    accumulate = 1;
                                }
                            }
                        }
                        for (int t9 = 0; t9 < 9 && !WRES; t9 += TPS) {
                            if (!mbar_wait(wfull0 + 8 * ws, wph, abort_flag)) { ok = false; break; }
                            tc_fence_after();
#pragma unroll
                            for (int sl = 0; sl < TPS; ++sl) {
                                const int t = P.mirror ? t9 + TPS - 1 - sl : t9 + sl;        // conv tap whose weights sit in slot sl
                                const int kh = t / 3, kw = t - kh * 3;
                                const uint64_t da = make_desc(smem_u32(w_base + (size_t)ws * WST_BYTES + sl * W_BYTES), 0, 8 * ROWB, SWZ);
                                // stride 2: tap 1 reads the even box, taps 0 and 2 the odd box 0 and 1 voxels in
                                const uint64_t db = ST == 1
                                    ? make_desc(plane + (kh * HALO_W + kw) * ROWB, 0, HALO_W * ROWB, SWZ)
                                    : make_desc(plane + ((kh != 1) * 2 + (kw != 1)) * S2_SUB_BYTES + ((kh == 2) * S2_BOX_W + (kw == 2)) * ROWB,
                                                0, S2_BOX_W * ROWB, SWZ);
#pragma unroll
                                for (int k = 0; k < KC / 16; ++k) {
                                    umma_bf16(d_tmem, da + 2 * k, db + 2 * k, IDESC, accumulate);
                                    accumulate = 1;
                                }
                            }
                            umma_commit(wempty0 + 8 * ws);
                            if (++ws == P.nw) { ws = 0; wph ^= 1; }
                        }
                        if (!ok) break;
                        umma_commit(pempty0 + 8 * ps);
                        if (++ps == P.np) { ps = 0; pph ^= 1; }
                    }
                }
                if (!ok) break;
                umma_commit(tfull0 + 8 * acc);
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1;
            }
        }
    } else {
        // -------------------------------------------------------------------- epilogue (warps 3..6)
        const int q = warp & 3;                                 // TMEM lane quarter of this warp
        float *tr = epi + (warp - 3) * 32 * 33;
        // which stacked output plane these 32 lanes belong to: block b = (q * 32) / COB carries tap kd = pi - (S - 1) + b
        // of output plane o0 + (S - 1 - b) in the forward pass, and of plane o0 + b with mirrored taps
        const int jplane = P.mirror ? (q * 32) / COB : S - 1 - (q * 32) / COB;
        const int co_in_blk = (q * 32) % COB;                   // first of this warp's 32 channels inside the block
        uint32_t acc = 0, acc_phase = 0;
        float s1 = 0.f, s2 = 0.f;                               // sums of this thread's channel
        int stat_n = -1, stat_ct = 0;
        bool ok = true;
        auto flush = [&]() {
            if (P.stats && stat_n >= 0) {
                double *dst = P.stats + ((int64_t)stat_n * P.co + stat_ct * 128 + co_in_blk + lane) * 2;
                atomicAdd(dst, (double)s1);
                atomicAdd(dst + 1, (double)s2);
            }
            s1 = 0.f; s2 = 0.f;
        };
        for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x) {
            const Item it = decode_item<S>(P, item);
            if (it.n != stat_n || it.ct != stat_ct) { flush(); stat_n = it.n; stat_ct = it.ct; }
            const int o = it.o0 + jplane;
            const bool plane_ok = o < P.D;
            const int cbase = it.ct * 128 + co_in_blk;          // first of this warp's channels in the tensor
            const float bias = P.bias ? __ldg(P.bias + cbase + lane) : 0.f;
            ok = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
#pragma unroll 1
            for (int c0 = 0; c0 < 256; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(trow + c0, r);
                tmem_ld_wait();
                if (plane_ok && !P.y_f32) {
                    // bf16 output: two voxels of a channel are rounded and packed into one word BEFORE the transpose, a
                    // lane then takes 16 channels of a voxel pair: half the shared-memory traffic of the fp32 form (the
                    // epilogue's shared-memory work slows the tensor pipe, which reads its operands from there too)
                    uint32_t *trw = reinterpret_cast<uint32_t *>(tr);
                    __syncwarp();
#pragma unroll
                    for (int jp = 0; jp < 16; ++jp) {
                        float f2[2];
#pragma unroll
                        for (int v = 0; v < 2; ++v) {
                            const int col = c0 + 2 * jp + v;
                            const bool valid = (it.w0 + (col & 7) < P.W) && (it.h0 + (col >> 3) < P.H);
                            const float f = valid ? __uint_as_float(r[2 * jp + v]) + bias : 0.f;
                            s1 += f;
                            s2 = fmaf(f, f, s2);
                            f2[v] = f;
                        }
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(f2[0], f2[1]);
                        trw[jp * 33 + lane] = *reinterpret_cast<uint32_t *>(&h2);
                    }
                    __syncwarp();
                    const int jp = lane >> 1, ch0 = (lane & 1) * 16;
                    uint32_t wv[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) wv[e] = trw[jp * 33 + ch0 + e];
#pragma unroll
                    for (int v = 0; v < 2; ++v) {
                        const int col = c0 + 2 * jp + v;
                        const int w = it.w0 + (col & 7), h = it.h0 + (col >> 3);
                        if (w < P.W && h < P.H) {
                            const int64_t vox = (((int64_t)it.n * P.D + o) * P.H + h) * P.W + w;
                            uint4 *dst = reinterpret_cast<uint4 *>((bf16 *)P.y + vox * P.y_pitch + cbase + ch0);
                            uint32_t ow[8];
#pragma unroll
                            for (int k = 0; k < 8; ++k) ow[k] = __byte_perm(wv[2 * k], wv[2 * k + 1], v ? 0x7632 : 0x5410);
                            dst[0] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                            dst[1] = make_uint4(ow[4], ow[5], ow[6], ow[7]);
                        }
                    }
                } else if (plane_ok) {
                    // r[j] = channel (cbase + lane) at voxel column c0 + j: column = hl * 8 + wx
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int col = c0 + j;
                        const bool valid = (it.w0 + (col & 7) < P.W) && (it.h0 + (col >> 3) < P.H);
                        const float f = valid ? __uint_as_float(r[j]) + bias : 0.f;
                        s1 += f;
                        s2 = fmaf(f, f, s2);
                        tr[j * 33 + lane] = f;
                    }
                    __syncwarp();
                    // this lane now stores voxel column c0 + lane: 32 consecutive channels
                    const int col = c0 + lane;
                    const int w = it.w0 + (col & 7), h = it.h0 + (col >> 3);
                    if (w < P.W && h < P.H) {
                        const int64_t vox = (((int64_t)it.n * P.D + o) * P.H + h) * P.W + w;
                        if (P.y_f32) {
                            float4 *dst = reinterpret_cast<float4 *>((float *)P.y + vox * P.y_pitch + cbase);
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                dst[e] = make_float4(tr[lane * 33 + 4 * e], tr[lane * 33 + 4 * e + 1], tr[lane * 33 + 4 * e + 2],
                                                     tr[lane * 33 + 4 * e + 3]);
                        } else {
                            uint4 *dst = reinterpret_cast<uint4 *>((bf16 *)P.y + vox * P.y_pitch + cbase);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float f8[8];
#pragma unroll
                                for (int u = 0; u < 8; ++u) f8[u] = tr[lane * 33 + 8 * e + u];
                                dst[e] = pack8(f8);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1;
        }
        flush();
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && P.status) atomicExch(P.status, (int)LAMP_ERR_TIMEOUT);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

PFN_cuTensorMapEncodeTiled_v12000 get_encode() { return (PFN_cuTensorMapEncodeTiled_v12000)tensor_map_encoder(); }

struct CtPlan { CtParams P; int KC, COB, ST; size_t smem; int grid; };

constexpr int EPI_BYTES = 4 * 32 * 33 * 4;
constexpr int CTRL_BYTES = 1024;
constexpr int SMEM_LIMIT = 227 * 1024;

bool make_ct_plan(const ConvGeom &g, CtPlan *out)
{
    if (!(g.k == 3 && (g.s == 1 || g.s == 2) && g.p == 1 && !g.transposed)) return false;
    if (g.ci % 32) return false;
    const int ST = g.s;
    int COB;
    if (g.co == 32 || g.co == 64) COB = g.co;
    else if (g.co % 128 == 0) COB = 128;
    else return false;
    const int KC = (g.ci % 64 == 0 && ST == 1) ? 64 : 32;
    const int S = 128 / COB;
    CtParams &P = out->P;
    P.N = g.n; P.D = g.od; P.H = g.oh; P.W = g.ow;            // the tiles cover the output tensor
    P.ID = g.d;
    P.chunks = g.ci / KC;
    const int rowb = KC * 2;
    P.plane_bytes = ST == 1 ? (int)align_up((size_t)HALO_W * HALO_H * rowb, 1024) : 4 * S2_SUB_BYTES;
    const int w_bytes = 128 * rowb * ((KC == 32 && ST == 1) ? 3 : 1);      // bytes of one weight stage
    const int budget = SMEM_LIMIT - 1024 - EPI_BYTES - CTRL_BYTES;
    int np = (KC == 64 || ST == 2) ? 2 : 4;
    int nw = (budget - np * P.plane_bytes) / w_bytes;
    if (nw > MAX_NW) nw = MAX_NW;
    if (nw < 3) return false;
    // 32 -> 32 channels: the weights are resident (nine regions of six 2 KB blocks plus three closing zero blocks)
    const bool wres = KC == 32 && COB == 32 && ST == 1;
    const size_t wres_bytes = (size_t)(9 * 6 + 3) * 32 * rowb;
    P.np = np; P.nw = nw;
    P.nwt = (g.ow + TW - 1) / TW;
    P.nht = (g.oh + TH - 1) / TH;
    P.ngr = (g.od + S - 1) / S;
    P.nct = g.co / (COB == 128 ? 128 : COB);
    const int64_t items = (int64_t)g.n * P.ngr * P.nht * P.nwt * P.nct;
    if (items > 0x7FFFFFFF || items <= 0) return false;
    P.total_items = (int32_t)items;
    P.co = g.co;
    const int sms = sm_count();
    out->KC = KC; out->COB = COB; out->ST = ST;
    out->smem = 1024 + (size_t)np * P.plane_bytes + (wres ? wres_bytes : (size_t)nw * w_bytes) + EPI_BYTES + CTRL_BYTES;
    if (out->smem > (size_t)SMEM_LIMIT) return false;
    out->grid = (int)(items < sms ? items : sms);
    return true;
}

template <int KC, int COB, int ST = 1>
lamp_status_t launch_ct(const CUtensorMap &mx, const CUtensorMap &mw, const CtPlan &pl, cudaStream_t st)
{
    static SmemAttrOnce attr;
    { const lamp_status_t as = attr.ensure(conv3_t_kernel<KC, COB, ST>, (int)(SMEM_LIMIT)); if (as != LAMP_OK) return as; }
    return launch_pdl(pl.P.total_items <= 4 * pl.grid, conv3_t_kernel<KC, COB, ST>, dim3(pl.grid), dim3(CT_THREADS), pl.smem, st, mx, mw, pl.P);
}

}  // namespace

bool ct_conv_fwd_supported(const ConvGeom &g, const TView &x, const TView &y)
{
    CtPlan pl;
    if ((int64_t)g.n * g.d * g.h * g.w == 0) return false;
    if (!make_ct_plan(g, &pl)) return false;
    // the 8 x 32 window must not be mostly padding
    const double used = (double)g.oh * g.ow / ((double)pl.P.nht * TH * pl.P.nwt * TW);
    if (used < 0.55) return false;
    if (x.pitch % 8 || ((uintptr_t)x.p & 15)) return false;
    if (y.f32 ? (y.pitch % 4 != 0) : (y.pitch % 8 != 0)) return false;
    if ((uintptr_t)y.p & 15) return false;
    return true;
}

lamp_status_t ct_conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                          double *stats, int mirror_taps, cudaStream_t st)
{
    CtPlan pl;
    if (!make_ct_plan(g, &pl)) return LAMP_ERR_UNSUPPORTED;
    PFN_cuTensorMapEncodeTiled_v12000 encode = get_encode();
    if (!encode) return LAMP_ERR_CUDA;
    CtParams &P = pl.P;
    P.mirror = mirror_taps; P.y_f32 = y.f32; P.y_pitch = y.pitch; P.y = y.p;
    P.bias = bias; P.stats = stats; P.status = status_word_ptr();
    const CUtensorMapSwizzle swz = pl.KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    CUtensorMap mx, mw;
    {
        const cuuint64_t dims[5] = {(cuuint64_t)g.ci, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.d, (cuuint64_t)g.n};
        const cuuint64_t strides[4] = {(cuuint64_t)x.pitch * 2, (cuuint64_t)x.pitch * 2 * g.w,
                                       (cuuint64_t)x.pitch * 2 * g.w * g.h, (cuuint64_t)x.pitch * 2 * g.w * g.h * g.d};
        // stride 2: a parity box takes every second voxel along w and h (the box spans twice what it delivers)
        const cuuint32_t s2 = pl.ST == 2;
        const cuuint32_t box[5] = {(cuuint32_t)pl.KC, s2 ? 2u * S2_BOX_W : (cuuint32_t)HALO_W, s2 ? 2u * S2_BOX_H : (cuuint32_t)HALO_H, 1, 1};
        const cuuint32_t es[5] = {1, s2 ? 2u : 1u, s2 ? 2u : 1u, 1, 1};
        if (encode(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, x.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    {
        // weights viewed as (c_in, c_out, kd, kh*3+kw): a box spans the stacked kd blocks, then the taps of a stage
        const cuuint64_t dims[4] = {(cuuint64_t)g.ci, (cuuint64_t)g.co, 3, 9};
        const cuuint64_t strides[3] = {(cuuint64_t)g.ci * 2, (cuuint64_t)g.ci * 2 * g.co * 9, (cuuint64_t)g.ci * 2 * g.co};
        const bool wres = pl.KC == 32 && pl.COB == 32 && pl.ST == 1;      // resident weights: one box = the three kd blocks of a tap
        // stride 2: the stacked blocks are two kd apart (block b of input plane pi carries kd = pi - 2 (S - 1) + 2 b)
        const cuuint32_t nblk = 128 / pl.COB;
        const cuuint32_t box[4] = {(cuuint32_t)pl.KC, (cuuint32_t)pl.COB, (cuuint32_t)(wres ? 3 : nblk * (pl.ST == 2 ? 2 : 1)),
                                   (cuuint32_t)(wres ? 1 : ((pl.KC == 32 && pl.ST == 1) ? 3 : 1))};
        const cuuint32_t es[4] = {1, 1, (cuuint32_t)(pl.ST == 2 ? 2 : 1), 1};
        if (encode(&mw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, (void *)w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    if (pl.ST == 2) {
        if (mirror_taps) return LAMP_ERR_UNSUPPORTED;
        switch (pl.COB) {
        case 32:  return launch_ct<32, 32, 2>(mx, mw, pl, st);
        case 64:  return launch_ct<32, 64, 2>(mx, mw, pl, st);
        case 128: return launch_ct<32, 128, 2>(mx, mw, pl, st);
        }
        return LAMP_ERR_UNSUPPORTED;
    }
    const int key = pl.KC * 1000 + pl.COB;
    switch (key) {
    case 64 * 1000 + 32:  return launch_ct<64, 32>(mx, mw, pl, st);
    case 64 * 1000 + 64:  return launch_ct<64, 64>(mx, mw, pl, st);
    case 64 * 1000 + 128: return launch_ct<64, 128>(mx, mw, pl, st);
    case 32 * 1000 + 32:  return launch_ct<32, 32>(mx, mw, pl, st);
    case 32 * 1000 + 64:  return launch_ct<32, 64>(mx, mw, pl, st);
    case 32 * 1000 + 128: return launch_ct<32, 128>(mx, mw, pl, st);
    }
    return LAMP_ERR_UNSUPPORTED;
}

}  // namespace lamp
