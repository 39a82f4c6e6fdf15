// 3x3x3 stride-1 pad-1 convolution as an implicit GEMM on the sm_100a tensor cores.
//
//   y[v, co] = b[co] + sum_{tap, ci} x[v + off(tap), ci] * w[tap][co][ci]
//   GEMM view: M = output voxels (tiles of 128 = tw x th x td), N = c_out (tile BN), K = 27 * c_in.
//
// Per CTA (persistent over tiles), warp-specialised:
//   warp 0   : TMA producer.  For each (tap, channel chunk) it loads the A tile - a tw x th x td box of
//              the NDHWC activation shifted by the tap offset, out-of-volume voxels zero-filled by the
//              TMA unit, which is exactly the zero padding - and the matching [BN x KC] weight tile,
//              both with the 128-byte (KC = 64) or 64-byte (KC = 32) shared-memory swizzle.
//   warp 1   : allocates TMEM and issues tcgen05.mma (M = 128, N = BN, K = 16 per instruction) from one
//              thread; fp32 accumulators live in TMEM, double-buffered so that the epilogue of tile i
//              overlaps the MMAs of tile i + 1.
//   warps 2-5: epilogue.  tcgen05.ld the accumulator rows (one voxel per thread), add the bias, reduce
//              the per-channel sum and sum of squares (InstanceNorm statistics), convert and store the
//              row into the output's channel slice.
// The data-gradient pass runs the same kernel on dy with the taps mirrored and the weights transposed.
// Every mbarrier wait is bounded; on expiry the CTA records LAMP_ERR_TIMEOUT and winds down.
#include <cuda.h>
#include <cudaTypedefs.h>
#include "common.cuh"
#include "umma_ptx.cuh"

namespace lamp {

namespace {

using namespace ptx;

struct UmmaParams {
    int32_t N, D, H, W;            // volume
    int32_t tw, th, td;            // voxel tile, tw * th * td = 128
    int32_t ntw, nth, ntd;         // tiles per axis
    int32_t nct;                   // c_out tiles
    int32_t chunks;                // c_in / KC
    int32_t total_tiles;
    int32_t co;                    // c_out
    int32_t mirror;                // 1: weight tap index = 26 - tap
    int32_t y_f32;
    int64_t y_pitch;
    void   *y;
    const float *bias;
    double *stats;                 // [N][co][2] or NULL
    int    *status;
};

constexpr int NUM_THREADS = 192;
constexpr int MAX_STAGES = 8;

template <int KC, int BN>
struct SmemLayout {
    static constexpr int A_BYTES = 128 * KC * 2;
    static constexpr int B_BYTES = BN * KC * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;      // multiple of 1024 for every (KC, BN)
    static constexpr int EPI_BYTES = 4 * 32 * 33 * 4;
    static constexpr int CTRL_BYTES = 1024;
    static constexpr int BUDGET = 227 * 1024 - 1024 /* alignment slack */ - EPI_BYTES - CTRL_BYTES;
    static constexpr int STAGES = (BUDGET / STAGE_BYTES) < MAX_STAGES ? (BUDGET / STAGE_BYTES) : MAX_STAGES;
    static constexpr int TOTAL = 1024 + STAGES * STAGE_BYTES + EPI_BYTES + CTRL_BYTES;
    static constexpr int TMEM_COLS = (2 * BN <= 32) ? 32 : (2 * BN <= 64) ? 64 : (2 * BN <= 128) ? 128 : (2 * BN <= 256) ? 256 : 512;
};

template <int KC, int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv3_umma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const UmmaParams P)
{
    using L = SmemLayout<KC, BN>;
    constexpr int STAGES = L::STAGES;
    constexpr uint32_t SWZ = (KC == 64) ? 2u : 4u;
    constexpr uint32_t SBO = 8 * KC * 2;                       // bytes per 8-row group
    constexpr uint32_t IDESC = make_idesc(BN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *stage_base = smem;
    float *epi = (float *)(smem + STAGES * L::STAGE_BYTES);
    uint64_t *bars = (uint64_t *)(smem + STAGES * L::STAGE_BYTES + L::EPI_BYTES);
    // bars: full[STAGES], empty[STAGES], tfull[2], tempty[2]; then tmem base (u32) and abort flag (int)
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * MAX_STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + MAX_STAGES);
    const uint32_t tfull0 = smem_u32(bars + 2 * MAX_STAGES), tempty0 = smem_u32(bars + 2 * MAX_STAGES + 2);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, 4); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), L::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int kiters = 27 * P.chunks;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x) {
                int t = tile;
                const int ct = t % P.nct; t /= P.nct;
                const int wt = t % P.ntw; t /= P.ntw;
                const int ht = t % P.nth; t /= P.nth;
                const int dt = t % P.ntd;
                const int n = t / P.ntd;
                const int w0 = wt * P.tw, h0 = ht * P.th, d0 = dt * P.td;
                for (int ki = 0; ki < kiters; ++ki) {
                    const int tap = ki / P.chunks, ch = ki - tap * P.chunks;
                    const int kd = tap / 9, kh = (tap / 3) % 3, kw = tap % 3;
                    if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t fb = full0 + 8 * stage;
                    mbar_expect_tx(fb, L::STAGE_BYTES);
                    const uint32_t sa = smem_u32(stage_base + stage * L::STAGE_BYTES);
                    tma_load_5d(sa, &map_x, fb, ch * KC, w0 + kw - 1, h0 + kh - 1, d0 + kd - 1, n);
                    tma_load_3d(sa + L::A_BYTES, &map_w, fb, ch * KC, ct * BN, P.mirror ? 26 - tap : tap);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x) {
                if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int ki = 0; ki < kiters; ++ki) {
                    if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(stage_base + stage * L::STAGE_BYTES);
                    const uint64_t da = make_desc(sa, 0, SBO, SWZ), db = make_desc(sa + L::A_BYTES, 0, SBO, SWZ);
#pragma unroll
                    for (int k = 0; k < KC / 16; ++k)       // 16 bf16 = 32 bytes = 2 descriptor address units
                        umma_bf16(d_tmem, da + 2 * k, db + 2 * k, IDESC, (ki | k) ? 1u : 0u);
                    umma_commit(empty0 + 8 * stage);        // frees the stage once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit(tfull0 + 8 * acc);              // accumulator complete
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                             // TMEM lane quarter this warp may read
        float *tr = epi + (warp - 2) * 32 * 33;
        uint32_t acc = 0, acc_phase = 0;
        float s1[BN / 32 + 1], s2[BN / 32 + 1];             // per-lane column sums: column (c0 + lane) of each chunk
#pragma unroll
        for (int i = 0; i < BN / 32 + 1; ++i) { s1[i] = 0.f; s2[i] = 0.f; }
        int stat_n = -1, stat_ct = 0;
        bool ok = true;
        auto flush = [&]() {
            if (P.stats && stat_n >= 0) {
#pragma unroll
                for (int i = 0; i < (BN + 31) / 32; ++i) {
                    const int c = i * 32 + lane;
                    if (c < BN) {
                        double *dst = P.stats + ((int64_t)stat_n * P.co + stat_ct * BN + c) * 2;
                        atomicAdd(dst, (double)s1[i]);
                        atomicAdd(dst + 1, (double)s2[i]);
                    }
                    s1[i] = 0.f; s2[i] = 0.f;
                }
            }
        };
        for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x) {
            int t = tile;
            const int ct = t % P.nct; t /= P.nct;
            const int wt = t % P.ntw; t /= P.ntw;
            const int ht = t % P.nth; t /= P.nth;
            const int dt = t % P.ntd;
            const int n = t / P.ntd;
            if (n != stat_n || ct != stat_ct) { flush(); stat_n = n; stat_ct = ct; }
            const int m = q * 32 + lane;
            const int wx = m % P.tw, hy = (m / P.tw) % P.th, dz = m / (P.tw * P.th);
            const int w = wt * P.tw + wx, h = ht * P.th + hy, d = dt * P.td + dz;
            const bool valid = (w < P.W) && (h < P.H) && (d < P.D);
            const int64_t vox = (((int64_t)n * P.D + d) * P.H + h) * P.W + w;
            // the whole warp takes the same decision, so no lane is left behind at a __syncwarp
            ok = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 32) {
                const int ncol = (BN - c0) < 32 ? (BN - c0) : 32;       // 32, or 16 for the last chunk
                uint32_t r[32];
                if (ncol == 32) tmem_ld32(trow + c0, r); else tmem_ld16(trow + c0, r);
                tmem_ld_wait();
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (j < ncol) {
                        float f = __uint_as_float(r[j]);
                        if (P.bias) f += __ldg(P.bias + ct * BN + c0 + j);
                        v[j] = valid ? f : 0.f;
                    } else v[j] = 0.f;
                }
                if (valid) {
                    if (P.y_f32) {
                        float4 *dst = reinterpret_cast<float4 *>((float *)P.y + vox * P.y_pitch + ct * BN + c0);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (4 * j < ncol) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    } else {
                        uint4 *dst = reinterpret_cast<uint4 *>((bf16 *)P.y + vox * P.y_pitch + ct * BN + c0);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (8 * j < ncol) {
                                float f8[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) f8[e] = v[8 * j + e];
                                dst[j] = pack8(f8);
                            }
                        }
                    }
                }
                if (P.stats) {
                    // transpose through shared memory: lane j then sums column j over the warp's 32 rows
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 32; ++j) tr[lane * 33 + j] = v[j];
                    __syncwarp();
                    float a = 0.f, b = 0.f;
#pragma unroll
                    for (int rr = 0; rr < 32; ++rr) { const float f = tr[rr * 33 + lane]; a += f; b = fmaf(f, f, b); }
                    s1[c0 / 32] += a;
                    s2[c0 / 32] += b;
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

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && P.status) atomicExch(P.status, (int)LAMP_ERR_TIMEOUT);
        // give copies that may still be in flight time to land before the shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

__global__ void transpose_weights_kernel(const bf16 *__restrict__ w, bf16 *__restrict__ wt, int co, int ci, int64_t total)
{
    // wt[t][ci][co] = w[t][co][ci]
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= total) return;
    const int o = (int)(e % co);
    const int i = (int)((e / co) % ci);
    const int64_t t = e / ((int64_t)co * ci);
    wt[e] = w[(t * co + o) * ci + i];
}

// ----------------------------------------------------------------------------------------------
// host side
// ----------------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 get_encode()
{
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (PFN_cuTensorMapEncodeTiled_v12000)p;
    }
    return fn;
}

int pick_bn(int co)
{
    if (co <= 256) return co;
    for (int bn = 256; bn >= 16; bn -= 16)
        if (co % bn == 0) return bn;
    return 0;
}

bool bn_instantiated(int bn) { return bn == 16 || bn == 32 || bn == 64 || bn == 128 || bn == 256; }

void pick_tile(int D, int H, int W, int *tw, int *th, int *td)
{
    // power-of-two box with 128 voxels that wastes the fewest padded voxels; ties go to the widest W extent
    long long best = -1;
    for (int a = 128; a >= 1; a >>= 1)
        for (int b = 128 / a; b >= 1; b >>= 1) {
            const int c = 128 / (a * b);
            const long long pad = (long long)((W + a - 1) / a * a) * ((H + b - 1) / b * b) * ((D + c - 1) / c * c);
            if (best < 0 || pad < best) { best = pad; *tw = a; *th = b; *td = c; }
        }
}

template <int KC, int BN>
lamp_status_t launch(const CUtensorMap &mx, const CUtensorMap &mw, const UmmaParams &P, cudaStream_t st)
{
    using L = SmemLayout<KC, BN>;
    static bool attr = false;
    if (!attr) {
        LAMP_CUDA_OK(cudaFuncSetAttribute(conv3_umma_kernel<KC, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL));
        attr = true;
    }
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int grid = P.total_tiles < sms ? P.total_tiles : sms;
    conv3_umma_kernel<KC, BN><<<grid, NUM_THREADS, L::TOTAL, st>>>(mx, mw, P);
    return launch_status();
}

template <int KC>
lamp_status_t launch_bn(int bn, const CUtensorMap &mx, const CUtensorMap &mw, const UmmaParams &P, cudaStream_t st)
{
    switch (bn) {
    case 16:  return launch<KC, 16>(mx, mw, P, st);
    case 32:  return launch<KC, 32>(mx, mw, P, st);
    case 64:  return launch<KC, 64>(mx, mw, P, st);
    case 128: return launch<KC, 128>(mx, mw, P, st);
    case 256: return launch<KC, 256>(mx, mw, P, st);
    }
    return LAMP_ERR_UNSUPPORTED;
}

}  // namespace

bool umma_conv_fwd_supported(const ConvGeom &g, const TView &x, const TView &y)
{
    if (!(g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed)) return false;
    if (g.ci % 32 || g.co % 16) return false;
    if (!bn_instantiated(pick_bn(g.co))) return false;
    if (x.pitch % 8 || ((uintptr_t)x.p & 15)) return false;
    if (y.f32 ? (y.pitch % 4 != 0) : (y.pitch % 8 != 0)) return false;
    if ((uintptr_t)y.p & 15) return false;
    return true;
}

size_t umma_dgrad_ws(const ConvGeom &g) { return align_up((size_t)27 * g.co * g.ci * sizeof(bf16), 256); }

lamp_status_t umma_transpose_weights(const bf16 *w, bf16 *wt, int taps, int co, int ci, cudaStream_t st)
{
    const int64_t total = (int64_t)taps * co * ci;
    transpose_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w, wt, co, ci, total);
    return launch_status();
}

lamp_status_t umma_conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                            double *stats, int mirror_taps, cudaStream_t st)
{
    if ((int64_t)g.n * g.d * g.h * g.w == 0) return LAMP_OK;
    PFN_cuTensorMapEncodeTiled_v12000 encode = get_encode();
    if (!encode) return LAMP_ERR_CUDA;
    const int KC = (g.ci % 64 == 0) ? 64 : 32;
    const int BN = pick_bn(g.co);
    UmmaParams P;
    P.N = g.n; P.D = g.d; P.H = g.h; P.W = g.w;
    pick_tile(g.d, g.h, g.w, &P.tw, &P.th, &P.td);
    P.ntw = (g.w + P.tw - 1) / P.tw; P.nth = (g.h + P.th - 1) / P.th; P.ntd = (g.d + P.td - 1) / P.td;
    P.nct = g.co / BN;
    P.chunks = g.ci / KC;
    const int64_t tiles = (int64_t)g.n * P.ntd * P.nth * P.ntw * P.nct;
    if (tiles > 0x7FFFFFFF) return LAMP_ERR_UNSUPPORTED;
    P.total_tiles = (int32_t)tiles;
    P.co = g.co; P.mirror = mirror_taps; P.y_f32 = y.f32; P.y_pitch = y.pitch; P.y = y.p;
    P.bias = bias; P.stats = stats; P.status = status_word_ptr();

    CUtensorMap mx, mw;
    {
        const cuuint64_t dims[5] = {(cuuint64_t)g.ci, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.d, (cuuint64_t)g.n};
        const cuuint64_t strides[4] = {(cuuint64_t)x.pitch * 2, (cuuint64_t)x.pitch * 2 * g.w,
                                       (cuuint64_t)x.pitch * 2 * g.w * g.h, (cuuint64_t)x.pitch * 2 * g.w * g.h * g.d};
        const cuuint32_t box[5] = {(cuuint32_t)KC, (cuuint32_t)P.tw, (cuuint32_t)P.th, (cuuint32_t)P.td, 1};
        const cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (encode(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, x.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    {
        const cuuint64_t dims[3] = {(cuuint64_t)g.ci, (cuuint64_t)g.co, 27};
        const cuuint64_t strides[2] = {(cuuint64_t)g.ci * 2, (cuuint64_t)g.ci * 2 * g.co};
        const cuuint32_t box[3] = {(cuuint32_t)KC, (cuuint32_t)BN, 1};
        const cuuint32_t es[3] = {1, 1, 1};
        if (encode(&mw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void *)w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    return KC == 64 ? launch_bn<64>(BN, mx, mw, P, st) : launch_bn<32>(BN, mx, mw, P, st);
}

}  // namespace lamp
