// Weight gradients on the sm_100a tensor cores.
//
//   3x3x3 s1 p1 :  dw[tap][co][ci] = sum_u dy[u - off(tap)][co] * x[u][ci]
//   3x3x3 s2 p1 :  dw[tap][co][ci] = sum_o dy[o][co] * x[2 o + off(tap)][ci]
//   2x2x2 s2 T  :  dw[tap][co][ci] = sum_j dy[2 j + tap][co] * x[j][ci]
//
// In each case one tensor is read at the tile's own voxels ("fixed", F) and the other at per-tap shifted
// (and possibly stride-2) voxels ("moving", G).  GEMM view per tap: D[G channels x F channels] = G_tap^T * F with
// the reduction over voxels.  Both operands are read straight from the NDHWC tensors, i.e. with the
// reduction (voxel) index as the shared-memory row and the channels contiguous: "MN-major" operands of
// tcgen05.mma.  A voxel tile (tw x th x td = 128 voxels) is one K = 128 slab: the F tile is loaded once,
// the G tile once per tap, at scale * j + shift(tap), out-of-volume voxels zero-filled by TMA (the
// conv's zero padding); a stride-2 G tile is fetched by a TMA box with element stride 2.
//
// M = 128 accumulator rows hold 128 G channels of one tap, two taps x 64 channels or four taps x 32
// channels; N = min(F channels, 256) columns.  The fp32 accumulators of up to 512 / N such blocks stay in
// TMEM while the CTA sweeps its share of the voxel tiles (split-K over CTAs); each CTA then writes its
// partial sums and a second kernel adds the partials in a fixed order (transposing where G is x), so
// the result does not depend on scheduling.
#include <cuda.h>
#include <cudaTypedefs.h>
#include "common.cuh"
#include "umma_ptx.cuh"

namespace lamp {

namespace {

using namespace ptx;

struct WgParams {
    int32_t N, D, H, W;
    int32_t tw, th, td, ntw, nth, ntd, ntiles;
    int32_t co, ci;          // channels of the moving tensor G (M side) and of the fixed tensor F (N side)
    int32_t ntaps;           // 27 or 8
    int32_t g_scale;         // G voxel = g_scale * j + shift(tap)
    int8_t  sd[27], sh[27], sw[27];
    int32_t co_blk;          // G channels per tap inside an M block: min(co, 128)
    int32_t tpm;             // taps per M block: 128 / co_blk
    int32_t co_chunks;       // co / co_blk
    int32_t MB;              // M blocks: ceil(ntaps / tpm) * co_chunks
    int32_t nchunks;         // ci / NC
    int32_t sps;             // accumulator slots per set (512 / NC, at most MB)
    int32_t sets_per_chunk;  // ceil(MB / sps)
    int32_t nsets, nsplit, nunits;
    int64_t entries;         // ntaps * co * ci
    float  *part;            // [nsplit][entries]
    int    *status;
};

constexpr int WG_THREADS = 192;
constexpr int A_STAGE_BYTES = 128 * 128 * 2;      // one M block: 128 voxels x 128 channel-rows of dy

template <int NC>
struct WgSmem {
    static constexpr int X_BYTES = 128 * NC * 2;
    static constexpr int NX = 2;
    static constexpr int CTRL = 1024;
    static constexpr int AVAIL = 227 * 1024 - 1024 - CTRL - NX * X_BYTES;
    static constexpr int NA = (AVAIL / A_STAGE_BYTES) < 6 ? (AVAIL / A_STAGE_BYTES) : 6;
    static constexpr int TOTAL = 1024 + NX * X_BYTES + NA * A_STAGE_BYTES + CTRL;
    static constexpr int TMEM_COLS = 512;
};

// BOXA / BOXB: channels per TMA box of dy / x (64 -> 128-byte swizzle, 32 -> 64-byte swizzle)
template <int NC, int BOXA, int BOXB>
__global__ void __launch_bounds__(WG_THREADS, 1)
wgrad_umma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_dy, const WgParams P)
{
    using L = WgSmem<NC>;
    constexpr int NA = L::NA, NX = L::NX;
    constexpr uint32_t SWA = BOXA == 64 ? 2u : 4u, SWB = BOXB == 64 ? 2u : 4u;
    constexpr uint32_t BOXA_BYTES = 128 * BOXA * 2, BOXB_BYTES = 128 * BOXB * 2;
    constexpr uint32_t SBO_A = 8 * BOXA * 2, SBO_B = 8 * BOXB * 2;         // 8 voxel rows
    constexpr uint32_t KSTEP_A = 16 * BOXA * 2, KSTEP_B = 16 * BOXB * 2;   // 16 voxel rows per MMA
    constexpr uint32_t IDESC = make_idesc(NC, 1, 1);
    constexpr int ABOXES = 128 / BOXA, XBOXES = NC / BOXB;

    extern __shared__ uint8_t smem_raw[];
    // aligned by offsetting the shared array itself, so that the compiler still sees shared-memory pointers
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *xs_base = smem;
    uint8_t *as_base = smem + NX * L::X_BYTES;
    uint64_t *bars = (uint64_t *)(as_base + NA * A_STAGE_BYTES);
    // xfull[2] xempty[2] afull[8] aempty[8] done drained
    const uint32_t xfull0 = smem_u32(bars), xempty0 = smem_u32(bars + 2);
    const uint32_t afull0 = smem_u32(bars + 4), aempty0 = smem_u32(bars + 12);
    const uint32_t done_bar = smem_u32(bars + 20), drained_bar = smem_u32(bars + 21);
    uint32_t *tmem_slot = (uint32_t *)(bars + 22);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < NX; ++s) { mbar_init(xfull0 + 8 * s, 1); mbar_init(xempty0 + 8 * s, 1); }
        for (int s = 0; s < NA; ++s) { mbar_init(afull0 + 8 * s, 1); mbar_init(aempty0 + 8 * s, 1); }
        mbar_init(done_bar, 1);
        mbar_init(drained_bar, 4);
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), L::TMEM_COLS);
    pdl_wait();                 // everything above touched shared and tensor memory only
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------------------- TMA producer
            int xs = 0, as = 0;
            uint32_t xph = 0, aph = 0;
            bool ok = true;
            for (int unit = blockIdx.x; unit < P.nunits && ok; unit += gridDim.x) {
                const int set = unit / P.nsplit, split = unit - set * P.nsplit;
                const int ncx = set / P.sets_per_chunk, sidx = set - ncx * P.sets_per_chunk;
                const int mb0 = sidx * P.sps, mb1 = min(P.MB, mb0 + P.sps);
                for (int tile = split; tile < P.ntiles && ok; tile += P.nsplit) {
                    int t = tile;
                    const int wt = t % P.ntw; t /= P.ntw;
                    const int ht = t % P.nth; t /= P.nth;
                    const int dt = t % P.ntd;
                    const int n = t / P.ntd;
                    const int w0 = wt * P.tw, h0 = ht * P.th, d0 = dt * P.td;
                    if (!mbar_wait(xempty0 + 8 * xs, xph ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(xfull0 + 8 * xs, L::X_BYTES);
                    const uint32_t xsm = smem_u32(xs_base + xs * L::X_BYTES);
#pragma unroll
                    for (int j = 0; j < XBOXES; ++j)
                        tma_load_5d(xsm + j * BOXB_BYTES, &map_x, xfull0 + 8 * xs, ncx * NC + j * BOXB, w0, h0, d0, n);
                    if (++xs == NX) { xs = 0; xph ^= 1; }
                    for (int mb = mb0; mb < mb1; ++mb) {
                        const int tg = mb / P.co_chunks, cc = mb - tg * P.co_chunks;
                        if (!mbar_wait(aempty0 + 8 * as, aph ^ 1, abort_flag)) { ok = false; break; }
                        int nvalid = 0;
#pragma unroll
                        for (int b = 0; b < ABOXES; ++b)
                            nvalid += (tg * P.tpm + (b * BOXA) / P.co_blk) < P.ntaps;
                        mbar_expect_tx(afull0 + 8 * as, nvalid * BOXA_BYTES);
                        const uint32_t asm_ = smem_u32(as_base + as * A_STAGE_BYTES);
#pragma unroll
                        for (int b = 0; b < ABOXES; ++b) {
                            const int m0 = b * BOXA;
                            const int tap = tg * P.tpm + m0 / P.co_blk;
                            if (tap < P.ntaps)
                                tma_load_5d(asm_ + b * BOXA_BYTES, &map_dy, afull0 + 8 * as, cc * P.co_blk + m0 % P.co_blk,
                                            P.g_scale * w0 + P.sw[tap], P.g_scale * h0 + P.sh[tap], P.g_scale * d0 + P.sd[tap], n);
                        }
                        if (++as == NA) { as = 0; aph ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------------------------------------------------------- MMA issuer
            int xs = 0, as = 0;
            uint32_t xph = 0, aph = 0, uph = 0;
            bool ok = true;
            for (int unit = blockIdx.x; unit < P.nunits && ok; unit += gridDim.x) {
                const int set = unit / P.nsplit, split = unit - set * P.nsplit;
                const int ncx = set / P.sets_per_chunk, sidx = set - ncx * P.sets_per_chunk;
                const int mb0 = sidx * P.sps, mb1 = min(P.MB, mb0 + P.sps);
                // the previous unit's accumulators must have been read out
                if (!mbar_wait(drained_bar, uph ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                bool first = true;
                for (int tile = split; tile < P.ntiles && ok; tile += P.nsplit) {
                    if (!mbar_wait(xfull0 + 8 * xs, xph, abort_flag)) { ok = false; break; }
                    const uint32_t xsm = smem_u32(xs_base + xs * L::X_BYTES);
                    const uint64_t db = make_desc(xsm, BOXB_BYTES, SBO_B, SWB);
                    for (int mb = mb0; mb < mb1; ++mb) {
                        if (!mbar_wait(afull0 + 8 * as, aph, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t da = make_desc(smem_u32(as_base + as * A_STAGE_BYTES), BOXA_BYTES, SBO_A, SWA);
                        const uint32_t d_tmem = tmem_base + (uint32_t)(mb - mb0) * NC;
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            umma_bf16(d_tmem, da + (uint64_t)(j * (KSTEP_A >> 4)), db + (uint64_t)(j * (KSTEP_B >> 4)), IDESC,
                                      (!first || j > 0) ? 1u : 0u);
                        umma_commit(aempty0 + 8 * as);
                        if (++as == NA) { as = 0; aph ^= 1; }
                    }
                    if (!ok) break;
                    umma_commit(xempty0 + 8 * xs);
                    if (++xs == NX) { xs = 0; xph ^= 1; }
                    first = false;
                }
                if (!ok) break;
                umma_commit(done_bar);
                uph ^= 1;
            }
        }
    } else {
        // -------------------------------------------------------------------- epilogue (warps 2..5)
        const int q = warp & 3;
        uint32_t uph = 0;
        bool ok = true;
        for (int unit = blockIdx.x; unit < P.nunits && ok; unit += gridDim.x) {
            const int set = unit / P.nsplit, split = unit - set * P.nsplit;
            const int ncx = set / P.sets_per_chunk, sidx = set - ncx * P.sets_per_chunk;
            const int mb0 = sidx * P.sps, mb1 = min(P.MB, mb0 + P.sps);
            ok = __all_sync(0xffffffffu, mbar_wait(done_bar, uph, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const int m = q * 32 + lane;
            for (int mb = mb0; mb < mb1; ++mb) {
                const int tg = mb / P.co_chunks, cc = mb - tg * P.co_chunks;
                const int tap = tg * P.tpm + m / P.co_blk;
                const int co = cc * P.co_blk + m % P.co_blk;
                float *dst = P.part + (int64_t)split * P.entries + ((int64_t)tap * P.co + co) * P.ci + ncx * NC;
                const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(mb - mb0) * NC;
#pragma unroll
                for (int c0 = 0; c0 < NC; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(trow + c0, r);
                    tmem_ld_wait();
                    if (tap < P.ntaps) {
                        float4 *d4 = reinterpret_cast<float4 *>(dst + c0);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            d4[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(drained_bar);
            uph ^= 1;
        }
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
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

PFN_cuTensorMapEncodeTiled_v12000 get_encode() { return (PFN_cuTensorMapEncodeTiled_v12000)tensor_map_encoder(); }

void pick_tile128(int D, int H, int W, int *tw, int *th, int *td)
{
    long long best = -1;
    for (int a = 128; a >= 1; a >>= 1)
        for (int b = 128 / a; b >= 1; b >>= 1) {
            const int c = 128 / (a * b);
            const long long pad = (long long)((W + a - 1) / a * a) * ((H + b - 1) / b * b) * ((D + c - 1) / c * c);
            if (best < 0 || pad < best) { best = pad; *tw = a; *th = b; *td = c; }
        }
}

bool encode_act(PFN_cuTensorMapEncodeTiled_v12000 encode, CUtensorMap *m, const TView &t, int box_c, int tw, int th, int td, int scale)
{
    const cuuint32_t s = (cuuint32_t)scale;
    const cuuint64_t dims[5] = {(cuuint64_t)t.c, (cuuint64_t)t.w, (cuuint64_t)t.h, (cuuint64_t)t.d, (cuuint64_t)t.n};
    const cuuint64_t strides[4] = {(cuuint64_t)t.pitch * 2, (cuuint64_t)t.pitch * 2 * t.w, (cuuint64_t)t.pitch * 2 * t.w * t.h,
                                   (cuuint64_t)t.pitch * 2 * t.w * t.h * t.d};
    const cuuint32_t box[5] = {(cuuint32_t)box_c, (cuuint32_t)tw * s, (cuuint32_t)th * s, (cuuint32_t)td * s, 1};
    const cuuint32_t es[5] = {1, s, s, s, 1};
    return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, t.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  box_c == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// out[t][b][a] = sum_s part[s][t][a][b]   (partials were accumulated as [tap][G channel][F channel] with G = x)
__global__ void __launch_bounds__(256)
reduce_transposed_kernel(const float *__restrict__ part, int64_t entries, int splits, int A, int Bc, float *__restrict__ out)
{
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;      // index into out: (t * Bc + b) * A + a
    if (e >= entries) return;
    const int a = (int)(e % A);
    const int b = (int)((e / A) % Bc);
    const int64_t t = e / ((int64_t)A * Bc);
    const int64_t src = (t * A + a) * Bc + b;
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += part[(int64_t)s * entries + src];
    out[e] = acc;
}

struct WgPlan { WgParams P; int NC, BOXA, BOXB; int grid; bool g_is_x; };

// Which tensor moves: s1 and transposed convs shift dy (G = dy, F = x); the stride-2 conv shifts x (G = x, F = dy).
bool make_wg_plan(const ConvGeom &g, WgPlan *out)
{
    const bool s1 = g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed;
    const bool s2 = g.k == 3 && g.s == 2 && g.p == 1 && !g.transposed;
    const bool tr = g.k == 2 && g.s == 2 && g.p == 0 && g.transposed;
    if (!s1 && !s2 && !tr) return false;
    out->g_is_x = s2;
    const int gc = s2 ? g.ci : g.co;                 // channels of G (M side)
    const int fc = s2 ? g.co : g.ci;                 // channels of F (N side)
    if (!(gc == 32 || gc == 64 || gc % 128 == 0)) return false;
    int NC;
    if (fc == 32 || fc == 64 || fc == 128) NC = fc;
    else if (fc % 256 == 0) NC = 256;
    else return false;
    WgParams &P = out->P;
    // the tile grid is F's voxel grid: x for s1 / transposed, dy for the stride-2 conv
    const int fd = s2 ? g.od : g.d, fh = s2 ? g.oh : g.h, fw = s2 ? g.ow : g.w;
    P.N = g.n; P.D = fd; P.H = fh; P.W = fw;
    pick_tile128(fd, fh, fw, &P.tw, &P.th, &P.td);
    P.ntw = (fw + P.tw - 1) / P.tw; P.nth = (fh + P.th - 1) / P.th; P.ntd = (fd + P.td - 1) / P.td;
    const int64_t nt = (int64_t)g.n * P.ntd * P.nth * P.ntw;
    if (nt > 0x7FFFFFFF || nt <= 0) return false;
    P.ntiles = (int32_t)nt;
    P.co = gc; P.ci = fc;
    P.ntaps = g.k * g.k * g.k;
    P.g_scale = s1 ? 1 : 2;
    for (int t = 0; t < P.ntaps; ++t) {
        const int kd = t / (g.k * g.k), kh = (t / g.k) % g.k, kw = t % g.k;
        if (s1)      { P.sd[t] = (int8_t)(1 - kd); P.sh[t] = (int8_t)(1 - kh); P.sw[t] = (int8_t)(1 - kw); }   // dy[u - (k - 1)]
        else if (s2) { P.sd[t] = (int8_t)(kd - 1); P.sh[t] = (int8_t)(kh - 1); P.sw[t] = (int8_t)(kw - 1); }   // x[2 o + k - 1]
        else         { P.sd[t] = (int8_t)kd; P.sh[t] = (int8_t)kh; P.sw[t] = (int8_t)kw; }                     // dy[2 j + tap]
    }
    P.co_blk = gc < 128 ? gc : 128;
    P.tpm = 128 / P.co_blk;
    P.co_chunks = gc / P.co_blk;
    P.MB = (P.ntaps + P.tpm - 1) / P.tpm * P.co_chunks;
    P.nchunks = fc / NC;
    P.sps = 512 / NC < P.MB ? 512 / NC : P.MB;
    P.sets_per_chunk = (P.MB + P.sps - 1) / P.sps;
    P.nsets = P.nchunks * P.sets_per_chunk;
    const int sms = sm_count();
    int nsplit = sms / P.nsets;
    if (nsplit < 1) nsplit = 1;
    if (nsplit > P.ntiles) nsplit = P.ntiles;
    P.nsplit = nsplit;
    P.nunits = P.nsets * nsplit;
    P.entries = (int64_t)P.ntaps * g.co * g.ci;
    out->NC = NC;
    out->BOXA = gc == 32 ? 32 : 64;
    out->BOXB = fc == 32 ? 32 : 64;
    out->grid = P.nunits < sms ? P.nunits : sms;
    return true;
}

template <int NC, int BOXA, int BOXB>
lamp_status_t launch_wg(const CUtensorMap &mx, const CUtensorMap &mdy, const WgPlan &pl, cudaStream_t st)
{
    using L = WgSmem<NC>;
    static SmemAttrOnce attr;
    { const lamp_status_t as = attr.ensure(wgrad_umma_kernel<NC, BOXA, BOXB>, (int)(L::TOTAL)); if (as != LAMP_OK) return as; }
    const lamp_status_t ls = launch_pdl((int64_t)pl.P.ntiles * pl.P.nunits <= 64 * (int64_t)pl.grid * pl.P.nsplit, wgrad_umma_kernel<NC, BOXA, BOXB>, dim3(pl.grid), dim3(WG_THREADS), L::TOTAL, st, mx, mdy, pl.P);
    if (ls != LAMP_OK) return ls;
    return launch_status();
}

}  // namespace

bool umma_wgrad_supported(const ConvGeom &g, const TView &x, const TView &dy)
{
    WgPlan pl;
    if ((int64_t)g.n * g.d * g.h * g.w == 0 || (int64_t)g.od * g.oh * g.ow == 0) return false;
    if (!make_wg_plan(g, &pl)) return false;
    if (x.pitch % 8 || dy.pitch % 8 || ((uintptr_t)x.p & 15) || ((uintptr_t)dy.p & 15)) return false;
    return true;
}

size_t umma_wgrad_ws(const ConvGeom &g)
{
    WgPlan pl;
    if (!make_wg_plan(g, &pl)) return 0;
    return align_up((size_t)pl.P.nsplit * pl.P.entries * sizeof(float), 256);
}

lamp_status_t umma_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, void *ws, size_t ws_bytes,
                         cudaStream_t st)
{
    WgPlan pl;
    if (!make_wg_plan(g, &pl)) return LAMP_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < umma_wgrad_ws(g)) return LAMP_ERR_WORKSPACE;
    PFN_cuTensorMapEncodeTiled_v12000 encode = get_encode();
    if (!encode) return LAMP_ERR_CUDA;
    // a single split needs no second pass: the CTAs write the gradient itself
    const bool direct = pl.P.nsplit == 1 && !pl.g_is_x;
    pl.P.part = direct ? dw : (float *)ws;
    pl.P.status = status_word_ptr();
    CUtensorMap mx, mdy;
    // first map = fixed tensor F (N side), second = moving tensor G (M side)
    const TView &F = pl.g_is_x ? dy : x, &G = pl.g_is_x ? x : dy;
    if (!encode_act(encode, &mx, F, pl.BOXB, pl.P.tw, pl.P.th, pl.P.td, 1)) return LAMP_ERR_CUDA;
    if (!encode_act(encode, &mdy, G, pl.BOXA, pl.P.tw, pl.P.th, pl.P.td, pl.P.g_scale)) return LAMP_ERR_CUDA;
    lamp_status_t s = LAMP_ERR_UNSUPPORTED;
    const int key = pl.NC * 10000 + pl.BOXA * 100 + pl.BOXB;
    switch (key) {
    case 32 * 10000 + 32 * 100 + 32:  s = launch_wg<32, 32, 32>(mx, mdy, pl, st); break;
    case 32 * 10000 + 64 * 100 + 32:  s = launch_wg<32, 64, 32>(mx, mdy, pl, st); break;
    case 64 * 10000 + 32 * 100 + 64:  s = launch_wg<64, 32, 64>(mx, mdy, pl, st); break;
    case 64 * 10000 + 64 * 100 + 64:  s = launch_wg<64, 64, 64>(mx, mdy, pl, st); break;
    case 128 * 10000 + 32 * 100 + 64: s = launch_wg<128, 32, 64>(mx, mdy, pl, st); break;
    case 128 * 10000 + 64 * 100 + 64: s = launch_wg<128, 64, 64>(mx, mdy, pl, st); break;
    case 256 * 10000 + 32 * 100 + 64: s = launch_wg<256, 32, 64>(mx, mdy, pl, st); break;
    case 256 * 10000 + 64 * 100 + 64: s = launch_wg<256, 64, 64>(mx, mdy, pl, st); break;
    }
    if (s != LAMP_OK || direct) return s;
    if (!pl.g_is_x) return reduce_partials(pl.P.part, pl.P.entries, pl.P.nsplit, dw, st);
    // partials are [tap][c_in][c_out]; dw is [tap][c_out][c_in]
    const int taps = g.k * g.k * g.k;
    if (transpose_sum_supported(taps, g.ci, g.co)) return transpose_sum_f32(pl.P.part, taps, g.ci, g.co, pl.P.nsplit, dw, st);
    reduce_transposed_kernel<<<(unsigned)((pl.P.entries + 255) / 256), 256, 0, st>>>(pl.P.part, pl.P.entries, pl.P.nsplit, g.ci, g.co, dw);
    return launch_status();
}

}  // namespace lamp
