// Weight gradient of the 3x3x3 stride-1 pad-1 convolution with N = 3 x 64 columns per MMA.
//
//   dw[kd,kh,kw][co][ci] = sum_u dy[u - (kd-1, kh-1, 0)][co] * x[u + (0, 0, kw-1)][ci]
//
// One tcgen05.mma (M = 128, K = 16) holds the tensor pipe for max(76, N/2) cycles, so the plain kernel
// (wgrad_umma.cu, N = c_in) runs a 64-channel layer at 42 % of the full rate.  Here the three kw taps
// sit side by side on N: the B operand is ONE x halo box (10 (w) x 16 (h) voxels x 64 channels, rows =
// voxels, MN-major) read through a descriptor whose three 64-channel blocks are the windows starting
// 0, 1 and 2 rows in (leading-dimension offset = one row, 8-voxel groups 10 rows apart).  N = 192 costs
// 96 cycles: the full rate.  The A operand is a window of a dy halo box (8 (w) x 18 (h) voxels of plane
// d + 1 - kd): it starts (2 - kh) lines in.  For c_out = 32 the 128 rows hold four windows one line apart (three kh
// taps per MMA).  For c_out = 64 they hold ANY two of the nine (kd, kh) taps: the second 64-row block is reached
// through the descriptor's block stride, which may lead into the dy box of the neighbouring plane (both boxes sit
// in the same stage), so nine taps take five M blocks instead of six.  Out-of-volume voxels are zero-filled by TMA (the
// conv's zero padding).  The swizzle is a function of the shared-memory address bits, so windows that
// start off the swizzle-atom boundary read exactly what TMA wrote.
//
// A CTA keeps two accumulators (128 x 192 fp32 each, one MMA-issuing thread each) in TMEM while it sweeps its share of the
// 8 x 16-voxel tiles (split-K over CTAs); partial sums go to scratch and are added in a fixed order.
#include <cuda.h>
#include <cudaTypedefs.h>
#include "common.cuh"
#include "umma_ptx.cuh"

namespace lamp {

namespace {

using namespace ptx;

constexpr int WW_THREADS = 224;
constexpr int TWW = 8, THH = 16;                   // tile: 8 (w) x 16 (h) voxels of one plane = K = 128
constexpr int XW = TWW + 2;                        // x box: w halo only
constexpr int DYH = THH + 2;                       // dy box: h halo only
constexpr int MAX_ST = 5;

struct WwParams {
    int32_t N, D, H, W;
    int32_t nwt, nht, ntiles;
    int32_t co, ci;
    int32_t cob;             // c_out channels per window inside an M block: min(co, 128)
    int32_t nmb;             // M blocks: 3 kd x (per-kd blocks) x (co / 128 or 1)
    int32_t mb_per_kd;       // cob = 128: 3 * (co / 128); cob = 64: 2; cob = 32: 1
    int32_t ncx;             // c_in chunks (of 64, or one of 32)
    int32_t pair_cx;         // 1: a set = one M block x two c_in chunks; 0: a set = two M blocks x the one chunk
    int32_t nsets, nsplit, nunits;
    int32_t nsplit_last;     // CTAs that share the LAST set (fewer where that set has one live accumulator: half the work per tile)
    int32_t nst;             // pipeline stages
    int32_t ndy;             // dy buffers per stage (2 where the two accumulators of a set can need different planes)
    int32_t dy_bytes, x_bytes, stage_bytes;
    int64_t entries;
    float  *part;
    int    *status;
};

// kd, ls0: plane tap and first line of the M block's first window.  c_out = 64 pairs any two of the nine (kd, kh)
// taps on the 128 rows: the second 64-row block is the window (kdB, lineB), which may lie in ANOTHER plane's dy box
// (reached through the descriptor's block stride); validB says whether it carries a tap at all.
struct Acc { int kd, ls0, nvalid, cc, cx; bool live; int kdB, lineB, validB; };

// accumulator a (0 or 1) of a set
__device__ __forceinline__ Acc decode_acc(const WwParams &P, int set, int a)
{
    Acc r;
    int mb, cx;
    if (P.pair_cx) { mb = set / (P.ncx / 2); cx = (set % (P.ncx / 2)) * 2 + a; }
    else           { mb = set * 2 + a; cx = 0; }
    r.live = mb < P.nmb;
    if (!r.live) mb = P.nmb - 1;
    r.cx = cx;
    r.kdB = 0; r.lineB = 0; r.validB = 0;
    if (P.cob == 64) {
        // five M blocks for nine taps (line = 2 - kh): (kd0: kh1, kh0) (kd0 kh2 | kd1 kh0) (kd1: kh2, kh1) (kd2: kh1, kh0) (kd2 kh2 | -)
        const int kdA[5] = {0, 0, 1, 2, 2}, lnA[5] = {1, 0, 0, 1, 0}, kdB[5] = {0, 1, 1, 2, 2}, lnB[5] = {2, 2, 1, 2, 1};
        r.cc = 0; r.kd = kdA[mb]; r.ls0 = lnA[mb]; r.kdB = kdB[mb]; r.lineB = lnB[mb]; r.validB = mb != 4;
        r.nvalid = r.validB ? 2 : 1;
        return r;
    }
    r.kd = mb / P.mb_per_kd;
    const int j = mb % P.mb_per_kd;
    if (P.cob >= 128)     { const int kh = j % 3; r.cc = j / 3; r.ls0 = 2 - kh; r.nvalid = 1; }
    else if (P.cob == 64) { r.cc = 0; r.ls0 = j == 0 ? 1 : 0; r.nvalid = j == 0 ? 2 : 1; }
    else                  { r.cc = 0; r.ls0 = 0; r.nvalid = 3; }
    return r;
}

// CBA / CBB: channels per TMA box of dy / x (64: 128-byte swizzle, 32: 64-byte swizzle)
template <int CBA, int CBB>
__global__ void __launch_bounds__(WW_THREADS, 1)
wgrad_win_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_dy, const WwParams P)
{
    constexpr uint32_t SWA = CBA == 64 ? 2u : 4u, SWB = CBB == 64 ? 2u : 4u;
    constexpr uint32_t ROWA = CBA * 2, ROWB = CBB * 2;
    constexpr uint32_t LINE_A = TWW * ROWA;                     // one h-line of the dy box = one 8-row group
    constexpr uint32_t DYBOX = TWW * DYH * ROWA, XBOX = XW * THH * ROWB;
    constexpr int NCOL = 3 * CBB;                               // 192 or 96
    constexpr uint32_t IDESC = make_idesc(NCOL, 1, 1);
    constexpr int ACC_COLS = 256;                               // TMEM column stride between the two accumulators

    extern __shared__ uint8_t smem_raw[];
    // aligned by offsetting the shared array itself, so that the compiler still sees shared-memory pointers
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t *bars = (uint64_t *)(smem + (size_t)P.nst * P.stage_bytes);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + MAX_ST);
    const uint32_t done_bar = smem_u32(bars + 2 * MAX_ST), drained_bar = smem_u32(bars + 2 * MAX_ST + 1);
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * MAX_ST + 2);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        // (each of the two accumulators has its own issuing thread: a stage is free, and a unit done, after both)
        for (int s = 0; s < MAX_ST; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 2); }
        mbar_init(done_bar, 2);
        mbar_init(drained_bar, 4);
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    pdl_wait();                 // everything above touched shared and tensor memory only
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int aboxes = P.cob >= 128 ? 2 : 1;                    // dy boxes per plane (64 channels each, or one of 32)

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------------------- TMA producer
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int unit = blockIdx.x; unit < P.nunits && ok; unit += gridDim.x) {
                const int full = (P.nsets - 1) * P.nsplit;
                const int set = unit < full ? unit / P.nsplit : P.nsets - 1, split = unit < full ? unit % P.nsplit : unit - full;
                const int stride = unit < full ? P.nsplit : P.nsplit_last;
                const Acc a0 = decode_acc(P, set, 0), a1 = decode_acc(P, set, 1);
                // c_out = 64: the set's dy planes: the first block's plane of accumulator 0, and the one other plane any of
                // the set's blocks uses (at most one)
                int kd_other = -1;
                if (P.cob == 64) {
                    const int cand[3] = {a0.validB ? a0.kdB : a0.kd, a1.live ? a1.kd : a0.kd, (a1.live && a1.validB) ? a1.kdB : a0.kd};
                    for (int i = 0; i < 3; ++i) if (cand[i] != a0.kd) kd_other = cand[i];
                }
                const bool two_dy = P.cob == 64 ? kd_other >= 0 : (P.ndy == 2 && (a1.kd != a0.kd || a1.cc != a0.cc));
                const bool two_x = P.pair_cx;
                const uint32_t bytes = (two_dy ? 2 : 1) * aboxes * DYBOX + (two_x ? 2 : 1) * XBOX;
                for (int tile = split; tile < P.ntiles && ok; tile += stride) {
                    int t = tile;
                    const int w0 = (t % P.nwt) * TWW; t /= P.nwt;
                    const int h0 = (t % P.nht) * THH; t /= P.nht;
                    const int d = t % P.D;
                    const int n = t / P.D;
                    if (!mbar_wait(empty0 + 8 * st, ph ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(full0 + 8 * st, bytes);
                    const uint32_t sb = smem_u32(smem + (size_t)st * P.stage_bytes);
                    for (int q = 0; q < (two_dy ? 2 : 1); ++q) {
                        const Acc &a = q ? a1 : a0;
                        const int kd = P.cob == 64 ? (q ? kd_other : a0.kd) : a.kd;
                        for (int b = 0; b < aboxes; ++b)
                            tma_load_5d(sb + q * P.dy_bytes + b * DYBOX, &map_dy, full0 + 8 * st, a.cc * 128 + b * 64, w0, h0 - 1,
                                        d + 1 - kd, n);
                    }
                    for (int q = 0; q < (two_x ? 2 : 1); ++q)
                        tma_load_5d(sb + P.ndy * P.dy_bytes + q * P.x_bytes, &map_x, full0 + 8 * st, (q ? a1.cx : a0.cx) * CBB, w0 - 1, h0, d, n);
                    if (++st == P.nst) { st = 0; ph ^= 1; }
                }
            }
        }
    } else if (warp == 1 || warp == 6) {
        if (lane == 0) {
            // ---------------------------------------------------------------- MMA issuers: warp 1 -> accumulator 0, warp 6 -> 1
            // One thread cannot issue faster than about one tcgen05.mma per 60-100 cycles (waits, descriptors and
            // commits included); with N = 96 (32 input channels) the pipe needs an instruction every 48 cycles, and a
            // single issuer left it idle more than half of the time.  Two threads, one accumulator each.
            const int q = warp == 1 ? 0 : 1;
            int st = 0;
            uint32_t ph = 0, uph = 0;
            bool ok = true;
            for (int unit = blockIdx.x; unit < P.nunits && ok; unit += gridDim.x) {
                const int full = (P.nsets - 1) * P.nsplit;
                const int set = unit < full ? unit / P.nsplit : P.nsets - 1, split = unit < full ? unit % P.nsplit : unit - full;
                const int stride = unit < full ? P.nsplit : P.nsplit_last;
                const Acc a0 = decode_acc(P, set, 0), a1 = decode_acc(P, set, 1);
                const bool two_dy = P.ndy == 2 && (a1.kd != a0.kd || a1.cc != a0.cc);      // (c_out = 64 has its own buffer rule below)
                if (!mbar_wait(drained_bar, uph ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                uint32_t accumulate = 0;
                for (int tile = split; tile < P.ntiles && ok; tile += stride) {
                    if (!mbar_wait(full0 + 8 * st, ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sb = smem_u32(smem + (size_t)st * P.stage_bytes);
                    {
                        const Acc &a = q ? a1 : a0;
                        if (!a.live) { mbar_arrive(empty0 + 8 * st); if (++st == P.nst) { st = 0; ph ^= 1; } accumulate = 1; continue; }
                        // c_out = 64: plane buffer 0 holds accumulator 0's first plane, buffer 1 the set's other plane
                        const int bufA = (P.cob == 64) ? (a.kd != a0.kd) : ((q && two_dy) ? 1 : 0);
                        const int bufB = (P.cob == 64) ? (a.kdB != a0.kd) : bufA;
                        const uint32_t dyb = sb + bufA * P.dy_bytes + a.ls0 * LINE_A;
                        const uint32_t lbo64 = (uint32_t)((bufB - bufA) * P.dy_bytes + (a.lineB - a.ls0) * (int)LINE_A);
                        const uint32_t xb = sb + P.ndy * P.dy_bytes + ((q && P.pair_cx) ? P.x_bytes : 0);
                        // A: blocks of 64 (32) rows = c_out channels of one window; next block = next 64 channels of
                        // the same window (cob = 128: next box) or the window one line further down (cob < 128)
                        const uint64_t da = make_desc(dyb, P.cob >= 128 ? DYBOX : (P.cob == 64 ? lbo64 : LINE_A), LINE_A, SWA);
                        // B: three blocks = the windows kw = 0, 1, 2 (one row apart); 8-voxel groups 10 rows apart
                        const uint64_t db = make_desc(xb, ROWB, XW * ROWB, SWB);
                        const uint32_t d_tmem = tmem_base + q * ACC_COLS;
#pragma unroll
                        for (int j = 0; j < 8; ++j)     // 16 voxels = two h-lines per MMA
                            umma_bf16(d_tmem, da + (uint64_t)(j * ((2 * LINE_A) >> 4)), db + (uint64_t)(j * ((2 * XW * ROWB) >> 4)), IDESC,
                                      (accumulate | j) ? 1u : 0u);
                    }
                    umma_commit(empty0 + 8 * st);
                    if (++st == P.nst) { st = 0; ph ^= 1; }
                    accumulate = 1;
                }
                if (!ok) break;
                if ((q ? a1 : a0).live) umma_commit(done_bar); else mbar_arrive(done_bar);
                uph ^= 1;
            }
        }
    } else {
        // -------------------------------------------------------------------- epilogue (warps 2..5)
        const int q4 = warp & 3;
        uint32_t uph = 0;
        bool ok = true;
        for (int unit = blockIdx.x; unit < P.nunits && ok; unit += gridDim.x) {
            const int full = (P.nsets - 1) * P.nsplit;
            const int set = unit < full ? unit / P.nsplit : P.nsets - 1, split = unit < full ? unit % P.nsplit : unit - full;
            ok = __all_sync(0xffffffffu, mbar_wait(done_bar, uph, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const int m = q4 * 32 + lane;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const Acc a = decode_acc(P, set, q);
                const int rows_per_win = P.cob >= 128 ? 128 : P.cob;
                const int b = m / rows_per_win;                     // window index inside the M block
                const int kh = P.cob == 64 ? (b ? 2 - a.lineB : 2 - a.ls0) : 2 - (a.ls0 + b);
                const int kd_row = (P.cob == 64 && b) ? a.kdB : a.kd;
                const bool row_ok = a.live && b < a.nvalid;
                const int co = a.cc * 128 + m % rows_per_win;
                const uint32_t trow = tmem_base + ((uint32_t)(q4 * 32) << 16) + q * ACC_COLS;
#pragma unroll
                for (int c0 = 0; c0 < NCOL; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(trow + c0, r);
                    tmem_ld_wait();
                    if (row_ok) {
                        const int kw = c0 / CBB, ci = a.cx * CBB + c0 % CBB;
                        const int tap = (kd_row * 3 + kh) * 3 + kw;
                        float4 *d4 = reinterpret_cast<float4 *>(P.part + (int64_t)split * P.entries +
                                                                ((int64_t)tap * P.co + co) * P.ci + ci);
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
        tmem_dealloc(tmem_base, 512);
    }
}

PFN_cuTensorMapEncodeTiled_v12000 get_encode() { return (PFN_cuTensorMapEncodeTiled_v12000)tensor_map_encoder(); }

bool encode_box(PFN_cuTensorMapEncodeTiled_v12000 encode, CUtensorMap *m, const TView &t, int box_c, int bw, int bh)
{
    const cuuint64_t dims[5] = {(cuuint64_t)t.c, (cuuint64_t)t.w, (cuuint64_t)t.h, (cuuint64_t)t.d, (cuuint64_t)t.n};
    const cuuint64_t strides[4] = {(cuuint64_t)t.pitch * 2, (cuuint64_t)t.pitch * 2 * t.w, (cuuint64_t)t.pitch * 2 * t.w * t.h,
                                   (cuuint64_t)t.pitch * 2 * t.w * t.h * t.d};
    const cuuint32_t box[5] = {(cuuint32_t)box_c, (cuuint32_t)bw, (cuuint32_t)bh, 1, 1};
    const cuuint32_t es[5] = {1, 1, 1, 1, 1};
    return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, t.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  box_c == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct WwPlan { WwParams P; int CBA, CBB; size_t smem; int grid; };

bool make_ww_plan(const ConvGeom &g, WwPlan *out)
{
    if (!(g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed)) return false;
    if (!(g.co == 32 || g.co == 64 || g.co % 128 == 0)) return false;
    int ncx, CBB;
    if (g.ci == 32) { ncx = 1; CBB = 32; }
    else if (g.ci == 64) { ncx = 1; CBB = 64; }
    else if (g.ci % 128 == 0) { ncx = g.ci / 64; CBB = 64; }
    else return false;
    // the fixed 8 x 16 tile must not be mostly padding (small or thin volumes go to the plain kernel)
    const int nwt = (g.w + TWW - 1) / TWW, nht = (g.h + THH - 1) / THH;
    if ((double)g.h * g.w < 0.6 * (double)nwt * TWW * nht * THH) return false;
    WwParams &P = out->P;
    P.N = g.n; P.D = g.d; P.H = g.h; P.W = g.w;
    P.nwt = nwt; P.nht = nht;
    const int64_t nt = (int64_t)g.n * g.d * nht * nwt;
    if (nt > 0x7FFFFFFF || nt <= 0) return false;
    P.ntiles = (int32_t)nt;
    P.co = g.co; P.ci = g.ci;
    P.cob = g.co < 128 ? g.co : 128;
    P.mb_per_kd = P.cob >= 128 ? 3 * (g.co / 128) : (P.cob == 64 ? 2 : 1);
    P.nmb = P.cob == 64 ? 5 : 3 * P.mb_per_kd;       // c_out = 64: nine taps in five blocks of two (decode_acc)
    P.ncx = ncx;
    P.pair_cx = ncx >= 2;
    P.nsets = P.pair_cx ? P.nmb * (ncx / 2) : (P.nmb + 1) / 2;
    const int CBA = g.co == 32 ? 32 : 64;
    const int aboxes = P.cob >= 128 ? 2 : 1;
    // one extra h-line behind the dy box: the fourth (unused) window of a 32-channel block reads it
    P.dy_bytes = (int)align_up((size_t)aboxes * TWW * DYH * CBA * 2 + TWW * CBA * 2, 1024);
    P.x_bytes = (int)align_up((size_t)XW * THH * CBB * 2, 1024);
    P.ndy = P.cob == 64 ? 2 : ((P.pair_cx || P.mb_per_kd % 2 == 0) ? 1 : 2);
    P.stage_bytes = P.ndy * P.dy_bytes + (P.pair_cx ? 2 : 1) * P.x_bytes;
    const int budget = 227 * 1024 - 1024 - 1024;
    int nst = budget / P.stage_bytes;
    if (nst > MAX_ST) nst = MAX_ST;
    if (nst < 2) return false;
    P.nst = nst;
    const int sms = sm_count();
    int nsplit = sms / P.nsets;
    if (nsplit < 1) nsplit = 1;
    if (nsplit > P.ntiles) nsplit = P.ntiles;
    P.nsplit = nsplit;
    P.nsplit_last = nsplit;
    // (32 output channels: three M blocks in two sets, the second with one live accumulator.  Giving that set a third
    // instead of half of the CTAs made the pass SLOWER, 782 -> 628 TFLOP/s: at this width a tile's time is set by its
    // loads and barrier round trips, not by its MMAs, so both kinds of set take the same time per tile.)
    // 64 output channels, one c_in chunk: five M blocks in three sets, the last with one live accumulator (2 : 2 : 1)
    if (P.cob == 64 && P.nsets == 3 && !P.pair_cx && sms >= 5 && P.ntiles >= sms) {
        P.nsplit = sms * 2 / 5;
        P.nsplit_last = sms - 2 * P.nsplit;
    }
    P.nunits = (P.nsets - 1) * P.nsplit + P.nsplit_last;
    P.entries = (int64_t)27 * g.co * g.ci;
    out->CBA = CBA; out->CBB = CBB;
    out->smem = 1024 + (size_t)nst * P.stage_bytes + 1024;
    out->grid = P.nunits < sms ? P.nunits : sms;
    return true;
}

template <int CBA, int CBB>
lamp_status_t launch_ww(const CUtensorMap &mx, const CUtensorMap &mdy, const WwPlan &pl, cudaStream_t st)
{
    static SmemAttrOnce attr;
    { const lamp_status_t as = attr.ensure(wgrad_win_kernel<CBA, CBB>, (int)(227 * 1024)); if (as != LAMP_OK) return as; }
    const lamp_status_t ls = launch_pdl((int64_t)pl.P.ntiles * pl.P.nsets <= 64 * (int64_t)pl.grid, wgrad_win_kernel<CBA, CBB>, dim3(pl.grid), dim3(WW_THREADS), pl.smem, st, mx, mdy, pl.P);
    if (ls != LAMP_OK) return ls;
    return launch_status();
}

}  // namespace

bool win_wgrad_supported(const ConvGeom &g, const TView &x, const TView &dy)
{
    WwPlan pl;
    if ((int64_t)g.n * g.d * g.h * g.w == 0) return false;
    if (!make_ww_plan(g, &pl)) return false;
    if (x.pitch % 8 || dy.pitch % 8 || ((uintptr_t)x.p & 15) || ((uintptr_t)dy.p & 15)) return false;
    return true;
}

size_t win_wgrad_ws(const ConvGeom &g)
{
    WwPlan pl;
    if (!make_ww_plan(g, &pl)) return 0;
    return align_up((size_t)pl.P.nsplit * pl.P.entries * sizeof(float), 256);
}

lamp_status_t win_wgrad(const ConvGeom &g, const TView &x, const TView &dy, float *dw, void *ws, size_t ws_bytes,
                        cudaStream_t st)
{
    WwPlan pl;
    if (!make_ww_plan(g, &pl)) return LAMP_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < win_wgrad_ws(g)) return LAMP_ERR_WORKSPACE;
    PFN_cuTensorMapEncodeTiled_v12000 encode = get_encode();
    if (!encode) return LAMP_ERR_CUDA;
    const bool direct = pl.P.nsplit == 1;
    pl.P.part = direct ? dw : (float *)ws;
    if (pl.P.nsplit_last < pl.P.nsplit) {
        // the last set (c_out = 64: tap (kd 2, kh 2), entries [24, 27) x c_out x c_in) writes fewer partial slices than the
        // reduction adds: the slices it does not write are zero
        const size_t tap_bytes = (size_t)g.co * g.ci * sizeof(float);
        const int first_tap = 24;
        LAMP_CUDA_OK(cudaMemset2DAsync((char *)pl.P.part + (size_t)pl.P.nsplit_last * pl.P.entries * sizeof(float) + first_tap * tap_bytes,
                                       (size_t)pl.P.entries * sizeof(float), 0, (27 - first_tap) * tap_bytes,
                                       (size_t)(pl.P.nsplit - pl.P.nsplit_last), st));
    }
    pl.P.status = status_word_ptr();
    CUtensorMap mx, mdy;
    if (!encode_box(encode, &mx, x, pl.CBB, XW, THH)) return LAMP_ERR_CUDA;
    if (!encode_box(encode, &mdy, dy, pl.CBA, TWW, DYH)) return LAMP_ERR_CUDA;
    lamp_status_t s;
    if (pl.CBA == 64 && pl.CBB == 64) s = launch_ww<64, 64>(mx, mdy, pl, st);
    else if (pl.CBA == 64 && pl.CBB == 32) s = launch_ww<64, 32>(mx, mdy, pl, st);
    else if (pl.CBA == 32 && pl.CBB == 64) s = launch_ww<32, 64>(mx, mdy, pl, st);
    else s = launch_ww<32, 32>(mx, mdy, pl, st);
    if (s != LAMP_OK || direct) return s;
    return reduce_partials(pl.P.part, pl.P.entries, pl.P.nsplit, dw, st);
}

}  // namespace lamp
