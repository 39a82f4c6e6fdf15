// Convolution passes as an implicit GEMM on the sm_100a tensor cores, "voxels x channels" form:
//   M = 128 output points (a tw x th x td box), N = output-channel tile (<= 256), K = taps x input channels.
//
// One kernel serves every pass whose result at a point j is a sum over taps of a [c_in]-vector read at
// (in_scale * j + shift(tap)) times a [c_out x c_in] weight tile:
//   3x3x3 s1 p1 forward            27 taps, shift k-1                      (c_out >= 256; narrower: conv_t.cu)
//   3x3x3 s1 p1 data gradient      the same on dy with taps mirrored, weights transposed
//   3x3x3 s2 p1 forward            27 taps, in_scale 2: the TMA box walks the input with element stride 2
//   3x3x3 s2 p1 data gradient      8 parity classes of dx (i = 2j + parity), 1..8 taps each, written with stride 2
//   2x2x2 s2 transposed forward    8 parity classes of y, one tap each
//   2x2x2 s2 transposed data grad. 8 taps, in_scale 2
// Which taps, shifts and weight tiles a class uses comes from a small table built on the host.
//
// Per CTA (persistent over tiles), warp-specialised:
//   warp 0   : TMA producer.  For each (tap, channel chunk) it loads the A tile - the tw x th x td box of
//              the NDHWC tensor at the tap's shift, out-of-volume voxels zero-filled by the TMA unit,
//              which is exactly the zero padding - and the matching [BN x KC] weight tile, both with
//              the 128-byte (KC = 64) or 64-byte (KC = 32) shared-memory swizzle.
//   warp 1   : allocates TMEM and issues tcgen05.mma (M = 128, N = BN, K = 16 per instruction) from one
//              thread; fp32 accumulators live in TMEM, double-buffered so that the epilogue of tile i
//              overlaps the MMAs of tile i + 1.
//   warps 2-5: epilogue.  tcgen05.ld the accumulator rows (one point per thread), add the bias, reduce
//              the per-channel sum and sum of squares (InstanceNorm statistics), convert and store the
//              row into the output's channel slice.
// Every mbarrier wait is bounded; on expiry the CTA records LAMP_ERR_TIMEOUT and winds down.
#include <cuda.h>
#include <cudaTypedefs.h>
#include "common.cuh"
#include <string.h>
#include "umma_ptx.cuh"

namespace lamp {

namespace {

using namespace ptx;

struct TapTable {                  // per parity class: the taps that contribute, their weight tile and input shift
    int8_t ntaps[8];
    uint32_t tap[8][27];           // one word per tap: bytes (weight tile, shift d, shift h, shift w), shifts signed
};

struct UmmaParams {
    int32_t N, D, H, W;            // batch; extents of the point grid j the tiles cover
    int32_t OD, OH, OW;            // extents of the output tensor
    int32_t in_scale, out_scale;   // input voxel = in_scale * j + shift; output voxel = out_scale * j + class parity
    int32_t nclass;                // 1, or 8 parity classes
    int32_t tw, th, td;            // voxel tile, tw * th * td = 128
    int32_t ntw, nth, ntd;         // tiles per axis
    int32_t nct;                   // c_out tiles
    int32_t ksplit;                // CTAs that share the (tap, chunk) range of one tile; > 1: y is the fp32 partial buffer
    int64_t part_stride;           // voxels between the partial results of consecutive splits
    int32_t chunks;                // c_in / KC
    int32_t total_tiles;
    int32_t step[7];               // the grid size in the tiles' mixed radix (ksplit, nct, ntw, nth, ntd, nclass, N)
    int32_t co;                    // c_out
    int32_t merge_co;              // > 0: the N axis carries (parity class, channel) pairs, class = column / merge_co
    int32_t y_f32;
    int32_t st32;                  // output rows may be written with 32-byte stores (base, pitch and slice offset allow it)
    int64_t y_pitch;
    void   *y;
    const float *bias;
    double *stats;                 // [N][co][2] or NULL
    int    *status;
    // head mode (1x1x1 conv + softmax over the hK <= 16 columns of a row): outputs instead of y
    int32_t hK;
    float *probs;                  // [voxel][hK] or NULL
    uint8_t *amax;                 // [voxel] or NULL
    const uint8_t *labels;         // [voxel], with dice
    double *dice;                  // [n][hK][3] = (sum p at the label, sum p, label count) or NULL
    TapTable taps;
};

struct Tile { int ks, ct, w0, h0, d0, cls, n; };

// A CTA visits tiles blockIdx.x, blockIdx.x + gridDim.x, ...  The tile index is a number in the mixed radix
// (ksplit, nct, ntw, nth, ntd, nclass, N); instead of dividing for every tile the walker divides once and then adds
// the grid size digit by digit (tiles with one short reduction step are otherwise bound by this index arithmetic).
struct TileWalker {
    int dg[7];
    __device__ __forceinline__ void init(const UmmaParams &P, int t)
    {
        dg[0] = t % P.ksplit; t /= P.ksplit;
        dg[1] = t % P.nct; t /= P.nct;
        dg[2] = t % P.ntw; t /= P.ntw;
        dg[3] = t % P.nth; t /= P.nth;
        dg[4] = t % P.ntd; t /= P.ntd;
        dg[5] = t % P.nclass;
        dg[6] = t / P.nclass;
    }
    __device__ __forceinline__ void next(const UmmaParams &P)
    {
        const int radix[6] = {P.ksplit, P.nct, P.ntw, P.nth, P.ntd, P.nclass};
        int carry = 0;
#pragma unroll
        for (int i = 0; i < 6; ++i) {
            int v = dg[i] + P.step[i] + carry;
            carry = v >= radix[i];
            if (carry) v -= radix[i];
            dg[i] = v;
        }
        dg[6] += P.step[6] + carry;
    }
    __device__ __forceinline__ Tile tile(const UmmaParams &P) const
    {
        Tile r;
        r.ks = dg[0]; r.ct = dg[1]; r.w0 = dg[2] * P.tw; r.h0 = dg[3] * P.th; r.d0 = dg[4] * P.td; r.cls = dg[5]; r.n = dg[6];
        return r;
    }
};

constexpr int MAX_STAGES = 8;
constexpr int MAX_ACC = 4;
constexpr int MAX_SBIAS = 2048;         // bias vectors up to this length are staged in shared memory


template <int KC, int BN>
struct SmemLayout {
    static constexpr int A_BYTES = 128 * KC * 2;
    static constexpr int B_BYTES = BN * KC * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;      // multiple of 1024 for every (KC, BN)
    static constexpr int EPI_BYTES = MAX_SBIAS * 4;                    // the staged bias
    // accumulators in TMEM, each drained by its own set of four epilogue warps (one warp per TMEM lane quarter)
    static constexpr int NACC = BN >= 256 ? 2 : (BN >= 64 ? 3 : 4);
    static constexpr int THREADS = 64 + 128 * NACC;
    static constexpr int CTRL_BYTES = 1024;
    static constexpr int BUDGET = 227 * 1024 - 1024 /* alignment slack */ - EPI_BYTES - CTRL_BYTES;
    static constexpr int STAGES = (BUDGET / STAGE_BYTES) < MAX_STAGES ? (BUDGET / STAGE_BYTES) : MAX_STAGES;
    static constexpr int TOTAL = 1024 + STAGES * STAGE_BYTES + EPI_BYTES + CTRL_BYTES;
    static constexpr int TMEM_COLS = (NACC * BN <= 32) ? 32 : (NACC * BN <= 64) ? 64 : (NACC * BN <= 128) ? 128 : (NACC * BN <= 256) ? 256 : 512;
};

// HEAD: 0, or the number of classes rounded up to a multiple of 4 (head mode, BN = 16)
template <int KC, int BN, int HEAD = 0>
__global__ void __launch_bounds__(SmemLayout<KC, BN>::THREADS, 1)
conv3_umma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const UmmaParams P)
{
    using L = SmemLayout<KC, BN>;
    constexpr int STAGES = L::STAGES;
    constexpr int NACC = L::NACC;
    constexpr uint32_t SWZ = (KC == 64) ? 2u : 4u;
    constexpr uint32_t SBO = 8 * KC * 2;                       // bytes per 8-row group
    constexpr uint32_t IDESC = make_idesc(BN);

    extern __shared__ uint8_t smem_raw[];
    // aligned by offsetting the shared array itself, so that the compiler still sees shared-memory pointers
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *stage_base = smem;
    float *epi = (float *)(smem + STAGES * L::STAGE_BYTES);
    uint64_t *bars = (uint64_t *)(smem + STAGES * L::STAGE_BYTES + L::EPI_BYTES);
    // bars: full[STAGES], empty[STAGES], tfull[NACC], tempty[NACC]; then tmem base (u32) and abort flag (int)
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * MAX_STAGES + 2 * MAX_ACC);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + MAX_STAGES);
    const uint32_t tfull0 = smem_u32(bars + 2 * MAX_STAGES), tempty0 = smem_u32(bars + 2 * MAX_STAGES + MAX_ACC);

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < NACC; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, 4); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), L::TMEM_COLS);
    pdl_wait();                 // everything above touched shared and tensor memory only
    float *sbias = epi;
    const bool bias_staged = P.bias && P.co <= MAX_SBIAS;
    if (bias_staged)
        for (int i = threadIdx.x; i < P.co; i += L::THREADS) sbias[i] = P.bias[i];
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            TileWalker tw_;
            tw_.init(P, blockIdx.x);
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x, tw_.next(P)) {
                const Tile T = tw_.tile(P);
                const int kit = P.taps.ntaps[T.cls] * P.chunks;
                int k0 = 0, k1 = kit, tp = 0, ch = 0;
                if (P.ksplit > 1) {
                    k0 = kit * T.ks / P.ksplit; k1 = kit * (T.ks + 1) / P.ksplit;
                    tp = k0 / P.chunks; ch = k0 - tp * P.chunks;
                }
                const int3 bw0 = make_int3(P.in_scale * T.w0, P.in_scale * T.h0, P.in_scale * T.d0);
                for (int ki = k0; ki < k1; ++ki) {
                    const uint32_t tw4 = P.taps.tap[T.cls][tp];
                    const int wt = (int)(tw4 & 0xFF);
                    const int cd = bw0.z + ((int)(tw4 << 16) >> 24);
                    const int chh = bw0.y + ((int)(tw4 << 8) >> 24);
                    const int cw = bw0.x + ((int)tw4 >> 24);
                    if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t fb = full0 + 8 * stage;
                    mbar_expect_tx(fb, L::STAGE_BYTES);
                    const uint32_t sa = smem_u32(stage_base + stage * L::STAGE_BYTES);
                    tma_load_5d(sa, &map_x, fb, ch * KC, cw, chh, cd, T.n);
                    tma_load_3d(sa + L::A_BYTES, &map_w, fb, ch * KC, T.ct * BN, wt);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    if (++ch == P.chunks) { ch = 0; ++tp; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            TileWalker tw_;
            tw_.init(P, blockIdx.x);
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x, tw_.next(P)) {
                const Tile T = tw_.tile(P);
                const int kit = P.taps.ntaps[T.cls] * P.chunks;
                // >= 1: ksplit <= taps * chunks
                const int kiters = P.ksplit > 1 ? kit * (T.ks + 1) / P.ksplit - kit * T.ks / P.ksplit : kit;
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
                if (++acc == NACC) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2 .. 2 + 4 NACC)
        // set e = (warp - 2) / 4 drains accumulator e, i.e. every NACC-th tile of this CTA
        const int q = warp & 3;                             // TMEM lane quarter this warp may read
        const uint32_t acc = (uint32_t)(warp - 2) >> 2;
        uint32_t acc_phase = 0;
        int it = 0;
        float s1[BN / 32 + 1], s2[BN / 32 + 1];             // per-lane column sums: column (c0 + lane) of each chunk
#pragma unroll
        for (int i = 0; i < BN / 32 + 1; ++i) { s1[i] = 0.f; s2[i] = 0.f; }
        int stat_n = -1, stat_ct = 0;
        bool ok = true;
        constexpr int HK = HEAD ? HEAD : 1;
        float hP[HK], hI[HK], hG[HK];                       // head mode: Dice sums of this thread's voxels
#pragma unroll
        for (int k = 0; k < HK; ++k) { hP[k] = 0.f; hI[k] = 0.f; hG[k] = 0.f; }
        auto flush = [&]() {
            if (HEAD && P.dice && stat_n >= 0) {
#pragma unroll
                for (int k = 0; k < HK; ++k) {
                    if (k < P.hK) {
                        float a = hI[k], b = hP[k], c = hG[k];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            a += __shfl_xor_sync(0xffffffffu, a, o);
                            b += __shfl_xor_sync(0xffffffffu, b, o);
                            c += __shfl_xor_sync(0xffffffffu, c, o);
                        }
                        if (lane == 0) {
                            double *dst = P.dice + ((int64_t)stat_n * P.hK + k) * 3;
                            atomicAdd(dst, (double)a); atomicAdd(dst + 1, (double)b); atomicAdd(dst + 2, (double)c);
                        }
                    }
                    hP[k] = 0.f; hI[k] = 0.f; hG[k] = 0.f;
                }
            }
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
        TileWalker tw_;
        tw_.init(P, blockIdx.x);
        for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x, ++it, tw_.next(P)) {
            if ((uint32_t)(it % NACC) != acc) continue;
            const Tile T = tw_.tile(P);
            const int ct = T.ct, n = T.n;
            if (n != stat_n || ct != stat_ct) { flush(); stat_n = n; stat_ct = ct; }
            const int m = q * 32 + lane;
            const int wx = m % P.tw, hy = (m / P.tw) % P.th, dz = m / (P.tw * P.th);
            const int jw = T.w0 + wx, jh = T.h0 + hy, jd = T.d0 + dz;
            const bool inside = (jw < P.W) && (jh < P.H) && (jd < P.D);
            // the whole warp takes the same decision, so no lane is left behind at a __syncwarp
            ok = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
            uint32_t r[32];
            if (BN >= 32) tmem_ld32(trow, r); else tmem_ld16(trow, r);
            if constexpr (HEAD > 0) {
                // the row holds the logits of the thread's voxel: softmax, arg max and the Dice sums
                tmem_ld_wait();
                const int64_t vox = (((int64_t)n * P.OD + jd) * P.OH + jh) * P.OW + jw;
                float l[HK];
#pragma unroll
                for (int k = 0; k < HK; ++k) l[k] = k < P.hK ? __uint_as_float(r[k]) + (bias_staged ? sbias[k] : 0.f) : -INFINITY;
                float mx = l[0];
                int am = 0;
#pragma unroll
                for (int k = 1; k < HK; ++k) if (l[k] > mx) { mx = l[k]; am = k; }
                float sum = 0.f;
                // exp(x) for x <= 0 as one exp2 of x * log2(e): relative error of a few 1e-7, far inside the
                // tolerance of the probabilities; classes beyond K contribute exp2(-inf) = 0
#pragma unroll
                for (int k = 0; k < HK; ++k) { l[k] = exp2f((l[k] - mx) * 1.4426950408889634f); sum += l[k]; }
                const float inv = 1.0f / sum;
                if (inside) {
                    const int lab = P.dice ? (int)P.labels[vox] : -1;
#pragma unroll
                    for (int k = 0; k < HK; ++k) {
                        const float p = l[k] * inv;
                        if (k < P.hK && P.probs) P.probs[vox * P.hK + k] = p;
                        hP[k] += p;
                        if (k == lab) { hI[k] += p; hG[k] += 1.f; }
                    }
                    if (P.amax) P.amax[vox] = (uint8_t)am;
                }
            } else {
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 32) {
                const int ncol = (BN - c0) < 32 ? (BN - c0) : 32;       // 32, or 16 for the last chunk
                // output voxel and first channel of this chunk of columns
                int cls = T.cls, ch0 = ct * BN + c0;
                if (P.merge_co) { cls = ch0 / P.merge_co; ch0 -= cls * P.merge_co; }
                const int w = P.out_scale * jw + (cls & 1), h = P.out_scale * jh + ((cls >> 1) & 1),
                          d = P.out_scale * jd + ((cls >> 2) & 1);
                const bool valid = inside && (w < P.OW) && (h < P.OH) && (d < P.OD);
                const int64_t vox = (((int64_t)n * P.OD + d) * P.OH + h) * P.OW + w + T.ks * P.part_stride;
                tmem_ld_wait();
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = (j < ncol && valid) ? __uint_as_float(r[j]) : 0.f;
                // the next chunk's accumulator columns travel while this one is converted and stored
                if (c0 + 32 < BN) {
                    if (BN - (c0 + 32) >= 32) tmem_ld32(trow + c0 + 32, r); else tmem_ld16(trow + c0 + 32, r);
                }
                if (valid && P.bias) {
                    if (bias_staged) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            if (j < ncol) {
                                const float4 b4 = *reinterpret_cast<const float4 *>(sbias + ch0 + j);
                                v[j] += b4.x; v[j + 1] += b4.y; v[j + 2] += b4.z; v[j + 3] += b4.w;
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) if (j < ncol) v[j] += __ldg(P.bias + ch0 + j);
                    }
                }
                if (valid) {
                    if (P.y_f32) {
                        float *dst = (float *)P.y + vox * P.y_pitch + ch0;
                        if (P.st32) {
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (8 * j < ncol) {
                                    uint32_t u[8];
#pragma unroll
                                    for (int e = 0; e < 8; ++e) u[e] = __float_as_uint(v[8 * j + e]);
                                    st_global_32B(dst + 8 * j, u);
                                }
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                if (4 * j < ncol)
                                    reinterpret_cast<float4 *>(dst)[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        }
                    } else {
                        bf16 *dst = (bf16 *)P.y + vox * P.y_pitch + ch0;
                        uint4 q4[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float f8[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) f8[e] = v[8 * j + e];
                            q4[j] = pack8(f8);
                        }
                        if (P.st32) {
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                if (16 * j < ncol) {
                                    const uint32_t u[8] = {q4[2 * j].x, q4[2 * j].y, q4[2 * j].z, q4[2 * j].w,
                                                           q4[2 * j + 1].x, q4[2 * j + 1].y, q4[2 * j + 1].z, q4[2 * j + 1].w};
                                    st_global_32B(dst + 16 * j, u);
                                }
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                if (8 * j < ncol) reinterpret_cast<uint4 *>(dst)[j] = q4[j];
                        }
                    }
                }
                if (P.stats) {
                    // lane j ends up with the sum (and sum of squares) of column j over the warp's 32 rows
                    float sq[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) sq[j] = v[j] * v[j];
                    s1[c0 / 32] += warp_colsum32(v, lane);
                    s2[c0 / 32] += warp_colsum32(sq, lane);
                }
            }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
            acc_phase ^= 1;
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

// Second step of a K-split pass: y = bias + sum over the splits (fixed order) of the fp32 partial results, plus the
// InstanceNorm sums of the finished values.  A block covers FIN_VOX voxels x 128 channels of one sample: thread =
// (4 channels, voxel lane), each voxel lane takes FIN_VOX / 8 voxels; the loads of one voxel are independent.
constexpr int FIN_VOX = 16, FIN_THREADS = 256, FIN_CG = 32;

__global__ void __launch_bounds__(FIN_THREADS)
splitk_finish_kernel(const float *__restrict__ part, int64_t split_elems, int ksplit, int64_t vox_per_n, int co,
                     const float *__restrict__ bias, void *__restrict__ y, int y_f32, int64_t y_pitch,
                     double *__restrict__ stats)
{
    __shared__ float4 red[2][FIN_THREADS];
    pdl_launch_dependents();
    pdl_wait();
    const int n = blockIdx.z;
    const int cl = threadIdx.x % FIN_CG, vl = threadIdx.x / FIN_CG;
    const int cg = blockIdx.y * FIN_CG + cl;                       // group of 4 channels
    const bool cok = 4 * cg < co;
    const int64_t v0 = (int64_t)blockIdx.x * FIN_VOX;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 b = (bias && cok) ? __ldg(reinterpret_cast<const float4 *>(bias) + cg) : zero;
    float4 s1 = zero, s2 = zero;
    if (cok) {
#pragma unroll
        for (int i = 0; i < FIN_VOX / 8; ++i) {
            const int64_t v = v0 + i * 8 + vl;
            if (v >= vox_per_n) break;
            const int64_t vox = (int64_t)n * vox_per_n + v;
            const float4 *src = reinterpret_cast<const float4 *>(part + vox * co) + cg;
            const size_t step = (size_t)(split_elems / 4);
            float4 a = zero;
            int s = 0;
            for (; s + 6 <= ksplit; s += 6) {
                float4 t[6];
#pragma unroll
                for (int u = 0; u < 6; ++u) t[u] = __ldcg(src + (size_t)(s + u) * step);
#pragma unroll
                for (int u = 0; u < 6; ++u) { a.x += t[u].x; a.y += t[u].y; a.z += t[u].z; a.w += t[u].w; }
            }
            for (; s < ksplit; ++s) {
                const float4 t = __ldcg(src + (size_t)s * step);
                a.x += t.x; a.y += t.y; a.z += t.z; a.w += t.w;
            }
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
            if (y_f32) {
                *reinterpret_cast<float4 *>((float *)y + vox * y_pitch + 4 * cg) = a;
            } else {
                __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
                uint2 u;
                u.x = *reinterpret_cast<uint32_t *>(&lo);
                u.y = *reinterpret_cast<uint32_t *>(&hi);
                *reinterpret_cast<uint2 *>((bf16 *)y + vox * y_pitch + 4 * cg) = u;
            }
            s1.x += a.x; s1.y += a.y; s1.z += a.z; s1.w += a.w;
            s2.x = fmaf(a.x, a.x, s2.x); s2.y = fmaf(a.y, a.y, s2.y); s2.z = fmaf(a.z, a.z, s2.z); s2.w = fmaf(a.w, a.w, s2.w);
        }
    }
    if (!stats) return;
    red[0][threadIdx.x] = s1;
    red[1][threadIdx.x] = s2;
    __syncthreads();
    if (vl == 0 && cok) {
        for (int r = 1; r < FIN_THREADS / FIN_CG; ++r) {           // fixed order over the voxel lanes
            const float4 p = red[0][r * FIN_CG + cl], q = red[1][r * FIN_CG + cl];
            s1.x += p.x; s1.y += p.y; s1.z += p.z; s1.w += p.w;
            s2.x += q.x; s2.y += q.y; s2.z += q.z; s2.w += q.w;
        }
        double *dst = stats + ((int64_t)n * co + 4 * cg) * 2;
        atomicAdd(dst + 0, (double)s1.x); atomicAdd(dst + 1, (double)s2.x);
        atomicAdd(dst + 2, (double)s1.y); atomicAdd(dst + 3, (double)s2.y);
        atomicAdd(dst + 4, (double)s1.z); atomicAdd(dst + 5, (double)s2.z);
        atomicAdd(dst + 6, (double)s1.w); atomicAdd(dst + 7, (double)s2.w);
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
PFN_cuTensorMapEncodeTiled_v12000 get_encode() { return (PFN_cuTensorMapEncodeTiled_v12000)tensor_map_encoder(); }

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

template <int KC, int BN, int HEAD = 0>
lamp_status_t launch(const CUtensorMap &mx, const CUtensorMap &mw, const UmmaParams &P, cudaStream_t st)
{
    using L = SmemLayout<KC, BN>;
    static SmemAttrOnce attr;
    { const lamp_status_t as = attr.ensure(conv3_umma_kernel<KC, BN, HEAD>, (int)(L::TOTAL)); if (as != LAMP_OK) return as; }
    const int sms = sm_count();
    const int grid = P.total_tiles < sms ? P.total_tiles : sms;
    UmmaParams Q = P;
    {
        const int radix[6] = {Q.ksplit, Q.nct, Q.ntw, Q.nth, Q.ntd, Q.nclass};
        int t = grid;
        for (int i = 0; i < 6; ++i) { Q.step[i] = t % radix[i]; t /= radix[i]; }
        Q.step[6] = t;
    }
    return launch_pdl(P.total_tiles <= 4 * grid, conv3_umma_kernel<KC, BN, HEAD>, dim3(grid), dim3(L::THREADS), L::TOTAL, st, mx, mw, Q);
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

struct KindInfo {
    int a_c, n_rows, taps;               // channels of the A tensor (GEMM K per tap), weight rows (GEMM N), taps in the weight tensor
    int ad, ah, aw;                      // extents of the A tensor
    int jd, jh, jw;                      // point grid
    int od, oh, ow;                      // output tensor extents
    int in_scale, out_scale, nclass;
};

bool kind_info(int kind, const ConvGeom &g, KindInfo *k)
{
    const bool s1 = g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed;
    const bool s2 = g.k == 3 && g.s == 2 && g.p == 1 && !g.transposed;
    const bool tr = g.k == 2 && g.s == 2 && g.p == 0 && g.transposed;
    k->in_scale = 1; k->out_scale = 1; k->nclass = 1;
    switch (kind) {
    case UK_S1_FWD:
        if (!s1) return false;
        *k = KindInfo{g.ci, g.co, 27, g.d, g.h, g.w, g.d, g.h, g.w, g.d, g.h, g.w, 1, 1, 1};
        return true;
    case UK_S1_DGRAD:
        if (!s1) return false;
        *k = KindInfo{g.co, g.ci, 27, g.d, g.h, g.w, g.d, g.h, g.w, g.d, g.h, g.w, 1, 1, 1};
        return true;
    case UK_S2_FWD:
        if (!s2) return false;
        *k = KindInfo{g.ci, g.co, 27, g.d, g.h, g.w, g.od, g.oh, g.ow, g.od, g.oh, g.ow, 2, 1, 1};
        return true;
    case UK_S2_DGRAD:
        if (!s2) return false;
        *k = KindInfo{g.co, g.ci, 27, g.od, g.oh, g.ow, g.od, g.oh, g.ow, g.d, g.h, g.w, 1, 2, 8};
        return true;
    case UK_T_FWD:
        if (!tr) return false;
        *k = KindInfo{g.ci, g.co, 8, g.d, g.h, g.w, g.d, g.h, g.w, g.od, g.oh, g.ow, 1, 2, 8};
        return true;
    case UK_T_DGRAD:
        if (!tr) return false;
        *k = KindInfo{g.co, g.ci, 8, g.od, g.oh, g.ow, g.d, g.h, g.w, g.d, g.h, g.w, 2, 1, 1};
        return true;
    case UK_T_FWD_MERGED:
        // the eight taps side by side on N: one GEMM [voxels x c_in] x [c_in x 8 c_out], each input tile read once
        if (!tr || g.co % 32) return false;
        *k = KindInfo{g.ci, 8 * g.co, 1, g.d, g.h, g.w, g.d, g.h, g.w, g.od, g.oh, g.ow, 1, 2, 1};
        return true;
    }
    return false;
}

void fill_taps(int kind, TapTable *T)
{
    memset(T, 0, sizeof(*T));
    auto set = [&](int cls, int wtap, int sd, int sh, int sw) {
        const int i = T->ntaps[cls]++;
        T->tap[cls][i] = (uint32_t)(wtap & 0xFF) | ((uint32_t)(sd & 0xFF) << 8) | ((uint32_t)(sh & 0xFF) << 16) | ((uint32_t)(sw & 0xFF) << 24);
    };
    if (kind == UK_S1_FWD || kind == UK_S2_FWD || kind == UK_S1_DGRAD) {
        // tap (kd,kh,kw) reads the input at shift k - 1; the data gradient uses the mirrored weight tap
        for (int t = 0; t < 27; ++t)
            set(0, kind == UK_S1_DGRAD ? 26 - t : t, t / 9 - 1, (t / 3) % 3 - 1, t % 3 - 1);
    } else if (kind == UK_T_FWD_MERGED) {
        set(0, 0, 0, 0, 0);
    } else if (kind == UK_T_DGRAD) {
        for (int t = 0; t < 8; ++t) set(0, t, t >> 2, (t >> 1) & 1, t & 1);
    } else if (kind == UK_T_FWD) {
        for (int c = 0; c < 8; ++c) set(c, c, 0, 0, 0);           // output parity (pd,ph,pw) = tap (a,b,c)
    } else {
        // stride-2 data gradient: dx[2j + parity] collects taps k with (parity + 1 - k) even, from dy[j + (parity + 1 - k) / 2]
        for (int c = 0; c < 8; ++c) {
            const int par[3] = {(c >> 2) & 1, (c >> 1) & 1, c & 1};
            for (int kd = 0; kd < 3; ++kd) {
                if ((par[0] + 1 - kd) & 1) continue;
                for (int kh = 0; kh < 3; ++kh) {
                    if ((par[1] + 1 - kh) & 1) continue;
                    for (int kw = 0; kw < 3; ++kw) {
                        if ((par[2] + 1 - kw) & 1) continue;
                        set(c, (kd * 3 + kh) * 3 + kw, (par[0] + 1 - kd) / 2, (par[1] + 1 - kh) / 2, (par[2] + 1 - kw) / 2);
                    }
                }
            }
        }
    }
}

struct TilePlan { int tw, th, td, ntw, nth, ntd, nct, chunks, KC, BN, ksplit; int64_t tiles; };

// Tiling of a pass, and over how many CTAs the (tap, chunk) range of a tile is split: deep U-Net levels have so few
// tiles that most SMs would idle, so their K range is shared out and a second small kernel adds the parts.
TilePlan plan_tiles(int kind, const ConvGeom &g, const KindInfo &k)
{
    TilePlan T;
    T.KC = (k.a_c % 64 == 0) ? 64 : 32;
    T.BN = pick_bn(k.n_rows);
    pick_tile(k.jd, k.jh, k.jw, &T.tw, &T.th, &T.td);
    T.ntw = (k.jw + T.tw - 1) / T.tw; T.nth = (k.jh + T.th - 1) / T.th; T.ntd = (k.jd + T.td - 1) / T.td;
    T.nct = T.BN ? k.n_rows / T.BN : 0;
    T.chunks = k.a_c / T.KC;
    T.tiles = (int64_t)g.n * k.nclass * T.ntd * T.nth * T.ntw * T.nct;
    TapTable tt;
    fill_taps(kind, &tt);
    int min_taps = 27;
    for (int c = 0; c < k.nclass; ++c) min_taps = tt.ntaps[c] < min_taps ? tt.ntaps[c] : min_taps;
    const int sms = sm_count();
    T.ksplit = 1;
    if (kind != UK_T_FWD_MERGED && T.tiles > 0 && T.tiles * 2 <= sms) {
        int s = (int)(sms / T.tiles);
        const int cap = min_taps * T.chunks / 4;          // at least four (tap, chunk) steps per CTA
        if (s > cap) s = cap;
        if (s >= 2) T.ksplit = s;
    }
    return T;
}

}  // namespace

size_t umma_splitk_ws(int kind, const ConvGeom &g)
{
    KindInfo k;
    if (kind == UK_T_FWD && kind_info(UK_T_FWD_MERGED, g, &k)) return 0;     // runs merged (when no statistics are asked for)
    if (!kind_info(kind, g, &k)) return 0;
    if (k.a_c % 32 || k.n_rows % 16 || !bn_instantiated(pick_bn(k.n_rows))) return 0;
    const TilePlan T = plan_tiles(kind, g, k);
    if (T.ksplit < 2) return 0;
    return align_up((size_t)T.ksplit * g.n * k.od * k.oh * k.ow * k.n_rows * sizeof(float), 256);
}

bool umma_conv_supported(int kind, const ConvGeom &g, const TView &a, const TView &y)
{
    KindInfo k;
    if (!kind_info(kind, g, &k)) return false;
    if (k.a_c % 32 || k.n_rows % 16) return false;
    if (!bn_instantiated(pick_bn(k.n_rows))) return false;
    if (a.pitch % 8 || ((uintptr_t)a.p & 15)) return false;
    if (y.f32 ? (y.pitch % 4 != 0) : (y.pitch % 8 != 0)) return false;
    if ((uintptr_t)y.p & 15) return false;
    return true;
}

bool umma_head_supported(const TView &z, int K)
{
    return K >= 1 && K <= 16 && z.c % 32 == 0 && z.c <= 256 && z.pitch % 8 == 0 && ((uintptr_t)z.p & 15) == 0;
}

// Head of the network on the tensor cores: logits = z * w^T + b as one [voxels x c] x [c x 16] GEMM (rows of w beyond
// K are out-of-range rows of the TMA box and arrive as zeros), softmax / arg max / Dice sums in the epilogue.
lamp_status_t umma_head(const TView &z, const bf16 *w, const float *b, int K, float *probs, uint8_t *argmax,
                        const uint8_t *labels, double *dice_sums, cudaStream_t st)
{
    if ((int64_t)z.n * z.d * z.h * z.w == 0) return LAMP_OK;
    PFN_cuTensorMapEncodeTiled_v12000 encode = get_encode();
    if (!encode) return LAMP_ERR_CUDA;
    const int KC = (z.c % 64 == 0) ? 64 : 32;
    UmmaParams P;
    memset(&P, 0, sizeof(P));
    P.N = z.n; P.D = z.d; P.H = z.h; P.W = z.w;
    P.OD = z.d; P.OH = z.h; P.OW = z.w;
    P.in_scale = 1; P.out_scale = 1; P.nclass = 1;
    pick_tile(z.d, z.h, z.w, &P.tw, &P.th, &P.td);
    P.ntw = (z.w + P.tw - 1) / P.tw; P.nth = (z.h + P.th - 1) / P.th; P.ntd = (z.d + P.td - 1) / P.td;
    P.nct = 1; P.ksplit = 1; P.part_stride = 0;
    P.chunks = z.c / KC;
    const int64_t tiles = (int64_t)z.n * P.ntd * P.nth * P.ntw;
    if (tiles > 0x7FFFFFFF) return LAMP_ERR_UNSUPPORTED;
    P.total_tiles = (int32_t)tiles;
    P.co = K; P.merge_co = 0;
    P.bias = b; P.status = status_word_ptr();
    P.hK = K; P.probs = probs; P.amax = argmax; P.labels = labels; P.dice = dice_sums;
    P.taps.ntaps[0] = 1;                                   // one tap, no shift, weight tile 0
    CUtensorMap mx, mw;
    {
        const cuuint64_t dims[5] = {(cuuint64_t)z.c, (cuuint64_t)z.w, (cuuint64_t)z.h, (cuuint64_t)z.d, (cuuint64_t)z.n};
        const cuuint64_t strides[4] = {(cuuint64_t)z.pitch * 2, (cuuint64_t)z.pitch * 2 * z.w,
                                       (cuuint64_t)z.pitch * 2 * z.w * z.h, (cuuint64_t)z.pitch * 2 * z.w * z.h * z.d};
        const cuuint32_t box[5] = {(cuuint32_t)KC, (cuuint32_t)P.tw, (cuuint32_t)P.th, (cuuint32_t)P.td, 1};
        const cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (encode(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, z.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    {
        const cuuint64_t dims[3] = {(cuuint64_t)z.c, (cuuint64_t)K, 1};
        const cuuint64_t strides[2] = {(cuuint64_t)z.c * 2, (cuuint64_t)z.c * 2 * K};
        const cuuint32_t box[3] = {(cuuint32_t)KC, 16, 1};
        const cuuint32_t es[3] = {1, 1, 1};
        if (encode(&mw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void *)w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    switch ((K + 3) / 4) {
    case 1:  return KC == 64 ? launch<64, 16, 4>(mx, mw, P, st) : launch<32, 16, 4>(mx, mw, P, st);
    case 2:  return KC == 64 ? launch<64, 16, 8>(mx, mw, P, st) : launch<32, 16, 8>(mx, mw, P, st);
    case 3:  return KC == 64 ? launch<64, 16, 12>(mx, mw, P, st) : launch<32, 16, 12>(mx, mw, P, st);
    default: return KC == 64 ? launch<64, 16, 16>(mx, mw, P, st) : launch<32, 16, 16>(mx, mw, P, st);
    }
}

size_t umma_dgrad_ws(const ConvGeom &g)
{
    return align_up((size_t)g.k * g.k * g.k * g.co * g.ci * sizeof(bf16), 256);
}

lamp_status_t umma_transpose_weights(const bf16 *w, bf16 *wt, int taps, int co, int ci, cudaStream_t st)
{
    const int64_t total = (int64_t)taps * co * ci;
    if (transpose_sum_supported(taps, co, ci)) return transpose_bf16(w, taps, co, ci, wt, st);
    transpose_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w, wt, co, ci, total);
    return launch_status();
}

// a: the tensor the taps read (x for forward kinds, dy for data-gradient kinds); w: [taps][n_rows][a_c] bf16
// (the layer's weights for forward kinds, their per-tap transpose for data-gradient kinds).
lamp_status_t umma_conv(int kind, const ConvGeom &g, const TView &a, const bf16 *w, const float *bias, const TView &y,
                        double *stats, void *part, size_t part_bytes, cudaStream_t st)
{
    KindInfo k;
    if (kind == UK_T_FWD && !stats && kind_info(UK_T_FWD_MERGED, g, &k) && bn_instantiated(pick_bn(k.n_rows)))
        kind = UK_T_FWD_MERGED;
    if (!kind_info(kind, g, &k)) return LAMP_ERR_UNSUPPORTED;
    if ((int64_t)g.n * k.jd * k.jh * k.jw == 0) return LAMP_OK;
    PFN_cuTensorMapEncodeTiled_v12000 encode = get_encode();
    if (!encode) return LAMP_ERR_CUDA;
    const TilePlan T = plan_tiles(kind, g, k);
    const int KC = T.KC, BN = T.BN;
    const int64_t out_vox = (int64_t)g.n * k.od * k.oh * k.ow;
    // the K range is split only when the caller's scratch can hold the partial results
    const bool split = T.ksplit > 1 && part && ((uintptr_t)part & 15) == 0 &&
                       part_bytes >= (size_t)T.ksplit * out_vox * k.n_rows * sizeof(float);
    UmmaParams P;
    P.N = g.n; P.D = k.jd; P.H = k.jh; P.W = k.jw;
    P.OD = k.od; P.OH = k.oh; P.OW = k.ow;
    P.in_scale = k.in_scale; P.out_scale = k.out_scale; P.nclass = k.nclass;
    P.tw = T.tw; P.th = T.th; P.td = T.td;
    P.ntw = T.ntw; P.nth = T.nth; P.ntd = T.ntd;
    P.nct = T.nct;
    P.chunks = T.chunks;
    P.ksplit = split ? T.ksplit : 1;
    P.part_stride = split ? out_vox : 0;
    const int64_t tiles = T.tiles * P.ksplit;
    if (tiles > 0x7FFFFFFF) return LAMP_ERR_UNSUPPORTED;
    P.total_tiles = (int32_t)tiles;
    P.co = k.n_rows; P.status = status_word_ptr();
    P.merge_co = kind == UK_T_FWD_MERGED ? g.co : 0;
    P.hK = 0; P.probs = nullptr; P.amax = nullptr; P.labels = nullptr; P.dice = nullptr;
    if (split) {
        P.y_f32 = 1; P.y_pitch = k.n_rows; P.y = part; P.bias = nullptr; P.stats = nullptr;
    } else {
        P.y_f32 = y.f32; P.y_pitch = y.pitch; P.y = y.p; P.bias = bias; P.stats = stats;
    }
    // a chunk of columns starts at a multiple of 16 channels, so rows are 32-byte aligned when base and pitch are
    P.st32 = ((uintptr_t)P.y & 31) == 0 && (P.y_pitch * (P.y_f32 ? 4 : 2)) % 32 == 0;
    fill_taps(kind, &P.taps);

    CUtensorMap mx, mw;
    {
        const cuuint32_t s = (cuuint32_t)k.in_scale;
        const cuuint64_t dims[5] = {(cuuint64_t)k.a_c, (cuuint64_t)k.aw, (cuuint64_t)k.ah, (cuuint64_t)k.ad, (cuuint64_t)g.n};
        const cuuint64_t strides[4] = {(cuuint64_t)a.pitch * 2, (cuuint64_t)a.pitch * 2 * k.aw,
                                       (cuuint64_t)a.pitch * 2 * k.aw * k.ah, (cuuint64_t)a.pitch * 2 * k.aw * k.ah * k.ad};
        // with an element stride s the box spans s times the number of voxels it delivers
        const cuuint32_t box[5] = {(cuuint32_t)KC, (cuuint32_t)P.tw * s, (cuuint32_t)P.th * s, (cuuint32_t)P.td * s, 1};
        const cuuint32_t es[5] = {1, s, s, s, 1};
        if (encode(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, a.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    {
        const cuuint64_t dims[3] = {(cuuint64_t)k.a_c, (cuuint64_t)k.n_rows, (cuuint64_t)k.taps};
        const cuuint64_t strides[2] = {(cuuint64_t)k.a_c * 2, (cuuint64_t)k.a_c * 2 * k.n_rows};
        const cuuint32_t box[3] = {(cuuint32_t)KC, (cuuint32_t)BN, 1};
        const cuuint32_t es[3] = {1, 1, 1};
        if (encode(&mw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void *)w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    const lamp_status_t s = KC == 64 ? launch_bn<64>(BN, mx, mw, P, st) : launch_bn<32>(BN, mx, mw, P, st);
    if (s != LAMP_OK || !split) return s;
    const int64_t vox_per_n = (int64_t)k.od * k.oh * k.ow;
    const dim3 grid((unsigned)((vox_per_n + FIN_VOX - 1) / FIN_VOX), (unsigned)((k.n_rows / 4 + FIN_CG - 1) / FIN_CG), (unsigned)g.n);
    return launch_pdl(true, splitk_finish_kernel, grid, dim3(FIN_THREADS), 0, st, (const float *)part, out_vox * k.n_rows, P.ksplit,
                      vox_per_n, k.n_rows, bias, y.p, y.f32, y.pitch, stats);
}

}  // namespace lamp
