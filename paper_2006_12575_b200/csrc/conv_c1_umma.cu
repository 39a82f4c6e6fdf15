// First layer of the network (one input channel, 3x3x3 s1 p1) on the sm_100a tensor cores.
//
// With a single input channel the w axis itself can serve as the reduction axis.  For a run of 8 output voxels
// w = 8a .. 8a+7 on the line (d, h), and 32 output channels,
//     y[d, h, 8a + j, c] = sum_{kd,kh} sum_{i=0..31} x[d+kd-1, h+kh-1, 8a-8+i] * T_{kd,kh}[i][(j, c)],
//     T_{kd,kh}[i][(j, c)] = w[kd, kh, kw = i - 7 - j][c]  if 0 <= kw <= 2, else 0,
// i.e. nine GEMMs whose A operand is a 64-byte piece of an input line (M = 128 lines, K = 32 positions starting at the
// 16-byte-aligned position 8a-8) and whose B operand is a banded matrix built once per CTA in shared memory
// (N = 8 x 32 = 256).  A tile is 128 lines (8 along h x 16 along d) x 8 voxels x 32 channels.  ONE TMA load per tile
// brings the 10 x 18 halo of line pieces (out-of-volume positions zero-filled = the padding); the A operand of tap
// (kd, kh) is the window of that box that starts kh + 10 kd rows in, with 10 rows between its 8-row groups.  The layer
// is then bound by writing y, not by arithmetic or by gathering neighbours.
// Wider layers run as c_out / 32 independent channel blocks, one per CTA.
//
// Per CTA (persistent over the tiles of its channel block), warp-specialised:
//   warp 0    : TMA producer, one halo box per tile into a ring of stages.
//   warp 1    : allocates TMEM, issues tcgen05.mma (two K = 16 steps per tap, nine taps per tile) into one of two
//               256-column accumulators.
//   warps 2-9 : epilogue, four warps (one per TMEM lane quarter) per accumulator.  A thread owns one line: per output
//               voxel it adds the bias and stores the 32 channels (its eight voxels are contiguous in memory); the
//               InstanceNorm sums of its values stay in registers over all its tiles and are added across the
//               warp's lines (shared-memory transpose) only when the sample changes or the CTA is done.
// Every mbarrier wait is bounded; on expiry the CTA records LAMP_ERR_TIMEOUT and winds down.
#include <cuda.h>
#include <cudaTypedefs.h>
#include "common.cuh"
#include "umma_ptx.cuh"

namespace lamp {

namespace {

using namespace ptx;

constexpr int STAGES = 3;
constexpr int TH = 8, TD = 16;                   // lines of a tile along h and d
constexpr int HALO_H = TH + 2, HALO_D = TD + 2;
constexpr int BOX_BYTES = HALO_H * HALO_D * 64;  // 180 line pieces of 32 positions
constexpr int A_BYTES = 12 * 1024;               // one stage (the box, rounded up to the swizzle alignment)
constexpr int B_BYTES = 256 * 64;                // one banded matrix: 256 (j, c) rows x 32 positions
constexpr int EPI_WARPS = 8;
constexpr int C1_THREADS = 64 + 32 * EPI_WARPS;
constexpr int TR_FLOATS = 32 * 33;               // per epilogue warp: 32 x 32 transpose (+1 pad)

struct C1Params {
    int32_t N, D, H, W;
    int32_t nth, ntd, nseg;                      // tiles along h, d; runs of 8 voxels along w
    int32_t tiles_per_part;                      // n * ntd * nth * nseg
    int32_t nparts;                              // c_out / 32
    int32_t co;
    int32_t y_f32, st32;
    int64_t y_pitch;
    const bf16 *w;                               // [27][co]
    const float *bias;
    void *y;
    double *stats;
    int *status;
};

// byte offset of 16-byte chunk c (8 K-elements) of row r in a K-major tile with 64-byte rows and the 64-byte swizzle
__device__ __forceinline__ uint32_t swz64(int r, int c) { return (uint32_t)(r * 64 + ((c ^ ((r >> 1) & 3)) << 4)); }

struct C1Tile { int seg, h0, d0, n; };

__device__ __forceinline__ C1Tile decode(const C1Params &P, int t)
{
    C1Tile r;
    r.seg = t % P.nseg; t /= P.nseg;
    r.h0 = (t % P.nth) * TH; t /= P.nth;
    r.d0 = (t % P.ntd) * TD;
    r.n = t / P.ntd;
    return r;
}

constexpr size_t C1_SMEM = 1024 + 9 * (size_t)B_BYTES + STAGES * (size_t)A_BYTES + EPI_WARPS * TR_FLOATS * 4 + 32 * 4 + 256;

__global__ void __launch_bounds__(C1_THREADS, 1)
conv_c1_umma_kernel(const __grid_constant__ CUtensorMap map_x, const C1Params P)
{
    extern __shared__ uint8_t smem_raw[];
    // aligned by offsetting the shared array itself, so that the compiler still sees shared-memory pointers
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *b_tiles = smem;                                    // 9 x [256 rows x 64 B]
    uint8_t *a_stages = smem + 9 * B_BYTES;                     // STAGES x [128 rows x 64 B]
    float *trans = (float *)(a_stages + STAGES * A_BYTES);      // EPI_WARPS x [32][33]
    float *sbias = trans + EPI_WARPS * TR_FLOATS;               // [32]
    uint64_t *bars = (uint64_t *)(sbias + 32);                  // full[STAGES], empty[STAGES], tfull[2], tempty[2]
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STAGES);
    const uint32_t tfull0 = smem_u32(bars + 2 * STAGES), tempty0 = smem_u32(bars + 2 * STAGES + 2);
    const int part = blockIdx.x % P.nparts;                     // the CTA's block of 32 output channels
    const int first = blockIdx.x / P.nparts, step = gridDim.x / P.nparts;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, 4); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    pdl_wait();                 // everything above touched shared and tensor memory only
    // the nine banded matrices: row (j, c), position i -> w[kd][kh][i - 7 - j][part * 32 + c] inside the band
    for (int idx = threadIdx.x; idx < 9 * 256 * 4; idx += C1_THREADS) {
        const int tap = idx / 1024, r = (idx >> 2) & 255, ch = idx & 3;
        const int j = r >> 5, c = r & 31;
        uint32_t u[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            uint32_t pr = 0;
#pragma unroll
            for (int hlf = 0; hlf < 2; ++hlf) {
                const int kw = 8 * ch + 2 * e + hlf - 7 - j;
                if (kw >= 0 && kw <= 2)
                    pr |= (uint32_t)__bfloat16_as_ushort(P.w[(tap * 3 + kw) * P.co + part * 32 + c]) << (16 * hlf);
            }
            u[e] = pr;
        }
        *reinterpret_cast<uint4 *>(b_tiles + tap * B_BYTES + swz64(r, ch)) = make_uint4(u[0], u[1], u[2], u[3]);
    }
    if (threadIdx.x < 32) sbias[threadIdx.x] = P.bias ? P.bias[part * 32 + threadIdx.x] : 0.f;
    fence_proxy_async();
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
            for (int t = first; t < P.tiles_per_part && ok; t += step) {
                const C1Tile T = decode(P, t);
                if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                const uint32_t fb = full0 + 8 * stage;
                mbar_expect_tx(fb, BOX_BYTES);
                tma_load_4d(smem_u32(a_stages + stage * A_BYTES), &map_x, fb, 8 * T.seg - 8, T.h0 - 1, T.d0 - 1, T.n);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t IDESC = make_idesc(256);
            int stage = 0;
            uint32_t phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int t = first; t < P.tiles_per_part && ok; t += step) {
                if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * 256;
                if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t box = smem_u32(a_stages + stage * A_BYTES);
#pragma unroll
                for (int tap = 0; tap < 9; ++tap) {
                    // lines (h0 + hy + kh - 1, d0 + dz + kd - 1): rows kh + hy + 10 (kd + dz) of the box
                    const uint64_t da = make_desc(box + (uint32_t)((tap % 3 + HALO_H * (tap / 3)) * 64), 0, HALO_H * 64, 4u);
                    const uint64_t db = make_desc(smem_u32(b_tiles + tap * B_BYTES), 0, 512, 4u);
                    umma_bf16(d_tmem, da, db, IDESC, tap ? 1u : 0u);
                    umma_bf16(d_tmem, da + 2, db + 2, IDESC, 1u);         // positions 16..31: +32 bytes
                }
                umma_commit(empty0 + 8 * stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
                umma_commit(tfull0 + 8 * acc);
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int e = warp - 2;
        const int q = warp & 3;                                  // TMEM lane quarter this warp may read
        const uint32_t acc = (uint32_t)(e >> 2);                 // accumulator drained by this warp: every other tile
        float *tr = trans + e * TR_FLOATS;
        const int m = q * 32 + lane;                             // the thread's line within a tile = accumulator lane
        const int hy = m % TH, dz = m / TH;
        float s1[32], s2[32];                                    // per channel: sum and sum of squares of this thread's values
#pragma unroll
        for (int c = 0; c < 32; ++c) { s1[c] = 0.f; s2[c] = 0.f; }
        int stat_n = -1;
        // lane c receives the warp's totals of channel c (fixed order over the 32 lines) and adds them to the statistics
        auto flush = [&]() {
            if (P.stats && stat_n >= 0) {
                float tot[2];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    __syncwarp();
#pragma unroll
                    for (int c = 0; c < 32; ++c) tr[lane * 33 + c] = k ? s2[c] : s1[c];
                    __syncwarp();
                    float a = 0.f;
#pragma unroll
                    for (int rr = 0; rr < 32; ++rr) a += tr[rr * 33 + lane];
                    tot[k] = a;
                }
                double *dst = P.stats + ((int64_t)stat_n * P.co + part * 32 + lane) * 2;
                atomicAdd(dst, (double)tot[0]);
                atomicAdd(dst + 1, (double)tot[1]);
            }
#pragma unroll
            for (int c = 0; c < 32; ++c) { s1[c] = 0.f; s2[c] = 0.f; }
        };
        uint32_t acc_phase = 0;
        int it = 0;
        bool ok = true;
        for (int t = first; t < P.tiles_per_part && ok; t += step, ++it) {
            if ((uint32_t)(it & 1) != acc) continue;
            const C1Tile T = decode(P, t);
            if (T.n != stat_n) { flush(); stat_n = T.n; }
            const int h = T.h0 + hy, d = T.d0 + dz;
            const bool valid = h < P.H && d < P.D;
            const int64_t vox0 = (((int64_t)T.n * P.D + d) * P.H + h) * P.W + 8 * T.seg;
            ok = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
            uint32_t r[32];
            tmem_ld32(trow, r);
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                tmem_ld_wait();
                float v[32];
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    const float4 b4 = *reinterpret_cast<const float4 *>(sbias + c);
                    v[c] = __uint_as_float(r[c]) + b4.x; v[c + 1] = __uint_as_float(r[c + 1]) + b4.y;
                    v[c + 2] = __uint_as_float(r[c + 2]) + b4.z; v[c + 3] = __uint_as_float(r[c + 3]) + b4.w;
                }
                if (jj < 7) tmem_ld32(trow + 32 * (jj + 1), r);  // the next voxel's columns travel meanwhile
                if (valid) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) { s1[c] += v[c]; s2[c] = fmaf(v[c], v[c], s2[c]); }
                    if (P.y_f32) {
                        float *dst = (float *)P.y + (vox0 + jj) * P.y_pitch + part * 32;
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            reinterpret_cast<float4 *>(dst)[c] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                    } else {
                        bf16 *dst = (bf16 *)P.y + (vox0 + jj) * P.y_pitch + part * 32;
                        uint4 q4[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            float f8[8];
#pragma unroll
                            for (int x = 0; x < 8; ++x) f8[x] = v[8 * c + x];
                            q4[c] = pack8(f8);
                        }
                        if (P.st32) {
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                const uint32_t w8[8] = {q4[2 * c].x, q4[2 * c].y, q4[2 * c].z, q4[2 * c].w,
                                                        q4[2 * c + 1].x, q4[2 * c + 1].y, q4[2 * c + 1].z, q4[2 * c + 1].w};
                                st_global_32B(dst + 16 * c, w8);
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 4; ++c) reinterpret_cast<uint4 *>(dst)[c] = q4[c];
                        }
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
        tmem_dealloc(tmem_base, 512);
    }
}

PFN_cuTensorMapEncodeTiled_v12000 get_encode() { return (PFN_cuTensorMapEncodeTiled_v12000)tensor_map_encoder(); }

}  // namespace

bool c1_umma_supported(const ConvGeom &g, const TView &x, const TView &y)
{
    if (!(g.ci == 1 && g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed)) return false;
    if (g.co % 32 || g.co > 256) return false;
    // the input is read by TMA as [n][d][h][w] with w innermost: unit pitch, rows that start on 16-byte boundaries
    if (x.pitch != 1 || g.w % 8 || ((uintptr_t)x.p & 15)) return false;
    if ((uintptr_t)y.p & 15) return false;
    return y.f32 ? y.pitch % 4 == 0 : y.pitch % 8 == 0;
}

lamp_status_t c1_umma_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                          double *stats, cudaStream_t st)
{
    if ((int64_t)g.n * g.d * g.h * g.w == 0) return LAMP_OK;
    PFN_cuTensorMapEncodeTiled_v12000 encode = get_encode();
    if (!encode) return LAMP_ERR_CUDA;
    C1Params P;
    P.N = g.n; P.D = g.d; P.H = g.h; P.W = g.w;
    P.nth = (g.h + TH - 1) / TH; P.ntd = (g.d + TD - 1) / TD; P.nseg = g.w / 8;
    const int64_t tiles = (int64_t)g.n * P.ntd * P.nth * P.nseg;
    if (tiles > 0x7FFFFFFF) return LAMP_ERR_UNSUPPORTED;
    P.tiles_per_part = (int32_t)tiles;
    P.nparts = g.co / 32;
    P.co = g.co;
    P.y_f32 = y.f32;
    P.st32 = ((uintptr_t)y.p & 31) == 0 && (y.pitch * (y.f32 ? 4 : 2)) % 32 == 0;
    P.y_pitch = y.pitch;
    P.w = w; P.bias = bias; P.y = y.p; P.stats = stats;
    P.status = status_word_ptr();

    CUtensorMap mx;
    {
        const cuuint64_t dims[4] = {(cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.d, (cuuint64_t)g.n};
        const cuuint64_t strides[3] = {(cuuint64_t)g.w * 2, (cuuint64_t)g.w * 2 * g.h, (cuuint64_t)g.w * 2 * g.h * g.d};
        const cuuint32_t box[4] = {32, HALO_H, HALO_D, 1};
        const cuuint32_t es[4] = {1, 1, 1, 1};
        if (encode(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, x.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    static SmemAttrOnce attr;
    { const lamp_status_t as = attr.ensure(conv_c1_umma_kernel, (int)((int)C1_SMEM)); if (as != LAMP_OK) return as; }
    const int sms = sm_count();
    // every CTA serves one channel block: the grid is a multiple of the number of blocks
    int64_t per_part = sms / P.nparts;
    if (per_part < 1) per_part = 1;
    if (per_part > tiles) per_part = tiles;
    const int grid = (int)(per_part * P.nparts);
    const lamp_status_t ls = launch_pdl(tiles * P.nparts <= 16 * (int64_t)grid, conv_c1_umma_kernel, dim3(grid), dim3(C1_THREADS), (size_t)C1_SMEM, st, mx, P);
    if (ls != LAMP_OK) return ls;
    return launch_status();
}

}  // namespace lamp
