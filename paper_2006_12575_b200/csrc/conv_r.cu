// 3x3x3 stride-1 pad-1 convolution of narrow layers (c_out = 64 or 32): "voxels x (kd, channels)" implicit
// GEMM whose accumulators rotate through three TMEM column slots.
//
// Why this shape.  One tcgen05.mma (M = 128, K = 16, bf16) holds the tensor pipe for N/2 cycles and one thread
// issues at most one every 60-100 cycles (measured), so c_out = 64 alone on N runs far below the full rate, and
// stacking the weights of two output planes on M (conv_t.cu) still spends a quarter of the MMAs on zero blocks.  Here the M rows are 128 OUTPUT
// VOXELS of one plane (8 (w) x 16 (h)) and the N columns are the THREE kd TAPS side by side:
//
//      D_p[voxel, (kd, co)] += X_p[voxel + (kh-1, kw-1), ci] * W[kd, kh, kw][co, ci]        (input plane p)
//
// Column block kd of input plane p belongs to output plane o = p + 1 - kd, so the three blocks of one MMA feed
// three CONSECUTIVE output planes.  Output plane o lives in TMEM column slot (o mod 3): every input plane
// writes all three slots (always 3 * c_out contiguous columns: no wrap-around, no zero blocks), only the ORDER
// of the kd blocks inside the weight tile rotates with p mod 3 - the weight producer places the three TMA boxes
// of a tile accordingly.  After input plane p the slot of output plane p - 1 is complete: the epilogue moves it
// to registers, stores zeros in its place (it becomes the fresh slot of plane p + 2) and hands it back.
//
//  * c_out = 32 (J = 2).  Three kd blocks of 32 channels would leave N = 96: 48 cycles, less than a thread's issue interval.  So a
//    slot holds TWO output rows side by side: the 128 M rows are the voxels of every second h row (8 (w) x 16 rows, the
//    descriptor steps two halo rows between 8-voxel groups), and column block (kd, jj) belongs to output row h + jj.
//    A window that starts hs rows into the halo box is tap kh = hs - jj of block jj: four window shifts hs = 0..3 x three
//    kw serve the nine in-plane taps of both rows, the blocks with kh outside 0..2 are fetched with an out-of-range tap
//    coordinate and arrive as zeros: 18 of 24 blocks carry work (75 % of the full rate; the stacked-plane form reaches
//    50 %).  Channels go in chunks of 32, and the three kw tiles of a shift share one pipeline stage.
//  * Two voxel windows per CTA (h rows 0..15 and 16..31 of one 8 x 32 window, one TMA halo box of 10 x 34 voxels
//    per input plane and channel chunk, out-of-volume voxels zero-filled = the zero padding) share every weight
//    tile, which halves the L2 -> SM weight traffic per MMA (the tiles are streamed: 27 * c_in * c_out * 2 bytes
//    do not fit beside the planes).  The nine in-plane taps are shifted windows of the halo box (descriptor
//    start (kh * 10 + kw) rows in, 10 rows between 8-voxel groups; the swizzle is a function of the address).
//  * Each window has its own MMA-issuing thread; both walk the same plane and weight stages, which are released once
//    both have committed them.  A window's slot hand-over (TMEM -> registers, zero store, barrier) after the last tile
//    of an input plane runs behind the other window's MMAs.
//  * A CTA owns a contiguous run of (window column, output plane) units; a run that starts or ends inside a
//    column costs one extra input plane each (the halo along d), columns that end at the volume border none.
//  * Epilogue: one voxel per thread with all its channels: bias, InstanceNorm sums (a transposing shuffle
//    butterfly per 32 columns), conversion and 32-byte stores of the voxel's channel run at the output's pitch.
//
// Warps: 0 = activation-plane TMA producer, 1 / 3 = MMA issuer of window 0 / 1 (warp 1 also owns the TMEM allocation),
// 2 = weight-tile TMA producer, 4..7 / 8..11 = epilogue of window 0 / 1.  All waits are bounded (LAMP_ERR_TIMEOUT on expiry).
#include <cuda.h>
#include <cudaTypedefs.h>
#include "common.cuh"
#include "umma_ptx.cuh"

namespace lamp {

namespace {

using namespace ptx;

constexpr int CR_THREADS = 384;
constexpr int TW = 8;                   // window pair: 8 (w) x 32 J (h) voxels = two windows of 128 M rows x J output rows
constexpr int HALO_W = TW + 2;
constexpr int MAX_NP = 4, MAX_NW = 8;
constexpr int CTRL_BYTES = 1024;
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr int WIN_COLS = 256;           // TMEM column stride between the two windows

struct CrParams {
    int32_t N, D, H, W;
    int32_t nwt, nht;                   // window pairs along w and h
    int32_t chunks;                     // c_in / KC
    int64_t units;                      // N * nht * nwt * D (window pair, output plane) units
    int32_t mirror, y_f32, st32;
    int32_t np, nw;                     // ring depths: activation planes, weight tiles
    int32_t plane_bytes;                // 1024-aligned bytes of one plane box
    int64_t y_pitch;
    void   *y;
    const float *bias;
    double *stats;
    int    *status;
};

// A run of output planes [o_lo, o_hi) of one window column.
struct Piece { int n, h0, w0, o_lo, o_hi; };

struct PieceWalker {
    int64_t u, u1;
    __device__ __forceinline__ void init(const CrParams &P)
    {
        u = P.units * (int64_t)blockIdx.x / gridDim.x;
        u1 = P.units * (int64_t)(blockIdx.x + 1) / gridDim.x;
    }
    __device__ __forceinline__ bool next(const CrParams &P, Piece &pc, int TH)
    {
        if (u >= u1) return false;
        int64_t col = u / P.D;
        pc.o_lo = (int)(u - col * P.D);
        const int64_t left = u1 - u;
        const int len = left < (int64_t)(P.D - pc.o_lo) ? (int)left : P.D - pc.o_lo;
        pc.o_hi = pc.o_lo + len;
        u += len;
        pc.w0 = (int)(col % P.nwt) * TW; col /= P.nwt;
        pc.h0 = (int)(col % P.nht) * TH;
        pc.n = (int)(col / P.nht);
        return true;
    }
};

__device__ __forceinline__ void tmem_st32_zero(uint32_t taddr)
{
    const uint32_t z = 0;
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                 ::"r"(taddr), "r"(z) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// KC: channels per chunk (64: 128-byte swizzle, 32: 64-byte swizzle).  CO x J = 64: output channels x output rows per slot.
template <int KC, int CO, int J>
__global__ void __launch_bounds__(CR_THREADS, 1)
conv3_r_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const CrParams P)
{
    static_assert(CO * J == 64, "a slot is 64 accumulator columns");
    constexpr int ROWB = KC * 2;
    constexpr uint32_t SWZ = KC == 64 ? 2u : 4u;
    constexpr int TH = 32 * J, HALO_H = TH + 2;
    constexpr uint32_t PLANE_BOX_BYTES = HALO_W * HALO_H * ROWB;
    constexpr uint32_t BLK_BYTES = CO * ROWB;                  // one (kd, jj) block of a weight tile
    constexpr uint32_t TILE_BYTES = 3 * J * BLK_BYTES;         // one (window shift, kw) tile: N = 192 rows
    constexpr int NT = 3 * (J + 2);                            // tiles per input plane and chunk: window shifts hs x kw
    constexpr int TPS = J == 2 ? 3 : 1;                        // tiles per pipeline stage
    constexpr uint32_t WST_BYTES = TPS * TILE_BYTES;
    constexpr int NCOL = 192;
    constexpr uint32_t IDESC = make_idesc(NCOL);

    extern __shared__ uint8_t smem_raw[];
    // aligned by offsetting the shared array itself, so that the compiler still sees shared-memory pointers
    uint8_t *smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t *p_base = smem;
    uint8_t *w_base = p_base + (size_t)P.np * P.plane_bytes;
    uint64_t *bars = (uint64_t *)(w_base + (size_t)P.nw * WST_BYTES);
    const uint32_t pfull0 = smem_u32(bars), pempty0 = smem_u32(bars + MAX_NP);
    const uint32_t wfull0 = smem_u32(bars + 2 * MAX_NP), wempty0 = smem_u32(bars + 2 * MAX_NP + MAX_NW);
    const uint32_t done0 = smem_u32(bars + 2 * MAX_NP + 2 * MAX_NW), free0 = done0 + 16;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * MAX_NP + 2 * MAX_NW + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    float *sbias = (float *)((uint8_t *)bars + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        // (a plane or weight stage is free again once BOTH windows' issuers have committed it)
        for (int s = 0; s < MAX_NP; ++s) { mbar_init(pfull0 + 8 * s, 1); mbar_init(pempty0 + 8 * s, 2); }
        for (int s = 0; s < MAX_NW; ++s) { mbar_init(wfull0 + 8 * s, 1); mbar_init(wempty0 + 8 * s, 2); }
        for (int s = 0; s < 2; ++s) { mbar_init(done0 + 8 * s, 1); mbar_init(free0 + 8 * s, 4); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    pdl_wait();                 // everything above touched shared and tensor memory only
    if (threadIdx.x < CO) sbias[threadIdx.x] = P.bias ? P.bias[threadIdx.x] : 0.f;
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
            PieceWalker pw;
            Piece pc;
            pw.init(P);
            while (ok && pw.next(P, pc, TH)) {
                const int p_lo = pc.o_lo > 0 ? pc.o_lo - 1 : 0, p_hi = pc.o_hi < P.D ? pc.o_hi : P.D - 1;
                for (int p = p_lo; p <= p_hi && ok; ++p) {
                    for (int c = 0; c < P.chunks; ++c) {
                        if (!mbar_wait(pempty0 + 8 * ps, pph ^ 1, abort_flag)) { ok = false; break; }
                        mbar_expect_tx(pfull0 + 8 * ps, PLANE_BOX_BYTES);
                        tma_load_5d(smem_u32(p_base + (size_t)ps * P.plane_bytes), &map_x, pfull0 + 8 * ps, c * KC, pc.w0 - 1,
                                    pc.h0 - 1, p, pc.n);
                        if (++ps == P.np) { ps = 0; pph ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 2) {
        // -------------------------------------------------------------------- weight tiles
        // The whole warp walks the stages; lane 0 waits for the stage and announces its bytes, then lane b issues box b
        // (one box = the J blocks of one (tile, kd): issuing the boxes of a stage from one thread, one after the
        // other, made the MMA issuer wait for weights a sixth of the time at 32 channels).
        constexpr int NBOX = 3 * TPS;
        const int ti = lane / 3, kd = lane - 3 * ti;            // this lane's box
        int ws = 0;
        uint32_t wph = 0;
        bool ok = true;
        PieceWalker pw;
        Piece pc;
        pw.init(P);
        while (ok && pw.next(P, pc, TH)) {
            const int p_lo = pc.o_lo > 0 ? pc.o_lo - 1 : 0, p_hi = pc.o_hi < P.D ? pc.o_hi : P.D - 1;
            for (int p = p_lo; p <= p_hi && ok; ++p) {
                // kd block of output plane o = p + 1 - kd goes to slot o mod 3 of the tile
                int slot = (p + 1) % 3 - kd;
                if (slot < 0) slot += 3;
                for (int c = 0; c < P.chunks && ok; ++c) {
                    for (int t0 = 0; t0 < NT; t0 += TPS) {
                        bool got = true;
                        if (lane == 0) {
                            got = mbar_wait(wempty0 + 8 * ws, wph ^ 1, abort_flag);
                            if (got) mbar_expect_tx(wfull0 + 8 * ws, WST_BYTES);
                        }
                        ok = __shfl_sync(0xffffffffu, (int)got, 0) != 0;
                        if (!ok) break;
                        if (lane < NBOX) {
                            // window shift hs serves tap kh = hs - jj of output row jj: the box spans kh = hs - J + 1 .. hs
                            // (block order jj = J - 1 .. 0); with mirrored taps the window (kd, kh, kw) reads weight tap
                            // (2 - kd, 2 - kh, 2 - kw), so the box spans 2 - hs .. 2 - hs + J - 1 (block order jj = 0 .. J - 1).
                            // Taps outside 0..2 are outside the tensor and arrive as zeros.
                            const int hs = (t0 + ti) / 3, kw = (t0 + ti) % 3;
                            tma_load_5d(smem_u32(w_base + (size_t)ws * WST_BYTES) + ti * TILE_BYTES + slot * (J * BLK_BYTES), &map_w,
                                        wfull0 + 8 * ws, c * KC, 0, P.mirror ? 2 - kw : kw, P.mirror ? 2 - hs : hs - J + 1,
                                        P.mirror ? 2 - kd : kd);
                        }
                        __syncwarp();
                        if (++ws == P.nw) { ws = 0; wph ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 1 || warp == 3) {
        if (lane == 0) {
            // ---------------------------------------------------------------- MMA issuers: warp 1 -> window 0, warp 3 -> window 1
            // One thread issuing both windows' MMAs spent 115-118 cycles per N = 192 instruction (barrier round trips,
            // descriptors and commits included) where the pipe needs 96: the tensor pipe idled a third of the time
            // waiting for its next instruction.  Each window therefore has its own issuing thread; the two share the
            // stages (every stage barrier expects both commits) and nothing else.
            const int j = warp == 1 ? 0 : 1;
            const uint32_t d_tmem = tmem_base + j * WIN_COLS;
            int ps = 0, ws = 0;
            uint32_t pph = 0, wph = 0, gs = 0;                  // gs: input planes issued so far (barrier phases)
            bool ok = true;
            PieceWalker pw;
            Piece pc;
            pw.init(P);
            while (ok && pw.next(P, pc, TH)) {
                const int p_lo = pc.o_lo > 0 ? pc.o_lo - 1 : 0, p_hi = pc.o_hi < P.D ? pc.o_hi : P.D - 1;
                for (int p = p_lo; p <= p_hi && ok; ++p, ++gs) {
                    for (int c = 0; c < P.chunks && ok; ++c) {
                        if (!mbar_wait(pfull0 + 8 * ps, pph, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        // window j: 16 groups of 8 voxels along w, J halo rows apart, from halo row hs + 16 J j
                        const uint32_t win = smem_u32(p_base + (size_t)ps * P.plane_bytes) + (16 * J * j) * HALO_W * ROWB;
                        if (c == 0) {
                            // the slot that input plane p starts afresh has been zeroed
                            if (!mbar_wait(free0 + 8 * j, gs & 1, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                        }
                        for (int t0 = 0; t0 < NT && ok; t0 += TPS) {
                            if (!mbar_wait(wfull0 + 8 * ws, wph, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                            const uint32_t wst = smem_u32(w_base + (size_t)ws * WST_BYTES);
#pragma unroll
                            for (int ti = 0; ti < TPS; ++ti) {
                                const int tt = t0 + ti, hs = tt / 3, kw = tt - hs * 3;
                                const uint64_t db = make_desc(wst + ti * TILE_BYTES, 0, 8 * ROWB, SWZ);
                                const uint64_t da = make_desc(win + (hs * HALO_W + kw) * ROWB, 0, J * HALO_W * ROWB, SWZ);
#pragma unroll
                                for (int k = 0; k < KC / 16; ++k) umma_bf16(d_tmem, da + 2 * k, db + 2 * k, IDESC, 1u);
                            }
                            if (c == P.chunks - 1 && t0 + TPS >= NT) umma_commit(done0 + 8 * j);
                            umma_commit(wempty0 + 8 * ws);
                            if (++ws == P.nw) { ws = 0; wph ^= 1; }
                        }
                        if (!ok) break;
                        umma_commit(pempty0 + 8 * ps);
                        if (++ps == P.np) { ps = 0; pph ^= 1; }
                    }
                }
            }
        }
    } else if (warp >= 4) {
        // -------------------------------------------------------------------- epilogue
        const int q = warp & 3;                                 // TMEM lane quarter of this warp
        const int j = (warp - 4) >> 2;                          // window
        const int m = q * 32 + lane;                            // M row of the window: output row(s) from hl, column wx
        const int hl = J * (16 * j + (m >> 3)), wx = m & 7;
        const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + j * WIN_COLS;
        uint32_t gs = 0;
        float s1[CO / 32], s2[CO / 32];                         // lane l: sums of channel (32 i + l)
#pragma unroll
        for (int i = 0; i < CO / 32; ++i) { s1[i] = 0.f; s2[i] = 0.f; }
        int stat_n = -1;
        bool ok = true;
        auto flush = [&]() {
            if (P.stats && stat_n >= 0) {
#pragma unroll
                for (int i = 0; i < CO / 32; ++i) {
                    double *dst = P.stats + ((int64_t)stat_n * CO + i * 32 + lane) * 2;
                    atomicAdd(dst, (double)s1[i]);
                    atomicAdd(dst + 1, (double)s2[i]);
                }
            }
#pragma unroll
            for (int i = 0; i < CO / 32; ++i) { s1[i] = 0.f; s2[i] = 0.f; }
        };
        // bias, statistics and store of 32 accumulator columns (the i-th 32 of the slot) of output plane o:
        // J = 1: channels 32 i .. 32 i + 31 of this thread's voxel; J = 2: all 32 channels of the voxel in row hl + i
        auto emit = [&](const Piece &pc, int o, int i32, const uint32_t (&r)[32]) {
            const int c0 = J == 1 ? 32 * i32 : 0;
            // J = 2: the slot's halves are the two output rows in the order the weight box delivered their taps
            const int h = pc.h0 + hl + (J == 2 ? (P.mirror ? i32 : 1 - i32) : 0), w = pc.w0 + wx;
            const bool valid = h < P.H && w < P.W;
            float v[32];
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                const float4 b4 = *reinterpret_cast<const float4 *>(sbias + c0 + e);
                v[e] = valid ? __uint_as_float(r[e]) + b4.x : 0.f;
                v[e + 1] = valid ? __uint_as_float(r[e + 1]) + b4.y : 0.f;
                v[e + 2] = valid ? __uint_as_float(r[e + 2]) + b4.z : 0.f;
                v[e + 3] = valid ? __uint_as_float(r[e + 3]) + b4.w : 0.f;
            }
            if (valid) {
                const int64_t vox = (((int64_t)pc.n * P.D + o) * P.H + h) * P.W + w;
                if (P.y_f32) {
                    float *dst = (float *)P.y + vox * P.y_pitch + c0;
                    if (P.st32) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            uint32_t u[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) u[i] = __float_as_uint(v[8 * e + i]);
                            st_global_32B(dst + 8 * e, u);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            reinterpret_cast<float4 *>(dst)[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                    }
                } else {
                    bf16 *dst = (bf16 *)P.y + vox * P.y_pitch + c0;
                    uint4 q4[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float f8[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) f8[i] = v[8 * e + i];
                        q4[e] = pack8(f8);
                    }
                    if (P.st32) {
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const uint32_t u[8] = {q4[2 * e].x, q4[2 * e].y, q4[2 * e].z, q4[2 * e].w,
                                                   q4[2 * e + 1].x, q4[2 * e + 1].y, q4[2 * e + 1].z, q4[2 * e + 1].w};
                            st_global_32B(dst + 16 * e, u);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) reinterpret_cast<uint4 *>(dst)[e] = q4[e];
                    }
                }
            }
            if (P.stats) {
                float sq[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) sq[e] = v[e] * v[e];
                s1[c0 / 32] += warp_colsum32(v, lane);
                s2[c0 / 32] += warp_colsum32(sq, lane);
            }
        };
        auto hand_back = [&]() {
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(free0 + 8 * j);
        };
        // all three slots start at zero
#pragma unroll
        for (int c0 = 0; c0 < NCOL; c0 += 32) tmem_st32_zero(trow + c0);
        hand_back();
        PieceWalker pw;
        Piece pc;
        pw.init(P);
        while (ok && pw.next(P, pc, TH)) {
            if (pc.n != stat_n) { flush(); stat_n = pc.n; }
            const int p_lo = pc.o_lo > 0 ? pc.o_lo - 1 : 0, p_hi = pc.o_hi < P.D ? pc.o_hi : P.D - 1;
            for (int p = p_lo; p <= p_hi && ok; ++p, ++gs) {
                ok = __all_sync(0xffffffffu, mbar_wait(done0 + 8 * j, gs & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                const uint32_t tdone = trow + (uint32_t)((p + 2) % 3) * 64;      // slot of output plane p - 1
                uint32_t r[2][32];
                if (p < p_hi) {
#pragma unroll
                    for (int i = 0; i < 2; ++i) tmem_ld32(tdone + 32 * i, r[i]);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 2; ++i) tmem_st32_zero(tdone + 32 * i);
                    hand_back();
                    if (p - 1 >= pc.o_lo) {
#pragma unroll
                        for (int i = 0; i < 2; ++i) emit(pc, p - 1, i, r[i]);
                    }
                } else {
                    // last input plane of the run: plane p - 1 is complete, and so is plane p where the volume ends;
                    // whatever the slots hold afterwards belongs to planes outside the run
                    if (p - 1 >= pc.o_lo) {
#pragma unroll
                        for (int i = 0; i < 2; ++i) tmem_ld32(tdone + 32 * i, r[i]);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 2; ++i) emit(pc, p - 1, i, r[i]);
                    }
                    if (p < pc.o_hi) {
                        const uint32_t tlast = trow + (uint32_t)(p % 3) * 64;
#pragma unroll
                        for (int i = 0; i < 2; ++i) tmem_ld32(tlast + 32 * i, r[i]);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 2; ++i) emit(pc, p, i, r[i]);
                    }
#pragma unroll
                    for (int c0 = 0; c0 < NCOL; c0 += 32) tmem_st32_zero(trow + c0);
                    hand_back();
                }
            }
        }
        flush();
    }

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

struct CrPlan { CrParams P; int KC, CO, J, TH; size_t smem; int grid; };

bool make_cr_plan(const ConvGeom &g, CrPlan *out)
{
    if (!(g.k == 3 && g.s == 1 && g.p == 1 && !g.transposed)) return false;
    if (g.co != 64 && g.co != 32) return false;
    if (g.ci % 32 || g.ci <= 0) return false;
    const int J = g.co == 64 ? 1 : 2;
    const int KC = (J == 1 && g.ci % 64 == 0) ? 64 : 32;       // two output rows per slot: planes twice as tall, 32-channel chunks
    const int TH = 32 * J;
    const int rowb = KC * 2;
    CrParams &P = out->P;
    P.N = g.n; P.D = g.od; P.H = g.oh; P.W = g.ow;
    P.chunks = g.ci / KC;
    P.plane_bytes = (int)align_up((size_t)HALO_W * (TH + 2) * rowb, 1024);
    const int wst = (J == 2 ? 3 : 1) * 192 * rowb;              // one stage: 1 or 3 tiles of 192 rows
    const int np = (KC == 64 || J == 2) ? 2 : 3;
    int nw = (SMEM_LIMIT - 1024 - CTRL_BYTES - np * P.plane_bytes) / wst;
    if (nw > MAX_NW) nw = MAX_NW;
    if (nw < 3) return false;
    P.np = np; P.nw = nw;
    P.nwt = (g.ow + TW - 1) / TW;
    P.nht = (g.oh + TH - 1) / TH;
    const int64_t units = (int64_t)g.n * P.nht * P.nwt * g.od;
    if (units <= 0 || units > 0x3FFFFFFF) return false;
    P.units = units;
    const int sms = sm_count();
    out->KC = KC; out->CO = g.co; out->J = J; out->TH = TH;
    out->smem = 1024 + (size_t)np * P.plane_bytes + (size_t)nw * wst + CTRL_BYTES;
    if (out->smem > (size_t)SMEM_LIMIT) return false;
    out->grid = (int)(units < sms ? units : sms);
    return true;
}

template <int KC, int CO, int J>
lamp_status_t launch_cr(const CUtensorMap &mx, const CUtensorMap &mw, const CrPlan &pl, cudaStream_t st)
{
    static SmemAttrOnce attr;
    { const lamp_status_t as = attr.ensure(conv3_r_kernel<KC, CO, J>, SMEM_LIMIT); if (as != LAMP_OK) return as; }
    return launch_pdl(pl.P.units <= 4 * (int64_t)pl.grid, conv3_r_kernel<KC, CO, J>, dim3(pl.grid), dim3(CR_THREADS), pl.smem, st, mx, mw, pl.P);
}

}  // namespace

bool cr_conv_fwd_supported(const ConvGeom &g, const TView &x, const TView &y)
{
    CrPlan pl;
    if ((int64_t)g.n * g.d * g.h * g.w == 0) return false;
    if (!make_cr_plan(g, &pl)) return false;
    // the window pair (8 x 32 or 8 x 64 voxels) must not be mostly padding
    const double used = (double)g.oh * g.ow / ((double)pl.P.nht * pl.TH * pl.P.nwt * TW);
    if (used < 0.55) return false;
    // a run cut inside a column pays two extra input planes: worth it only for runs of some length (shorter ones
    // go to the stacked-plane kernel, which pays a fixed quarter)
    const int64_t run = pl.P.units / pl.grid;
    if (run < g.od && run < 10) return false;
    if (x.pitch % 8 || ((uintptr_t)x.p & 15)) return false;
    if (y.f32 ? (y.pitch % 4 != 0) : (y.pitch % 8 != 0)) return false;
    if ((uintptr_t)y.p & 15) return false;
    return true;
}

lamp_status_t cr_conv_fwd(const ConvGeom &g, const TView &x, const bf16 *w, const float *bias, const TView &y,
                          double *stats, int mirror_taps, cudaStream_t st)
{
    CrPlan pl;
    if (!make_cr_plan(g, &pl)) return LAMP_ERR_UNSUPPORTED;
    PFN_cuTensorMapEncodeTiled_v12000 encode = (PFN_cuTensorMapEncodeTiled_v12000)tensor_map_encoder();
    if (!encode) return LAMP_ERR_CUDA;
    CrParams &P = pl.P;
    P.mirror = mirror_taps; P.y_f32 = y.f32; P.y_pitch = y.pitch; P.y = y.p;
    P.bias = bias; P.stats = stats; P.status = status_word_ptr();
    const size_t es_y = y.f32 ? 4 : 2;
    P.st32 = (((uintptr_t)y.p & 31) == 0) && ((y.pitch * es_y) % 32 == 0);
    const CUtensorMapSwizzle swz = pl.KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    CUtensorMap mx, mw;
    {
        const cuuint64_t dims[5] = {(cuuint64_t)g.ci, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.d, (cuuint64_t)g.n};
        const cuuint64_t strides[4] = {(cuuint64_t)x.pitch * 2, (cuuint64_t)x.pitch * 2 * g.w,
                                       (cuuint64_t)x.pitch * 2 * g.w * g.h, (cuuint64_t)x.pitch * 2 * g.w * g.h * g.d};
        const cuuint32_t box[5] = {(cuuint32_t)pl.KC, (cuuint32_t)HALO_W, (cuuint32_t)(pl.TH + 2), 1, 1};
        const cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (encode(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, x.p, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    {
        // weights [kd][kh][kw][row = output channel of this pass][k = reduced channel] as a 5-D tensor, so that a tap
        // coordinate outside 0..2 delivers a block of zeros; one box = the J consecutive kh blocks of one (kd, kw)
        const cuuint64_t dims[5] = {(cuuint64_t)g.ci, (cuuint64_t)g.co, 3, 3, 3};
        const cuuint64_t tapb = (cuuint64_t)g.ci * 2 * g.co;
        const cuuint64_t strides[4] = {(cuuint64_t)g.ci * 2, tapb, 3 * tapb, 9 * tapb};
        const cuuint32_t box[5] = {(cuuint32_t)pl.KC, (cuuint32_t)pl.CO, 1, (cuuint32_t)pl.J, 1};
        const cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (encode(&mw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, (void *)w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LAMP_ERR_CUDA;
    }
    lamp_status_t s;
    if (pl.J == 2) s = launch_cr<32, 32, 2>(mx, mw, pl, st);
    else if (pl.KC == 64) s = launch_cr<64, 64, 1>(mx, mw, pl, st);
    else s = launch_cr<32, 64, 1>(mx, mw, pl, st);
    if (s != LAMP_OK) return s;
    return launch_status();
}

}  // namespace lamp
