// U-Net executor: layer plan, workspace arena, forward pass, training step, sliding window.
//
// Network (Sec. 2.2, Eq. 2): encoder blocks e_1..e_L, decoder blocks d_{L-1}..d_1 with
// d_i = s_i(e_i, d_{i+1}), s_i = channel concatenation, softmax at the end; widths per level
// are given by the spec (Sec. 3: doubled per encoder block, decoder symmetric).  The output of
// encoder block l is used twice (Eq. 3 writes it as e_{l,0}, e_{l,1}): it is stored once, in
// channels [0, C_l) of level l's concat buffer, read by the down conv and by the decoder; its
// gradient is the sum of the two consumers' gradients, formed inside the norm-backward kernel.
#include <vector>
#include <new>
#include "common.cuh"

using namespace lamp;

enum { K_CONV = 0, K_DOWN = 1, K_UP = 2, K_HEAD = 3 };

struct Layer {
    int kind, level;            // level of the layer's OUTPUT
    int c_in, c_out, taps;
    size_t w_off, b_off;
    bool to_cat;                // output is E_l, written to the concat buffer slice [0, C_l)
    bool from_cat;              // input is the full concat buffer (2 C_l channels)
    // SEU-Net variant: the level's last conv ends in a squeeze-and-excitation residual step, out = r + e * z with
    // r = the output of the level's first conv (layer res_of).  se_cr > 0: hidden units; its fp32 parameters
    // W1 [cr][c], b1 [cr], W2 [c][cr], b2 [c] sit in the bias buffer from se_off.  The level's first conv then gets the
    // block output's gradient as a second gradient source (res_from = index of that last conv, else -1).
    int se_cr = 0;
    size_t se_off = 0;
    int res_of = -1;
    int res_from = -1;
};

struct lamp_unet {
    lamp_unet_spec_t spec;
    std::vector<Layer> layers;
    size_t n_w, n_b;
    // Host-side resources of the training step: a second stream on which the weight gradients (and the per-step
    // weight transposes) run beside the data-gradient chain, and the events that order the two.  Created on the
    // first training step on a device, destroyed with the handle.
    mutable int side_dev = -1;
    mutable cudaStream_t side = nullptr;
    mutable cudaEvent_t ev_fork = nullptr, ev_wt = nullptr, ev_dy = nullptr, ev_join = nullptr;
};

namespace {

struct Arena {
    char *base;
    size_t off;
    void *take(size_t bytes)
    {
        off = align_up(off, 256);
        void *p = base ? base + off : nullptr;
        off += bytes;
        return p;
    }
};

struct LayerBuf {
    TView in, out;              // activation views (out: normalised z / up output / unused for head)
    TView y;                    // raw conv output (norm layers)
    double *stats;              // [n][c_out][2]
    float *mr;                  // [n][c_out][2]
    double *bsums;              // InstanceNorm backward sums [n][c_out][2] (train mode)
    double *db_acc;             // bias-gradient totals [c_out] in fp64 and the ticket counter of their reduction
    unsigned *db_count;
    TView dy;                   // gradient w.r.t. the raw conv output (norm layers; train mode)
    TView din;                  // gradient w.r.t. the layer's input (train mode; empty for layer 0)
    TView dout, dout2;          // gradient w.r.t. the layer's output: main source and skip source (may be empty)
    ConvGeom g;
    lamp_conv_desc_t desc;
    // squeeze-and-excitation step of a level's last conv (SEU-Net variant)
    double *se_sums, *se_de;    // [n][c] fp64: sum_v z, sum_v dout * z
    float *se_e, *se_mean, *se_hid, *se_dsv;
    TView dsum, dz;             // train mode: dout + dout2 where the block output has two consumers; e * dout + ds / V
};

struct Plan {
    std::vector<LayerBuf> lb;
    std::vector<TView> cat, dcat;       // per level (levels - 1 entries)
    float *probs;                       // [V][K] when the caller gave none
    double *dice;                       // [n][K][3]
    void *bwd_pool;                     // per normalised layer: fp64 sums [n][c][2], fp64 db totals [c], ticket counter
    size_t bwd_pool_bytes;
    void *stats_pool;                   // fp64 [n][c_out][2] of every normalised layer, back to back
    size_t stats_pool_bytes;
    void *scratch;                      // conv workspace of the main chain (split-K partials, head backward)
    size_t scratch_bytes;
    void *scratch_side;                 // conv workspace of the weight-gradient passes (train mode)
    size_t scratch_side_bytes;
    std::vector<void *> wt;             // per layer: the weights as the data gradient reads them (train mode), or NULL
    std::vector<size_t> wt_bytes;
    size_t total;
};

TView view(void *p, int n, int d, int h, int w, int c, int64_t pitch, int c_off)
{
    TView v;
    v.p = p ? (char *)p + (size_t)c_off * 2 : nullptr;
    v.n = n; v.d = d; v.h = h; v.w = w; v.c = c; v.pitch = pitch; v.f32 = 0;
    return v;
}

lamp_conv_desc_t layer_desc(const Layer &L)
{
    lamp_conv_desc_t d;
    d.c_in = L.c_in; d.c_out = L.c_out;
    switch (L.kind) {
    case K_CONV: d.ksize = 3; d.stride = 1; d.pad = 1; d.transposed = 0; break;
    case K_DOWN: d.ksize = 3; d.stride = 2; d.pad = 1; d.transposed = 0; break;
    case K_UP:   d.ksize = 2; d.stride = 2; d.pad = 0; d.transposed = 1; break;
    default:     d.ksize = 1; d.stride = 1; d.pad = 0; d.transposed = 0; break;
    }
    return d;
}

// Lays every buffer of one pass out in the workspace (base may be NULL: sizing only).
void make_plan(const lamp_unet *net, void *base, const void *x_ptr, int64_t x_pitch, int n, int d, int h, int w,
               int mode, bool need_probs, Plan *P)
{
    const lamp_unet_spec_t &S = net->spec;
    Arena A{(char *)base, 0};
    const int L = S.levels;
    auto dd = [&](int l) { return d >> l; };
    auto hh = [&](int l) { return h >> l; };
    auto ww = [&](int l) { return w >> l; };
    auto vox = [&](int l) { return (size_t)n * dd(l) * hh(l) * ww(l); };
    P->cat.resize(L > 1 ? L - 1 : 0);
    P->dcat.resize(L > 1 ? L - 1 : 0);
    for (int l = 0; l + 1 < L; ++l) {
        void *p = A.take(vox(l) * 2 * S.channels[l] * sizeof(bf16));
        P->cat[l] = view(p, n, dd(l), hh(l), ww(l), 2 * S.channels[l], 2 * S.channels[l], 0);
    }
    size_t ymax = 0;
    for (const Layer &Ly : net->layers) {
        if (Ly.kind == K_CONV || Ly.kind == K_DOWN) ymax = ymax > vox(Ly.level) * Ly.c_out ? ymax : vox(Ly.level) * Ly.c_out;
    }
    bf16 *yshared = (mode == LAMP_MODE_INFER) ? (bf16 *)A.take(ymax * sizeof(bf16)) : nullptr;
    P->lb.resize(net->layers.size());
    size_t stats_total = 0;
    for (const Layer &Ly : net->layers)
        if (Ly.kind == K_CONV || Ly.kind == K_DOWN) stats_total += align_up((size_t)n * Ly.c_out * 2 * sizeof(double), 256);
    P->stats_pool = stats_total ? A.take(stats_total) : nullptr;
    P->stats_pool_bytes = stats_total;
    size_t stats_off = 0;
    TView cur = view((void *)x_ptr, n, d, h, w, S.in_channels, x_pitch, 0);
    size_t scratch = 0, scratch_side = 0;
    for (size_t i = 0; i < net->layers.size(); ++i) {
        const Layer &Ly = net->layers[i];
        LayerBuf &B = P->lb[i];
        const int l = Ly.level;
        B.in = cur;
        B.desc = layer_desc(Ly);
        B.stats = nullptr; B.mr = nullptr;
        B.y = TView{};
        {
            ConvGeom g;
            g.n = n; g.d = cur.d; g.h = cur.h; g.w = cur.w;
            g.od = dd(l); g.oh = hh(l); g.ow = ww(l);
            g.ci = Ly.c_in; g.co = Ly.c_out; g.k = B.desc.ksize; g.s = B.desc.stride; g.p = B.desc.pad;
            g.transposed = B.desc.transposed;
            B.g = g;
        }
        if (Ly.kind != K_HEAD) {
            const size_t s0 = conv_ws_bytes(B.g, LAMP_PASS_FWD);
            scratch = scratch > s0 ? scratch : s0;
        }
        if (mode == LAMP_MODE_TRAIN && Ly.kind == K_HEAD) {
            const size_t s3 = head_bwd_ws((int64_t)cur.d * cur.h * cur.w, n, S.num_classes, Ly.c_in);
            scratch = scratch > s3 ? scratch : s3;
        }
        if (mode == LAMP_MODE_TRAIN && Ly.kind != K_HEAD) {
            // the data gradient's transposed weights have their own per-layer buffers (below)
            const size_t s1 = conv_ws_bytes(B.g, LAMP_PASS_WGRAD);
            const size_t s2 = conv_ws_bytes(B.g, LAMP_PASS_DGRAD) - conv_ws_min_bytes(B.g, LAMP_PASS_DGRAD);
            scratch_side = scratch_side > s1 ? scratch_side : s1;
            scratch = scratch > s2 ? scratch : s2;
        }
        if (Ly.kind == K_CONV || Ly.kind == K_DOWN) {
            void *yp = yshared ? (void *)yshared : A.take(vox(l) * Ly.c_out * sizeof(bf16));
            B.y = view(yp, n, dd(l), hh(l), ww(l), Ly.c_out, Ly.c_out, 0);
            B.stats = P->stats_pool ? (double *)((char *)P->stats_pool + stats_off) : nullptr;
            stats_off += align_up((size_t)n * Ly.c_out * 2 * sizeof(double), 256);
            B.mr = (float *)A.take((size_t)n * Ly.c_out * 2 * sizeof(float));
            B.se_sums = nullptr; B.se_de = nullptr; B.se_e = nullptr; B.se_mean = nullptr; B.se_hid = nullptr; B.se_dsv = nullptr;
            if (Ly.se_cr) {
                B.se_sums = (double *)A.take((size_t)n * Ly.c_out * sizeof(double));
                B.se_de = (double *)A.take((size_t)n * Ly.c_out * sizeof(double));
                B.se_e = (float *)A.take((size_t)n * Ly.c_out * sizeof(float));
                B.se_mean = (float *)A.take((size_t)n * Ly.c_out * sizeof(float));
                B.se_dsv = (float *)A.take((size_t)n * Ly.c_out * sizeof(float));
                B.se_hid = (float *)A.take((size_t)n * Ly.se_cr * sizeof(float));
            }
            if (Ly.to_cat) {
                B.out = P->cat[l];
                B.out.c = Ly.c_out;                      // slice [0, C_l)
            } else {
                void *zp = A.take(vox(l) * Ly.c_out * sizeof(bf16));
                B.out = view(zp, n, dd(l), hh(l), ww(l), Ly.c_out, Ly.c_out, 0);
            }
            cur = B.out;
        } else if (Ly.kind == K_UP) {
            B.out = P->cat[l];
            B.out.p = B.out.p ? (char *)B.out.p + (size_t)Ly.c_out * 2 : nullptr;   // slice [C_l, 2 C_l)
            B.out.c = Ly.c_out;
            cur = P->cat[l];                             // the next conv reads all 2 C_l channels
        } else {
            B.out = TView{};
        }
    }
    const size_t V0 = vox(0);
    P->probs = need_probs ? (float *)A.take(V0 * S.num_classes * sizeof(float)) : nullptr;
    P->dice = nullptr; P->bwd_pool = nullptr; P->bwd_pool_bytes = 0;
    P->scratch = nullptr; P->scratch_bytes = 0;
    P->scratch_side = nullptr; P->scratch_side_bytes = 0;
    P->wt.assign(net->layers.size(), nullptr);
    P->wt_bytes.assign(net->layers.size(), 0);
    for (LayerBuf &B : P->lb) {
        B.dy = TView{}; B.din = TView{}; B.dout = TView{}; B.dout2 = TView{}; B.dsum = TView{}; B.dz = TView{};
        B.bsums = nullptr; B.db_acc = nullptr; B.db_count = nullptr;
    }
    if (mode == LAMP_MODE_TRAIN) {
        // Every gradient tensor gets its own buffer (nothing is recycled), so that each step of the
        // backward pass can be inspected after the call.
        P->dice = (double *)A.take((size_t)n * S.num_classes * 3 * sizeof(double));
        size_t pool = 0;
        for (const Layer &Ly : net->layers)
            if (Ly.kind == K_CONV || Ly.kind == K_DOWN)
                pool += align_up((size_t)n * Ly.c_out * 2 * sizeof(double), 256) + align_up((size_t)Ly.c_out * sizeof(double), 256) + 256;
        P->bwd_pool = A.take(pool);
        P->bwd_pool_bytes = pool;
        size_t poff = 0;
        for (size_t i = 0; i < net->layers.size(); ++i) {
            const Layer &Ly = net->layers[i];
            LayerBuf &B = P->lb[i];
            B.bsums = nullptr; B.db_acc = nullptr; B.db_count = nullptr;
            if (Ly.kind != K_CONV && Ly.kind != K_DOWN) continue;
            char *base = (char *)P->bwd_pool;
            B.bsums = base ? (double *)(base + poff) : nullptr;
            poff += align_up((size_t)n * Ly.c_out * 2 * sizeof(double), 256);
            B.db_acc = base ? (double *)(base + poff) : nullptr;
            poff += align_up((size_t)Ly.c_out * sizeof(double), 256);
            B.db_count = base ? (unsigned *)(base + poff) : nullptr;
            poff += 256;
        }
        for (int l = 0; l + 1 < L; ++l) {
            void *p = A.take(vox(l) * 2 * S.channels[l] * sizeof(bf16));
            P->dcat[l] = view(p, n, dd(l), hh(l), ww(l), 2 * S.channels[l], 2 * S.channels[l], 0);
        }
        TView g{};
        for (int i = (int)net->layers.size() - 1; i >= 0; --i) {
            const Layer &Ly = net->layers[i];
            LayerBuf &B = P->lb[i];
            B.dout = g;
            if (Ly.kind == K_CONV || Ly.kind == K_DOWN) {
                void *p = A.take(vox(Ly.level) * Ly.c_out * sizeof(bf16));
                B.dy = view(p, n, dd(Ly.level), hh(Ly.level), ww(Ly.level), Ly.c_out, Ly.c_out, 0);
                if (Ly.to_cat) {                        // E_l also fed the skip: slice [0, C_l) of dcat_l
                    B.dout2 = P->dcat[Ly.level];
                    B.dout2.c = Ly.c_out;
                }
                if (Ly.se_cr) {
                    void *pz = A.take(vox(Ly.level) * Ly.c_out * sizeof(bf16));
                    B.dz = view(pz, n, dd(Ly.level), hh(Ly.level), ww(Ly.level), Ly.c_out, Ly.c_out, 0);
                    if (Ly.to_cat) {
                        void *ps = A.take(vox(Ly.level) * Ly.c_out * sizeof(bf16));
                        B.dsum = view(ps, n, dd(Ly.level), hh(Ly.level), ww(Ly.level), Ly.c_out, Ly.c_out, 0);
                    }
                }
            } else if (Ly.kind == K_UP) {
                B.dy = g;                               // no norm / activation after the up conv
            }
            if (i == 0) break;                          // the network input needs no gradient
            if (Ly.from_cat) {
                B.din = P->dcat[Ly.level];              // all 2 C_l channels, kept for the encoder
                g = B.din;                              // the up conv's output gradient: slice [C_l, 2 C_l)
                g.p = g.p ? (char *)g.p + (size_t)(Ly.c_in / 2) * 2 : nullptr;
                g.c = Ly.c_in / 2;
            } else {
                void *p = A.take((size_t)B.in.n * B.in.d * B.in.h * B.in.w * Ly.c_in * sizeof(bf16));
                B.din = view(p, B.in.n, B.in.d, B.in.h, B.in.w, Ly.c_in, Ly.c_in, 0);
                g = B.din;
            }
        }
    }
    if (scratch) {
        P->scratch = A.take(scratch);
        P->scratch_bytes = scratch;
    }
    if (mode == LAMP_MODE_TRAIN) {
        if (scratch_side) {
            P->scratch_side = A.take(scratch_side);
            P->scratch_side_bytes = scratch_side;
        }
        for (size_t i = 1; i < net->layers.size(); ++i) {
            if (net->layers[i].kind == K_HEAD) continue;
            const size_t b = conv_ws_min_bytes(P->lb[i].g, LAMP_PASS_DGRAD);
            if (!b) continue;
            P->wt[i] = A.take(b);
            P->wt_bytes[i] = b;
        }
    }
    P->total = align_up(A.off, 256);
}

lamp_status_t check_input(const lamp_unet *net, const lamp_tensor_t *x)
{
    if (!net || !x || !x->ptr) return LAMP_ERR_INVALID_ARG;
    const lamp_unet_spec_t &S = net->spec;
    if (x->dtype != LAMP_BF16) return LAMP_ERR_UNSUPPORTED;
    if (x->c != S.in_channels || x->c_offset != 0 || x->c_pitch < x->c) return LAMP_ERR_INVALID_ARG;
    if (x->n <= 0 || x->d <= 0 || x->h <= 0 || x->w <= 0) return LAMP_ERR_INVALID_ARG;
    const int m = 1 << (S.levels - 1);
    if (x->d % m || x->h % m || x->w % m) return LAMP_ERR_UNSUPPORTED;
    if (((uintptr_t)x->ptr & 15) != 0) return LAMP_ERR_INVALID_ARG;
    return LAMP_OK;
}

#define TRY(expr)                                   \
    do {                                            \
        lamp_status_t s__ = (expr);                 \
        if (s__ != LAMP_OK) return s__;             \
    } while (0)

// layers [first, last) of the forward pass (the whole network by default)
lamp_status_t run_forward(const lamp_unet *net, const Plan &P, const bf16 *W, const float *Bv, float *probs,
                          uint8_t *argmax, const uint8_t *labels, double *dice, cudaStream_t st, size_t first = 0,
                          size_t last = (size_t)-1)
{
    const lamp_unet_spec_t &S = net->spec;
    if (last > net->layers.size()) last = net->layers.size();
    // the InstanceNorm sums of all layers sit in one pool: one memset clears them
    if (P.stats_pool_bytes) LAMP_CUDA_OK(cudaMemsetAsync(P.stats_pool, 0, P.stats_pool_bytes, st));
    for (size_t i = first; i < last; ++i) {
        const Layer &Ly = net->layers[i];
        const LayerBuf &B = P.lb[i];
        const bf16 *w = W + Ly.w_off;
        const float *b = Bv + Ly.b_off;
        if (Ly.se_cr) {
            // last conv of a level in the SEU-Net variant: out = r + e * relu(norm(y)), r = the output of the level's first conv
            TRY(conv_fwd(B.g, B.in, w, b, B.y, B.stats, P.scratch, P.scratch_bytes, st));
            TRY(k_mu_rstd(B.stats, (int64_t)B.y.d * B.y.h * B.y.w, S.in_eps, B.mr, B.y.n * Ly.c_out, st));
            TRY(k_se_fwd(B.y, B.mr, Bv + Ly.se_off, Ly.se_cr, B.se_sums, B.se_e, B.se_hid, B.se_mean, &P.lb[Ly.res_of].out, B.out, st));
        } else if (Ly.kind == K_CONV || Ly.kind == K_DOWN) {
            TRY(conv_fwd(B.g, B.in, w, b, B.y, B.stats, P.scratch, P.scratch_bytes, st));
            TRY(k_instnorm_relu_fwd(B.y, B.stats, S.in_eps, B.mr, B.out, st));
        } else if (Ly.kind == K_UP) {
            TRY(conv_fwd(B.g, B.in, w, b, B.out, nullptr, P.scratch, P.scratch_bytes, st));
        } else {
            TRY(k_head_softmax(B.in, w, b, S.num_classes, probs, argmax, labels, dice, st));
        }
    }
    return LAMP_OK;
}

void release_side(const lamp_unet *net)
{
    if (net->ev_fork) cudaEventDestroy(net->ev_fork);
    if (net->ev_wt) cudaEventDestroy(net->ev_wt);
    if (net->ev_dy) cudaEventDestroy(net->ev_dy);
    if (net->ev_join) cudaEventDestroy(net->ev_join);
    if (net->side) cudaStreamDestroy(net->side);
    net->ev_fork = net->ev_wt = net->ev_dy = net->ev_join = nullptr;
    net->side = nullptr;
    net->side_dev = -1;
}

// The side stream and its events on the current device; false if they cannot be had (the step then runs on one
// stream).  Creation is not allowed while the caller's stream is being captured, hence "first call before capture".
bool ensure_side(const lamp_unet *net)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (net->side && net->side_dev == dev) return true;
    release_side(net);
    bool ok = cudaStreamCreateWithFlags(&net->side, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&net->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&net->ev_wt, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&net->ev_dy, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&net->ev_join, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        release_side(net);
        return false;
    }
    net->side_dev = dev;
    return true;
}

}  // namespace

extern "C" {

lamp_status_t lamp_unet_create(const lamp_unet_spec_t *spec, lamp_unet_t **out)
{
    if (!spec || !out) return LAMP_ERR_INVALID_ARG;
    if (spec->levels < 1 || spec->levels > 8 || spec->convs_per_level < 1) return LAMP_ERR_INVALID_ARG;
    if (spec->num_classes < 2 || spec->num_classes > 16) return LAMP_ERR_UNSUPPORTED;
    if (spec->in_channels != 1 && (spec->in_channels <= 0 || spec->in_channels % 8)) return LAMP_ERR_UNSUPPORTED;
    for (int l = 0; l < spec->levels; ++l)
        if (spec->channels[l] <= 0 || spec->channels[l] % 8 || spec->channels[l] > 2048) return LAMP_ERR_UNSUPPORTED;
    if (spec->channels[0] > 128) return LAMP_ERR_UNSUPPORTED;          // the head's backward kernel keeps 256 voxels x channels[0] in shared memory
    if (!(spec->in_eps > 0.f)) return LAMP_ERR_INVALID_ARG;
    if (spec->se_ratio < 0) return LAMP_ERR_INVALID_ARG;
    // the residual branch of the squeeze-and-excitation block is the output of the level's first conv
    if (spec->se_ratio > 0 && spec->convs_per_level < 2) return LAMP_ERR_UNSUPPORTED;
    lamp_unet *net = new (std::nothrow) lamp_unet;
    if (!net) return LAMP_ERR_INVALID_ARG;
    net->spec = *spec;
    const int L = spec->levels;
    const int32_t *ch = spec->channels;
    size_t wo = 0, bo = 0;
    auto add = [&](int kind, int level, int ci, int co, int taps, bool to_cat, bool from_cat, bool se_last = false) {
        Layer y{kind, level, ci, co, taps, wo, bo, to_cat, from_cat};
        wo += (size_t)taps * ci * co;
        wo = (wo + 7) / 8 * 8;                  // keep every layer's weights 16-byte aligned
        bo += (size_t)co;
        if (se_last && spec->se_ratio > 0) {
            y.se_cr = co / spec->se_ratio > 0 ? co / spec->se_ratio : 1;
            y.se_off = bo;
            bo += (size_t)2 * co * y.se_cr + co + y.se_cr;
            y.res_of = (int)net->layers.size() - (spec->convs_per_level - 1);      // the level's first conv
            net->layers[y.res_of].res_from = (int)net->layers.size();
        }
        net->layers.push_back(y);
    };
    int c = spec->in_channels;
    for (int l = 0; l < L; ++l) {
        for (int j = 0; j < spec->convs_per_level; ++j) {
            add(K_CONV, l, c, ch[l], 27, j == spec->convs_per_level - 1 && l < L - 1, false, j == spec->convs_per_level - 1);
            c = ch[l];
        }
        if (l < L - 1) { add(K_DOWN, l + 1, ch[l], ch[l + 1], 27, false, false); c = ch[l + 1]; }
    }
    for (int l = L - 2; l >= 0; --l) {
        add(K_UP, l, ch[l + 1], ch[l], 8, false, false);
        c = 2 * ch[l];
        for (int j = 0; j < spec->convs_per_level; ++j) { add(K_CONV, l, c, ch[l], 27, false, j == 0, j == spec->convs_per_level - 1); c = ch[l]; }
    }
    add(K_HEAD, 0, ch[0], spec->num_classes, 1, false, false);
    net->n_w = wo;
    net->n_b = bo;
    *out = net;
    return LAMP_OK;
}

void lamp_unet_destroy(lamp_unet_t *net)
{
    if (!net) return;
    release_side(net);
    delete net;
}
int32_t lamp_unet_num_layers(const lamp_unet_t *net) { return net ? (int32_t)net->layers.size() : 0; }
size_t lamp_unet_weight_count(const lamp_unet_t *net) { return net ? net->n_w : 0; }
size_t lamp_unet_bias_count(const lamp_unet_t *net) { return net ? net->n_b : 0; }

lamp_status_t lamp_unet_se_layout(const lamp_unet_t *net, int32_t layer, size_t *se_off, int32_t *cr)
{
    if (!net || layer < 0 || layer >= (int32_t)net->layers.size() || !se_off || !cr) return LAMP_ERR_INVALID_ARG;
    *se_off = net->layers[layer].se_off;
    *cr = net->layers[layer].se_cr;
    return LAMP_OK;
}

lamp_status_t lamp_unet_param_layout(const lamp_unet_t *net, int32_t layer, size_t *w_off, size_t *b_off,
                                     lamp_conv_desc_t *desc)
{
    if (!net || layer < 0 || layer >= (int32_t)net->layers.size()) return LAMP_ERR_INVALID_ARG;
    const Layer &L = net->layers[layer];
    if (w_off) *w_off = L.w_off;
    if (b_off) *b_off = L.b_off;
    if (desc) *desc = layer_desc(L);
    return LAMP_OK;
}

size_t lamp_unet_workspace_bytes(const lamp_unet_t *net, int32_t n, int32_t d, int32_t h, int32_t w, int32_t mode)
{
    if (!net || n <= 0 || d <= 0 || h <= 0 || w <= 0) return 0;
    Plan P;
    make_plan(net, nullptr, nullptr, net->spec.in_channels, n, d, h, w, mode, true, &P);
    return P.total;
}

lamp_status_t lamp_unet_tensor_layout(const lamp_unet_t *net, int32_t n, int32_t d, int32_t h, int32_t w, int32_t mode,
                                      int32_t layer, int32_t which, lamp_tensor_t *out, size_t *offset)
{
    if (!net || !out || !offset || n <= 0 || d <= 0 || h <= 0 || w <= 0) return LAMP_ERR_INVALID_ARG;
    if (layer < 0 || layer >= (int32_t)net->layers.size()) return LAMP_ERR_INVALID_ARG;
    Plan P;
    char *const fake = (char *)(uintptr_t)(1ull << 40);          // offsets are measured from this base
    char *const fake_x = (char *)(uintptr_t)(1ull << 20);
    make_plan(net, fake, fake_x, net->spec.in_channels, n, d, h, w, mode, mode == LAMP_MODE_TRAIN, &P);
    const LayerBuf &B = P.lb[layer];
    TView v{};
    int f32 = 0, f64 = 0;
    switch (which) {
    case LAMP_T_IN: v = B.in; break;
    case LAMP_T_Y: v = B.y; break;
    case LAMP_T_OUT: v = B.out; break;
    case LAMP_T_DY: v = B.dy; break;
    case LAMP_T_DIN: v = B.din; break;
    case LAMP_T_DOUT: v = B.dout; break;
    case LAMP_T_DOUT2: v = B.dout2; break;
    case LAMP_T_MU_RSTD:
        if (B.mr) { v.p = B.mr; v.n = n; v.d = v.h = v.w = 1; v.c = 2 * B.g.co; v.pitch = v.c; f32 = 1; }
        break;
    case LAMP_T_STATS:
        if (B.stats) { v.p = B.stats; v.n = n; v.d = v.h = v.w = 1; v.c = 2 * B.g.co; v.pitch = v.c; f64 = 1; }
        break;
    case LAMP_T_PROBS:
        v.p = P.probs; v.n = n; v.d = d; v.h = h; v.w = w; v.c = net->spec.num_classes; v.pitch = v.c; f32 = 1;
        break;
    default: return LAMP_ERR_INVALID_ARG;
    }
    if (!v.p) return LAMP_ERR_UNSUPPORTED;                        // this layer / mode has no such tensor
    if ((char *)v.p < fake) return LAMP_ERR_UNSUPPORTED;          // the network input lives in the caller's buffer
    out->ptr = nullptr;
    out->dtype = f32 ? LAMP_F32 : LAMP_BF16;
    out->n = v.n; out->d = v.d; out->h = v.h; out->w = v.w; out->c = v.c;
    out->c_pitch = v.pitch;
    out->c_offset = 0;
    *offset = (size_t)((char *)v.p - fake);
    (void)f64;
    return LAMP_OK;
}

lamp_status_t lamp_unet_forward(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                const lamp_tensor_t *x, float *probs, uint8_t *argmax,
                                void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!weights_bf16 || !biases_f32) return LAMP_ERR_INVALID_ARG;
    TRY(check_input(net, x));
    if (!ws || ((uintptr_t)ws & 255)) return LAMP_ERR_WORKSPACE;
    Plan P;
    make_plan(net, ws, x->ptr, x->c_pitch, x->n, x->d, x->h, x->w, LAMP_MODE_INFER, false, &P);
    if (P.total > ws_bytes) return LAMP_ERR_WORKSPACE;
    return run_forward(net, P, (const bf16 *)weights_bf16, biases_f32, probs, argmax, nullptr, nullptr,
                       (cudaStream_t)cuda_stream);
}

// bucket_start / bucket_events: see lamp_unet_train_step_buckets (n_buckets = 0: none)
static lamp_status_t train_step_impl(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                     const lamp_tensor_t *x, const uint8_t *labels, float *loss,
                                     float *grad_w, float *grad_b, float *probs,
                                     void *ws, size_t ws_bytes, void *cuda_stream,
                                     const int64_t *bucket_start, int32_t n_buckets, void *const *bucket_events)
{
    if (!weights_bf16 || !biases_f32 || !labels || !loss || !grad_w || !grad_b) return LAMP_ERR_INVALID_ARG;
    TRY(check_input(net, x));
    if (n_buckets < 0 || (n_buckets > 0 && (!bucket_start || !bucket_events))) return LAMP_ERR_INVALID_ARG;
    for (int b = 0; b < n_buckets; ++b) {
        if (!bucket_events[b] || bucket_start[b] < 0 || (size_t)bucket_start[b] >= net->n_w) return LAMP_ERR_INVALID_ARG;
        if (b == 0 ? bucket_start[0] != 0 : bucket_start[b] <= bucket_start[b - 1]) return LAMP_ERR_INVALID_ARG;
    }
    if (!ws || ((uintptr_t)ws & 255)) return LAMP_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const lamp_unet_spec_t &S = net->spec;
    Plan P;
    make_plan(net, ws, x->ptr, x->c_pitch, x->n, x->d, x->h, x->w, LAMP_MODE_TRAIN, true, &P);
    if (P.total > ws_bytes) return LAMP_ERR_WORKSPACE;
    const bf16 *W = (const bf16 *)weights_bf16;
    if (!probs) probs = P.probs;
    // Two streams.  The caller's stream carries the chain forward pass -> loss -> InstanceNorm backward / data
    // gradient, layer by layer.  The side stream carries what nothing in that chain waits for: first the per-step
    // transposes of the weights the data gradients read (beside the forward pass), then every weight gradient as soon
    // as its dy exists - tensor-core work that runs beside the HBM-bound InstanceNorm backward of the next layer and
    // fills the SMs the small deep-level kernels leave idle.  The side stream starts after everything the caller
    // enqueued before this call and is joined before the call returns.
    const bool two = ensure_side(net);
    const cudaStream_t sd = two ? net->side : st;
    if (two) {
        LAMP_CUDA_OK(cudaEventRecord(net->ev_fork, st));
        LAMP_CUDA_OK(cudaStreamWaitEvent(sd, net->ev_fork, 0));
    }
    lamp_status_t rs = LAMP_OK;
    // Buckets of grad_w whose last contribution has been enqueued get their event recorded: the layers are visited
    // last to first and their weights lie in layer order, so once the layer at offset `done_from` is enqueued every
    // bucket that starts at or behind it is final.  The weight gradients run on the side stream (the head's on the
    // caller's stream: `on_main`), so that is where the events go.
    int buckets_left = n_buckets;
    auto mark_final = [&](size_t done_from, bool on_main) -> lamp_status_t {
        if (buckets_left == 0 || (size_t)bucket_start[buckets_left - 1] < done_from) return LAMP_OK;
        if (on_main && two) {
            LAMP_CUDA_OK(cudaEventRecord(net->ev_dy, st));
            LAMP_CUDA_OK(cudaStreamWaitEvent(sd, net->ev_dy, 0));
        }
        while (buckets_left > 0 && (size_t)bucket_start[buckets_left - 1] >= done_from) {
            LAMP_CUDA_OK(cudaEventRecord((cudaEvent_t)bucket_events[buckets_left - 1], sd));
            --buckets_left;
        }
        return LAMP_OK;
    };
    auto body = [&]() -> lamp_status_t {
        for (size_t i = 1; i < net->layers.size(); ++i) {
            if (net->layers[i].kind == K_HEAD) continue;
            const LayerBuf &B = P.lb[i];
            TRY(conv_dgrad_prepare(B.g, B.dy, B.din, W + net->layers[i].w_off, P.wt[i], P.wt_bytes[i], sd));
        }
        if (two) LAMP_CUDA_OK(cudaEventRecord(net->ev_wt, sd));
        TRY(run_forward(net, P, W, biases_f32, probs, nullptr, labels, P.dice, st));
        TRY(k_dice_loss(P.dice, x->n, S.num_classes, loss, st));

        // backward, last layer first; one memset clears every layer's reduction scratch
        LAMP_CUDA_OK(cudaMemsetAsync(P.bwd_pool, 0, P.bwd_pool_bytes, st));
        if (two) LAMP_CUDA_OK(cudaStreamWaitEvent(st, net->ev_wt, 0));
        for (int i = (int)net->layers.size() - 1; i >= 0; --i) {
            const Layer &Ly = net->layers[i];
            const LayerBuf &B = P.lb[i];
            const bf16 *w = W + Ly.w_off;
            float *dw = grad_w + Ly.w_off, *db = grad_b + Ly.b_off;
            if (Ly.kind == K_HEAD) {
                TRY(k_head_bwd(B.in, w, S.num_classes, probs, labels, P.dice, B.din, dw, db, nullptr, P.scratch, P.scratch_bytes, st));
                TRY(mark_final(Ly.w_off, true));
                continue;
            }
            if (Ly.se_cr) {
                // gradient of the block output (both consumers where it also fed the skip), through the
                // squeeze-and-excitation step to dz, then the InstanceNorm backward of this conv
                const TView *src = &B.dout;
                if (Ly.to_cat) { TRY(k_add2(B.dout, B.dout2, B.dsum, st)); src = &B.dsum; }
                TRY(k_se_bwd(*src, B.y, B.mr, biases_f32 + Ly.se_off, Ly.se_cr, B.se_e, B.se_hid, B.se_mean, B.se_de, B.se_dsv,
                             grad_b + Ly.se_off, B.dz, st));
                TRY(k_instnorm_relu_bwd(B.dz, nullptr, B.y, B.mr, B.bsums, true, B.dy, B.db_acc, B.db_count, db, st));
            } else if (Ly.kind != K_UP) {
                // (the first conv of a squeeze-and-excitation level also receives the block output's gradient: the residual)
                const TView *second = Ly.to_cat ? &B.dout2 : nullptr;
                if (Ly.res_from >= 0) {
                    const LayerBuf &R = P.lb[Ly.res_from];
                    second = net->layers[Ly.res_from].to_cat ? &R.dsum : &R.dout;
                }
                TRY(k_instnorm_relu_bwd(B.dout, second, B.y, B.mr, B.bsums, true, B.dy, B.db_acc, B.db_count, db, st));
            }
            // dy is complete on the caller's stream: the weight gradient starts from here on the side stream (the
            // bias gradient of a normalised layer came out of the InstanceNorm backward kernel above)
            if (two) {
                LAMP_CUDA_OK(cudaEventRecord(net->ev_dy, st));
                LAMP_CUDA_OK(cudaStreamWaitEvent(sd, net->ev_dy, 0));
            }
            TRY(conv_wgrad(B.g, B.in, B.dy, dw, Ly.kind == K_UP ? db : nullptr, P.scratch_side, P.scratch_side_bytes, sd));
            TRY(mark_final(Ly.w_off, false));
            if (i == 0) break;
            TRY(conv_dgrad_run(B.g, B.dy, w, P.wt[i], B.din, P.scratch, P.scratch_bytes, st));
        }
        return LAMP_OK;
    };
    rs = body();
    if (two) {
        // joined on every path, so that a stream capture of the caller never ends with the side stream still forked
        const bool j = cudaEventRecord(net->ev_join, sd) == cudaSuccess && cudaStreamWaitEvent(st, net->ev_join, 0) == cudaSuccess;
        if (!j && rs == LAMP_OK) rs = LAMP_ERR_CUDA;
    }
    return rs;
}

lamp_status_t lamp_unet_forward_layers(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                       const lamp_tensor_t *x, int32_t first_layer, int32_t last_layer,
                                       float *probs, uint8_t *argmax, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!weights_bf16 || !biases_f32) return LAMP_ERR_INVALID_ARG;
    TRY(check_input(net, x));
    if (first_layer < 0 || last_layer <= first_layer || last_layer > (int32_t)net->layers.size()) return LAMP_ERR_INVALID_ARG;
    if (!ws || ((uintptr_t)ws & 255)) return LAMP_ERR_WORKSPACE;
    Plan P;
    make_plan(net, ws, x->ptr, x->c_pitch, x->n, x->d, x->h, x->w, LAMP_MODE_INFER, false, &P);
    if (P.total > ws_bytes) return LAMP_ERR_WORKSPACE;
    return run_forward(net, P, (const bf16 *)weights_bf16, biases_f32, probs, argmax, nullptr, nullptr,
                       (cudaStream_t)cuda_stream, (size_t)first_layer, (size_t)last_layer);
}

lamp_status_t lamp_unet_train_step(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                   const lamp_tensor_t *x, const uint8_t *labels, float *loss,
                                   float *grad_w, float *grad_b, float *probs,
                                   void *ws, size_t ws_bytes, void *cuda_stream)
{
    return train_step_impl(net, weights_bf16, biases_f32, x, labels, loss, grad_w, grad_b, probs, ws, ws_bytes, cuda_stream,
                           nullptr, 0, nullptr);
}

lamp_status_t lamp_unet_train_step_buckets(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                           const lamp_tensor_t *x, const uint8_t *labels, float *loss,
                                           float *grad_w, float *grad_b, float *probs,
                                           void *ws, size_t ws_bytes, void *cuda_stream,
                                           const int64_t *bucket_start, int32_t n_buckets, void *const *bucket_events)
{
    return train_step_impl(net, weights_bf16, biases_f32, x, labels, loss, grad_w, grad_b, probs, ws, ws_bytes, cuda_stream,
                           bucket_start, n_buckets, bucket_events);
}

static void window_grid(int len, int patch, float overlap, int32_t *nst, int32_t *stride)
{
    int s = (int)lrintf(patch * (1.0f - overlap));
    if (s < 1) s = 1;
    const int last = len > patch ? len - patch : 0;
    int n = last / s + 1;
    if ((n - 1) * s != last) ++n;
    *nst = n;
    *stride = s;
}

static lamp_status_t sw_check(const lamp_unet_t *net, int d, int h, int w, const int32_t patch[3], float overlap,
                              int sw_batch)
{
    if (!net || !patch || sw_batch < 1 || !(overlap >= 0.f && overlap < 1.f)) return LAMP_ERR_INVALID_ARG;
    const int dims[3] = {d, h, w};
    const int m = 1 << (net->spec.levels - 1);
    for (int a = 0; a < 3; ++a) {
        if (patch[a] <= 0 || patch[a] > dims[a]) return LAMP_ERR_INVALID_ARG;
        if (patch[a] % m) return LAMP_ERR_UNSUPPORTED;
        if (patch[a] > 1024) return LAMP_ERR_UNSUPPORTED;
    }
    return LAMP_OK;
}

size_t lamp_sliding_window_workspace_bytes(const lamp_unet_t *net, int32_t d, int32_t h, int32_t w,
                                           const int32_t patch[3], float overlap, int32_t sw_batch)
{
    if (sw_check(net, d, h, w, patch, overlap, sw_batch) != LAMP_OK) return 0;
    int32_t nst[3], str[3];
    window_grid(d, patch[0], overlap, &nst[0], &str[0]);
    window_grid(h, patch[1], overlap, &nst[1], &str[1]);
    window_grid(w, patch[2], overlap, &nst[2], &str[2]);
    const size_t np = (size_t)nst[0] * nst[1] * nst[2];
    const size_t pv = (size_t)patch[0] * patch[1] * patch[2];
    size_t total = align_up(np * pv * net->spec.num_classes * sizeof(float), 256);
    total += align_up((size_t)sw_batch * pv * net->spec.in_channels * sizeof(bf16), 256);
    total += lamp_unet_workspace_bytes(net, sw_batch, patch[0], patch[1], patch[2], LAMP_MODE_INFER);
    return total;
}

// Patches first_patch .. first_patch + num_patches - 1 of the grid (num_patches < 0: all of them): forward pass of each,
// then the blend.  wsum == NULL: normalised probabilities and arg max; otherwise the un-normalised sums and weight totals
// of these patches alone.
static lamp_status_t sliding_window_run(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                        const lamp_tensor_t *volume, const int32_t patch[3], float overlap,
                                        int32_t sw_batch, int32_t window, int32_t first_patch, int32_t num_patches,
                                        float *probs_planar, float *wsum, uint8_t *argmax,
                                        void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!weights_bf16 || !biases_f32 || !volume || !volume->ptr) return LAMP_ERR_INVALID_ARG;
    if (volume->n != 1 || volume->dtype != LAMP_BF16 || volume->c != (net ? net->spec.in_channels : 0)) return LAMP_ERR_INVALID_ARG;
    TRY(sw_check(net, volume->d, volume->h, volume->w, patch, overlap, sw_batch));
    if (!ws || ((uintptr_t)ws & 255)) return LAMP_ERR_WORKSPACE;
    if (ws_bytes < lamp_sliding_window_workspace_bytes(net, volume->d, volume->h, volume->w, patch, overlap, sw_batch))
        return LAMP_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const lamp_unet_spec_t &S = net->spec;
    int32_t nst[3], str[3];
    window_grid(volume->d, patch[0], overlap, &nst[0], &str[0]);
    window_grid(volume->h, patch[1], overlap, &nst[1], &str[1]);
    window_grid(volume->w, patch[2], overlap, &nst[2], &str[2]);
    const int np = nst[0] * nst[1] * nst[2];
    if (num_patches < 0) { first_patch = 0; num_patches = np; }
    if (first_patch < 0 || first_patch + num_patches > np) return LAMP_ERR_INVALID_ARG;
    const size_t pv = (size_t)patch[0] * patch[1] * patch[2];
    char *p = (char *)ws;
    float *pprobs = (float *)p;
    p += align_up((size_t)np * pv * S.num_classes * sizeof(float), 256);
    bf16 *pin = (bf16 *)p;
    p += align_up((size_t)sw_batch * pv * S.in_channels * sizeof(bf16), 256);
    void *nws = p;
    TView vol = make_view(volume);
    const int end = first_patch + num_patches;
    for (int first = first_patch; first < end; first += sw_batch) {
        const int b = end - first < sw_batch ? end - first : sw_batch;
        TView pt = view(pin, b, patch[0], patch[1], patch[2], S.in_channels, S.in_channels, 0);
        TRY(k_gather_patches(vol, pt, first, nst, str, st));
        Plan P;
        make_plan(net, nws, pin, S.in_channels, b, patch[0], patch[1], patch[2], LAMP_MODE_INFER, false, &P);
        TRY(run_forward(net, P, (const bf16 *)weights_bf16, biases_f32, pprobs + (size_t)(first - first_patch) * pv * S.num_classes,
                        nullptr, nullptr, nullptr, st));
    }
    return k_overlap_add(pprobs, S.num_classes, volume->d, volume->h, volume->w, patch, nst, str, window,
                         probs_planar, argmax, st, first_patch, num_patches, wsum);
}

lamp_status_t lamp_sliding_window_infer(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                        const lamp_tensor_t *volume, const int32_t patch[3], float overlap,
                                        int32_t sw_batch, int32_t window, float *probs_planar, uint8_t *argmax,
                                        void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!argmax && !probs_planar) return LAMP_ERR_INVALID_ARG;
    return sliding_window_run(net, weights_bf16, biases_f32, volume, patch, overlap, sw_batch, window, 0, -1, probs_planar,
                              nullptr, argmax, ws, ws_bytes, cuda_stream);
}

int32_t lamp_sliding_window_num_patches(int32_t d, int32_t h, int32_t w, const int32_t patch[3], float overlap)
{
    if (!patch || !(overlap >= 0.f && overlap < 1.f)) return 0;
    const int dims[3] = {d, h, w};
    int n = 1;
    for (int a = 0; a < 3; ++a) {
        if (patch[a] <= 0 || patch[a] > dims[a]) return 0;
        int32_t nst, str;
        window_grid(dims[a], patch[a], overlap, &nst, &str);
        n *= nst;
    }
    return n;
}

lamp_status_t lamp_sliding_window_partial(const lamp_unet_t *net, const void *weights_bf16, const float *biases_f32,
                                          const lamp_tensor_t *volume, const int32_t patch[3], float overlap,
                                          int32_t sw_batch, int32_t window, int32_t first_patch, int32_t num_patches,
                                          float *sums_planar, float *weight_sums, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!sums_planar || !weight_sums || num_patches < 0) return LAMP_ERR_INVALID_ARG;
    if (((uintptr_t)sums_planar | (uintptr_t)weight_sums) & 15) return LAMP_ERR_INVALID_ARG;
    return sliding_window_run(net, weights_bf16, biases_f32, volume, patch, overlap, sw_batch, window, first_patch, num_patches,
                              sums_planar, weight_sums, nullptr, ws, ws_bytes, cuda_stream);
}

lamp_status_t lamp_sliding_window_finish(float *sums_planar, const float *weight_sums, int32_t k, int64_t voxels,
                                         int32_t write_probs, uint8_t *argmax, void *cuda_stream)
{
    if (!sums_planar || !weight_sums || voxels < 0 || (!write_probs && !argmax)) return LAMP_ERR_INVALID_ARG;
    return k_overlap_finish(sums_planar, weight_sums, k, voxels, write_probs, argmax, (cudaStream_t)cuda_stream);
}

lamp_status_t lamp_overlap_add(const float *patch_probs, int32_t k, int32_t d, int32_t h, int32_t w,
                               const int32_t patch[3], float overlap, int32_t window,
                               float *probs_planar, uint8_t *argmax, void *cuda_stream)
{
    if (!patch_probs || !patch || d <= 0 || h <= 0 || w <= 0 || (!probs_planar && !argmax)) return LAMP_ERR_INVALID_ARG;
    if (!(overlap >= 0.f && overlap < 1.f)) return LAMP_ERR_INVALID_ARG;
    const int dims[3] = {d, h, w};
    int32_t nst[3], str[3];
    for (int a = 0; a < 3; ++a) {
        if (patch[a] <= 0 || patch[a] > dims[a] || patch[a] > 1024) return LAMP_ERR_INVALID_ARG;
        window_grid(dims[a], patch[a], overlap, &nst[a], &str[a]);
    }
    return k_overlap_add(patch_probs, k, d, h, w, patch, nst, str, window, probs_planar, argmax,
                         (cudaStream_t)cuda_stream);
}

}  // extern "C"
