// C ABI: context, convolution entry points, and the training step over a layer list.
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.h"

using namespace b2c;

// Default L2 budget (MB) for the largest tensor of a layer per launch inside b2c_train_step; 0 = whole passes.
#ifndef B2C_DEFAULT_CHUNK_MB
#define B2C_DEFAULT_CHUNK_MB 0
#endif

extern "C" {

b2c_status b2c_create(b2c_ctx** out, int device)
{
    if (!out) return B2C_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return B2C_ERR_CUDA;
    cudaDeviceProp prop;
    B2C_CUDA(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return B2C_ERR_ARCH;
    B2C_CUDA(cudaSetDevice(device));
    b2c_ctx* ctx = new (std::nothrow) b2c_ctx();
    if (!ctx) return B2C_ERR_CUDA;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->spin_limit = 1u << 22;
    ctx->stall_counters = nullptr;
    ctx->smem_optin_done = 0u;
    {
        const char* env = std::getenv("B2C_CTA_PAIRS");
        ctx->use_pairs = env ? (env[0] == '3' ? 3 : env[0] == '2' ? 2 : env[0] == '1' ? 1 : 0) : 1;   // 0 never, 1 for 3x3 stride-1 layers with tiles of 128 channels or more (default), 2 wherever possible, 3 for 128-channel tiles only
    }
    {
        const char* env = std::getenv("B2C_FULL_HALO");
        ctx->use_full_halo = env ? (env[0] != '0') : 1;
    }
    {
        const char* env = std::getenv("B2C_WGRAD_FRAME");
        ctx->use_wgrad_frame = env ? (env[0] != '0') : 1;
    }
    {
        const char* env = std::getenv("B2C_ISSUE_SPLIT");
        ctx->use_issue_split = env ? (env[0] != '0') : 1;
    }
    {
        const char* env = std::getenv("B2C_PDL");
        ctx->use_pdl = env ? (env[0] != '0') : 1;
    }
    {
        const char* env = std::getenv("B2C_HMERGE");
        ctx->use_hmerge = env ? (env[0] != '0') : 1;
    }
    {
        const char* env = std::getenv("B2C_GROUP_KBLOCKS");
        ctx->use_group_kblocks = env ? (env[0] != '0') : 1;
    }
    {
        const char* env = std::getenv("B2C_WGRAD_ISSUERS");
        ctx->use_wgrad_two_issuers = env ? (env[0] != '1') : 1;   // B2C_WGRAD_ISSUERS=1: one issuing thread
    }
    {
        const char* env = std::getenv("B2C_BN_GROUPED");
        ctx->use_bn_grouped = env ? (env[0] != '0') : 0;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr ||
        qres != cudaDriverEntryPointSuccess) {
        delete ctx;
        return B2C_ERR_CUDA;
    }
    ctx->encode_tiled = reinterpret_cast<b2c_encode_tiled_fn>(fn);
    if (cudaMalloc(&ctx->d_status, sizeof(unsigned)) != cudaSuccess || cudaMemset(ctx->d_status, 0, sizeof(unsigned)) != cudaSuccess) {
        delete ctx;
        return B2C_ERR_CUDA;
    }
    *out = ctx;
    return B2C_OK;
}

void b2c_destroy(b2c_ctx* ctx)
{
    if (!ctx) return;
    cudaFree(ctx->d_status);
    delete ctx;
}

const char* b2c_status_string(b2c_status s)
{
    switch (s) {
        case B2C_OK: return "ok";
        case B2C_ERR_INVALID_ARG: return "invalid argument";
        case B2C_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case B2C_ERR_MISALIGNED: return "misaligned pointer";
        case B2C_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case B2C_ERR_CUDA: return "CUDA runtime or driver error";
        case B2C_ERR_ARCH: return "device is not compute capability 10.x";
        case B2C_ERR_DEVICE_TIMEOUT: return "a device-side wait exhausted its spin budget";
        case B2C_ERR_BAD_LABEL: return "label outside [0, classes)";
    }
    return "unknown status";
}

b2c_status b2c_get_device_status(b2c_ctx* ctx, void* stream)
{
    if (!ctx) return B2C_ERR_INVALID_ARG;
    unsigned word = 0;
    B2C_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    B2C_CUDA(cudaMemcpy(&word, ctx->d_status, sizeof(word), cudaMemcpyDeviceToHost));
    if (word) B2C_CUDA(cudaMemset(ctx->d_status, 0, sizeof(word)));
    if (word & B2C_DEV_TIMEOUT) return B2C_ERR_DEVICE_TIMEOUT;
    if (word & B2C_DEV_BAD_LABEL) return B2C_ERR_BAD_LABEL;
    return B2C_OK;
}

void b2c_set_stall_counters(b2c_ctx* ctx, unsigned long long* counters) { if (ctx) ctx->stall_counters = counters; }

void b2c_set_spin_limit(b2c_ctx* ctx, unsigned limit)
{
    if (ctx && limit > 0) ctx->spin_limit = limit;
}

// ------------------------------------------------------------------------------ convolution
static b2c_status check_desc(const b2c_conv_desc* d, int* p, int* q)
{
    if (!d) return B2C_ERR_INVALID_ARG;
    if (d->n < 1 || d->h < 1 || d->w < 1 || d->c < 1 || d->k < 1) return B2C_ERR_INVALID_ARG;
    if (d->r != d->s || !(d->r == 1 || d->r == 3) || !(d->stride == 1 || d->stride == 2) || d->pad != (d->r - 1) / 2)
        return B2C_ERR_UNSUPPORTED_SHAPE;
    *p = (d->h + 2 * d->pad - d->r) / d->stride + 1;
    *q = (d->w + 2 * d->pad - d->s) / d->stride + 1;
    if (*p * d->stride != d->h || *q * d->stride != d->w) return B2C_ERR_UNSUPPORTED_SHAPE;
    return B2C_OK;
}

size_t b2c_conv2d_workspace_bytes(const b2c_conv_desc* d, int which)
{
    (void)d; (void)which;
    return 0;   // forward, data gradient and weight gradient keep everything they need in shared memory and TMEM
}

b2c_status b2c_conv2d_fwd(b2c_ctx* ctx, const b2c_conv_desc* d, const void* x, const void* w_krsc, void* y, int y_is_f32, const float* bias,
                          double* ch_stats, void* stream)
{
    if (!ctx || !x || !w_krsc || !y) return B2C_ERR_INVALID_ARG;
    int p, q;
    b2c_status st = check_desc(d, &p, &q);
    if (st != B2C_OK) return st;
    if (ch_stats && y_is_f32) return B2C_ERR_INVALID_ARG;
    KMajorProblem pb{};
    pb.n = d->n; pb.ih = d->h; pb.iw = d->w; pb.ic = d->c;
    pb.oh = p; pb.ow = q; pb.oc = d->k;
    pb.r = d->r; pb.stride = d->stride; pb.pad = d->pad;
    pb.dgrad = false;
    pb.in = x; pb.wt = w_krsc; pb.out = y;
    pb.out_f32 = y_is_f32 != 0; pb.bias = bias; pb.stats = ch_stats;
    return launch_conv_kmajor(ctx, pb, (cudaStream_t)stream);
}

b2c_status b2c_conv2d_dgrad(b2c_ctx* ctx, const b2c_conv_desc* d, const void* dy, const void* w_crsk_flipped, void* dx, void* stream)
{
    if (!ctx || !dy || !w_crsk_flipped || !dx) return B2C_ERR_INVALID_ARG;
    int p, q;
    b2c_status st = check_desc(d, &p, &q);
    if (st != B2C_OK) return st;
    KMajorProblem pb{};
    pb.n = d->n; pb.ih = p; pb.iw = q; pb.ic = d->k;
    pb.oh = d->h; pb.ow = d->w; pb.oc = d->c;
    pb.r = d->r; pb.stride = d->stride; pb.pad = d->pad;
    pb.dgrad = true;
    pb.in = dy; pb.wt = w_crsk_flipped; pb.out = dx;
    pb.out_f32 = false; pb.bias = nullptr; pb.stats = nullptr;
    return launch_conv_kmajor(ctx, pb, (cudaStream_t)stream);
}

b2c_status b2c_conv2d_wgrad(b2c_ctx* ctx, const b2c_conv_desc* d, const void* dy, const void* x, float* dw_krsc, int accumulate, void* stream)
{
    if (!ctx || !dy || !x || !dw_krsc) return B2C_ERR_INVALID_ARG;
    int p, q;
    b2c_status st = check_desc(d, &p, &q);
    if (st != B2C_OK) return st;
    WgradProblem pb{};
    pb.n = d->n; pb.h = d->h; pb.w = d->w; pb.c = d->c;
    pb.p = p; pb.q = q; pb.k = d->k;
    pb.r = d->r; pb.stride = d->stride; pb.pad = d->pad;
    pb.dy = dy; pb.x = x; pb.dw = dw_krsc;
    // everything the launcher would reject is rejected here, before anything is enqueued
    if (d->c < 16 || d->c % 16 || d->k < 16 || d->k % 16) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_is_pow2(p) || !b2c_is_pow2(q) || p > 128 || q > 128) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(dy) || !b2c_aligned16(x) || !b2c_aligned16(dw_krsc)) return B2C_ERR_MISALIGNED;
    if (!accumulate) B2C_CUDA(cudaMemsetAsync(dw_krsc, 0, sizeof(float) * (size_t)d->k * d->r * d->s * d->c, (cudaStream_t)stream));
    return launch_conv_wgrad(ctx, pb, (cudaStream_t)stream);
}

}  // extern "C"

// ------------------------------------------------------------------------------ layer list
namespace {

struct TensorPlan {
    int n = 0, h = 1, w = 1, c = 0;  // c = stored (padded) channels
    bool f32 = false;
    bool exists = false;
    long long act_off = -1;        // bytes into the workspace (-1 for tensor 0 when it is read in place)
    long long stats_off = -1;      // fp64 [groups][2c] sum / sum of squares, for convolution outputs
    bool fused_stats = false;      // the producing convolution accumulates them in its epilogue
    long long grad_off[2] = {-1, -1};
    int n_contrib = 0;             // gradient contributions expected
    int producer = -1;             // layer index
    size_t elems() const { return (size_t)n * h * w * c; }
};

struct LayerPlan {
    b2c_layer_desc d;
    int c_pad = 0, k_pad = 0;      // stored input / output channels of conv and fc layers
    int gemm_r = 0;                // filter size the convolution kernels see (1 for the patch-matrix stem)
    int p = 0, q = 0;
    long long w_off = -1, gamma_off = -1, beta_off = -1, bias_off = -1;   // elements into the flat parameter arrays
    long long mean_off = -1, invstd_off = -1, bwd_ws_off = -1, mask_off = -1, arrive_off = -1;   // bytes into the workspace
    long long run_off = -1;                                                // elements into the running-statistics array
    int src_slot = -1, res_slot = -1;                                     // which gradient buffer of src / res this layer writes
    int chunk_groups = 1;          // micro-batches of a pass this layer takes per launch (divides n_conc)
    int seg_index = -1;            // position of this layer's filter bank among the weight layers (conv, fc)
};

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

}  // namespace

struct b2c_net {
    b2c_ctx* ctx = nullptr;
    int micro_batch = 0;
    int n_conc = 1;            // micro-batches processed side by side in one pass
    int image_h = 0, image_w = 0, image_c = 0, image_c_pad = 0;
    bool stem_im2col = false;   // the first convolution runs as a 1x1 GEMM on the 3x3 patch matrix of the images
    std::vector<LayerPlan> layers;
    std::vector<TensorPlan> tensors;
    std::vector<b2c_weight_seg> segs;
    size_t param_count = 0;
    size_t ws_bytes = 0;
    long long stats_begin = 0, stats_end = 0;   // fp64 region zeroed before every forward pass
    float *w = nullptr, *v = nullptr, *g = nullptr;
    char *w_bf16 = nullptr, *w_dgrad = nullptr, *ws = nullptr;
    bool fuse_stats = true;
    // optional per-launch timing (CUDA events on the step's stream), summed per kernel family
    bool profile = false;
    struct Span { cudaEvent_t a, b; int kind, layer, pass; };   // layer -1: not a layer's launch site; pass 0 forward, 1 parameter gradient, 2 data gradient
    std::vector<Span> spans;      // event pool, reused every step
    size_t spans_used = 0;
    long long launches[B2C_PROF_KINDS] = {0};   // kernels launched since the last profile read
    // gradient-ready events of the update buckets: event k is recorded once the weight layer first_layer[k] has finished its
    // parameter gradient in the last pass of a step (the backward pass completes weight layers last to first)
    // running statistics of the BatchNorm layers (optional): caller-owned array, one [mean c][var c] block per layer
    std::vector<BnRunEntry> run_entries;
    size_t run_count = 0;
    float* run_stats = nullptr;
    float run_momentum = 0.1f;
    std::vector<int> bucket_first_layer;
    std::vector<cudaEvent_t> bucket_events;
    ~b2c_net()
    {
        for (Span& sp : spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
        for (cudaEvent_t e : bucket_events) cudaEventDestroy(e);
    }
};

namespace {
// Brackets one launch site with events when profiling is on, and counts its kernels.
struct ProfScope {
    b2c_net* net; cudaStream_t stream; b2c_net::Span* sp = nullptr;
    ProfScope(b2c_net* n, cudaStream_t st, int kind, int kernels, int layer = -1, int pass = 0) : net(n), stream(st)
    {
        net->launches[kind] += kernels;
        if (!net->profile) return;
        if (net->spans_used == net->spans.size()) {
            b2c_net::Span fresh{};
            if (cudaEventCreate(&fresh.a) != cudaSuccess || cudaEventCreate(&fresh.b) != cudaSuccess) return;
            net->spans.push_back(fresh);
        }
        sp = &net->spans[net->spans_used++];
        sp->kind = kind;
        sp->layer = layer;
        sp->pass = pass;
        cudaEventRecord(sp->a, stream);
    }
    ~ProfScope() { if (sp) cudaEventRecord(sp->b, stream); }
};
}  // namespace

extern "C" {

b2c_status b2c_net_create(b2c_ctx* ctx, const b2c_layer_desc* layers, int n_layers, int micro_batch, b2c_net** out)
{
    return b2c_net_create_concurrent(ctx, layers, n_layers, micro_batch, 1, out);
}

b2c_status b2c_net_create_concurrent(b2c_ctx* ctx, const b2c_layer_desc* layers, int n_layers, int micro_batch, int n_concurrent, b2c_net** out)
{
    if (!ctx || !layers || !out || n_layers < 1 || micro_batch < 1 || n_concurrent < 1) return B2C_ERR_INVALID_ARG;
    *out = nullptr;
    b2c_net* net = new (std::nothrow) b2c_net();
    if (!net) return B2C_ERR_CUDA;
    net->ctx = ctx;
    net->micro_batch = micro_batch;
    net->n_conc = n_concurrent;
    const int batch = micro_batch * n_concurrent;   // images per pass
    const char* env = std::getenv("B2C_FUSE_BN_STATS");
    net->fuse_stats = !(env && env[0] == '0');
    net->layers.resize(n_layers);
    net->tensors.resize(n_layers + 1);
    auto fail = [&](b2c_status s) { delete net; return s; };

    size_t ws = 0;
    auto alloc = [&](size_t bytes) { long long off = (long long)ws; ws += (bytes + 255) & ~size_t(255); return off; };
    size_t pc = 0;
    auto palloc = [&](size_t elems) { long long off = (long long)pc; pc += (elems + 7) & ~size_t(7); return off; };

    // the first layer must be a convolution reading tensor 0: it fixes the image shape
    if (layers[0].kind != B2C_LAYER_CONV || layers[0].src != 0) return fail(B2C_ERR_INVALID_ARG);
    net->image_h = layers[0].h; net->image_w = layers[0].w; net->image_c = layers[0].c;
    net->image_c_pad = round_up(layers[0].c, 16);
    net->stem_im2col = layers[0].r == 3 && layers[0].stride == 1 && layers[0].c * 9 <= 32;
    if (net->stem_im2col) net->image_c_pad = 32;
    {
        TensorPlan& t0 = net->tensors[0];
        t0.n = batch; t0.h = net->image_h; t0.w = net->image_w; t0.c = net->image_c_pad; t0.exists = true;
        if (net->image_c_pad != net->image_c) t0.act_off = alloc(t0.elems() * 2);
    }
    // forward shapes and parameters
    for (int i = 0; i < n_layers; ++i) {
        LayerPlan& L = net->layers[i];
        L.d = layers[i];
        const b2c_layer_desc& d = L.d;
        if (d.src < 0 || d.src > i || !net->tensors[d.src].exists) return fail(B2C_ERR_INVALID_ARG);
        const TensorPlan& in = net->tensors[d.src];
        TensorPlan& o = net->tensors[i + 1];
        o.producer = i;
        switch (d.kind) {
            case B2C_LAYER_CONV: {
                const bool patch = net->stem_im2col && i == 0;   // this layer reads the patch matrix: a 1x1 GEMM over 32 columns
                if (in.f32 || d.h != in.h || d.w != in.w || (!patch && round_up(d.c, 16) != in.c)) return fail(B2C_ERR_INVALID_ARG);
                if (d.k % 16 || !(d.r == 1 || d.r == 3) || !(d.stride == 1 || d.stride == 2)) return fail(B2C_ERR_UNSUPPORTED_SHAPE);
                if (d.src != 0 && d.c % 16) return fail(B2C_ERR_UNSUPPORTED_SHAPE);
                const int pad = (d.r - 1) / 2;
                L.c_pad = in.c; L.k_pad = d.k;
                L.p = (d.h + 2 * pad - d.r) / d.stride + 1; L.q = (d.w + 2 * pad - d.r) / d.stride + 1;
                if (L.p * d.stride != d.h || L.q * d.stride != d.w || !b2c_is_pow2(L.p) || !b2c_is_pow2(L.q)) return fail(B2C_ERR_UNSUPPORTED_SHAPE);
                o.n = batch; o.h = L.p; o.w = L.q; o.c = d.k; o.exists = true;
                o.act_off = alloc(o.elems() * 2);
                L.gemm_r = patch ? 1 : d.r;
                L.w_off = palloc((size_t)d.k * L.gemm_r * L.gemm_r * L.c_pad);
                L.seg_index = (int)net->segs.size();
                net->segs.push_back(b2c_weight_seg{L.w_off, d.k, L.gemm_r * L.gemm_r, L.c_pad});
                break;
            }
            case B2C_LAYER_BN: {
                if (in.f32 || d.c != in.c || d.c % 8) return fail(B2C_ERR_INVALID_ARG);
                if (d.res >= 0) {
                    if (d.res > i || !net->tensors[d.res].exists) return fail(B2C_ERR_INVALID_ARG);
                    const TensorPlan& r = net->tensors[d.res];
                    if (r.n != in.n || r.h != in.h || r.w != in.w || r.c != in.c || d.res == 0) return fail(B2C_ERR_INVALID_ARG);
                }
                o = in; o.producer = i; o.n_contrib = 0; o.grad_off[0] = o.grad_off[1] = -1; o.stats_off = -1; o.fused_stats = false;
                o.act_off = alloc(o.elems() * 2);
                if (d.relu) L.mask_off = alloc(o.elems() / 8);   // one bit per output for the backward pass
                break;
            }
            case B2C_LAYER_AVGPOOL: {
                if (in.f32 || d.c != in.c) return fail(B2C_ERR_INVALID_ARG);
                o.n = batch; o.h = 1; o.w = 1; o.c = in.c; o.exists = true;
                o.act_off = alloc(o.elems() * 2);
                break;
            }
            case B2C_LAYER_FC: {
                if (in.f32 || in.h != 1 || in.w != 1 || d.c != in.c || d.c % 16 || d.k < 1) return fail(B2C_ERR_INVALID_ARG);
                L.c_pad = in.c; L.k_pad = round_up(d.k, 64);
                L.p = L.q = 1;
                o.n = batch; o.h = 1; o.w = 1; o.c = L.k_pad; o.f32 = true; o.exists = true;
                o.act_off = alloc(o.elems() * 4);
                L.w_off = palloc((size_t)L.k_pad * L.c_pad);
                L.seg_index = (int)net->segs.size();
                net->segs.push_back(b2c_weight_seg{L.w_off, L.k_pad, 1, L.c_pad});
                break;
            }
            case B2C_LAYER_XENT: {
                if (!in.f32 || i != n_layers - 1 || net->layers[in.producer].d.kind != B2C_LAYER_FC || d.k != net->layers[in.producer].d.k)
                    return fail(B2C_ERR_INVALID_ARG);
                break;
            }
            default: return fail(B2C_ERR_INVALID_ARG);
        }
    }
    if (layers[n_layers - 1].kind != B2C_LAYER_XENT) return fail(B2C_ERR_INVALID_ARG);
    if (net->segs.size() > 128) return fail(B2C_ERR_UNSUPPORTED_SHAPE);
    // BatchNorm / bias parameters after all filter banks
    for (int i = 0; i < n_layers; ++i) {
        LayerPlan& L = net->layers[i];
        if (L.d.kind == B2C_LAYER_BN) { L.gamma_off = palloc(L.d.c); L.beta_off = palloc(L.d.c); }
        if (L.d.kind == B2C_LAYER_FC) L.bias_off = palloc(L.k_pad);
    }
    net->param_count = (pc + 3) & ~size_t(3);

    // backward plan: gradient buffers, in the order the backward pass produces them
    auto add_contrib = [&](int t) -> int {
        TensorPlan& T = net->tensors[t];
        if (T.n_contrib >= 2) return -1;
        const int slot = T.n_contrib++;
        T.grad_off[slot] = alloc(T.elems() * 2);
        return slot;
    };
    for (int i = n_layers - 1; i >= 0; --i) {
        LayerPlan& L = net->layers[i];
        const int kind = L.d.kind;
        if (kind == B2C_LAYER_XENT || kind == B2C_LAYER_FC || kind == B2C_LAYER_AVGPOOL || kind == B2C_LAYER_BN ||
            (kind == B2C_LAYER_CONV && L.d.src != 0)) {
            if (kind != B2C_LAYER_XENT && net->tensors[i + 1].n_contrib < 1) return fail(B2C_ERR_INVALID_ARG);   // dead output
            if (kind != B2C_LAYER_BN && kind != B2C_LAYER_XENT && net->tensors[i + 1].n_contrib != 1) return fail(B2C_ERR_UNSUPPORTED_SHAPE);
            if ((L.src_slot = add_contrib(L.d.src)) < 0) return fail(B2C_ERR_UNSUPPORTED_SHAPE);
            if (kind == B2C_LAYER_BN && L.d.res >= 0 && (L.res_slot = add_contrib(L.d.res)) < 0) return fail(B2C_ERR_UNSUPPORTED_SHAPE);
        }
    }
    // small per-layer buffers; the fp64 statistics are contiguous so one memset clears them
    for (int i = 0; i < n_layers; ++i) {
        LayerPlan& L = net->layers[i];
        if (L.d.kind == B2C_LAYER_BN) { L.mean_off = alloc(4 * (size_t)L.d.c * n_concurrent); L.invstd_off = alloc(4 * (size_t)L.d.c * n_concurrent); }
    }
    net->stats_begin = (long long)ws;
    for (int i = 0; i < n_layers; ++i) {
        LayerPlan& L = net->layers[i];
        if (L.d.kind == B2C_LAYER_CONV) {
            TensorPlan& o = net->tensors[i + 1];
            o.stats_off = alloc(16 * (size_t)L.d.k * n_concurrent);
            // the epilogue can own the statistics only if no 128-pixel tile straddles two micro-batches
            const int pix = L.p * L.q;
            const int imgs_per_tile = pix >= 128 ? 1 : 128 / pix;
            o.fused_stats = net->fuse_stats && (micro_batch % imgs_per_tile == 0);
            // Tiles wider than 64 channels sum their columns with a shuffle butterfly (about 1400 cycles per 32 columns and
            // unit, measured); where that exceeds the unit's MMA time the epilogue becomes the bottleneck and one more pass
            // over the output (mostly still in L2) is cheaper.  Tiles of up to 64 channels keep their sums in registers.
            {
                int n_tile = 16;
                for (int cand = 256; cand >= 16; cand -= 16)
                    if (L.d.k % cand == 0) { n_tile = cand; break; }
                const long long mma_cycles = (long long)(L.c_pad * L.gemm_r * L.gemm_r / 16) * (n_tile / 2 > 48 ? n_tile / 2 : 48);
                const long long sum_cycles = 1400ll * n_tile / 32;
                const char* e2 = std::getenv("B2C_FUSE_WIDE");   // 1: always fuse; 0: never on wide tiles; default: by the estimate
                const bool wide_ok = e2 ? e2[0] != '0' : mma_cycles >= sum_cycles;
                if (n_tile > 64 && !wide_ok) o.fused_stats = false;
            }
        }
        if (L.d.kind == B2C_LAYER_BN) {
            L.bwd_ws_off = alloc(b2c_bn_relu_bwd_workspace_bytes(L.d.c) * n_concurrent);
            L.arrive_off = alloc(sizeof(unsigned) * (size_t)n_concurrent);   // one arrival counter per statistics group, cleared with the sums
        }
    }
    net->stats_end = (long long)ws;
    net->ws_bytes = ws;
    // running statistics: every BatchNorm whose input is a convolution output (its sums stay in the workspace for the pass)
    for (int i = 0; i < n_layers; ++i) {
        LayerPlan& L = net->layers[i];
        if (L.d.kind != B2C_LAYER_BN) continue;
        const TensorPlan& in = net->tensors[L.d.src];
        if (in.stats_off < 0) continue;
        L.run_off = (long long)net->run_count;
        net->run_entries.push_back(BnRunEntry{in.stats_off, in.c, (int)net->run_count, (float)((long long)micro_batch * in.h * in.w)});
        net->run_count += 2 * (size_t)in.c;
    }
    // Chunking for L2: a layer takes as many micro-batches per launch as keep its largest tensor under the budget (a
    // power-of-two divisor of the pass; B2C_CHUNK_MB sets the budget in MB, 0 = whole passes).
    {
        const char* cenv = std::getenv("B2C_CHUNK_MB");
        const double budget = (cenv ? std::atof(cenv) : (double)B2C_DEFAULT_CHUNK_MB) * 1e6;
        for (int i = 0; i < n_layers; ++i) {
            LayerPlan& L = net->layers[i];
            int gc = n_concurrent;
            if (budget > 0.0) {
                const TensorPlan& a = net->tensors[L.d.src];
                const TensorPlan& b = net->tensors[i + 1];
                double per_mb = (double)micro_batch * a.h * a.w * a.c * (a.f32 ? 4 : 2);
                if (b.exists) {
                    const double pb = (double)micro_batch * b.h * b.w * b.c * (b.f32 ? 4 : 2);
                    if (pb > per_mb) per_mb = pb;
                }
                while (gc > 1 && (gc * per_mb > budget || n_concurrent % gc != 0)) --gc;
            }
            L.chunk_groups = gc;
        }
    }
    *out = net;
    return B2C_OK;
}

void b2c_net_destroy(b2c_net* net) { delete net; }
size_t b2c_net_param_count(const b2c_net* net) { return net ? net->param_count : 0; }
size_t b2c_net_workspace_bytes(const b2c_net* net) { return net ? net->ws_bytes : 0; }
int b2c_net_padded_image_channels(const b2c_net* net) { return net ? net->image_c_pad : 0; }
int b2c_net_first_conv_im2col(const b2c_net* net) { return net && net->stem_im2col ? 1 : 0; }

long long b2c_net_param_offset(const b2c_net* net, int layer, int which)
{
    if (!net || layer < 0 || layer >= (int)net->layers.size()) return -1;
    const LayerPlan& L = net->layers[layer];
    switch (which) {
        case 0: return L.w_off;
        case 1: return L.gamma_off;
        case 2: return L.beta_off;
        case 3: return L.bias_off;
    }
    return -1;
}

long long b2c_net_tensor_offset(const b2c_net* net, int tensor, int grad, int which)
{
    if (!net || tensor < 0 || tensor >= (int)net->tensors.size()) return -1;
    const TensorPlan& T = net->tensors[tensor];
    if (!grad) return T.act_off;
    if (which < 0 || which > 1) return -1;
    return T.grad_off[which];
}

b2c_status b2c_net_bind(b2c_net* net, float* w_master, float* velocity, float* grad_sum, void* w_bf16, void* w_bf16_dgrad, void* workspace,
                        size_t workspace_bytes)
{
    if (!net || !w_master || !velocity || !grad_sum || !w_bf16 || !w_bf16_dgrad || !workspace) return B2C_ERR_INVALID_ARG;
    if (workspace_bytes < net->ws_bytes) return B2C_ERR_WORKSPACE_TOO_SMALL;
    if (!b2c_aligned16(w_master) || !b2c_aligned16(velocity) || !b2c_aligned16(grad_sum) || !b2c_aligned16(w_bf16) ||
        !b2c_aligned16(w_bf16_dgrad) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return B2C_ERR_MISALIGNED;
    net->w = w_master; net->v = velocity; net->g = grad_sum;
    net->w_bf16 = reinterpret_cast<char*>(w_bf16); net->w_dgrad = reinterpret_cast<char*>(w_bf16_dgrad);
    net->ws = reinterpret_cast<char*>(workspace);
    return B2C_OK;
}

static b2c_status net_pack_dgrad(b2c_net* net, void* stream)
{
    return b2c_weight_pack_dgrad(net->ctx, net->segs.data(), (int)net->segs.size(), net->w_bf16, net->w_dgrad, stream);
}

size_t b2c_net_running_stats_count(const b2c_net* net) { return net ? net->run_count : 0; }

long long b2c_net_running_stats_offset(const b2c_net* net, int layer)
{
    if (!net || layer < 0 || layer >= (int)net->layers.size()) return -1;
    return net->layers[layer].run_off;
}

b2c_status b2c_net_bind_running_stats(b2c_net* net, float* running, float momentum)
{
    if (!net || momentum < 0.f || momentum > 1.f) return B2C_ERR_INVALID_ARG;
    if (running && (reinterpret_cast<uintptr_t>(running) & 3u)) return B2C_ERR_MISALIGNED;
    net->run_stats = running;
    net->run_momentum = momentum;
    return B2C_OK;
}

b2c_status b2c_net_set_buckets(b2c_net* net, int n_buckets, const int* first_layer)
{
    if (!net || n_buckets < 0 || (n_buckets > 0 && !first_layer)) return B2C_ERR_INVALID_ARG;
    for (int b = 0; b < n_buckets; ++b)
        if (first_layer[b] < 0 || first_layer[b] >= (int)net->segs.size()) return B2C_ERR_INVALID_ARG;
    for (cudaEvent_t e : net->bucket_events) cudaEventDestroy(e);
    net->bucket_events.clear();
    net->bucket_first_layer.assign(first_layer, first_layer + n_buckets);
    for (int b = 0; b < n_buckets; ++b) {
        cudaEvent_t e;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return B2C_ERR_CUDA;
        net->bucket_events.push_back(e);
    }
    return B2C_OK;
}

b2c_status b2c_net_bucket_wait(b2c_net* net, int bucket, void* stream)
{
    if (!net || bucket < 0 || bucket >= (int)net->bucket_events.size()) return B2C_ERR_INVALID_ARG;
    B2C_CUDA(cudaStreamWaitEvent((cudaStream_t)stream, net->bucket_events[bucket], 0));
    return B2C_OK;
}

b2c_status b2c_net_refresh_dgrad_weights(b2c_net* net, void* stream)
{
    if (!net || !net->ws) return B2C_ERR_INVALID_ARG;
    return net_pack_dgrad(net, stream);
}

b2c_status b2c_net_weight_range(const b2c_net* net, int index, long long* begin, long long* end)
{
    if (!net || !begin || !end || index < 0 || index >= (int)net->segs.size()) return B2C_ERR_INVALID_ARG;
    const b2c_weight_seg& sg = net->segs[index];
    *begin = sg.offset;
    *end = sg.offset + (long long)sg.k * sg.rs * sg.c;
    return B2C_OK;
}

int b2c_net_weight_layer_count(const b2c_net* net) { return net ? (int)net->segs.size() : 0; }

b2c_status b2c_net_sync_weights(b2c_net* net, void* stream)
{
    if (!net || !net->ws) return B2C_ERR_INVALID_ARG;
    // lr = 0, momentum = 1, wd = 0, zero gradient scale: leaves w and v untouched and writes the bf16 copy
    b2c_status st = b2c_grad_accum_sgd_momentum(net->ctx, net->param_count, net->w, net->v, net->g, 0.f, 0.f, 1.f, 0.f, net->w_bf16, 0, stream);
    if (st != B2C_OK) return st;
    return net_pack_dgrad(net, stream);
}

b2c_status b2c_net_apply_update(b2c_net* net, int n_avg, float lr, float momentum, float wd, void* stream_)
{
    if (!net || !net->ws || n_avg < 1) return B2C_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    ProfScope ps_(net, stream, B2C_PROF_UPDATE, 2);
    b2c_status st = b2c_grad_accum_sgd_momentum(net->ctx, net->param_count, net->w, net->v, net->g, 1.f / (float)n_avg, lr, momentum, wd,
                                                net->w_bf16, 1, stream_);
    if (st != B2C_OK) return st;
    return net_pack_dgrad(net, stream_);
}

#define B2C_TRY(call)                   \
    do {                                \
        b2c_status s_ = (call);         \
        if (s_ != B2C_OK) return s_;    \
    } while (0)

b2c_status b2c_train_step(b2c_net* net, const void* images, const int32_t* labels, int n_micro, float lr, float momentum, float wd,
                          float* loss_dev, int update, void* stream_)
{
    if (!net || !net->ws || !images || !labels || !loss_dev || n_micro < 1) return B2C_ERR_INVALID_ARG;
    if (n_micro % net->n_conc) return B2C_ERR_INVALID_ARG;   // whole passes only
    if (!b2c_aligned16(images)) return B2C_ERR_MISALIGNED;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (net->profile && net->spans_used > (1u << 20)) return B2C_ERR_INVALID_ARG;   // read the profile between steps
    b2c_ctx* ctx = net->ctx;
    const int G = net->n_conc;                 // statistics groups per pass
    const int N = net->micro_batch * G;        // images per pass
    const int n_passes = n_micro / G;
    const int n_layers = (int)net->layers.size();
    const __nv_bfloat16* w_bf16 = reinterpret_cast<const __nv_bfloat16*>(net->w_bf16);
    const __nv_bfloat16* w_dg = reinterpret_cast<const __nv_bfloat16*>(net->w_dgrad);
    // Tensors hold the images of a pass back to back, so a run of whole micro-batches (statistics groups g0 .. g0 + Gc) of any
    // tensor or per-group array is the same array at an offset: img0 = first image of the run.
    auto act = [&](int t, int img0) -> void* {
        const TensorPlan& T = net->tensors[t];
        return net->ws + T.act_off + (long long)img0 * T.h * T.w * T.c * (T.f32 ? 4 : 2);
    };
    auto grad = [&](int t, int slot, int img0) -> void* {
        const TensorPlan& T = net->tensors[t];
        return slot >= 0 && T.grad_off[slot] >= 0 ? net->ws + T.grad_off[slot] + (long long)img0 * T.h * T.w * T.c * 2 : nullptr;
    };

    const size_t image_bytes = (size_t)N * net->image_h * net->image_w * net->image_c * 2;
    if (image_bytes % 16) return B2C_ERR_MISALIGNED;
    B2C_CUDA(cudaMemsetAsync(loss_dev, 0, sizeof(float), stream));
    const int mbs = net->micro_batch;

    for (int mb = 0; mb < n_passes; ++mb) {
        const char* img = reinterpret_cast<const char*>(images) + (size_t)mb * image_bytes;
        const int32_t* lab = labels + (size_t)mb * N;
        const bool staged_input = net->tensors[0].act_off >= 0;
        auto act_in = [&](int t, int img0) -> const void* {
            if (t == 0 && !staged_input) return img + (size_t)img0 * net->image_h * net->image_w * net->image_c * 2;
            return act(t, img0);
        };
        B2C_CUDA(cudaMemsetAsync(net->ws + net->stats_begin, 0, (size_t)(net->stats_end - net->stats_begin), stream));

        // forward pass of layer i over the micro-batches g0 .. g0 + Gc of the pass
        auto forward_layer = [&](int i, int g0, int Gc) -> b2c_status {
            const LayerPlan& L = net->layers[i];
            const b2c_layer_desc& d = L.d;
            const TensorPlan& o = net->tensors[i + 1];
            const int img0 = g0 * mbs, Nc = Gc * mbs;
            if (i == 0 && staged_input) {   // the first layer's chunk of the image batch, expanded on the device
                ProfScope ps_(net, stream, B2C_PROF_OTHER, 1);
                const char* src = img + (size_t)img0 * net->image_h * net->image_w * net->image_c * 2;
                if (net->stem_im2col)
                    B2C_TRY(b2c_im2col_3x3(ctx, Nc, net->image_h, net->image_w, net->image_c, net->image_c_pad, src, act(0, img0), stream));
                else
                    B2C_TRY(b2c_pad_channels(ctx, (long)Nc * net->image_h * net->image_w, net->image_c, net->image_c_pad, src, act(0, img0), stream));
            }
            switch (d.kind) {
                case B2C_LAYER_CONV: {
                    KMajorProblem pb{};
                    pb.n = Nc; pb.ih = d.h; pb.iw = d.w; pb.ic = L.c_pad; pb.oh = L.p; pb.ow = L.q; pb.oc = d.k;
                    pb.r = L.gemm_r; pb.stride = d.stride; pb.pad = (L.gemm_r - 1) / 2; pb.dgrad = false;
                    pb.in = act_in(d.src, img0); pb.wt = w_bf16 + L.w_off; pb.out = act(i + 1, img0);
                    pb.stats = o.fused_stats ? reinterpret_cast<double*>(net->ws + o.stats_off) + (size_t)g0 * 2 * d.k : nullptr;
                    pb.stats_group_images = mbs;
                    ProfScope ps_(net, stream, B2C_PROF_CONV_FWD, 1, i, 0);
                    B2C_TRY(launch_conv_kmajor(ctx, pb, stream));
                    break;
                }
                case B2C_LAYER_BN: {
                    const TensorPlan& in = net->tensors[d.src];
                    const bool ready = in.fused_stats;
                    double* stats = reinterpret_cast<double*>(net->ws + (in.stats_off >= 0 ? in.stats_off : L.bwd_ws_off)) + (size_t)g0 * 2 * in.c;
                    ProfScope ps_(net, stream, B2C_PROF_BN_FWD, ready ? 1 : 2, i, 0);
                    B2C_TRY(launch_bn_fwd(ctx, Gc, (long long)mbs * in.h * in.w, in.c, act(d.src, img0), stats,
                                          ready ? 1 : (in.stats_off >= 0 ? 2 : 0),   // a convolution output's sums live in the region cleared once per pass
                                          net->w + L.gamma_off,
                                          net->w + L.beta_off, d.res >= 0 ? act(d.res, img0) : nullptr, d.relu, 1e-5f, act(i + 1, img0),
                                          reinterpret_cast<float*>(net->ws + L.mean_off) + (size_t)g0 * in.c,
                                          reinterpret_cast<float*>(net->ws + L.invstd_off) + (size_t)g0 * in.c, nullptr, nullptr, 0.f,
                                          L.mask_off >= 0 ? net->ws + L.mask_off + (long long)img0 * in.h * in.w * in.c / 8 : nullptr, stream));
                    break;
                }
                case B2C_LAYER_AVGPOOL: {
                    const TensorPlan& in = net->tensors[d.src];
                    ProfScope ps_(net, stream, B2C_PROF_OTHER, 1, i, 0);
                    B2C_TRY(b2c_avgpool_fwd(ctx, Nc, in.h * in.w, in.c, act(d.src, img0), act(i + 1, img0), stream));
                    break;
                }
                case B2C_LAYER_FC: {
                    KMajorProblem pb{};
                    pb.n = Nc; pb.ih = 1; pb.iw = 1; pb.ic = L.c_pad; pb.oh = 1; pb.ow = 1; pb.oc = L.k_pad;
                    pb.r = 1; pb.stride = 1; pb.pad = 0; pb.dgrad = false;
                    pb.in = act(d.src, img0); pb.wt = w_bf16 + L.w_off; pb.out = act(i + 1, img0);
                    pb.out_f32 = true; pb.bias = net->w + L.bias_off;
                    ProfScope ps_(net, stream, B2C_PROF_OTHER, 1, i, 0);
                    B2C_TRY(launch_conv_kmajor(ctx, pb, stream));
                    break;
                }
                case B2C_LAYER_XENT: {
                    const TensorPlan& in = net->tensors[d.src];
                    ProfScope ps_(net, stream, B2C_PROF_OTHER, 1, i, 0);
                    B2C_TRY(b2c_softmax_xent_fwd_bwd(ctx, Nc, d.k, reinterpret_cast<const float*>(act(d.src, img0)), in.c, lab + img0,
                                                     1.f / ((float)mbs * (float)n_micro), 1.f / (float)mbs, loss_dev,
                                                     grad(d.src, L.src_slot, img0), in.c, stream));
                    break;
                }
            }
            return B2C_OK;
        };

        // the parameter gradient of weight layer `seg` is complete for this step: release the buckets that waited for it
        auto weights_done = [&](int seg, int g0, int Gc) {
            if (mb != n_passes - 1 || g0 + Gc != G) return;
            for (size_t b = 0; b < net->bucket_events.size(); ++b)
                if (net->bucket_first_layer[b] == seg) cudaEventRecord(net->bucket_events[b], stream);
        };
        // backward pass of layer i over the same kind of run; parameter gradients are summed into the flat gradient array
        auto backward_layer = [&](int i, int g0, int Gc) -> b2c_status {
            const LayerPlan& L = net->layers[i];
            const b2c_layer_desc& d = L.d;
            const TensorPlan& o = net->tensors[i + 1];
            const int img0 = g0 * mbs, Nc = Gc * mbs;
            switch (d.kind) {
                case B2C_LAYER_XENT: break;
                case B2C_LAYER_FC: {
                    const void* dz = grad(i + 1, 0, img0);
                    WgradProblem wp{};
                    wp.n = Nc; wp.h = 1; wp.w = 1; wp.c = L.c_pad; wp.p = 1; wp.q = 1; wp.k = L.k_pad; wp.r = 1; wp.stride = 1; wp.pad = 0;
                    wp.dy = dz; wp.x = act(d.src, img0); wp.dw = net->g + L.w_off;
                    ProfScope ps_(net, stream, B2C_PROF_OTHER, 3, i, 1);
                    B2C_TRY(launch_conv_wgrad(ctx, wp, stream));
                    B2C_TRY(b2c_bias_grad(ctx, Nc, L.k_pad, L.k_pad, dz, net->g + L.bias_off, 1, stream));
                    weights_done(L.seg_index, g0, Gc);
                    KMajorProblem pb{};
                    pb.n = Nc; pb.ih = 1; pb.iw = 1; pb.ic = L.k_pad; pb.oh = 1; pb.ow = 1; pb.oc = L.c_pad;
                    pb.r = 1; pb.stride = 1; pb.pad = 0; pb.dgrad = true;
                    pb.in = dz; pb.wt = w_dg + L.w_off; pb.out = grad(d.src, L.src_slot, img0);
                    B2C_TRY(launch_conv_kmajor(ctx, pb, stream));
                    break;
                }
                case B2C_LAYER_AVGPOOL: {
                    const TensorPlan& in = net->tensors[d.src];
                    ProfScope ps_(net, stream, B2C_PROF_OTHER, 1, i, 2);
                    B2C_TRY(b2c_avgpool_bwd(ctx, Nc, in.h * in.w, in.c, grad(i + 1, 0, img0), grad(d.src, L.src_slot, img0), stream));
                    break;
                }
                case B2C_LAYER_BN: {
                    const TensorPlan& in = net->tensors[d.src];
                    ProfScope ps_(net, stream, B2C_PROF_BN_BWD, 2, i, 2);
                    B2C_TRY(launch_bn_bwd(ctx, Gc, (long long)mbs * in.h * in.w, in.c, grad(i + 1, 0, img0),
                                          o.n_contrib > 1 ? grad(i + 1, 1, img0) : nullptr, act(d.src, img0), act(i + 1, img0), net->w + L.gamma_off,
                                          reinterpret_cast<float*>(net->ws + L.mean_off) + (size_t)g0 * in.c,
                                          reinterpret_cast<float*>(net->ws + L.invstd_off) + (size_t)g0 * in.c, d.relu, grad(d.src, L.src_slot, img0),
                                          d.res >= 0 ? grad(d.res, L.res_slot, img0) : nullptr, net->g + L.gamma_off, net->g + L.beta_off, 1,
                                          reinterpret_cast<double*>(net->ws + L.bwd_ws_off) + (size_t)g0 * 2 * in.c, /*sums_zeroed=*/in.stats_off >= 0,
                                          L.mask_off >= 0 ? net->ws + L.mask_off + (long long)img0 * in.h * in.w * in.c / 8 : nullptr,
                                          ctx->use_bn_grouped ? reinterpret_cast<unsigned*>(net->ws + L.arrive_off) + g0 : nullptr, stream));
                    break;
                }
                case B2C_LAYER_CONV: {
                    const void* dy = grad(i + 1, 0, img0);
                    WgradProblem wp{};
                    wp.n = Nc; wp.h = d.h; wp.w = d.w; wp.c = L.c_pad; wp.p = L.p; wp.q = L.q; wp.k = d.k;
                    wp.r = L.gemm_r; wp.stride = d.stride; wp.pad = (L.gemm_r - 1) / 2;
                    wp.dy = dy; wp.x = act_in(d.src, img0); wp.dw = net->g + L.w_off;
                    {
                        ProfScope ps_(net, stream, B2C_PROF_CONV_WGRAD, 1, i, 1);
                        B2C_TRY(launch_conv_wgrad(ctx, wp, stream));
                    }
                    weights_done(L.seg_index, g0, Gc);
                    if (d.src != 0) {
                        KMajorProblem pb{};
                        pb.n = Nc; pb.ih = L.p; pb.iw = L.q; pb.ic = d.k; pb.oh = d.h; pb.ow = d.w; pb.oc = L.c_pad;
                        pb.r = d.r; pb.stride = d.stride; pb.pad = (d.r - 1) / 2; pb.dgrad = true;
                        pb.in = dy; pb.wt = w_dg + L.w_off; pb.out = grad(d.src, L.src_slot, img0);
                        ProfScope ps_(net, stream, B2C_PROF_CONV_DGRAD, 1, i, 2);
                        B2C_TRY(launch_conv_kmajor(ctx, pb, stream));
                    }
                    break;
                }
            }
            return B2C_OK;
        };

        // Layers whose tensors exceed the L2 budget run in segments: a run of consecutive layers with the same chunk size
        // is taken chunk by chunk (a few micro-batches at a time), so that a tensor is still in L2 when its consumer (and
        // the second pass of the BatchNorm backward) reads it.  Every layer acts on images independently except through the
        // per-micro-batch BatchNorm statistics, so any run of whole micro-batches is a valid chunk.
        for (int seg = 0; seg < n_layers;) {
            const int Gc = net->layers[seg].chunk_groups;
            int seg_end = seg + 1;
            while (seg_end < n_layers && net->layers[seg_end].chunk_groups == Gc) ++seg_end;
            for (int g0 = 0; g0 < G; g0 += Gc)
                for (int i = seg; i < seg_end; ++i) B2C_TRY(forward_layer(i, g0, Gc));
            seg = seg_end;
        }
        if (net->run_stats != nullptr && !net->run_entries.empty()) {   // the forward pass of all micro-batches of the pass is enqueued
            ProfScope ps_(net, stream, B2C_PROF_BN_FWD, (int)((net->run_entries.size() + 63) / 64));
            B2C_TRY(launch_bn_running_update(ctx, net->run_entries.data(), (int)net->run_entries.size(), net->ws, net->run_stats, G, net->run_momentum,
                                             stream));
        }
        for (int seg_end = n_layers; seg_end > 0;) {
            const int Gc = net->layers[seg_end - 1].chunk_groups;
            int seg = seg_end - 1;
            while (seg > 0 && net->layers[seg - 1].chunk_groups == Gc) --seg;
            for (int g0 = 0; g0 < G; g0 += Gc)
                for (int i = seg_end - 1; i >= seg; --i) B2C_TRY(backward_layer(i, g0, Gc));
            seg_end = seg;
        }
    }
    // ---------------- gradient average + parameter update, refresh of both bf16 weight copies
    if (update) B2C_TRY(b2c_net_apply_update(net, n_micro, lr, momentum, wd, stream_));
    return B2C_OK;
}

b2c_status b2c_net_profile_enable(b2c_net* net, int enable)
{
    if (!net) return B2C_ERR_INVALID_ARG;
    net->profile = enable != 0;
    net->spans_used = 0;
    for (int k = 0; k < B2C_PROF_KINDS; ++k) net->launches[k] = 0;
    return B2C_OK;
}

b2c_status b2c_net_profile_read_layers(b2c_net* net, double* ms, int n_layers, void* stream)
{
    if (!net || !ms || n_layers != (int)net->layers.size()) return B2C_ERR_INVALID_ARG;
    B2C_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    for (int i = 0; i < 3 * n_layers; ++i) ms[i] = 0.0;
    for (size_t i = 0; i < net->spans_used; ++i) {
        const b2c_net::Span& sp = net->spans[i];
        float t = 0.f;
        if (sp.layer >= 0 && sp.layer < n_layers && cudaEventElapsedTime(&t, sp.a, sp.b) == cudaSuccess) ms[3 * sp.layer + sp.pass] += t;
    }
    return B2C_OK;
}

int b2c_net_layer_count(const b2c_net* net) { return net ? (int)net->layers.size() : 0; }

b2c_status b2c_net_profile_read(b2c_net* net, double* ms, long long* launches, void* stream)
{
    if (!net || !ms || !launches) return B2C_ERR_INVALID_ARG;
    B2C_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    for (int k = 0; k < B2C_PROF_KINDS; ++k) { ms[k] = 0.0; launches[k] = net->launches[k]; net->launches[k] = 0; }
    for (size_t i = 0; i < net->spans_used; ++i) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, net->spans[i].a, net->spans[i].b) == cudaSuccess) ms[net->spans[i].kind] += t;
    }
    net->spans_used = 0;
    return B2C_OK;
}

}  // extern "C"
