// Host-side shared declarations of the library: context, status helpers, kernel launchers.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/b2c.h"

// Bits of the sticky device status word.
#define B2C_DEV_TIMEOUT 1u
#define B2C_DEV_BAD_LABEL 2u

typedef CUresult (*b2c_encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                        const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                        CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct b2c_ctx {
    int device;
    int sm_count;
    unsigned* d_status;  // one device word
    unsigned spin_limit;
    b2c_encode_tiled_fn encode_tiled;
    int use_full_halo;                   // 3x3 stride-1 convolutions with a resident filter bank stage one framed tile for all nine taps
    int use_pairs;                       // forward / data-gradient convolutions may run on CTA pairs (cta_group::2)
    unsigned long long* stall_counters;  // optional device array the convolution kernels add their wait cycles to
    int use_wgrad_frame;                 // weight gradient of 3x3 stride-1 layers stages x once per chunk with a one-pixel frame (all three shifts from one box)
    int use_issue_split;                 // forward / data-gradient tiles wider than 128 channels: two MMA-issuing threads share every unit
    int use_pdl;                         // kernels are launched with programmatic stream serialization (their set-up overlaps the previous kernel's tail)
    int use_hmerge;                      // forward / data gradient of 3x3 stride-1 layers with 64 output channels: horizontal taps merged into N = 192 MMAs
    int use_group_kblocks;               // short k-blocks of stride-2 and 1x1 layers share ring slots (fewer barrier waits per MMA)
    int use_wgrad_two_issuers;           // weight gradient: two MMA-issuing threads on alternate chunks of one accumulator where the ring depth is even
    int use_bn_grouped;                  // BatchNorm backward of the training step: both passes in one cooperative launch, group by group
    // Launch plans (kernel parameter blocks with their tensor maps, grid and shared-memory size) of the convolution
    // kernels, keyed by the bytes of the problem description: pointers and shapes of a bound network repeat every
    // step, so a plan is built once and its launches cost one parameter copy.
    std::unordered_map<std::string, std::vector<unsigned char>> plan_cache;
    unsigned smem_optin_done;            // kernels whose dynamic shared-memory opt-in was set on this context's device (B2C_OPTIN_* bits)
};
#define B2C_OPTIN_KMAJOR 1u
#define B2C_OPTIN_WGRAD 2u
#define B2C_OPTIN_BN_BWD 4u
#define B2C_OPTIN_BN_GROUPED 8u

#define B2C_CUDA(call)                               \
    do {                                             \
        cudaError_t e_ = (call);                     \
        if (e_ != cudaSuccess) return B2C_ERR_CUDA;  \
    } while (0)

// Kernel launch.  With ctx->use_pdl the launch carries the programmatic-stream-serialization attribute: the kernel may be
// scheduled while the previous kernel of the stream drains, and it orders itself behind that kernel with pdl_wait()
// (every kernel of the library calls it before its first global access).  cluster > 1 launches thread-block clusters.
template <typename... KArgs, typename... Args>
static inline cudaError_t b2c_launch(const b2c_ctx* ctx, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     unsigned cluster, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (ctx->use_pdl) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

static inline bool b2c_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline bool b2c_is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

namespace b2c {

// Filter taps of one launch: which tensor map (parity view) a tap gathers from, its pixel
// offset inside that view, and its index in the weight tensor's tap dimension.
struct TapList {
    int count;
    int8_t map[9], dh[9], dw[9], rs[9];
};

// bf16 activation tensor [n][h][w][c] as a 4-D tensor map (c, w/step, h/step, n); step 2 selects
// rows of parity ph and columns of parity pw.  Box = (box_c, box_w, box_h, box_n); swizzle = box_c*2 bytes.
bool encode_activation_map(b2c_ctx* ctx, CUtensorMap* tm, const void* base, int n, int h, int w, int c, int step, int ph, int pw, int box_c,
                           int box_w, int box_h, int box_n);
// Taps of a forward convolution in terms of (parity view, offset): input row = p*stride + r - pad.
void forward_taps(TapList& tl, int R, int stride, int pad);

// Geometry of one implicit-GEMM launch with K-major operands (forward and data gradient):
// the "input" is the activation tensor that is gathered (x for fprop, dy for dgrad), the
// "output" the tensor that is written.  in_pitch / out_pitch are channel strides in elements.
struct KMajorProblem {
    int n;                 // images
    int ih, iw, ic;        // gathered tensor
    int oh, ow, oc;        // written tensor
    int r, stride, pad;    // filter taps (r x r), forward stride and padding of the convolution
    bool dgrad;            // false: forward; true: data gradient (input = dy, weights in [c,r,s,k] flipped layout)
    const void* in;
    const void* wt;        // [oc][r*r][ic] bf16
    void* out;
    bool out_f32;
    const float* bias;
    double* stats;         // fp64 [groups][2*oc] or nullptr
    int stats_group_images;  // images per statistics group (0: one group)
};
b2c_status launch_conv_kmajor(b2c_ctx* ctx, const KMajorProblem& pb, cudaStream_t stream);

struct WgradProblem {
    int n, h, w, c;        // x
    int p, q, k;           // dy
    int r, stride, pad;
    const void* dy;
    const void* x;
    float* dw;             // [k][r*r][c] fp32, accumulated into
};
b2c_status launch_conv_wgrad(b2c_ctx* ctx, const WgradProblem& pb, cudaStream_t stream);

// BatchNorm over G statistics groups (micro-batches) of m rows each; stats / sums are fp64 [G][2c],
// save_mean / save_invstd fp32 [G][c].  G > 1 requires acc != 0 in the backward pass.  stats_ready: 1 = `stats` holds the
// sums already (convolution epilogue), 0 = clear and compute them, 2 = compute them into `stats` the caller has cleared.  relu_mask (optional): one bit per
// element, "stored output > 0" (a byte per 8 channels), written by the forward pass and read by the backward pass
// in place of the output tensor.  sums_zeroed: the caller has already cleared `sums` (and `arrivals`).  arrivals (optional): G
// zeroed counters; with them the two passes run in one cooperative launch, group by group (bn_bwd_grouped_kernel).
b2c_status launch_bn_fwd(b2c_ctx* ctx, int G, long long m, int c, const void* y, double* stats, int stats_ready, const float* gamma,
                         const float* beta, const void* residual, int relu, float eps, void* a, float* save_mean, float* save_invstd,
                         float* run_mean, float* run_var, float momentum, void* relu_mask, cudaStream_t stream);
b2c_status launch_bn_bwd(b2c_ctx* ctx, int G, long long m, int c, const void* da1, const void* da2, const void* y, const void* a,
                         const float* gamma, const float* save_mean, const float* save_invstd, int relu, void* dy, void* dres, float* dgamma,
                         float* dbeta, int acc, double* sums, bool sums_zeroed, const void* relu_mask, unsigned* arrivals, cudaStream_t stream);

// Running statistics of the BatchNorm layers of a step (momentum update with the unbiased variance), taken from the fp64
// sums the forward pass left in the workspace.  One entry per layer; the G statistics groups of a pass are applied in
// order, as if the micro-batches had run one after the other.
struct BnRunEntry {
    long long stats_off;   // bytes into the workspace: fp64 [G][2c] sum / sum of squares
    int c;                 // channels
    int run_off;           // elements into the running-statistics array: [mean c][var c]
    float m;               // rows per group
};
b2c_status launch_bn_running_update(b2c_ctx* ctx, const BnRunEntry* entries, int n_entries, const char* ws, float* run, int G, float momentum,
                                    cudaStream_t stream);

}  // namespace b2c
