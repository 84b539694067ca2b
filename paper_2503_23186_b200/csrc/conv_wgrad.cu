// Weight gradient as an implicit GEMM on tcgen05 with both operands MN-major:
//
//   dw[k, tap, c] += sum over pixels  dy[pixel, k] * x[pixel shifted by tap, c]
//
// GEMM M = 128 output channels (k), N = ct input channels (c), reduction = pixels.  Both dy and
// x are stored pixel-major with channels contiguous, i.e. the reduction index is the slow one:
// TMA boxes of (cw channels, pb pixels) land in shared memory exactly in the swizzled MN-major
// canonical layout (rows = pixels, cw*2 = 32/64/128 bytes per row).  One CTA owns a
// (k-tile, c-tile, tap group) and a range of pixel chunks; a stage holds one chunk: the dy boxes
// (shared by all taps of the group) and, per tap, the x boxes shifted by that tap (zero-filled
// outside the image by TMA).  Each tap accumulates into its own TMEM column range.  Partial sums
// of the pixel ranges are added to dw with vector fp32 reductions.
#include "common.h"
#include "ptx.cuh"

namespace b2c {

struct alignas(64) WgradParams {
    CUtensorMap tmDy;
    CUtensorMap tmX[4];
    TapList taps;
    int bw, bh, bn, tiles_w, tiles_h;  // pixel chunk box and chunk grid
    int pb;                            // pixels per chunk
    int cw, swz;                       // channels per box, descriptor swizzle code
    int ct;                            // x channels per CTA (UMMA N)
    int n_ktiles, n_ctiles, n_groups, taps_per_group, n_splits;
    int chunks_total;
    int stages, tmem_cols;
    int box_bytes, a_boxes, b_boxes;   // bytes per box; dy boxes per stage; x boxes per tap
    int stage_bytes;
    int k_total, c_total, rs_total;
    float* dw;
    unsigned* status;
    unsigned spin_limit;
};

static constexpr int kWgStages = 4;
static constexpr int kWgThreads = 192;
static constexpr uint32_t kWgDrainPolls = 1u << 22;

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

__global__ void __launch_bounds__(kWgThreads, 1) conv_wgrad_kernel(const __grid_constant__ WgradParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kWgStages], empty_bar[kWgStages], accum_bar, drain_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t abort_flag;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;

    int t = blockIdx.x;
    const int ktile = t % p.n_ktiles;
    t /= p.n_ktiles;
    const int ctile = t % p.n_ctiles;
    t /= p.n_ctiles;
    const int group = t % p.n_groups;
    const int split = t / p.n_groups;
    const int chunk_begin = (int)((long long)p.chunks_total * split / p.n_splits);
    const int chunk_end = (int)((long long)p.chunks_total * (split + 1) / p.n_splits);
    const int n_chunks = chunk_end - chunk_begin;
    const int tap0 = group * p.taps_per_group;
    const int n_taps = min(p.taps_per_group, p.taps.count - tap0);
    const int row_bytes = p.cw * 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&accum_bar, 1);
        mbar_init(&drain_bar, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(&tmem_slot, (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    int issued = 0;  // producer lane: chunks whose loads were issued

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&p.tmDy);
            const uint32_t tx = (uint32_t)((p.a_boxes + n_taps * p.b_boxes) * p.box_bytes);
            for (int it = 0; it < n_chunks; ++it, ++issued) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, p.spin_limit, &abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    break;
                }
                int ch = chunk_begin + it;
                const int ow0 = (ch % p.tiles_w) * p.bw;
                ch /= p.tiles_w;
                const int oh0 = (ch % p.tiles_h) * p.bh;
                const int n0 = (ch / p.tiles_h) * p.bn;
                uint8_t* dst = smem + (size_t)s * p.stage_bytes;
                mbar_expect_tx(&full_bar[s], tx);
                for (int j = 0; j < p.a_boxes; ++j)  // boxes past the last channel are zero-filled
                    tma_load_4d(dst + (size_t)j * p.box_bytes, &p.tmDy, &full_bar[s], ktile * 128 + j * p.cw, ow0, oh0, n0);
                dst += (size_t)p.a_boxes * p.box_bytes;
                for (int tl = 0; tl < n_taps; ++tl) {
                    const int tap = tap0 + tl;
                    for (int j = 0; j < p.b_boxes; ++j)
                        tma_load_4d(dst + (size_t)(tl * p.b_boxes + j) * p.box_bytes, &p.tmX[p.taps.map[tap]], &full_bar[s],
                                    ctile * p.ct + j * p.cw, ow0 + p.taps.dw[tap], oh0 + p.taps.dh[tap], n0);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, p.ct, true, true);
            const uint32_t sbo = 8u * (uint32_t)row_bytes;   // eight pixel rows
            const uint32_t lbo = (uint32_t)p.box_bytes;      // next block of cw channels
            const int ksteps = p.pb >> 4;
            bool ok = true;
            for (int it = 0; it < n_chunks; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait_bounded(&full_bar[s], ph, p.spin_limit, &abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t a_addr = smem_u32(smem + (size_t)s * p.stage_bytes);
                const uint32_t b_addr = a_addr + (uint32_t)(p.a_boxes * p.box_bytes);
                for (int tl = 0; tl < n_taps; ++tl) {
                    for (int kk = 0; kk < ksteps; ++kk) {
                        const uint32_t koff = (uint32_t)(kk * 16 * row_bytes);
                        umma_bf16(tmem_base + (uint32_t)(tl * p.ct), make_smem_desc(a_addr + koff, lbo, sbo, (uint32_t)p.swz),
                                  make_smem_desc(b_addr + (uint32_t)(tl * p.b_boxes * p.box_bytes) + koff, lbo, sbo, (uint32_t)p.swz), idesc,
                                  (uint32_t)((it | kk) != 0));
                    }
                }
                umma_commit(&empty_bar[s]);
            }
            if (ok && n_chunks > 0) umma_commit(&accum_bar);
        }
    } else {
        const int q = warp & 3;
        const int m = q * 32 + lane;
        const int k = ktile * 128 + m;
        bool ok = n_chunks > 0;
        if (ok) {
            ok = mbar_wait_bounded(&accum_bar, 0u, p.spin_limit, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok && lane == 0) atomicOr(p.status, B2C_DEV_TIMEOUT);
            tc_fence_after();
        }
        if (ok) {
            for (int tl = 0; tl < n_taps; ++tl) {
                const int rs = p.taps.rs[tap0 + tl];
                float* dst_row = p.dw + ((long long)k * p.rs_total + rs) * p.c_total + ctile * p.ct;
                for (int c0 = 0; c0 < p.ct; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(tl * p.ct + c0), r);
                    tmem_ld_wait();
                    if (k < p.k_total) {
#pragma unroll
                        for (int i = 0; i < 16; i += 4)
                            red_add_v4(dst_row + c0 + i, __uint_as_float(r[i]), __uint_as_float(r[i + 1]), __uint_as_float(r[i + 2]),
                                       __uint_as_float(r[i + 3]));
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (abort_flag) {
        // A wait gave up: let the issued bulk copies land and the issued MMAs retire before exit.
        if (warp == 0 && lane == 0) {
            for (int back = 0; back < S && back < issued; ++back) {
                const int it = issued - 1 - back;
                for (uint32_t i = 0; i < kWgDrainPolls && !mbar_try_wait(&full_bar[it % S], (uint32_t)(it / S) & 1u); ++i) {}
            }
        }
        if (warp == 1 && lane == 0) {
            umma_commit(&drain_bar);
            for (uint32_t i = 0; i < kWgDrainPolls && !mbar_try_wait(&drain_bar, 0u); ++i) {}
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

b2c_status launch_conv_wgrad(b2c_ctx* ctx, const WgradProblem& pb, cudaStream_t stream)
{
    static bool attr_set = false;
    WgradParams p;
    memset(&p, 0, sizeof(p));
    const int R = pb.r;
    if (!(R == 1 || R == 3) || !(pb.stride == 1 || pb.stride == 2) || pb.pad != (R - 1) / 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (pb.n < 1 || pb.c < 16 || pb.c % 16 || pb.k < 16 || pb.k % 16) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (pb.h != pb.p * pb.stride || pb.w != pb.q * pb.stride) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_is_pow2(pb.p) || !b2c_is_pow2(pb.q) || pb.p > 128 || pb.q > 128) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(pb.dy) || !b2c_aligned16(pb.x) || !b2c_aligned16(pb.dw)) return B2C_ERR_MISALIGNED;

    // channels per box: one swizzle row; both tensors use the same width so that one descriptor geometry serves both
    p.cw = (pb.c % 64 == 0 && pb.k % 64 == 0) ? 64 : (pb.c % 32 == 0 && pb.k % 32 == 0) ? 32 : 16;
    p.swz = p.cw == 64 ? SWZ_128B : p.cw == 32 ? SWZ_64B : SWZ_32B;
    p.taps_per_group = R == 3 ? 3 : 1;
    p.n_groups = R == 3 ? 3 : 1;
    // x-channel tile: largest divisor of c that is a multiple of cw, at most 160 (three taps fit 512 TMEM columns)
    p.ct = p.cw;
    for (int cand = 160; cand >= p.cw; cand -= 16)
        if (pb.c % cand == 0 && cand % p.cw == 0) { p.ct = cand; break; }
    p.n_ctiles = pb.c / p.ct;
    p.n_ktiles = (pb.k + 127) / 128;
    p.a_boxes = 128 / p.cw;
    p.b_boxes = p.ct / p.cw;
    p.tmem_cols = 32;
    while (p.tmem_cols < p.taps_per_group * p.ct) p.tmem_cols *= 2;
    if (p.tmem_cols > 512) return B2C_ERR_UNSUPPORTED_SHAPE;

    // pixel chunk: 64 pixels, or 32 when a 64-pixel stage would not leave room for three stages
    p.pb = 64;
    for (;;) {
        p.box_bytes = p.pb * p.cw * 2;
        p.stage_bytes = (p.a_boxes + p.taps_per_group * p.b_boxes) * p.box_bytes;
        if (p.stage_bytes * 3 <= 200 * 1024 || p.pb == 32) break;
        p.pb = 32;
    }
    int stages = (200 * 1024) / p.stage_bytes;
    if (stages > kWgStages) stages = kWgStages;
    if (stages < 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    p.stages = stages;
    p.bw = pb.q < p.pb ? pb.q : p.pb;
    p.bh = (p.pb / p.bw) < pb.p ? (p.pb / p.bw) : pb.p;
    p.bn = p.pb / (p.bw * p.bh);
    p.tiles_w = pb.q / p.bw;
    p.tiles_h = pb.p / p.bh;
    const int tiles_n = (pb.n + p.bn - 1) / p.bn;
    p.chunks_total = p.tiles_w * p.tiles_h * tiles_n;
    const int base = p.n_ktiles * p.n_ctiles * p.n_groups;
    int n_splits = (2 * ctx->sm_count + base - 1) / base;
    if (n_splits > p.chunks_total / 4) n_splits = p.chunks_total / 4;
    if (n_splits < 1) n_splits = 1;
    p.n_splits = n_splits;

    if (!encode_activation_map(ctx, &p.tmDy, pb.dy, pb.n, pb.p, pb.q, pb.k, 1, 0, 0, p.cw, p.bw, p.bh, p.bn)) return B2C_ERR_CUDA;
    if (pb.stride == 2) {
        for (int ph = 0; ph < 2; ++ph)
            for (int pw = 0; pw < 2; ++pw)
                if (!encode_activation_map(ctx, &p.tmX[ph * 2 + pw], pb.x, pb.n, pb.h, pb.w, pb.c, 2, ph, pw, p.cw, p.bw, p.bh, p.bn))
                    return B2C_ERR_CUDA;
    } else {
        if (!encode_activation_map(ctx, &p.tmX[0], pb.x, pb.n, pb.h, pb.w, pb.c, 1, 0, 0, p.cw, p.bw, p.bh, p.bn)) return B2C_ERR_CUDA;
    }
    forward_taps(p.taps, R, pb.stride, pb.pad);
    p.k_total = pb.k;
    p.c_total = pb.c;
    p.rs_total = R * R;
    p.dw = pb.dw;
    p.status = ctx->d_status;
    p.spin_limit = ctx->spin_limit;

    if (!attr_set) {
        B2C_CUDA(cudaFuncSetAttribute(conv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
        attr_set = true;
    }
    const size_t smem_bytes = (size_t)p.stages * p.stage_bytes + 1024;
    dim3 grid((unsigned)(base * n_splits));
    conv_wgrad_kernel<<<grid, kWgThreads, smem_bytes, stream>>>(p);
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

}  // namespace b2c
