// Implicit-GEMM convolution with K-major operands on tcgen05: forward pass and data gradient.
//
//   D[128 pixels x n_tile channels] = sum over (tap, channel block) A[128 x kb] * B[n_tile x kb]^T
//
// A is an im2col tile staged by TMA: a 4-D box (kb channels, bw x bh pixels, bn images) of the
// gathered activation tensor, shifted by the tap's offset; rows that fall outside the image are
// zero-filled by the TMA unit, which implements the padding.  Stride-2 forward convolutions
// gather from four "parity views" of the input (even/odd rows x even/odd columns), each a plain
// strided tensor map; the stride-2 data gradient is four sub-problems, one per output parity.
// B is a box (kb channels, one tap, n_tile output channels) of the [out][tap][in] weights.
// Accumulators live in TMEM; four epilogue warps read them back, add the bias, round to bf16,
// accumulate per-channel sum / sum of squares for BatchNorm, and store.
//
// Warp roles: warp 0 = TMA producer (one lane), warp 1 = TMEM owner + MMA issuer (one lane),
// warps 2..5 = epilogue.  Every mbarrier wait is bounded.
#include "common.h"
#include "ptx.cuh"

namespace b2c {

struct alignas(64) ConvKParams {
    CUtensorMap tmA[4];
    CUtensorMap tmB;
    TapList taps[4];
    int bw, bh, bn;                  // pixel box; bw*bh*bn == 128
    int tiles_w, tiles_h, tiles_n;   // tiles of the output grid
    int n_ktiles, n_tile;            // output-channel tiles, UMMA N
    int kb, c_blocks;                // channels per k-block, k-blocks per tap
    int stages, swz, tmem_cols;
    int a_bytes, b_bytes;            // per stage (b rounded up to 1 KB so that every stage stays 1 KB aligned)
    int tx_bytes;                    // bytes the two TMA loads of a stage deliver
    int n_valid, oc_valid;           // images / output channels that exist
    long long os_n, os_h, os_w;      // output element strides along the tile grid
    long long off[4];                // output element offset per parity
    void* out;
    int out_is_f32;
    const float* bias;
    double* stats;
    int stats_group_images;          // images per BatchNorm statistics group (0: one group)
    unsigned* status;
    unsigned spin_limit;
};

static constexpr int kMaxStages = 8;
static constexpr int kThreads = 192;
static constexpr uint32_t kDrainPolls = 1u << 22;

__global__ void __launch_bounds__(kThreads, 1) conv_kmajor_kernel(const __grid_constant__ ConvKParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], accum_bar, drain_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t abort_flag;
    __shared__ float s_stats[512];

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int par = blockIdx.z;
    const TapList& tl = p.taps[par];
    const int n_iters = tl.count * p.c_blocks;
    const int S = p.stages;

    // tile decode: neighbouring CTAs share the activation tile and differ in the channel tile
    int t = blockIdx.x;
    const int ktile = t % p.n_ktiles;
    t /= p.n_ktiles;
    const int tw = t % p.tiles_w;
    t /= p.tiles_w;
    const int th = t % p.tiles_h;
    const int tn = t / p.tiles_h;
    const int ow0 = tw * p.bw, oh0 = th * p.bh, n0 = tn * p.bn;

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
    const int stage_bytes = p.a_bytes + p.b_bytes;
    int issued = 0;  // producer lane: k-blocks whose loads were issued

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&p.tmB);
            for (int it = 0; it < n_iters; ++it, ++issued) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, p.spin_limit, &abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    break;
                }
                const int tap = it / p.c_blocks, cb = it - tap * p.c_blocks;
                uint8_t* a_dst = smem + (size_t)s * stage_bytes;
                uint8_t* b_dst = a_dst + p.a_bytes;
                mbar_expect_tx(&full_bar[s], (uint32_t)p.tx_bytes);
                tma_load_4d(a_dst, &p.tmA[tl.map[tap]], &full_bar[s], cb * p.kb, ow0 + tl.dw[tap], oh0 + tl.dh[tap], n0);
                tma_load_3d(b_dst, &p.tmB, &full_bar[s], cb * p.kb, tl.rs[tap], ktile * p.n_tile);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, p.n_tile, false, false);
            const uint32_t sbo = 8u * (uint32_t)p.kb * 2u;  // eight rows of kb bf16
            bool ok = true;
            for (int it = 0; it < n_iters; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait_bounded(&full_bar[s], ph, p.spin_limit, &abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                const uint32_t b_addr = a_addr + (uint32_t)p.a_bytes;
                const int ksteps = p.kb >> 4;
                for (int k = 0; k < ksteps; ++k) {
                    umma_bf16(tmem_base, make_smem_desc(a_addr + k * 32, 16, sbo, (uint32_t)p.swz),
                              make_smem_desc(b_addr + k * 32, 16, sbo, (uint32_t)p.swz), idesc, (uint32_t)((it | k) != 0));
                }
                umma_commit(&empty_bar[s]);  // frees the stage once these MMAs have read it
            }
            if (ok && n_iters > 0) umma_commit(&accum_bar);
        }
    } else {
        // ---------------------------------------------------------------- epilogue (128 threads)
        const int q = warp & 3;          // TMEM lane quarter this warp may read
        const int m = q * 32 + lane;     // accumulator row = pixel of the tile (w fastest, then h, then image)
        const int et = threadIdx.x - 64; // 0..127
        const int lw = m % p.bw, lh = (m / p.bw) % p.bh, ln = m / (p.bw * p.bh);
        const bool row_valid = (n0 + ln) < p.n_valid;
        const long long row_off = (long long)(n0 + ln) * p.os_n + (long long)(oh0 + lh) * p.os_h + (long long)(ow0 + lw) * p.os_w + p.off[par];
        const bool do_stats = p.stats != nullptr;

        if (do_stats) {
            for (int i = et; i < 512; i += 128) s_stats[i] = 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");

        bool ok = true;
        if (n_iters > 0) {
            ok = mbar_wait_bounded(&accum_bar, 0u, p.spin_limit, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok && lane == 0) atomicOr(p.status, B2C_DEV_TIMEOUT);
            tc_fence_after();
        }
        if (ok) {
            for (int c0 = 0; c0 < p.n_tile; c0 += 16) {
                uint32_t r[16];
                if (n_iters > 0) {
                    tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = 0u;
                }
                const int ch0 = ktile * p.n_tile + c0;  // first output channel of this chunk
                float v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
                if (p.bias != nullptr) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] += (ch0 + i < p.oc_valid) ? __ldg(p.bias + ch0 + i) : 0.f;
                }
                if (p.out_is_f32) {
                    if (row_valid) {
                        float* dst = reinterpret_cast<float*>(p.out) + row_off + ch0;
#pragma unroll
                        for (int i = 0; i < 16; i += 4)
                            if (ch0 + i < p.oc_valid) *reinterpret_cast<float4*>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    }
                } else {
                    uint32_t pk[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) pk[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
                    if (row_valid) {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + row_off + ch0;
                        if (ch0 < p.oc_valid) *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        if (ch0 + 8 < p.oc_valid) *reinterpret_cast<uint4*>(dst + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    }
                    if (do_stats) {
                        // Column sums over the warp's 32 rows of the values as stored: a butterfly that
                        // halves the number of columns each lane carries (16 -> 8 -> 4 -> 2 -> 1).
                        float a[16], b[16];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            __nv_bfloat162 h = *reinterpret_cast<__nv_bfloat162*>(&pk[i]);
                            const float lo = row_valid ? __low2float(h) : 0.f, hi = row_valid ? __high2float(h) : 0.f;
                            a[2 * i] = lo;
                            a[2 * i + 1] = hi;
                            b[2 * i] = lo * lo;
                            b[2 * i + 1] = hi * hi;
                        }
#pragma unroll
                        for (int width = 8, bit = 16; width >= 1; width >>= 1, bit >>= 1) {
                            const bool upper = (lane & bit) != 0;
#pragma unroll
                            for (int i = 0; i < width; ++i) {
                                const float sa = upper ? a[i] : a[i + width], ka = upper ? a[i + width] : a[i];
                                const float sb = upper ? b[i] : b[i + width], kb_ = upper ? b[i + width] : b[i];
                                a[i] = ka + __shfl_xor_sync(0xffffffffu, sa, bit);
                                b[i] = kb_ + __shfl_xor_sync(0xffffffffu, sb, bit);
                            }
                        }
                        a[0] += __shfl_xor_sync(0xffffffffu, a[0], 1);
                        b[0] += __shfl_xor_sync(0xffffffffu, b[0], 1);
                        if ((lane & 1) == 0) {
                            const int col = c0 + (lane >> 1);  // lane bits 4..1 select the column of the chunk
                            atomicAdd(&s_stats[col], a[0]);
                            atomicAdd(&s_stats[256 + col], b[0]);
                        }
                    }
                }
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (do_stats && ok) {
            for (int c = et; c < p.n_tile; c += 128) {
                const int ch = ktile * p.n_tile + c;
                if (ch < p.oc_valid) {
                    double* st = p.stats + (size_t)(p.stats_group_images > 0 ? n0 / p.stats_group_images : 0) * 2 * p.oc_valid;
                    atomicAdd(st + ch, (double)s_stats[c]);
                    atomicAdd(st + p.oc_valid + ch, (double)s_stats[256 + c]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (abort_flag) {
        // A wait gave up.  Before the CTA may exit, let every bulk copy it issued land and every
        // MMA it issued retire (both finish on their own; the polls here only bound the wait).
        if (warp == 0 && lane == 0) {
            for (int back = 0; back < S && back < issued; ++back) {
                const int it = issued - 1 - back;
                for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(&full_bar[it % S], (uint32_t)(it / S) & 1u); ++i) {}
            }
        }
        if (warp == 1 && lane == 0) {
            umma_commit(&drain_bar);
            for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(&drain_bar, 0u); ++i) {}
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------ host side
static bool encode_map(b2c_ctx* ctx, CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                       const cuuint32_t* box, int inner_bytes)
{
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUtensorMapSwizzle swz = inner_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : inner_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    CUresult r = ctx->encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes, box, estr,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Activation tensor [n][h][w][c] viewed with a spatial step (1: plain; 2: one parity of rows/cols).
bool encode_activation_map(b2c_ctx* ctx, CUtensorMap* tm, const void* base, int n, int h, int w, int c, int step, int ph, int pw, int box_c,
                           int box_w, int box_h, int box_n)
{
    const char* b = reinterpret_cast<const char*>(base) + ((size_t)ph * w + pw) * c * 2;
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)(w / step), (cuuint64_t)(h / step), (cuuint64_t)n};
    cuuint64_t str[3] = {(cuuint64_t)step * c * 2, (cuuint64_t)step * w * c * 2, (cuuint64_t)h * w * c * 2};
    cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)box_w, (cuuint32_t)box_h, (cuuint32_t)box_n};
    return encode_map(ctx, tm, b, 4, dims, str, box, box_c * 2);
}

static int floordiv2(int e) { return (e >= 0) ? e / 2 : -((-e + 1) / 2); }

void forward_taps(TapList& tl, int R, int stride, int pad)
{
    tl.count = 0;
    for (int r = 0; r < R; ++r)
        for (int s = 0; s < R; ++s) {
            const int i = tl.count++;
            const int eh = r - pad, ew = s - pad;
            if (stride == 1) {
                tl.map[i] = 0; tl.dh[i] = (int8_t)eh; tl.dw[i] = (int8_t)ew;
            } else {
                const int hp = eh & 1, wp = ew & 1;
                tl.map[i] = (int8_t)(hp * 2 + wp);
                tl.dh[i] = (int8_t)floordiv2(eh);
                tl.dw[i] = (int8_t)floordiv2(ew);
            }
            tl.rs[i] = (int8_t)(r * R + s);
        }
}

b2c_status launch_conv_kmajor(b2c_ctx* ctx, const KMajorProblem& pb, cudaStream_t stream)
{
    static bool attr_set = false;
    ConvKParams p;
    memset(&p, 0, sizeof(p));
    const int R = pb.r;
    if (!(R == 1 || R == 3) || !(pb.stride == 1 || pb.stride == 2) || pb.pad != (R - 1) / 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (pb.n < 1 || pb.ic < 16 || pb.ic % 16 || pb.oc < 16 || pb.oc % 16) return B2C_ERR_UNSUPPORTED_SHAPE;
    // tile grid = spatial grid each CTA's 128 accumulator rows walk over
    int gh, gw, n_par = 1;
    if (!pb.dgrad) {
        gh = pb.oh; gw = pb.ow;
        if (pb.ih != pb.oh * pb.stride || pb.iw != pb.ow * pb.stride) return B2C_ERR_UNSUPPORTED_SHAPE;
    } else {
        gh = pb.ih; gw = pb.iw;  // the dy grid; for stride 2 each parity of dx has exactly this size
        if (pb.oh != pb.ih * pb.stride || pb.ow != pb.iw * pb.stride) return B2C_ERR_UNSUPPORTED_SHAPE;
        n_par = pb.stride * pb.stride;
    }
    if (!b2c_is_pow2(gh) || !b2c_is_pow2(gw) || gh > 128 || gw > 128) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(pb.in) || !b2c_aligned16(pb.wt) || !b2c_aligned16(pb.out)) return B2C_ERR_MISALIGNED;

    p.bw = gw < 128 ? gw : 128;
    p.bh = (128 / p.bw) < gh ? (128 / p.bw) : gh;
    p.bn = 128 / (p.bw * p.bh);
    p.tiles_w = gw / p.bw;
    p.tiles_h = gh / p.bh;
    p.tiles_n = (pb.n + p.bn - 1) / p.bn;

    p.kb = (pb.ic % 64 == 0) ? 64 : (pb.ic % 32 == 0) ? 32 : 16;
    p.c_blocks = pb.ic / p.kb;
    p.swz = p.kb == 64 ? SWZ_128B : p.kb == 32 ? SWZ_64B : SWZ_32B;
    // output-channel tile: the largest multiple of 16 up to 256 that splits oc evenly
    int n_tile = 16;
    for (int cand = 256; cand >= 16; cand -= 16)
        if (pb.oc % cand == 0) { n_tile = cand; break; }
    p.n_tile = n_tile;
    p.n_ktiles = pb.oc / n_tile;
    p.tmem_cols = 32;
    while (p.tmem_cols < n_tile) p.tmem_cols *= 2;
    p.a_bytes = 128 * p.kb * 2;
    p.b_bytes = ((n_tile * p.kb * 2) + 1023) & ~1023;
    p.tx_bytes = p.a_bytes + n_tile * p.kb * 2;
    const int stage_bytes = p.a_bytes + p.b_bytes;
    int stages = (96 * 1024) / stage_bytes;            // two CTAs per SM when the ring is small
    if (stages < 4) stages = (200 * 1024) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    p.stages = stages;
    const size_t smem_bytes = (size_t)stages * stage_bytes + 1024;

    // tensor maps
    if (!pb.dgrad && pb.stride == 2) {
        for (int ph = 0; ph < 2; ++ph)
            for (int pw = 0; pw < 2; ++pw)
                if (!encode_activation_map(ctx, &p.tmA[ph * 2 + pw], pb.in, pb.n, pb.ih, pb.iw, pb.ic, 2, ph, pw, p.kb, p.bw, p.bh, p.bn))
                    return B2C_ERR_CUDA;
    } else {
        if (!encode_activation_map(ctx, &p.tmA[0], pb.in, pb.n, pb.ih, pb.iw, pb.ic, 1, 0, 0, p.kb, p.bw, p.bh, p.bn)) return B2C_ERR_CUDA;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)pb.ic, (cuuint64_t)(R * R), (cuuint64_t)pb.oc};
        cuuint64_t str[2] = {(cuuint64_t)pb.ic * 2, (cuuint64_t)R * R * pb.ic * 2};
        cuuint32_t box[3] = {(cuuint32_t)p.kb, 1u, (cuuint32_t)n_tile};
        if (!encode_map(ctx, &p.tmB, pb.wt, 3, dims, str, box, p.kb * 2)) return B2C_ERR_CUDA;
    }

    // tap tables
    if (!pb.dgrad) {
        forward_taps(p.taps[0], R, pb.stride, pb.pad);
        p.os_n = (long long)pb.oh * pb.ow * pb.oc; p.os_h = (long long)pb.ow * pb.oc; p.os_w = pb.oc;
    } else if (pb.stride == 1) {
        TapList& tl = p.taps[0];
        for (int r = 0; r < R; ++r)   // r, s index the flipped filter
            for (int s = 0; s < R; ++s) {
                const int i = tl.count++;
                tl.map[i] = 0; tl.dh[i] = (int8_t)(r - (R - 1 - pb.pad)); tl.dw[i] = (int8_t)(s - (R - 1 - pb.pad));
                tl.rs[i] = (int8_t)(r * R + s);
            }
        p.os_n = (long long)pb.oh * pb.ow * pb.oc; p.os_h = (long long)pb.ow * pb.oc; p.os_w = pb.oc;
    } else {
        for (int ph = 0; ph < 2; ++ph)
            for (int pw = 0; pw < 2; ++pw) {
                TapList& tl = p.taps[ph * 2 + pw];
                for (int rf = 0; rf < R; ++rf)
                    for (int sf = 0; sf < R; ++sf) {
                        const int r = R - 1 - rf, s = R - 1 - sf;   // tap of the forward filter
                        const int eh = ph + pb.pad - r, ew = pw + pb.pad - s;
                        if ((eh & 1) || (ew & 1)) continue;
                        const int i = tl.count++;
                        tl.map[i] = 0; tl.dh[i] = (int8_t)(eh / 2); tl.dw[i] = (int8_t)(ew / 2);
                        tl.rs[i] = (int8_t)(rf * R + sf);
                    }
                p.off[ph * 2 + pw] = ((long long)ph * pb.ow + pw) * pb.oc;
            }
        p.os_n = (long long)pb.oh * pb.ow * pb.oc; p.os_h = 2ll * pb.ow * pb.oc; p.os_w = 2ll * pb.oc;
    }
    p.n_valid = pb.n;
    p.oc_valid = pb.oc;
    p.out = pb.out;
    p.out_is_f32 = pb.out_f32 ? 1 : 0;
    p.bias = pb.bias;
    p.stats = pb.out_f32 ? nullptr : pb.stats;
    p.stats_group_images = pb.stats_group_images;
    if (p.stats && p.stats_group_images > 0 && (p.stats_group_images % p.bn) != 0) return B2C_ERR_UNSUPPORTED_SHAPE;  // a tile must not straddle groups
    p.status = ctx->d_status;
    p.spin_limit = ctx->spin_limit;

    if (!attr_set) {
        B2C_CUDA(cudaFuncSetAttribute(conv_kmajor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
        attr_set = true;
    }
    dim3 grid((unsigned)(p.tiles_w * p.tiles_h * p.tiles_n * p.n_ktiles), 1, (unsigned)n_par);
    conv_kmajor_kernel<<<grid, kThreads, smem_bytes, stream>>>(p);
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

}  // namespace b2c
