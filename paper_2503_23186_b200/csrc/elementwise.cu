// HBM-bound kernels of the training step: BatchNorm(+residual)+ReLU forward and backward,
// global average pool, softmax cross-entropy, bias gradient, the fused gradient-average +
// SGD-momentum update, channel padding and the dgrad weight re-layout.
//
// Access pattern common to the BatchNorm kernels: the tensor is [m rows][c channels] bf16 with
// channels contiguous; a thread owns 8 consecutive channels (one 16-byte vector) and walks rows
// with a grid stride, so a warp reads whole 128-byte lines and per-channel reductions stay in
// registers until the end of the walk.  Row sums are combined in shared memory, then added to
// global fp64 accumulators (fp32 partials over few rows, fp64 across them: var = E[y^2] - E[y]^2
// stays accurate for channels whose mean is large against their spread).
#include <cstdlib>
#include "common.h"
#include "ptx.cuh"

namespace b2c {

static constexpr int kEwThreads = 256;

struct bf16x8 {
    uint4 raw;
};
__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8])
{
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __low2float(h[i]);
        f[2 * i + 1] = __high2float(h[i]);
    }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    return make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
}
__device__ __forceinline__ uint4 ld16(const void* base, long long vec_index) { return __ldg(reinterpret_cast<const uint4*>(base) + vec_index); }

// Row/channel-group decomposition shared by the row-walking kernels.  blockIdx.y selects the
// statistics group (a micro-batch): rows [g*m, (g+1)*m) of the tensor, its own accumulators and
// its own saved mean / invstd.  Each thread keeps several independent 16-byte loads per tensor
// in flight (rows beyond the end read as zero and contribute nothing).
struct RowWalk {
    int groups;         // c / 8
    int rows_per_iter;  // rows a block covers per step
    __device__ RowWalk(int c) : groups(c >> 3), rows_per_iter(kEwThreads / (c >> 3)) {}
};
__device__ __forceinline__ uint4 ld16_or_zero(const void* base, long long vec_index, bool ok)
{
    return ok ? __ldg(reinterpret_cast<const uint4*>(base) + vec_index) : make_uint4(0u, 0u, 0u, 0u);
}

// A thread's 8 + 8 per-channel sums into the block's shared accumulators.  Threads of a warp whose lanes differ by a
// multiple of the group count hold the same channels: where the group count is a power of two below 32 those lanes add
// up with shuffles first and one lane per channel group issues the shared-memory atomics, which leaves one contender
// per warp and address instead of one per row (32 rows on the same address took several microseconds per block).
// `whole_warps`: every lane of every calling warp is active (the group count divides the block).
__device__ __forceinline__ void block_accumulate(float* s_acc, int c, int groups, int g, float (&a)[8], float (&b)[8], bool active)
{
    const bool warp_reduce = groups < 32 && (groups & (groups - 1)) == 0;   // uniform over the block; all threads are active then
    if (warp_reduce) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            if (off >= groups) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    a[i] += __shfl_xor_sync(0xffffffffu, a[i], off);
                    b[i] += __shfl_xor_sync(0xffffffffu, b[i], off);
                }
            }
        }
        if ((int)(threadIdx.x & 31) >= groups) return;
    }
    if (!active) return;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        atomicAdd(&s_acc[g * 8 + i], a[i]);
        atomicAdd(&s_acc[c + g * 8 + i], b[i]);
    }
}

// ------------------------------------------------------------------------------ BN forward
// Rows in flight per thread in the statistics pass: it reads one tensor only (see bn_apply_kernel).
static constexpr int kStatsUnroll = 8;
__global__ void __launch_bounds__(kEwThreads, 2) bn_stats_kernel(const void* __restrict__ y, long long m, int c, double* __restrict__ stats)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    extern __shared__ float s_acc[];  // [2*c]
    for (int i = threadIdx.x; i < 2 * c; i += kEwThreads) s_acc[i] = 0.f;
    __syncthreads();
    const RowWalk rw(c);
    const int g = threadIdx.x % rw.groups, rl = threadIdx.x / rw.groups;
    const long long base = (long long)blockIdx.y * m * rw.groups;
    if (rl < rw.rows_per_iter) {
        float s[8], ss[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) s[i] = ss[i] = 0.f;
        const long long step = (long long)gridDim.x * rw.rows_per_iter;
        for (long long r = (long long)blockIdx.x * rw.rows_per_iter + rl; r < m; r += kStatsUnroll * step) {
            uint4 v[kStatsUnroll];
#pragma unroll
            for (int u = 0; u < kStatsUnroll; ++u) v[u] = ld16_or_zero(y, base + (r + u * step) * rw.groups + g, r + u * step < m);
#pragma unroll
            for (int u = 0; u < kStatsUnroll; ++u) {
                float f[8];
                unpack8(v[u], f);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    s[i] += f[i];
                    ss[i] = fmaf(f[i], f[i], ss[i]);
                }
            }
        }
        block_accumulate(s_acc, c, rw.groups, g, s, ss, true);
    }
    __syncthreads();
    double* out = stats + (size_t)blockIdx.y * 2 * c;
    for (int i = threadIdx.x; i < 2 * c; i += kEwThreads) atomicAdd(out + i, (double)s_acc[i]);
}

// mean and 1/sqrt(var+eps) from the fp64 sums, identically in every thread that needs them.
__device__ __forceinline__ void bn_moments(const double* stats, int c, int ch, double inv_m, float eps, float& mean, float& invstd, float& var)
{
    const double mu = stats[ch] * inv_m;
    double v = stats[c + ch] * inv_m - mu * mu;
    v = v < 0.0 ? 0.0 : v;
    mean = (float)mu;
    var = (float)v;
    invstd = rsqrtf((float)v + eps);
}

// UNROLL independent 16-byte loads per tensor and thread are in flight: without a residual the kernel reads one tensor,
// so it takes twice the rows per step to keep as many bytes in flight as the residual variant (HBM latency x bandwidth).
template <int UNROLL, bool RES>
__global__ void __launch_bounds__(kEwThreads, 2) bn_apply_kernel(const void* __restrict__ y, long long m, int c, const double* __restrict__ stats_all,
                                                                 const float* __restrict__ gamma, const float* __restrict__ beta,
                                                                 const void* __restrict__ residual, int relu, float eps, void* __restrict__ a,
                                                                 float* save_mean, float* save_invstd, float* run_mean, float* run_var,
                                                                 float momentum, uint8_t* __restrict__ relu_mask)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const RowWalk rw(c);
    const int g = threadIdx.x % rw.groups, rl = threadIdx.x / rw.groups;
    const double inv_m = 1.0 / (double)m;
    const double* stats = stats_all + (size_t)blockIdx.y * 2 * c;
    const long long base = (long long)blockIdx.y * m * rw.groups;
    if (blockIdx.x == 0) {
        for (int ch = threadIdx.x; ch < c; ch += kEwThreads) {
            float mean, invstd, var;
            bn_moments(stats, c, ch, inv_m, eps, mean, invstd, var);
            save_mean[(size_t)blockIdx.y * c + ch] = mean;
            save_invstd[(size_t)blockIdx.y * c + ch] = invstd;
            if (run_mean != nullptr) {
                const float unbiased = m > 1 ? var * (float)((double)m / (double)(m - 1)) : var;
                run_mean[ch] = (1.f - momentum) * run_mean[ch] + momentum * mean;
                run_var[ch] = (1.f - momentum) * run_var[ch] + momentum * unbiased;
            }
        }
    }
    if (rl >= rw.rows_per_iter) return;
    float scale[8], shift[8], bt[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float mean, invstd, var;
        bn_moments(stats, c, g * 8 + i, inv_m, eps, mean, invstd, var);
        // z = gamma*(y-mean)*invstd + beta, evaluated as (y-mean)*(gamma*invstd) + beta
        scale[i] = gamma[g * 8 + i] * invstd;
        shift[i] = mean;
        bt[i] = beta[g * 8 + i];
    }
    const long long step = (long long)gridDim.x * rw.rows_per_iter;
    for (long long r = (long long)blockIdx.x * rw.rows_per_iter + rl; r < m; r += UNROLL * step) {
        uint4 vy[UNROLL], vr[RES ? UNROLL : 1];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const bool ok = r + u * step < m;
            const long long vi = base + (r + u * step) * rw.groups + g;
            vy[u] = ld16_or_zero(y, vi, ok);
            if constexpr (RES) vr[u] = ld16_or_zero(residual, vi, ok);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            if (r + u * step >= m) break;
            float f[8], res[8];
            unpack8(vy[u], f);
            if constexpr (RES) unpack8(vr[u], res);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float z = fmaf(f[i] - shift[i], scale[i], bt[i]);
                if constexpr (RES) z += res[i];
                f[i] = (relu && z < 0.f) ? 0.f : z;
            }
            const uint4 packed = pack8(f);
            reinterpret_cast<uint4*>(a)[base + (r + u * step) * rw.groups + g] = packed;
            if (relu_mask != nullptr) {   // one bit per stored output: "a > 0", read by the backward pass instead of a
                float st[8];
                unpack8(packed, st);
                unsigned bits = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) bits |= (st[i] > 0.f ? 1u : 0u) << i;
                relu_mask[base + (r + u * step) * rw.groups + g] = (uint8_t)bits;
            }
        }
    }
}

// ------------------------------------------------------------------------------ BN backward
// Pass 1: S1 = sum dz, S2 = sum dz*y per channel (dgamma = invstd*(S2 - mean*S1) is formed in fp64 by pass 2).
__global__ void __launch_bounds__(kEwThreads, 2) bn_bwd_reduce_kernel(const void* __restrict__ da1, const void* __restrict__ da2,
                                                                      const void* __restrict__ y, const void* __restrict__ a, long long m, int c,
                                                                      int relu, double* __restrict__ sums_all /* [G][2c] */,
                                                                      const uint8_t* __restrict__ relu_mask)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    extern __shared__ float s_acc[];
    for (int i = threadIdx.x; i < 2 * c; i += kEwThreads) s_acc[i] = 0.f;
    __syncthreads();
    const RowWalk rw(c);
    const int g = threadIdx.x % rw.groups, rl = threadIdx.x / rw.groups;
    const long long base = (long long)blockIdx.y * m * rw.groups;
    if (rl < rw.rows_per_iter) {
        float sb[8], sg[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) sb[i] = sg[i] = 0.f;
        const long long step = (long long)gridDim.x * rw.rows_per_iter;
        constexpr int U = 2;
        for (long long r = (long long)blockIdx.x * rw.rows_per_iter + rl; r < m; r += U * step) {
            uint4 v1[U], v2[U], vy[U], va[U];
            unsigned mk[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool ok = r + u * step < m;
                const long long vi = base + (r + u * step) * rw.groups + g;
                v1[u] = ld16_or_zero(da1, vi, ok);
                if (da2 != nullptr) v2[u] = ld16_or_zero(da2, vi, ok);
                vy[u] = ld16_or_zero(y, vi, ok);
                mk[u] = 0xffu;
                if (relu) {
                    if (relu_mask != nullptr) mk[u] = ok ? (unsigned)__ldg(relu_mask + vi) : 0u;
                    else va[u] = ld16_or_zero(a, vi, ok);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float d[8], d2[8], fy[8], fa[8];
                unpack8(v1[u], d);
                if (da2 != nullptr) unpack8(v2[u], d2);
                unpack8(vy[u], fy);
                if (relu && relu_mask == nullptr) {
                    unpack8(va[u], fa);
                    unsigned bits = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) bits |= (fa[i] > 0.f ? 1u : 0u) << i;
                    mk[u] = bits;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float dz = d[i];
                    if (da2 != nullptr) dz += d2[i];
                    if (!((mk[u] >> i) & 1u)) dz = 0.f;
                    sb[i] += dz;
                    sg[i] = fmaf(dz, fy[i], sg[i]);
                }
            }
        }
        block_accumulate(s_acc, c, rw.groups, g, sb, sg, true);
    }
    __syncthreads();
    double* out = sums_all + (size_t)blockIdx.y * 2 * c;
    for (int i = threadIdx.x; i < 2 * c; i += kEwThreads) atomicAdd(out + i, (double)s_acc[i]);
}

// Pass 2: dy = gamma*invstd*(dz - dbeta/m - xhat*dgamma/m), dres = dz; block 0 of each group emits dgamma, dbeta.
__global__ void __launch_bounds__(kEwThreads, 2) bn_bwd_apply_kernel(const void* __restrict__ da1, const void* __restrict__ da2,
                                                                     const void* __restrict__ y, const void* __restrict__ a, long long m, int c,
                                                                     const float* __restrict__ gamma, const float* __restrict__ mean_all,
                                                                     const float* __restrict__ invstd_all, int relu,
                                                                     const double* __restrict__ sums_all, void* __restrict__ dy,
                                                                     void* __restrict__ dres, float* dgamma, float* dbeta, int acc,
                                                                     const uint8_t* __restrict__ relu_mask)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const RowWalk rw(c);
    const int g = threadIdx.x % rw.groups, rl = threadIdx.x / rw.groups;
    const double* sums = sums_all + (size_t)blockIdx.y * 2 * c;
    const float* mean = mean_all + (size_t)blockIdx.y * c;
    const float* invstd = invstd_all + (size_t)blockIdx.y * c;
    const long long base = (long long)blockIdx.y * m * rw.groups;
    if (blockIdx.x == 0) {
        for (int ch = threadIdx.x; ch < c; ch += kEwThreads) {
            const double s1 = sums[ch], s2 = sums[c + ch];
            const float db = (float)s1, dg = (float)((double)invstd[ch] * (s2 - (double)mean[ch] * s1));
            if (gridDim.y == 1) {
                dbeta[ch] = acc ? dbeta[ch] + db : db;
                dgamma[ch] = acc ? dgamma[ch] + dg : dg;
            } else {   // several groups add into the same gradient (always accumulating)
                atomicAdd(dbeta + ch, db);
                atomicAdd(dgamma + ch, dg);
            }
        }
    }
    if (rl >= rw.rows_per_iter) return;
    const double inv_m = 1.0 / (double)m;
    float mu[8], k0[8], kb[8], kg[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int ch = g * 8 + i;
        const double s1 = sums[ch], s2 = sums[c + ch];
        const double is = (double)invstd[ch], dgam = is * (s2 - (double)mean[ch] * s1);
        mu[i] = mean[ch];
        k0[i] = gamma[ch] * invstd[ch];                        // gamma*invstd
        kb[i] = (float)(s1 * inv_m);                           // dbeta/m
        kg[i] = (float)(dgam * inv_m * is);                    // (dgamma/m)*invstd, multiplies (y-mean)
    }
    const long long step = (long long)gridDim.x * rw.rows_per_iter;
    constexpr int U = 2;
    for (long long r = (long long)blockIdx.x * rw.rows_per_iter + rl; r < m; r += U * step) {
        uint4 v1[U], v2[U], vy[U], va[U];
        unsigned mk[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool ok = r + u * step < m;
            const long long vi = base + (r + u * step) * rw.groups + g;
            v1[u] = ld16_or_zero(da1, vi, ok);
            if (da2 != nullptr) v2[u] = ld16_or_zero(da2, vi, ok);
            vy[u] = ld16_or_zero(y, vi, ok);
            mk[u] = 0xffu;
            if (relu) {
                if (relu_mask != nullptr) mk[u] = ok ? (unsigned)__ldg(relu_mask + vi) : 0u;
                else va[u] = ld16_or_zero(a, vi, ok);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (r + u * step >= m) break;
            float d[8], d2[8], fy[8], fa[8], o[8];
            unpack8(v1[u], d);
            if (da2 != nullptr) unpack8(v2[u], d2);
            unpack8(vy[u], fy);
            if (relu && relu_mask == nullptr) {
                unpack8(va[u], fa);
                unsigned bits = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) bits |= (fa[i] > 0.f ? 1u : 0u) << i;
                mk[u] = bits;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float dz = d[i];
                if (da2 != nullptr) dz += d2[i];
                if (!((mk[u] >> i) & 1u)) dz = 0.f;
                d[i] = dz;
                o[i] = k0[i] * (dz - kb[i] - (fy[i] - mu[i]) * kg[i]);
            }
            const long long vi = base + (r + u * step) * rw.groups + g;
            reinterpret_cast<uint4*>(dy)[vi] = pack8(o);
            if (dres != nullptr) reinterpret_cast<uint4*>(dres)[vi] = pack8(d);
        }
    }
}

// ------------------------------------------------------------------------------ BN backward, staged through shared memory
// The same two passes fed by bulk copies: a producer thread streams chunks of every input tensor (and of the ReLU bit
// mask) into a ring of shared-memory stages with cp.async.bulk, eight consumer warps work from shared memory.  A
// register-staged row walk keeps two 16-byte loads per tensor and thread in flight, too few bytes to hide the DRAM
// latency at two blocks per SM; the ring keeps kStStages x ~25 KB per block in flight and costs no registers.
//   chunk = 2 * rows_per_iter rows = 2 vectors per active thread and tensor (about 8 KB per tensor); chunk k of a group
//   goes to block k % gridDim.x; a ragged last chunk is read with plain loads.
static constexpr int kStStages = 4;
static constexpr int kStThreads = kEwThreads + 32;   // consumer warps + the producer warp

struct StagedWalk {
    int groups, rpi, active, chunk_rows, chunk_vecs, nt, mask_stride, stage_bytes;
    long long n_full;
    __device__ StagedWalk(int c, long long m, int n_tensors, bool has_mask, int vecs = 2)   // vecs: vectors per thread, tensor and stage
    {
        groups = c >> 3;
        rpi = kEwThreads / groups;
        active = rpi * groups;
        chunk_rows = vecs * rpi;
        chunk_vecs = vecs * active;
        nt = n_tensors;
        mask_stride = has_mask ? ((chunk_vecs + 127) & ~127) : 0;
        stage_bytes = nt * chunk_vecs * 16 + mask_stride;
        n_full = m / chunk_rows;
    }
};

// Producer side: one thread.  Returns the number of chunks it issued (for the drain after an aborted wait).
__device__ __forceinline__ int staged_produce(const StagedWalk& sw, uint8_t* ring, uint64_t* full, uint64_t* empty, const void* t0, const void* t1,
                                              const void* t2, const uint8_t* mask, long long base_vec, unsigned spin_limit, uint32_t* abort_flag,
                                              unsigned* status)
{
    int i = 0;
    const uint32_t tbytes = (uint32_t)sw.chunk_vecs * 16u;
    const uint32_t tx = (uint32_t)sw.nt * tbytes + (mask != nullptr ? (uint32_t)sw.chunk_vecs : 0u);
    for (long long k = blockIdx.x; k < sw.n_full; k += gridDim.x, ++i) {
        const int s = i % kStStages;
        if (!mbar_wait_bounded(&empty[s], (((uint32_t)(i / kStStages)) & 1u) ^ 1u, spin_limit, abort_flag)) {
            atomicOr(status, B2C_DEV_TIMEOUT);
            break;
        }
        uint8_t* dst = ring + (size_t)s * sw.stage_bytes;
        const long long v0 = base_vec + k * sw.chunk_vecs;
        mbar_expect_tx(&full[s], tx);
        bulk_load(dst, reinterpret_cast<const uint4*>(t0) + v0, tbytes, &full[s]);
        bulk_load(dst + tbytes, reinterpret_cast<const uint4*>(t1) + v0, tbytes, &full[s]);
        if (sw.nt > 2) bulk_load(dst + 2 * tbytes, reinterpret_cast<const uint4*>(t2) + v0, tbytes, &full[s]);
        if (mask != nullptr) bulk_load(dst + sw.nt * tbytes, mask + v0, (uint32_t)sw.chunk_vecs, &full[s]);
    }
    return i;
}
// After an aborted wait: the copies already issued must land before the block may exit.
__device__ __forceinline__ void staged_drain(int issued, uint64_t* full, int S = kStStages)
{
    for (int back = 0; back < S && back < issued; ++back) {
        const int it = issued - 1 - back;
        for (uint32_t i = 0; i < (1u << 22) && !mbar_try_wait(&full[it % S], (uint32_t)(it / S) & 1u); ++i) {}
    }
}
// Consumer side of one chunk: wait (one poller per warp), then the caller reads its two vectors per tensor.
__device__ __forceinline__ bool staged_wait(uint64_t* full, int i, int lane, unsigned spin_limit, uint32_t* abort_flag, unsigned* status,
                                            int S = kStStages)
{
    bool ok = true;
    if (lane == 0) {
        ok = mbar_wait_bounded(&full[i % S], (uint32_t)(i / S) & 1u, spin_limit, abort_flag);
        if (!ok) atomicOr(status, B2C_DEV_TIMEOUT);
    }
    return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void staged_release(uint64_t* empty, int i, int lane, int S = kStStages)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[i % S]);
}
__device__ __forceinline__ void staged_init(uint64_t* full, uint64_t* empty, uint32_t* abort_flag)
{
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kEwThreads / 32);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
}

__global__ void __launch_bounds__(kStThreads, 2) bn_bwd_reduce_staged_kernel(const void* __restrict__ da1, const void* __restrict__ da2,
                                                                             const void* __restrict__ y, long long m, int c, int relu,
                                                                             double* __restrict__ sums_all, const uint8_t* __restrict__ relu_mask,
                                                                             unsigned spin_limit, unsigned* status)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    extern __shared__ uint8_t st_raw[];
    __shared__ uint64_t full[kStStages], empty[kStStages];
    __shared__ uint32_t abort_flag;
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(st_raw) + 127u) & ~uintptr_t(127));
    const StagedWalk sw(c, m, da2 != nullptr ? 3 : 2, relu != 0);
    float* s_acc = reinterpret_cast<float*>(ring + (size_t)kStStages * sw.stage_bytes);
    for (int i = threadIdx.x; i < 2 * c; i += kStThreads) s_acc[i] = 0.f;
    staged_init(full, empty, &abort_flag);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long base = (long long)blockIdx.y * m * sw.groups;
    const uint8_t* mask = relu ? relu_mask : nullptr;
    int issued = 0;
    if (warp == kEwThreads / 32) {
        if (lane == 0) issued = staged_produce(sw, ring, full, empty, da1, y, da2, mask, base, spin_limit, &abort_flag, status);
    } else {
        const int g = threadIdx.x % sw.groups;
        const bool act = threadIdx.x < sw.active;
        const uint32_t tbytes = (uint32_t)sw.chunk_vecs * 16u;
        float sb[8], sg[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) sb[i] = sg[i] = 0.f;
        auto accumulate = [&](const uint4& v1, const uint4& vy, const uint4& v2, bool two, unsigned mk) {
            float d[8], d2[8], fy[8];
            unpack8(v1, d);
            if (two) unpack8(v2, d2);
            unpack8(vy, fy);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float dz = d[i];
                if (two) dz += d2[i];
                if (!((mk >> i) & 1u)) dz = 0.f;
                sb[i] += dz;
                sg[i] = fmaf(dz, fy[i], sg[i]);
            }
        };
        int i = 0;
        bool ok = true;
        for (long long k = blockIdx.x; k < sw.n_full; k += gridDim.x, ++i) {
            ok = staged_wait(full, i, lane, spin_limit, &abort_flag, status);
            if (!ok) break;
            if (act) {
                const uint8_t* st = ring + (size_t)(i % kStStages) * sw.stage_bytes;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int v = u * sw.active + threadIdx.x;
                    const uint4 v1 = reinterpret_cast<const uint4*>(st)[v];
                    const uint4 vy = reinterpret_cast<const uint4*>(st + tbytes)[v];
                    uint4 v2 = make_uint4(0u, 0u, 0u, 0u);
                    if (sw.nt > 2) v2 = reinterpret_cast<const uint4*>(st + 2 * tbytes)[v];
                    const unsigned mk = mask != nullptr ? (unsigned)st[sw.nt * tbytes + v] : 0xffu;
                    accumulate(v1, vy, v2, sw.nt > 2, mk);
                }
            }
            staged_release(empty, i, lane);
        }
        // ragged tail of the group: plain loads, by the block whose turn it would be
        if (ok && act && (long long)sw.n_full * sw.chunk_rows < m && (sw.n_full % gridDim.x) == blockIdx.x) {
            for (long long r = sw.n_full * sw.chunk_rows + threadIdx.x / sw.groups; r < m; r += sw.rpi) {
                const long long vi = base + r * sw.groups + g;
                const uint4 v1 = ld16(da1, vi), vy = ld16(y, vi);
                const uint4 v2 = da2 != nullptr ? ld16(da2, vi) : make_uint4(0u, 0u, 0u, 0u);
                const unsigned mk = mask != nullptr ? (unsigned)__ldg(mask + vi) : 0xffu;
                accumulate(v1, vy, v2, da2 != nullptr, mk);
            }
        }
        block_accumulate(s_acc, c, sw.groups, g, sb, sg, act);
    }
    __syncthreads();
    if (abort_flag && warp == kEwThreads / 32 && lane == 0) staged_drain(issued, full);
    double* out = sums_all + (size_t)blockIdx.y * 2 * c;
    for (int i = threadIdx.x; i < 2 * c; i += kStThreads) atomicAdd(out + i, (double)s_acc[i]);
    __syncthreads();
}

__global__ void __launch_bounds__(kStThreads, 2) bn_bwd_apply_staged_kernel(const void* __restrict__ da1, const void* __restrict__ da2,
                                                                            const void* __restrict__ y, long long m, int c,
                                                                            const float* __restrict__ gamma, const float* __restrict__ mean_all,
                                                                            const float* __restrict__ invstd_all, int relu,
                                                                            const double* __restrict__ sums_all, void* __restrict__ dy,
                                                                            void* __restrict__ dres, float* dgamma, float* dbeta, int acc,
                                                                            const uint8_t* __restrict__ relu_mask, unsigned spin_limit,
                                                                            unsigned* status)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    extern __shared__ uint8_t st_raw[];
    __shared__ uint64_t full[kStStages], empty[kStStages];
    __shared__ uint32_t abort_flag;
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(st_raw) + 127u) & ~uintptr_t(127));
    const StagedWalk sw(c, m, da2 != nullptr ? 3 : 2, relu != 0);
    staged_init(full, empty, &abort_flag);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const double* sums = sums_all + (size_t)blockIdx.y * 2 * c;
    const float* mean = mean_all + (size_t)blockIdx.y * c;
    const float* invstd = invstd_all + (size_t)blockIdx.y * c;
    const long long base = (long long)blockIdx.y * m * sw.groups;
    const uint8_t* mask = relu ? relu_mask : nullptr;
    int issued = 0;
    if (warp == kEwThreads / 32) {
        if (lane == 0) issued = staged_produce(sw, ring, full, empty, da1, y, da2, mask, base, spin_limit, &abort_flag, status);
    } else {
        if (blockIdx.x == 0) {
            for (int ch = threadIdx.x; ch < c; ch += kEwThreads) {
                const double s1 = sums[ch], s2 = sums[c + ch];
                const float db = (float)s1, dg = (float)((double)invstd[ch] * (s2 - (double)mean[ch] * s1));
                if (gridDim.y == 1) {
                    dbeta[ch] = acc ? dbeta[ch] + db : db;
                    dgamma[ch] = acc ? dgamma[ch] + dg : dg;
                } else {   // several groups add into the same gradient (always accumulating)
                    atomicAdd(dbeta + ch, db);
                    atomicAdd(dgamma + ch, dg);
                }
            }
        }
        const int g = threadIdx.x % sw.groups;
        const bool act = threadIdx.x < sw.active;
        const uint32_t tbytes = (uint32_t)sw.chunk_vecs * 16u;
        const double inv_m = 1.0 / (double)m;
        float mu[8], k0[8], kb[8], kg[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int ch = g * 8 + i;
            const double s1 = sums[ch], s2 = sums[c + ch];
            const double is = (double)invstd[ch], dgam = is * (s2 - (double)mean[ch] * s1);
            mu[i] = mean[ch];
            k0[i] = gamma[ch] * invstd[ch];                        // gamma*invstd
            kb[i] = (float)(s1 * inv_m);                           // dbeta/m
            kg[i] = (float)(dgam * inv_m * is);                    // (dgamma/m)*invstd, multiplies (y-mean)
        }
        auto emit = [&](const uint4& v1, const uint4& vy, const uint4& v2, bool two, unsigned mk, long long vi) {
            float d[8], d2[8], fy[8], o[8];
            unpack8(v1, d);
            if (two) unpack8(v2, d2);
            unpack8(vy, fy);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float dz = d[i];
                if (two) dz += d2[i];
                if (!((mk >> i) & 1u)) dz = 0.f;
                d[i] = dz;
                o[i] = k0[i] * (dz - kb[i] - (fy[i] - mu[i]) * kg[i]);
            }
            reinterpret_cast<uint4*>(dy)[vi] = pack8(o);
            if (dres != nullptr) reinterpret_cast<uint4*>(dres)[vi] = pack8(d);
        };
        int i = 0;
        bool ok = true;
        for (long long k = blockIdx.x; k < sw.n_full; k += gridDim.x, ++i) {
            ok = staged_wait(full, i, lane, spin_limit, &abort_flag, status);
            if (!ok) break;
            if (act) {
                const uint8_t* st = ring + (size_t)(i % kStStages) * sw.stage_bytes;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int v = u * sw.active + threadIdx.x;
                    const uint4 v1 = reinterpret_cast<const uint4*>(st)[v];
                    const uint4 vy = reinterpret_cast<const uint4*>(st + tbytes)[v];
                    uint4 v2 = make_uint4(0u, 0u, 0u, 0u);
                    if (sw.nt > 2) v2 = reinterpret_cast<const uint4*>(st + 2 * tbytes)[v];
                    const unsigned mk = mask != nullptr ? (unsigned)st[sw.nt * tbytes + v] : 0xffu;
                    emit(v1, vy, v2, sw.nt > 2, mk, base + k * sw.chunk_vecs + v);
                }
            }
            staged_release(empty, i, lane);
        }
        if (ok && act && (long long)sw.n_full * sw.chunk_rows < m && (sw.n_full % gridDim.x) == blockIdx.x) {
            for (long long r = sw.n_full * sw.chunk_rows + threadIdx.x / sw.groups; r < m; r += sw.rpi) {
                const long long vi = base + r * sw.groups + g;
                const uint4 v1 = ld16(da1, vi), vy = ld16(y, vi);
                const uint4 v2 = da2 != nullptr ? ld16(da2, vi) : make_uint4(0u, 0u, 0u, 0u);
                const unsigned mk = mask != nullptr ? (unsigned)__ldg(mask + vi) : 0xffu;
                emit(v1, vy, v2, da2 != nullptr, mk, vi);
            }
        }
    }
    __syncthreads();
    if (abort_flag && warp == kEwThreads / 32 && lane == 0) staged_drain(issued, full);
    __syncthreads();
}

// ------------------------------------------------------------------------------ BN backward, both passes in one launch
// One cooperative launch walks the statistics groups (micro-batches) in order: the reduction pass R(g) of a group, a
// grid-wide barrier, then the apply pass A(g) of the same group, which finds the group's tensors still in L2 (a group
// of a 1024-image layer is an eighth of the tensor: da and y of 17 MB each against 134 MB for all groups, which do not
// fit the L2).  HBM traffic per element drops from 10.25 bytes (two passes over da and y, one write) to about 6.1.
// The barrier of group g is split: a block arrives after R(g), runs the reduction passes of the next `ahead` groups, and
// only then needs the group's sums, so the barrier latency hides behind useful work; a helper warp does the arriving,
// the waiting and the coefficient arithmetic beside the streaming warps.  Small layers (whole tensor in L2
// anyway) look further ahead; they gain the second launch.  The launch is cooperative (all blocks co-resident), every
// wait is bounded, and a block that gives up raises the status word and winds down like the other staged kernels.
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEwThreads) : "memory"); }
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Producer: the full chunks of one group, continuing the ring at stage index i.  False if a wait gave up.
__device__ __forceinline__ bool staged_produce_group(const StagedWalk& sw, uint8_t* ring, uint64_t* full, uint64_t* empty, const void* t0,
                                                     const void* t1, const void* t2, const uint8_t* mask, long long base_vec, int& i,
                                                     unsigned spin_limit, uint32_t* abort_flag, unsigned* status, uint64_t policy, int S)
{
    const uint32_t tbytes = (uint32_t)sw.chunk_vecs * 16u;
    const uint32_t tx = (uint32_t)sw.nt * tbytes + (mask != nullptr ? (uint32_t)sw.chunk_vecs : 0u);
    for (long long k = blockIdx.x; k < sw.n_full; k += gridDim.x, ++i) {
        const int s = i % S;
        if (!mbar_wait_bounded(&empty[s], (((uint32_t)(i / S)) & 1u) ^ 1u, spin_limit, abort_flag)) {
            atomicOr(status, B2C_DEV_TIMEOUT);
            return false;
        }
        uint8_t* dst = ring + (size_t)s * sw.stage_bytes;
        const long long v0 = base_vec + k * sw.chunk_vecs;
        mbar_expect_tx(&full[s], tx);
        bulk_load_hint(dst, reinterpret_cast<const uint4*>(t0) + v0, tbytes, &full[s], policy);
        bulk_load_hint(dst + tbytes, reinterpret_cast<const uint4*>(t1) + v0, tbytes, &full[s], policy);
        if (sw.nt > 2) bulk_load_hint(dst + 2 * tbytes, reinterpret_cast<const uint4*>(t2) + v0, tbytes, &full[s], policy);
        if (mask != nullptr) bulk_load_hint(dst + sw.nt * tbytes, mask + v0, (uint32_t)sw.chunk_vecs, &full[s], policy);
    }
    return true;
}

// Block of the grouped kernel: eight consumer warps, the producer warp, and a helper warp that takes the work between
// two passes off the consumers' path (adding the block's partial sums to the group's global sums, the arrival at the
// group's barrier, the wait for the other blocks and the group's coefficients), so that the consumers only stream.
static constexpr int kGrThreads = kEwThreads + 64;
// Named barriers between the consumers (c) and the helper (h); a barrier completes once kEwThreads + 32 threads have
// arrived or synchronised on it.  Every role runs the same sequence of barrier operations whether or not a wait has
// given up (after a failure only the work in between is skipped), so none of them can be left waiting.
//   2: partial sums of R(t) are in shared memory        (c arrive, h sync)
//   3: the partial-sum slots may be overwritten          (h arrive, c sync)
//   4: coefficients of A(ga) are in shared memory        (h arrive, c sync)
//   5: the coefficient table may be overwritten          (c arrive, h sync)
__device__ __forceinline__ void named_sync(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(kEwThreads + 32) : "memory"); }
__device__ __forceinline__ void named_arrive(int id) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "n"(kEwThreads + 32) : "memory"); }

__global__ void __launch_bounds__(kGrThreads, 2) bn_bwd_grouped_kernel(const void* __restrict__ da1, const void* __restrict__ da2,
                                                                       const void* __restrict__ y, long long m, int c, int n_groups, int ahead,
                                                                       const float* __restrict__ gamma, const float* __restrict__ mean_all,
                                                                       const float* __restrict__ invstd_all, int relu, double* sums_all,
                                                                       unsigned* arrivals, void* __restrict__ dy, void* __restrict__ dres,
                                                                       float* dgamma, float* dbeta, int acc, const uint8_t* __restrict__ relu_mask,
                                                                       unsigned spin_limit, unsigned* status, int vecs, int S)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    extern __shared__ uint8_t st_raw[];
    __shared__ uint64_t full[kStStages], empty[kStStages];
    __shared__ uint32_t abort_flag;
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(st_raw) + 127u) & ~uintptr_t(127));
    const StagedWalk sw(c, m, da2 != nullptr ? 3 : 2, relu != 0, vecs);   // S ring stages of `vecs` vectors per thread and tensor
    // Per-block partial sums without atomics: every consumer thread owns one (row, channel group) pair, so it stores
    // its 16 sums into its own slot [slot][2c]; channel groups narrower than a warp first add up the rows a warp holds
    // with shuffles (slot = warp), otherwise slot = the thread's row.  The helper warp adds the slots up.
    const bool warp_reduce = sw.groups < 32 && (sw.groups & (sw.groups - 1)) == 0;
    const int n_slots = warp_reduce ? kEwThreads / 32 : sw.rpi;
    float* s_part = reinterpret_cast<float*>(ring + (size_t)S * sw.stage_bytes);   // [n_slots][2c]
    float* s_coef = s_part + (size_t)n_slots * 2 * c;                                     // [4][c]: mean, gamma*invstd, dbeta/m, (dgamma/m)*invstd
    staged_init(full, empty, &abort_flag);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint8_t* mask = relu ? relu_mask : nullptr;
    const long long group_vecs = m * sw.groups;
    const int n_steps = n_groups + ahead;   // step t: R(t) if t < n_groups, then A(t - ahead) if t >= ahead
    const double inv_m = 1.0 / (double)m;
    int i = 0;                              // ring stage index, advanced identically by the producer and the consumers
    if (warp == kEwThreads / 32) {
        // ------------------------------------------------------------------------------------ producer
        if (lane == 0) {
            // the reduction pass asks L2 to keep the group's lines (the apply pass reads them again), the apply pass releases them
            const uint64_t keep = l2_policy_evict_last(), release = l2_policy_evict_first();
            bool ok = true;
            for (int t = 0; ok && t < n_steps; ++t) {
                if (t < n_groups)
                    ok = staged_produce_group(sw, ring, full, empty, da1, y, da2, mask, t * group_vecs, i, spin_limit, &abort_flag, status, keep, S);
                if (ok && t >= ahead)
                    ok = staged_produce_group(sw, ring, full, empty, da1, y, da2, mask, (t - ahead) * group_vecs, i, spin_limit, &abort_flag, status,
                                              release, S);
            }
        }
    } else if (warp == kEwThreads / 32 + 1) {
        // ------------------------------------------------------------------------------------ helper
        named_arrive(3);   // the partial-sum slots start out free
        for (int t = 0; t < n_steps; ++t) {
            // first the coefficients of the apply pass of this step (its group's arrivals were posted a whole reduction pass
            // ago), then this step's own sums: the consumers find the table ready when they get there
            if (t >= ahead) {
                const int ga = t - ahead;
                bool ok = *(volatile uint32_t*)&abort_flag == 0u;
                if (ok && lane == 0) {   // every block has added its sums of group ga
                    bool seen = false;
                    for (unsigned poll = 0; poll < spin_limit; ++poll) {
                        if (ld_acquire_gpu(arrivals + ga) >= gridDim.x) { seen = true; break; }
                        if (*(volatile uint32_t*)&abort_flag) break;
                        __nanosleep(100);
                    }
                    if (!seen) {
                        *(volatile uint32_t*)&abort_flag = 1u;
                        atomicOr(status, B2C_DEV_TIMEOUT);
                    }
                }
                __syncwarp();
                ok = *(volatile uint32_t*)&abort_flag == 0u;
                named_sync(5);   // the consumers have taken the previous group's coefficients
                if (ok) {
                    const double* sums = sums_all + (size_t)ga * 2 * c;
                    const float* mean = mean_all + (size_t)ga * c;
                    const float* invstd = invstd_all + (size_t)ga * c;
                    for (int ch = lane; ch < c; ch += 32) {
                        const double s1 = __ldcg(sums + ch), s2 = __ldcg(sums + c + ch);
                        const float mn = mean[ch], istd = invstd[ch];
                        const double dgam = (double)istd * (s2 - (double)mn * s1);
                        s_coef[ch] = mn;
                        s_coef[c + ch] = gamma[ch] * istd;                          // gamma*invstd
                        s_coef[2 * c + ch] = (float)(s1 * inv_m);                   // dbeta/m
                        s_coef[3 * c + ch] = (float)(dgam * inv_m * (double)istd);  // (dgamma/m)*invstd, multiplies (y-mean)
                        if (blockIdx.x == 0) {   // block 0 also emits the parameter gradients
                            const float db = (float)s1, dg = (float)dgam;
                            if (n_groups == 1) {
                                dbeta[ch] = acc ? dbeta[ch] + db : db;
                                dgamma[ch] = acc ? dgamma[ch] + dg : dg;
                            } else {   // several groups add into the same gradient (always accumulating)
                                atomicAdd(dbeta + ch, db);
                                atomicAdd(dgamma + ch, dg);
                            }
                        }
                    }
                }
                named_arrive(4);
            }
            if (t < n_groups) {
                named_sync(2);
                const bool ok = *(volatile uint32_t*)&abort_flag == 0u;
                if (ok) {
                    double* out = sums_all + (size_t)t * 2 * c;
                    for (int j = lane; j < 2 * c; j += 32) {
                        float tot = 0.f;
                        for (int sl = 0; sl < n_slots; ++sl) tot += s_part[(size_t)sl * 2 * c + j];
                        atomicAdd(out + j, (double)tot);
                    }
                }
                if (t + 1 < n_groups) named_arrive(3);   // the slots have been read (nobody waits for it after the last group)
                if (ok) {
                    __threadfence();   // this block's sums are visible device-wide before its arrival is
                    __syncwarp();
                    if (lane == 0) atomicAdd(arrivals + t, 1u);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------------------------ consumers
        const int g = threadIdx.x % sw.groups;
        const bool act = threadIdx.x < sw.active;
        const uint32_t tbytes = (uint32_t)sw.chunk_vecs * 16u;
        const bool two = sw.nt > 2;
        const bool ragged = (long long)sw.n_full * sw.chunk_rows < m && (sw.n_full % gridDim.x) == blockIdx.x;   // this block takes the group's tail
        named_arrive(5);   // the coefficient table starts out free
        bool ok = true;
        for (int t = 0; t < n_steps; ++t) {
            if (t < n_groups) {
                // ---------------------------------------------------------------- R(t): S1 = sum dz, S2 = sum dz*y
                float sb[8], sg[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) sb[j] = sg[j] = 0.f;
                if (ok) {
                    const long long base = t * group_vecs;
                    auto accumulate = [&](const uint4& v1, const uint4& vy, const uint4& v2, unsigned mk) {
                        float d[8], d2[8], fy[8];
                        unpack8(v1, d);
                        if (two) unpack8(v2, d2);
                        unpack8(vy, fy);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float dz = d[j];
                            if (two) dz += d2[j];
                            if (!((mk >> j) & 1u)) dz = 0.f;
                            sb[j] += dz;
                            sg[j] = fmaf(dz, fy[j], sg[j]);
                        }
                    };
                    for (long long k = blockIdx.x; k < sw.n_full; k += gridDim.x, ++i) {
                        ok = staged_wait(full, i, lane, spin_limit, &abort_flag, status, S);
                        if (!ok) break;
                        if (act) {
                            const uint8_t* st = ring + (size_t)(i % S) * sw.stage_bytes;
#pragma unroll 2
                            for (int u = 0; u < vecs; ++u) {
                                const int v = u * sw.active + threadIdx.x;
                                const uint4 v1 = reinterpret_cast<const uint4*>(st)[v];
                                const uint4 vy = reinterpret_cast<const uint4*>(st + tbytes)[v];
                                uint4 v2 = make_uint4(0u, 0u, 0u, 0u);
                                if (two) v2 = reinterpret_cast<const uint4*>(st + 2 * tbytes)[v];
                                const unsigned mk = mask != nullptr ? (unsigned)st[sw.nt * tbytes + v] : 0xffu;
                                accumulate(v1, vy, v2, mk);
                            }
                        }
                        staged_release(empty, i, lane, S);
                    }
                    if (ok && act && ragged) {
                        for (long long r = sw.n_full * sw.chunk_rows + threadIdx.x / sw.groups; r < m; r += sw.rpi) {
                            const long long vi = base + r * sw.groups + g;
                            const uint4 v1 = ld16(da1, vi), vy = ld16(y, vi);
                            const uint4 v2 = two ? ld16(da2, vi) : make_uint4(0u, 0u, 0u, 0u);
                            const unsigned mk = mask != nullptr ? (unsigned)__ldg(mask + vi) : 0xffu;
                            accumulate(v1, vy, v2, mk);
                        }
                    }
                }
                if (warp_reduce) {   // every lane of the warp is active here (the group count divides the block); uniform branch
#pragma unroll
                    for (int off = 16; off >= 1; off >>= 1) {
                        if (off >= sw.groups) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                sb[j] += __shfl_xor_sync(0xffffffffu, sb[j], off);
                                sg[j] += __shfl_xor_sync(0xffffffffu, sg[j], off);
                            }
                        }
                    }
                }
                named_sync(3);   // the helper has read the previous group's partial sums
                if (act && (!warp_reduce || lane < sw.groups)) {
                    float* mine = s_part + (size_t)(warp_reduce ? warp : threadIdx.x / sw.groups) * 2 * c + g * 8;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        mine[j] = sb[j];
                        mine[c + j] = sg[j];
                    }
                }
                named_arrive(2);   // hand the partial sums to the helper and go on streaming
            }
            if (t >= ahead) {
                // ---------------------------------------------------------------- A(ga): dy (and dres) from the coefficients the helper has prepared
                const int ga = t - ahead;
                named_sync(4);
                if (*(volatile uint32_t*)&abort_flag) ok = false;
                float mu[8], k0[8], kb[8], kg[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int ch = act ? g * 8 + j : 0;
                    mu[j] = s_coef[ch];
                    k0[j] = s_coef[c + ch];
                    kb[j] = s_coef[2 * c + ch];
                    kg[j] = s_coef[3 * c + ch];
                }
                if (t + 1 < n_steps) named_arrive(5);   // the table may be rewritten (nobody waits for it after the last group)
                if (ok) {
                    const long long base = ga * group_vecs;
                    auto emit = [&](const uint4& v1, const uint4& vy, const uint4& v2, unsigned mk, long long vi) {
                        float d[8], d2[8], fy[8], o[8];
                        unpack8(v1, d);
                        if (two) unpack8(v2, d2);
                        unpack8(vy, fy);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float dz = d[j];
                            if (two) dz += d2[j];
                            if (!((mk >> j) & 1u)) dz = 0.f;
                            d[j] = dz;
                            o[j] = k0[j] * (dz - kb[j] - (fy[j] - mu[j]) * kg[j]);
                        }
                        __stcs(reinterpret_cast<uint4*>(dy) + vi, pack8(o));   // streaming stores: the outputs should not push the waiting group out of L2
                        if (dres != nullptr) __stcs(reinterpret_cast<uint4*>(dres) + vi, pack8(d));
                    };
                    for (long long k = blockIdx.x; k < sw.n_full; k += gridDim.x, ++i) {
                        ok = staged_wait(full, i, lane, spin_limit, &abort_flag, status, S);
                        if (!ok) break;
                        if (act) {
                            const uint8_t* st = ring + (size_t)(i % S) * sw.stage_bytes;
#pragma unroll 2
                            for (int u = 0; u < vecs; ++u) {
                                const int v = u * sw.active + threadIdx.x;
                                const uint4 v1 = reinterpret_cast<const uint4*>(st)[v];
                                const uint4 vy = reinterpret_cast<const uint4*>(st + tbytes)[v];
                                uint4 v2 = make_uint4(0u, 0u, 0u, 0u);
                                if (two) v2 = reinterpret_cast<const uint4*>(st + 2 * tbytes)[v];
                                const unsigned mk = mask != nullptr ? (unsigned)st[sw.nt * tbytes + v] : 0xffu;
                                emit(v1, vy, v2, mk, base + k * sw.chunk_vecs + v);
                            }
                        }
                        staged_release(empty, i, lane, S);
                    }
                    if (ok && act && ragged) {
                        for (long long r = sw.n_full * sw.chunk_rows + threadIdx.x / sw.groups; r < m; r += sw.rpi) {
                            const long long vi = base + r * sw.groups + g;
                            const uint4 v1 = ld16(da1, vi), vy = ld16(y, vi);
                            const uint4 v2 = two ? ld16(da2, vi) : make_uint4(0u, 0u, 0u, 0u);
                            const unsigned mk = mask != nullptr ? (unsigned)__ldg(mask + vi) : 0xffu;
                            emit(v1, vy, v2, mk, vi);
                        }
                    }
                }
            }
        }
    }
    __syncthreads();
    // After an aborted wait the copies already issued must land before the block may exit.
    if (abort_flag && warp == kEwThreads / 32 && lane == 0) staged_drain(i, full, S);   // the producer lane's i = stages it issued
    __syncthreads();
}

// ------------------------------------------------------------------------------ pooling, padding
__global__ void avgpool_fwd_kernel(const void* __restrict__ a, int n, int hw, int c, void* __restrict__ pooled)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const int groups = c >> 3;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)n * groups) return;
    const int g = (int)(idx % groups);
    const long long img = idx / groups;
    float s[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = 0.f;
    for (int j = 0; j < hw; ++j) {
        float f[8];
        unpack8(ld16(a, (img * hw + j) * groups + g), f);
#pragma unroll
        for (int i = 0; i < 8; ++i) s[i] += f[i];
    }
    const float inv = 1.f / (float)hw;
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] *= inv;
    reinterpret_cast<uint4*>(pooled)[idx] = pack8(s);
}

__global__ void avgpool_bwd_kernel(const void* __restrict__ dpooled, int n, int hw, int c, void* __restrict__ da)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const int groups = c >> 3;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)n * hw * groups) return;
    const int g = (int)(idx % groups);
    const long long img = idx / ((long long)groups * hw);
    float f[8];
    unpack8(ld16(dpooled, img * groups + g), f);
    const float inv = 1.f / (float)hw;
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] *= inv;
    reinterpret_cast<uint4*>(da)[idx] = pack8(f);
}

__global__ void pad_channels_kernel(const __nv_bfloat16* __restrict__ x, long long m, int c_in, int c_out, void* __restrict__ y)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const int groups = c_out >> 3;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= m * groups) return;
    const int g = (int)(idx % groups);
    const long long row = idx / groups;
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int ch = g * 8 + i;
        f[i] = ch < c_in ? __bfloat162float(x[row * c_in + ch]) : 0.f;
    }
    reinterpret_cast<uint4*>(y)[idx] = pack8(f);
}

// Patch matrix of a 3x3, stride 1, pad 1 convolution over a narrow image: y[pixel, (r*3+s)*c_in + ch] = x[n, h+r-1, w+s-1, ch]
// (zero outside the image), columns 9*c_in .. c_out-1 zero.  Turns the first convolution into a 1x1-shaped GEMM.
template <int C_IN>
__global__ void im2col3x3_kernel(const __nv_bfloat16* __restrict__ x, int n, int h, int w, int c_out, void* __restrict__ y)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    // one thread per pixel: 9*C_IN (<= 32) values gathered with static tap offsets, written as whole 16-byte vectors
    const long long pix = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (pix >= (long long)n * h * w) return;
    const int ww = (int)(pix % w);
    const int hh = (int)((pix / w) % h);
    const long long img = pix / ((long long)w * h);
    float f[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) f[i] = 0.f;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int ih = hh + r - 1;
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            const int iw = ww + q - 1;
            if (ih >= 0 && ih < h && iw >= 0 && iw < w) {
                const __nv_bfloat16* src = x + ((img * h + ih) * w + iw) * C_IN;
#pragma unroll
                for (int ch = 0; ch < C_IN; ++ch) f[(r * 3 + q) * C_IN + ch] = __bfloat162float(src[ch]);
            }
        }
    }
    uint4* dst = reinterpret_cast<uint4*>(y) + pix * (c_out >> 3);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = f[g * 8 + i];
        dst[g] = pack8(v);
    }
    for (int g = 4; g < (c_out >> 3); ++g) dst[g] = make_uint4(0u, 0u, 0u, 0u);
}

// ------------------------------------------------------------------------------ loss
// One warp per row.
__global__ void softmax_xent_kernel(const float* __restrict__ logits, int logits_pitch, const int32_t* __restrict__ labels, int n, int classes,
                                    float loss_scale, float grad_scale, float* loss, __nv_bfloat16* __restrict__ dlogits, int pitch,
                                    unsigned* status)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    const float* z = logits + (long long)row * logits_pitch;
    const int label = labels[row];
    const bool bad = label < 0 || label >= classes;
    float mx = -INFINITY;
    for (int j = lane; j < classes; j += 32) mx = fmaxf(mx, z[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float se = 0.f;
    for (int j = lane; j < classes; j += 32) se += expf(z[j] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    const float lse = mx + logf(se);
    if (lane == 0) {
        if (bad)
            atomicOr(status, B2C_DEV_BAD_LABEL);
        else
            atomicAdd(loss, loss_scale * (lse - z[label]));
    }
    __nv_bfloat16* d = dlogits + (long long)row * pitch;
    for (int j = lane; j < pitch; j += 32) {
        float gval = 0.f;
        if (j < classes && !bad) gval = (expf(z[j] - lse) - (j == label ? 1.f : 0.f)) * grad_scale;
        d[j] = __float2bfloat16_rn(gval);
    }
}

// db[ch] (+)= sum over rows of dz[row, ch]: a block per 32 channels x a slice of rows, warp-shuffle free (each thread
// owns a channel and a row lane, partial sums meet in shared memory), one atomic per channel and block.
__global__ void bias_grad_kernel(const __nv_bfloat16* __restrict__ dz, int m, int k, int pitch, float* db)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    __shared__ float part[8][33];
    const int ch = blockIdx.x * 32 + threadIdx.x;        // blockDim = (32, 8)
    float s = 0.f;
    if (ch < k)
        for (int r = blockIdx.y * 8 + threadIdx.y; r < m; r += gridDim.y * 8) s += __bfloat162float(dz[(long long)r * pitch + ch]);
    part[threadIdx.y][threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y == 0 && ch < k) {
        float t = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) t += part[j][threadIdx.x];
        atomicAdd(db + ch, t);
    }
}

// ------------------------------------------------------------------------------ update
__global__ void __launch_bounds__(kEwThreads) sgd_momentum_kernel(float4* __restrict__ w, float4* __restrict__ v, float4* __restrict__ gsum,
                                                                  long long count4, float inv_n, float lr, float mu, float wd,
                                                                  uint2* __restrict__ w_bf16, int zero_grad)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const long long step = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count4; i += step) {
        float4 wi = w[i], vi = v[i];
        const float4 gi = gsum[i];
        float* pw = reinterpret_cast<float*>(&wi);
        float* pv = reinterpret_cast<float*>(&vi);
        const float* pg = reinterpret_cast<const float*>(&gi);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float g = fmaf(wd, pw[j], pg[j] * inv_n);   // g = g_sum*inv_n + wd*w
            pv[j] = fmaf(mu, pv[j], g);                      // v = mu*v + g
            pw[j] = fmaf(-lr, pv[j], pw[j]);                 // w = w - lr*v
        }
        w[i] = wi;
        v[i] = vi;
        if (zero_grad) gsum[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (w_bf16 != nullptr) w_bf16[i] = make_uint2(pack_bf16x2(pw[0], pw[1]), pack_bf16x2(pw[2], pw[3]));
    }
}

struct PackSegs {
    b2c_weight_seg seg[128];
    int first_block[129];   // running total of (taps x tiles) per segment: block b belongs to the segment with first_block[s] <= b < first_block[s + 1]
    int n_segs;
};
// dst[c][rs-1-t][k] = src[k][t][c] per segment: for a fixed tap this is a k x c -> c x k transpose, done in 32 x 32
// tiles through shared memory so that both the reads (c contiguous) and the writes (k contiguous) are coalesced.
// One block per (segment, tap, tile of the (k, c) plane), numbered consecutively over all segments.
__global__ void weight_pack_dgrad_kernel(const __grid_constant__ PackSegs segs, const __nv_bfloat16* __restrict__ src,
                                         __nv_bfloat16* __restrict__ dst)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    __shared__ __nv_bfloat16 tile[32][33];
    int lo = 0, hi = segs.n_segs;   // binary search for the segment of this block
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int)blockIdx.x >= segs.first_block[mid]) lo = mid;
        else hi = mid;
    }
    const b2c_weight_seg sg = segs.seg[lo];
    const int local = (int)blockIdx.x - segs.first_block[lo];
    const int tiles_c = (sg.c + 31) / 32, tiles_k = (sg.k + 31) / 32;
    const int t = local / (tiles_c * tiles_k), tile_id = local - t * (tiles_c * tiles_k);
    if (t >= sg.rs) return;
    const int k0 = (tile_id / tiles_c) * 32, c0 = (tile_id % tiles_c) * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {          // blockDim = (32, 8)
        const int k = k0 + j, c = c0 + threadIdx.x;
        tile[j][threadIdx.x] = (k < sg.k && c < sg.c) ? src[sg.offset + ((long long)k * sg.rs + t) * sg.c + c] : __float2bfloat16(0.f);
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int c = c0 + j, k = k0 + threadIdx.x;
        if (c < sg.c && k < sg.k) dst[sg.offset + ((long long)c * sg.rs + (sg.rs - 1 - t)) * sg.k + k] = tile[threadIdx.x][j];
    }
}

// ------------------------------------------------------------------------------ running statistics
static constexpr int kRunEntries = 64;
struct BnRunTable {
    BnRunEntry e[kRunEntries];
};
__global__ void bn_running_update_kernel(const __grid_constant__ BnRunTable tab, const char* __restrict__ ws, float* __restrict__ run, int G, float momentum)
{
    pdl_wait();   // first global access comes after the previous kernel of the stream
    pdl_launch_dependents();
    const BnRunEntry& en = tab.e[blockIdx.x];
    const double* stats = reinterpret_cast<const double*>(ws + en.stats_off);
    const double inv_m = 1.0 / (double)en.m;
    const float unbias = en.m > 1.f ? (float)((double)en.m / ((double)en.m - 1.0)) : 1.f;
    for (int ch = threadIdx.x; ch < en.c; ch += blockDim.x) {
        float rm = run[en.run_off + ch], rv = run[en.run_off + en.c + ch];
        for (int g = 0; g < G; ++g) {
            float mean, invstd, var;
            bn_moments(stats + (size_t)g * 2 * en.c, en.c, ch, inv_m, 0.f, mean, invstd, var);
            rm = (1.f - momentum) * rm + momentum * mean;
            rv = (1.f - momentum) * rv + momentum * var * unbias;
        }
        run[en.run_off + ch] = rm;
        run[en.run_off + en.c + ch] = rv;
    }
}

// ------------------------------------------------------------------------------ launchers
// Blocks per statistics group: one wave of two resident blocks per SM across all groups.
static int ew_grid(b2c_ctx* ctx, int n_groups, long long m, int rows_per_iter)
{
    long long blocks = (m + rows_per_iter - 1) / rows_per_iter;
    long long cap = ((long long)ctx->sm_count * 2 + n_groups - 1) / n_groups;
    if (cap < 1) cap = 1;
    return (int)(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
}

b2c_status launch_bn_fwd(b2c_ctx* ctx, int G, long long m, int c, const void* y, double* stats, int stats_ready, const float* gamma,
                         const float* beta, const void* residual, int relu, float eps, void* a, float* save_mean, float* save_invstd,
                         float* run_mean, float* run_var, float momentum, void* relu_mask, cudaStream_t stream)
{
    const int rows_per_iter = kEwThreads / (c / 8);
    dim3 grid((unsigned)ew_grid(ctx, G, m, rows_per_iter), (unsigned)G);
    if (stats_ready != 1) {
        if (stats_ready == 0) B2C_CUDA(cudaMemsetAsync(stats, 0, sizeof(double) * 2 * c * G, stream));
        B2C_CUDA(b2c_launch(ctx, bn_stats_kernel, dim3(grid), dim3(kEwThreads), sizeof(float) * 2 * c, stream, 1u, y, m, c, stats));
    }
    uint8_t* mask_out = relu ? reinterpret_cast<uint8_t*>(relu_mask) : nullptr;
    if (residual != nullptr)
        B2C_CUDA(b2c_launch(ctx, bn_apply_kernel<4, true>, dim3(grid), dim3(kEwThreads), 0, stream, 1u, y, m, c, stats, gamma, beta, residual, relu, eps, a,
                            save_mean, save_invstd, run_mean, run_var, momentum, mask_out));
    else
        B2C_CUDA(b2c_launch(ctx, bn_apply_kernel<8, false>, dim3(grid), dim3(kEwThreads), 0, stream, 1u, y, m, c, stats, gamma, beta, residual, relu, eps, a,
                            save_mean, save_invstd, run_mean, run_var, momentum, mask_out));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status launch_bn_running_update(b2c_ctx* ctx, const BnRunEntry* entries, int n_entries, const char* ws, float* run, int G, float momentum,
                                    cudaStream_t stream)
{
    for (int first = 0; first < n_entries; first += kRunEntries) {
        BnRunTable tab;
        const int n = n_entries - first < kRunEntries ? n_entries - first : kRunEntries;
        for (int i = 0; i < n; ++i) tab.e[i] = entries[first + i];
        B2C_CUDA(b2c_launch(ctx, bn_running_update_kernel, dim3((unsigned)n), dim3(128), 0, stream, 1u, tab, ws, run, G, momentum));
    }
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status launch_bn_bwd(b2c_ctx* ctx, int G, long long m, int c, const void* da1, const void* da2, const void* y, const void* a,
                         const float* gamma, const float* save_mean, const float* save_invstd, int relu, void* dy, void* dres, float* dgamma,
                         float* dbeta, int acc, double* sums, bool sums_zeroed, const void* relu_mask, unsigned* arrivals, cudaStream_t stream)
{
    const int rows_per_iter = kEwThreads / (c / 8);
    dim3 grid((unsigned)ew_grid(ctx, G, m, rows_per_iter), (unsigned)G);
    const uint8_t* mask = relu ? reinterpret_cast<const uint8_t*>(relu_mask) : nullptr;
    if (!sums_zeroed) {
        B2C_CUDA(cudaMemsetAsync(sums, 0, sizeof(double) * 2 * c * G, stream));
        if (arrivals != nullptr) B2C_CUDA(cudaMemsetAsync(arrivals, 0, sizeof(unsigned) * G, stream));
    }
    // Both passes in one cooperative launch, group by group (the apply pass of a group re-reads its tensors from L2).
    if (arrivals != nullptr) {
        // Stage size (vectors per thread and tensor) and ring depth: as many stages as fit, four at most.
        const int groups = c / 8, active = rows_per_iter * groups;
        const int nt = da2 != nullptr ? 3 : 2;
        const bool warp_reduce = groups < 32 && (groups & (groups - 1)) == 0;
        const int n_slots = warp_reduce ? kEwThreads / 32 : rows_per_iter;
        const size_t extra = sizeof(float) * ((size_t)n_slots * 2 * c + 4 * (size_t)c) + 128;
        int vecs = 2, ring_stages = 0;   // (stages of four vectors leave a ring of two or three and measured slower: 159 against 136 us on the 64-channel layers)
        size_t stage = 0;
        for (;;) {
            const int cv = vecs * active;
            stage = (size_t)nt * cv * 16 + (relu ? ((cv + 127) & ~127) : 0);
            ring_stages = (int)((110 * 1024 - extra) / stage);
            if (ring_stages > kStStages) ring_stages = kStStages;
            if ((ring_stages >= 2 && m / (vecs * rows_per_iter) >= 4ll * ctx->sm_count) || vecs == 2) break;
            vecs = 2;
        }
        const int chunk_vecs = vecs * active;
        const size_t smem = (size_t)(ring_stages > 0 ? ring_stages : 1) * stage + extra;
        const long long n_full = m / (vecs * rows_per_iter);
        const bool eligible = ring_stages >= 2 && (!relu || mask != nullptr) && chunk_vecs % 16 == 0 && (m * groups) % 16 == 0 && n_full >= 1 &&
                              reinterpret_cast<uintptr_t>(mask) % 16 == 0 && smem <= 110 * 1024;
        if (eligible) {
            if (!(ctx->smem_optin_done & B2C_OPTIN_BN_GROUPED)) {
                B2C_CUDA(cudaFuncSetAttribute(bn_bwd_grouped_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
                ctx->smem_optin_done |= B2C_OPTIN_BN_GROUPED;
            }
            int per_sm = 0;
            B2C_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bn_bwd_grouped_kernel, kGrThreads, smem));
            if (per_sm > 2) per_sm = 2;
            if (per_sm >= 1) {
                long long blocks = (long long)per_sm * ctx->sm_count;   // all blocks co-resident: the groups' barriers need every block running
                if (blocks > n_full) blocks = n_full;
                // Groups whose reduction pass runs ahead of a group's apply pass: as many as keep the inputs of the waiting
                // groups (da, y, second gradient, mask) within a part of the L2, at least one.
                const double group_bytes = (double)m * c * (2.0 * nt + 0.125);
                int ahead = (int)(40e6 / group_bytes);
                if (ahead < 1) ahead = 1;
                if (ahead > G) ahead = G;
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3((unsigned)blocks);
                cfg.blockDim = dim3(kGrThreads);
                cfg.dynamicSmemBytes = smem;
                cfg.stream = stream;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeCooperative;
                attr[0].val.cooperative = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 1;
                B2C_CUDA(cudaLaunchKernelEx(&cfg, bn_bwd_grouped_kernel, da1, da2, y, m, c, G, ahead, gamma, save_mean, save_invstd, relu, sums, arrivals, dy,
                                            dres, dgamma, dbeta, acc, mask, ctx->spin_limit, ctx->d_status, vecs, ring_stages));
                B2C_CUDA(cudaGetLastError());
                return B2C_OK;
            }
        }
    }
    // The staged kernels need the ReLU mask (not the activation), chunk offsets that keep the mask copies 16-byte
    // aligned, and at least one full chunk per block to be worth their set-up.
    const int groups = c / 8, active = rows_per_iter * groups, chunk_vecs = 2 * active;
    const bool staged = (!relu || mask != nullptr) && chunk_vecs % 16 == 0 && (m * groups) % 16 == 0 && m >= 2ll * rows_per_iter * grid.x &&
                        reinterpret_cast<uintptr_t>(mask) % 16 == 0;
    if (staged) {
        const int nt = da2 != nullptr ? 3 : 2;
        const size_t stage = (size_t)nt * chunk_vecs * 16 + (relu ? ((chunk_vecs + 127) & ~127) : 0);
        const size_t smem = kStStages * stage + sizeof(float) * 2 * c + 128;
        if (smem <= 110 * 1024) {
            if (!(ctx->smem_optin_done & B2C_OPTIN_BN_BWD)) {
                B2C_CUDA(cudaFuncSetAttribute(bn_bwd_reduce_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
                B2C_CUDA(cudaFuncSetAttribute(bn_bwd_apply_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
                ctx->smem_optin_done |= B2C_OPTIN_BN_BWD;
            }
            B2C_CUDA(b2c_launch(ctx, bn_bwd_reduce_staged_kernel, dim3(grid), dim3(kStThreads), smem, stream, 1u, da1, da2, y, m, c, relu, sums, mask, ctx->spin_limit, ctx->d_status));
            B2C_CUDA(b2c_launch(ctx, bn_bwd_apply_staged_kernel, dim3(grid), dim3(kStThreads), smem, stream, 1u, da1, da2, y, m, c, gamma, save_mean, save_invstd, relu, sums, dy, dres,
                                                                            dgamma, dbeta, acc, mask, ctx->spin_limit, ctx->d_status));
            B2C_CUDA(cudaGetLastError());
            return B2C_OK;
        }
    }
    B2C_CUDA(b2c_launch(ctx, bn_bwd_reduce_kernel, dim3(grid), dim3(kEwThreads), sizeof(float) * 2 * c, stream, 1u, da1, da2, y, a, m, c, relu, sums, mask));
    B2C_CUDA(b2c_launch(ctx, bn_bwd_apply_kernel, dim3(grid), dim3(kEwThreads), 0, stream, 1u, da1, da2, y, a, m, c, gamma, save_mean, save_invstd, relu, sums, dy, dres, dgamma, dbeta,
                                                         acc, mask));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

}  // namespace b2c

using namespace b2c;

extern "C" {

b2c_status b2c_bn_relu_fwd(b2c_ctx* ctx, int n, int h, int w, int c, const void* y, double* ch_stats, int stats_ready, const float* gamma,
                           const float* beta, const void* residual, int relu, float eps, void* a, float* save_mean, float* save_invstd,
                           float* run_mean, float* run_var, float momentum, void* relu_mask, void* stream_)
{
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!ctx || !y || !ch_stats || !gamma || !beta || !a || !save_mean || !save_invstd) return B2C_ERR_INVALID_ARG;
    if (n < 1 || h < 1 || w < 1 || c < 8 || c % 8 || c > 2048) return B2C_ERR_UNSUPPORTED_SHAPE;
    if ((run_mean == nullptr) != (run_var == nullptr)) return B2C_ERR_INVALID_ARG;
    if (!b2c_aligned16(y) || !b2c_aligned16(a) || (residual && !b2c_aligned16(residual)) || (reinterpret_cast<uintptr_t>(ch_stats) & 7u))
        return B2C_ERR_MISALIGNED;
    return launch_bn_fwd(ctx, 1, (long long)n * h * w, c, y, ch_stats, stats_ready != 0, gamma, beta, residual, relu, eps, a, save_mean, save_invstd,
                         run_mean, run_var, momentum, relu_mask, stream);
}

size_t b2c_bn_relu_bwd_workspace_bytes(int c) { return c > 0 ? sizeof(double) * 2 * (size_t)c : 0; }

b2c_status b2c_bn_relu_bwd(b2c_ctx* ctx, int n, int h, int w, int c, const void* da1, const void* da2, const void* y, const void* a,
                           const float* gamma, const float* save_mean, const float* save_invstd, int relu, void* dy, void* dres, float* dgamma,
                           float* dbeta, int acc, const void* relu_mask, void* ws, size_t ws_bytes, void* stream_)
{
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!ctx || !da1 || !y || !gamma || !save_mean || !save_invstd || !dy || !dgamma || !dbeta || !ws) return B2C_ERR_INVALID_ARG;
    if (relu && !a && !relu_mask) return B2C_ERR_INVALID_ARG;
    if (n < 1 || h < 1 || w < 1 || c < 8 || c % 8 || c > 2048) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (ws_bytes < b2c_bn_relu_bwd_workspace_bytes(c)) return B2C_ERR_WORKSPACE_TOO_SMALL;
    if (!b2c_aligned16(da1) || (da2 && !b2c_aligned16(da2)) || !b2c_aligned16(y) || (a && !b2c_aligned16(a)) || !b2c_aligned16(dy) ||
        (dres && !b2c_aligned16(dres)) || (reinterpret_cast<uintptr_t>(ws) & 7u))
        return B2C_ERR_MISALIGNED;
    return launch_bn_bwd(ctx, 1, (long long)n * h * w, c, da1, da2, y, a, gamma, save_mean, save_invstd, relu, dy, dres, dgamma, dbeta, acc,
                         reinterpret_cast<double*>(ws), false, relu_mask, nullptr, stream);
}

size_t b2c_bn_relu_bwd_groups_workspace_bytes(int c, int groups)
{
    if (c <= 0 || groups <= 0) return 0;
    return sizeof(double) * 2 * (size_t)c * groups + ((sizeof(unsigned) * (size_t)groups + 7) & ~size_t(7));   // sums, then arrival counters
}

b2c_status b2c_bn_relu_bwd_groups(b2c_ctx* ctx, int groups, long long rows_per_group, int c, const void* da1, const void* da2, const void* y,
                                  const float* gamma, const float* save_mean, const float* save_invstd, int relu, void* dy, void* dres,
                                  float* dgamma, float* dbeta, int acc, const void* relu_mask, void* ws, size_t ws_bytes, void* stream_)
{
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!ctx || !da1 || !y || !gamma || !save_mean || !save_invstd || !dy || !dgamma || !dbeta || !ws) return B2C_ERR_INVALID_ARG;
    if (relu && !relu_mask) return B2C_ERR_INVALID_ARG;
    if (groups < 1 || groups > 4096 || rows_per_group < 1 || c < 8 || c % 8 || c > 2048) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (ws_bytes < b2c_bn_relu_bwd_groups_workspace_bytes(c, groups)) return B2C_ERR_WORKSPACE_TOO_SMALL;
    if (!b2c_aligned16(da1) || (da2 && !b2c_aligned16(da2)) || !b2c_aligned16(y) || !b2c_aligned16(dy) || (dres && !b2c_aligned16(dres)) ||
        (relu_mask && !b2c_aligned16(relu_mask)) || (reinterpret_cast<uintptr_t>(ws) & 7u))
        return B2C_ERR_MISALIGNED;
    if ((rows_per_group * (c / 8)) % 16) return B2C_ERR_UNSUPPORTED_SHAPE;   // a group's slice of the bit mask must start on a 16-byte boundary
    double* sums = reinterpret_cast<double*>(ws);
    unsigned* arrivals = reinterpret_cast<unsigned*>(sums + (size_t)2 * c * groups);
    B2C_CUDA(cudaMemsetAsync(ws, 0, b2c_bn_relu_bwd_groups_workspace_bytes(c, groups), stream));
    if (!acc && groups > 1) {   // several groups always add into the gradients: start them at zero
        B2C_CUDA(cudaMemsetAsync(dgamma, 0, sizeof(float) * c, stream));
        B2C_CUDA(cudaMemsetAsync(dbeta, 0, sizeof(float) * c, stream));
    }
    return launch_bn_bwd(ctx, groups, rows_per_group, c, da1, da2, y, nullptr, gamma, save_mean, save_invstd, relu, dy, dres, dgamma, dbeta,
                         groups > 1 ? 1 : acc, sums, true, relu_mask, arrivals, stream);
}

b2c_status b2c_avgpool_fwd(b2c_ctx* ctx, int n, int hw, int c, const void* a, void* pooled, void* stream_)
{
    if (!ctx || !a || !pooled) return B2C_ERR_INVALID_ARG;
    if (n < 1 || hw < 1 || c < 8 || c % 8) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(a) || !b2c_aligned16(pooled)) return B2C_ERR_MISALIGNED;
    const long long total = (long long)n * (c / 8);
    B2C_CUDA(b2c_launch(ctx, avgpool_fwd_kernel, dim3((unsigned)((total + 127) / 128)), dim3(128), 0, (cudaStream_t)stream_, 1u, a, n, hw, c, pooled));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status b2c_avgpool_bwd(b2c_ctx* ctx, int n, int hw, int c, const void* dpooled, void* da, void* stream_)
{
    if (!ctx || !dpooled || !da) return B2C_ERR_INVALID_ARG;
    if (n < 1 || hw < 1 || c < 8 || c % 8) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(dpooled) || !b2c_aligned16(da)) return B2C_ERR_MISALIGNED;
    const long long total = (long long)n * hw * (c / 8);
    B2C_CUDA(b2c_launch(ctx, avgpool_bwd_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, (cudaStream_t)stream_, 1u, dpooled, n, hw, c, da));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status b2c_pad_channels(b2c_ctx* ctx, long m, int c_in, int c_out, const void* x, void* y, void* stream_)
{
    if (!ctx || !x || !y) return B2C_ERR_INVALID_ARG;
    if (m < 1 || c_in < 1 || c_out < c_in || c_out % 8) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(y) || (reinterpret_cast<uintptr_t>(x) & 1u)) return B2C_ERR_MISALIGNED;
    const long long total = (long long)m * (c_out / 8);
    B2C_CUDA(b2c_launch(ctx, pad_channels_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, (cudaStream_t)stream_, 1u, reinterpret_cast<const __nv_bfloat16*>(x), m, c_in,
                                                                                            c_out, y));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status b2c_im2col_3x3(b2c_ctx* ctx, int n, int h, int w, int c_in, int c_out, const void* x, void* y, void* stream_)
{
    if (!ctx || !x || !y) return B2C_ERR_INVALID_ARG;
    if (n < 1 || h < 1 || w < 1 || c_in < 1 || c_out < 32 || c_out % 8) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(y) || (reinterpret_cast<uintptr_t>(x) & 1u)) return B2C_ERR_MISALIGNED;
    if (c_in > 3) return B2C_ERR_UNSUPPORTED_SHAPE;
    const long long total = (long long)n * h * w;
    const unsigned blocks = (unsigned)((total + 127) / 128);
    const __nv_bfloat16* xs = reinterpret_cast<const __nv_bfloat16*>(x);
    if (c_in == 3) B2C_CUDA(b2c_launch(ctx, im2col3x3_kernel<3>, dim3(blocks), dim3(128), 0, (cudaStream_t)stream_, 1u, xs, n, h, w, c_out, y));
    else if (c_in == 2) B2C_CUDA(b2c_launch(ctx, im2col3x3_kernel<2>, dim3(blocks), dim3(128), 0, (cudaStream_t)stream_, 1u, xs, n, h, w, c_out, y));
    else B2C_CUDA(b2c_launch(ctx, im2col3x3_kernel<1>, dim3(blocks), dim3(128), 0, (cudaStream_t)stream_, 1u, xs, n, h, w, c_out, y));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status b2c_softmax_xent_fwd_bwd(b2c_ctx* ctx, int n, int classes, const float* logits, int logits_pitch, const int32_t* labels,
                                    float loss_scale, float grad_scale, float* loss, void* dlogits, int pitch, void* stream_)
{
    if (!ctx || !logits || !labels || !loss || !dlogits) return B2C_ERR_INVALID_ARG;
    if (n < 1 || classes < 1 || logits_pitch < classes || pitch < classes || pitch % 8) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(dlogits)) return B2C_ERR_MISALIGNED;
    const int warps = 4;
    B2C_CUDA(b2c_launch(ctx, softmax_xent_kernel, dim3((n + warps - 1) / warps), dim3(warps * 32), 0, (cudaStream_t)stream_, 1u, logits, logits_pitch, labels, n, classes, loss_scale,
                                                                                          grad_scale, loss, reinterpret_cast<__nv_bfloat16*>(dlogits),
                                                                                          pitch, ctx->d_status));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status b2c_bias_grad(b2c_ctx* ctx, int m, int k, int pitch, const void* dz, float* db, int accumulate, void* stream_)
{
    if (!ctx || !dz || !db) return B2C_ERR_INVALID_ARG;
    if (m < 1 || k < 1 || pitch < k) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!accumulate) B2C_CUDA(cudaMemsetAsync(db, 0, sizeof(float) * (size_t)k, (cudaStream_t)stream_));
    int row_blocks = (m + 63) / 64;
    if (row_blocks > 64) row_blocks = 64;
    B2C_CUDA(b2c_launch(ctx, bias_grad_kernel, dim3(dim3((unsigned)((k + 31) / 32), (unsigned)row_blocks)), dim3(dim3(32, 8)), 0, (cudaStream_t)stream_, 1u, 
        reinterpret_cast<const __nv_bfloat16*>(dz), m, k, pitch, db));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status b2c_grad_accum_sgd_momentum(b2c_ctx* ctx, size_t count, float* w, float* v, float* g_accum, float inv_n_micro, float lr,
                                       float momentum, float wd, void* w_bf16, int zero_grad, void* stream_)
{
    if (!ctx || !w || !v || !g_accum) return B2C_ERR_INVALID_ARG;
    if (count == 0 || count % 4) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(w) || !b2c_aligned16(v) || !b2c_aligned16(g_accum) || (w_bf16 && (reinterpret_cast<uintptr_t>(w_bf16) & 7u)))
        return B2C_ERR_MISALIGNED;
    const long long count4 = (long long)(count / 4);
    long long blocks = (count4 + kEwThreads - 1) / kEwThreads;
    const long long cap = (long long)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    B2C_CUDA(b2c_launch(ctx, sgd_momentum_kernel, dim3((unsigned)blocks), dim3(kEwThreads), 0, (cudaStream_t)stream_, 1u, reinterpret_cast<float4*>(w), reinterpret_cast<float4*>(v),
                                                                                   reinterpret_cast<float4*>(g_accum), count4, inv_n_micro, lr,
                                                                                   momentum, wd, reinterpret_cast<uint2*>(w_bf16), zero_grad));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

b2c_status b2c_weight_pack_dgrad(b2c_ctx* ctx, const b2c_weight_seg* segs, int n_segs, const void* src_bf16, void* dst_bf16, void* stream_)
{
    if (!ctx || !segs || !src_bf16 || !dst_bf16) return B2C_ERR_INVALID_ARG;
    if (n_segs < 1 || n_segs > 128) return B2C_ERR_UNSUPPORTED_SHAPE;
    PackSegs ps;
    long long blocks = 0;
    for (int i = 0; i < n_segs; ++i) {
        if (segs[i].k < 1 || segs[i].rs < 1 || segs[i].c < 1 || segs[i].offset < 0) return B2C_ERR_INVALID_ARG;
        ps.seg[i] = segs[i];
        ps.first_block[i] = (int)blocks;
        blocks += (long long)segs[i].rs * ((segs[i].k + 31) / 32) * ((segs[i].c + 31) / 32);
        if (blocks > 0x7fffffffll) return B2C_ERR_UNSUPPORTED_SHAPE;
    }
    ps.first_block[n_segs] = (int)blocks;
    ps.n_segs = n_segs;
    dim3 grid((unsigned)blocks);
    B2C_CUDA(b2c_launch(ctx, weight_pack_dgrad_kernel, dim3(grid), dim3(dim3(32, 8)), 0, (cudaStream_t)stream_, 1u, ps, reinterpret_cast<const __nv_bfloat16*>(src_bf16),
                                                                              reinterpret_cast<__nv_bfloat16*>(dst_bf16)));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

// ------------------------------------------------------------------------------ allocation-free variant
// Scratch of b2c_bn_relu_bwd_static: the two fp64 accumulators per channel, for up to
// B2C_BN_BWD_STATIC_MAX_C channels.  It is part of the library image, so every GPU that loads the
// library holds these 32 KB until the process exits.
static __device__ __align__(256) double g_bn_bwd_static_scratch[2 * B2C_BN_BWD_STATIC_MAX_C];

// Device address of the array above, looked up once per device.  In host code the symbol's name
// is only a handle: the kernels must be given the address cudaGetSymbolAddress reports.
static double* g_bn_bwd_static_ptr[64] = {nullptr};

b2c_status b2c_bn_relu_bwd_static(b2c_ctx* ctx, int n, int h, int w, int c, const void* da1, const void* da2, const void* y, const void* a,
                                  const float* gamma, const float* save_mean, const float* save_invstd, int relu, void* dy, void* dres,
                                  float* dgamma, float* dbeta, int acc, void* stream_)
{
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!ctx || !da1 || !y || !gamma || !save_mean || !save_invstd || !dy || !dgamma || !dbeta) return B2C_ERR_INVALID_ARG;
    if (relu && !a) return B2C_ERR_INVALID_ARG;
    if (n < 1 || h < 1 || w < 1 || c < 8 || c % 8) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (c > B2C_BN_BWD_STATIC_MAX_C) return B2C_ERR_WORKSPACE_TOO_SMALL;   // the built-in scratch holds at most that many channels
    if (!b2c_aligned16(da1) || (da2 && !b2c_aligned16(da2)) || !b2c_aligned16(y) || (a && !b2c_aligned16(a)) || !b2c_aligned16(dy) ||
        (dres && !b2c_aligned16(dres)))
        return B2C_ERR_MISALIGNED;
    int current = -1;
    B2C_CUDA(cudaGetDevice(&current));
    if (current != ctx->device || current < 0 || current >= 64) return B2C_ERR_INVALID_ARG;   // the context's device must be current
    if (g_bn_bwd_static_ptr[current] == nullptr) {
        double* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_bn_bwd_static_scratch) != cudaSuccess || ptr == nullptr) return B2C_ERR_CUDA;
        g_bn_bwd_static_ptr[current] = ptr;
    }
    // the array keeps the previous call's sums: the launcher clears the part this call uses
    return launch_bn_bwd(ctx, 1, (long long)n * h * w, c, da1, da2, y, a, gamma, save_mean, save_invstd, relu, dy, dres, dgamma, dbeta, acc,
                         g_bn_bwd_static_ptr[current], false, nullptr, nullptr, stream);
}

}  // extern "C"
