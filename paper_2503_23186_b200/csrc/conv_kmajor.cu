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
//
// The kernel is persistent: one CTA per SM walks a list of (pixel tile, channel tile) units.
//   * Two or four accumulators in TMEM (four where 4 x n_tile columns fit): while the epilogue warps drain unit i
//     (bias, bf16 rounding, BatchNorm sums, stores), the MMA threads already accumulate the next units into the
//     others, and the TMA producers run ahead through the shared-memory ring across unit boundaries.
//   * Vertical tap reuse (3x3, stride 1, tile inside one image): a stage holds the tile plus one
//     halo row above and below for one horizontal shift; the three vertical taps read it at row
//     offsets of one image row (a multiple of the swizzle period), so the input is fetched three
//     times instead of nine.
//   * Small filter banks stay resident in shared memory for the whole launch.
// Warp roles: warp 0 = first TMA producer (one lane), warp 1 = TMEM owner + first MMA issuer (one lane),
// warps 2..9 = epilogue (two per TMEM lane quarter, splitting the columns), warp 10 = second MMA issuer (one lane;
// the two issuers take alternate units), warp 11 = second TMA producer (one lane; the two producers take alternate
// stages).  Every mbarrier wait is bounded.
#include "common.h"
#include "ptx.cuh"

namespace b2c {

struct alignas(64) ConvKParams {
    CUtensorMap tmA[4];
    CUtensorMap tmB;
    TapList taps[4];
    int bw, bh, bn;                  // pixel box of an output tile; bw*bh*bn == 128
    int tiles_w, tiles_h, tiles_n;   // tiles of the output grid
    int tw_shift, th_shift, nk_shift, grp_shift, cb_shift;   // log2 of tiles_w, tiles_h, n_ktiles, stats_group_images, c_blocks (-1: not a power of two)
    int n_ktiles, n_tile;            // output-channel tiles, UMMA N
    int n_par;                       // output parities (stride-2 data gradient: 4)
    int total_units;
    int kb, c_blocks;                // channels per k-block, k-blocks per tap
    int stages, swz;
    int tmem_cols, acc_cols;         // allocation, columns per accumulator
    int acc_bufs, acc_shift;         // accumulators in TMEM (2 or 4) and log2 of that: unit j uses accumulator j % acc_bufs
    int vreuse;                      // a stage serves the three vertical taps of one horizontal shift
    int fh;                          // full halo: a stage holds the tile with a one-pixel frame and serves all nine taps
    int hm;                          // merged horizontal taps: one N = 3 x n_tile MMA per vertical tap and k-step, the three column blocks are
                                     // shifted by one pixel and added in the epilogue (tiles of whole image rows, 64 output channels)
    int mma_n;                       // UMMA N (n_tile, or 3 x n_tile with merged horizontal taps)
    int nb;                          // B tiles per stage (1, or 3 with vreuse)
    int b_merged;                    // the three B tiles of a stage come with one load (box of three filter rows)
    int r_filter;                    // filter height = width
    int a_bytes, b_bytes;            // shared-memory footprint of the A tile / one B tile (multiples of 1 KB)
    int tx_a, tx_b;                  // bytes one A / B load delivers
    int a_step;                      // byte offset of one image row inside the A tile (vreuse)
    int issuers;                     // MMA-issuing threads at work (1 or 2)
    int gsub;                        // k-blocks that share a ring slot, one barrier wait and one commit (short k-blocks: the waits would bound the issuing threads)
    int issue_split;                 // the two issuing threads share every unit: alternate stages into one accumulator (tiles wider than 128 channels)
    int pair;                        // CTA pairs (cta_group::2): M = 256 per MMA, each CTA holds half of every B tile
    int resident;                    // filter bank of this CTA's channel tile stays in shared memory
    int resident_bytes;
    int n_valid, oc_valid;           // images / output channels that exist
    long long os_n, os_h, os_w;      // output element strides along the tile grid
    long long off[4];                // output element offset per parity
    void* out;
    int out_is_f32;
    int out_v8;                      // the output base is 32-byte aligned: bf16 chunks go out as one 256-bit store per lane
    const float* bias;
    double* stats;
    int stats_group_images;          // images per BatchNorm statistics group (0: one group)
    unsigned* status;
    unsigned spin_limit;
    unsigned long long* stall;       // optional [5]: cycles waited by producer / MMA (ring) / MMA (accumulator) / epilogue, CTA lifetime
};

static constexpr int kMaxStages = 8;
static constexpr int kMaxAccBufs = 4;
static constexpr int kEpiWarps = 8;
static constexpr int kIssuers = 2;       // MMA-issuing threads: warp 1 and the warps after the epilogue warps
static constexpr int kProducers = 2;     // TMA-issuing threads: warp 0 and the warp after the issuer warps; they take alternate stages
static constexpr int kThreads = 64 + 32 * kEpiWarps + 32 * (kIssuers - 1) + 32 * (kProducers - 1);
static constexpr int kProducerWarp1 = 2 + kEpiWarps + (kIssuers - 1);   // warp index of the second producer
static constexpr uint32_t kDrainPolls = 1u << 22;

struct UnitCoord {
    int par, ktile, ow0, oh0, n0;
};
// tiles_w and tiles_h are powers of two (the grid sides are); the channel-tile count and the stats group size usually are
__device__ __forceinline__ UnitCoord decode_unit(const ConvKParams& p, int u)
{
    UnitCoord c;
    if (p.nk_shift >= 0) {
        c.ktile = u & (p.n_ktiles - 1);
        u >>= p.nk_shift;
    } else {
        c.ktile = u % p.n_ktiles;
        u /= p.n_ktiles;
    }
    c.ow0 = (u & (p.tiles_w - 1)) * p.bw;
    u >>= p.tw_shift;
    c.oh0 = (u & (p.tiles_h - 1)) * p.bh;
    u >>= p.th_shift;
    if (p.n_par > 1) {
        c.n0 = (u % p.tiles_n) * p.bn;
        c.par = u / p.tiles_n;
    } else {
        c.n0 = u * p.bn;
        c.par = 0;
    }
    return c;
}
// Units of this CTA: plain kernels walk units blockIdx.x, +gridDim.x, ...; CTA pairs walk pair-units (two pixel tiles
// next to each other, same channel tile) and CTA `rank` of the pair takes tile 2*m + rank.
struct UnitWalk {
    int first, stride, count, rank, pair;
    __device__ UnitWalk(const ConvKParams& p, int rank_) : rank(rank_), pair(p.pair)
    {
        first = pair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
        stride = pair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
        count = pair ? p.total_units >> 1 : p.total_units;
    }
    __device__ int unit(const ConvKParams& p, int pu) const
    {
        return pair ? (2 * (pu / p.n_ktiles) + rank) * p.n_ktiles + pu % p.n_ktiles : pu;
    }
};
__device__ __forceinline__ int unit_iters(const ConvKParams& p, int par)
{
    const int taps = p.taps[par].count;
    if (p.fh || p.hm) return p.c_blocks;
    return (p.vreuse ? taps / 3 : taps) * p.c_blocks;
}

// ring slots a unit takes: gsub k-blocks per slot, the last slot of a unit possibly with fewer
__device__ __forceinline__ int unit_stages(const ConvKParams& p, int par)
{
    const int n = unit_iters(p, par);
    return p.gsub > 1 ? (n + p.gsub - 1) / p.gsub : n;
}

// Column sums over the 32 rows a warp holds (one row per lane, 16 columns each): a butterfly that halves the
// number of columns each lane carries (16 -> 8 -> 4 -> 2 -> 1).  On return lane l holds in a[0], b[0] the totals of
// column (l >> 1) of the chunk.
__device__ __forceinline__ void butterfly16(float (&a)[16], float (&b)[16], int lane)
{
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
}

// Epilogue of one warp over all units of the CTA.  Epilogue warp e reads the TMEM lane quarter its warp index selects and the column half e >> 2
// of every accumulator.  NCH > 0: the warp owns exactly NCH 16-column chunks per unit and keeps the BatchNorm sums of
// its rows in registers across units, reducing them over rows once per statistics group.  NCH == 0: any width; sums
// are reduced over rows per unit into a per-warp shared-memory array.
template <int NCH, bool HM = false>
__device__ __forceinline__ void epilogue_loop(const ConvKParams& p, uint32_t tmem_base, uint64_t* acc_full, uint64_t* acc_empty,
                                              uint32_t* abort_flag, float* my_stats, int e, int lane, int rank)
{
    const UnitWalk walk(p, rank);
    // the accumulator-free barrier lives in the leader CTA of a pair: the peer's warps arrive on it remotely
    const bool remote_empty = p.pair && rank != 0;
    const int q = (e + 2) & 3;       // TMEM lane quarter this warp may read: (warp index in the CTA) % 4, epilogue warps start at 2
    const int m = q * 32 + lane;     // accumulator row = pixel of the tile (w fastest, then h, then image)
    const int lw = m % p.bw, lh = (m / p.bw) % p.bh, ln = m / (p.bw * p.bh);
    const bool do_stats = p.stats != nullptr;
    const int n_chunks_all = p.n_tile >> 4;
    const int first_half = (n_chunks_all + 1) >> 1;
    const int ck_begin = (e >> 2) ? first_half : 0;
    const int n_chunks = (e >> 2) ? n_chunks_all - first_half : first_half;   // chunks this warp handles
    const int col_begin = ck_begin * 16;
    constexpr int NA = NCH > 0 ? NCH * 16 : 1;
    float acc_s[NA], acc_q[NA];
#pragma unroll
    for (int i = 0; i < NA; ++i) acc_s[i] = acc_q[i] = 0.f;
    for (int i = lane; i < 256; i += 32) my_stats[i] = 0.f;
    __syncwarp();
    int jacc = 0, cur_group = -1, cur_ktile = 0;
    bool ok = true;
    long long epi_wait = 0;

    auto flush_stats = [&]() {   // this warp's partial sums of the finished statistics group -> global fp64
        double* st = p.stats + (size_t)cur_group * 2 * p.oc_valid;
        if constexpr (NCH > 0) {
#pragma unroll
            for (int ck = 0; ck < NCH; ++ck) {
                float a[16], b[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    a[i] = acc_s[ck * 16 + i];
                    b[i] = acc_q[ck * 16 + i];
                    acc_s[ck * 16 + i] = 0.f;
                    acc_q[ck * 16 + i] = 0.f;
                }
                butterfly16(a, b, lane);
                const int ch = cur_ktile * p.n_tile + col_begin + ck * 16 + (lane >> 1);
                if ((lane & 1) == 0 && ck < n_chunks && ch < p.oc_valid) {
                    atomicAdd(st + ch, (double)a[0]);
                    atomicAdd(st + p.oc_valid + ch, (double)b[0]);
                }
            }
        } else {
            __syncwarp();
            for (int c = lane; c < n_chunks * 16; c += 32) {
                const int ch = cur_ktile * p.n_tile + col_begin + c;
                if (ch < p.oc_valid) {
                    atomicAdd(st + ch, (double)my_stats[c]);
                    atomicAdd(st + p.oc_valid + ch, (double)my_stats[128 + c]);
                }
                my_stats[c] = 0.f;
                my_stats[128 + c] = 0.f;
            }
            __syncwarp();
        }
    };

    // The coordinates of a unit are worked out one unit ahead, between the probe of the current unit's accumulator barrier
    // and the use of its answer: the barrier's latency and the integer chain of the decode (about 350 cycles each, measured)
    // run side by side instead of one after the other.
    UnitCoord c_next = decode_unit(p, walk.unit(p, walk.first < walk.count ? walk.first : 0));
    for (int pu = walk.first; pu < walk.count; pu += walk.stride) {
        const UnitCoord c = c_next;
        const int n_it = unit_iters(p, c.par);
        int buf = 0;
        uint32_t full_now = 0;
        if (n_it > 0) {
            buf = jacc & (p.acc_bufs - 1);
            full_now = mbar_try_wait(&acc_full[buf], (uint32_t)(jacc >> p.acc_shift) & 1u) ? 1u : 0u;   // all lanes, one address
        }
        if (pu + walk.stride < walk.count) c_next = decode_unit(p, walk.unit(p, pu + walk.stride));
        const bool row_valid = (c.n0 + ln) < p.n_valid;
        const long long row_off = (long long)(c.n0 + ln) * p.os_n + (long long)(c.oh0 + lh) * p.os_h + (long long)(c.ow0 + lw) * p.os_w + p.off[c.par];
        if (n_it > 0) {
            if (!__all_sync(0xffffffffu, full_now != 0u)) {   // not full yet: one poller per warp
                const long long w3 = clock64();
                ok = true;
                if (lane == 0) ok = mbar_wait_bounded(&acc_full[buf], (uint32_t)(jacc >> p.acc_shift) & 1u, p.spin_limit, abort_flag);
                epi_wait += clock64() - w3;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) {
                    if (lane == 0) atomicOr(p.status, B2C_DEV_TIMEOUT);
                    break;
                }
            }
            tc_fence_after();
            ++jacc;
        }
        // A new statistics group: the finished group's sums go out.  Narrow tiles (sums in registers) do that after this unit's
        // accumulator has been read and handed back, so that the MMA threads do not wait for the reduction over rows.
        bool flush_pending = false;
        int next_group = cur_group;
        if (do_stats) {
            const int grp = p.stats_group_images > 0 ? (p.grp_shift >= 0 ? c.n0 >> p.grp_shift : c.n0 / p.stats_group_images) : 0;
            if (grp != cur_group) {
                if (cur_group >= 0) {
                    if constexpr (NCH > 0) flush_pending = true;
                    else flush_stats();
                }
                next_group = grp;
                if constexpr (NCH == 0) cur_group = grp;
            }
            if constexpr (NCH == 0) cur_ktile = c.ktile;
        }
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * p.acc_cols + col_begin);
        // the accumulator is handed back to the MMA thread as soon as this warp has read its last column
        auto release = [&]() {
            if (n_it > 0) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (remote_empty) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[buf]), 0));
                    else mbar_arrive(&acc_empty[buf]);
                }
            }
        };
        // bias, rounding and stores of one 16-column chunk; returns the values as stored in pk
        auto store_chunk = [&](const uint32_t (&r)[16], int c0, uint32_t (&pk)[8]) {
            const int ch0 = c.ktile * p.n_tile + col_begin + c0;  // first output channel of this chunk
            float v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
            if (!HM && p.bias != nullptr) {   // (merged-tap plans have neither a bias nor fp32 output)
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] += (ch0 + i < p.oc_valid) ? __ldg(p.bias + ch0 + i) : 0.f;
            }
            if (!HM && p.out_is_f32) {
                if (row_valid) {
                    float* dst = reinterpret_cast<float*>(p.out) + row_off + ch0;
#pragma unroll
                    for (int i = 0; i < 16; i += 4)
                        if (ch0 + i < p.oc_valid) *reinterpret_cast<float4*>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                }
                return;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) pk[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
            if (row_valid) {
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + row_off + ch0;
                if (p.out_v8 && ch0 + 8 < p.oc_valid) {
                    st_global_v8(dst, pk);   // one full 32-byte sector per lane
                } else {
                    if (ch0 < p.oc_valid) *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    if (ch0 + 8 < p.oc_valid) *reinterpret_cast<uint4*>(dst + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
            }
        };

        if constexpr (NCH > 0) {
            // narrow tiles: read all of this warp's columns at once, free the accumulator, then work from registers
            uint32_t r[NCH][16];
            if constexpr (HM) {
                // Merged horizontal taps: the accumulator holds three blocks of n_tile columns, block s = the contribution of
                // filter column s evaluated at this row's own pixel.  Output pixel w takes block 0 of pixel w - 1, block 1 of its
                // own pixel and block 2 of pixel w + 1; a warp's 32 rows are whole image rows, so the neighbours are the
                // adjacent lanes, and the first / last pixel of an image row has no left / right neighbour (zero padding).
                const float m_left = lw != 0 ? 1.f : 0.f, m_right = lw != p.bw - 1 ? 1.f : 0.f;
#pragma unroll
                for (int ck = 0; ck < NCH; ++ck) {
                    uint32_t d0[16], d1[16], d2[16];
                    tmem_ld16(t_row + (uint32_t)(ck * 16), d0);
                    tmem_ld16(t_row + (uint32_t)(p.n_tile + ck * 16), d1);
                    tmem_ld16(t_row + (uint32_t)(2 * p.n_tile + ck * 16), d2);
                    tmem_ld_wait();
                    if (ck == NCH - 1) release();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float left = __shfl_up_sync(0xffffffffu, __uint_as_float(d0[i]), 1);
                        const float right = __shfl_down_sync(0xffffffffu, __uint_as_float(d2[i]), 1);
                        r[ck][i] = __float_as_uint(fmaf(left, m_left, fmaf(right, m_right, __uint_as_float(d1[i]))));
                    }
                }
            } else {
#pragma unroll
            for (int ck = 0; ck < NCH; ++ck) {
                if (n_it > 0 && ck < n_chunks) {
                    tmem_ld16(t_row + (uint32_t)(ck * 16), r[ck]);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[ck][i] = 0u;
                }
            }
            if (n_it > 0) tmem_ld_wait();
            release();
            }
            if (flush_pending) flush_stats();   // still the previous group's sums and channel tile
            cur_group = next_group;
            cur_ktile = c.ktile;
#pragma unroll
            for (int ck = 0; ck < NCH; ++ck) {
                if (ck < n_chunks) {
                    uint32_t pk[8];
                    store_chunk(r[ck], ck * 16, pk);
                    if (do_stats && row_valid) {   // sums of the values as stored, kept per row in registers
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            __nv_bfloat162 h = *reinterpret_cast<__nv_bfloat162*>(&pk[i]);
                            const float lo = __low2float(h), hi = __high2float(h);
                            acc_s[ck * 16 + 2 * i] += lo;
                            acc_s[ck * 16 + 2 * i + 1] += hi;
                            acc_q[ck * 16 + 2 * i] = fmaf(lo, lo, acc_q[ck * 16 + 2 * i]);
                            acc_q[ck * 16 + 2 * i + 1] = fmaf(hi, hi, acc_q[ck * 16 + 2 * i + 1]);
                        }
                    }
                }
            }
        } else {
            auto process = [&](const uint32_t (&r)[16], int c0) {
                uint32_t pk[8];
                store_chunk(r, c0, pk);
                if (do_stats && !p.out_is_f32) {
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
                    butterfly16(a, b, lane);
                    if ((lane & 1) == 0) {   // the array is private to this warp
                        const int col = c0 + (lane >> 1);
                        my_stats[col] += a[0];
                        my_stats[128 + col] += b[0];
                    }
                }
            };
            uint32_t ra[16], rb[16];
            if (n_it > 0 && n_chunks > 0) {
                tmem_ld16(t_row, ra);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) ra[i] = rb[i] = 0u;
            }
            if (n_chunks <= 1) release();
            for (int ck = 0; ck < n_chunks; ck += 2) {
                // chunk ck is in ra; fetch ck+1 into rb while ra is processed, then ck+2 into ra while rb is processed
                if (n_it > 0 && ck + 1 < n_chunks) tmem_ld16(t_row + (uint32_t)((ck + 1) * 16), rb);
                process(ra, ck * 16);
                if (ck + 1 < n_chunks) {
                    if (n_it > 0) {
                        tmem_ld_wait();
                        if (ck + 2 == n_chunks) release();
                        if (ck + 2 < n_chunks) tmem_ld16(t_row + (uint32_t)((ck + 2) * 16), ra);
                    }
                    process(rb, (ck + 1) * 16);
                    if (n_it > 0 && ck + 2 < n_chunks) {
                        tmem_ld_wait();
                        if (ck + 3 == n_chunks) release();
                    }
                }
            }
        }
    }
    if (do_stats && cur_group >= 0 && ok) flush_stats();
    if (p.stall != nullptr && e == 0 && lane == 0) atomicAdd(p.stall + 3, (unsigned long long)epi_wait);
}

// Issues the MMAs of one stage: NB sub-tiles (vertical taps) x KS k-steps of 16 channels, fully unrolled so that
// the issuing thread spends a handful of independent instructions per MMA (its own dependent-issue latency, not the
// tensor pipe, bounds small-N tiles otherwise).  Descriptor low words advance by 32 bytes per k-step inside the
// swizzle atom and by a_step / b_step per sub-tile.
template <int KS, int NB, bool PAIR>
__device__ __forceinline__ void issue_stage(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                            uint32_t a_step16, uint32_t b_step16, uint32_t accumulate_first)
{
#pragma unroll
    for (int j = 0; j < NB; ++j) {
#pragma unroll
        for (int k = 0; k < KS; ++k) {
            const uint64_t ad = ((uint64_t)desc_hi << 32) | (uint64_t)(a_lo + (uint32_t)j * a_step16 + 2u * k);
            const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(b_lo + (uint32_t)j * b_step16 + 2u * k);
            if constexpr (PAIR) umma_bf16_pair(d_tmem, ad, bd, idesc, (j == 0 && k == 0) ? accumulate_first : 1u);
            else umma_bf16(d_tmem, ad, bd, idesc, (j == 0 && k == 0) ? accumulate_first : 1u);
        }
    }
}

// Full-halo stage: the A tile is a box of (bw + 2) x (bh + 2) pixels with bw = 8, so every image row of the tile is
// one 8-row group of the K-major operand and the group stride (SBO) is bw + 2 rows.  Tap (r, s) reads the same box
// starting r image rows and s pixels further in: a start address that is a whole number of 128-byte rows off the
// swizzle atom, which works because the swizzle is keyed on absolute shared-memory address bits (measured: exact
// results for arbitrary row offsets and group strides).  B tiles come from the resident bank, order [s][cb][r].
template <int KS, bool PAIR>
__device__ __forceinline__ void issue_stage_fh(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_hi, uint32_t b_hi, uint32_t idesc,
                                               uint32_t a_row16, uint32_t a_rowpitch16, uint32_t b_tile16, uint32_t b_s16,
                                               uint32_t accumulate_first)
{
#pragma unroll
    for (int sft = 0; sft < 3; ++sft) {
#pragma unroll
        for (int r = 0; r < 3; ++r) {
#pragma unroll
            for (int k = 0; k < KS; ++k) {
                const uint64_t ad = ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + (uint32_t)r * a_rowpitch16 + (uint32_t)sft * a_row16 + 2u * k);
                const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + (uint32_t)sft * b_s16 + (uint32_t)r * b_tile16 + 2u * k);
                const uint32_t acc = (sft == 0 && r == 0 && k == 0) ? accumulate_first : 1u;
                if constexpr (PAIR) umma_bf16_pair(d_tmem, ad, bd, idesc, acc);
                else umma_bf16(d_tmem, ad, bd, idesc, acc);
            }
        }
    }
}

// One MMA-issuing thread.  The CTA runs kIssuers of them (in different warps): issuer `my` accumulates the CTA's units
// my, my + kIssuers, ... (unit j always into accumulator j % acc_bufs) and steps over the ring stages of the others.  A single
// thread cannot keep the tensor pipe busy on narrow tiles: it pays roughly 45 cycles per tcgen05.mma, 180 per barrier
// wait and 55 per commit, all serial, against 48-64 cycles the pipe needs per MMA at N <= 128; two threads working on
// different accumulators can.
template <int KS, int NB, bool PAIR, bool GROUP, bool FH>
__device__ __forceinline__ void mma_issuer(const ConvKParams& p, const UnitWalk& walk, int my, uint32_t tmem_base, uint32_t smem_addr,
                                           uint32_t ring_addr, int stage_bytes, uint64_t* full_bar, uint64_t* empty_bar, uint64_t* acc_full,
                                           uint64_t* acc_empty, uint64_t* w_bar, uint64_t* init_bar, uint32_t* abort_flag, const int* slot_stage)
{
    const uint32_t idesc = make_idesc_bf16(PAIR ? 256 : 128, p.mma_n, false, false);
    const uint32_t sbo = 8u * (uint32_t)p.kb * 2u;  // eight rows of kb bf16
    const uint64_t desc_proto = make_smem_desc(0u, 16u, sbo, (uint32_t)p.swz);
    const uint32_t desc_hi = (uint32_t)(desc_proto >> 32), desc_lo_base = (uint32_t)desc_proto;
    // full halo: A groups are (bw + 2) rows apart
    const uint32_t a_hi_fh = (uint32_t)(make_smem_desc(0u, 16u, (uint32_t)(p.bw + 2) * (uint32_t)p.kb * 2u, (uint32_t)p.swz) >> 32);
    const uint32_t a_row16 = ((uint32_t)p.kb * 2u) >> 4, a_rowpitch16 = (uint32_t)(p.bw + 2) * a_row16;
    const uint32_t b_s16 = (uint32_t)(p.c_blocks * 3 * p.b_bytes) >> 4;
    const uint32_t a_to_b16 = (uint32_t)p.a_bytes >> 4, a_step16 = (uint32_t)p.a_step >> 4;
    // B tiles of consecutive vertical taps are adjacent, in a stage and in the resident bank alike
    const uint32_t b_step16 = (uint32_t)p.b_bytes >> 4;
    const uint32_t b_cb16 = (uint32_t)(p.nb * p.b_bytes) >> 4, stage16 = (uint32_t)stage_bytes >> 4;
    const int G = GROUP ? p.gsub : 1;
    const uint32_t sub16 = GROUP ? stage16 / (uint32_t)G : stage16;   // one k-block inside a slot
    const uint32_t ring_lo = desc_lo_base + (ring_addr >> 4), bank_lo = desc_lo_base + (smem_addr >> 4);
    const int S = p.stages;
    const bool timed = p.stall != nullptr;
    const int units_per_par = p.n_par > 1 ? p.total_units / p.n_par : 1;
    const int n_it_fixed = unit_iters(p, 0);
    bool ok = true;
    if (p.resident && !mbar_wait_bounded(w_bar, 0u, p.spin_limit, abort_flag)) {
        atomicOr(p.status, B2C_DEV_TIMEOUT);
        ok = false;
    }
    int s = 0, j = 0, i_stage = 0;   // ring slot and index of the next stage in CTA order, count of units that have stages
    uint32_t ph = 0;
    long long wait_ring = 0, wait_acc = 0;
    for (int pu = walk.first; ok && pu < walk.count; pu += walk.stride) {
        int n_sub = n_it_fixed;   // k-blocks of the unit
        if (p.n_par > 1) n_sub = unit_iters(p, walk.unit(p, pu) / units_per_par);
        if (n_sub == 0) continue;   // a parity without taps: the epilogue stores zeros without an accumulator
        const int n_it = GROUP ? (n_sub + G - 1) / G : n_sub;   // ring slots of the unit
        if ((j % p.issuers) != my) {   // another issuer's unit: step over its stages
            i_stage += n_it;
            s += n_it;
            while (s >= S) { s -= S; ph ^= 1u; }
            ++j;
            continue;
        }
        const int buf = j & (p.acc_bufs - 1);
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.acc_cols);
        uint32_t b_res = bank_lo;   // resident bank: B tile of (tap or horizontal shift, channel block), consecutive per stage
        for (int it = 0; it < n_it; ++it) {
            int n_k = 1;   // k-blocks in this slot
            if constexpr (GROUP) n_k = n_sub - it * G < G ? n_sub - it * G : G;
            const long long w2 = timed ? clock64() : 0;
            // A parity wait tells a barrier's phases apart only modulo two, and with two issuers this thread may reach a
            // slot before the slot's previous stage (another issuer's) was even loaded.  A producer issues the load of
            // stage i only after the previous stage in that slot was consumed, and then stamps the slot with i + 1:
            // seeing the stamp pass i makes the parity wait unambiguous.
            if (p.issuers > 1) {
                uint32_t polls = 0;
                while (ld_volatile_shared(&slot_stage[s]) <= i_stage) {
                    if (++polls > p.spin_limit || *(volatile uint32_t*)abort_flag != 0u) {
                        ok = false;
                        break;
                    }
                }
            }
            if (!ok || !mbar_wait_bounded(&full_bar[s], ph, p.spin_limit, abort_flag)) {
                *(volatile uint32_t*)abort_flag = 1u;
                atomicOr(p.status, B2C_DEV_TIMEOUT);
                ok = false;
                break;
            }
            if (timed) wait_ring += clock64() - w2;
            // The accumulator comes second: the unit's first slot is usually full long before the epilogue hands the accumulator
            // back, so the slot's stamp and barrier (600-700 cycles of this thread) are off the path from "accumulator free" to
            // the first MMA, the loop that bounds narrow tiles with two accumulators.
            if (it == 0) {
                const long long w1 = timed ? clock64() : 0;
                if (!mbar_wait_bounded(&acc_empty[buf], ((uint32_t)(j >> p.acc_shift) & 1u) ^ 1u, p.spin_limit, abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    ok = false;
                    break;
                }
                if (timed) wait_acc += clock64() - w1;
            }
            tc_fence_after();
            // descriptors differ from stage to stage only in the 14-bit address field: add offsets to the low word
            if constexpr (GROUP) {   // (never with full-halo or merged-tap stages)
                uint32_t a_lo = ring_lo + (uint32_t)s * stage16;
                for (int g = 0; g < n_k; ++g) {
                    const uint32_t b_lo = p.resident ? b_res : a_lo + a_to_b16;
                    issue_stage<KS, NB, PAIR>(d_tmem, a_lo, b_lo, desc_hi, idesc, a_step16, b_step16, (it | g) != 0 ? 1u : 0u);
                    b_res += b_cb16;
                    a_lo += sub16;
                }
            } else {
                const uint32_t a_lo = ring_lo + (uint32_t)s * stage16;
                const uint32_t b_lo = p.resident ? b_res : a_lo + a_to_b16;
                if constexpr (FH) issue_stage_fh<KS, PAIR>(d_tmem, a_lo, b_lo, a_hi_fh, desc_hi, idesc, a_row16, a_rowpitch16, b_step16, b_s16, it != 0 ? 1u : 0u);
                else issue_stage<KS, NB, PAIR>(d_tmem, a_lo, b_lo, desc_hi, idesc, a_step16, b_step16, it != 0 ? 1u : 0u);
                b_res += b_cb16;
            }
            // frees the stage (in both CTAs of a pair) once these MMAs have read it
            if constexpr (PAIR) umma_commit_pair(&empty_bar[s], (uint16_t)3);
            else umma_commit(&empty_bar[s]);
            ++i_stage;
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        if constexpr (PAIR) umma_commit_pair(&acc_full[buf], (uint16_t)3);
        else umma_commit(&acc_full[buf]);
        ++j;
    }
    if (timed) {
        atomicAdd(p.stall + 1, (unsigned long long)wait_ring);
        atomicAdd(p.stall + 2, (unsigned long long)wait_acc);
    }
}

// The two MMA-issuing threads of a CTA sharing every unit (tiles wider than 128 channels, where TMEM holds two accumulators
// and the threads cannot take alternate units).  Stage i of the CTA belongs to thread i % 2; the ring depth is even, so
// thread `my` owns the slots my, my + 2, ... and walks them in order with its own phase bit: a slot has one consumer and
// needs no stamp.  Both threads accumulate into the unit's accumulator (accumulation commutes; the tensor pipe runs MMAs
// one after the other).  The thread that does not own a unit's first stage, whose first MMA overwrites the accumulator,
// waits for that stage's completion barrier instead of the accumulator-free barrier (the first stage was issued after
// the accumulator had been freed); both threads commit to the accumulator-full barrier (count 2).  This thread's chain
// of dependent instructions per slot is what bounds these layers, so the loop carries nothing it does not need.
template <int KS, int NB, bool PAIR, bool GROUP>
__device__ __forceinline__ void mma_issuer_split(const ConvKParams& p, const UnitWalk& walk, int my, uint32_t tmem_base, uint32_t smem_addr,
                                                 uint32_t ring_addr, int stage_bytes, uint64_t* full_bar, uint64_t* empty_bar, uint64_t* acc_full,
                                                 uint64_t* acc_empty, uint64_t* w_bar, uint64_t* init_bar, uint32_t* abort_flag)
{
    const uint32_t idesc = make_idesc_bf16(PAIR ? 256 : 128, p.mma_n, false, false);
    const uint64_t desc_proto = make_smem_desc(0u, 16u, 8u * (uint32_t)p.kb * 2u, (uint32_t)p.swz);
    const uint32_t desc_hi = (uint32_t)(desc_proto >> 32), desc_lo_base = (uint32_t)desc_proto;
    const uint32_t a_to_b16 = (uint32_t)p.a_bytes >> 4, a_step16 = (uint32_t)p.a_step >> 4, b_step16 = (uint32_t)p.b_bytes >> 4;
    const uint32_t b_cb16 = (uint32_t)(p.nb * p.b_bytes) >> 4, stage16 = (uint32_t)stage_bytes >> 4;
    const int G = GROUP ? p.gsub : 1;
    const uint32_t sub16 = GROUP ? stage16 / (uint32_t)G : stage16;
    const uint32_t ring_lo = desc_lo_base + (ring_addr >> 4), bank_lo = desc_lo_base + (smem_addr >> 4);
    const int S = p.stages;
    const bool timed = p.stall != nullptr, resident = p.resident != 0;
    const int n_sub_fixed = unit_iters(p, 0);
    const int units_per_par = p.n_par > 1 ? p.total_units / p.n_par : 1;
    long long wait_ring = 0, wait_acc = 0;
    bool ok = true;
    if (resident && !mbar_wait_bounded(w_bar, 0u, p.spin_limit, abort_flag)) {
        atomicOr(p.status, B2C_DEV_TIMEOUT);
        ok = false;
    }
    int s = my, k = my;   // this thread's next slot, and the index (in CTA order) of the stage that goes there
    uint32_t ph = 0;
    int i0 = 0, j = 0;    // index of the unit's first stage, count of units with stages
    for (int pu = walk.first; ok && pu < walk.count; pu += walk.stride) {
        int n_sub = n_sub_fixed;
        if (p.n_par > 1) n_sub = unit_iters(p, walk.unit(p, pu) / units_per_par);
        if (n_sub == 0) continue;
        const int i_end = i0 + (GROUP ? (n_sub + G - 1) / G : n_sub);
        const int buf = j & (p.acc_bufs - 1);
        const uint32_t acc_par = (uint32_t)(j >> p.acc_shift) & 1u;
        if (k < i_end) {
            const long long w1 = timed ? clock64() : 0;
            const bool mine_first = k == i0;
            if (!mbar_wait_bounded(mine_first ? &acc_empty[buf] : &init_bar[buf], mine_first ? acc_par ^ 1u : acc_par, p.spin_limit, abort_flag)) {
                atomicOr(p.status, B2C_DEV_TIMEOUT);
                ok = false;
                break;
            }
            if (timed) wait_acc += clock64() - w1;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.acc_cols);
            do {
                const int it = k - i0;
                const long long w2 = timed ? clock64() : 0;
                if (!mbar_wait_bounded(&full_bar[s], ph, p.spin_limit, abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    ok = false;
                    break;
                }
                if (timed) wait_ring += clock64() - w2;
                tc_fence_after();
                uint32_t a_lo = ring_lo + (uint32_t)s * stage16;
                if constexpr (GROUP) {
                    const int n_k = n_sub - it * G < G ? n_sub - it * G : G;
                    uint32_t b_res = bank_lo + (uint32_t)(it * G) * b_cb16;
                    for (int g = 0; g < n_k; ++g) {
                        issue_stage<KS, NB, PAIR>(d_tmem, a_lo, resident ? b_res : a_lo + a_to_b16, desc_hi, idesc, a_step16, b_step16, (it | g) != 0 ? 1u : 0u);
                        b_res += b_cb16;
                        a_lo += sub16;
                    }
                } else {
                    issue_stage<KS, NB, PAIR>(d_tmem, a_lo, resident ? bank_lo + (uint32_t)it * b_cb16 : a_lo + a_to_b16, desc_hi, idesc, a_step16, b_step16,
                                              it != 0 ? 1u : 0u);
                }
                if constexpr (PAIR) umma_commit_pair(&empty_bar[s], (uint16_t)3);   // frees the stage in both CTAs of a pair
                else umma_commit(&empty_bar[s]);
                if (it == 0) {   // the overwriting stage (both issuing threads live in the leader CTA of a pair)
                    if constexpr (PAIR) umma_commit_pair(&init_bar[buf], (uint16_t)1);
                    else umma_commit(&init_bar[buf]);
                }
                k += 2;
                s += 2;
                if (s >= S) { s = my; ph ^= 1u; }
            } while (k < i_end);
            if (!ok) break;
        }
        if constexpr (PAIR) umma_commit_pair(&acc_full[buf], (uint16_t)3);
        else umma_commit(&acc_full[buf]);
        i0 = i_end;
        ++j;
    }
    if (timed) {
        atomicAdd(p.stall + 1, (unsigned long long)wait_ring);
        atomicAdd(p.stall + 2, (unsigned long long)wait_acc);
    }
}

// The kernel comes in four kinds, one per family of launch plans, so that each carries only the issuing and epilogue code its
// plans use (with all of them in one kernel the code of a launch was spread over several hundred KB and the 64- and
// 128-channel layers ran 7-12 % slower inside a training step, where every launch starts on a cold instruction cache):
// general (one MMA per tap or vertical tap reuse, any tile width up to 128 channels), split (tiles wider than 128 channels:
// two issuing threads share every unit), merged horizontal taps, full-halo stages.
enum : int { KIND_GENERAL = 0, KIND_SPLIT = 1, KIND_HMERGE = 2, KIND_FULL_HALO = 3 };
template <bool PAIR, int KIND>
__global__ void __launch_bounds__(kThreads, 1) conv_kmajor_kernel(const __grid_constant__ ConvKParams p)
{
    const int rank = PAIR ? (int)cluster_ctarank() : 0;   // 0 = leader of the pair: issues the MMAs, owns the barriers the pair shares
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], acc_full[kMaxAccBufs], acc_empty[kMaxAccBufs], init_bar[kMaxAccBufs], w_bar, drain_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t abort_flag;
    __shared__ int slot_stage[kMaxStages];   // per ring slot: 1 + index of the stage whose loads were issued into it last
    __shared__ float s_stats[kEpiWarps][256];   // per epilogue warp (128 columns at most): [0,128) sums, [128,256) sums of squares

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~uintptr_t(1023));
    uint8_t* ring = smem + p.resident_bytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;
    const int sub_bytes = p.a_bytes + (p.resident ? 0 : p.nb * p.b_bytes);   // one k-block: the A tile and, unless the bank is resident, its filter tiles
    const int stage_bytes = p.gsub * sub_bytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < kMaxAccBufs; ++b) {
            mbar_init(&acc_full[b], p.issue_split ? 2 : 1);   // shared units: both issuing threads commit
            mbar_init(&init_bar[b], 1);
            mbar_init(&acc_empty[b], PAIR ? 2 * kEpiWarps : kEpiWarps);   // one arrival per epilogue warp (of both CTAs of a pair)
        }
        mbar_init(&w_bar, 1);
        mbar_init(&drain_bar, kIssuers);
        abort_flag = 0;
        for (int i = 0; i < kMaxStages; ++i) slot_stage[i] = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        if constexpr (PAIR) {
            tmem_alloc_pair(&tmem_slot, (uint32_t)p.tmem_cols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(&tmem_slot, (uint32_t)p.tmem_cols);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();   // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    // set-up done (it touched no global data): order behind the previous kernel of the stream, then let the next one in
    pdl_wait();
    pdl_launch_dependents();
    const long long t_start = clock64();
    const UnitWalk walk(p, rank);
    int last_issued = -1;  // producer lanes: index of the last stage whose loads this lane issued

    if (warp == 0 || warp == kProducerWarp1) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producers
            // Producer w fills the ring slots w, w + kProducers, ...: the chain wait -> expect -> issue of one thread
            // (several hundred cycles) would otherwise bound short stages.  Splitting by slot (not by stage) keeps
            // every slot with one producer that uses it strictly in order, which a parity wait on its barrier needs.
            const int w = warp == 0 ? 0 : 1;
            prefetch_tensormap(&p.tmB);
            prefetch_tensormap(&p.tmA[0]);
            // a pair counts the bytes of both CTAs on the leader's barriers; b_row = first filter row this CTA fetches
            const int b_rows = PAIR ? p.n_tile >> 1 : p.n_tile;
            const int R = p.r_filter;
            const uint32_t w_bar_cl = PAIR ? map_to_cta(smem_u32(&w_bar), 0) : 0u;
            if (KIND == KIND_HMERGE && w == 0) {
                // merged horizontal taps: per channel block one box of all nine taps, landing as [r][s][out][64 in]:
                // three tiles (one per filter row) of 3 x n_tile rows
                const int oc0 = (walk.first % p.n_ktiles) * p.n_tile;
                mbar_expect_tx(&w_bar, (uint32_t)(p.c_blocks * 3 * p.tx_b));
                for (int cb = 0; cb < p.c_blocks; ++cb)
                    tma_load_4d(smem + (size_t)cb * 3 * p.b_bytes, &p.tmB, &w_bar, cb * p.kb, oc0, 0, 0);
            } else if (KIND != KIND_HMERGE && p.resident && w == 0) {
                // bank order: [tap or horizontal shift][channel block][vertical tap]
                const int ktile = walk.first % p.n_ktiles;   // the walk stride is a multiple of n_ktiles: fixed per CTA
                const TapList& tl = p.taps[0];
                const int oc0 = ktile * p.n_tile + rank * b_rows;
                if (rank == 0) mbar_expect_tx(&w_bar, (uint32_t)((PAIR ? 2 : 1) * tl.count * p.c_blocks * p.tx_b));
                const int groups = (p.vreuse || p.fh) ? tl.count / 3 : tl.count;
                for (int t = 0; t < groups; ++t)
                    for (int cb = 0; cb < p.c_blocks; ++cb) {
                        uint8_t* dst = smem + (size_t)(t * p.c_blocks + cb) * p.nb * p.b_bytes;
                        const int n_loads = p.b_merged ? 1 : p.nb;
                        for (int v = 0; v < n_loads; ++v) {
                            const int rs = tl.rs[t + 3 * v];
                            if constexpr (PAIR) tma_load_4d_pair(dst + (size_t)v * p.b_bytes, &p.tmB, w_bar_cl, cb * p.kb, rs % R, oc0, rs / R);
                            else tma_load_4d(dst + (size_t)v * p.b_bytes, &p.tmB, &w_bar, cb * p.kb, rs % R, oc0, rs / R);
                        }
                    }
            }
            bool ok = true;
            long long waited = 0;
            const bool timed = p.stall != nullptr;
            int i = w, i_base = 0;   // this producer's next stage and the first stage of the current unit, in CTA order
            int s = w;   // w < kProducers <= S
            uint32_t ph = 0u;
            const uint32_t stage_tx = (uint32_t)(p.tx_a + (p.resident ? 0 : p.nb * p.tx_b));
            const int n_b_loads = p.resident ? 0 : (p.b_merged ? 1 : p.nb);
            for (int pu = walk.first; ok && pu < walk.count; pu += walk.stride) {
                const int u = walk.unit(p, pu);
                const int n_sub = unit_iters(p, p.n_par > 1 ? u / (p.total_units / p.n_par) : 0);
                const int G = (KIND == KIND_GENERAL || KIND == KIND_SPLIT) ? p.gsub : 1;   // (full-halo and merged-tap stages are never grouped)
                const int n_it = G > 1 ? (n_sub + G - 1) / G : n_sub;   // ring slots of the unit
                if (i >= i_base + n_it) {   // no stage of this unit is mine
                    i_base += n_it;
                    continue;
                }
                const UnitCoord c = decode_unit(p, u);
                const TapList& tl = p.taps[c.par];
                const int oc0 = c.ktile * p.n_tile + rank * b_rows;
                while (i < i_base + n_it) {
                    const int it = i - i_base;
                    // waits until the slot's previous stage has been consumed; that stage's barrier phase is then over, and the
                    // stamp lets issuers that take alternate units tell the slot's phases apart (a relaxed store: the wait orders it)
                    auto wait_empty = [&]() -> bool {
                        const long long w0 = timed ? clock64() : 0;
                        if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, p.spin_limit, &abort_flag)) {
                            atomicOr(p.status, B2C_DEV_TIMEOUT);
                            ok = false;
                            return false;
                        }
                        if (timed) waited += clock64() - w0;
                        if (p.issuers > 1 && !p.issue_split) st_volatile_shared(&slot_stage[s], i + 1);
                        return true;
                    };
                    if (G > 1) {
                        if (!wait_empty()) break;
                        // the k-blocks that share this slot (one, except where short k-blocks are grouped)
                        const int k_first = it * G, n_k = n_sub - k_first < G ? n_sub - k_first : G;
                        if constexpr (PAIR) {
                            if (rank == 0) mbar_expect_tx(&full_bar[s], 2u * (uint32_t)n_k * stage_tx);
                        } else {
                            mbar_expect_tx(&full_bar[s], (uint32_t)n_k * stage_tx);
                        }
                        for (int g = 0; g < n_k; ++g) {
                            const int kblk = k_first + g;
                            const int t0 = p.cb_shift >= 0 ? kblk >> p.cb_shift : kblk / p.c_blocks;   // tap
                            const int cb = kblk - t0 * p.c_blocks;                                       // channel block
                            uint8_t* a_dst = ring + (size_t)s * stage_bytes + (size_t)g * sub_bytes;
                            if constexpr (PAIR) {
                                const uint32_t full_cl = map_to_cta(smem_u32(&full_bar[s]), 0);
                                tma_load_4d_pair(a_dst, &p.tmA[tl.map[t0]], full_cl, cb * p.kb, c.ow0 + tl.dw[t0], c.oh0 + tl.dh[t0], c.n0);
                                for (int v = 0; v < n_b_loads; ++v) {
                                    const int rs = tl.rs[t0 + 3 * v], fr = (rs * 11) >> 5;   // rs / 3 for rs < 9 (R is 1 or 3)
                                    tma_load_4d_pair(a_dst + p.a_bytes + (size_t)v * p.b_bytes, &p.tmB, full_cl, cb * p.kb, rs - fr * R, oc0, fr);
                                }
                            } else {
                                tma_load_4d(a_dst, &p.tmA[tl.map[t0]], &full_bar[s], cb * p.kb, c.ow0 + tl.dw[t0], c.oh0 + tl.dh[t0], c.n0);
                                for (int v = 0; v < n_b_loads; ++v) {
                                    const int rs = tl.rs[t0 + 3 * v], fr = (rs * 11) >> 5;   // rs / 3 for rs < 9 (R is 1 or 3)
                                    tma_load_4d(a_dst + p.a_bytes + (size_t)v * p.b_bytes, &p.tmB, &full_bar[s], cb * p.kb, rs - fr * R, oc0, fr);
                                }
                            }
                        }
                    } else {
                        // (operands first, the wait second: the address arithmetic is off the chain wait -> expect -> issue)
                        int t0 = p.cb_shift >= 0 ? it >> p.cb_shift : it / p.c_blocks;   // tap (or horizontal shift)
                        const int cb = it - t0 * p.c_blocks;                               // channel block
                        if (KIND == KIND_HMERGE || KIND == KIND_FULL_HALO) t0 = 0;   // one box per channel block: the entry of tap (0, 0) carries its origin
                        uint8_t* a_dst = ring + (size_t)s * stage_bytes;
                        // with vreuse the table entry of vertical tap 0 carries the shift of the whole haloed tile
                        const CUtensorMap* map_a = &p.tmA[tl.map[t0]];
                        const int ca = cb * p.kb, wa = c.ow0 + (KIND == KIND_HMERGE ? 0 : tl.dw[t0]), ha = c.oh0 + tl.dh[t0];   // merged taps: no horizontal shift
                        int b_s[3], b_r[3];
#pragma unroll
                        for (int v = 0; v < 3; ++v) {
                            const int rs = v < n_b_loads ? tl.rs[t0 + 3 * v] : 0, fr = (rs * 11) >> 5;   // rs / 3 for rs < 9 (R is 1 or 3)
                            b_s[v] = rs - fr * R;
                            b_r[v] = fr;
                        }
                        if (!wait_empty()) break;
                        if constexpr (PAIR) {
                            const uint32_t full_cl = map_to_cta(smem_u32(&full_bar[s]), 0);
                            if (rank == 0) mbar_expect_tx(&full_bar[s], 2u * stage_tx);
                            tma_load_4d_pair(a_dst, map_a, full_cl, ca, wa, ha, c.n0);
#pragma unroll
                            for (int v = 0; v < 3; ++v)
                                if (v < n_b_loads) tma_load_4d_pair(a_dst + p.a_bytes + (size_t)v * p.b_bytes, &p.tmB, full_cl, ca, b_s[v], oc0, b_r[v]);
                        } else {
                            mbar_expect_tx(&full_bar[s], stage_tx);
                            tma_load_4d(a_dst, map_a, &full_bar[s], ca, wa, ha, c.n0);
#pragma unroll
                            for (int v = 0; v < 3; ++v)
                                if (v < n_b_loads) tma_load_4d(a_dst + p.a_bytes + (size_t)v * p.b_bytes, &p.tmB, &full_bar[s], ca, b_s[v], oc0, b_r[v]);
                        }
                    }
                    last_issued = i;
                    if (s + kProducers < S) {
                        i += kProducers;
                        s += kProducers;
                    } else {   // wrap to this producer's first slot
                        i += S - s + w;
                        s = w;
                        ph ^= 1u;
                    }
                }
                i_base += n_it;
            }
            if (p.stall != nullptr && rank == 0 && w == 0) {
                atomicAdd(p.stall + 0, (unsigned long long)waited);
                atomicAdd(p.stall + 4, (unsigned long long)(clock64() - t_start));
            }
        }
    } else if (warp == 1 || (warp >= 2 + kEpiWarps && warp < kProducerWarp1)) {
        if (lane == 0 && rank == 0) {
            // ------------------------------------------------------------ MMA issuers (in the leader CTA of a pair)
            const int my = warp == 1 ? 0 : warp - (2 + kEpiWarps) + 1;
            if (my < p.issuers) {
            const uint32_t smem_addr = smem_u32(smem), ring_addr = smem_u32(ring);
            const int ksteps = p.kb >> 4;
            if constexpr (KIND == KIND_SPLIT) {
#define B2C_ISSUER_S(KS, NB, GR) mma_issuer_split<KS, NB, PAIR, GR>(p, walk, my, tmem_base, smem_addr, ring_addr, stage_bytes, full_bar, empty_bar, acc_full, acc_empty, &w_bar, init_bar, &abort_flag)
                if (p.nb == 3) {
                    if (ksteps == 4) B2C_ISSUER_S(4, 3, false);
                    else if (ksteps == 2) B2C_ISSUER_S(2, 3, false);
                    else B2C_ISSUER_S(1, 3, false);
                } else if (p.gsub > 1) {
                    if (ksteps == 4) B2C_ISSUER_S(4, 1, true);
                    else if (ksteps == 2) B2C_ISSUER_S(2, 1, true);
                    else B2C_ISSUER_S(1, 1, true);
                } else {
                    if (ksteps == 4) B2C_ISSUER_S(4, 1, false);
                    else if (ksteps == 2) B2C_ISSUER_S(2, 1, false);
                    else B2C_ISSUER_S(1, 1, false);
                }
#undef B2C_ISSUER_S
            } else {
#define B2C_ISSUER(KS, NB, GR, FH) mma_issuer<KS, NB, PAIR, GR, FH>(p, walk, my, tmem_base, smem_addr, ring_addr, stage_bytes, full_bar, empty_bar, acc_full, acc_empty, &w_bar, init_bar, &abort_flag, slot_stage)
                if constexpr (KIND == KIND_HMERGE) {
                    B2C_ISSUER(4, 3, false, false);   // 64-channel k-blocks, the three filter rows of a channel block per stage
                } else if constexpr (KIND == KIND_FULL_HALO) {
                    B2C_ISSUER(4, 3, false, true);
                } else if (p.nb == 3) {
                    if (ksteps == 4) B2C_ISSUER(4, 3, false, false);
                    else if (ksteps == 2) B2C_ISSUER(2, 3, false, false);
                    else B2C_ISSUER(1, 3, false, false);
                } else if (p.gsub > 1) {
                    if (ksteps == 4) B2C_ISSUER(4, 1, true, false);
                    else if (ksteps == 2) B2C_ISSUER(2, 1, true, false);
                    else B2C_ISSUER(1, 1, true, false);
                } else {
                    if (ksteps == 4) B2C_ISSUER(4, 1, false, false);
                    else if (ksteps == 2) B2C_ISSUER(2, 1, false, false);
                    else B2C_ISSUER(1, 1, false, false);
                }
#undef B2C_ISSUER
            }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (8 warps)
        const int e = warp - 2;
        if constexpr (KIND == KIND_SPLIT) {   // tiles wider than 128 channels
            epilogue_loop<0>(p, tmem_base, acc_full, acc_empty, &abort_flag, s_stats[e], e, lane, rank);
        } else if constexpr (KIND == KIND_HMERGE) {
            epilogue_loop<2, true>(p, tmem_base, acc_full, acc_empty, &abort_flag, s_stats[e], e, lane, rank);
        } else {
            if (KIND == KIND_GENERAL && p.n_tile <= 32 && !p.out_is_f32)
                epilogue_loop<1>(p, tmem_base, acc_full, acc_empty, &abort_flag, s_stats[e], e, lane, rank);
            else if (p.n_tile <= 64 && !p.out_is_f32)
                epilogue_loop<2>(p, tmem_base, acc_full, acc_empty, &abort_flag, s_stats[e], e, lane, rank);
            else
                epilogue_loop<0>(p, tmem_base, acc_full, acc_empty, &abort_flag, s_stats[e], e, lane, rank);
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();   // both CTAs have left their loops: nothing new will be issued
    if (abort_flag) {
        // A wait gave up.  Before the CTA may exit, let every bulk copy it issued land and every
        // MMA it issued retire (both finish on their own; the polls here only bound the wait).
        // In a pair the leader's barriers count the peer's copies too.
        if ((warp == 0 || warp == kProducerWarp1) && lane == 0 && rank == 0) {
            if (p.resident && warp == 0)
                for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(&w_bar, 0u); ++i) {}
            // the last stage issued into each of the own slots (older ones were consumed, so they had landed)
            const int w = warp == 0 ? 0 : 1;
            for (int sl = w; sl < S; sl += kProducers) {
                if (last_issued < sl) continue;
                const int it = last_issued - ((last_issued - sl) % S);   // largest stage index <= last_issued in slot sl
                for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(&full_bar[sl], (uint32_t)(it / S) & 1u); ++i) {}
            }
        }
        if ((warp == 1 || (warp >= 2 + kEpiWarps && warp < kProducerWarp1)) && lane == 0 && rank == 0) {   // a commit covers the MMAs of the thread that makes it
            if constexpr (PAIR) umma_commit_pair(&drain_bar, (uint16_t)1);
            else umma_commit(&drain_bar);
            if (warp == 1)
                for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(&drain_bar, 0u); ++i) {}
        }
        __syncthreads();
    }
    if constexpr (PAIR) cluster_sync_all();   // the peer must not exit while the leader still drains copies into it
    if (warp == 1) {
        tc_fence_after();
        if constexpr (PAIR) tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
        else tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
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

static int log2_exact(int v)
{
    if (v <= 0 || (v & (v - 1)) != 0) return -1;
    int l = 0;
    while ((1 << l) < v) ++l;
    return l;
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

// A launch plan: the kernel's parameter block (tensor maps included), launch shape and shared-memory size.
struct KMajorPlan {
    ConvKParams p;
    int grid;
    size_t smem_bytes;
};

static b2c_status build_kmajor_plan(b2c_ctx* ctx, const KMajorProblem& pb, KMajorPlan& plan)
{
    ConvKParams& p = plan.p;
    memset(&plan, 0, sizeof(plan));
    const int R = pb.r;
    if (!(R == 1 || R == 3) || !(pb.stride == 1 || pb.stride == 2) || pb.pad != (R - 1) / 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (pb.n < 1 || pb.ic < 16 || pb.ic % 16 || pb.oc < 16 || pb.oc % 16) return B2C_ERR_UNSUPPORTED_SHAPE;
    // tile grid = spatial grid each unit's 128 accumulator rows walk over
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
    p.n_par = n_par;

    // output-channel tile: the largest multiple of 16 up to 256 that splits oc evenly
    int n_tile = 16;
    for (int cand = 256; cand >= 16; cand -= 16)
        if (pb.oc % cand == 0) { n_tile = cand; break; }
    p.n_tile = n_tile;
    p.n_ktiles = pb.oc / n_tile;
    p.acc_cols = ((n_tile + 31) / 32) * 32;
    // four accumulators where TMEM has room: the issuers then run a unit or two ahead of the epilogue
    p.acc_bufs = (4 * p.acc_cols <= 512) ? 4 : 2;
    p.acc_shift = p.acc_bufs == 4 ? 2 : 1;
    p.tmem_cols = 32;
    while (p.tmem_cols < p.acc_bufs * p.acc_cols) p.tmem_cols *= 2;
    p.total_units = n_par * p.tiles_n * p.tiles_h * p.tiles_w * p.n_ktiles;

    // CTA pairs (cta_group::2): two neighbouring pixel tiles share every filter tile, each CTA holding half of its
    // rows, which halves the shared-memory operand traffic per MMA.  Needs an even number of pixel tiles and a channel
    // tile that splits into two multiples of 16; the fp32 / bias / multi-parity cases stay on single CTAs.
    const int m_tiles = p.tiles_n * p.tiles_h * p.tiles_w;
    // Measured on B200 (1024-image layers): pairs gain ~30 % at 128-channel tiles, where the filter traffic from L2
    // bounds single CTAs, and lose 5-30 % at 64 and 256 and on the short reductions of 1x1 and stride-2 layers; so by
    // default only 3x3 stride-1 layers with 128-channel tiles use them (use_pairs: 0 = never, 1 = those, 2 = every
    // eligible problem).
    const bool pair_ok = n_par == 1 && !pb.out_f32 && pb.bias == nullptr && n_tile % 32 == 0 && m_tiles % 2 == 0 && ctx->sm_count >= 2;
    p.pair = (pair_ok && (ctx->use_pairs == 2 || (ctx->use_pairs == 1 && n_tile >= 128 && R == 3 && pb.stride == 1) ||
                          (ctx->use_pairs == 3 && n_tile == 128 && R == 3 && pb.stride == 1))) ? 1 : 0;
    const int b_rows = p.pair ? n_tile / 2 : n_tile;   // filter rows one CTA fetches per tile

    // launch shape: one persistent CTA per SM; the unit walk stride (CTAs, or pairs) is a multiple of n_ktiles so that a
    // CTA keeps its channel tile
    const int walkers_max = p.pair ? ctx->sm_count / 2 : ctx->sm_count;
    const int walk_units = p.pair ? p.total_units / 2 : p.total_units;
    int walkers = walkers_max < walk_units ? walkers_max : walk_units;
    walkers -= walkers % p.n_ktiles;
    if (walkers < p.n_ktiles) walkers = p.n_ktiles;
    const int grid = p.pair ? 2 * walkers : walkers;
    const int units_per_cta = (walk_units + walkers - 1) / walkers;

    // Full-halo plan (3x3, stride 1, 64-channel k-blocks, images of at least 8 x 16 pixels, filter bank resident): tiles
    // of 8 x 16 pixels, one framed box per channel block serves all nine taps, so the input crosses L2 -> SM once
    // (three times with vertical tap reuse, nine without) and a ring slot holds a whole channel block of a unit.
    const bool fh_ok = R == 3 && pb.stride == 1 && n_par == 1 && pb.ic % 64 == 0 && gw >= 8 && gh >= 16 && ctx->use_full_halo &&
                       9 * (pb.ic / 64) * b_rows * 64 * 2 <= (p.pair ? 148 : 96) * 1024;
    // shared-memory plan.  Preference: haloed stages (vertical tap reuse) with 64-channel k-blocks, then with
    // 32-channel k-blocks (smaller stages, so that a ring of at least four still fits), else one tap per stage.
    const int ring_budget = 217 * 1024;   // 227 KB per CTA less the static arrays (8.3 KB) and the alignment slack
    const int kb_natural = (pb.ic % 64 == 0) ? 64 : (pb.ic % 32 == 0) ? 32 : 16;
    const bool can_vreuse = (R == 3 && pb.stride == 1 && p.bn == 1);
    const int taps_total = R * R;
    const int attempts[3][2] = {{kb_natural, 1}, {32, 1}, {kb_natural, 0}};   // (kb, vreuse)
    bool planned = false;
    // Merged horizontal taps (3x3, stride 1, one channel tile of 64, 64-channel k-blocks, image rows of 8 / 16 / 32 pixels that
    // fill a tile with whole rows): per vertical tap and k-step ONE MMA with N = 192 against the three filter columns, so
    // the A operand crosses the shared-memory port once per 192 columns instead of once per 64 (an N = 64 MMA is bound by
    // its operand fetch: 48 cycles for 32 cycles of tensor work).  The stage is the tile with a halo row above and below
    // (vertical taps are row offsets, as with vertical tap reuse); the horizontal shifts are applied to the three column
    // blocks of the accumulator by the epilogue.
    const bool hm_ok = ctx->use_hmerge && !p.pair && R == 3 && pb.stride == 1 && n_par == 1 && n_tile == 64 && pb.oc == 64 && pb.ic % 64 == 0 && !pb.out_f32 &&
                       pb.bias == nullptr && (gw == 8 || gw == 16 || gw == 32) && gh >= 128 / gw && 9 * pb.ic * 64 * 2 <= 148 * 1024;
    if (hm_ok && units_per_cta >= 2) {
        const int bank = 9 * pb.ic * 64 * 2;
        p.bw = gw; p.bh = 128 / gw; p.bn = 1;
        p.tiles_w = 1; p.tiles_h = gh / p.bh; p.tiles_n = pb.n;
        p.total_units = p.tiles_n * p.tiles_h * p.n_ktiles;
        const int a_bytes = (p.bh + 2) * p.bw * 128;   // multiples of 1 KB for every row length used here
        int stages = (ring_budget - bank) / a_bytes;
        if (stages > kMaxStages) stages = kMaxStages;
        if (stages >= 3) {
            p.hm = 1; p.fh = 0; p.vreuse = 0; p.pair = 0;
            p.kb = 64; p.c_blocks = pb.ic / 64; p.swz = SWZ_128B;
            p.nb = 3; p.b_merged = 1;
            p.tx_b = 3 * 64 * 64 * 2; p.b_bytes = p.tx_b;          // one tile = the three filter columns of one filter row: 192 rows of 128 bytes
            p.tx_a = a_bytes; p.a_bytes = a_bytes; p.a_step = p.bw * 128;   // one image row per vertical tap
            p.resident = 1; p.resident_bytes = bank;
            p.stages = stages;
            p.acc_cols = 192; p.acc_bufs = 2; p.acc_shift = 1; p.tmem_cols = 512;
            planned = true;
        }
    }
    if (!planned && fh_ok && units_per_cta >= 2) {
        const int tx_b = b_rows * 64 * 2, bank = taps_total * (pb.ic / 64) * tx_b, a_bytes = ((10 * 18 * 128) + 1023) & ~1023;
        int stages = (ring_budget - bank) / a_bytes;
        if (stages > kMaxStages) stages = kMaxStages;
        if (stages >= (p.pair ? 2 : 3)) {
            p.bw = 8; p.bh = 16; p.bn = 1;
            p.tiles_w = gw / 8; p.tiles_h = gh / 16; p.tiles_n = pb.n;
            p.fh = 1; p.vreuse = 0;
            p.kb = 64; p.c_blocks = pb.ic / 64; p.swz = SWZ_128B;
            p.tx_b = tx_b; p.b_bytes = tx_b; p.b_merged = 1; p.nb = 3;   // bank order [s][cb][r], three filter rows per load
            p.tx_a = 10 * 18 * 128; p.a_bytes = a_bytes; p.a_step = 0;
            p.resident = 1; p.resident_bytes = bank;
            p.stages = stages;
            planned = true;
        }
    }
    for (int a = 0; a < 3 && !planned; ++a) {
        const int kb = attempts[a][0], vr = attempts[a][1];
        if (vr && !can_vreuse) continue;
        if (kb > kb_natural) continue;
        p.kb = kb;
        p.c_blocks = pb.ic / kb;
        p.swz = kb == 64 ? SWZ_128B : kb == 32 ? SWZ_64B : SWZ_32B;
        p.vreuse = vr;
        p.tx_b = b_rows * kb * 2;
        p.b_merged = (vr && p.tx_b % 1024 == 0) ? 1 : 0;   // tiles of one load lie back to back: they must keep the swizzle alignment
        p.b_bytes = (p.tx_b + 1023) & ~1023;
        const int a_rows = vr ? (p.bh + 2) * p.bw : 128;
        p.tx_a = a_rows * kb * 2;
        p.a_bytes = (p.tx_a + 1023) & ~1023;
        p.nb = vr ? 3 : 1;
        p.a_step = vr ? p.bw * kb * 2 : 0;
        // (a pair could keep its half of a 3x3x128x128 bank, 148 KB, resident; measured slower than streaming it: the
        // ring left over is short)
        const int bank_bytes = taps_total * p.c_blocks * p.b_bytes;
        p.resident = (n_par == 1 && bank_bytes <= 96 * 1024 && units_per_cta >= 2) ? 1 : 0;
        p.resident_bytes = p.resident ? bank_bytes : 0;
        const int stage_bytes = p.a_bytes + (p.resident ? 0 : p.nb * p.b_bytes);
        int stages = (ring_budget - p.resident_bytes) / stage_bytes;
        if (stages > kMaxStages) stages = kMaxStages;
        p.stages = stages;
        if (stages >= 4 || !vr) break;
    }
    if (p.stages < 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    p.mma_n = p.hm ? 3 * p.n_tile : p.n_tile;
    // Short k-blocks share a ring slot.  An issuing thread pays 700-900 cycles per slot on top of its MMAs (the slot's stamp,
    // the barrier wait, two commits; measured inside the running kernel), which bounds the stride-2 and 1x1 layers
    // (one k-block = 2-4 MMAs of 48-128 cycles): group k-blocks while a slot holds less than about 1000 tensor-pipe
    // cycles, three slots remain (four where two threads take alternate slots) and the unit has that many k-blocks.
    p.gsub = 1;
    if (ctx->use_group_kblocks && !p.fh && !p.hm && !p.vreuse) {
        // k-blocks of the longest unit (stride-2 data gradient: the parity that takes every other tap in both directions)
        const int max_sub = (n_par > 1 ? ((R + 1) / 2) * ((R + 1) / 2) : taps_total) * p.c_blocks;
        const int per_sub = (p.kb / 16) * (p.mma_n / 2 > 48 ? p.mma_n / 2 : 48);
        const bool split = p.n_tile > 128 && ctx->use_issue_split;   // two threads on alternate slots: an even ring, and four slots so that each keeps two
        int g = 1;
        while (g < 4 && g * per_sub < 1000 && 2 * g <= max_sub) {
            int slots = p.stages / (2 * g);
            if (split) slots &= ~1;
            if (slots < (split ? 4 : 3)) break;
            g *= 2;
        }
        p.gsub = g;
        p.stages /= g;
    }
    // Two issuing threads where one cannot keep the tensor pipe busy: tiles of at most 128 channels.
    p.issuers = p.n_tile <= 128 ? kIssuers : 1;
    // Wider tiles: both threads work on every unit, alternate stages (needs an even ring).
    if (p.n_tile > 128 && ctx->use_issue_split && p.stages >= 2) {
        p.stages &= ~1;
        p.issuers = kIssuers;
        p.issue_split = 1;
    }
    const int stage_bytes = p.gsub * (p.a_bytes + (p.resident ? 0 : p.nb * p.b_bytes));
    const size_t smem_bytes = (size_t)p.resident_bytes + (size_t)p.stages * stage_bytes + 1024;

    // tensor maps
    const int box_h = (p.vreuse || p.fh || p.hm) ? p.bh + 2 : p.bh;
    const int box_w = p.fh ? p.bw + 2 : p.bw;
    if (!pb.dgrad && pb.stride == 2) {
        for (int ph = 0; ph < 2; ++ph)
            for (int pw = 0; pw < 2; ++pw)
                if (!encode_activation_map(ctx, &p.tmA[ph * 2 + pw], pb.in, pb.n, pb.ih, pb.iw, pb.ic, 2, ph, pw, p.kb, box_w, box_h, p.bn))
                    return B2C_ERR_CUDA;
    } else {
        if (!encode_activation_map(ctx, &p.tmA[0], pb.in, pb.n, pb.ih, pb.iw, pb.ic, 1, 0, 0, p.kb, box_w, box_h, p.bn)) return B2C_ERR_CUDA;
    }
    if (p.hm) {
        // weights [out][r][s][in] viewed as (in, out, s, r): a box of all nine taps lands as [r][s][out][in], i.e. per filter row
        // one K-major tile whose 192 rows are the three filter columns of the 64 output channels
        cuuint64_t dims[4] = {(cuuint64_t)pb.ic, (cuuint64_t)pb.oc, (cuuint64_t)R, (cuuint64_t)R};
        cuuint64_t str[3] = {(cuuint64_t)R * R * pb.ic * 2, (cuuint64_t)pb.ic * 2, (cuuint64_t)R * pb.ic * 2};
        cuuint32_t box[4] = {64u, 64u, 3u, 3u};
        if (!encode_map(ctx, &p.tmB, pb.wt, 4, dims, str, box, 128)) return B2C_ERR_CUDA;
    } else {
        // weights [out][r][s][in] viewed as (in, s, out, r): a box of three filter rows lands as three tiles [r][out][in]
        cuuint64_t dims[4] = {(cuuint64_t)pb.ic, (cuuint64_t)R, (cuuint64_t)pb.oc, (cuuint64_t)R};
        cuuint64_t str[3] = {(cuuint64_t)pb.ic * 2, (cuuint64_t)R * R * pb.ic * 2, (cuuint64_t)R * pb.ic * 2};
        cuuint32_t box[4] = {(cuuint32_t)p.kb, 1u, (cuuint32_t)b_rows, p.b_merged ? 3u : 1u};
        if (!encode_map(ctx, &p.tmB, pb.wt, 4, dims, str, box, p.kb * 2)) return B2C_ERR_CUDA;
    }

    // tap tables (row-major over (r, s); with vreuse entry s of row 0 carries the shift of the haloed tile)
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
    p.r_filter = R;
    p.n_valid = pb.n;
    p.oc_valid = pb.oc;
    p.out = pb.out;
    p.out_is_f32 = pb.out_f32 ? 1 : 0;
    p.out_v8 = (reinterpret_cast<uintptr_t>(pb.out) % 32 == 0) ? 1 : 0;   // row pitches are multiples of 32 bytes (16 channels)
    p.bias = pb.bias;
    p.stats = pb.out_f32 ? nullptr : pb.stats;
    p.stats_group_images = pb.stats_group_images;
    p.tw_shift = log2_exact(p.tiles_w);
    p.th_shift = log2_exact(p.tiles_h);
    p.nk_shift = log2_exact(p.n_ktiles);
    p.grp_shift = log2_exact(p.stats_group_images);
    p.cb_shift = log2_exact(p.c_blocks);
    if (p.stats && p.stats_group_images > 0 && (p.stats_group_images % p.bn) != 0) return B2C_ERR_UNSUPPORTED_SHAPE;  // a tile must not straddle groups
    plan.grid = grid;
    plan.smem_bytes = smem_bytes;
    return B2C_OK;
}

// Appends the bytes of a value to a cache key.
template <typename T>
static inline void key_add(std::string& key, const T& v)
{
    key.append(reinterpret_cast<const char*>(&v), sizeof(T));
}

b2c_status launch_conv_kmajor(b2c_ctx* ctx, const KMajorProblem& pb, cudaStream_t stream)
{
    // plans are keyed by everything the planner reads: the problem and the context's switches
    std::string key("K");
    key_add(key, pb.n); key_add(key, pb.ih); key_add(key, pb.iw); key_add(key, pb.ic); key_add(key, pb.oh); key_add(key, pb.ow); key_add(key, pb.oc);
    key_add(key, pb.r); key_add(key, pb.stride); key_add(key, pb.pad); key_add(key, pb.dgrad); key_add(key, pb.in); key_add(key, pb.wt);
    key_add(key, pb.out); key_add(key, pb.out_f32); key_add(key, pb.bias); key_add(key, pb.stats); key_add(key, pb.stats_group_images);
    key_add(key, ctx->use_pairs); key_add(key, ctx->use_full_halo); key_add(key, ctx->use_issue_split); key_add(key, ctx->use_hmerge); key_add(key, ctx->use_group_kblocks);
    auto it = ctx->plan_cache.find(key);
    if (it == ctx->plan_cache.end()) {
        KMajorPlan fresh;
        b2c_status st = build_kmajor_plan(ctx, pb, fresh);
        if (st != B2C_OK) return st;
        if (ctx->plan_cache.size() >= 8192) ctx->plan_cache.clear();   // callers that pass new buffers every call: keep the table bounded
        std::vector<unsigned char> bytes(sizeof(KMajorPlan));
        memcpy(bytes.data(), &fresh, sizeof(KMajorPlan));
        it = ctx->plan_cache.emplace(std::move(key), std::move(bytes)).first;
    }
    KMajorPlan plan;   // a copy: the 64-byte alignment of the tensor maps is the parameter block's, not the table's
    memcpy(&plan, it->second.data(), sizeof(KMajorPlan));
    ConvKParams& p = plan.p;
    const int grid = plan.grid;
    const size_t smem_bytes = plan.smem_bytes;
    p.status = ctx->d_status;
    p.spin_limit = ctx->spin_limit;
    p.stall = ctx->stall_counters;

    // the kernel kind of the plan (merged taps run on single CTAs only)
    typedef void (*kernel_t)(const ConvKParams);
    static const kernel_t kernels[2][4] = {
        {conv_kmajor_kernel<false, KIND_GENERAL>, conv_kmajor_kernel<false, KIND_SPLIT>, conv_kmajor_kernel<false, KIND_HMERGE>, conv_kmajor_kernel<false, KIND_FULL_HALO>},
        {conv_kmajor_kernel<true, KIND_GENERAL>, conv_kmajor_kernel<true, KIND_SPLIT>, nullptr, conv_kmajor_kernel<true, KIND_FULL_HALO>}};
    const int kind = p.hm ? KIND_HMERGE : p.fh ? KIND_FULL_HALO : p.issue_split ? KIND_SPLIT : KIND_GENERAL;
    const kernel_t kernel = kernels[p.pair ? 1 : 0][kind];
    if (kernel == nullptr) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!(ctx->smem_optin_done & B2C_OPTIN_KMAJOR)) {   // the attribute belongs to the device: kept per context, not per process
        for (int a = 0; a < 2; ++a)
            for (int b = 0; b < 4; ++b)
                if (kernels[a][b] != nullptr) B2C_CUDA(cudaFuncSetAttribute(kernels[a][b], cudaFuncAttributeMaxDynamicSharedMemorySize, 218 * 1024));
        ctx->smem_optin_done |= B2C_OPTIN_KMAJOR;
    }
    B2C_CUDA(b2c_launch(ctx, kernel, dim3((unsigned)grid), dim3(kThreads), smem_bytes, stream, p.pair ? 2u : 1u, p));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

}  // namespace b2c
