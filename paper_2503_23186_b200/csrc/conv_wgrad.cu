// Weight gradient as an implicit GEMM on tcgen05 with both operands MN-major:
//
//   dw[k, tap, c] += sum over pixels  dy[pixel, k] * x[pixel shifted by tap, c]
//
// GEMM M = 128 output channels (k), N = input channels (c) of one or more taps, reduction = pixels.
// Both dy and x are stored pixel-major with channels contiguous, i.e. the reduction index is the
// slow one: TMA boxes of (cw channels, pb pixels) land in shared memory exactly in the swizzled
// MN-major canonical layout (rows = pixels, cw*2 = 32/64/128 bytes per row).  One CTA owns a
// (k-tile, c-tile, tap group) and a range of pixel chunks; a stage holds one chunk: the dy boxes
// and, per x shift of the group, the x boxes gathered at that shift (zero-filled outside the image by
// TMA).  The x boxes of consecutive shifts are adjacent, so one MMA covers several taps (N up to 256).
//
// Layers with 64 output channels would leave half of M = 128 empty.  There two copies of dy, the
// second gathered one row higher, are stacked on M: with x gathered at (r0 - pad, s - pad) the rows of
// copy a accumulate tap (r0 + a, s), since sum_p dy[p - (a,0)] x[p + t] = sum_p dy[p] x[p + t + (a,0)].
// Partial sums of the pixel ranges are added to dw with vector fp32 reductions.
//
// Framed x stages (3x3, stride 1, image rows of at least 8 pixels, 64-channel x boxes): instead of one x box per
// horizontal shift, a stage holds each 64-channel block of the chunk once, with one extra pixel left and right of every
// image row (box of bw + 2 pixels).  The operand of shift s is the same box read from a start address s pixel rows
// (s x 128 bytes) further in: the k-step of 16 pixels starts at row h * (bw + 2) + w0 + s, and the three shifts are the
// three 64-column blocks of one N = 192 MMA whose block stride (LBO) is one pixel row.  The 128-byte swizzle is keyed on
// absolute shared-memory address bits, so a start that is not a multiple of the 8-row atom reads the right data
// (the parity tests cover it).  The x tensor crosses L2 -> SM once per filter row instead of three times.
#include "common.h"
#include "ptx.cuh"

namespace b2c {

struct WgGroup {
    int nb;                        // x shifts of the group (column blocks of ct channels)
    int8_t map[3], dh[3], dw[3];   // tensor map (parity view) and pixel offset of each shift
    int8_t rs[2][3];               // filter tap accumulated by (dy copy, shift); -1: not used
};

struct alignas(64) WgradParams {
    CUtensorMap tmDy;
    CUtensorMap tmX[4];
    WgGroup groups[3];
    int n_groups;
    int stack;                         // two dy copies stacked on M (64 output channels)
    int bw, bh, bn, tiles_w, tiles_h;  // pixel chunk box and chunk grid (tiles_h covers one extra row when stacked)
    int pb;                            // pixels per chunk
    int cw_a, swz_a, cw_b, swz_b;      // channels per box (= one swizzle row) and descriptor swizzle code: dy, x
    int ct;                            // x channels per CTA
    int n_ktiles, n_ctiles, n_splits;
    int chunks_total;
    int stages, tmem_cols;
    int box_a, box_b, a_boxes, b_boxes;   // bytes per dy / x box; dy boxes per stage; x boxes per shift
    int a_bytes, a_lbo;                   // dy bytes per stage; byte distance between the two 64-row halves of the A operand
    int tw_shift;                         // log2(tiles_w)
    int stage_bytes;                      // bytes of a ring slot = gsub chunks
    int gsub, sub_bytes;                  // pixel chunks that share a ring slot, one barrier wait and one commit; bytes of one chunk's operands
    int n_pieces, piece_t0[3], piece_nt[3];   // MMAs per k-step: first shift and number of shifts each covers
    int fx;                               // framed x stages: one box of (bw + 2) x bh pixels per 64-channel block serves the three shifts
    int fx_box, fx_tx;                    // shared-memory footprint (1 KB multiple) and bytes delivered per framed box
    uint32_t fx_koff[4];                  // start of k-step kk inside a framed box, in 16-byte units
    uint32_t fx_sbo;                      // byte distance between the two 8-pixel groups of a k-step
    int issuers;                          // MMA-issuing threads at work: 2 with an even ring depth, else 1
    int k_total, c_total, rs_total;
    float* dw;
    unsigned* status;
    unsigned spin_limit;
    unsigned long long* stall;            // optional [8]: wait and lifetime cycles of the roles (see b2c_set_stall_counters)
};

static constexpr int kWgStages = 6;
static constexpr int kWgProducers = 3;   // warp 0 and the warps after the epilogue warps; producer w fills ring slots w, w + 3, ...
static constexpr int kWgProducerWarp1 = 6;
static constexpr int kWgThreads = 256;
// MMA-issuing threads (lane 0 of warps 1 and 2).  They take alternate chunks and accumulate into the same TMEM tile: one
// thread pays about 100 cycles per MMA with a wait and a commit every four, against 96 the pipe needs at N = 192.  The
// second thread starts once the first chunk (the one that overwrites instead of accumulating) has completed.  The ring
// depth is even, so a slot always returns to the same thread and its barrier phases stay unambiguous.
static constexpr int kWgIssuers = 2;
static constexpr uint32_t kWgDrainPolls = 1u << 22;

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// One MMA per k-step of 16 pixels, unrolled: descriptors differ only in their low (address) word.
// Framed x: the B operand of k-step kk starts at its own row offset inside the framed box.
template <int KS>
__device__ __forceinline__ void wg_issue_framed(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_hi, uint32_t b_hi, uint32_t idesc,
                                                uint32_t kstep_a, uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3, uint32_t accumulate_first)
{
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
        const uint32_t koff = kk == 0 ? k0 : kk == 1 ? k1 : kk == 2 ? k2 : k3;
        const uint64_t ad = ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + (uint32_t)kk * kstep_a);
        const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + koff);
        umma_bf16(d_tmem, ad, bd, idesc, kk == 0 ? accumulate_first : 1u);
    }
}
template <int KS>
__device__ __forceinline__ void wg_issue(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_hi, uint32_t b_hi, uint32_t idesc,
                                         uint32_t kstep_a, uint32_t kstep_b, uint32_t accumulate_first)
{
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
        const uint64_t ad = ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + (uint32_t)kk * kstep_a);
        const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + (uint32_t)kk * kstep_b);
        umma_bf16(d_tmem, ad, bd, idesc, kk == 0 ? accumulate_first : 1u);
    }
}

__global__ void __launch_bounds__(kWgThreads, 1) conv_wgrad_kernel(const __grid_constant__ WgradParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kWgStages], empty_bar[kWgStages], accum_bar, drain_bar, init_bar;
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
    const int gi = t % p.n_groups;
    const int split = t / p.n_groups;
    const WgGroup& grp = p.groups[gi];
    const int chunk_begin = (int)((long long)p.chunks_total * split / p.n_splits);
    const int chunk_end = (int)((long long)p.chunks_total * (split + 1) / p.n_splits);
    const int n_chunks = chunk_end - chunk_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&accum_bar, (uint32_t)p.issuers);   // one commit per MMA-issuing thread
        mbar_init(&drain_bar, (uint32_t)p.issuers);
        mbar_init(&init_bar, 1);
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
    // set-up done (it touched no global data): order behind the previous kernel of the stream, then let the next one in
    pdl_wait();
    pdl_launch_dependents();
    const long long t_kernel = clock64();
    int last_issued = -1;  // producer lanes: last chunk whose loads this lane issued

    if (warp == 0 || warp >= kWgProducerWarp1) {
        const int w = warp == 0 ? 0 : warp - kWgProducerWarp1 + 1;
        if (lane == 0 && w < S) {
            // Producer w fills the ring slots w, w + kWgProducers, ...: one thread's wait -> expect -> issue chain is
            // longer than the MMAs of a stage take.  Each slot keeps one producer, which uses it strictly in order.
            prefetch_tensormap(&p.tmDy);
            prefetch_tensormap(&p.tmX[0]);
            const uint32_t tx = p.fx ? (uint32_t)(p.a_bytes + p.b_boxes * p.fx_tx) : (uint32_t)(p.a_bytes + grp.nb * p.b_boxes * p.box_b);
            int it = w, s = w;   // it counts ring slots; a slot holds G consecutive chunks (the last one of the CTA possibly fewer)
            uint32_t ph = 0u;
            const bool timed = p.stall != nullptr && w == 0;
            long long waited = 0;
            const int G = p.gsub, n_slots = (n_chunks + G - 1) / G;
            while (it < n_slots) {
                const long long w0 = timed ? clock64() : 0;
                if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, p.spin_limit, &abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    break;
                }
                if (timed) waited += clock64() - w0;
                const int n_g = n_chunks - it * G < G ? n_chunks - it * G : G;
                mbar_expect_tx(&full_bar[s], (uint32_t)n_g * tx);
                for (int g = 0; g < n_g; ++g) {
                int ch = chunk_begin + it * G + g;
                const int ow0 = (ch & (p.tiles_w - 1)) * p.bw;
                ch >>= p.tw_shift;
                const int th = ch / p.tiles_h;
                const int oh0 = (ch - th * p.tiles_h) * p.bh;
                const int n0 = th * p.bn;
                uint8_t* dst = smem + (size_t)s * p.stage_bytes + (size_t)g * p.sub_bytes;
                if (p.stack) {
                    // one box with a halo row on top: copy 1 of dy (gathered one row higher) is its first pb pixels,
                    // copy 0 starts one image row further down
                    tma_load_4d(dst, &p.tmDy, &full_bar[s], 0, ow0, oh0 - 1, n0);
                } else {
                    for (int j = 0; j < p.a_boxes; ++j)  // boxes past the last channel are zero-filled
                        tma_load_4d(dst + (size_t)j * p.box_a, &p.tmDy, &full_bar[s], ktile * 128 + j * p.cw_a, ow0, oh0, n0);
                }
                dst += p.a_bytes;
                if (p.fx) {   // one framed box per channel block, gathered at the first shift (one pixel to the left)
                    for (int j = 0; j < p.b_boxes; ++j)
                        tma_load_4d(dst + (size_t)j * p.fx_box, &p.tmX[grp.map[0]], &full_bar[s], ctile * p.ct + j * p.cw_b, ow0 + grp.dw[0],
                                    oh0 + grp.dh[0], n0);
                } else
                for (int b = 0; b < grp.nb; ++b)
                    for (int j = 0; j < p.b_boxes; ++j)
                        tma_load_4d(dst + (size_t)(b * p.b_boxes + j) * p.box_b, &p.tmX[grp.map[b]], &full_bar[s], ctile * p.ct + j * p.cw_b,
                                    ow0 + grp.dw[b], oh0 + grp.dh[b], n0);
                }
                last_issued = it;
                if (s + kWgProducers < S) {
                    it += kWgProducers;
                    s += kWgProducers;
                } else {   // wrap to this producer's first slot
                    it += S - s + w;
                    s = w;
                    ph ^= 1u;
                }
            }
            if (timed) atomicAdd(p.stall + 0, (unsigned long long)waited);
        }
    } else if (warp == 1 || warp == 2) {
        if (lane == 0 && warp - 1 < p.issuers) {
            const int my = warp - 1;
            // SBO = eight pixel rows, LBO = next block of cw channels (the next box)
            const uint64_t proto_a = make_smem_desc(0u, (uint32_t)p.a_lbo, 16u * (uint32_t)p.cw_a, (uint32_t)p.swz_a);
            // framed x: the column blocks of an MMA are the three shifts, one pixel row (cw_b channels) apart
            const uint64_t proto_b = p.fx ? make_smem_desc(0u, 2u * (uint32_t)p.cw_b, p.fx_sbo, (uint32_t)p.swz_b)
                                          : make_smem_desc(0u, (uint32_t)p.box_b, 16u * (uint32_t)p.cw_b, (uint32_t)p.swz_b);
            const uint32_t a_hi = (uint32_t)(proto_a >> 32), a_lo_base = (uint32_t)proto_a;
            const uint32_t b_hi = (uint32_t)(proto_b >> 32), b_lo_base = (uint32_t)proto_b;
            const uint32_t kstep_a = (uint32_t)(16 * p.cw_a * 2) >> 4, kstep_b = (uint32_t)(16 * p.cw_b * 2) >> 4;   // 16 pixel rows
            const int ksteps = p.pb >> 4;
            // up to three MMAs per k-step (kept in scalars: the issuing thread must not index local memory)
            uint32_t idesc0 = 0, idesc1 = 0, idesc2 = 0, boff0 = 0, boff1 = 0, boff2 = 0, dcol0 = 0, dcol1 = 0, dcol2 = 0;
            int n_pieces = 0;
            for (int i = 0; i < p.n_pieces; ++i) {
                if (p.piece_t0[i] >= grp.nb) break;
                const int nt = min(p.piece_nt[i], grp.nb - p.piece_t0[i]);
                const uint32_t id = make_idesc_bf16(128, nt * p.ct, true, true);
                const uint32_t bo = (uint32_t)(p.a_bytes + p.piece_t0[i] * p.b_boxes * p.box_b) >> 4;
                const uint32_t dc = (uint32_t)(p.piece_t0[i] * p.ct);
                if (i == 0) { idesc0 = id; boff0 = bo; dcol0 = dc; }
                else if (i == 1) { idesc1 = id; boff1 = bo; dcol1 = dc; }
                else { idesc2 = id; boff2 = bo; dcol2 = dc; }
                ++n_pieces;
            }
            bool ok = true;
            const bool timed = p.stall != nullptr;
            const long long t_begin = timed ? clock64() : 0;
            long long waited = 0, issuing = 0;
            const int G = p.gsub, n_slots = (n_chunks + G - 1) / G;
            const uint32_t sub16 = (uint32_t)p.sub_bytes >> 4;
            if (my != 0 && n_slots > 1 && !mbar_wait_bounded(&init_bar, 0u, p.spin_limit, &abort_flag)) {   // slot 0 has initialised the accumulator
                atomicOr(p.status, B2C_DEV_TIMEOUT);
                ok = false;
            }
            if (my != 0) tc_fence_after();
            // (this thread's chain of dependent instructions per slot bounds chunks with few MMAs: nothing is recomputed in the loop)
            const bool fx = p.fx != 0;
            const int n_issuers = p.issuers, b_boxes = p.b_boxes;
            const uint32_t id_fx = make_idesc_bf16(128, 3 * p.cw_b, true, true);
            const uint32_t fx_b_first = (uint32_t)p.a_bytes >> 4, fx_b_next = (uint32_t)p.fx_box >> 4, fx_d_next = 3u * (uint32_t)p.cw_b;
            const uint32_t fk0 = p.fx_koff[0], fk1 = p.fx_koff[1], fk2 = p.fx_koff[2], fk3 = p.fx_koff[3];
            const uint32_t stage16 = (uint32_t)p.stage_bytes >> 4, smem16 = smem_u32(smem) >> 4;
            int s = my;            // S is even with two threads: a thread's slots are my, my + 2, ...
            uint32_t ph = 0u;
            for (int it = my; ok && it < n_slots; it += n_issuers) {
                const long long w0 = timed ? clock64() : 0;
                if (!mbar_wait_bounded(&full_bar[s], ph, p.spin_limit, &abort_flag)) {
                    atomicOr(p.status, B2C_DEV_TIMEOUT);
                    ok = false;
                    break;
                }
                const long long w1 = timed ? clock64() : 0;
                waited += w1 - w0;
                tc_fence_after();
                const uint32_t st16 = smem16 + (uint32_t)s * stage16;
                const int n_g = n_chunks - it * G < G ? n_chunks - it * G : G;
                for (int g = 0; g < n_g; ++g) {
                const uint32_t a_lo = a_lo_base + st16 + (uint32_t)g * sub16, b_lo = b_lo_base + st16 + (uint32_t)g * sub16;
                const uint32_t acc0 = (it | g) != 0 ? 1u : 0u;
                if (fx) {   // chunks of 64 pixels: four k-steps; one MMA per channel block, N = three shifts x cw_b channels
                    const uint32_t b_first = b_lo + fx_b_first;
                    for (int i = 0; i < b_boxes; ++i)
                        wg_issue_framed<4>(tmem_base + (uint32_t)i * fx_d_next, a_lo, b_first + (uint32_t)i * fx_b_next, a_hi, b_hi, id_fx, kstep_a, fk0, fk1, fk2,
                                           fk3, acc0);
                } else if (ksteps == 4) {
                    wg_issue<4>(tmem_base + dcol0, a_lo, b_lo + boff0, a_hi, b_hi, idesc0, kstep_a, kstep_b, acc0);
                    if (n_pieces > 1) wg_issue<4>(tmem_base + dcol1, a_lo, b_lo + boff1, a_hi, b_hi, idesc1, kstep_a, kstep_b, acc0);
                    if (n_pieces > 2) wg_issue<4>(tmem_base + dcol2, a_lo, b_lo + boff2, a_hi, b_hi, idesc2, kstep_a, kstep_b, acc0);
                } else {
                    wg_issue<2>(tmem_base + dcol0, a_lo, b_lo + boff0, a_hi, b_hi, idesc0, kstep_a, kstep_b, acc0);
                    if (n_pieces > 1) wg_issue<2>(tmem_base + dcol1, a_lo, b_lo + boff1, a_hi, b_hi, idesc1, kstep_a, kstep_b, acc0);
                    if (n_pieces > 2) wg_issue<2>(tmem_base + dcol2, a_lo, b_lo + boff2, a_hi, b_hi, idesc2, kstep_a, kstep_b, acc0);
                }
                }
                umma_commit(&empty_bar[s]);
                if (it == 0) umma_commit(&init_bar);
                if (timed) issuing += clock64() - w1;
                s += n_issuers;
                if (s >= S) { s -= S; ph ^= 1u; }
            }
            if (ok && n_chunks > 0) umma_commit(&accum_bar);
            if (timed && my == 0) {
                atomicAdd(p.stall + 1, (unsigned long long)waited);
                atomicAdd(p.stall + 4, (unsigned long long)(clock64() - t_begin));
                atomicAdd(p.stall + 6, (unsigned long long)issuing);
            }
        }
    }
    // ------------------------------------------------------------------ epilogue: all eight warps
    // The producer and MMA warps have nothing left to do once their loops end, so they help the four epilogue warps:
    // two warps per TMEM lane quarter, each sending half of the channel chunks of every shift to dw.
    {
        const int q = warp & 3, part = warp >> 2;
        const int m = q * 32 + lane;
        const int copy = p.stack ? 1 - (m >> 6) : 0;                   // which dy copy this accumulator row belongs to (copy 1 comes first)
        const int k = p.stack ? (m & 63) : ktile * 128 + m;
        __syncwarp();
        bool ok = n_chunks > 0;
        if (ok) {
            if (lane == 0) ok = mbar_wait_bounded(&accum_bar, 0u, p.spin_limit, &abort_flag);   // one poller per warp
            ok = __all_sync(0xffffffffu, ok);
            if (!ok && lane == 0) atomicOr(p.status, B2C_DEV_TIMEOUT);
            tc_fence_after();
        }
        if (ok) {
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
            const int n_ck = p.ct >> 4;
            const int ck_begin = part == 0 ? 0 : (n_ck + 1) >> 1, ck_end = part == 0 ? (n_ck + 1) >> 1 : n_ck;   // this warp's chunks
            for (int b = 0; b < grp.nb && ck_begin < ck_end; ++b) {
                const int rs = grp.rs[copy][b];
                const bool live = rs >= 0 && k < p.k_total;
                float* dst_row = p.dw + ((long long)(live ? k : 0) * p.rs_total + (live ? rs : 0)) * p.c_total + ctile * p.ct;
                // accumulator column of 16-channel chunk ck of shift b (framed x: [channel block][shift][64 channels])
                auto col = [&](int ck) -> uint32_t {
                    const int per_block = p.cw_b >> 4;   // 16-channel chunks per x box
                    return p.fx ? (uint32_t)((ck / per_block) * 3 * p.cw_b + b * p.cw_b + (ck % per_block) * 16) : (uint32_t)(b * p.ct + ck * 16);
                };
                auto send = [&](const uint32_t (&r)[16], int ck) {
                    if (live) {
#pragma unroll
                        for (int i = 0; i < 16; i += 4)
                            red_add_v4(dst_row + ck * 16 + i, __uint_as_float(r[i]), __uint_as_float(r[i + 1]), __uint_as_float(r[i + 2]),
                                       __uint_as_float(r[i + 3]));
                    }
                };
                // two chunks in flight: the next one is fetched while the current one is sent out
                uint32_t ra[16], rb[16];
                tmem_ld16(t_row + col(ck_begin), ra);
                tmem_ld_wait();
                for (int ck = ck_begin; ck < ck_end; ck += 2) {
                    if (ck + 1 < ck_end) tmem_ld16(t_row + col(ck + 1), rb);
                    send(ra, ck);
                    if (ck + 1 < ck_end) {
                        tmem_ld_wait();
                        if (ck + 2 < ck_end) tmem_ld16(t_row + col(ck + 2), ra);
                        send(rb, ck + 1);
                        if (ck + 2 < ck_end) tmem_ld_wait();
                    }
                }
            }
        }
        if (p.stall != nullptr && lane == 0) atomicMax(p.stall + 7, (unsigned long long)(clock64() - t_kernel));   // the slowest warp of the slowest CTA
        if (p.stall != nullptr && warp == 2 && lane == 0) atomicAdd(p.stall + 5, (unsigned long long)(clock64() - t_kernel));
    }
    tc_fence_before();
    __syncthreads();
    if (abort_flag) {
        // A wait gave up: let the issued bulk copies land and the issued MMAs retire before exit.
        if ((warp == 0 || warp >= kWgProducerWarp1) && lane == 0) {
            const int w = warp == 0 ? 0 : warp - kWgProducerWarp1 + 1;
            for (int sl = w; sl < S; sl += kWgProducers) {   // the last chunk issued into each of the own slots
                if (last_issued < sl) continue;
                const int it = last_issued - ((last_issued - sl) % S);
                for (uint32_t i = 0; i < kWgDrainPolls && !mbar_try_wait(&full_bar[sl], (uint32_t)(it / S) & 1u); ++i) {}
            }
        }
        if ((warp == 1 || warp == 2) && lane == 0 && warp - 1 < p.issuers) {   // a commit covers the MMAs of the thread that makes it
            umma_commit(&drain_bar);
            if (warp == 1)
                for (uint32_t i = 0; i < kWgDrainPolls && !mbar_try_wait(&drain_bar, 0u); ++i) {}
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

struct WgradPlan {
    WgradParams p;
    int grid;
    size_t smem_bytes;
};

static b2c_status build_wgrad_plan(b2c_ctx* ctx, const WgradProblem& pb, WgradPlan& plan)
{
    WgradParams& p = plan.p;
    memset(&plan, 0, sizeof(plan));
    const int R = pb.r;
    if (!(R == 1 || R == 3) || !(pb.stride == 1 || pb.stride == 2) || pb.pad != (R - 1) / 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (pb.n < 1 || pb.c < 16 || pb.c % 16 || pb.k < 16 || pb.k % 16) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (pb.h != pb.p * pb.stride || pb.w != pb.q * pb.stride) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_is_pow2(pb.p) || !b2c_is_pow2(pb.q) || pb.p > 128 || pb.q > 128) return B2C_ERR_UNSUPPORTED_SHAPE;
    if (!b2c_aligned16(pb.dy) || !b2c_aligned16(pb.x) || !b2c_aligned16(pb.dw)) return B2C_ERR_MISALIGNED;

    // channels per box = one swizzle row, chosen per tensor
    p.cw_a = (pb.k % 64 == 0) ? 64 : (pb.k % 32 == 0) ? 32 : 16;
    p.cw_b = (pb.c % 64 == 0) ? 64 : (pb.c % 32 == 0) ? 32 : 16;
    p.swz_a = p.cw_a == 64 ? SWZ_128B : p.cw_a == 32 ? SWZ_64B : SWZ_32B;
    p.swz_b = p.cw_b == 64 ? SWZ_128B : p.cw_b == 32 ? SWZ_64B : SWZ_32B;
    // stacking needs chunks that stay inside one image (at least 64 pixels per image)
    p.stack = (R == 3 && pb.stride == 1 && pb.k == 64 && pb.p * pb.q >= 64 && pb.q >= 8) ? 1 : 0;   // q >= 8: the second copy starts on a swizzle-atom boundary
    // x-channel tile: largest divisor of c that is a multiple of cw_b, at most 160 (three shifts fit 512 TMEM columns)
    p.ct = p.cw_b;
    for (int cand = 160; cand >= p.cw_b; cand -= 16)
        if (pb.c % cand == 0 && cand % p.cw_b == 0) { p.ct = cand; break; }
    // framed x stages: 64 pixels of one image per chunk, 64-channel x boxes, at most two of them per CTA (2 x 192 TMEM columns)
    p.fx = (R == 3 && pb.stride == 1 && pb.q >= 8 && pb.p * pb.q >= 64 && p.cw_b >= 32 && ctx->use_wgrad_frame) ? 1 : 0;
    if (p.fx) {   // as many boxes per CTA as TMEM holds (three shifts of cw_b columns each): 2 of 64 channels, up to 5 of 32
        const int max_boxes = 512 / (3 * p.cw_b);
        p.ct = p.cw_b;
        for (int nb = max_boxes; nb >= 1; --nb)
            if (pb.c % (nb * p.cw_b) == 0) { p.ct = nb * p.cw_b; break; }
    }
    p.n_ctiles = pb.c / p.ct;
    p.n_ktiles = p.stack ? 1 : (pb.k + 127) / 128;
    p.a_boxes = p.stack ? 2 : 128 / p.cw_a;
    p.b_boxes = p.ct / p.cw_b;
    const int shifts = R == 3 ? 3 : 1;
    p.tmem_cols = 32;
    while (p.tmem_cols < (p.fx ? p.b_boxes * 3 * p.cw_b : shifts * p.ct)) p.tmem_cols *= 2;
    if (p.tmem_cols > 512) return B2C_ERR_UNSUPPORTED_SHAPE;
    // MMAs per k-step: merge the column blocks of consecutive shifts while N stays within 256
    if (p.fx) {
        p.n_pieces = 0;   // framed x: one MMA per x box, laid out by the kernel
    } else if (shifts * p.ct <= 256) {
        p.n_pieces = 1; p.piece_t0[0] = 0; p.piece_nt[0] = shifts;
    } else if (2 * p.ct <= 256) {
        p.n_pieces = 2; p.piece_t0[0] = 0; p.piece_nt[0] = 2; p.piece_t0[1] = 2; p.piece_nt[1] = 1;
    } else {
        p.n_pieces = shifts;
        for (int i = 0; i < shifts; ++i) { p.piece_t0[i] = i; p.piece_nt[i] = 1; }
    }

    // tap groups
    TapList fw;
    forward_taps(fw, R, pb.stride, pb.pad);
    if (R == 1) {
        p.n_groups = 1;
        WgGroup& g = p.groups[0];
        g.nb = 1; g.map[0] = fw.map[0]; g.dh[0] = fw.dh[0]; g.dw[0] = fw.dw[0];
        g.rs[0][0] = 0; g.rs[1][0] = -1;
    } else if (!p.stack) {
        p.n_groups = 3;   // one group per filter row
        for (int r = 0; r < 3; ++r) {
            WgGroup& g = p.groups[r];
            g.nb = 3;
            for (int s = 0; s < 3; ++s) {
                g.map[s] = fw.map[r * 3 + s]; g.dh[s] = fw.dh[r * 3 + s]; g.dw[s] = fw.dw[r * 3 + s];
                g.rs[0][s] = (int8_t)(r * 3 + s); g.rs[1][s] = -1;
            }
        }
    } else {
        p.n_groups = 2;   // rows {0,1} and {1,2}; the second group's copy 0 repeats row 1 and is dropped
        for (int gi = 0; gi < 2; ++gi) {
            WgGroup& g = p.groups[gi];
            const int r0 = gi;   // x is gathered at filter row r0; dy copy a lands on row r0 + a
            g.nb = 3;
            for (int s = 0; s < 3; ++s) {
                g.map[s] = fw.map[r0 * 3 + s]; g.dh[s] = fw.dh[r0 * 3 + s]; g.dw[s] = fw.dw[r0 * 3 + s];
                g.rs[0][s] = gi == 0 ? (int8_t)(r0 * 3 + s) : (int8_t)-1;
                g.rs[1][s] = (int8_t)((r0 + 1) * 3 + s);
            }
        }
    }

    // pixel chunk: 64 pixels, or 32 when a 64-pixel stage would not leave room for three stages
    p.pb = 64;
    for (;;) {
        p.box_a = p.pb * p.cw_a * 2;
        p.box_b = p.pb * p.cw_b * 2;
        p.a_bytes = p.stack ? (p.pb + (pb.q < p.pb ? pb.q : p.pb)) * p.cw_a * 2 : p.a_boxes * p.box_a;   // stacked: one box with a halo row
        p.stage_bytes = p.a_bytes + shifts * p.b_boxes * p.box_b;
        if (p.fx) {
            const int bw = pb.q < p.pb ? pb.q : p.pb, bh = p.pb / bw;
            p.fx_tx = (bw + 2) * bh * p.cw_b * 2;
            p.fx_box = (p.fx_tx + 1023) & ~1023;
            p.stage_bytes = p.a_bytes + p.b_boxes * p.fx_box;
        }
        if (p.stage_bytes * 3 <= 200 * 1024 || p.pb == 32) break;
        p.pb = 32;
    }
    if (p.fx && p.pb != 64) return B2C_ERR_UNSUPPORTED_SHAPE;   // cannot happen: a framed stage is under 40 KB
    // Chunks with few MMAs share a ring slot (an issuing thread pays 700-900 cycles per slot for the barrier wait and the
    // commits on top of its MMAs): two chunks per slot where one holds under half of that in tensor-pipe cycles and four
    // slots remain.
    p.sub_bytes = p.stage_bytes;
    p.gsub = 1;
    {
        const int total_cols = p.fx ? p.b_boxes * 3 * p.cw_b : shifts * p.ct;
        const int per_chunk = (p.pb / 16) * (total_cols / 2);
        if (ctx->use_group_kblocks && per_chunk < 500 && ((216 * 1024) / p.sub_bytes) / 2 >= 4) p.gsub = 2;
    }
    p.stage_bytes = p.gsub * p.sub_bytes;
    int stages = ((p.gsub > 1 ? 216 : 200) * 1024) / p.stage_bytes;
    if (stages > kWgStages) stages = kWgStages;
    if (stages < 2) return B2C_ERR_UNSUPPORTED_SHAPE;
    // Two issuing threads need an even ring.  Measured: four stages with two threads beat five with one (128 -> 128:
    // 67 us against 79 us), three stages with one thread beat two with two (512 -> 512 at 4x4: 79 us against 106 us).
    if (stages >= 4) stages &= ~1;
    p.issuers = (stages % 2 == 0 && ctx->use_wgrad_two_issuers) ? kWgIssuers : 1;
    p.stages = stages;
    p.bw = pb.q < p.pb ? pb.q : p.pb;
    p.bh = (p.pb / p.bw) < pb.p ? (p.pb / p.bw) : pb.p;
    p.bn = p.pb / (p.bw * p.bh);
    if (p.stack && p.bn != 1) return B2C_ERR_UNSUPPORTED_SHAPE;   // cannot happen: 64 pixels per image guarantee bn == 1
    if (p.fx) {
        if (p.bn != 1) return B2C_ERR_UNSUPPORTED_SHAPE;   // cannot happen: at least 64 pixels per image
        for (int kk = 0; kk < 4; ++kk) {
            const int pix = 16 * kk, h = pix / p.bw, w0 = pix % p.bw;   // bw == 8: a k-step covers image rows 2kk and 2kk + 1
            p.fx_koff[kk] = (uint32_t)((h * (p.bw + 2) + w0) * p.cw_b * 2) >> 4;
        }
        p.fx_sbo = (uint32_t)((p.bw == 8 ? 10 : 8) * p.cw_b * 2);   // eight pixel rows, or one framed image row of ten
    }
    p.tiles_w = pb.q / p.bw;
    p.tw_shift = 0;
    while ((1 << p.tw_shift) < p.tiles_w) ++p.tw_shift;
    p.a_lbo = p.stack ? p.bw * p.cw_a * 2 : p.box_a;   // stacked: copy 0 starts one image row below copy 1
    p.tiles_h = (pb.p + (p.stack ? 1 : 0) + p.bh - 1) / p.bh;   // stacked: dy copy 1 of row p-1 is met at chunk row p
    const int tiles_n = (pb.n + p.bn - 1) / p.bn;
    p.chunks_total = p.tiles_w * p.tiles_h * tiles_n;
    const int base = p.n_ktiles * p.n_ctiles * p.n_groups;
    int n_splits = ctx->sm_count / base;   // one wave of one CTA per SM
    if (n_splits > p.chunks_total / 4) n_splits = p.chunks_total / 4;
    if (n_splits < 1) n_splits = 1;
    p.n_splits = n_splits;

    if (!encode_activation_map(ctx, &p.tmDy, pb.dy, pb.n, pb.p, pb.q, pb.k, 1, 0, 0, p.cw_a, p.bw, p.stack ? p.bh + 1 : p.bh, p.bn)) return B2C_ERR_CUDA;
    if (pb.stride == 2) {
        for (int ph = 0; ph < 2; ++ph)
            for (int pw = 0; pw < 2; ++pw)
                if (!encode_activation_map(ctx, &p.tmX[ph * 2 + pw], pb.x, pb.n, pb.h, pb.w, pb.c, 2, ph, pw, p.cw_b, p.bw, p.bh, p.bn))
                    return B2C_ERR_CUDA;
    } else {
        if (!encode_activation_map(ctx, &p.tmX[0], pb.x, pb.n, pb.h, pb.w, pb.c, 1, 0, 0, p.cw_b, p.fx ? p.bw + 2 : p.bw, p.bh, p.bn)) return B2C_ERR_CUDA;
    }
    p.k_total = pb.k;
    p.c_total = pb.c;
    p.rs_total = R * R;
    p.dw = pb.dw;
    plan.smem_bytes = (size_t)p.stages * p.stage_bytes + 1024;
    plan.grid = base * n_splits;
    return B2C_OK;
}

template <typename T>
static inline void key_add(std::string& key, const T& v)
{
    key.append(reinterpret_cast<const char*>(&v), sizeof(T));
}

b2c_status launch_conv_wgrad(b2c_ctx* ctx, const WgradProblem& pb, cudaStream_t stream)
{
    std::string key("W");
    key_add(key, pb.n); key_add(key, pb.h); key_add(key, pb.w); key_add(key, pb.c); key_add(key, pb.p); key_add(key, pb.q); key_add(key, pb.k);
    key_add(key, pb.r); key_add(key, pb.stride); key_add(key, pb.pad); key_add(key, pb.dy); key_add(key, pb.x); key_add(key, pb.dw);
    key_add(key, ctx->use_wgrad_frame); key_add(key, ctx->use_wgrad_two_issuers); key_add(key, ctx->use_group_kblocks);
    auto it = ctx->plan_cache.find(key);
    if (it == ctx->plan_cache.end()) {
        WgradPlan fresh;
        b2c_status st = build_wgrad_plan(ctx, pb, fresh);
        if (st != B2C_OK) return st;
        if (ctx->plan_cache.size() >= 8192) ctx->plan_cache.clear();
        std::vector<unsigned char> bytes(sizeof(WgradPlan));
        memcpy(bytes.data(), &fresh, sizeof(WgradPlan));
        it = ctx->plan_cache.emplace(std::move(key), std::move(bytes)).first;
    }
    WgradPlan plan;
    memcpy(&plan, it->second.data(), sizeof(WgradPlan));
    WgradParams& p = plan.p;
    p.status = ctx->d_status;
    p.spin_limit = ctx->spin_limit;
    p.stall = ctx->stall_counters;

    if (!(ctx->smem_optin_done & B2C_OPTIN_WGRAD)) {
        B2C_CUDA(cudaFuncSetAttribute(conv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 218 * 1024));
        ctx->smem_optin_done |= B2C_OPTIN_WGRAD;
    }
    const size_t smem_bytes = plan.smem_bytes;
    dim3 grid((unsigned)plan.grid);
    B2C_CUDA(b2c_launch(ctx, conv_wgrad_kernel, grid, dim3(kWgThreads), smem_bytes, stream, 1u, p));
    B2C_CUDA(cudaGetLastError());
    return B2C_OK;
}

}  // namespace b2c
