// Stride-1 R x S convolution with the activation transform applied ONCE per staged input
// pixel ("window" kernel).
//
// The im2col form of the fused kernel stages a shifted copy of the input for every filter
// tap, so every input byte is copied into shared memory and transformed R*S times.  Here a
// CTA's output tile is TR whole output rows of one image, laid out with the PADDED width
// Wp = W + 2*pad_w (slot i = tr * Wp + ow; the S-1 slots at the end of each row are junk and
// are never stored).  With that layout tap (r, s) of slot i reads padded-input pixel
// i + r*Wp + s: every tap is the SAME shared-memory matrix shifted by r*Wp + s rows.  So
//   * one tiled TMA box (CB channels x Wp x (TR+R-1) rows, zero fill outside the image)
//     brings the tile's input window in once per channel block,
//   * the transform warps rewrite it in place once (bSPARQ / vSPARQ, Sections 3.1-3.2),
//   * the MMA warp issues tcgen05.mma kind::i8 for every (channel block, tap) with an A
//     descriptor whose start address is advanced by (r*Wp + s) rows.  The 128-/64-byte
//     swizzle is a function of the shared-memory address, so a row-shifted start reads the
//     bytes TMA wrote.
// Weights either stay resident in shared memory for the whole kernel (B_RESIDENT: all
// R*S*C/CB blocks of BN x CB, loaded once per CTA) or stream through a ring of stages.
// Warp roles, bounded waits and the epilogue are those of sparq_gemm_kernel.
#pragma once

#include "sparq_gemm_kernel.cuh"

namespace sparq {

struct WindowArgs {
    // GEMM view for the epilogue
    int64_t N;              // cout
    int64_t K;              // r * s * c
    // geometry
    int n_img, H, W, C, R, S, pad_h, pad_w, Ho, Wo;
    int Wp;                 // W + 2 * pad_w
    int TR;                 // output rows per tile
    int tiles_per_img;      // ceil(Ho / TR)
    int c_blocks;           // C / CB
    int box_bytes;          // CB * Wp * (TR + R - 1): one channel block of one tile's window
    int plane_bytes;        // shared-memory bytes reserved per channel block (>= rows the MMA may touch)
    int win_bufs;           // window buffers in the ring
    int b_stages;           // weight stages (stream mode) or resident blocks (resident mode)
    // transform
    XformDev xf;
    // epilogue
    const float *scale;
    const float *bias;
    int relu;
    float inv_out_scale;
    int32_t *acc_out;
    float *f32_out;
    uint8_t *u8_out;
    unsigned int *status;
    // producer-side transform of u8_out (mode NONE = off)
    int next_mode, next_rnd;
    XformDev next_xf;
    const uint8_t *residual;
    float residual_scale;
};

// dynamic shared memory the kernel may ask for: 227 KB minus room for its static variables
constexpr int kWindowMaxDynSmem = 232448 - 4096;
constexpr int kMaxWinBufs = 4;
constexpr int kMaxBStages = 8;

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c, int w, int h, int n)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        :: "r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n) : "memory");
}

template <int BN, int CB, int MODE, int XN, bool RND, bool B_RESIDENT>
__global__ void __launch_bounds__(kGemmThreads, 1)
sparq_conv_window_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                         const WindowArgs g)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_win_full[kMaxWinBufs], bar_win_xf[kMaxWinBufs], bar_win_empty[kMaxWinBufs];
    __shared__ __align__(8) uint64_t bar_b_full[kMaxBStages], bar_b_empty[kMaxBStages];
    __shared__ __align__(8) uint64_t bar_acc_full[2], bar_acc_empty[2], bar_done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_word;
    __shared__ __align__(16) float s_scale[BN], s_bias[BN];

    constexpr int kBBlock = BN * CB;                   // one (tap, channel block) of weights
    constexpr int kTmemCols = (2 * BN < 32) ? 32 : 2 * BN;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    volatile uint32_t *abort_flag = &abort_word;
    const long long cta_t0 = SPARQ_PROF_NOW();

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t win_bytes = (uint32_t)g.plane_bytes * (uint32_t)g.c_blocks;
    auto win_buf = [&](int b) { return smem_base + (uint32_t)b * win_bytes; };
    const uint32_t b_base = smem_base + (uint32_t)g.win_bufs * win_bytes;
    auto b_slot = [&](int s) { return b_base + (uint32_t)s * kBBlock; };

    const int taps = g.R * g.S;
    const int kb_count = taps * g.c_blocks;            // weight blocks per tile

    if (threadIdx.x == 0) {
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
        for (int b = 0; b < kMaxWinBufs; ++b) {
            mbar_init(smem_u32(&bar_win_full[b]), 1);
            mbar_init(smem_u32(&bar_win_xf[b]), kNumXfWarps);
            mbar_init(smem_u32(&bar_win_empty[b]), 1);
        }
        for (int s = 0; s < kMaxBStages; ++s) {
            mbar_init(smem_u32(&bar_b_full[s]), 1);
            mbar_init(smem_u32(&bar_b_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bar_acc_full[a]), 1);
            mbar_init(smem_u32(&bar_acc_empty[a]), epi_warps(MODE));
        }
        mbar_init(smem_u32(&bar_done), 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    dep_launch();
    dep_wait();

    // With resident weights there is one column tile (host guarantees N <= BN).
    const int64_t n_tiles = (g.N + BN - 1) / BN;
    const int64_t m_tiles = (int64_t)g.n_img * g.tiles_per_img;
    const int64_t total_tiles = m_tiles * n_tiles;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t wt = 0;      // window counter
            uint32_t it = 0;      // streamed weight-block counter
            bool b_issued = false;  // resident weights requested
            long long pw = 0;
            const long long pt0 = SPARQ_PROF_NOW();
            for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++wt) {
                const int64_t mt = tile / n_tiles, nt = tile % n_tiles;
                const int img = (int)(mt / g.tiles_per_img);
                const int oh0 = (int)(mt % g.tiles_per_img) * g.TR;
                const int b = wt % g.win_bufs;
                const uint32_t use = wt / g.win_bufs;
                if (use > 0) SPARQ_PROF_WAIT(pw, mbar_wait(smem_u32(&bar_win_empty[b]), (use - 1) & 1, abort_flag, g.status));
                if (*abort_flag) break;
                const uint32_t wfull = smem_u32(&bar_win_full[b]);
                mbar_expect_tx(wfull, (uint32_t)g.box_bytes * (uint32_t)g.c_blocks);
                for (int cb = 0; cb < g.c_blocks; ++cb)
                    tma_load_4d(win_buf(b) + (uint32_t)cb * g.plane_bytes, &map_x, wfull,
                                cb * CB, -g.pad_w, oh0 - g.pad_h, img);
                if (B_RESIDENT && wt == 0) {
                    // all weight blocks, once per CTA, on stage barrier 0 -- after the first
                    // window so that the activations (which come from HBM and still have to
                    // be transformed) are requested first
                    const uint32_t full = smem_u32(&bar_b_full[0]);
                    mbar_expect_tx(full, (uint32_t)kb_count * kBBlock);
                    for (int kb = 0; kb < kb_count; ++kb) {
                        const int cb = kb / taps, tap = kb % taps;
                        tma_load_2d(b_slot(kb), &map_w, full, tap * g.C + cb * CB, 0);
                    }
                    b_issued = true;
                }
                if (!B_RESIDENT) {
                    for (int kb = 0; kb < kb_count; ++kb, ++it) {
                        const int s = it % g.b_stages;
                        const uint32_t buse = it / g.b_stages;
                        if (buse > 0) mbar_wait(smem_u32(&bar_b_empty[s]), (buse - 1) & 1, abort_flag, g.status);
                        if (*abort_flag) break;
                        const int cb = kb / taps, tap = kb % taps;
                        const uint32_t full = smem_u32(&bar_b_full[s]);
                        mbar_expect_tx(full, kBBlock);
                        tma_load_2d(b_slot(s), &map_w, full, tap * g.C + cb * CB, (int)(nt * BN));
                    }
                }
                // an abort noticed here is acted on at the top of the next iteration, after this
                // tile's window has been counted in wt (the drain below waits for it)
            }
            SPARQ_PROF_STORE(0, pw);
            SPARQ_PROF_STORE(1, SPARQ_PROF_NOW() - pt0);
            if (*abort_flag) {
                // wait (bounded) for copies still in flight so that none lands after exit
                const uint32_t wfirst = wt > (uint32_t)g.win_bufs ? wt - g.win_bufs : 0;
                for (uint32_t j = wfirst; j < wt; ++j)
                    mbar_wait(smem_u32(&bar_win_full[j % g.win_bufs]), (j / g.win_bufs) & 1, abort_flag, g.status, true);
                if (B_RESIDENT) {
                    // the weight copies were issued together with the first window
                    if (b_issued) mbar_wait(smem_u32(&bar_b_full[0]), 0, abort_flag, g.status, true);
                } else {
                    const uint32_t first = it > (uint32_t)g.b_stages ? it - g.b_stages : 0;
                    for (uint32_t j = first; j < it; ++j)
                        mbar_wait(smem_u32(&bar_b_full[j % g.b_stages]), (j / g.b_stages) & 1, abort_flag, g.status, true);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // The whole warp runs this loop converged and one elected lane issues: the descriptor
        // arithmetic below is on warp-uniform values only (kernel arguments, loop counters),
        // which lets it stay in the uniform datapath that feeds tcgen05.mma.
        {
            const uint32_t elected = elect_one();
            constexpr uint32_t idesc = make_idesc_i8(BN);
            // descriptors of window buffer 0 and of weight slot 0; offsets are added in units of
            // 16 bytes to the start-address field (the low word never carries into the next field)
            const uint64_t win_desc0 = make_smem_desc<CB>(smem_base);
            const uint64_t b_desc0 = make_smem_desc<CB>(b_base);
            uint32_t wt = 0;
            int b = 0;  uint32_t wph = 0;      // window buffer and its phase parity
            int s = 0;  uint32_t bph = 0;      // streamed weight stage and its phase parity
            long long mw = 0, ma = 0, mb = 0, mi = 0;
            const long long mt0 = SPARQ_PROF_NOW();
            // descriptor steps, in 16-byte units: one padded input row, one channel-block plane
            const uint32_t row16 = (uint32_t)(g.Wp * CB) >> 4;
            const uint32_t plane16 = (uint32_t)g.plane_bytes >> 4;
            if (B_RESIDENT) SPARQ_PROF_WAIT(mb, mbar_wait(smem_u32(&bar_b_full[0]), 0, abort_flag, g.status));
            for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++wt) {
                const int acc = wt & 1;
                const uint32_t acc_use = wt >> 1;
                if (acc_use > 0) SPARQ_PROF_WAIT(ma, mbar_wait(smem_u32(&bar_acc_empty[acc]), (acc_use - 1) & 1, abort_flag, g.status));
                if (MODE == SPARQ_MODE_NONE) SPARQ_PROF_WAIT(mw, mbar_wait(smem_u32(&bar_win_full[b]), wph, abort_flag, g.status));
                else SPARQ_PROF_WAIT(mw, mbar_wait(smem_u32(&bar_win_xf[b]), wph, abort_flag, g.status));
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                const uint64_t a_desc0 = win_desc0 + (uint64_t)((uint32_t)b * (win_bytes >> 4));
                const long long is0 = SPARQ_PROF_NOW();
                // One (tap, channel block) of the tile: wait for its weights when they are
                // streamed, then CB / 32 MMAs.  The descriptors are sums of warp-uniform
                // loop-carried values (no table, no division), so the address arithmetic of
                // consecutive MMAs is a couple of adds.
                auto issue_block = [&](const uint32_t kb, const uint64_t adesc) {
                    uint64_t bdesc;
                    if (B_RESIDENT) {
                        bdesc = b_desc0 + (uint64_t)(kb * (uint32_t)(kBBlock >> 4));
                    } else {
                        SPARQ_PROF_WAIT(mb, mbar_wait(smem_u32(&bar_b_full[s]), bph, abort_flag, g.status));
                        tc_fence_after();
                        bdesc = b_desc0 + (uint64_t)((uint32_t)s * (uint32_t)(kBBlock >> 4));
                    }
#pragma unroll
                    for (int k = 0; k < CB / 32; ++k)
                        tc_mma_i8_if(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                                     (kb > 0 || k > 0) ? 1u : 0u, elected);
                    if (!B_RESIDENT) {
                        tc_commit_if(smem_u32(&bar_b_empty[s]), elected);
                        if (++s == g.b_stages) { s = 0; bph ^= 1u; }
                    }
                };
                uint32_t kb = 0;
                uint64_t a_cb = a_desc0;
                if (g.R == 3 && g.S == 3) {
                    for (int cb = 0; cb < g.c_blocks; ++cb, a_cb += plane16) {
#pragma unroll
                        for (int r = 0; r < 3; ++r)
#pragma unroll
                            for (int sx = 0; sx < 3; ++sx, ++kb)
                                issue_block(kb, a_cb + (uint64_t)((uint32_t)r * row16 + (uint32_t)(sx * (CB >> 4))));
                    }
                } else {
                    for (int cb = 0; cb < g.c_blocks; ++cb, a_cb += plane16) {
                        uint64_t a_r = a_cb;
                        for (int r = 0; r < g.R; ++r, a_r += row16)
                            for (int sx = 0; sx < g.S; ++sx, ++kb)
                                issue_block(kb, a_r + (uint64_t)(uint32_t)(sx * (CB >> 4)));
                    }
                }
                mi += SPARQ_PROF_NOW() - is0;
                tc_commit_if(smem_u32(&bar_win_empty[b]), elected);       // window reusable once these MMAs retire
                tc_commit_if(smem_u32(&bar_acc_full[acc]), elected);      // accumulator complete
                if (++b == g.win_bufs) { b = 0; wph ^= 1u; }
            }
            SPARQ_PROF_STORE(2, mw);
            SPARQ_PROF_STORE(3, ma);
            SPARQ_PROF_STORE(11, mb);
            SPARQ_PROF_STORE(12, mi);
            SPARQ_PROF_STORE(4, SPARQ_PROF_NOW() - mt0);
            tc_commit_if(smem_u32(&bar_done), elected);
            mbar_wait(smem_u32(&bar_done), 0, abort_flag, g.status, true);
        }
        __syncwarp();
    } else if (warp < kFirstEpiWarp + epi_warps(MODE)) {
        // ================= epilogue =================
        constexpr int kEpi = epi_warps(MODE);
        constexpr int kColsPerWarp = BN / (kEpi / 4);     // the tile's columns are split over the warps of a quarter
        const int quarter = warp & 3;
        const int part = (warp - kFirstEpiWarp) >> 2;
        const int et = threadIdx.x - kFirstEpiWarp * 32;
        const EpiView ev = make_epi_view(g);
        uint32_t wt = 0;
        int64_t staged_nt = -1;
        // this thread's slot inside a tile: row tr of the tile, padded column ow
        const int slot = quarter * 32 + lane;
        const int tr = slot / g.Wp;
        const int ow = slot - tr * g.Wp;
        const bool slot_ok = (tr < g.TR) && (ow < g.Wo);
        long long ew = 0;
        const long long et0 = SPARQ_PROF_NOW();
        // 64-wide tiles have one column tile and 16 or 32 columns per warp.  When only the
        // requantized bytes are wanted (the form every layer of a network uses), the warp keeps
        // the scale and bias of its columns in registers for the whole launch -- shared-memory
        // reads queue behind the tensor core's operand fetches -- and takes the accumulator in
        // 16-column pieces so that those registers fit beside it.
        if (BN == 64 && ev.need_f && !g.acc_out && !g.f32_out && !g.residual && g.N == 64) {
            epi_stage_scale_bias<kEpi>(g, 0, BN, et, s_scale, s_bias);
            const int cbase = part * kColsPerWarp;
            float rs[kColsPerWarp], rb[kColsPerWarp];
#pragma unroll
            for (int i = 0; i < kColsPerWarp; ++i) {
                rs[i] = s_scale[cbase + i];
                rb[i] = s_bias[cbase + i];
            }
            const uint32_t tiles32 = (uint32_t)total_tiles, tpi = (uint32_t)g.tiles_per_img;
            for (uint32_t tile = blockIdx.x; tile < tiles32; tile += gridDim.x, ++wt) {
                const uint32_t acc = wt & 1u;
                // coordinates first: they do not depend on the accumulator
                const uint32_t img = tile / tpi;
                const int oh = (int)(tile - img * tpi) * g.TR + tr;
                const bool row_ok = slot_ok && (oh < g.Ho);
                uint8_t *dst = g.u8_out + (((int64_t)img * g.Ho + oh) * g.Wo + ow) * 64 + cbase;
                const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + (uint32_t)cbase;
                SPARQ_PROF_WAIT(ew, mbar_wait(smem_u32(&bar_acc_full[acc]), (wt >> 1) & 1u, abort_flag, g.status));
                tc_fence_after();
#pragma unroll
                for (int hh = 0; hh < kColsPerWarp / 16; ++hh) {
                    uint32_t v[16];
                    tmem_ld_32x16_issue(taddr0 + (uint32_t)(hh * 16), v);
                    tmem_ld_wait();
                    if (hh + 1 == kColsPerWarp / 16) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
                    }
                    if (!row_ok) continue;
                    uint32_t w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t b[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int c = hh * 16 + 4 * q + j;
                            const float y = ev.small_acc ? dequant<true>((int32_t)v[4 * q + j], rs[c], rb[c], ev.relu_op)
                                                         : dequant<false>((int32_t)v[4 * q + j], rs[c], rb[c], ev.relu_op);
                            b[j] = requant_bits(y, ev.inv_out_scale);
                        }
                        w[q] = pack4(b[0], b[1], b[2], b[3]);
                    }
                    if (ev.next_mode != SPARQ_MODE_NONE) {
                        const bool fast4 = ev.next_xf.n == 4 && ev.next_xf.rounds == 0;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (ev.next_mode == SPARQ_MODE_VSPARQ) {
                                if (fast4) w[q] = ev.next_rnd ? xform_word<SPARQ_MODE_VSPARQ, 4, true, false>(w[q], ev.next_xf)
                                                              : xform_word<SPARQ_MODE_VSPARQ, 4, false, false>(w[q], ev.next_xf);
                                else w[q] = ev.next_rnd ? xform_word<SPARQ_MODE_VSPARQ, 0, true, true>(w[q], ev.next_xf)
                                                        : xform_word<SPARQ_MODE_VSPARQ, 0, false, true>(w[q], ev.next_xf);
                            } else {
                                if (fast4) w[q] = ev.next_rnd ? xform_word<SPARQ_MODE_BSPARQ, 4, true, false>(w[q], ev.next_xf)
                                                              : xform_word<SPARQ_MODE_BSPARQ, 4, false, false>(w[q], ev.next_xf);
                                else w[q] = ev.next_rnd ? xform_word<SPARQ_MODE_BSPARQ, 0, true, true>(w[q], ev.next_xf)
                                                        : xform_word<SPARQ_MODE_BSPARQ, 0, false, true>(w[q], ev.next_xf);
                            }
                        }
                    }
                    *reinterpret_cast<uint4 *>(dst + hh * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        } else
        for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++wt) {
            const int64_t mt = tile / n_tiles, nt = tile % n_tiles;
            const int acc = wt & 1;
            const uint32_t acc_use = wt >> 1;
            if (ev.need_f && nt != staged_nt) {
                staged_nt = nt;
                epi_stage_scale_bias<kEpi>(g, nt * BN, BN, et, s_scale, s_bias);
            }
            SPARQ_PROF_WAIT(ew, mbar_wait(smem_u32(&bar_acc_full[acc]), acc_use & 1, abort_flag, g.status));
            tc_fence_after();
            const int img = (int)(mt / g.tiles_per_img);
            const int oh = (int)(mt % g.tiles_per_img) * g.TR + tr;
            const bool row_ok = slot_ok && (oh < g.Ho);
            const int64_t row = ((int64_t)img * g.Ho + oh) * g.Wo + ow;
            const int cbase = part * kColsPerWarp;
            const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + cbase);
            epi_warp_columns<kColsPerWarp>(ev, taddr0, cbase, row, row_ok, nt * BN, s_scale, s_bias,
                                      smem_u32(&bar_acc_empty[acc]), lane);
        }
        if (warp == kFirstEpiWarp && lane == 0) {
            SPARQ_PROF_STORE(5, ew);
            SPARQ_PROF_STORE(6, SPARQ_PROF_NOW() - et0);
        }
    } else if (MODE != SPARQ_MODE_NONE) {
        // ================= transform: once per window =================
        const int xt = threadIdx.x - kFirstXfWarp * 32;
        constexpr int kXfThreads = kNumXfWarps * 32;
        const XformDev xf = g.xf;
        // whole groups of kXfThreads * 4 vectors; the tail group runs into the plane's slack
        // rows, which no valid output reads (the host sizes the plane for it)
        const int groups = (g.box_bytes + kXfThreads * 64 - 1) / (kXfThreads * 64);
        uint32_t wt = 0;
        long long xw = 0;
        const long long xt0 = SPARQ_PROF_NOW();
        for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++wt) {
            const int b = wt % g.win_bufs;
            SPARQ_PROF_WAIT(xw, mbar_wait(smem_u32(&bar_win_full[b]), (wt / g.win_bufs) & 1, abort_flag, g.status));
            for (int cb = 0; cb < g.c_blocks; ++cb) {
                const uint32_t base = win_buf(b) + (uint32_t)cb * g.plane_bytes + (uint32_t)xt * 16u;
                for (int grp = 0; grp < groups; ++grp) {
                    const uint32_t gbase = base + (uint32_t)grp * (kXfThreads * 64);
                    uint4 v[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(v[j].x), "=r"(v[j].y), "=r"(v[j].z), "=r"(v[j].w)
                                     : "r"(gbase + (uint32_t)(j * kXfThreads * 16)));
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        v[j].x = xform_word<MODE, XN, RND, XN == 0>(v[j].x, xf);
                        v[j].y = xform_word<MODE, XN, RND, XN == 0>(v[j].y, xf);
                        v[j].z = xform_word<MODE, XN, RND, XN == 0>(v[j].z, xf);
                        v[j].w = xform_word<MODE, XN, RND, XN == 0>(v[j].w, xf);
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};"
                                     :: "r"(gbase + (uint32_t)(j * kXfThreads * 16)),
                                        "r"(v[j].x), "r"(v[j].y), "r"(v[j].z), "r"(v[j].w) : "memory");
                    }
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_win_xf[b]));
        }
        if (warp == kFirstXfWarp && lane == 0) {
            SPARQ_PROF_STORE(7, xw);
            SPARQ_PROF_STORE(8, SPARQ_PROF_NOW() - xt0);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) SPARQ_PROF_STORE(10, SPARQ_PROF_NOW() - cta_t0);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     :: "r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

template <int BN, int CB, bool B_RESIDENT>
cudaError_t launch_window_shape(const CUtensorMap &mx, const CUtensorMap &mw, const WindowArgs &g,
                                int mode, int n, int rnd, int grid, int smem_bytes, cudaStream_t st);

#define SPARQ_LAUNCH_WINDOW_VARIANT(MODE_, XN_, RND_)                                                  \
    do {                                                                                               \
        auto kfn = sparq_conv_window_kernel<BN, CB, MODE_, XN_, RND_, RES>;                            \
        static bool attr_set[64] = {};   /* per device ordinal */                                     \
        int dev_ = 0;                                                                                  \
        cudaError_t e_ = cudaGetDevice(&dev_);                                                         \
        if (e_ != cudaSuccess) return e_;                                                              \
        if (dev_ < 0 || dev_ >= 64 || !attr_set[dev_]) {                                               \
            e_ = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize,                \
                                      kWindowMaxDynSmem);                                              \
            if (e_ != cudaSuccess) return e_;                                                          \
            if (dev_ >= 0 && dev_ < 64) attr_set[dev_] = true;                                         \
        }                                                                                              \
        return launch_pdl(kfn, grid, smem_bytes, st, mx, mw, g);                                       \
    } while (0)

#define SPARQ_DEFINE_WINDOW_SHAPE(BN_, CB_, RES_)                                                      \
    template <>                                                                                        \
    cudaError_t launch_window_shape<BN_, CB_, RES_>(const CUtensorMap &mx, const CUtensorMap &mw,      \
                                                    const WindowArgs &g, int mode, int n, int rnd,     \
                                                    int grid, int smem_bytes, cudaStream_t st)         \
    {                                                                                                  \
        constexpr int BN = BN_, CB = CB_;                                                              \
        constexpr bool RES = RES_;                                                                     \
        if (mode == SPARQ_MODE_NONE) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_NONE, 4, false);           \
        if (mode == SPARQ_MODE_BSPARQ) {                                                               \
            if (n == 4) { if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 4, true);            \
                          else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 4, false); }             \
            if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 0, true);                          \
            else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 0, false);                             \
        }                                                                                              \
        if (n == 4) { if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 4, true);                \
                      else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 4, false); }                 \
        if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 0, true);                              \
        else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 0, false);                                 \
    }

}  // namespace sparq
