// Stride-1 R x S convolution with the activation transform applied once per staged input
// row ("window" kernel).
//
// The im2col form of the fused kernel stages a shifted copy of the input for every filter
// tap, so every input byte is copied into shared memory and transformed R*S times.  Here a
// CTA's output tile is TR whole output rows of one image, laid out with the PADDED width
// Wp = W + 2*pad_w (slot i = tr * Wp + ow; the S-1 slots at the end of each row are junk and
// are never stored).  With that layout tap (r, s) of slot i reads padded-input pixel
// i + r*Wp + s: every tap is the SAME shared-memory matrix shifted by r*Wp + s rows.
//
// Up to G consecutive tiles of one image form a GROUP that shares one window buffer of
// G*TR + R-1 input rows, so the R-1 halo rows between neighbouring tiles are staged and
// transformed once instead of once per tile.  The window arrives in pieces -- the first is
// TR+R-1 rows, every later one TR rows -- each with its own pair of barriers, and tile j of
// the group needs pieces 0..j only: the tensor core starts on the first tile while later
// pieces are still in flight or being transformed.
//   * tiled TMA boxes (CB channels x Wp x piece rows, zero fill outside the image) bring the
//     pieces in, once per channel block; the swizzle of a box is a function of the
//     shared-memory address, so pieces written at consecutive row offsets form one
//     consistently swizzled matrix,
//   * the transform warps rewrite each piece in place once (bSPARQ / vSPARQ, Sections 3.1-3.2),
//   * the MMA warp issues tcgen05.mma kind::i8 for every (channel block, tap) with an A
//     descriptor whose start address is advanced by (j*TR*Wp + r*Wp + s) rows.
// Each CTA owns a contiguous range of the tile sequence (balanced to within one tile) and
// cuts it into groups at image boundaries.
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
    int G;                  // most tiles that share one window (1 when there are several column tiles)
    int piece0_bytes;       // CB * Wp * (TR + R - 1): first piece of a group, one channel block
    int piece_bytes;        // CB * Wp * TR: every later piece
    int plane_bytes;        // shared-memory bytes reserved per channel block (>= rows the MMA may touch)
    int win_bufs;           // window buffers in the ring
    int b_stages;           // weight stages (stream mode) or resident blocks (resident mode)
    int early_weights;      // resident weights may be fetched before the previous kernel on the stream has finished
    int issuers;            // 2: the two issuer warps alternate (resident weights); 1: warp 1 issues every tile (streamed weights)
    int w_one_copy;         // resident weights: map_w is the 3-D (bytes, rows, blocks) view and one copy brings all blocks
    uint32_t n_tiles;       // column tiles
    uint32_t units;         // n_img * tiles_per_img * n_tiles, column tile fastest
    uint32_t groups;        // streamed weights on 128-wide tiles: n_img * n_tiles * ceil(tiles_per_img / G) whole
                            // groups of up to G row tiles of one (image, column tile), which share one pass over
                            // the weights; CTAs own whole groups there, contiguous shares of the unit sequence else
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
    long long wait_limit;   // cycles after which a device-side wait gives up
    // producer-side transform of u8_out (mode NONE = off)
    int next_mode, next_rnd;
    XformDev next_xf;
    const uint8_t *residual;
    float residual_scale;
};

// dynamic shared memory the kernel may ask for: 227 KB minus room for its static variables
constexpr int kWindowMaxDynSmem = 232448 - 4096;
constexpr int kMaxWinBufs = 4;
constexpr int kMaxG = 8;
constexpr int kMaxBStages = 12;
// Two warps issue MMAs, taking the tiles of a CTA alternately (each owns one of the two
// accumulators): whatever one of them does between two tiles -- commits, barrier reads that
// queue behind the tensor core's own shared-memory traffic, descriptor set-up -- happens
// while the other one's MMAs keep the tensor core busy.
constexpr int kMmaBWarp = kFirstXfWarp + kNumXfWarps;      // the second issuer is the last warp
constexpr int kWindowThreads = kGemmThreads + 32;

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c, int w, int h, int n)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        :: "r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n) : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}

// Walks the groups of one CTA's share of the tile sequence.  Every warp role runs the same
// walk, so that window buffers, accumulators and barrier phases line up without any
// communication.
template <bool BY_GROUP>
struct GroupWalk {
    uint32_t u, u_end;          // units (BY_GROUP: whole groups) still to do: [u, u_end)
    uint32_t n_tiles, tpi, G;
    uint32_t img, tin, nt, cnt; // current group: image, first tile inside it, column tile, tiles

    __device__ __forceinline__ GroupWalk(const WindowArgs &g)
    {
        // the sequence is split into gridDim.x contiguous shares that differ by at most one
        const uint32_t total = BY_GROUP ? g.groups : g.units;
        const uint32_t q = total / gridDim.x, rem = total - q * gridDim.x;
        u = blockIdx.x * q + (blockIdx.x < rem ? blockIdx.x : rem);
        u_end = u + q + (blockIdx.x < rem ? 1u : 0u);
        n_tiles = g.n_tiles; tpi = (uint32_t)g.tiles_per_img; G = (uint32_t)g.G;
        img = tin = nt = cnt = 0;
    }
    __device__ __forceinline__ bool next()
    {
        if (u >= u_end) return false;
        if (BY_GROUP) {
            // group number u = (image * n_tiles + column tile) * gpt + k: tiles k*G .. of that image
            const uint32_t gpt = (tpi + G - 1) / G;
            const uint32_t key = u / gpt, k = u - key * gpt;
            img = key / n_tiles;
            nt = key - img * n_tiles;
            tin = k * G;
            cnt = tpi - tin < G ? tpi - tin : G;
            u += 1;
            return true;
        }
        uint32_t mt = u;
        nt = 0;
        if (n_tiles != 1) { mt = u / n_tiles; nt = u - mt * n_tiles; }
        img = mt / tpi;
        tin = mt - img * tpi;
        uint32_t c = 1;
        if (n_tiles == 1) {
            c = tpi - tin;
            if (c > G) c = G;
            if (c > u_end - u) c = u_end - u;
        }
        cnt = c;
        u += c;
        return true;
    }
};

template <int BN, int CB, int MODE, int XN, bool RND, bool B_RESIDENT>
__global__ void __launch_bounds__(kWindowThreads, 1)
sparq_conv_window_kernel(const __grid_constant__ CUtensorMap map_x0, const __grid_constant__ CUtensorMap map_x1,
                         const __grid_constant__ CUtensorMap map_w, const WindowArgs g)
{
    extern __shared__ uint8_t smem_raw[];
    // one pair per (window buffer, piece): bytes landed / piece transformed
    __shared__ __align__(8) uint64_t bar_win_full[kMaxWinBufs * kMaxG], bar_win_xf[kMaxWinBufs * kMaxG];
    __shared__ __align__(8) uint64_t bar_win_empty[kMaxWinBufs];
    __shared__ __align__(8) uint64_t bar_b_full[kMaxBStages], bar_b_empty[kMaxBStages];
    // Accumulator stages in tensor memory; tile number t uses stage t % kAcc.  (Four stages were
    // measured and changed nothing for tiles that run one after the other: the epilogue hands a
    // stage back well within one tile.)  Streamed weights on 128-wide tiles: the tiles of a group
    // are accumulated TOGETHER during one pass over the weights (kBatched), so a group holds up
    // to two stages and four let the next group start while the previous one is in its epilogue.
    constexpr bool kBatched = !B_RESIDENT && BN == 128;
    constexpr int kAcc = kBatched ? 4 : 2;
    __shared__ __align__(8) uint64_t bar_acc_full[kAcc], bar_acc_empty[kAcc], bar_done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_word;
    __shared__ __align__(16) float s_scale[BN], s_bias[BN];

    constexpr int kBBlock = BN * CB;                   // one (tap, channel block) of weights
    constexpr int kTmemCols = kAcc * BN;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    volatile uint32_t *abort_flag = &abort_word;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t win_bytes = (uint32_t)g.plane_bytes * (uint32_t)g.c_blocks;
    auto win_buf = [&](int b) { return smem_base + (uint32_t)b * win_bytes; };
    const uint32_t b_base = smem_base + (uint32_t)g.win_bufs * win_bytes;
    auto b_slot = [&](int s) { return b_base + (uint32_t)s * kBBlock; };
    // byte offset of piece j inside a channel block's plane, and its size
    auto piece_off = [&](int j) { return j ? (uint32_t)((j * g.TR + g.R - 1) * g.Wp * CB) : 0u; };
    auto piece_len = [&](int j) { return (uint32_t)(j ? g.piece_bytes : g.piece0_bytes); };

    const int taps = g.R * g.S;
    const int kb_count = taps * g.c_blocks;            // weight blocks per tile
    // A tile's epilogue is mostly latency (barrier read, tensor-memory loads, stores), not
    // arithmetic.  When only requantized bytes are wanted and there is one column tile, the epilogue
    // warps split into two teams, one per accumulator stage, each warp taking twice the columns of
    // its lane quarter, so that the epilogues of two consecutive tiles overlap.
    // (Measured: a gain on 64-wide tiles and on 128-wide tiles with a transform, whose eight epilogue
    // warps are latency-bound; a loss where sixteen warps are already bound by instruction issue or
    // where a warp would hold a 256-column accumulator for eight loads.)
    constexpr bool kTeamsPay = BN == 64 || (BN == 128 && MODE != SPARQ_MODE_NONE);
    const bool epi_teams = kTeamsPay && g.u8_out && !g.acc_out && !g.f32_out && !g.residual && g.next_mode == SPARQ_MODE_NONE &&
                           g.n_tiles == 1 && (g.N % 32) == 0 && (!g.relu || g.inv_out_scale > 0.0f) &&
                           (reinterpret_cast<uintptr_t>(g.u8_out) & 31u) == 0;
    if (threadIdx.x == 0) {
        prefetch_tensormap(&map_x0);
        prefetch_tensormap(&map_x1);
        prefetch_tensormap(&map_w);
    }
    if (warp == 0) {
        // barrier set-up spread over the lanes of one warp
        for (int b = lane; b < kMaxWinBufs * kMaxG; b += 32) {
            mbar_init(smem_u32(&bar_win_full[b]), 1);
            mbar_init(smem_u32(&bar_win_xf[b]), kNumXfWarps);
        }
        if (lane < kMaxWinBufs) mbar_init(smem_u32(&bar_win_empty[lane]), 2);     // one arrival per issuing warp
        if (lane < kMaxBStages) {
            mbar_init(smem_u32(&bar_b_full[lane]), 1);
            mbar_init(smem_u32(&bar_b_empty[lane]), 1);
        }
        if (lane < kAcc) {
            mbar_init(smem_u32(&bar_acc_full[lane]), 1);
            mbar_init(smem_u32(&bar_acc_empty[lane]), epi_teams ? epi_warps(MODE) / 2 : epi_warps(MODE));
        }
        if (lane == 0) {
            mbar_init(smem_u32(&bar_done), 2);
            abort_word = 0;
        }
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
    // this CTA's share of the tile sequence: kernel arguments only, so it is worked out (two
    // integer divisions) while the previous kernel may still be running
    GroupWalk<kBatched> walk(g);
    bool have = walk.next();       // the first group, too
    // All weight blocks, once per CTA, on stage barrier 0: every CTA reads the same bytes, so
    // they come out of L2 one reader after the other, and they are what the first tile waits
    // for longest.  Block (tap, cb) = bytes [tap*C + cb*CB, +CB) of every filter lands in slot
    // tap * c_blocks + cb.
    auto issue_resident_weights = [&]() {
        const uint32_t full = smem_u32(&bar_b_full[0]);
        mbar_expect_tx(full, (uint32_t)kb_count * kBBlock);
        if (g.w_one_copy) {
            tma_load_3d(b_slot(0), &map_w, full, 0, 0, 0);
        } else {
            for (int kb = 0; kb < kb_count; ++kb) tma_load_2d(b_slot(kb), &map_w, full, kb * CB, 0);
        }
    };
    // The weights are not an output of the kernel that runs before this one (the host checks
    // that and sets early_weights), so their copy may start before that kernel has finished:
    // in a chain of layers the wait for the weights then overlaps the predecessor's tail.
    bool b_issued = false;
    if (B_RESIDENT && g.early_weights && threadIdx.x == 0 && have) {
        issue_resident_weights();
        b_issued = true;
    }
    dep_launch();
    dep_wait();


    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t gi = 0;                   // group counter
            int rb = 0; uint32_t ruse = 0;     // its window buffer (gi % win_bufs) and that buffer's use count (gi / win_bufs)
            uint32_t it = 0;      // streamed weight-block counter
            for (; have; have = walk.next()) {
                const int b = rb;                 // window buffer of this group and how often it was used before
                const uint32_t use = ruse;
                if (use > 0) mbar_wait(smem_u32(&bar_win_empty[b]), (use - 1) & 1, abort_flag, g.status, g.wait_limit);
                if (*abort_flag) break;
                const int oh0 = (int)walk.tin * g.TR;
                if (B_RESIDENT && !b_issued) {
                    issue_resident_weights();
                    b_issued = true;
                }
                for (int j = 0; j < g.G; ++j) {
                    const uint32_t wfull = smem_u32(&bar_win_full[b * kMaxG + j]);
                    if (j < (int)walk.cnt) {
                        mbar_expect_tx(wfull, piece_len(j) * (uint32_t)g.c_blocks);
                        const int h0 = oh0 - g.pad_h + (j ? j * g.TR + g.R - 1 : 0);
                        uint32_t dst = win_buf(b) + piece_off(j);
                        for (int cb = 0; cb < g.c_blocks; ++cb, dst += (uint32_t)g.plane_bytes)
                            tma_load_4d(dst, j ? &map_x1 : &map_x0, wfull, cb * CB, -g.pad_w, h0, (int)walk.img);
                    } else {
                        // a piece this group does not have: complete its phase so that the
                        // parity of every barrier of the buffer advances once per use
                        mbar_arrive(wfull);
                    }
                }
                ++gi;
            if (++rb == g.win_bufs) { rb = 0; ++ruse; }
                if (!B_RESIDENT) {
                    bool stop = false;
                    const int passes = kBatched ? 1 : (int)walk.cnt;     // batched: one pass serves the whole group
                    for (int j = 0; j < passes && !stop; ++j) {
                        for (int cb = 0; cb < g.c_blocks && !stop; ++cb) {
                            for (int tap = 0; tap < taps; ++tap, ++it) {
                                const int s = it % g.b_stages;
                                const uint32_t buse = it / g.b_stages;
                                if (buse > 0) mbar_wait(smem_u32(&bar_b_empty[s]), (buse - 1) & 1, abort_flag, g.status, g.wait_limit);
                                if (*abort_flag) { stop = true; break; }
                                const uint32_t full = smem_u32(&bar_b_full[s]);
                                mbar_expect_tx(full, kBBlock);
                                tma_load_2d(b_slot(s), &map_w, full, tap * g.C + cb * CB, (int)(walk.nt * BN));
                            }
                        }
                    }
                    if (stop) break;
                }
            }
            if (*abort_flag) {
                // wait (bounded) for copies still in flight so that none lands after exit
                const uint32_t gfirst = gi > (uint32_t)g.win_bufs ? gi - g.win_bufs : 0;
                for (uint32_t q = gfirst; q < gi; ++q)
                    for (int j = 0; j < g.G; ++j)
                        mbar_wait(smem_u32(&bar_win_full[(q % g.win_bufs) * kMaxG + j]), (q / g.win_bufs) & 1,
                                  abort_flag, g.status, g.wait_limit, true);
                if (B_RESIDENT) {
                    if (b_issued) mbar_wait(smem_u32(&bar_b_full[0]), 0, abort_flag, g.status, g.wait_limit, true);
                } else {
                    const uint32_t first = it > (uint32_t)g.b_stages ? it - g.b_stages : 0;
                    for (uint32_t q = first; q < it; ++q)
                        mbar_wait(smem_u32(&bar_b_full[q % g.b_stages]), (q / g.b_stages) & 1, abort_flag, g.status, g.wait_limit, true);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == kMmaBWarp) {
        // ================= MMA issuers =================
        // Issuer `me` (0: warp 1, 1: the last warp) takes the tiles whose running number has
        // parity `me`; tile number t goes into accumulator stage t % kAcc.  Each warp runs its loop converged and one elected
        // lane issues: the descriptor arithmetic below is on warp-uniform values only (kernel
        // arguments, loop counters), which lets it stay in the uniform datapath that feeds
        // tcgen05.mma.
        {
            const uint32_t me = (warp == 1) ? 0u : 1u;
            const uint32_t elected = elect_one();
            constexpr uint32_t idesc = make_idesc_i8(BN);
            // descriptors of window buffer 0 and of weight slot 0; offsets are added in units of
            // 16 bytes to the start-address field (the low word never carries into the next field)
            const uint64_t win_desc0 = make_smem_desc<CB>(smem_base);
            const uint64_t b_desc0 = make_smem_desc<CB>(b_base);
            uint32_t wt = 0;                   // tile counter (both issuers count every tile)
            uint32_t gi = 0;                   // group counter
            int rb = 0; uint32_t ruse = 0;     // its window buffer (gi % win_bufs) and that buffer's use count (gi / win_bufs)
            int s = 0;  uint32_t bph = 0;      // streamed weight stage and its phase parity
            // descriptor steps, in 16-byte units: one padded input row, one channel-block plane,
            // the rows of one tile
            const uint32_t row16 = (uint32_t)(g.Wp * CB) >> 4;
            const uint32_t plane16 = (uint32_t)g.plane_bytes >> 4;
            const uint32_t tile16 = (uint32_t)(g.TR * g.Wp * CB) >> 4;
            if (B_RESIDENT) mbar_wait(smem_u32(&bar_b_full[0]), 0, abort_flag, g.status, g.wait_limit);
            for (; have; have = walk.next()) {
                const int b = rb;
                const uint32_t wph = ruse & 1u;
                const uint64_t a_grp = win_desc0 + (uint64_t)((uint32_t)b * (win_bytes >> 4));
                bool issued = false;
                // Barrier reads go through the shared-memory pipe, which the tensor core's operand
                // fetches keep saturated, so a read takes hundreds of cycles.  The two barriers of
                // this issuer's NEXT tile of the group are therefore looked at (non-blocking, both
                // reads in flight together) after the first few MMAs of the current tile have been
                // queued; when both say "ready" -- the usual case -- that tile starts without
                // touching shared memory.
                uint32_t pre_acc = 0, pre_ops = 0;
                if constexpr (kBatched) {
                    // One pass over the streamed weights for all tiles of the group: every weight
                    // block is fetched from L2 once per group instead of once per tile.  Warp 1
                    // issues; the other issuer only keeps its counters in step.
                    const int cnt = (int)walk.cnt;
                    if (me == 0) {
                        issued = true;
                        for (int j = 0; j < cnt; ++j) {
                            const uint32_t t = wt + (uint32_t)j, use = t / (uint32_t)kAcc;
                            if (use > 0) mbar_wait(smem_u32(&bar_acc_empty[t & (uint32_t)(kAcc - 1)]), (use - 1) & 1, abort_flag, g.status, g.wait_limit);
                        }
                        // all pieces of the group: the transform warps finish them in order; without a
                        // transform the copies land in any order
                        if (MODE == SPARQ_MODE_NONE) {
                            for (int j = 0; j < cnt; ++j)
                                mbar_wait(smem_u32(&bar_win_full[b * kMaxG + j]), wph, abort_flag, g.status, g.wait_limit);
                        } else {
                            mbar_wait(smem_u32(&bar_win_xf[b * kMaxG + cnt - 1]), wph, abort_flag, g.status, g.wait_limit);
                        }
                        tc_fence_after();
                        uint64_t a_cb = a_grp;
                        for (uint32_t cb = 0; cb < (uint32_t)g.c_blocks; ++cb, a_cb += plane16) {
                            uint64_t a_r = a_cb;
                            for (int r = 0; r < g.R; ++r, a_r += row16) {
                                for (int sx = 0; sx < g.S; ++sx) {
                                    mbar_wait(smem_u32(&bar_b_full[s]), bph, abort_flag, g.status, g.wait_limit);
                                    tc_fence_after();
                                    const uint64_t bdesc = b_desc0 + (uint64_t)((uint32_t)s * (uint32_t)(kBBlock >> 4));
                                    const uint64_t a_tap = a_r + (uint64_t)(uint32_t)(sx * (CB >> 4));
                                    const uint32_t first = (cb == 0 && r == 0 && sx == 0) ? 0u : 1u;
                                    for (int j = 0; j < cnt; ++j) {
                                        const uint32_t d_tmem = tmem_base + ((wt + (uint32_t)j) & (uint32_t)(kAcc - 1)) * (uint32_t)BN;
                                        const uint64_t adesc = a_tap + (uint64_t)((uint32_t)j * tile16);
#pragma unroll
                                        for (int k = 0; k < CB / 32; ++k)
                                            tc_mma_i8_if(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                                                         (first || k > 0) ? 1u : 0u, elected);
                                    }
                                    tc_commit_if(smem_u32(&bar_b_empty[s]), elected);
                                    if (++s == g.b_stages) { s = 0; bph ^= 1u; }
                                }
                            }
                        }
                        for (int j = 0; j < cnt; ++j)
                            tc_commit_if(smem_u32(&bar_acc_full[(wt + (uint32_t)j) & (uint32_t)(kAcc - 1)]), elected);
                    }
                    wt += (uint32_t)cnt;
                } else
                for (int j = 0; j < (int)walk.cnt; ++j, ++wt) {
                    if (g.issuers == 2 ? (wt & 1u) != me : me != 0u) {
                        if (!B_RESIDENT) {
                            // the other issuer consumes this tile's weight stages
                            s += kb_count;
                            while (s >= g.b_stages) { s -= g.b_stages; bph ^= 1u; }
                        }
                        continue;
                    }
                    issued = true;
                    const uint32_t acc = wt & (uint32_t)(kAcc - 1);
                    const uint32_t acc_use = wt / (uint32_t)kAcc;
                    const uint32_t d_tmem = tmem_base + acc * (uint32_t)BN;
                    if (acc_use > 0 && !pre_acc) mbar_wait(smem_u32(&bar_acc_empty[acc]), (acc_use - 1) & 1, abort_flag, g.status, g.wait_limit);
                    // Tile j reads pieces 0..j.  The transform warps finish pieces in order, so with
                    // a transform piece j's barrier covers the earlier ones.  Without one the copies
                    // land in any order: this issuer waits for pieces j-1 and j (its previous tile
                    // of the group, j-2, waited for the two before).
                    const uint32_t ops_bar = smem_u32(MODE == SPARQ_MODE_NONE ? &bar_win_full[b * kMaxG + j] : &bar_win_xf[b * kMaxG + j]);
                    if (!pre_ops) {
                        if (MODE == SPARQ_MODE_NONE && j > 0) mbar_wait(ops_bar - 8u, wph, abort_flag, g.status, g.wait_limit);
                        mbar_wait(ops_bar, wph, abort_flag, g.status, g.wait_limit);
                    }
                    tc_fence_after();
                    pre_acc = pre_ops = 0;
                    const uint32_t step = (uint32_t)g.issuers;          // this issuer's next tile is number wt + step
                    const bool look_ahead = j + (int)step < (int)walk.cnt;
                    auto look = [&]() {
                        if (!look_ahead) return;
                        // a stage's first use needs no wait (the piece barrier stands in for it in the look)
                        const uint32_t nacc = (wt + step) & (uint32_t)(kAcc - 1), nuse = (wt + step) / (uint32_t)kAcc;
                        const uint32_t m = mbar_test3(nuse ? smem_u32(&bar_acc_empty[nacc]) : ops_bar, nuse ? (nuse - 1u) & 1u : wph,
                                                      ops_bar + 8u, wph, ops_bar + 8u * step, wph);
                        pre_acc = nuse ? (m & 1u) : 1u;
                        pre_ops = (MODE == SPARQ_MODE_NONE) ? (uint32_t)((m & 6u) == 6u) : (m >> 2);
                    };
                    const uint64_t a_desc0 = a_grp + (uint64_t)((uint32_t)j * tile16);
                    // One (tap, channel block) of the tile: wait for its weights when they are
                    // streamed, then CB / 32 MMAs.  The descriptors are sums of warp-uniform
                    // loop-carried values (no table, no division), so the address arithmetic of
                    // consecutive MMAs is a couple of adds.
                    auto issue_block = [&](const bool first, const uint32_t slot, const uint64_t adesc) {
                        uint64_t bdesc;
                        if (B_RESIDENT) {
                            bdesc = b_desc0 + (uint64_t)(slot * (uint32_t)(kBBlock >> 4));
                        } else {
                            mbar_wait(smem_u32(&bar_b_full[s]), bph, abort_flag, g.status, g.wait_limit);
                            tc_fence_after();
                            bdesc = b_desc0 + (uint64_t)((uint32_t)s * (uint32_t)(kBBlock >> 4));
                        }
#pragma unroll
                        for (int k = 0; k < CB / 32; ++k)
                            tc_mma_i8_if(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                                         (!first || k > 0) ? 1u : 0u, elected);
                        if (!B_RESIDENT) {
                            tc_commit_if(smem_u32(&bar_b_empty[s]), elected);
                            if (++s == g.b_stages) { s = 0; bph ^= 1u; }
                        }
                    };
                    // channel block outer, tap inner; the resident slot of (tap, cb) is tap * c_blocks + cb
                    uint64_t a_cb = a_desc0;
                    const uint32_t cbs = (uint32_t)g.c_blocks;
                    if (g.R == 3 && g.S == 3) {
                        for (uint32_t cb = 0; cb < cbs; ++cb, a_cb += plane16) {
#pragma unroll
                            for (int r = 0; r < 3; ++r) {
#pragma unroll
                                for (int sx = 0; sx < 3; ++sx)
                                    issue_block(cb == 0 && r == 0 && sx == 0, (uint32_t)(r * 3 + sx) * cbs + cb,
                                                a_cb + (uint64_t)((uint32_t)r * row16 + (uint32_t)(sx * (CB >> 4))));
                                if (r == 0 && cb == 0) look();
                            }
                        }
                    } else {
                        for (uint32_t cb = 0; cb < cbs; ++cb, a_cb += plane16) {
                            uint64_t a_r = a_cb;
                            uint32_t slot = cb;
                            for (int r = 0; r < g.R; ++r, a_r += row16) {
                                for (int sx = 0; sx < g.S; ++sx, slot += cbs)
                                    issue_block(cb == 0 && r == 0 && sx == 0, slot, a_r + (uint64_t)(uint32_t)(sx * (CB >> 4)));
                                if (r == 0 && cb == 0) look();
                            }
                        }
                    }
                    tc_commit_if(smem_u32(&bar_acc_full[acc]), elected);      // accumulator complete
                }
                // The buffer goes back to the producer once both issuers have arrived and their
                // MMAs have retired.  With a transform, first make sure that every transform warp
                // is past all of this use's barriers (they arrive on the last piece's barrier
                // last), so that none of them can still be waiting on a phase when the producer
                // starts the next.
                if (MODE != SPARQ_MODE_NONE && (int)walk.cnt < g.G)
                    mbar_wait(smem_u32(&bar_win_xf[b * kMaxG + g.G - 1]), wph, abort_flag, g.status, g.wait_limit);
                if (issued) {
                    tc_commit_if(smem_u32(&bar_win_empty[b]), elected);
                } else {
                    // No tile of this group was this issuer's.  It arrives only once the producer has
                    // started this use of the buffer (its first piece has landed), i.e. after the
                    // previous use's phase of the barrier has completed.
                    mbar_wait(smem_u32(&bar_win_full[b * kMaxG]), wph, abort_flag, g.status, g.wait_limit);
                    if (elected) mbar_arrive(smem_u32(&bar_win_empty[b]));
                }
                ++gi;
            if (++rb == g.win_bufs) { rb = 0; ++ruse; }
            }
            // all tensor-core work of this CTA has retired before tensor memory is freed
            tc_commit_if(smem_u32(&bar_done), elected);
            mbar_wait(smem_u32(&bar_done), 0, abort_flag, g.status, g.wait_limit, true);
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
        // 64-wide tiles have one column tile and 16 or 32 columns per warp.  When only the
        // requantized bytes are wanted (the form every layer of a network uses), the warp keeps
        // the scale and bias of its columns in registers for the whole launch -- shared-memory
        // reads queue behind the tensor core's operand fetches -- and takes the accumulator in
        // 16-column pieces so that those registers fit beside it.
        if (epi_teams) {
            constexpr int kTeamWarps = kEpi / 2;
            constexpr int kTeamCols = BN / (kTeamWarps / 4);      // columns per warp
            epi_stage_scale_bias<kEpi>(g, 0, BN, et, s_scale, s_bias);
            const uint32_t team = (uint32_t)(warp - kFirstEpiWarp) / kTeamWarps;     // team t takes the tiles of parity t (kAcc is even)
            const int cbase = (((warp - kFirstEpiWarp) % kTeamWarps) >> 2) * kTeamCols;
            for (; have; have = walk.next()) {
                for (int j = 0; j < (int)walk.cnt; ++j, ++wt) {
                    if ((wt & 1u) != team) continue;
                    const int oh = ((int)walk.tin + j) * g.TR + tr;
                    const bool row_ok = slot_ok && (oh < g.Ho);
                    const int64_t row = ((int64_t)walk.img * g.Ho + oh) * g.Wo + ow;
                    const uint32_t acc = wt & (uint32_t)(kAcc - 1);
                    const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + (uint32_t)cbase;
                    mbar_wait(smem_u32(&bar_acc_full[acc]), (wt / (uint32_t)kAcc) & 1u, abort_flag, g.status, g.wait_limit);
                    tc_fence_after();
#pragma unroll 1
                    for (int ch = 0; ch < kTeamCols / 32; ++ch) {
                        uint32_t v[32];
                        tmem_ld_32x32_issue(taddr0 + (uint32_t)(ch * 32), v);
                        tmem_ld_wait();
                        if (ch + 1 == kTeamCols / 32) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
                        }
                        const int ct = cbase + ch * 32;
                        if (!row_ok || ct >= (int)g.N) continue;       // N is a multiple of 32 here
                        if (ev.small_acc) epi_chunk_u8<true>(ev, v, row, ct, ct, s_scale, s_bias);
                        else epi_chunk_u8<false>(ev, v, row, ct, ct, s_scale, s_bias);
                    }
                }
            }
        } else
        if (BN == 64 && ev.need_f && !g.acc_out && !g.f32_out && !g.residual && g.N == 64) {
            epi_stage_scale_bias<kEpi>(g, 0, BN, et, s_scale, s_bias);
            const int cbase = part * kColsPerWarp;
            float rs[kColsPerWarp], rb[kColsPerWarp];
#pragma unroll
            for (int i = 0; i < kColsPerWarp; ++i) {
                rs[i] = s_scale[cbase + i];
                rb[i] = s_bias[cbase + i];
            }
            uint32_t pre_full = 0;     // the next tile's accumulator was seen complete
            for (; have; have = walk.next()) {
              for (int j = 0; j < (int)walk.cnt; ++j, ++wt) {
                const uint32_t acc = wt & (uint32_t)(kAcc - 1);
                // coordinates first: they do not depend on the accumulator
                const int oh = ((int)walk.tin + j) * g.TR + tr;
                const bool row_ok = slot_ok && (oh < g.Ho);
                uint8_t *dst = g.u8_out + (((int64_t)walk.img * g.Ho + oh) * g.Wo + ow) * 64 + cbase;
                const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + (uint32_t)cbase;
                if (!pre_full) mbar_wait(smem_u32(&bar_acc_full[acc]), (wt / (uint32_t)kAcc) & 1u, abort_flag, g.status, g.wait_limit);
                tc_fence_after();
                pre_full = 0;
#pragma unroll
                for (int hh = 0; hh < kColsPerWarp / 16; ++hh) {
                    uint32_t v[16];
                    tmem_ld_32x16_issue(taddr0 + (uint32_t)(hh * 16), v);
                    // While the load is in flight: has the next tile of the group been accumulated
                    // already?  A barrier read takes hundreds of cycles behind the tensor core's
                    // shared-memory traffic; here it overlaps the tensor-memory load, and a "yes"
                    // lets the next tile start without one.
                    if (hh == 0 && j + 1 < (int)walk.cnt)
                        pre_full = mbar_test(smem_u32(&bar_acc_full[(wt + 1u) & (uint32_t)(kAcc - 1)]), ((wt + 1u) / (uint32_t)kAcc) & 1u);
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
                        float z[4];
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {
                            const int c = hh * 16 + 4 * q + jj;
                            const float y = ev.small_acc ? dequant<true>((int32_t)v[4 * q + jj], rs[c], rb[c], ev.relu_op)
                                                         : dequant<false>((int32_t)v[4 * q + jj], rs[c], rb[c], ev.relu_op);
                            z[jj] = __fmul_rn(y, ev.inv_out_scale);
                        }
                        w[q] = requant_pack4(z[0], z[1], z[2], z[3]);
                    }
                    if (ev.next_mode != SPARQ_MODE_NONE) next_xform_words(w, 4, ev.next_mode, ev.next_rnd, ev.next_xf);
                    *reinterpret_cast<uint4 *>(dst + hh * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                }
              }
            }
        } else
        for (; have; have = walk.next()) {
          for (int j = 0; j < (int)walk.cnt; ++j, ++wt) {
            const int64_t nt = (int64_t)walk.nt;
            const int acc = (int)(wt & (uint32_t)(kAcc - 1));
            const uint32_t acc_use = wt / (uint32_t)kAcc;
            if (ev.need_f && nt != staged_nt) {
                staged_nt = nt;
                epi_stage_scale_bias<kEpi>(g, nt * BN, BN, et, s_scale, s_bias);
            }
            mbar_wait(smem_u32(&bar_acc_full[acc]), acc_use & 1, abort_flag, g.status, g.wait_limit);
            tc_fence_after();
            const int oh = ((int)walk.tin + j) * g.TR + tr;
            const bool row_ok = slot_ok && (oh < g.Ho);
            const int64_t row = ((int64_t)walk.img * g.Ho + oh) * g.Wo + ow;
            const int cbase = part * kColsPerWarp;
            const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + cbase);
            epi_warp_columns<kColsPerWarp>(ev, taddr0, cbase, row, row_ok, nt * BN, s_scale, s_bias,
                                      smem_u32(&bar_acc_empty[acc]), lane);
          }
        }
    } else if (MODE != SPARQ_MODE_NONE) {
        // ================= transform: once per piece =================
        const uint32_t xt = threadIdx.x - kFirstXfWarp * 32;
        constexpr uint32_t kXfThreads = kNumXfWarps * 32;
        const XformDev xf = g.xf;
        uint32_t gi = 0;
        int rb = 0; uint32_t ruse = 0;         // window buffer of the group (gi % win_bufs) and its use count (gi / win_bufs)
        for (; have; have = walk.next()) {
            const int b = rb;
            const uint32_t wph = ruse & 1u;
            for (int j = 0; j < g.G; ++j) {
                mbar_wait(smem_u32(&bar_win_full[b * kMaxG + j]), wph, abort_flag, g.status, g.wait_limit);
                if (j < (int)walk.cnt) {
                    const uint32_t nvec = piece_len(j) >> 4;
                    uint32_t pbase = win_buf(b) + piece_off(j);
                    for (int cb = 0; cb < g.c_blocks; ++cb, pbase += (uint32_t)g.plane_bytes) {
                        // four independent 16-byte vectors per thread and step; the last step of a
                        // piece may be short
                        for (uint32_t v0 = xt; v0 < nvec; v0 += 4 * kXfThreads) {
                            uint4 v[4];
                            bool ok[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                ok[q] = v0 + (uint32_t)q * kXfThreads < nvec;
                                if (ok[q])
                                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                                 : "=r"(v[q].x), "=r"(v[q].y), "=r"(v[q].z), "=r"(v[q].w)
                                                 : "r"(pbase + (v0 + (uint32_t)q * kXfThreads) * 16u));
                            }
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                if (!ok[q]) continue;
                                v[q].x = xform_fused<MODE, XN, RND>(v[q].x, xf);
                                v[q].y = xform_fused<MODE, XN, RND>(v[q].y, xf);
                                v[q].z = xform_fused<MODE, XN, RND>(v[q].z, xf);
                                v[q].w = xform_fused<MODE, XN, RND>(v[q].w, xf);
                                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};"
                                             :: "r"(pbase + (v0 + (uint32_t)q * kXfThreads) * 16u),
                                                "r"(v[q].x), "r"(v[q].y), "r"(v[q].z), "r"(v[q].w) : "memory");
                            }
                        }
                    }
                    fence_proxy_async_smem();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_win_xf[b * kMaxG + j]));
            }
            ++gi;
            if (++rb == g.win_bufs) { rb = 0; ++ruse; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     :: "r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

template <int BN, int CB, bool B_RESIDENT>
cudaError_t launch_window_shape(const CUtensorMap &mx0, const CUtensorMap &mx1, const CUtensorMap &mw, const WindowArgs &g,
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
        return launch_pdl<kWindowThreads>(kfn, grid, smem_bytes, st, mx0, mx1, mw, g);                                       \
    } while (0)

#define SPARQ_DEFINE_WINDOW_SHAPE(BN_, CB_, RES_)                                                      \
    template <>                                                                                        \
    cudaError_t launch_window_shape<BN_, CB_, RES_>(const CUtensorMap &mx0, const CUtensorMap &mx1,    \
                                                    const CUtensorMap &mw,                             \
                                                    const WindowArgs &g, int mode, int n, int rnd,     \
                                                    int grid, int smem_bytes, cudaStream_t st)         \
    {                                                                                                  \
        constexpr int BN = BN_, CB = CB_;                                                              \
        constexpr bool RES = RES_;                                                                     \
        if (mode == SPARQ_MODE_NONE) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_NONE, 4, false);           \
        if (mode == SPARQ_MODE_BSPARQ) {                                                               \
            if (n == 8) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 8, true);                       \
            if (n == 4) { if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 4, true);            \
                          else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 4, false); }             \
            if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 0, true);                          \
            else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_BSPARQ, 0, false);                             \
        }                                                                                              \
        if (n == 8) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 8, true);                           \
        if (n == 4) { if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 4, true);                \
                      else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 4, false); }                 \
        if (rnd) SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 0, true);                              \
        else SPARQ_LAUNCH_WINDOW_VARIANT(SPARQ_MODE_VSPARQ, 0, false);                                 \
    }

}  // namespace sparq
