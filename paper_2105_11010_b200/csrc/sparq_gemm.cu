// Host side of the fused entry points: validation, tile-shape choice, TMA tensor maps
// (tiled for the GEMM view, im2col for the convolution), launch.
#include <cuda.h>

#include <cstdlib>
#include <cstring>
#include <mutex>

#include "sparq_conv_window_kernel.cuh"

namespace sparq {


// Limit of the device-side waits of every fused launch, in SM cycles.
static long long g_wait_limit = kWaitLimitCycles;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static int driver_fn(const char *name, void **fn)
{
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPointByVersion(name, fn, 12000, cudaEnableDefault, &q);
    if (e != cudaSuccess) return cuda_error(e, name);
    if (q != cudaDriverEntryPointSuccess || !*fn)
        return set_error(SPARQ_ERR_CUDA, "driver entry point %s is unavailable", name);
    return SPARQ_OK;
}

static CUtensorMapSwizzle swizzle_for(int bk) { return bk == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B; }

// A tensor map is a pure function of the arguments it is encoded from (address, extents,
// strides, box, swizzle), and encoding one costs the host several microseconds -- as much as
// a small layer takes on the device.  Networks call the same layers with the same buffers
// over and over, so encoded maps are kept in a small direct-mapped table keyed by those
// arguments.  Host memory only; nothing to release.
struct MapKey {
    uint64_t v[14];
    bool operator==(const MapKey &o) const { return memcmp(v, o.v, sizeof(v)) == 0; }
};
struct MapSlot { bool used; MapKey key; CUtensorMap map; };
constexpr int kMapSlots = 256;
static MapSlot g_map_cache[kMapSlots];
static std::mutex g_map_mutex;

// Forgets the cached tensor maps (host memory only; they are re-encoded on demand).
void release_gemm_state()
{
    std::lock_guard<std::mutex> lock(g_map_mutex);
    for (MapSlot &s : g_map_cache) s.used = false;
}

static unsigned map_hash(const MapKey &k)
{
    uint64_t h = 1469598103934665603ull;
    for (uint64_t x : k.v) { h ^= x; h *= 1099511628211ull; h ^= h >> 29; }
    return (unsigned)(h % kMapSlots);
}
static bool map_lookup(const MapKey &k, CUtensorMap *out)
{
    std::lock_guard<std::mutex> lock(g_map_mutex);
    const MapSlot &s = g_map_cache[map_hash(k)];
    if (!s.used || !(s.key == k)) return false;
    *out = s.map;
    return true;
}
static void map_store(const MapKey &k, const CUtensorMap &m)
{
    std::lock_guard<std::mutex> lock(g_map_mutex);
    MapSlot &s = g_map_cache[map_hash(k)];
    s.used = true; s.key = k; s.map = m;
}

// 2-D K-contiguous matrix [rows][K] with row pitch ld bytes; box = bk x box_rows.
static int encode_2d(CUtensorMap *map, const void *ptr, int64_t K, int64_t rows, int64_t ld, int bk, int box_rows)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        int rc = driver_fn("cuTensorMapEncodeTiled", (void **)&fn);
        if (rc != SPARQ_OK) return rc;
    }
    const MapKey key = {{1, (uint64_t)(uintptr_t)ptr, (uint64_t)K, (uint64_t)rows, (uint64_t)ld, (uint64_t)bk, (uint64_t)box_rows}};
    if (map_lookup(key, map)) return SPARQ_OK;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {(cuuint32_t)bk, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(bk), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(SPARQ_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    map_store(key, *map);
    return SPARQ_OK;
}

// NHWC activation tensor read as im2col columns of 128 output pixels x bk channels.
static int encode_im2col(CUtensorMap *map, const void *ptr, int n, int h, int w, int c, int r, int s,
                         int stride_h, int stride_w, int pad_h, int pad_w, int bk)
{
    static EncodeIm2colFn fn = nullptr;
    if (!fn) {
        int rc = driver_fn("cuTensorMapEncodeIm2col", (void **)&fn);
        if (rc != SPARQ_OK) return rc;
    }
    const MapKey key = {{2, (uint64_t)(uintptr_t)ptr, (uint64_t)n, (uint64_t)h, (uint64_t)w, (uint64_t)c, (uint64_t)r, (uint64_t)s,
                         (uint64_t)stride_h, (uint64_t)stride_w, (uint64_t)(int64_t)pad_h, (uint64_t)(int64_t)pad_w, (uint64_t)bk}};
    if (map_lookup(key, map)) return SPARQ_OK;
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {(cuuint64_t)c, (cuuint64_t)c * w, (cuuint64_t)c * w * h};
    // Base pixels (the filter's top-left tap) run from -pad to dim - 1 + upper.
    int lower[2] = {-pad_w, -pad_h};
    int upper[2] = {pad_w - (s - 1), pad_h - (r - 1)};
    cuuint32_t estr[4] = {1, (cuuint32_t)stride_w, (cuuint32_t)stride_h, 1};
    CUresult res = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(ptr), dims, strides, lower, upper,
                      (cuuint32_t)bk, (cuuint32_t)kBM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(bk),
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (res != CUDA_SUCCESS) return set_error(SPARQ_ERR_CUDA, "cuTensorMapEncodeIm2col failed with CUresult %d", (int)res);
    map_store(key, *map);
    return SPARQ_OK;
}

static int device_info(int *sms)
{
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_error(e, "device query");
    if (major != 10) return set_error(SPARQ_ERR_UNSUPPORTED, "the fused kernels need an sm_100 device (found sm_%d0)", major);
    return SPARQ_OK;
}

// Validates e->next_transform and turns it into kernel arguments (mode NONE when absent).
static int next_transform_args(const sparq_epilogue *e, int64_t N, int *mode, int *rnd, XformDev *xf)
{
    *mode = SPARQ_MODE_NONE;
    *rnd = 0;
    *xf = XformDev{0u, 0, 4};
    fill_fullset(xf, 4, 0);
    if (!e->next_transform || e->next_transform->mode == SPARQ_MODE_NONE) return SPARQ_OK;
    XformArgs nx;
    int rc = validate_params(e->next_transform, &nx);
    if (rc != SPARQ_OK) return rc;
    if (!e->u8_out) return set_error(SPARQ_ERR_INVALID_ARG, "next_transform needs u8_out");
    if (N % 4) return set_error(SPARQ_ERR_UNSUPPORTED, "next_transform needs N (%lld) to be a multiple of 4", (long long)N);
    *mode = nx.mode;
    *rnd = nx.rnd;
    *xf = XformDev{nx.widen_c, nx.widen_rounds, nx.n};
    fill_fullset(xf, nx.n, nx.rnd);
    return SPARQ_OK;
}

static int check_epilogue(const sparq_epilogue *e)
{
    if (!e) return set_error(SPARQ_ERR_INVALID_ARG, "sparq_epilogue is NULL");
    if (!e->acc_out && !e->f32_out && !e->u8_out)
        return set_error(SPARQ_ERR_INVALID_ARG, "no output requested (acc_out, f32_out and u8_out are all NULL)");
    if ((e->f32_out || e->u8_out) && !e->scale)
        return set_error(SPARQ_ERR_INVALID_ARG, "scale is NULL but a dequantized output is requested");
    if ((e->acc_out && ((uintptr_t)e->acc_out & 15u)) || (e->f32_out && ((uintptr_t)e->f32_out & 15u)) ||
        (e->u8_out && ((uintptr_t)e->u8_out & 15u)))
        return set_error(SPARQ_ERR_UNSUPPORTED, "output pointers must be 16-byte aligned");
    if (e->residual) {
        if (!e->f32_out && !e->u8_out)
            return set_error(SPARQ_ERR_INVALID_ARG, "residual needs a dequantized output (f32_out or u8_out)");
        if ((uintptr_t)e->residual & 15u)
            return set_error(SPARQ_ERR_UNSUPPORTED, "residual must be 16-byte aligned");
    }
    return SPARQ_OK;
}

// Tile width for the 128 x BN kernel.  Per reduction step (128 bytes of K) a CTA needs about
//   max( transform of the A stage  ~1250 cycles when a SPARQ mode is on,
//        MMA                       2 * BN cycles,
//        operand fetch from L2     ~4.4 cycles per 128-byte row of A and B )
// and the kernel takes ceil(tiles / SMs) such passes; narrow tiles add CTAs but re-fetch
// and re-transform A once per column tile.  Pick the width with the lowest estimate.
static int pick_bn(int64_t M, int64_t N, int sms, bool transform)
{
    const int cand[3] = {256, 128, 64};
    const int64_t m_tiles = (M + kBM - 1) / kBM;
    int best = 64;
    double best_cost = 0.0;
    for (int i = 0; i < 3; ++i) {
        const int bn = cand[i];
        if (bn > 64 && N <= bn / 2) continue;          // would be mostly padding
        const int64_t tiles = m_tiles * ((N + bn - 1) / bn);
        const int64_t rounds = (tiles + sms - 1) / sms;
        double step = 2.0 * bn;
        const double fetch = 4.4 * (kBM + bn);
        if (fetch > step) step = fetch;
        if (transform && step < 1250.0) step = 1250.0;
        const double cost = (double)rounds * (step + 150.0);   // + fixed per-step hand-off cost
        if (best_cost == 0.0 || cost < best_cost) {
            best_cost = cost;
            best = bn;
        }
    }
    return best;
}

// ---- what the previous fused launch on a stream wrote ---------------------------------------------
// The fused kernels are launched with programmatic stream serialization and let their successor
// start early; a successor may fetch its WEIGHTS before it waits for them -- provided the weights
// are not among their outputs.  Every fused launch records its output ranges per (device,
// stream) here and learns whether its own weights are clear of the previous launch's.  Kernels
// of other libraries never release their successor early, so only these launches matter.  A
// stream that is not in the table (first launch, or evicted) counts as "not clear".
struct LastLaunch {
    bool used;
    int dev;
    cudaStream_t stream;
    uint64_t age;
    uintptr_t lo[3], hi[3];
};
constexpr int kLastSlots = 32;
static LastLaunch g_last[kLastSlots];
static uint64_t g_last_age = 0;
static std::mutex g_last_mutex;

static bool record_launch_weights_clear(cudaStream_t st, const sparq_epilogue *e, size_t out_elems, const void *wgt, size_t wgt_bytes)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
    std::lock_guard<std::mutex> lock(g_last_mutex);
    LastLaunch *slot = nullptr, *oldest = &g_last[0];
    for (LastLaunch &l : g_last) {
        if (l.used && l.dev == dev && l.stream == st) { slot = &l; break; }
        if (!l.used || l.age < oldest->age || oldest->used && !l.used) oldest = &l;
    }
    bool clear = false;
    if (slot) {
        clear = true;
        const uintptr_t w0 = (uintptr_t)wgt, w1 = w0 + wgt_bytes;
        for (int i = 0; i < 3; ++i)
            if (slot->lo[i] < w1 && w0 < slot->hi[i]) clear = false;
    } else {
        slot = oldest;
    }
    const void *outs[3] = {e->acc_out, e->f32_out, e->u8_out};
    const size_t width[3] = {4, 4, 1};
    slot->used = true; slot->dev = dev; slot->stream = st; slot->age = ++g_last_age;
    for (int i = 0; i < 3; ++i) {
        slot->lo[i] = (uintptr_t)outs[i];
        slot->hi[i] = outs[i] ? (uintptr_t)outs[i] + out_elems * width[i] : 0;
    }
    return clear;
}

// Variant argument of the launchers: 4 = n = 4 with all five placements, 8 = another full
// placement set (6opt, 7opt), 0 = the general kernels.
static int variant_n(const XformArgs &x) { return x.widen_rounds != 0 ? 0 : (x.n == 4 ? 4 : 8); }

// Kernel-side transform constants.
static XformDev xform_dev(const XformArgs &x)
{
    XformDev d{x.widen_c, x.widen_rounds, x.n};
    fill_fullset(&d, x.n, x.rnd);
    return d;
}

static cudaError_t launch(int bn, int bk, const CUtensorMap &ma, const CUtensorMap &mb, const GemmArgs &g,
                          const XformArgs &x, int grid, cudaStream_t st)
{
    if (bn == 64 && bk == 64) return launch_gemm_shape<64, 64>(ma, mb, g, x.mode, variant_n(x), x.rnd, grid, st);
    if (bn == 64) return launch_gemm_shape<64, 128>(ma, mb, g, x.mode, variant_n(x), x.rnd, grid, st);
    if (bn == 128 && bk == 64) return launch_gemm_shape<128, 64>(ma, mb, g, x.mode, variant_n(x), x.rnd, grid, st);
    if (bn == 128) return launch_gemm_shape<128, 128>(ma, mb, g, x.mode, variant_n(x), x.rnd, grid, st);
    if (bk == 64) return launch_gemm_shape<256, 64>(ma, mb, g, x.mode, variant_n(x), x.rnd, grid, st);
    return launch_gemm_shape<256, 128>(ma, mb, g, x.mode, variant_n(x), x.rnd, grid, st);
}

static int fill_common(GemmArgs *g, const XformArgs &x, const sparq_epilogue *e, unsigned int *status)
{
    g->xf = xform_dev(x);
    g->scale = e->scale;
    g->bias = e->bias;
    g->relu = e->relu ? 1 : 0;
    g->inv_out_scale = e->inv_out_scale;
    g->acc_out = e->acc_out;
    g->f32_out = e->f32_out;
    g->u8_out = e->u8_out;
    g->status = status;
    g->wait_limit = g_wait_limit;
    g->residual = e->residual;
    g->residual_scale = e->residual_scale;
    return next_transform_args(e, g->N, &g->next_mode, &g->next_rnd, &g->next_xf);
}

int gemm_with_status(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb, int64_t M, int64_t N, int64_t K,
                     const XformArgs &x, const sparq_epilogue *e, unsigned int *status, cudaStream_t st);

// The fused GEMM with the library's own status word (allocated on first use).
static int gemm_impl(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb, int64_t M, int64_t N, int64_t K,
                     const XformArgs &x, const sparq_epilogue *e, cudaStream_t st)
{
    unsigned int *status = nullptr;
    int rc = get_status_word(&status);
    if (rc != SPARQ_OK) return rc;
    return gemm_with_status(A, lda, B, ldb, M, N, K, x, e, status, st);
}

// NHWC activation tensor read as a box of cb channels x wp columns x rows input rows of one
// image (zero fill outside the image).
static int encode_window(CUtensorMap *map, const void *ptr, int n, int h, int w, int c, int cb, int wp, int rows)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        int rc = driver_fn("cuTensorMapEncodeTiled", (void **)&fn);
        if (rc != SPARQ_OK) return rc;
    }
    const MapKey key = {{3, (uint64_t)(uintptr_t)ptr, (uint64_t)n, (uint64_t)h, (uint64_t)w, (uint64_t)c, (uint64_t)cb, (uint64_t)wp, (uint64_t)rows}};
    if (map_lookup(key, map)) return SPARQ_OK;
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {(cuuint64_t)c, (cuuint64_t)c * w, (cuuint64_t)c * w * h};
    cuuint32_t box[4] = {(cuuint32_t)cb, (cuuint32_t)wp, (cuuint32_t)rows, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(cb), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(SPARQ_ERR_CUDA, "cuTensorMapEncodeTiled (window) failed with CUresult %d", (int)r);
    map_store(key, *map);
    return SPARQ_OK;
}

// Weights [cout][K] seen as (cb bytes, cout rows, K / cb blocks): one box brings every
// (tap, channel block) of bn filters into consecutive bn x cb shared-memory blocks.
// Returns the driver's result; the caller falls back to one copy per block if it is refused.
static CUresult encode_weight_blocks(CUtensorMap *map, const void *ptr, int64_t K, int cout, int cb, int bn, int blocks)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn && driver_fn("cuTensorMapEncodeTiled", (void **)&fn) != SPARQ_OK) return CUDA_ERROR_NOT_FOUND;
    const MapKey key = {{4, (uint64_t)(uintptr_t)ptr, (uint64_t)K, (uint64_t)cout, (uint64_t)cb, (uint64_t)bn, (uint64_t)blocks}};
    if (map_lookup(key, map)) return CUDA_SUCCESS;
    cuuint64_t dims[3] = {(cuuint64_t)cb, (cuuint64_t)cout, (cuuint64_t)blocks};
    cuuint64_t strides[2] = {(cuuint64_t)K, (cuuint64_t)cb};
    cuuint32_t box[3] = {(cuuint32_t)cb, (cuuint32_t)bn, (cuuint32_t)blocks};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(cb), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r == CUDA_SUCCESS) map_store(key, *map);
    return r;
}

constexpr int kMaxDynSmem = kWindowMaxDynSmem;

// Stride-1 filters larger than 1x1: the window kernel, when its tiling fits.  Returns
// 1 if it launched, 0 if the shape should take the im2col kernel, < 0 on error.
static int try_window_conv(const uint8_t *x_in, int n, int h, int w, int c, const int8_t *wgt, int cout, int r, int s,
                           int pad_h, int pad_w, int ho, int wo, const XformArgs &x, const sparq_epilogue *e,
                           int sms, unsigned int *status, cudaStream_t st)
{
    const int wp = w + 2 * pad_w;
    if (wp > 128 || wo < 1) return 0;
    const int cb = (c % 128 == 0) ? 128 : (c == 64 ? 64 : 0);
    if (!cb) return 0;
    int tr = 128 / wp;
    if (tr > ho) tr = ho;
    if (tr < 1 || tr * wo < 64) return 0;               // less than half of the MMA rows would be useful
    const int c_blocks = c / cb;
    const int taps = r * s;
    const int kb_count = taps * c_blocks;
    const int tiles_per_img = (ho + tr - 1) / tr;
    const int64_t m_tiles = (int64_t)n * tiles_per_img;

    int bn;
    if (cb == 64) {
        if (cout > 64) return 0;
        bn = 64;
    } else {
        if (cout <= 64) return 0;
        bn = (cout > 128 && m_tiles * ((cout + 255) / 256) >= sms) ? 256 : 128;
    }
    const int b_block = bn * cb;
    const int n_tiles = (cout + bn - 1) / bn;
    const int64_t units = m_tiles * n_tiles;
    if (units >= (int64_t)1 << 31) return 0;
    int grid = (int)(units < sms ? units : sms);

    // Shared memory of one window buffer when up to `grp` tiles share it: a plane (one channel
    // block) holds every row the MMA of the group's last tile may touch.
    auto plane_for = [&](int grp) {
        const int rows_alloc = (grp - 1) * tr * wp + (r - 1) * wp + (s - 1) + 128;
        return (rows_alloc * cb + 1023) / 1024 * 1024;
    };
    // Tiles per group: with one column tile, as many as a CTA's share of the tile sequence
    // has (more would never be used) while two window buffers still fit beside the weights.
    // A later piece must land on a 128-byte boundary (TMA destination alignment).
    int gmax = 1;
    if (n_tiles == 1) {
        gmax = (int)((units + grid - 1) / grid);
        if (gmax > tiles_per_img) gmax = tiles_per_img;
        if (gmax > kMaxG) gmax = kMaxG;
        if (cb == 64 && (((tr * wp) & 1) || (((r - 1) * wp) & 1))) gmax = 1;
    }
    bool resident = false, batched = false;
    int win_bufs = 2, b_stages = 0, grp = 1;
    if (bn != 256 && n_tiles == 1 && 1024 + 2 * plane_for(1) * c_blocks + kb_count * b_block <= kMaxDynSmem) {
        resident = true;
        b_stages = kb_count;
        grp = gmax;
        while (grp > 1 && 1024 + 2 * plane_for(grp) * c_blocks + kb_count * b_block > kMaxDynSmem) --grp;
        // more buffers only help while a CTA has more groups than buffers
        const int groups_per_cta = (int)((units + grid - 1) / grid + grp - 1) / grp + 1;
        while (win_bufs < kMaxWinBufs && win_bufs < groups_per_cta &&
               1024 + (win_bufs + 1) * plane_for(grp) * c_blocks + kb_count * b_block <= kMaxDynSmem) ++win_bufs;
    } else {
        if (bn == 64) return 0;                          // only the resident form is built for 64-wide tiles
        // 128-wide tiles: up to two row tiles of one (image, column tile) are accumulated together
        // during ONE pass over the streamed weights (four accumulator stages: two groups in
        // flight), which halves the weight traffic out of L2 -- the bound of these layers.
        batched = bn == 128;
        grp = batched ? (tiles_per_img < 2 ? tiles_per_img : 2) : gmax;
        while (grp > 1 && kMaxDynSmem - 1024 - 2 * plane_for(grp) * c_blocks < 4 * b_block) --grp;
        const int win_bytes1 = plane_for(grp) * c_blocks;
        // a CTA that owns a single group needs no second window buffer: the room goes to the
        // weight ring, whose depth (bytes in flight) bounds how fast one SM can pull the weights
        const int64_t groups_b = (int64_t)n * n_tiles * ((tiles_per_img + grp - 1) / grp);
        if (batched && groups_b <= sms) win_bufs = 1;
        const int left = kMaxDynSmem - 1024 - win_bufs * win_bytes1;
        b_stages = left / b_block;
        if (b_stages > kMaxBStages) b_stages = kMaxBStages;
        if (b_stages < 2) return 0;
        // spare room beyond four weight stages goes to a third window buffer
        if (win_bufs == 2 && b_stages > 4 && 1024 + 3 * win_bytes1 + 4 * b_block <= kMaxDynSmem) {
            win_bufs = 3;
            b_stages = (kMaxDynSmem - 1024 - 3 * win_bytes1) / b_block;
            if (b_stages > kMaxBStages) b_stages = kMaxBStages;
        }
    }
    const int plane_bytes = plane_for(grp);
    const int win_bytes = plane_bytes * c_blocks;
    const int smem_bytes = 1024 + win_bufs * win_bytes + b_stages * b_block;

    CUtensorMap mx, mx1, mw;
    int rc = encode_window(&mx, x_in, n, h, w, c, cb, wp, tr + r - 1);
    if (rc != SPARQ_OK) return rc;
    rc = encode_window(&mx1, x_in, n, h, w, c, cb, wp, tr);
    if (rc != SPARQ_OK) return rc;
    const int64_t K = (int64_t)r * s * c;
    bool w_one_copy = resident && kb_count <= 256 &&
                      encode_weight_blocks(&mw, wgt, K, cout, cb, bn, kb_count) == CUDA_SUCCESS;
    if (!w_one_copy) {
        rc = encode_2d(&mw, wgt, K, cout, K, cb, bn);
        if (rc != SPARQ_OK) return rc;
    }

    WindowArgs g;
    memset(&g, 0, sizeof(g));
    g.w_one_copy = w_one_copy ? 1 : 0;
    // Streamed weights pass through a ring that is shorter than one tile's blocks, in tile order:
    // two issuers on different tiles would wait on the same stage barriers several phases apart,
    // which a parity wait cannot tell apart.  One issuer then; two with resident weights.
    g.issuers = resident ? 2 : 1;
    g.N = cout; g.K = K;
    g.n_img = n; g.H = h; g.W = w; g.C = c; g.R = r; g.S = s; g.pad_h = pad_h; g.pad_w = pad_w; g.Ho = ho; g.Wo = wo;
    g.Wp = wp; g.TR = tr; g.tiles_per_img = tiles_per_img; g.c_blocks = c_blocks;
    g.G = grp;
    g.piece0_bytes = cb * wp * (tr + r - 1);
    g.piece_bytes = cb * wp * tr;
    g.n_tiles = (uint32_t)n_tiles;
    g.units = (uint32_t)units;
    if (batched) {
        // CTAs own whole groups, so that a group is never cut at a share boundary
        const int64_t groups = (int64_t)n * n_tiles * ((tiles_per_img + grp - 1) / grp);
        g.groups = (uint32_t)groups;
        grid = (int)(groups < sms ? groups : sms);
    }
    g.plane_bytes = plane_bytes;
    g.win_bufs = win_bufs;
    g.b_stages = b_stages;
    g.xf = xform_dev(x);
    g.scale = e->scale; g.bias = e->bias; g.relu = e->relu ? 1 : 0; g.inv_out_scale = e->inv_out_scale;
    g.acc_out = e->acc_out; g.f32_out = e->f32_out; g.u8_out = e->u8_out;
    g.status = status;
    g.wait_limit = g_wait_limit;
    g.residual = e->residual;
    g.residual_scale = e->residual_scale;
    rc = next_transform_args(e, g.N, &g.next_mode, &g.next_rnd, &g.next_xf);
    if (rc != SPARQ_OK) return rc;
    g.early_weights = record_launch_weights_clear(st, e, (size_t)n * ho * wo * (size_t)cout, wgt, (size_t)cout * (size_t)K) ? 1 : 0;
    cudaError_t ce;
    if (bn == 64) ce = launch_window_shape<64, 64, true>(mx, mx1, mw, g, x.mode, variant_n(x), x.rnd, grid, smem_bytes, st);
    else if (bn == 128 && resident) ce = launch_window_shape<128, 128, true>(mx, mx1, mw, g, x.mode, variant_n(x), x.rnd, grid, smem_bytes, st);
    else if (bn == 128) ce = launch_window_shape<128, 128, false>(mx, mx1, mw, g, x.mode, variant_n(x), x.rnd, grid, smem_bytes, st);
    else ce = launch_window_shape<256, 128, false>(mx, mx1, mw, g, x.mode, variant_n(x), x.rnd, grid, smem_bytes, st);
    if (ce != cudaSuccess) return cuda_error(ce, "sparq_conv_window_kernel launch");
    return 1;
}

// Tile choice, tensor maps and launch of the fused GEMM.  The caller brings the status word (a
// device pointer); nothing here allocates device memory.
int gemm_with_status(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb, int64_t M, int64_t N, int64_t K,
                     const XformArgs &x, const sparq_epilogue *e, unsigned int *status, cudaStream_t st)
{
    int sms = 0;
    int rc = device_info(&sms);
    if (rc != SPARQ_OK) return rc;
    const int64_t pad128 = (K + 127) / 128 * 128, pad64 = (K + 63) / 64 * 64;
    // the step that pads K the least; ties go to the wider one -- and so does a long reduction whose
    // padding stays below an eighth (K = 576: five 128-byte steps instead of nine 64-byte ones: each
    // step is a hand-off between three warp roles, which is what a small launch is made of)
    const int bk = (pad64 < pad128 && !(pad64 >= 320 && pad128 * 8 <= pad64 * 9)) ? 64 : 128;
    const int bn = pick_bn(M, N, sms, x.mode != SPARQ_MODE_NONE);
    CUtensorMap ma, mb;
    rc = encode_2d(&ma, A, K, M, lda, bk, kBM);
    if (rc != SPARQ_OK) return rc;
    rc = encode_2d(&mb, B, K, N, ldb, bk, bn);
    if (rc != SPARQ_OK) return rc;
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.M = M; g.N = N; g.K = K;
    g.k_blocks = (int)((K + bk - 1) / bk);
    rc = fill_common(&g, x, e, status);
    if (rc != SPARQ_OK) return rc;
    const int64_t tiles = ((M + kBM - 1) / kBM) * ((N + bn - 1) / bn);
    if (tiles >= ((int64_t)1 << 31)) return set_error(SPARQ_ERR_UNSUPPORTED, "more than 2^31 output tiles");
    const int grid = (int)(tiles < sms ? tiles : sms);
    record_launch_weights_clear(st, e, (size_t)M * (size_t)N, B, (size_t)N * (size_t)ldb);
    cudaError_t ce = launch(bn, bk, ma, mb, g, x, grid, st);
    if (ce != cudaSuccess) return cuda_error(ce, "sparq_gemm_kernel launch");
    return SPARQ_OK;
}

int check_epilogue_args(const sparq_epilogue *e) { return check_epilogue(e); }

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_gemm_s8(const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                             int64_t M, int64_t N, int64_t K,
                             const sparq_params *p, const sparq_epilogue *e, void *stream)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    rc = check_epilogue(e);
    if (rc != SPARQ_OK) return rc;
    if (M < 0 || N < 0 || K < 0) return set_error(SPARQ_ERR_INVALID_ARG, "negative dimension");
    if (M == 0 || N == 0) return SPARQ_OK;
    if (!A || !B) return set_error(SPARQ_ERR_INVALID_ARG, "A or B is NULL");
    if (K == 0 || K % 16 || K > 65536) return set_error(SPARQ_ERR_UNSUPPORTED, "K = %lld must be a multiple of 16 in [16, 65536]", (long long)K);
    if (lda < K || ldb < K || lda % 16 || ldb % 16)
        return set_error(SPARQ_ERR_UNSUPPORTED, "lda/ldb must be multiples of 16 and at least K");
    if (((uintptr_t)A | (uintptr_t)B) & 15u) return set_error(SPARQ_ERR_UNSUPPORTED, "A and B must be 16-byte aligned");
    if (M > (int64_t)1 << 31 || N > (int64_t)1 << 31) return set_error(SPARQ_ERR_UNSUPPORTED, "M or N too large");
    return gemm_impl(A, lda, B, ldb, M, N, K, x, e, (cudaStream_t)stream);
}

extern "C" int sparq_conv2d_nhwc_s8(const uint8_t *x_in, int n, int h, int w, int c,
                                    const int8_t *wgt, int cout, int r, int s,
                                    int stride_h, int stride_w, int pad_h, int pad_w,
                                    const sparq_params *p, const sparq_epilogue *e, void *stream)
{
    XformArgs x;
    int rc = validate_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    rc = check_epilogue(e);
    if (rc != SPARQ_OK) return rc;
    if (n < 0 || h < 0 || w < 0 || c < 0 || cout < 0) return set_error(SPARQ_ERR_INVALID_ARG, "negative dimension");
    if (r < 1 || s < 1 || stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0)
        return set_error(SPARQ_ERR_INVALID_ARG, "filter size and strides must be >= 1, pads >= 0");
    if (r > 7 || s > 7 || stride_h > 8 || stride_w > 8 || pad_h >= r || pad_w >= s)
        return set_error(SPARQ_ERR_UNSUPPORTED, "filter up to 7x7, strides up to 8, pads below the filter size");
    if (n == 0 || cout == 0) return SPARQ_OK;
    if (h + 2 * pad_h < r || w + 2 * pad_w < s) return set_error(SPARQ_ERR_INVALID_ARG, "filter larger than the padded image");
    if (!x_in || !wgt) return set_error(SPARQ_ERR_INVALID_ARG, "x or wgt is NULL");
    if (c == 0 || c % 16) return set_error(SPARQ_ERR_UNSUPPORTED, "c = %d must be a positive multiple of 16", c);
    if (((uintptr_t)x_in | (uintptr_t)wgt) & 15u) return set_error(SPARQ_ERR_UNSUPPORTED, "x and wgt must be 16-byte aligned");
    const int ho = (h + 2 * pad_h - r) / stride_h + 1;
    const int wo = (w + 2 * pad_w - s) / stride_w + 1;
    const int64_t M = (int64_t)n * ho * wo;
    const int64_t K = (int64_t)r * s * c;
    if (K > 65536) return set_error(SPARQ_ERR_UNSUPPORTED, "r*s*c = %lld exceeds 65536", (long long)K);
    cudaStream_t st = (cudaStream_t)stream;

    // A 1x1 filter with unit stride reads the NHWC tensor as the M x c matrix it already is.
    if (r == 1 && s == 1 && stride_h == 1 && stride_w == 1 && pad_h == 0 && pad_w == 0)
        return gemm_impl(x_in, c, wgt, c, M, cout, c, x, e, st);

    int sms = 0;
    rc = device_info(&sms);
    if (rc != SPARQ_OK) return rc;
    unsigned int *status = nullptr;
    rc = get_status_word(&status);
    if (rc != SPARQ_OK) return rc;
    if (stride_h == 1 && stride_w == 1) {
        rc = try_window_conv(x_in, n, h, w, c, wgt, cout, r, s, pad_h, pad_w, ho, wo, x, e, sms, status, st);
        if (rc != 0) return rc < 0 ? rc : SPARQ_OK;
    }
    const int bk = (c % 128 == 0) ? 128 : 64;
    const int bn = pick_bn(M, cout, sms, x.mode != SPARQ_MODE_NONE);
    CUtensorMap ma, mb;
    rc = encode_im2col(&ma, x_in, n, h, w, c, r, s, stride_h, stride_w, pad_h, pad_w, bk);
    if (rc != SPARQ_OK) return rc;
    rc = encode_2d(&mb, wgt, K, cout, K, bk, bn);
    if (rc != SPARQ_OK) return rc;
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.M = M; g.N = cout; g.K = K;
    // A channel count that is not a multiple of 64 takes a last block that reaches past C: the
    // im2col copy fills those channels with zeros.
    g.c_blocks = (c + bk - 1) / bk;
    g.k_blocks = r * s * g.c_blocks;
    g.conv = 1;
    g.tap_k = c;
    g.S = s;
    g.Ho = ho; g.Wo = wo;
    g.stride_h = stride_h; g.stride_w = stride_w; g.pad_h = pad_h; g.pad_w = pad_w;
    rc = fill_common(&g, x, e, status);
    if (rc != SPARQ_OK) return rc;
    const int64_t tiles = ((M + kBM - 1) / kBM) * ((cout + bn - 1) / bn);
    if (tiles >= ((int64_t)1 << 31)) return set_error(SPARQ_ERR_UNSUPPORTED, "more than 2^31 output tiles");
    const int grid = (int)(tiles < sms ? tiles : sms);
    record_launch_weights_clear(st, e, (size_t)M * (size_t)cout, wgt, (size_t)cout * (size_t)K);
    cudaError_t ce = launch(bn, bk, ma, mb, g, x, grid, st);
    if (ce != cudaSuccess) return cuda_error(ce, "sparq_gemm_kernel (convolution) launch");
    return SPARQ_OK;
}

