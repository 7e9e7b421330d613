// Packed SPARQ stream (n = 4): what the multiplier of Eq. 4 consumes instead of the 8-bit
// activation -- two 4-bit inputs per pair (one data byte) and the pair's control state
// (both placements, or which slot holds a lone value; Sections 3.1 and 5.1).
//
//   data plane   one byte per pair, (in1 << 4) | in2
//   ctrl plane   per unit of 16 activations the 8 pair states, CB bits each, pair j at
//                bits [j*CB, (j+1)*CB) of a little-endian integer of CB bytes
//   state        both non-zero: id(shift1) * ns + id(shift2) with ns placements in the set
//                and id = rank of the shift in the set; ns*ns: second slot zero, data is the
//                first activation whole; ns*ns + 1: first slot zero (vSPARQ only)
//
// Both kernels are streaming kernels: a thread owns whole units (one 16-byte vector of
// activations <-> 8 data bytes + CB control bytes), control bytes go through shared
// memory so that global accesses stay coalesced, and the per-byte window / placement comes
// from a 256-entry table built on the host from the same packed transform the other
// kernels use.
#include "sparq_common.cuh"

namespace sparq {

namespace {

constexpr int kThreads = 256;
constexpr int kUnits = 4;      // units per thread per tile

// Per activation byte x: bits 0-3 window of bSPARQ(x), bits 4-7 id of its placement,
// bits 8-12 id * ns.
struct PackLut {
    uint16_t e[256];
};

// Per state: bits 0-2 shift of the first slot, bits 4-6 shift of the second, bit 8: lone
// value in the first slot, bit 9: lone value in the second slot.
struct UnpackLut {
    uint16_t e[32];
};

__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ uint2 ld_stream8(const void *p)
{
    uint2 v;
    asm volatile("ld.global.cs.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream16(void *p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ void st_stream8(void *p, uint2 v)
{
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(v.x), "r"(v.y) : "memory");
}

// One tile = kThreads * kUnits consecutive units; unit (i, t) of the tile is
// tile0 + i * kThreads + t, so that a warp's loads and stores are contiguous.
template <int MODE, int CB>
__global__ void __launch_bounds__(kThreads)
pack_kernel(const uint8_t *__restrict__ in, uint8_t *__restrict__ data, uint8_t *__restrict__ ctrl,
            size_t units, const __grid_constant__ PackLut lut, int ns)
{
    __shared__ uint16_t s_lut[256];
    __shared__ __align__(16) uint8_t s_ctrl[kUnits * kThreads * CB];
    s_lut[threadIdx.x] = lut.e[threadIdx.x];
    __syncthreads();
    const uint32_t lone_state = (uint32_t)(ns * ns);
    const size_t tile_units = (size_t)kThreads * kUnits;
    for (size_t tile0 = (size_t)blockIdx.x * tile_units; tile0 < units; tile0 += (size_t)gridDim.x * tile_units) {
        uint4 v[kUnits];
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = tile0 + (size_t)i * kThreads + threadIdx.x;
            if (u < units) v[i] = ld_stream16(in + 16 * u);
        }
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = tile0 + (size_t)i * kThreads + threadIdx.x;
            if (u >= units) continue;
            const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
            uint32_t d[2] = {0u, 0u};
            uint64_t c = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t pair = (w[j >> 1] >> (16 * (j & 1))) & 0xFFFFu;
                const uint32_t a = pair & 0xFFu, b = pair >> 8;
                const uint32_t ea = s_lut[a], eb = s_lut[b];
                uint32_t dat = ((ea & 15u) << 4) | (eb & 15u);
                uint32_t st = (ea >> 8) + ((eb >> 4) & 15u);
                if (MODE == SPARQ_MODE_VSPARQ) {
                    // Eq. 2 / Eq. 3: a lone value is kept whole as its two nibbles
                    if (b == 0u) { dat = a; st = lone_state; }
                    else if (a == 0u) { dat = b; st = lone_state + 1u; }
                }
                d[j >> 2] |= dat << (8 * (j & 3));
                c |= (uint64_t)st << (j * CB);
            }
            st_stream8(data + 8 * u, make_uint2(d[0], d[1]));
            uint8_t *sc = s_ctrl + ((size_t)i * kThreads + threadIdx.x) * CB;
#pragma unroll
            for (int k = 0; k < CB; ++k) sc[k] = (uint8_t)(c >> (8 * k));
        }
        __syncthreads();
        // the tile's control bytes are contiguous in the stream: copy them out in words
        const size_t left = units - tile0;
        const size_t n_units = left < tile_units ? left : tile_units;
        const uint32_t bytes = (uint32_t)n_units * CB;
        uint8_t *dst = ctrl + tile0 * CB;                 // 4-byte aligned: tile0 is a multiple of 1024
        for (uint32_t o = threadIdx.x * 4u; o + 4u <= bytes; o += kThreads * 4u)
            *reinterpret_cast<uint32_t *>(dst + o) = *reinterpret_cast<const uint32_t *>(s_ctrl + o);
        if (threadIdx.x < (bytes & 3u)) dst[(bytes & ~3u) + threadIdx.x] = s_ctrl[(bytes & ~3u) + threadIdx.x];
        __syncthreads();
    }
}

template <int CB>
__global__ void __launch_bounds__(kThreads)
unpack_kernel(const uint8_t *__restrict__ data, const uint8_t *__restrict__ ctrl, uint8_t *__restrict__ out,
              size_t units, const __grid_constant__ UnpackLut lut)
{
    __shared__ uint16_t s_lut[32];
    __shared__ __align__(16) uint8_t s_ctrl[kUnits * kThreads * CB];
    if (threadIdx.x < 32) s_lut[threadIdx.x] = lut.e[threadIdx.x];
    const size_t tile_units = (size_t)kThreads * kUnits;
    for (size_t tile0 = (size_t)blockIdx.x * tile_units; tile0 < units; tile0 += (size_t)gridDim.x * tile_units) {
        const size_t left = units - tile0;
        const size_t n_units = left < tile_units ? left : tile_units;
        const uint32_t bytes = (uint32_t)n_units * CB;
        const uint8_t *src = ctrl + tile0 * CB;
        uint2 dv[kUnits];
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = tile0 + (size_t)i * kThreads + threadIdx.x;
            if (u < units) dv[i] = ld_stream8(data + 8 * u);
        }
        for (uint32_t o = threadIdx.x * 4u; o + 4u <= bytes; o += kThreads * 4u)
            *reinterpret_cast<uint32_t *>(s_ctrl + o) = __ldcs(reinterpret_cast<const uint32_t *>(src + o));
        if (threadIdx.x < (bytes & 3u)) s_ctrl[(bytes & ~3u) + threadIdx.x] = src[(bytes & ~3u) + threadIdx.x];
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = tile0 + (size_t)i * kThreads + threadIdx.x;
            if (u >= units) continue;
            const uint8_t *sc = s_ctrl + ((size_t)i * kThreads + threadIdx.x) * CB;
            uint64_t c = 0;
#pragma unroll
            for (int k = 0; k < CB; ++k) c |= (uint64_t)sc[k] << (8 * k);
            const uint32_t d[2] = {dv[i].x, dv[i].y};
            uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t st = (uint32_t)(c >> (j * CB)) & ((1u << CB) - 1u);
                const uint32_t dat = (d[j >> 2] >> (8 * (j & 3))) & 0xFFu;
                const uint32_t e = s_lut[st];
                // Eq. 4 with unit weights: 2^opt1 * in1 and 2^opt2 * in2
                uint32_t qa = (dat >> 4) << (e & 7u);
                uint32_t qb = (dat & 15u) << ((e >> 4) & 7u);
                if (e & 0x100u) { qa = dat; qb = 0u; }
                if (e & 0x200u) { qa = 0u; qb = dat; }
                w[j >> 1] |= (qa | (qb << 8)) << (16 * (j & 1));
            }
            st_stream16(out + 16 * u, make_uint4(w[0], w[1], w[2], w[3]));
        }
        __syncthreads();
    }
}

int set_size(uint32_t mask) { return __builtin_popcount(mask & 0x1Fu); }

int state_bits(int mode, uint32_t mask)
{
    const int ns = set_size(mask);
    const int states = ns * ns + (mode == SPARQ_MODE_VSPARQ ? 2 : 0);
    int bits = 0;
    while ((1 << bits) < states) ++bits;
    return bits;
}

// Validates the parameters of the packed form: a SPARQ mode with 4-bit windows.
int check_pack_params(const sparq_params *p, XformArgs *x)
{
    int rc = validate_params(p, x);
    if (rc != SPARQ_OK) return rc;
    if (x->mode == SPARQ_MODE_NONE) return set_error(SPARQ_ERR_INVALID_ARG, "the packed form needs mode BSPARQ or VSPARQ");
    if (x->n != 4) return set_error(SPARQ_ERR_UNSUPPORTED, "the packed form is defined for 4-bit windows (window_bits = %d)", x->n);
    return SPARQ_OK;
}

int check_stream(const void *a, const void *b, const void *c, const void *d, size_t rows, size_t row_len, size_t *units)
{
    if (!a || !b || !c || !d) return set_error(SPARQ_ERR_INVALID_ARG, "a stream pointer is NULL");
    if (row_len % 16) return set_error(SPARQ_ERR_UNSUPPORTED, "row_len (%zu) must be a multiple of 16", row_len);
    if (rows > ((size_t)1 << 62) / row_len) return set_error(SPARQ_ERR_INVALID_ARG, "rows * row_len overflows");
    if ((((uintptr_t)a | (uintptr_t)b | (uintptr_t)c | (uintptr_t)d) & 15u) != 0)
        return set_error(SPARQ_ERR_UNSUPPORTED, "stream pointers must be 16-byte aligned");
    *units = rows * row_len / 16;
    return SPARQ_OK;
}

int grid_for(size_t units, int *blocks)
{
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_error(e, "device query");
    const size_t tile = (size_t)kThreads * kUnits;
    const size_t want = (units + tile - 1) / tile;
    const size_t cap = (size_t)sms * 32;
    *blocks = (int)(want < cap ? want : cap);
    return SPARQ_OK;
}

// Lowest allowed placement that holds q (q is a bSPARQ result, so its bits below that
// placement are zero).
int placement_of(uint32_t q, uint32_t mask)
{
    for (int s = 0; s <= 4; ++s)
        if (((mask >> s) & 1u) && (q >> s) < 16u) return s;
    return 4;
}

int rank_of(int s, uint32_t mask) { return __builtin_popcount(mask & ((1u << s) - 1u)); }

template <int MODE>
cudaError_t launch_pack(int cb, const uint8_t *in, uint8_t *data, uint8_t *ctrl, size_t units, const PackLut &lut,
                        int ns, int blocks, cudaStream_t st)
{
    switch (cb) {
    case 2: pack_kernel<MODE, 2><<<blocks, kThreads, 0, st>>>(in, data, ctrl, units, lut, ns); break;
    case 3: pack_kernel<MODE, 3><<<blocks, kThreads, 0, st>>>(in, data, ctrl, units, lut, ns); break;
    case 4: pack_kernel<MODE, 4><<<blocks, kThreads, 0, st>>>(in, data, ctrl, units, lut, ns); break;
    default: pack_kernel<MODE, 5><<<blocks, kThreads, 0, st>>>(in, data, ctrl, units, lut, ns); break;
    }
    return cudaGetLastError();
}

}  // namespace

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_packed_ctrl_bits(const sparq_params *p)
{
    XformArgs x;
    int rc = check_pack_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    return state_bits(x.mode, x.mask);
}

extern "C" int sparq_pack(const uint8_t *in, size_t rows, size_t row_len, const sparq_params *p,
                          uint8_t *data, uint8_t *ctrl, void *stream)
{
    XformArgs x;
    int rc = check_pack_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    if (rows == 0 || row_len == 0) return SPARQ_OK;
    size_t units = 0;
    if ((rc = check_stream(in, data, ctrl, in, rows, row_len, &units)) != SPARQ_OK) return rc;
    const int ns = set_size(x.mask);
    const int cb = state_bits(x.mode, x.mask);
    // window and placement of bSPARQ(v) for every byte value, from the packed transform
    PackLut lut;
    const XformDev d{x.widen_c, x.widen_rounds, 4};
    for (uint32_t v = 0; v < 256; ++v) {
        const uint32_t q = (x.rnd ? xform_word<SPARQ_MODE_BSPARQ, 0, true, true>(v, d)
                                  : xform_word<SPARQ_MODE_BSPARQ, 0, false, true>(v, d)) & 0xFFu;
        const int s = placement_of(q, x.mask);
        const int id = rank_of(s, x.mask);
        lut.e[v] = (uint16_t)((q >> s) | (uint32_t)(id << 4) | (uint32_t)((id * ns) << 8));
    }
    int blocks = 0;
    if ((rc = grid_for(units, &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = x.mode == SPARQ_MODE_VSPARQ
                        ? launch_pack<SPARQ_MODE_VSPARQ>(cb, in, data, ctrl, units, lut, ns, blocks, st)
                        : launch_pack<SPARQ_MODE_BSPARQ>(cb, in, data, ctrl, units, lut, ns, blocks, st);
    if (e != cudaSuccess) return cuda_error(e, "pack_kernel launch");
    return SPARQ_OK;
}

extern "C" int sparq_unpack(const uint8_t *data, const uint8_t *ctrl, size_t rows, size_t row_len,
                            const sparq_params *p, uint8_t *out, void *stream)
{
    XformArgs x;
    int rc = check_pack_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    if (rows == 0 || row_len == 0) return SPARQ_OK;
    size_t units = 0;
    if ((rc = check_stream(data, ctrl, out, out, rows, row_len, &units)) != SPARQ_OK) return rc;
    const int ns = set_size(x.mask);
    const int cb = state_bits(x.mode, x.mask);
    int shift_of[5], r = 0;
    for (int s = 0; s <= 4; ++s)
        if ((x.mask >> s) & 1u) shift_of[r++] = s;
    UnpackLut lut;
    for (int st = 0; st < 32; ++st) {
        uint32_t e = 0;
        if (st < ns * ns) e = (uint32_t)shift_of[st / ns] | ((uint32_t)shift_of[st % ns] << 4);
        else if (st == ns * ns + 1 && x.mode == SPARQ_MODE_VSPARQ) e = 0x200u;
        else e = 0x100u;   // ns*ns; states a valid stream never holds decode like it
        lut.e[st] = (uint16_t)e;
    }
    int blocks = 0;
    if ((rc = grid_for(units, &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    switch (cb) {
    case 2: unpack_kernel<2><<<blocks, kThreads, 0, st>>>(data, ctrl, out, units, lut); break;
    case 3: unpack_kernel<3><<<blocks, kThreads, 0, st>>>(data, ctrl, out, units, lut); break;
    case 4: unpack_kernel<4><<<blocks, kThreads, 0, st>>>(data, ctrl, out, units, lut); break;
    default: unpack_kernel<5><<<blocks, kThreads, 0, st>>>(data, ctrl, out, units, lut); break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_error(e, "unpack_kernel launch");
    return SPARQ_OK;
}
