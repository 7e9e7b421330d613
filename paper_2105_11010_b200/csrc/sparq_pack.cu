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
// activations <-> 8 data bytes + CB control bytes) and control bytes go through shared
// memory so that global accesses stay coalesced.  The per-activation work is table
// look-ups; the tables (512 words, built on the host from the same packed transform the
// other kernels use) are replicated once per lane in shared memory, word (index, lane) at
// word address index * 32 + lane, so that a warp's 32 look-ups always hit 32 different
// banks whatever the data.
#include "sparq_common.cuh"

namespace sparq {

// 3- and 2-bit windows: sparq_pack_narrow.cu
int narrow_ctrl_bits(const XformArgs &x);
int pack_narrow(const uint8_t *in, uint8_t *data, uint8_t *ctrl, size_t units, const XformArgs &x, cudaStream_t st);
int unpack_narrow(const uint8_t *data, const uint8_t *ctrl, uint8_t *out, size_t units, const XformArgs &x, cudaStream_t st);

namespace {

constexpr int kThreads = 512;
constexpr int kUnits = 4;                        // units per thread per tile
constexpr int kLutWords = 512;
constexpr int kLutBytes = kLutWords * 32 * 4;    // one copy per lane

// Encoder table.  The data byte and the state of a pair are the SUM of one half-word per
// slot, half-word = data contribution | state contribution << 8.  Word index = x * 2 + z
// with x the slot's activation and z = 1 when the partner slot is zero (vSPARQ only):
//   low half, first slot    z = 0: window(x) << 4 | (id(x) * ns) << 8
//                           z = 1: x | (ns*ns) << 8                    (x whole)
//   high half, second slot  z = 0: window(x) | id(x) << 8
//                           z = 1: x | (ns*ns + 1) << 8, 0 for x = 0
// Decoder table.  The two activations of a pair as (first | second << 8) are the sum of the
// low half of word [nibble_hi * 32 + state] and the high half of word [nibble_lo * 32 + state]
// (Eq. 4 with unit weights: 2^opt1 * in1 and 2^opt2 * in2, routed to the slot(s) the state
// names).
struct Lut {
    uint32_t w[kLutWords];
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

// One copy of the table per lane (all threads of the block call this).
__device__ __forceinline__ void fill_lut(uint32_t *s_lut, const Lut &lut)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = warp; i < kLutWords; i += kThreads / 32) s_lut[i * 32 + lane] = lut.w[i];
}

// Half-word of the lane's table copy at byte offset `off` (= word index * 128 + lane * 4 + half * 2)
__device__ __forceinline__ uint32_t lut_half(const uint8_t *s_lut, uint32_t off)
{
    return *reinterpret_cast<const uint16_t *>(s_lut + off);
}

// CB-bit field `st` into bits [POS, POS + CB) of the 64-bit word (lo, hi)
template <int POS, int CB>
__device__ __forceinline__ void put_state(uint32_t &lo, uint32_t &hi, uint32_t st)
{
    if constexpr (POS >= 32) {
        hi |= st << (POS - 32);
    } else {
        lo |= st << POS;
        if constexpr (POS + CB > 32) hi |= st >> (32 - POS);
    }
}

template <int POS, int CB>
__device__ __forceinline__ uint32_t get_state(uint32_t lo, uint32_t hi)
{
    uint32_t v;
    if constexpr (POS >= 32) v = hi >> (POS - 32);
    else if constexpr (POS + CB > 32) v = __funnelshift_r(lo, hi, POS);
    else v = lo >> POS;
    return v & ((1u << CB) - 1u);
}

// Two pairs (one 32-bit word of activations): their sums data | state << 8.
// lanes = (lane * 4) in every byte: the lane's offset inside a table word row.
template <int MODE>
__device__ __forceinline__ void pack_word(uint32_t x, uint32_t lanes, const uint8_t *s_lut, uint32_t &s0, uint32_t &s1)
{
    uint32_t low = lanes;                                                // byte: z << 7 | lane << 2
    if (MODE == SPARQ_MODE_VSPARQ) {
        const uint32_t nz = ((x & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | x;      // bit 7 of each byte: byte != 0
        low = (~prmt(nz, nz, 0xAB89u) & 0x80808080u) | lanes;            // bit 7: the partner is zero
    }
    // byte offsets of the four look-ups: activation << 8 | z << 7 | lane << 2
    const uint32_t o01 = prmt(x, low, 0x1504u), o23 = prmt(x, low, 0x3726u);
    s0 = lut_half(s_lut, o01 & 0xFFFFu) + lut_half(s_lut + 2, o01 >> 16);
    s1 = lut_half(s_lut, o23 & 0xFFFFu) + lut_half(s_lut + 2, o23 >> 16);
}

// low bytes of four words -> one word
__device__ __forceinline__ uint32_t bytes4(uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    return prmt(prmt(a, b, 0x0040u), prmt(c, d, 0x0040u), 0x5410u);
}

// A warp owns chunks of kUnits * 32 consecutive units (unit (i, lane) of a chunk is
// chunk0 + i * 32 + lane, so its loads and stores are contiguous); the chunk's control bytes
// are contiguous in the stream too, and go through a warp-private staging area, so the only
// block-wide barrier is the one after the table fill.
constexpr int kChunkUnits = kUnits * 32;

template <int MODE, int CB>
__global__ void __launch_bounds__(kThreads)
pack_kernel(const uint8_t *__restrict__ in, uint8_t *__restrict__ data, uint8_t *__restrict__ ctrl,
            size_t units, const __grid_constant__ Lut lut)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t *s_lut = smem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t *s_ctrl = smem + kLutBytes + warp * (kChunkUnits * CB);
    fill_lut(reinterpret_cast<uint32_t *>(s_lut), lut);
    __syncthreads();
    const uint32_t lanes = (uint32_t)lane * 0x04040404u;
    const size_t n_chunks = (units + kChunkUnits - 1) / kChunkUnits;
    const size_t stride = (size_t)gridDim.x * (kThreads / 32);
    for (size_t ch = (size_t)blockIdx.x * (kThreads / 32) + warp; ch < n_chunks; ch += stride) {
        const size_t chunk0 = ch * kChunkUnits;
        uint4 v[kUnits];
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = chunk0 + (size_t)i * 32 + lane;
            if (u < units) v[i] = ld_stream16(in + 16 * u);
        }
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = chunk0 + (size_t)i * 32 + lane;
            if (u >= units) continue;
            uint32_t s[8];
            pack_word<MODE>(v[i].x, lanes, s_lut, s[0], s[1]);
            pack_word<MODE>(v[i].y, lanes, s_lut, s[2], s[3]);
            pack_word<MODE>(v[i].z, lanes, s_lut, s[4], s[5]);
            pack_word<MODE>(v[i].w, lanes, s_lut, s[6], s[7]);
            st_stream8(data + 8 * u, make_uint2(bytes4(s[0], s[1], s[2], s[3]), bytes4(s[4], s[5], s[6], s[7])));
            uint32_t lo = 0u, hi = 0u;
            put_state<0 * CB, CB>(lo, hi, s[0] >> 8);
            put_state<1 * CB, CB>(lo, hi, s[1] >> 8);
            put_state<2 * CB, CB>(lo, hi, s[2] >> 8);
            put_state<3 * CB, CB>(lo, hi, s[3] >> 8);
            put_state<4 * CB, CB>(lo, hi, s[4] >> 8);
            put_state<5 * CB, CB>(lo, hi, s[5] >> 8);
            put_state<6 * CB, CB>(lo, hi, s[6] >> 8);
            put_state<7 * CB, CB>(lo, hi, s[7] >> 8);
            uint8_t *sc = s_ctrl + (i * 32 + lane) * CB;
#pragma unroll
            for (int k = 0; k < CB; ++k) sc[k] = (uint8_t)((k < 4 ? lo : hi) >> (8 * (k & 3)));
        }
        __syncwarp();
        // the chunk's control bytes, contiguous in the stream, in words (CB words per lane)
        const size_t left = units - chunk0;
        const uint32_t bytes = (uint32_t)(left < (size_t)kChunkUnits ? left : (size_t)kChunkUnits) * CB;
        uint8_t *dst = ctrl + chunk0 * CB;                // 16-byte aligned: chunk0 is a multiple of 128
#pragma unroll
        for (int k = 0; k < CB; ++k) {
            const uint32_t o = (uint32_t)(k * 32 + lane) * 4u;
            if (o + 4u <= bytes) *reinterpret_cast<uint32_t *>(dst + o) = *reinterpret_cast<const uint32_t *>(s_ctrl + o);
        }
        if ((uint32_t)lane < (bytes & 3u)) dst[(bytes & ~3u) + lane] = s_ctrl[(bytes & ~3u) + lane];
        __syncwarp();
    }
}

// Pair J of a unit.  hn / ln: the data bytes' high / low nibbles in the top half of each byte
// (nibble << 12 once the byte sits in bits 8-15 of the offset); base = lane << 2.
template <int J, int CB>
__device__ __forceinline__ uint32_t unpack_pair(uint32_t lo, uint32_t hi, uint32_t hn, uint32_t ln, uint32_t base,
                                                const uint8_t *s_lut)
{
    const uint32_t row = get_state<J * CB, CB>(lo, hi) * 128u + base;
    const uint32_t oh = prmt(hn, 0u, 0x4404u + ((J & 3) << 4)) | row;    // nibble << 12 | state << 7 | lane << 2
    const uint32_t ol = prmt(ln, 0u, 0x4404u + ((J & 3) << 4)) | row;
    return lut_half(s_lut, oh) + lut_half(s_lut + 2, ol);
}

template <int CB>
__global__ void __launch_bounds__(kThreads)
unpack_kernel(const uint8_t *__restrict__ data, const uint8_t *__restrict__ ctrl, uint8_t *__restrict__ out,
              size_t units, const __grid_constant__ Lut lut)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t *s_lut = smem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t *s_ctrl = smem + kLutBytes + warp * (kChunkUnits * CB);
    fill_lut(reinterpret_cast<uint32_t *>(s_lut), lut);
    __syncthreads();
    const uint32_t base = (uint32_t)lane * 4u;
    const size_t n_chunks = (units + kChunkUnits - 1) / kChunkUnits;
    const size_t stride = (size_t)gridDim.x * (kThreads / 32);
    for (size_t ch = (size_t)blockIdx.x * (kThreads / 32) + warp; ch < n_chunks; ch += stride) {
        const size_t chunk0 = ch * kChunkUnits;
        const size_t left = units - chunk0;
        const uint32_t bytes = (uint32_t)(left < (size_t)kChunkUnits ? left : (size_t)kChunkUnits) * CB;
        const uint8_t *src = ctrl + chunk0 * CB;
        uint2 dv[kUnits];
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = chunk0 + (size_t)i * 32 + lane;
            if (u < units) dv[i] = ld_stream8(data + 8 * u);
        }
#pragma unroll
        for (int k = 0; k < CB; ++k) {
            const uint32_t o = (uint32_t)(k * 32 + lane) * 4u;
            if (o + 4u <= bytes) *reinterpret_cast<uint32_t *>(s_ctrl + o) = __ldcs(reinterpret_cast<const uint32_t *>(src + o));
        }
        if ((uint32_t)lane < (bytes & 3u)) s_ctrl[(bytes & ~3u) + lane] = src[(bytes & ~3u) + lane];
        __syncwarp();
#pragma unroll
        for (int i = 0; i < kUnits; ++i) {
            const size_t u = chunk0 + (size_t)i * 32 + lane;
            if (u >= units) continue;
            const uint8_t *sc = s_ctrl + (i * 32 + lane) * CB;
            uint32_t lo = 0u, hi = 0u;
#pragma unroll
            for (int k = 0; k < CB; ++k) {
                if (k < 4) lo |= (uint32_t)sc[k] << (8 * k);
                else hi |= (uint32_t)sc[k] << (8 * (k - 4));
            }
            const uint32_t hn0 = dv[i].x & 0xF0F0F0F0u, ln0 = (dv[i].x << 4) & 0xF0F0F0F0u;
            const uint32_t hn1 = dv[i].y & 0xF0F0F0F0u, ln1 = (dv[i].y << 4) & 0xF0F0F0F0u;
            const uint32_t p0 = unpack_pair<0, CB>(lo, hi, hn0, ln0, base, s_lut);
            const uint32_t p1 = unpack_pair<1, CB>(lo, hi, hn0, ln0, base, s_lut);
            const uint32_t p2 = unpack_pair<2, CB>(lo, hi, hn0, ln0, base, s_lut);
            const uint32_t p3 = unpack_pair<3, CB>(lo, hi, hn0, ln0, base, s_lut);
            const uint32_t p4 = unpack_pair<4, CB>(lo, hi, hn1, ln1, base, s_lut);
            const uint32_t p5 = unpack_pair<5, CB>(lo, hi, hn1, ln1, base, s_lut);
            const uint32_t p6 = unpack_pair<6, CB>(lo, hi, hn1, ln1, base, s_lut);
            const uint32_t p7 = unpack_pair<7, CB>(lo, hi, hn1, ln1, base, s_lut);
            st_stream16(out + 16 * u, make_uint4(prmt(p0, p1, 0x5410u), prmt(p2, p3, 0x5410u),
                                                 prmt(p4, p5, 0x5410u), prmt(p6, p7, 0x5410u)));
        }
        __syncwarp();
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

// Validates the parameters of the packed form: a SPARQ mode.
int check_pack_params(const sparq_params *p, XformArgs *x)
{
    int rc = validate_params(p, x);
    if (rc != SPARQ_OK) return rc;
    if (x->mode == SPARQ_MODE_NONE) return set_error(SPARQ_ERR_INVALID_ARG, "the packed form needs mode BSPARQ or VSPARQ");
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
    const size_t cap = (size_t)sms * 3;      // three resident blocks per SM, each fills its tables once
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

// Launch with the tables' and the control staging's shared memory (above the default limit).
template <class Kernel, class... Args>
cudaError_t launch_codec(Kernel kernel, int cb, int blocks, cudaStream_t st, Args... args)
{
    const int smem = kLutBytes + kUnits * kThreads * cb;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kernel<<<blocks, kThreads, smem, st>>>(args...);
    return cudaGetLastError();
}

template <int MODE>
cudaError_t launch_pack(int cb, const uint8_t *in, uint8_t *data, uint8_t *ctrl, size_t units, const Lut &lut,
                        int blocks, cudaStream_t st)
{
    switch (cb) {
    case 2: return launch_codec(pack_kernel<MODE, 2>, cb, blocks, st, in, data, ctrl, units, lut);
    case 3: return launch_codec(pack_kernel<MODE, 3>, cb, blocks, st, in, data, ctrl, units, lut);
    case 4: return launch_codec(pack_kernel<MODE, 4>, cb, blocks, st, in, data, ctrl, units, lut);
    default: return launch_codec(pack_kernel<MODE, 5>, cb, blocks, st, in, data, ctrl, units, lut);
    }
}

}  // namespace

}  // namespace sparq

using namespace sparq;

extern "C" int sparq_packed_ctrl_bits(const sparq_params *p)
{
    XformArgs x;
    int rc = check_pack_params(p, &x);
    if (rc != SPARQ_OK) return rc;
    return x.n == 4 ? state_bits(x.mode, x.mask) : narrow_ctrl_bits(x);
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
    if (x.n != 4) return pack_narrow(in, data, ctrl, units, x, (cudaStream_t)stream);
    const int ns = set_size(x.mask);
    const int cb = state_bits(x.mode, x.mask);
    // window and placement of bSPARQ(v) for every byte value, from the packed transform
    Lut lut;
    const XformDev d{x.widen_c, x.widen_rounds, 4};
    const bool pairs = x.mode == SPARQ_MODE_VSPARQ;
    for (uint32_t v = 0; v < 256; ++v) {
        const uint32_t q = (x.rnd ? xform_word<SPARQ_MODE_BSPARQ, 0, true, true>(v, d)
                                  : xform_word<SPARQ_MODE_BSPARQ, 0, false, true>(v, d)) & 0xFFu;
        const int s = placement_of(q, x.mask);
        const uint32_t id = (uint32_t)rank_of(s, x.mask), win = q >> s;
        const uint32_t first = (win << 4) | ((id * ns) << 8), second = win | (id << 8);
        lut.w[2 * v] = first | (second << 16);
        // partner zero (reached with vSPARQ only)
        const uint32_t first_z = v | ((uint32_t)(ns * ns) << 8), second_z = v ? (v | ((uint32_t)(ns * ns + 1) << 8)) : 0u;
        lut.w[2 * v + 1] = pairs ? (first_z | (second_z << 16)) : lut.w[2 * v];
    }
    int blocks = 0;
    if ((rc = grid_for(units, &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = x.mode == SPARQ_MODE_VSPARQ
                        ? launch_pack<SPARQ_MODE_VSPARQ>(cb, in, data, ctrl, units, lut, blocks, st)
                        : launch_pack<SPARQ_MODE_BSPARQ>(cb, in, data, ctrl, units, lut, blocks, st);
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
    if (x.n != 4) return unpack_narrow(data, ctrl, out, units, x, (cudaStream_t)stream);
    const int ns = set_size(x.mask);
    const int cb = state_bits(x.mode, x.mask);
    int shift_of[5], r = 0;
    for (int s = 0; s <= 4; ++s)
        if ((x.mask >> s) & 1u) shift_of[r++] = s;
    Lut lut;
    for (int st = 0; st < 32; ++st) {
        for (uint32_t nib = 0; nib < 16; ++nib) {
            uint32_t h = 0, l = 0;
            if (st < ns * ns) {                                   // two windows
                h = nib << shift_of[st / ns];
                l = (nib << shift_of[st % ns]) << 8;
            } else if (st == ns * ns) {                           // lone value in the first slot
                h = nib << 4;
                l = nib;
            } else if (st == ns * ns + 1 && x.mode == SPARQ_MODE_VSPARQ) {   // ... in the second
                h = (nib << 4) << 8;
                l = nib << 8;
            }                                                      // states a valid stream never holds: 0
            lut.w[nib * 32 + st] = h | (l << 16);
        }
    }
    int blocks = 0;
    if ((rc = grid_for(units, &blocks)) != SPARQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    switch (cb) {
    case 2: e = launch_codec(unpack_kernel<2>, cb, blocks, st, data, ctrl, out, units, lut); break;
    case 3: e = launch_codec(unpack_kernel<3>, cb, blocks, st, data, ctrl, out, units, lut); break;
    case 4: e = launch_codec(unpack_kernel<4>, cb, blocks, st, data, ctrl, out, units, lut); break;
    default: e = launch_codec(unpack_kernel<5>, cb, blocks, st, data, ctrl, out, units, lut); break;
    }
    if (e != cudaSuccess) return cuda_error(e, "unpack_kernel launch");
    return SPARQ_OK;
}
