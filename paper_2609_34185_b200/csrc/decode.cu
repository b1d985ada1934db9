// Fused EntroPack decode for sm_100a (paper Sec. 3.7): tiled 32-state rANS symbol decode (Eq. 18),
// arithmetic inverse of the field representation (Eq. 5), multiplication by the fp32 row scale and
// rounding to the output type (Eq. 19), written straight to the weight tensor.  No symbol tensor,
// no codebook, no tensor cores (the path is not a contraction).
//
// Mapping: one warp per tile, one rANS state per lane (the paper's layout); a CTA of 32 warps
// builds the seventeen slot->(frequency, offset, value) lookup tables once in shared memory from the
// stream's frequency tables and then streams tiles through them.  A lookup entry is one 32-bit word
//     [31:20] f      [19:11] code     [10:0] u - F
// where `code` is the symbol's coordinate relative to an even base zlo (z - zlo; 2m - zlo for the m
// field; 32c for the coset, which makes (entry & 0xFF800) the byte offset of coset c's tables).
// (entry & 0xFF800) | 0x45800000 is the fp32 number 4096 + code, so one subtraction of
// 4096 - zlo - c/2 yields the lattice coordinate p exactly, and one fp32 multiply by the row scale
// gives the product of Eq. 19 with the same operands and rounding as the definition.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "stream.hpp"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr uint32_t kLutEntries = 2048;                 // 2^11 slots per table
constexpr uint32_t kLutStride = kLutEntries * 4;       // bytes per table in shared memory
constexpr uint32_t kCosetTableOff = 16 * kLutStride;   // coset table sits after the 16 coordinate tables
constexpr uint32_t kLutBytes = 17 * kLutStride;        // 139264
constexpr uint32_t kCodeMask = 0x000FF800u;
constexpr uint32_t kExp4096 = 0x45800000u;             // fp32 bit pattern of 4096.0

__device__ unsigned int g_ep_status = 0;

struct JobParams {
    const uint8_t *stream;        // blob base (device)
    const uint32_t *tile_index;   // n_tiles records of 33 words + 1 final word
    const float *scales;
    void *out;
    uint32_t off_freq;            // byte offset of the u16 frequency arrays inside the blob
    uint32_t off_payload;
    uint32_t total_words;
    uint32_t n_vec;
    uint32_t per_row;             // C / 8
    uint32_t V, n_tiles, b;
    int32_t zlo;                  // even, <= -2
    uint32_t cta_begin, cta_count;
    int16_t tmin[EP_NUM_TABLES];
    uint16_t tK[EP_NUM_TABLES];
    uint16_t foff[EP_NUM_TABLES]; // start of table t's frequencies, in u16 units
};

struct BatchParams {
    JobParams job[EP_MAX_BATCH];
    int32_t n_jobs;
};

// ---- small PTX helpers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ldg_u16(const uint16_t *p) {
    uint16_t v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void prefetch_l1(const void *p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

// two fp32 lanes per instruction (sm_100 packed fp32)
__device__ __forceinline__ void sub2(float &a0, float &a1, float k) {
    asm("{ .reg .b64 ta, tb; mov.b64 ta, {%0, %1}; mov.b64 tb, {%2, %2}; sub.rn.f32x2 ta, ta, tb; mov.b64 {%0, %1}, ta; }"
        : "+f"(a0), "+f"(a1) : "f"(k));
}
__device__ __forceinline__ void mul2(float &a0, float &a1, float k) {
    asm("{ .reg .b64 ta, tb; mov.b64 ta, {%0, %1}; mov.b64 tb, {%2, %2}; mul.rn.f32x2 ta, ta, tb; mov.b64 {%0, %1}, ta; }"
        : "+f"(a0), "+f"(a1) : "f"(k));
}

// snap_tau of Eq. 19 for two neighbouring weights (lo = lower address)
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pack_fp16_sat(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pack_e4m3(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t cvt_s8(float v) {
    int32_t r;
    asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(r) : "f"(v));
    return uint32_t(r) & 0xFFu;
}

// ---- lookup-table construction (per CTA, from the stream's frequency tables) ---------------------
// Warp t fills table t.  Symbols are taken 32 at a time: a warp scan gives each lane its symbol's
// first slot, every lane writes the first four slots of its own symbol, and symbols with more than
// four slots are then filled by the whole warp.
__device__ __forceinline__ void build_tables_smem(const JobParams &J, uint32_t lut_addr, uint32_t warp, uint32_t lane) {
    if (warp >= EP_NUM_TABLES) return;
    const uint32_t t = warp;
    const uint32_t K = J.tK[t];
    if (K == 0) return;
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(J.stream + J.off_freq) + J.foff[t];
    const int32_t tmin = J.tmin[t];
    const uint32_t base = lut_addr + (t == 0 ? kCosetTableOff : (t - 1) * kLutStride);
    const bool is_m = (t != 0) && (((t - 1) & 7) == 7);
    uint32_t run = 0;
    for (uint32_t j0 = 0; j0 < K; j0 += 32) {
        const uint32_t j = j0 + lane;
        const uint32_t f = j < K ? uint32_t(fq[j]) : 0u;
        uint32_t incl = f;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= uint32_t(d)) incl += n;
        }
        const uint32_t first = run + incl - f;
        const int32_t v = tmin + int32_t(j);
        const uint32_t code = t == 0 ? uint32_t(v) * 32u : uint32_t((is_m ? 2 * v : v) - J.zlo);
        const uint32_t entry = (f << 20) | ((code & 0x1FFu) << 11);
#pragma unroll
        for (uint32_t u = 0; u < 4; ++u)
            if (u < f && first + u < kLutEntries) sts32(base + 4u * (first + u), entry | u);
        uint32_t big = __ballot_sync(0xFFFFFFFFu, f > 4);
        while (big) {
            const int i = __ffs(big) - 1;
            big &= big - 1;
            const uint32_t fi = __shfl_sync(0xFFFFFFFFu, f, i);
            const uint32_t Fi = __shfl_sync(0xFFFFFFFFu, first, i);
            const uint32_t ei = __shfl_sync(0xFFFFFFFFu, entry, i);
            for (uint32_t u = 4 + lane; u < fi && Fi + u < kLutEntries; u += 32) sts32(base + 4u * (Fi + u), ei | u);
        }
        run += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
}

// ---- one rANS symbol (Eq. 18) followed by renormalisation --------------------------------------
// x: this lane's state; ptr: the tile's word cursor (warp-uniform, absolute word index in the payload).
// Lanes that need a word take them in lane order: lane l reads word ptr + popc(ballot & lanes below l).
template <bool TAIL, bool CAREFUL>
__device__ __forceinline__ uint32_t rans_step(uint32_t &x, uint32_t table_addr, uint32_t mask, uint32_t b, uint32_t &ptr,
                                              const uint16_t *pay, uint32_t lt, bool act, uint32_t last_word) {
    uint32_t e = 0;
    bool need = false;
    if (!TAIL || act) {
        const uint32_t u = x & mask;
        e = lds32(table_addr + (u << 2));
        x = (e >> 20) * (x >> b) + (e & 0x7FFu);
        need = x < ep::kStateLow;
    }
    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, need);
    if (need) {
        uint32_t idx = ptr + __popc(bal & lt);
        if (CAREFUL) idx = min(idx, last_word);
        x = (x << 16) | ldg_u16(pay + idx);
    }
    ptr += __popc(bal);
    return e;
}

template <int DT>
struct Out;   // per output type: bytes per 8-weight block and the store of one block

template <>
struct Out<EP_BF16> {
    static constexpr uint32_t kBlockBytes = 16;
    static __device__ __forceinline__ void store(void *dst, const float (&w)[8]) {
        uint4 q = make_uint4(pack_bf16(w[0], w[1]), pack_bf16(w[2], w[3]), pack_bf16(w[4], w[5]), pack_bf16(w[6], w[7]));
        *reinterpret_cast<uint4 *>(dst) = q;
    }
};
template <>
struct Out<EP_FP16> {
    static constexpr uint32_t kBlockBytes = 16;
    static __device__ __forceinline__ void store(void *dst, const float (&w)[8]) {
        uint4 q = make_uint4(pack_fp16_sat(w[0], w[1]), pack_fp16_sat(w[2], w[3]), pack_fp16_sat(w[4], w[5]),
                             pack_fp16_sat(w[6], w[7]));
        *reinterpret_cast<uint4 *>(dst) = q;
    }
};
template <>
struct Out<EP_FP8_E4M3> {
    static constexpr uint32_t kBlockBytes = 8;
    static __device__ __forceinline__ void store(void *dst, const float (&w)[8]) {
        uint2 q = make_uint2(pack_e4m3(w[0], w[1]) | (pack_e4m3(w[2], w[3]) << 16),
                             pack_e4m3(w[4], w[5]) | (pack_e4m3(w[6], w[7]) << 16));
        *reinterpret_cast<uint2 *>(dst) = q;
    }
};
template <>
struct Out<EP_INT8> {
    static constexpr uint32_t kBlockBytes = 8;
    static __device__ __forceinline__ void store(void *dst, const float (&w)[8]) {
        uint2 q = make_uint2(cvt_s8(w[0]) | (cvt_s8(w[1]) << 8) | (cvt_s8(w[2]) << 16) | (cvt_s8(w[3]) << 24),
                             cvt_s8(w[4]) | (cvt_s8(w[5]) << 8) | (cvt_s8(w[6]) << 16) | (cvt_s8(w[7]) << 24));
        *reinterpret_cast<uint2 *>(dst) = q;
    }
};

// ---- one group of 32 vectors: nine symbols per lane, then Eq. 5 / Eq. 19 and the store ------------
template <int DT, bool TAIL, bool CAREFUL>
__device__ __forceinline__ void decode_group(uint32_t &x, uint32_t &ptr, const uint16_t *pay, uint32_t lut_addr, uint32_t mask,
                                             uint32_t b, uint32_t lt, bool act, uint32_t last_word, float k0, float sigma,
                                             int32_t zlo, void *dst) {
    uint32_t e[9];
    e[0] = rans_step<TAIL, CAREFUL>(x, lut_addr + kCosetTableOff, mask, b, ptr, pay, lt, act, last_word);
    const uint32_t coff = e[0] & kCodeMask;          // 0 or 65536: byte offset of this coset's tables
    const uint32_t tab = lut_addr + coff;
#pragma unroll
    for (int k = 1; k <= 8; ++k)
        e[k] = rans_step<TAIL, CAREFUL>(x, tab + uint32_t(k - 1) * kLutStride, mask, b, ptr, pay, lt, act, last_word);
    if (TAIL && !act) return;
    // parity of z1 + ... + z7 = xor of the codes' lowest bits (zlo is even); it is the lowest bit of z8
    const uint32_t par = (e[1] ^ e[2] ^ e[3] ^ e[4] ^ e[5] ^ e[6] ^ e[7]) & 0x800u;
    if constexpr (DT == EP_FIELDS_I32) {
        int32_t *f = reinterpret_cast<int32_t *>(dst);
        f[0] = int32_t(coff >> 16);
#pragma unroll
        for (int k = 1; k <= 7; ++k) f[k] = int32_t((e[k] & kCodeMask) >> 11) + zlo;
        f[8] = (int32_t((e[8] & kCodeMask) >> 11) + zlo) >> 1;
        return;
    } else {
        // 4096 + code as fp32; subtracting kc = 4096 - zlo - c/2 gives p = z + c/2 exactly
        const float kc = __uint_as_float(__float_as_uint(k0) - (coff >> 6));   // one ulp here is 2^-11: c/2 = 1024 ulps
        float w[8];
#pragma unroll
        for (int k = 1; k <= 7; ++k) w[k - 1] = __uint_as_float((e[k] & kCodeMask) | kExp4096);
        w[7] = __uint_as_float((e[8] & kCodeMask) | par | kExp4096);
#pragma unroll
        for (int i = 0; i < 8; i += 2) {
            sub2(w[i], w[i + 1], kc);
            mul2(w[i], w[i + 1], sigma);
        }
        Out<DT>::store(dst, w);
    }
}

template <int DT>
struct BlockBytes { static constexpr uint32_t value = Out<DT>::kBlockBytes; };
template <>
struct BlockBytes<EP_FIELDS_I32> { static constexpr uint32_t value = 36; };

template <int DT, bool CAREFUL>
__device__ __forceinline__ void decode_tile(const JobParams &J, uint32_t tile, uint32_t lut_addr, uint32_t lane) {
    const uint32_t *rec = J.tile_index + size_t(tile) * 33u;
    uint32_t x = rec[lane];
    uint32_t ptr = rec[32];
    const uint32_t end = (tile + 1 < J.n_tiles) ? rec[33 + 32] : rec[33];
    const uint32_t v0 = tile * J.V;
    const uint32_t nv = min(J.V, J.n_vec - v0);
    const uint32_t b = J.b, mask = (1u << b) - 1u, lt = (1u << lane) - 1u;
    const uint16_t *pay = reinterpret_cast<const uint16_t *>(J.stream + J.off_payload);
    const uint32_t last_word = J.total_words ? J.total_words - 1 : 0;
    const float k0 = float(4096 - J.zlo);
    uint32_t v = v0 + lane;
    uint32_t row = v / J.per_row, col = v - row * J.per_row;
    uint8_t *dst = static_cast<uint8_t *>(J.out) + size_t(v) * BlockBytes<DT>::value;
    const uint32_t full = nv >> 5;
    for (uint32_t g = 0; g < full; ++g) {
        if (lane < 4) prefetch_l1(pay + min(ptr + 256u + 64u * lane, last_word));   // next lines of this tile's words
        const float sigma = (DT == EP_FIELDS_I32) ? 0.f : __ldg(J.scales + row);
        decode_group<DT, false, CAREFUL>(x, ptr, pay, lut_addr, mask, b, lt, true, last_word, k0, sigma, J.zlo, dst);
        dst += 32u * BlockBytes<DT>::value;
        col += 32;
        while (col >= J.per_row) { col -= J.per_row; ++row; }
    }
    if (nv & 31u) {
        const bool act = lane < (nv & 31u);
        const float sigma = (DT == EP_FIELDS_I32 || !act) ? 0.f : __ldg(J.scales + row);
        decode_group<DT, true, CAREFUL>(x, ptr, pay, lut_addr, mask, b, lt, act, last_word, k0, sigma, J.zlo, dst);
    }
    // integrity: the encoder started every state at 2^15 and the tile's words end where the next tile's begin
    const bool bad = (x != ep::kStateLow) || (ptr != end);
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(&g_ep_status, 1u);
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1) ep_decode_smem_kernel(const __grid_constant__ BatchParams P) {
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    int j = 0;
    while (j + 1 < P.n_jobs && blockIdx.x >= P.job[j + 1].cta_begin) ++j;
    const JobParams &J = P.job[j];
    const uint32_t lut_addr = uint32_t(__cvta_generic_to_shared(smem));
    build_tables_smem(J, lut_addr, warp, lane);
    __syncthreads();
    const uint32_t cta = blockIdx.x - J.cta_begin;
    for (uint32_t tile = cta * kWarps + warp; tile < J.n_tiles; tile += J.cta_count * kWarps) {
        // a damaged stream could ask for up to one word per symbol: only tiles that close to the end of the
        // payload need their word index clamped
        const uint32_t off = J.tile_index[size_t(tile) * 33u + 32u];
        const uint32_t nv = min(J.V, J.n_vec - tile * J.V);
        if (uint64_t(off) + 9ull * nv >= J.total_words) decode_tile<DT, true>(J, tile, lut_addr, lane);
        else decode_tile<DT, false>(J, tile, lut_addr, lane);
    }
}

// ---- host side -----------------------------------------------------------------------------------

int g_num_sms = 0;

int num_sms() {
    if (g_num_sms == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        g_num_sms = n;
    }
    return g_num_sms;
}

struct Range { int64_t lo, hi; bool any; };

// coordinate range from the table directory (the header's coord_min/max are not trusted)
Range coord_range(const ep_info &I) {
    Range r{0, 0, false};
    for (int c = 0; c < 2; ++c)
        for (int k = 1; k <= 8; ++k) {
            const int t = ep::table_id(c, k);
            if (!I.table_K[t]) continue;
            int64_t lo = I.table_min[t], hi = int64_t(I.table_min[t]) + I.table_K[t] - 1;
            if (k == 8) { lo *= 2; hi = 2 * hi + 1; }
            if (!r.any) { r = {lo, hi, true}; }
            else { r.lo = lo < r.lo ? lo : r.lo; r.hi = hi > r.hi ? hi : r.hi; }
        }
    return r;
}

int64_t even_base(const Range &r) {
    int64_t zlo = r.any ? r.lo : 0;
    if (zlo > -2) zlo = -2;
    return zlo & ~int64_t(1);   // floor to even
}

bool fits_smem_tables(const ep_info &I) {
    if (I.b > 11) return false;
    const Range r = coord_range(I);
    const int64_t zlo = even_base(r);
    if (r.any && r.hi - zlo > 511) return false;
    if (zlo < -512) return false;
    for (int t = 0; t < EP_NUM_TABLES; ++t) if (I.table_K[t] > kLutEntries) return false;
    return true;
}

template <int DT>
cudaError_t launch_smem(const BatchParams &P, uint32_t grid, cudaStream_t st) {
    static bool configured[64] = {};   // the attribute is per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(ep_decode_smem_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kLutBytes));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    ep_decode_smem_kernel<DT><<<grid, kThreads, kLutBytes, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

extern "C" size_t ep_decode_scratch_bytes(const ep_info *info) {
    if (!info) return 0;
    if (fits_smem_tables(*info)) return 0;
    return size_t(EP_NUM_TABLES) * (size_t(1) << info->b) * 8u;
}

extern "C" int ep_decode_batch(const ep_decode_job *jobs, int32_t n_jobs, void *stream) {
    if (!jobs || n_jobs <= 0 || n_jobs > EP_MAX_BATCH) return EP_ERR_BAD_ARG;
    const int sms = num_sms();
    if (sms <= 0) return EP_ERR_CUDA;
    BatchParams P;
    std::memset(&P, 0, sizeof(P));
    P.n_jobs = n_jobs;
    const int32_t dt = jobs[0].out_dtype;
    uint64_t tiles_total = 0;
    for (int i = 0; i < n_jobs; ++i) {
        const ep_decode_job &jb = jobs[i];
        if (!jb.info || !jb.d_stream || !jb.d_tile_index || !jb.d_out) return EP_ERR_BAD_ARG;
        if (jb.out_dtype != dt) return EP_ERR_BAD_ARG;   // one output type per launch
        if (dt != EP_FIELDS_I32 && !jb.d_row_scales) return EP_ERR_BAD_ARG;
        const ep_info &I = *jb.info;
        if (I.C == 0 || I.C % 8 || I.R == 0 || I.V == 0 || I.b < 9 || I.b > 15 || I.J != ep::kStates) return EP_ERR_BAD_ARG;
        if ((reinterpret_cast<uintptr_t>(jb.d_stream) & 3) || (reinterpret_cast<uintptr_t>(jb.d_tile_index) & 3) ||
            (reinterpret_cast<uintptr_t>(jb.d_out) & 15))
            return EP_ERR_BAD_ARG;
        if (I.table_K[0] == 0 || I.table_min[0] < 0 || int64_t(I.table_min[0]) + I.table_K[0] > 2) return EP_ERR_BAD_STREAM;
        if (!fits_smem_tables(I)) return EP_ERR_UNSUPPORTED;
        tiles_total += I.n_tiles;
    }
    // persistent CTAs: a single tensor gets one CTA per SM (or fewer if it has under 32 tiles per SM);
    // a batch shares twice the SM count in proportion to the tensors' tile counts
    const uint64_t budget = n_jobs == 1 ? uint64_t(sms) : 2ull * sms;
    uint32_t next = 0;
    for (int i = 0; i < n_jobs; ++i) {
        const ep_decode_job &jb = jobs[i];
        const ep_info &I = *jb.info;
        JobParams &J = P.job[i];
        const uint64_t want = (uint64_t(I.n_tiles) + kWarps - 1) / kWarps;
        uint64_t share = (budget * I.n_tiles + tiles_total - 1) / tiles_total;
        if (share < 1) share = 1;
        if (share > want) share = want;
        J.stream = static_cast<const uint8_t *>(jb.d_stream);
        J.tile_index = static_cast<const uint32_t *>(jb.d_tile_index);
        J.scales = jb.d_row_scales;
        J.out = jb.d_out;
        J.off_freq = I.off_tables + 8u * EP_NUM_TABLES;
        J.off_payload = I.off_payload;
        J.total_words = uint32_t(I.total_words);
        J.n_vec = uint32_t(uint64_t(I.R) * (I.C / 8));
        J.per_row = I.C / 8;
        J.V = I.V;
        J.n_tiles = I.n_tiles;
        J.b = I.b;
        J.zlo = int32_t(even_base(coord_range(I)));
        J.cta_begin = next;
        J.cta_count = uint32_t(share);
        uint32_t acc = 0;
        for (int t = 0; t < EP_NUM_TABLES; ++t) {
            J.tmin[t] = int16_t(I.table_min[t]);
            J.tK[t] = uint16_t(I.table_K[t]);
            J.foff[t] = uint16_t(acc);
            acc += I.table_K[t];
        }
        next += uint32_t(share);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (dt) {
    case EP_BF16: e = launch_smem<EP_BF16>(P, next, st); break;
    case EP_FP16: e = launch_smem<EP_FP16>(P, next, st); break;
    case EP_FP8_E4M3: e = launch_smem<EP_FP8_E4M3>(P, next, st); break;
    case EP_INT8: e = launch_smem<EP_INT8>(P, next, st); break;
    case EP_FIELDS_I32: e = launch_smem<EP_FIELDS_I32>(P, next, st); break;
    default: return EP_ERR_BAD_ARG;
    }
    return e == cudaSuccess ? EP_OK : EP_ERR_CUDA;
}

extern "C" int ep_decode_tensor(const ep_info *info, const void *d_stream, const void *d_tile_index,
                                const float *d_row_scales, int32_t out_dtype, void *d_out, void *d_scratch,
                                size_t scratch_bytes, void *stream) {
    ep_decode_job jb;
    jb.info = info;
    jb.d_stream = d_stream;
    jb.d_tile_index = d_tile_index;
    jb.d_row_scales = d_row_scales;
    jb.out_dtype = out_dtype;
    jb.d_out = d_out;
    jb.d_scratch = d_scratch;
    jb.scratch_bytes = scratch_bytes;
    return ep_decode_batch(&jb, 1, stream);
}

extern "C" int ep_last_device_status(void *stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return EP_ERR_CUDA;
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_ep_status, sizeof(v)) != cudaSuccess) return EP_ERR_CUDA;
    if (v && cudaMemcpyToSymbol(g_ep_status, &zero, sizeof(zero)) != cudaSuccess) return EP_ERR_CUDA;
    return v ? EP_ERR_BAD_STREAM : EP_OK;
}
