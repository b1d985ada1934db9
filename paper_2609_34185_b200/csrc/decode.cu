// Fused EntroPack decode for sm_100a (paper Sec. 3.7): tiled 32-state rANS symbol decode (Eq. 18),
// arithmetic inverse of the field representation (Eq. 5), multiplication by the fp32 row scale and
// rounding to the output type (Eq. 19), written straight to the weight tensor.  No symbol tensor,
// no codebook, no tensor cores (the path is not a contraction).
//
// Mapping: one warp per tile, one rANS state per lane (the paper's layout); a CTA of 32 warps
// builds the seventeen slot->(frequency, offset, value) lookup tables once in shared memory from the
// stream's frequency tables and then streams tiles through them.  A lookup entry is one 32-bit word
//     [31:21] f      [20:11] code     [10:0] u - F
// where `code` is the symbol's coordinate relative to an even base zlo (z - zlo; 2m - zlo for the m
// field; 32c for the coset, which makes (entry & 0x1FF800) the byte offset of coset c's tables).
// f < 2^11 always: a table with a single symbol at b = 11 (f = 2^11) goes to the large-table path.
// (entry & 0x1FF800) | 0x45800000 is the fp32 number 4096 + code, so one subtraction of
// 4096 - zlo - c/2 yields the lattice coordinate p exactly, and one fp32 multiply by the row scale
// gives the product of Eq. 19 with the same operands and rounding as the definition.
//
// Payload words reach the lanes through a per-warp ring in shared memory, filled 512 bytes at a
// time by cp.async (16 bytes per lane, source clamped to the end of the payload) a few chunks ahead
// of the read cursor; the first 640 bytes of the ring are mirrored behind its end so that the nine
// steps of a group never have to wrap an address.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "stream.hpp"

namespace {

constexpr int kThreads = 1024;                         // one CTA per SM: 32 warps = 32 tiles in flight
constexpr int kWarps = kThreads / 32;
constexpr uint32_t kLutEntries = 2048;                 // 2^11 slots per table
constexpr uint32_t kLutStride = kLutEntries * 4;       // bytes per table in shared memory
constexpr uint32_t kCosetTableOff = 16 * kLutStride;   // coset table sits after the 16 coordinate tables
constexpr uint32_t kLutBytes = 17 * kLutStride;        // 139264
constexpr uint32_t kRingBytes = 2048;                  // four 512-byte chunks per warp
constexpr uint32_t kRingMirror = 640;                  // >= 9 steps * 32 words * 2 bytes + one lane span
constexpr uint32_t kRingStride = kRingBytes + kRingMirror;
constexpr uint32_t kSmemBytes = kLutBytes + kWarps * kRingStride;   // 225280
constexpr uint32_t kCodeMask = 0x001FF800u;            // 10-bit code field
constexpr uint32_t kExp4096 = 0x45800000u;             // fp32 bit pattern of 4096.0
constexpr uint32_t kOwnSlots = 16;                     // table build: slots of a symbol that its own lane writes

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
    uint32_t V, n_tiles, b;       // n_tiles: tiles of the whole tensor
    uint32_t tile0, tile_cnt;     // the tiles this launch decodes: [tile0, tile0 + tile_cnt)
    int32_t zlo;                  // even, <= -2
    uint32_t rounds;              // ceil(tile_cnt / warps): in one round the 32 warps of a CTA take 32 consecutive tiles
    uint32_t round_cost;          // work of one round in groups of 32 vectors (ceil(V / 32))
    uint32_t cost_begin;          // sum of rounds * round_cost over the jobs before this one
    int16_t tmin[EP_NUM_TABLES];
    uint16_t tK[EP_NUM_TABLES];
    uint16_t foff[EP_NUM_TABLES]; // start of table t's frequencies, in u16 units
};

struct BatchParams {
    JobParams job[EP_MAX_BATCH];
    uint32_t cost_per_cta;        // ceil(sum of rounds * round_cost over all jobs / CTAs of the launch)
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
__device__ __forceinline__ void cp_async16(uint32_t dst, uint64_t src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// two fp32 lanes per instruction (sm_100 packed fp32), operands kept as 64-bit register pairs
__device__ __forceinline__ uint64_t pack64(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ void unpack64(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
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
__device__ __forceinline__ uint32_t pack_e5m2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t cvt_u8(float v) {
    uint32_t r;
    asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r & 0xFFu;
}
__device__ __forceinline__ uint32_t cvt_s8(float v) {
    int32_t r;
    asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(r) : "f"(v));
    return uint32_t(r) & 0xFFu;
}

// ---- lookup-table construction (per CTA, from the stream's frequency tables) ---------------------
// Warp t fills table t.  Symbols are taken 32 at a time: a warp scan gives each lane its symbol's
// first slot, every lane writes the first sixteen slots of its own symbol, and the few symbols with more
// slots than that are then filled by the whole warp, one after the other (that loop is serial: its length,
// not the number of stores, is what the build time depends on).
__device__ __forceinline__ void build_tables_smem(const JobParams &J, uint32_t lut_addr, uint32_t warp, uint32_t lane) {
  for (uint32_t t = warp; t < EP_NUM_TABLES; t += kWarps) {
    const uint32_t K = J.tK[t];
    if (K == 0) continue;
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
        const uint32_t entry = (f << 21) | ((code & 0x3FFu) << 11);
        if (f >= kLutEntries) atomicOr(&g_ep_status, 1u);   // not a stream the launcher sends here: f does not fit its field
#pragma unroll
        for (uint32_t u = 0; u < kOwnSlots; ++u)
            if (u < f && first + u < kLutEntries) sts32(base + 4u * (first + u), entry | u);
        uint32_t big = __ballot_sync(0xFFFFFFFFu, f > kOwnSlots);
        while (big) {
            const int i = __ffs(big) - 1;
            big &= big - 1;
            const uint32_t fi = __shfl_sync(0xFFFFFFFFu, f, i);
            const uint32_t Fi = __shfl_sync(0xFFFFFFFFu, first, i);
            const uint32_t ei = __shfl_sync(0xFFFFFFFFu, entry, i);
            for (uint32_t u = kOwnSlots + lane; u < fi && Fi + u < kLutEntries; u += 32) sts32(base + 4u * (Fi + u), ei | u);
        }
        run += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    // frequencies of a damaged stream may sum to less than 2^b: no slot keeps what an earlier CTA left there
    // (the coset entry's code field is added to a shared-memory address)
    for (uint32_t u = run + lane; u < (1u << J.b) && u < kLutEntries; u += 32) sts32(base + 4u * u, 0u);
  }
}

// ---- one rANS symbol (Eq. 18) followed by renormalisation --------------------------------------
// x: this lane's state; wa: shared-memory byte address of the tile's word cursor (same in all lanes).
// Lanes that need a word take them in lane order: lane l reads the word popc(ballot & lanes below l)
// places after the cursor (every lane reads, only the needy merge); the cursor then advances by
// popc(ballot) words.  Returns the table entry.
template <uint32_t TABLE_OFF>
__device__ __forceinline__ uint32_t rans_step(uint32_t &x, uint32_t table_addr, uint32_t mask, uint32_t b, uint32_t &wa,
                                              uint32_t lt) {
    uint32_t e;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .b32 u, f, q, bias, bal, t, w;\n\t"
        "and.b32 u, %1, %3;\n\t"
        "shl.b32 u, u, 2;\n\t"
        "add.u32 u, u, %5;\n\t"
        "ld.shared.u32 %0, [u + %7];\n\t"
        "shr.u32 f, %0, 21;\n\t"
        "and.b32 bias, %0, 0x7FF;\n\t"
        "shr.u32 q, %1, %4;\n\t"
        "mad.lo.u32 %1, f, q, bias;\n\t"
        "setp.lt.u32 p, %1, 32768;\n\t"
        "vote.sync.ballot.b32 bal, p, 0xffffffff;\n\t"
        "and.b32 t, bal, %6;\n\t"
        "popc.b32 t, t;\n\t"
        "shl.b32 t, t, 1;\n\t"
        "add.u32 t, t, %2;\n\t"
        "ld.shared.u16 w, [t];\n\t"
        "@p mad.lo.u32 %1, %1, 65536, w;\n\t"
        "popc.b32 t, bal;\n\t"
        "shl.b32 t, t, 1;\n\t"
        "add.u32 %2, %2, t;\n\t"
        "}"
        : "=&r"(e), "+r"(x), "+r"(wa)
        : "r"(mask), "r"(b), "r"(table_addr), "r"(lt), "n"(TABLE_OFF)
        : "memory");
    return e;
}

// the same for the last, partly filled group of a tile: lanes without a vector leave their state alone
__device__ __forceinline__ uint32_t rans_step_tail(uint32_t &x, uint32_t table_addr, uint32_t mask, uint32_t b, uint32_t &wa,
                                                   uint32_t lt, bool act) {
    uint32_t e = 0;
    bool need = false;
    if (act) {
        e = lds32(table_addr + ((x & mask) << 2));
        x = (e >> 21) * (x >> b) + (e & 0x7FFu);
        need = x < ep::kStateLow;
    }
    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, need);
    if (need) {
        uint16_t w;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(w) : "r"(wa + 2u * __popc(bal & lt)));
        x = (x << 16) | w;
    }
    wa += 2u * __popc(bal);
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

template <>
struct Out<EP_FP32> {
    static constexpr uint32_t kBlockBytes = 32;
    static __device__ __forceinline__ void store(void *dst, const float (&w)[8]) {
        reinterpret_cast<float4 *>(dst)[0] = make_float4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<float4 *>(dst)[1] = make_float4(w[4], w[5], w[6], w[7]);
    }
};
template <>
struct Out<EP_FP8_E5M2> {
    static constexpr uint32_t kBlockBytes = 8;
    static __device__ __forceinline__ void store(void *dst, const float (&w)[8]) {
        uint2 q = make_uint2(pack_e5m2(w[0], w[1]) | (pack_e5m2(w[2], w[3]) << 16),
                             pack_e5m2(w[4], w[5]) | (pack_e5m2(w[6], w[7]) << 16));
        *reinterpret_cast<uint2 *>(dst) = q;
    }
};
template <>
struct Out<EP_UINT8> {
    static constexpr uint32_t kBlockBytes = 8;
    static __device__ __forceinline__ void store(void *dst, const float (&w)[8]) {
        uint2 q = make_uint2(cvt_u8(w[0]) | (cvt_u8(w[1]) << 8) | (cvt_u8(w[2]) << 16) | (cvt_u8(w[3]) << 24),
                             cvt_u8(w[4]) | (cvt_u8(w[5]) << 8) | (cvt_u8(w[6]) << 16) | (cvt_u8(w[7]) << 24));
        *reinterpret_cast<uint2 *>(dst) = q;
    }
};

template <int DT>
struct BlockBytes { static constexpr uint32_t value = Out<DT>::kBlockBytes; };
template <>
struct BlockBytes<EP_FIELDS_I32> { static constexpr uint32_t value = 36; };

// ---- one group of 32 vectors: nine symbols per lane, then Eq. 5 / Eq. 19 and the store ------------
template <int DT, bool TAIL>
__device__ __forceinline__ void decode_group(uint32_t &x, uint32_t &wa, uint32_t lut_addr, uint32_t mask, uint32_t b, uint32_t lt,
                                             bool act, uint32_t k0_bits, float sigma, int32_t zlo, void *dst) {
    uint32_t e[9];
    e[0] = TAIL ? rans_step_tail(x, lut_addr + kCosetTableOff, mask, b, wa, lt, act)
                : rans_step<kCosetTableOff>(x, lut_addr, mask, b, wa, lt);
    // 0 or 65536: byte offset of this coset's tables (one bit only, so that a damaged table cannot point elsewhere)
    const uint32_t coff = e[0] & 0x10000u;
    const uint32_t tab = lut_addr + coff;
    if (TAIL) {
#pragma unroll
        for (int k = 1; k <= 8; ++k) e[k] = rans_step_tail(x, tab + uint32_t(k - 1) * kLutStride, mask, b, wa, lt, act);
    } else {
        e[1] = rans_step<0 * kLutStride>(x, tab, mask, b, wa, lt);
        e[2] = rans_step<1 * kLutStride>(x, tab, mask, b, wa, lt);
        e[3] = rans_step<2 * kLutStride>(x, tab, mask, b, wa, lt);
        e[4] = rans_step<3 * kLutStride>(x, tab, mask, b, wa, lt);
        e[5] = rans_step<4 * kLutStride>(x, tab, mask, b, wa, lt);
        e[6] = rans_step<5 * kLutStride>(x, tab, mask, b, wa, lt);
        e[7] = rans_step<6 * kLutStride>(x, tab, mask, b, wa, lt);
        e[8] = rans_step<7 * kLutStride>(x, tab, mask, b, wa, lt);
    }
    if (TAIL && !act) return;
    // parity of z1 + ... + z7 = xor of the codes' lowest bits (zlo is even); it is the lowest bit of z8
    const uint32_t par = (e[1] ^ e[2] ^ e[3] ^ e[4] ^ e[5] ^ e[6] ^ e[7]) & 0x800u;
    if constexpr (DT == EP_FIELDS_I32) {
        int32_t *f = reinterpret_cast<int32_t *>(dst);
        f[0] = int32_t(coff >> 16);
#pragma unroll
        for (int k = 1; k <= 7; ++k) f[k] = int32_t((e[k] & kCodeMask) >> 11) + zlo;
        f[8] = (int32_t((e[8] & kCodeMask) >> 11) + zlo) >> 1;
    } else {
        // (entry & mask) | 0x45800000 is 4096 + code as fp32; subtracting kc = 4096 - zlo - c/2 gives
        // p = z + c/2 exactly (one ulp here is 2^-11, so c/2 is 1024 ulps of the bit pattern)
        const uint32_t kc = k0_bits - (coff >> 6);
        const uint64_t kk = pack64(kc, kc);
        const uint64_t ss = pack64(__float_as_uint(sigma), __float_as_uint(sigma));
        uint32_t xb[8];
#pragma unroll
        for (int k = 1; k <= 7; ++k) xb[k - 1] = (e[k] & kCodeMask) | kExp4096;
        xb[7] = (e[8] & kCodeMask) | par | kExp4096;
        float w[8];
#pragma unroll
        for (int i = 0; i < 8; i += 2) unpack64(mul2(sub2(pack64(xb[i], xb[i + 1]), kk), ss), w[i], w[i + 1]);
        Out<DT>::store(dst, w);
    }
}

// ---- payload ring ------------------------------------------------------------------------------------
// chunk c of a tile = global bytes [a0 + 512c, a0 + 512c + 512), a0 = tile's first word rounded down to
// 16 bytes; it lives in ring slot c & 3.  `room` = bytes from a0 to the end of the payload: nothing
// beyond it is read (cp.async zero-fills the rest).
__device__ __forceinline__ void ring_issue(uint32_t ring, uint64_t a0, uint32_t room, uint32_t c, uint32_t lane) {
    uint32_t o = 512u * c + 16u * lane;
    uint32_t n = 16;
    if (o + 16u > room) {
        n = o < room ? room - o : 0u;
        if (n == 0) o = 0;                       // nothing is read, but keep the address a valid one
    }
    const uint32_t slot = c & 3u;
    const uint32_t dst = ring + 512u * slot + 16u * lane;
    cp_async16(dst, a0 + o, n);
    if (slot == 0 || (slot == 1 && lane < 8)) cp_async16(dst + kRingBytes, a0 + o, n);   // mirror of the first 640 bytes
    cp_async_commit();
}

// The cursor entered a new 512-byte chunk: request chunks up to three ahead of it and wait for all but
// the newest.  `threshold` = start of the chunk after the cursor's at the previous service; chunks up
// to (threshold >> 9) + 2 have been requested.  A group touches at most 576 + 62 bytes from its start,
// i.e. chunks cur .. cur+2, which are complete after this call.
__device__ __forceinline__ void ring_service(uint32_t ring, uint64_t a0, uint32_t room, uint32_t pos, uint32_t &threshold,
                                             uint32_t lane) {
    const uint32_t cur = pos >> 9;
    for (uint32_t c = (threshold >> 9) + 3u; c < cur + 4u; ++c) ring_issue(ring, a0, room, c, lane);
    cp_async_wait<1>();
    __syncwarp();
    threshold = 512u * (cur + 1u);
}

// Plain C++ version of the tile loop, used for the field-dump mode and for tensors with fewer than 32
// blocks per row (WIDE = false: a group may then cross several rows).
template <int DT, bool WIDE>
__device__ __forceinline__ void decode_tile(const JobParams &J, uint32_t tile, uint32_t lut_addr, uint32_t ring, uint32_t lane) {
    const uint32_t *rec = J.tile_index + size_t(tile) * 33u;
    uint32_t x = rec[lane];
    const uint32_t off = min(rec[32], J.total_words);   // a damaged index must not move reads outside the payload
    const uint32_t end = (tile + 1 < J.n_tiles) ? rec[33 + 32] : rec[33];
    const uint32_t v0 = tile * J.V;
    const uint32_t nv = min(J.V, J.n_vec - v0);
    const uint32_t b = J.b, mask = (1u << b) - 1u, lt = (1u << lane) - 1u;
    const uint32_t per_row = J.per_row;
    const uint64_t pay = reinterpret_cast<uint64_t>(J.stream + J.off_payload);
    const uint64_t first = pay + 2ull * off;
    const uint64_t a0 = first & ~15ull;
    const uint32_t lead = uint32_t(first - a0);
    const uint32_t room = uint32_t(pay + 2ull * J.total_words - a0);     // the payload is shorter than 4 GB
    uint32_t pos = lead;          // byte position of the cursor relative to a0
    uint32_t threshold;           // next chunk boundary the cursor has not yet crossed
    for (uint32_t c = 0; c < 4; ++c) ring_issue(ring, a0, room, c, lane);
    cp_async_wait<1>();
    __syncwarp();
    threshold = 512u;
    const uint32_t k0_bits = __float_as_uint(float(4096 - J.zlo));
    uint32_t v = v0 + lane;
    uint32_t row = v / per_row, col = v - row * per_row;
    uint8_t *dst = static_cast<uint8_t *>(J.out) + size_t(v) * BlockBytes<DT>::value;
    const uint32_t full = nv >> 5;
    for (uint32_t g = 0; g < full; ++g) {
        if (__any_sync(0xFFFFFFFFu, pos >= threshold)) ring_service(ring, a0, room, pos, threshold, lane);
        const uint32_t wa0 = ring + (pos & (kRingBytes - 1u));
        uint32_t wa = wa0;
        const float sigma = (DT == EP_FIELDS_I32) ? 0.f : __ldg(J.scales + row);
        decode_group<DT, false>(x, wa, lut_addr, mask, b, lt, true, k0_bits, sigma, J.zlo, dst);
        pos += wa - wa0;
        dst += 32u * BlockBytes<DT>::value;
        col += 32;
        if (WIDE) {
            const bool wrap = col >= per_row;
            col -= wrap ? per_row : 0u;
            row += wrap ? 1u : 0u;
        } else {
            while (col >= per_row) { col -= per_row; ++row; }
        }
    }
    if (nv & 31u) {
        if (__any_sync(0xFFFFFFFFu, pos >= threshold)) ring_service(ring, a0, room, pos, threshold, lane);
        const uint32_t wa0 = ring + (pos & (kRingBytes - 1u));
        uint32_t wa = wa0;
        const bool act = lane < (nv & 31u);
        const float sigma = (DT == EP_FIELDS_I32 || !act) ? 0.f : __ldg(J.scales + row);
        decode_group<DT, true>(x, wa, lut_addr, mask, b, lt, act, k0_bits, sigma, J.zlo, dst);
        pos += wa - wa0;
    }
    cp_async_wait<0>();          // nothing may still be landing in the ring when the next tile starts
    __syncwarp();
    // integrity: the encoder started every state at 2^15 and the tile's words end where the next tile's begin
    const bool bad = (x != ep::kStateLow) || (off + ((pos - lead) >> 1) != end);
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(&g_ep_status, 1u);
}

// ---- the hot loop in PTX -------------------------------------------------------------------------------
// All full groups of one tile.  Written as one asm statement so that every branch can be marked
// warp-uniform (bra.uni) and the rare work - refilling the payload ring, moving to the next row, leaving
// the loop - sits out of line behind ONE warp vote per group.  Per group: 9 x rans step, Eq. 5 / Eq. 19
// on eight weights, one vector store.
//
// Register roles (asm operands):
//   x      rANS state                      wa    cursor (shared-memory byte address)
//   wthr   cursor value that triggers the next ring service (next 512-byte chunk boundary)
//   wbase  wa - (byte position of the cursor relative to a0)
//   doff   byte offset of this lane's block in the output
//   chg    value of doff at which this lane enters its next row;  row = row index;  sig = row scale bits
//   lim    min(chg, endo): the fast path compares doff with this alone;  endo = doff after the last group
//   srcp, rem, nextc  ring refill state: global address of this lane's 16 bytes of chunk nextc and
//                     the payload bytes left from there (may be <= 0)
#define EP_S_FQ(E)                                              \
    "shr.u32 f, " E ", 21;\n\t"                                 \
    "shr.u32 q, %0, %14;\n\t"
#define EP_S_FETCH                                              \
    "and.b32 t, bal, %12;\n\t"                                  \
    "popc.b32 t, t;\n\t"                                        \
    "shl.b32 t, t, 1;\n\t"                                      \
    "add.u32 t, t, %1;\n\t"                                     \
    "ld.shared.u16 w, [t];\n\t"                                 \
    "@p mad.lo.u32 %0, %0, 65536, w;\n\t"                       \
    "popc.b32 t, bal;\n\t"                                      \
    "shl.b32 t, t, 1;\n\t"                                      \
    "add.u32 %1, %1, t;\n\t"
#define EP_S_STEP(E, TAB, OFF)                                  \
    "and.b32 u, %0, %13;\n\t"                                   \
    "shl.b32 u, u, 2;\n\t"                                      \
    "add.u32 u, u, " TAB ";\n\t"                                \
    "ld.shared.u32 " E ", [u+" OFF "];\n\t"                     \
    EP_S_FQ(E)                                                  \
    "and.b32 bias, " E ", 0x7FF;\n\t"                           \
    "mad.lo.u32 %0, f, q, bias;\n\t"                            \
    "setp.lt.u32 p, %0, 32768;\n\t"                             \
    "vote.sync.ballot.b32 bal, p, 0xffffffff;\n\t"              \
    EP_S_FETCH

#define EP_S_PAIR(P, XA, XB, WA, WB)                            \
    "mov.b64 " P ", {" XA ", " XB "};\n\t"                      \
    "sub.rn.f32x2 " P ", " P ", kk;\n\t"                        \
    "mul.rn.f32x2 " P ", " P ", ss;\n\t"                        \
    "mov.b64 {" WA ", " WB "}, " P ";\n\t"

#define EP_S_STORE_BF16                                         \
    "cvt.rn.bf16x2.f32 o0, w1, w0;\n\t"                         \
    "cvt.rn.bf16x2.f32 o1, w3, w2;\n\t"                         \
    "cvt.rn.bf16x2.f32 o2, w5, w4;\n\t"                         \
    "cvt.rn.bf16x2.f32 o3, w7, w6;\n\t"                         \
    "st.global.v4.b32 [ad], {o0, o1, o2, o3};\n\t"
#define EP_S_STORE_FP16                                         \
    "cvt.rn.satfinite.f16x2.f32 o0, w1, w0;\n\t"                \
    "cvt.rn.satfinite.f16x2.f32 o1, w3, w2;\n\t"                \
    "cvt.rn.satfinite.f16x2.f32 o2, w5, w4;\n\t"                \
    "cvt.rn.satfinite.f16x2.f32 o3, w7, w6;\n\t"                \
    "st.global.v4.b32 [ad], {o0, o1, o2, o3};\n\t"
#define EP_S_STORE_E4M3                                         \
    "cvt.rn.satfinite.e4m3x2.f32 h0, w1, w0;\n\t"               \
    "cvt.rn.satfinite.e4m3x2.f32 h1, w3, w2;\n\t"               \
    "cvt.rn.satfinite.e4m3x2.f32 h2, w5, w4;\n\t"               \
    "cvt.rn.satfinite.e4m3x2.f32 h3, w7, w6;\n\t"               \
    "mov.b32 o0, {h0, h1};\n\t"                                 \
    "mov.b32 o1, {h2, h3};\n\t"                                 \
    "st.global.v2.b32 [ad], {o0, o1};\n\t"
#define EP_S_STORE_FP32                                         \
    "mov.b32 o0, w0;\n\t"                                       \
    "mov.b32 o1, w1;\n\t"                                       \
    "mov.b32 o2, w2;\n\t"                                       \
    "mov.b32 o3, w3;\n\t"                                       \
    "st.global.v4.b32 [ad], {o0, o1, o2, o3};\n\t"              \
    "mov.b32 o0, w4;\n\t"                                       \
    "mov.b32 o1, w5;\n\t"                                       \
    "mov.b32 o2, w6;\n\t"                                       \
    "mov.b32 o3, w7;\n\t"                                       \
    "st.global.v4.b32 [ad+16], {o0, o1, o2, o3};\n\t"
#define EP_S_STORE_E5M2                                         \
    "cvt.rn.satfinite.e5m2x2.f32 h0, w1, w0;\n\t"               \
    "cvt.rn.satfinite.e5m2x2.f32 h1, w3, w2;\n\t"               \
    "cvt.rn.satfinite.e5m2x2.f32 h2, w5, w4;\n\t"               \
    "cvt.rn.satfinite.e5m2x2.f32 h3, w7, w6;\n\t"               \
    "mov.b32 o0, {h0, h1};\n\t"                                 \
    "mov.b32 o1, {h2, h3};\n\t"                                 \
    "st.global.v2.b32 [ad], {o0, o1};\n\t"
/* one-byte integers: round to nearest even into s32 (out-of-range values end at INT_MIN / INT_MAX, NaN at 0), then
   saturate and pack four at a time: cvt.pack d, a, b, c gives (c << 16) | sat(a) << 8 | sat(b) */
#define EP_S_STORE_UINT8                                        \
    "cvt.rni.s32.f32 x1, w0;\n\t"                               \
    "cvt.rni.s32.f32 x2, w1;\n\t"                               \
    "cvt.rni.s32.f32 x3, w2;\n\t"                               \
    "cvt.rni.s32.f32 x4, w3;\n\t"                               \
    "cvt.rni.s32.f32 x5, w4;\n\t"                               \
    "cvt.rni.s32.f32 x6, w5;\n\t"                               \
    "cvt.rni.s32.f32 x7, w6;\n\t"                               \
    "cvt.rni.s32.f32 x8, w7;\n\t"                               \
    "cvt.pack.sat.u8.s32.b32 o2, x4, x3, 0;\n\t"                \
    "cvt.pack.sat.u8.s32.b32 o0, x2, x1, o2;\n\t"               \
    "cvt.pack.sat.u8.s32.b32 o3, x8, x7, 0;\n\t"                \
    "cvt.pack.sat.u8.s32.b32 o1, x6, x5, o3;\n\t"               \
    "st.global.v2.b32 [ad], {o0, o1};\n\t"
#define EP_S_STORE_INT8                                         \
    "cvt.rni.s32.f32 x1, w0;\n\t"                               \
    "cvt.rni.s32.f32 x2, w1;\n\t"                               \
    "cvt.rni.s32.f32 x3, w2;\n\t"                               \
    "cvt.rni.s32.f32 x4, w3;\n\t"                               \
    "cvt.rni.s32.f32 x5, w4;\n\t"                               \
    "cvt.rni.s32.f32 x6, w5;\n\t"                               \
    "cvt.rni.s32.f32 x7, w6;\n\t"                               \
    "cvt.rni.s32.f32 x8, w7;\n\t"                               \
    "cvt.pack.sat.s8.s32.b32 o2, x4, x3, 0;\n\t"                \
    "cvt.pack.sat.s8.s32.b32 o0, x2, x1, o2;\n\t"               \
    "cvt.pack.sat.s8.s32.b32 o3, x8, x7, 0;\n\t"                \
    "cvt.pack.sat.s8.s32.b32 o1, x6, x5, o3;\n\t"               \
    "st.global.v2.b32 [ad], {o0, o1};\n\t"

#define EP_FULL_GROUPS_ASM(STORE, GROUP_BYTES)                                                                        \
    asm volatile(                                                                                                     \
        "{\n\t"                                                                                                       \
        ".reg .pred p, ps, pw, pa, pl, pq, pr, pv, pm;\n\t"                                                           \
        ".reg .b32 u, f, q, bias, bal, t, w, coff, tab, kc, par, pos, cur, clim, n, slot, d, mlim;\n\t"               \
        ".reg .b32 e0, e1, e2, e3, e4, e5, e6, e7, e8, x1, x2, x3, x4, x5, x6, x7, x8, o0, o1, o2, o3;\n\t"           \
        ".reg .b16 h0, h1, h2, h3;\n\t"                                                                               \
        ".reg .f32 w0, w1, w2, w3, w4, w5, w6, w7;\n\t"                                                               \
        ".reg .b64 kk, ss, p0, p1, p2, p3, ad, src;\n\t"                                                              \
        "setp.ge.u32 pl, %7, %23;\n\t"                                                                                \
        "vote.sync.any.pred pl, pl, 0xffffffff;\n\t"                                                                  \
        "@pl bra.uni EP_DONE;\n\t"                                                                                    \
        "EP_LOOP:\n\t"                                                                                                \
        EP_S_STEP("e0", "%15", "131072")                                                                              \
        "and.b32 coff, e0, 0x1FF800;\n\t"                                                                              \
        "add.u32 tab, %15, coff;\n\t"                                                                                 \
        EP_S_STEP("e1", "tab", "0")                                                                                   \
        EP_S_STEP("e2", "tab", "8192")                                                                                \
        EP_S_STEP("e3", "tab", "16384")                                                                               \
        EP_S_STEP("e4", "tab", "24576")                                                                               \
        EP_S_STEP("e5", "tab", "32768")                                                                               \
        EP_S_STEP("e6", "tab", "40960")                                                                               \
        EP_S_STEP("e7", "tab", "49152")                                                                               \
        EP_S_STEP("e8", "tab", "57344")                                                                               \
        /* Eq. 5: 4096 + code as fp32, minus kc = 4096 - zlo - c/2 (one ulp = 2^-11, c/2 = 1024 ulps) */              \
        "shr.u32 t, coff, 6;\n\t"                                                                                     \
        "sub.u32 kc, %18, t;\n\t"                                                                                     \
        "lop3.b32 x1, e1, 0x1FF800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 x2, e2, 0x1FF800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 x3, e3, 0x1FF800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 x4, e4, 0x1FF800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 x5, e5, 0x1FF800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 x6, e6, 0x1FF800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 x7, e7, 0x1FF800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 par, e1, e2, e3, 0x96;\n\t"                                                                         \
        "lop3.b32 par, par, e4, e5, 0x96;\n\t"                                                                        \
        "lop3.b32 par, par, e6, e7, 0x96;\n\t"                                                                        \
        "lop3.b32 par, par, 0x800, 0x45800000, 0xEA;\n\t"                                                             \
        "lop3.b32 x8, e8, 0x1FF800, par, 0xEA;\n\t"                                                                    \
        "mov.b64 kk, {kc, kc};\n\t"                                                                                   \
        "mov.b64 ss, {%6, %6};\n\t"                                                                                   \
        EP_S_PAIR("p0", "x1", "x2", "w0", "w1")                                                                       \
        EP_S_PAIR("p1", "x3", "x4", "w2", "w3")                                                                       \
        EP_S_PAIR("p2", "x5", "x6", "w4", "w5")                                                                       \
        EP_S_PAIR("p3", "x7", "x8", "w6", "w7")                                                                       \
        "cvt.u64.u32 ad, %7;\n\t"                                                                                     \
        "add.s64 ad, ad, %19;\n\t"                                                                                    \
        STORE                                                                                                         \
        "add.u32 %7, %7, " #GROUP_BYTES ";\n\t"                                                                       \
        /* one vote for everything rare: go on only if no lane crossed a chunk boundary or reached its lim */        \
        "setp.lt.u32 ps, %1, %2;\n\t"                                                                                 \
        "setp.lt.and.u32 pq, %7, %8, ps;\n\t"                                                                         \
        "vote.sync.all.pred pq, pq, 0xffffffff;\n\t"   /* a vote result is uniform to the compiler as well */         \
        "@pq bra.uni EP_LOOP;\n\t"                                                                                    \
        "setp.ge.u32 pr, %7, %8;\n\t"                                                                                 \
        "vote.sync.any.pred pr, pr, 0xffffffff;\n\t"                                                                  \
        "@!pr bra.uni EP_SVCCHK;\n\t"                                                                                 \
        /* ---- some lane moved to the next row (reload its scale), or the tile's full groups are done ---- */        \
        "setp.ge.u32 pw, %7, %4;\n\t"                                                                                 \
        "@pw add.u32 %4, %4, %17;\n\t"                                                                                \
        "@pw add.u32 %5, %5, 1;\n\t"                                                                                  \
        "min.u32 t, %5, %22;\n\t"                                                                                     \
        "mul.wide.u32 ad, t, 4;\n\t"                                                                                  \
        "add.s64 ad, ad, %20;\n\t"                                                                                    \
        "@pw ld.global.nc.b32 %6, [ad];\n\t"                                                                          \
        "min.u32 %8, %4, %23;\n\t"                                                                                    \
        "setp.ge.u32 pl, %7, %23;\n\t"                                                                                \
        "vote.sync.any.pred pl, pl, 0xffffffff;\n\t"                                                                  \
        "@pl bra.uni EP_DONE;\n\t"                                                                                    \
        "EP_SVCCHK:\n\t"                                                                                              \
        "setp.ge.u32 ps, %1, %2;\n\t"                                                                                 \
        "vote.sync.any.pred ps, ps, 0xffffffff;\n\t"                                                                  \
        "@!ps bra.uni EP_LOOP;\n\t"                                                                                   \
        /* ---- the cursor entered a new 512-byte chunk: request chunks up to cur+3, wait for all but the newest */   \
        "sub.u32 pos, %1, %3;\n\t"                                                                                    \
        "shr.u32 cur, pos, 9;\n\t"                                                                                    \
        "add.u32 clim, cur, 4;\n\t"                                                                                   \
        "sub.u32 t, %24, %16;\n\t"                     /* 16 * lane */                                                \
        "setp.lt.u32 pm, t, 128;\n\t"                                                                                 \
        "selp.u32 mlim, 2, 1, pm;\n\t"                 /* slot 0 is mirrored whole, slot 1 by lanes 0..7 */           \
        "EP_SVC_LOOP:\n\t"                                                                                            \
        "setp.ge.u32 pq, %11, clim;\n\t"                                                                              \
        "vote.sync.any.pred pq, pq, 0xffffffff;\n\t"                                                                  \
        "@pq bra.uni EP_SVC_DONE;\n\t"                                                                                \
        "min.s32 n, %10, 16;\n\t"                                                                                     \
        "max.s32 n, n, 0;\n\t"                                                                                        \
        "setp.gt.s32 pv, %10, 0;\n\t"                                                                                 \
        "selp.b64 src, %9, %21, pv;\n\t"                                                                              \
        "and.b32 slot, %11, 3;\n\t"                                                                                   \
        "mad.lo.u32 d, slot, 512, %24;\n\t"                                                                           \
        "cp.async.cg.shared.global [d], [src], 16, n;\n\t"                                                            \
        "setp.lt.u32 pm, slot, mlim;\n\t"                                                                             \
        "@pm cp.async.cg.shared.global [d+2048], [src], 16, n;\n\t"                                                   \
        "cp.async.commit_group;\n\t"                                                                                  \
        "add.s64 %9, %9, 512;\n\t"                                                                                    \
        "sub.s32 %10, %10, 512;\n\t"                                                                                  \
        "add.u32 %11, %11, 1;\n\t"                                                                                    \
        "bra.uni EP_SVC_LOOP;\n\t"                                                                                    \
        "EP_SVC_DONE:\n\t"                                                                                            \
        "cp.async.wait_group 1;\n\t"                                                                                  \
        "bar.warp.sync 0xffffffff;\n\t"                                                                               \
        "and.b32 t, pos, 2047;\n\t"                                                                                   \
        "add.u32 %1, %16, t;\n\t"                                                                                     \
        "sub.u32 %3, %1, pos;\n\t"                                                                                    \
        "shl.b32 t, cur, 9;\n\t"                                                                                      \
        "add.u32 t, t, 512;\n\t"                                                                                      \
        "add.u32 %2, %3, t;\n\t"                                                                                      \
        "bra.uni EP_LOOP;\n\t"                                                                                        \
        "EP_DONE:\n\t"                                                                                                \
        "}"                                                                                                           \
        /* every read-write operand is early-clobber: the loop reads the inputs after it has updated them */         \
        : "+&r"(x), "+&r"(wa), "+&r"(wthr), "+&r"(wbase), "+&r"(chg), "+&r"(row), "+&r"(sig), "+&r"(doff),            \
          "+&r"(lim), "+&l"(srcp), "+&r"(rem), "+&r"(nextc)                                                           \
        : "r"(lt), "r"(mask), "r"(b), "r"(lut_addr), "r"(ring), "r"(row_bytes), "r"(k0_bits), "l"(out_base),         \
          "l"(scales), "l"(a0), "r"(row_max), "r"(endo), "r"(ring_lane)                                               \
        : "memory")

// One tile of a tensor whose rows hold at least 32 blocks: the full groups in PTX, a last partial group
// through decode_group.  `valid` is false for a warp whose slot lies past the last tile (`tile` is then
// the last tile, only so that addresses stay inside the stream): it does no group at all.  The number of
// groups is data here, not control flow the compiler reasons about: every branch on it is a bra.uni.
template <int DT>
__device__ __forceinline__ void decode_tile_fast(const JobParams &J, uint32_t tile, bool valid, uint32_t lut_addr,
                                                 uint32_t ring, uint32_t lane) {
    const uint32_t *rec = J.tile_index + size_t(tile) * 33u;
    uint32_t x = rec[lane];
    const uint32_t off = min(rec[32], J.total_words);   // a damaged index must not move reads outside the payload
    const uint32_t end = (tile + 1 < J.n_tiles) ? rec[33 + 32] : rec[33];
    const uint32_t v0 = tile * J.V;
    const uint32_t nv = valid ? min(J.V, J.n_vec - v0) : 0u;
    const uint32_t b = J.b, mask = (1u << b) - 1u, lt = (1u << lane) - 1u;
    const uint32_t per_row = J.per_row;
    const uint64_t pay = reinterpret_cast<uint64_t>(J.stream + J.off_payload);
    const uint64_t first = pay + 2ull * off;
    const uint64_t a0 = first & ~15ull;
    const uint32_t lead = uint32_t(first - a0);
    const uint32_t room = uint32_t(pay + 2ull * J.total_words - a0);     // the payload is shorter than 2 GB
    const uint32_t lane16 = 16u * lane;
    for (uint32_t c = 0; c < 4; ++c) ring_issue(ring, a0, room, c, lane);
    cp_async_wait<1>();
    __syncwarp();
    uint32_t wa = ring + lead;                    // cursor
    uint32_t wbase = ring;                        // wa - position
    uint32_t wthr = ring + 512u;                  // next chunk boundary
    uint64_t srcp = a0 + 2048u + lane16;          // this lane's part of chunk 4
    uint32_t rem = room - (2048u + lane16);       // signed in the asm: may be negative
    uint32_t nextc = 4;
    const uint32_t ring_lane = ring + lane16;
    const uint32_t k0_bits = __float_as_uint(float(4096 - J.zlo));
    const uint32_t v = v0 + lane;
    uint32_t row = v / per_row;
    const float *scales = J.scales;
    uint32_t sig = __float_as_uint(__ldg(scales + row));
    uint32_t doff = v * Out<DT>::kBlockBytes;
    const uint64_t out_base = reinterpret_cast<uint64_t>(J.out);
    // The loop runs on byte offsets into the output: this lane leaves its row when doff reaches chg and the tile's
    // full groups are done when it reaches endo.  The group count is the same in all lanes but comes from loaded
    // data, which the compiler treats as possibly different per lane; the loop therefore branches on warp votes of
    // these comparisons (see the asm), never on the values themselves.  nv >> 5 may be 0: the asm falls through.
    const uint32_t row_bytes = per_row * Out<DT>::kBlockBytes;
    uint32_t chg = (row + 1u) * row_bytes;
    const uint32_t endo = doff + (nv >> 5) * (32u * Out<DT>::kBlockBytes);
    uint32_t lim = min(chg, endo);
    const uint32_t row_max = J.n_vec / per_row - 1u;   // the wrap after a tensor's last block must not read past the scales
    if constexpr (DT == EP_BF16) EP_FULL_GROUPS_ASM(EP_S_STORE_BF16, 512);
    else if constexpr (DT == EP_FP16) EP_FULL_GROUPS_ASM(EP_S_STORE_FP16, 512);
    else if constexpr (DT == EP_FP8_E4M3) EP_FULL_GROUPS_ASM(EP_S_STORE_E4M3, 256);
    else if constexpr (DT == EP_FP32) EP_FULL_GROUPS_ASM(EP_S_STORE_FP32, 1024);
    else if constexpr (DT == EP_FP8_E5M2) EP_FULL_GROUPS_ASM(EP_S_STORE_E5M2, 256);
    else if constexpr (DT == EP_UINT8) EP_FULL_GROUPS_ASM(EP_S_STORE_UINT8, 256);
    else EP_FULL_GROUPS_ASM(EP_S_STORE_INT8, 256);
    uint32_t pos = wa - wbase;
    if (nv & 31u) {
        uint32_t threshold = wthr - wbase;
        // chunks up to (threshold >> 9) + 2 are requested: the same bookkeeping as ring_service expects
        if (__any_sync(0xFFFFFFFFu, pos >= threshold)) ring_service(ring, a0, room, pos, threshold, lane);
        const uint32_t wa0 = ring + (pos & (kRingBytes - 1u));
        uint32_t wt = wa0;
        const bool act = lane < (nv & 31u);
        decode_group<DT, true>(x, wt, lut_addr, mask, b, lt, act, k0_bits, __uint_as_float(sig), J.zlo,
                               static_cast<uint8_t *>(J.out) + doff);
        pos += wt - wa0;
    }
    cp_async_wait<0>();
    __syncwarp();
    const bool bad = valid && ((x != ep::kStateLow) || (off + ((pos - lead) >> 1) != end));
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(&g_ep_status, 1u);
}

// One persistent CTA per SM.  The rounds of all jobs of the launch form one list (job after job); CTA k takes the
// rounds whose cumulative cost at their start lies in [k, k + 1) * ceil(total / gridDim.x) - a contiguous stretch,
// usually inside one job - and rebuilds the lookup tables when the stretch crosses into the next job.  Everything
// that steers this (loop bounds, job changes) depends on blockIdx and kernel parameters only, so the compiler
// sees warp-uniform control flow and puts no divergence guards around the warp votes of the hot loop; in the last
// round of a job a warp past the job's last tile goes through the same code with zero groups to do.
// SINGLE: the launch has one job (the common single-tensor call); its parameters then sit at fixed offsets of
// the parameter block and the job loop disappears.
template <int DT, bool SINGLE>
__global__ void __launch_bounds__(kThreads, 1) ep_decode_smem_kernel(const __grid_constant__ BatchParams P) {
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t lut_addr = uint32_t(__cvta_generic_to_shared(smem));
    const uint32_t ring = lut_addr + kLutBytes + warp * kRingStride;
    bool tables_in_use = false;
    const int n_jobs = SINGLE ? 1 : P.n_jobs;
    for (int j = 0; j < n_jobs; ++j) {
        const JobParams &J = P.job[SINGLE ? 0 : j];
        // rounds r of this job with cost_begin + r * round_cost in [lo, hi), this CTA's share of the total cost
        // (recomputed per job rather than kept in registers across the decode loops)
        const uint32_t lo = P.cost_per_cta * blockIdx.x, hi = lo + P.cost_per_cta;      // below 2^31 (see the launcher)
        const uint32_t a = lo > J.cost_begin ? lo - J.cost_begin : 0u, b = hi > J.cost_begin ? hi - J.cost_begin : 0u;
        const uint32_t r0 = min((a + J.round_cost - 1u) / J.round_cost, J.rounds);
        const uint32_t r1 = min((b + J.round_cost - 1u) / J.round_cost, J.rounds);
        if (r0 >= r1) continue;
        {   // while the tables are built, bring this warp's first tile record and the start of its payload into L2
            const uint32_t t_first = J.tile0 + min(r0 * kWarps + warp, J.tile_cnt - 1u);
            const uint32_t *rec = J.tile_index + size_t(t_first) * 33u;
            if (lane < 2) prefetch_l2(rec + 32u * lane);                     // the record spans two 128-byte lines
            const uint32_t off = min(rec[32], J.total_words);
            const uint64_t at = 2ull * off + 128u * lane;                      // 4 KB: the ring's first fill and more
            if (at < 2ull * J.total_words) prefetch_l2(J.stream + J.off_payload + at);
        }
        if (tables_in_use) __syncthreads();          // every warp is done with the previous job's tables
        build_tables_smem(J, lut_addr, warp, lane);
        __syncthreads();
        tables_in_use = true;
        const bool wide = J.per_row >= 32u;
        for (uint32_t r = r0; r < r1; ++r) {
            const uint32_t base = r * kWarps;
            const bool mine = base + warp < J.tile_cnt;
            const uint32_t tile = J.tile0 + min(base + warp, J.tile_cnt - 1u);
            if constexpr (DT != EP_FIELDS_I32) {
                if (wide && J.V < (1u << 20)) {
                    decode_tile_fast<DT>(J, tile, mine, lut_addr, ring, lane);
                    continue;
                }
            }
            if (mine) {
                if (wide) decode_tile<DT, true>(J, tile, lut_addr, ring, lane);
                else decode_tile<DT, false>(J, tile, lut_addr, ring, lane);
            }
        }
    }
}

// ======================================================================================================
// Large-table path: b >= 12, a coordinate range above 1024, or a single-symbol table at b = 11.  The
// seventeen tables (2^b slots of 4 bytes: symbol index << 16 | u - F) are built into caller-provided
// scratch by one launch and read through L1/L2 by the decode launch that follows on the same stream; a
// symbol's frequency comes from the stream's own frequency arrays (a few KB, resident in L1) and its value
// is the table's minimum plus the index.  Slots are hit uniformly at random, so the traffic between L2 and
// L1 is what bounds this path: four-byte entries halve the table set (278 KB at b = 12, most of it
// L1-resident).  Same tile / lane / word order as above; payload words are read straight from global
// memory with the index clamped to the payload.
// ======================================================================================================

struct GJobParams {
    const uint8_t *stream;
    const uint32_t *tile_index;
    const float *scales;
    void *out;
    uint32_t *lut;                // scratch: 17 << b entries
    uint32_t off_tables;          // byte offset of the table section (directory, then frequencies)
    uint32_t off_payload;
    uint32_t total_words;
    uint32_t n_vec;
    uint32_t per_row;
    uint32_t V, n_tiles, b;
    uint32_t tile0, tile_cnt;     // the tiles this launch decodes
    uint32_t cta_begin, cta_count;
};

struct GBatchParams {
    GJobParams job[EP_MAX_BATCH];
    int32_t n_jobs;
};

constexpr int kGThreads = 256;
constexpr int kGWarps = kGThreads / 32;

// one CTA per (table, job): exclusive prefix sums of the frequencies in shared memory (as u16; the last
// entry 2^b <= 32768 still fits), then every slot finds its symbol by binary search
__global__ void __launch_bounds__(1024) ep_build_tables_kernel(const __grid_constant__ GBatchParams P) {
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ uint32_t part[1024];
    const GJobParams &J = P.job[blockIdx.y];
    const uint32_t t = blockIdx.x, tid = threadIdx.x;
    const uint8_t *dir = J.stream + J.off_tables;
    const uint32_t *Ks = reinterpret_cast<const uint32_t *>(dir) + EP_NUM_TABLES;
    const uint32_t K = Ks[t];
    if (K == 0) return;
    uint32_t before = 0;
    for (uint32_t i = 0; i < t; ++i) before += Ks[i];
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(dir + 8 * EP_NUM_TABLES) + before;
    uint16_t *F = reinterpret_cast<uint16_t *>(smem);              // K + 1 entries
    const uint32_t per = (K + blockDim.x - 1) / blockDim.x;
    const uint32_t j0 = min(tid * per, K), j1 = min(j0 + per, K);
    uint32_t sum = 0;
    for (uint32_t j = j0; j < j1; ++j) sum += fq[j];
    part[tid] = sum;
    __syncthreads();
    if (tid == 0) {
        uint32_t run = 0;
        for (uint32_t i = 0; i < blockDim.x; ++i) { const uint32_t v = part[i]; part[i] = run; run += v; }
        F[K] = uint16_t(run);                                        // = 2^b for a valid stream
    }
    __syncthreads();
    uint32_t run = part[tid];
    for (uint32_t j = j0; j < j1; ++j) { F[j] = uint16_t(run); run += fq[j]; }
    __syncthreads();
    const uint32_t M = 1u << J.b;
    uint32_t *lut = J.lut + (size_t(t) << J.b);
    for (uint32_t u = tid; u < M; u += blockDim.x) {
        uint32_t lo = 0, hi = K;                                     // largest j with F[j] <= u; F[K] = 2^b > u
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (uint32_t(F[mid]) <= u) lo = mid; else hi = mid;
        }
        lut[u] = (lo << 16) | (u - uint32_t(F[lo]));                 // K <= 65535 and u - F < 2^15
    }
}

// one symbol: returns its index inside table t's symbol range (0 for an idle lane)
__device__ __forceinline__ uint32_t grans_step(uint32_t &x, const uint32_t *table, const uint16_t *freq, uint32_t mask,
                                               uint32_t b, uint32_t &ptr, const uint16_t *pay, uint32_t lt, bool act,
                                               uint32_t last_word) {
    uint32_t sym = 0;
    bool need = false;
    if (act) {
        const uint32_t e = __ldg(table + (x & mask));
        sym = e >> 16;
        x = uint32_t(__ldg(freq + sym)) * (x >> b) + (e & 0xFFFFu);
        need = x < ep::kStateLow;
    }
    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, need);
    if (need) x = (x << 16) | __ldg(pay + min(ptr + __popc(bal & lt), last_word));
    ptr += __popc(bal);
    return sym;
}

template <int DT>
__global__ void __launch_bounds__(kGThreads) ep_decode_glut_kernel(const __grid_constant__ GBatchParams P) {
    __shared__ uint32_t s_foff[EP_NUM_TABLES];     // start of table t's frequencies, in u16 units
    __shared__ int32_t s_tmin[EP_NUM_TABLES];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    int j = 0;
    while (j + 1 < P.n_jobs && blockIdx.x >= P.job[j + 1].cta_begin) ++j;
    const GJobParams &J = P.job[j];
    const uint8_t *dir = J.stream + J.off_tables;
    if (threadIdx.x == 0) {
        const uint32_t *Ks = reinterpret_cast<const uint32_t *>(dir) + EP_NUM_TABLES;
        uint32_t acc = 0;
        for (int t = 0; t < EP_NUM_TABLES; ++t) {
            s_foff[t] = acc;
            s_tmin[t] = reinterpret_cast<const int32_t *>(dir)[t];
            acc += Ks[t];
        }
    }
    __syncthreads();
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(dir + 8 * EP_NUM_TABLES);
    const uint32_t b = J.b, mask = (1u << b) - 1u, lt = (1u << lane) - 1u;
    const uint16_t *pay = reinterpret_cast<const uint16_t *>(J.stream + J.off_payload);
    const uint32_t last_word = J.total_words ? J.total_words - 1u : 0u;
    const uint32_t cta = blockIdx.x - J.cta_begin;
    const uint32_t foff0 = s_foff[0];
    for (uint32_t local = cta * kGWarps + warp; local < J.tile_cnt; local += J.cta_count * kGWarps) {
        const uint32_t tile = J.tile0 + local;
        const uint32_t *rec = J.tile_index + size_t(tile) * 33u;
        uint32_t x = rec[lane];
        uint32_t ptr = rec[32];
        const uint32_t end = (tile + 1 < J.n_tiles) ? rec[33 + 32] : rec[33];
        const uint32_t v0 = tile * J.V;
        const uint32_t nv = min(J.V, J.n_vec - v0);
        for (uint32_t g = 0; g * 32u < nv; ++g) {
            const uint32_t i = g * 32u + lane;
            const bool act = i < nv;
            int32_t fld[9];
            fld[0] = int32_t(grans_step(x, J.lut, fq + foff0, mask, b, ptr, pay, lt, act, last_word)) + s_tmin[0];
            const uint32_t t0 = 1u + 8u * uint32_t(fld[0] & 1);          // first coordinate table of this coset
#pragma unroll
            for (uint32_t k = 0; k < 8; ++k)
                fld[k + 1] = int32_t(grans_step(x, J.lut + (size_t(t0 + k) << b), fq + s_foff[t0 + k], mask, b, ptr, pay, lt,
                                                act, last_word)) + s_tmin[t0 + k];
            if (!act) continue;
            const uint32_t v = v0 + i;
            if constexpr (DT == EP_FIELDS_I32) {
                int32_t *o = static_cast<int32_t *>(J.out) + size_t(v) * 9u;
#pragma unroll
                for (int k = 0; k < 9; ++k) o[k] = fld[k];
            } else {
                // Eq. 5 on doubled coordinates q = 2p (integers), then p = q/2 exactly and Eq. 19
                const float sigma = __ldg(J.scales + v / J.per_row);
                int32_t s7 = 0;
                float w[8];
#pragma unroll
                for (int k = 1; k <= 7; ++k) {
                    s7 += fld[k];
                    w[k - 1] = __fmul_rn(sigma, float(2 * fld[k] + fld[0]) * 0.5f);
                }
                w[7] = __fmul_rn(sigma, float(2 * (2 * fld[8] + (s7 & 1)) + fld[0]) * 0.5f);
                Out<DT>::store(static_cast<uint8_t *>(J.out) + size_t(v) * Out<DT>::kBlockBytes, w);
            }
        }
        const bool bad = (x != ep::kStateLow) || (ptr != end);
        if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(&g_ep_status, 1u);
    }
}

// ---- host side -----------------------------------------------------------------------------------

// the tiles a job asks for: its range, or the whole tensor when both range fields are 0
inline uint32_t job_tile0(const ep_decode_job &jb) { return jb.tile_count ? jb.tile_begin : 0u; }
inline uint32_t job_tiles(const ep_decode_job &jb) { return jb.tile_count ? jb.tile_count : jb.info->n_tiles; }

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
    if (r.any && r.hi - zlo > 1023) return false;     // 10-bit code field
    if (zlo < -1024) return false;                    // 4096 - zlo - c/2 stays below 8192: same fp32 exponent as 4096 + code
    for (int t = 0; t < EP_NUM_TABLES; ++t) {
        if (I.table_K[t] > kLutEntries) return false;
        if (I.b == 11 && I.table_K[t] == 1) return false;   // a lone symbol has f = 2^11: one bit more than the f field
    }
    return true;
}

template <int DT>
cudaError_t launch_smem(const BatchParams &P, uint32_t grid, cudaStream_t st) {
    static bool configured[64] = {};   // the attribute is per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(ep_decode_smem_kernel<DT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemBytes));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(ep_decode_smem_kernel<DT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemBytes));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    if (P.n_jobs == 1) ep_decode_smem_kernel<DT, true><<<grid, kThreads, kSmemBytes, st>>>(P);
    else ep_decode_smem_kernel<DT, false><<<grid, kThreads, kSmemBytes, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

extern "C" size_t ep_decode_scratch_bytes(const ep_info *info) {
    if (!info) return 0;
    if (fits_smem_tables(*info)) return 0;
    return size_t(EP_NUM_TABLES) * (size_t(1) << info->b) * 4u;
}

namespace {

template <int DT>
cudaError_t launch_glut(const GBatchParams &P, uint32_t grid, cudaStream_t st) {
    ep_decode_glut_kernel<DT><<<grid, kGThreads, 0, st>>>(P);
    return cudaGetLastError();
}

// jobs whose tables do not fit shared memory: build the tables into scratch, then decode from them
int decode_large_tables(const ep_decode_job *const *jobs, int n_jobs, int32_t dt, int sms, cudaStream_t st) {
    GBatchParams P;
    std::memset(&P, 0, sizeof(P));
    P.n_jobs = n_jobs;
    uint32_t next = 0, max_K = 1;
    for (int i = 0; i < n_jobs; ++i) {
        const ep_decode_job &jb = *jobs[i];
        const ep_info &I = *jb.info;
        const size_t need = size_t(EP_NUM_TABLES) * (size_t(1) << I.b) * 4u;
        if (!jb.d_scratch || jb.scratch_bytes < need || (reinterpret_cast<uintptr_t>(jb.d_scratch) & 255)) return EP_ERR_SCRATCH;
        for (int t = 0; t < EP_NUM_TABLES; ++t) {
            if (I.table_K[t] > 65535u) return EP_ERR_UNSUPPORTED;
            if (I.table_K[t] > max_K) max_K = I.table_K[t];
        }
        GJobParams &J = P.job[i];
        J.stream = static_cast<const uint8_t *>(jb.d_stream);
        J.tile_index = static_cast<const uint32_t *>(jb.d_tile_index);
        J.scales = jb.d_row_scales;
        J.out = jb.d_out;
        J.lut = static_cast<uint32_t *>(jb.d_scratch);
        J.off_tables = I.off_tables;
        J.off_payload = I.off_payload;
        J.total_words = uint32_t(I.total_words);
        J.n_vec = uint32_t(uint64_t(I.R) * (I.C / 8));
        J.per_row = I.C / 8;
        J.V = I.V;
        J.n_tiles = I.n_tiles;
        J.b = I.b;
        J.tile0 = job_tile0(jb);
        J.tile_cnt = job_tiles(jb);
        const uint64_t want = (uint64_t(J.tile_cnt) + kGWarps - 1) / kGWarps;
        const uint64_t cap = uint64_t(sms) * 8u;
        J.cta_begin = next;
        J.cta_count = uint32_t(want < cap ? want : cap);
        next += J.cta_count;
    }
    const size_t smem = 2u * (size_t(max_K) + 1u);
    if (smem > 48u * 1024u) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return EP_ERR_CUDA;
        if (cudaFuncSetAttribute(ep_build_tables_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
            return EP_ERR_CUDA;
    }
    ep_build_tables_kernel<<<dim3(EP_NUM_TABLES, n_jobs), 1024, smem, st>>>(P);
    if (cudaGetLastError() != cudaSuccess) return EP_ERR_CUDA;
    cudaError_t e;
    switch (dt) {
    case EP_BF16: e = launch_glut<EP_BF16>(P, next, st); break;
    case EP_FP16: e = launch_glut<EP_FP16>(P, next, st); break;
    case EP_FP8_E4M3: e = launch_glut<EP_FP8_E4M3>(P, next, st); break;
    case EP_INT8: e = launch_glut<EP_INT8>(P, next, st); break;
    case EP_FP32: e = launch_glut<EP_FP32>(P, next, st); break;
    case EP_FP8_E5M2: e = launch_glut<EP_FP8_E5M2>(P, next, st); break;
    case EP_UINT8: e = launch_glut<EP_UINT8>(P, next, st); break;
    case EP_FIELDS_I32: e = launch_glut<EP_FIELDS_I32>(P, next, st); break;
    default: return EP_ERR_BAD_ARG;
    }
    return e == cudaSuccess ? EP_OK : EP_ERR_CUDA;
}

}  // namespace

extern "C" int ep_decode_batch(const ep_decode_job *jobs_in, int32_t n_in, void *stream) {
    if (!jobs_in || n_in <= 0 || n_in > EP_MAX_BATCH) return EP_ERR_BAD_ARG;
    const int sms = num_sms();
    if (sms <= 0) return EP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int32_t dt = jobs_in[0].out_dtype;
    if (dt != EP_BF16 && dt != EP_FP16 && dt != EP_FP8_E4M3 && dt != EP_INT8 && dt != EP_FP32 && dt != EP_FP8_E5M2 &&
        dt != EP_UINT8 && dt != EP_FIELDS_I32)
        return EP_ERR_BAD_ARG;
    const ep_decode_job *fast[EP_MAX_BATCH], *large[EP_MAX_BATCH];
    int n_jobs = 0, n_large = 0;
    for (int i = 0; i < n_in; ++i) {
        const ep_decode_job &jb = jobs_in[i];
        if (!jb.info || !jb.d_stream || !jb.d_tile_index || !jb.d_out) return EP_ERR_BAD_ARG;
        if (jb.out_dtype != dt) return EP_ERR_BAD_ARG;   // one output type per launch
        if (dt != EP_FIELDS_I32 && !jb.d_row_scales) return EP_ERR_BAD_ARG;
        const ep_info &I = *jb.info;
        if (I.C == 0 || I.C % 8 || I.R == 0 || I.V == 0 || I.b < 9 || I.b > 15 || I.J != ep::kStates) return EP_ERR_BAD_ARG;
        // one vector store per block: 16 bytes for the two-byte types (two of them for FP32), 8 for the one-byte types
        const uintptr_t out_mask = dt == EP_FIELDS_I32 ? 3u : (dt == EP_FP8_E4M3 || dt == EP_FP8_E5M2 || dt == EP_INT8 || dt == EP_UINT8) ? 7u : 15u;
        if ((reinterpret_cast<uintptr_t>(jb.d_stream) & 3) || (reinterpret_cast<uintptr_t>(jb.d_tile_index) & 3) ||
            (reinterpret_cast<uintptr_t>(jb.d_out) & out_mask))
            return EP_ERR_BAD_ARG;
        if (I.table_K[0] == 0 || I.table_min[0] < 0 || int64_t(I.table_min[0]) + I.table_K[0] > 2) return EP_ERR_BAD_STREAM;
        // 32-bit byte offsets into the output (one row and one group beyond the end still representable) and a
        // signed 32-bit payload remainder in the kernels
        if ((uint64_t(I.R) + 1u) * I.C * 4u + 1024u >= (1ull << 32) || I.total_words >= (1ull << 30)) return EP_ERR_UNSUPPORTED;
        if (jb.tile_count != 0 || jb.tile_begin != 0) {     // a tile range: inside the tensor and not empty
            if (jb.tile_count == 0 || jb.tile_begin >= I.n_tiles || jb.tile_count > I.n_tiles - jb.tile_begin) return EP_ERR_BAD_ARG;
        }
        if (fits_smem_tables(I)) { fast[n_jobs++] = &jb; }
        else large[n_large++] = &jb;
    }
    if (n_large) {
        const int rc = decode_large_tables(large, n_large, dt, sms, st);
        if (rc) return rc;
    }
    if (n_jobs == 0) return EP_OK;
    BatchParams P;
    std::memset(&P, 0, sizeof(P));
    P.n_jobs = n_jobs;
    // persistent CTAs, one per SM (fewer if the launch has fewer rounds than SMs); the kernel splits the
    // cost-weighted list of all rounds evenly over them
    uint64_t rounds_total = 0, cost = 0;
    for (int i = 0; i < n_jobs; ++i) {
        const ep_decode_job &jb = *fast[i];
        const ep_info &I = *jb.info;
        JobParams &J = P.job[i];
        const uint32_t my_tiles = job_tiles(jb);
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
        J.tile0 = job_tile0(jb);
        J.tile_cnt = my_tiles;
        J.b = I.b;
        J.zlo = int32_t(even_base(coord_range(I)));
        J.rounds = (my_tiles + uint32_t(kWarps) - 1u) / uint32_t(kWarps);
        J.round_cost = (I.V + 31u) / 32u;
        J.cost_begin = uint32_t(cost);
        cost += uint64_t(J.rounds) * J.round_cost;
        rounds_total += J.rounds;
        uint32_t acc = 0;
        for (int t = 0; t < EP_NUM_TABLES; ++t) {
            J.tmin[t] = int16_t(I.table_min[t]);
            J.tK[t] = uint16_t(I.table_K[t]);
            J.foff[t] = uint16_t(acc);
            acc += I.table_K[t];
        }
    }
    const uint32_t next = uint32_t(rounds_total < uint64_t(sms) ? rounds_total : uint64_t(sms));   // grid size
    // a tensor has under 2^27 blocks, so sixteen of them cost under 2^26 groups: 32-bit arithmetic in the kernel
    if (cost + next >= (1ull << 31)) return EP_ERR_UNSUPPORTED;
    P.cost_per_cta = uint32_t((cost + next - 1u) / next);
    cudaError_t e;
    switch (dt) {
    case EP_BF16: e = launch_smem<EP_BF16>(P, next, st); break;
    case EP_FP16: e = launch_smem<EP_FP16>(P, next, st); break;
    case EP_FP8_E4M3: e = launch_smem<EP_FP8_E4M3>(P, next, st); break;
    case EP_INT8: e = launch_smem<EP_INT8>(P, next, st); break;
    case EP_FP32: e = launch_smem<EP_FP32>(P, next, st); break;
    case EP_FP8_E5M2: e = launch_smem<EP_FP8_E5M2>(P, next, st); break;
    case EP_UINT8: e = launch_smem<EP_UINT8>(P, next, st); break;
    case EP_FIELDS_I32: e = launch_smem<EP_FIELDS_I32>(P, next, st); break;
    default: return EP_ERR_BAD_ARG;
    }
    return e == cudaSuccess ? EP_OK : EP_ERR_CUDA;
}

extern "C" int ep_decode_tiles(const ep_info *info, const void *d_stream, const void *d_tile_index,
                               const float *d_row_scales, int32_t out_dtype, void *d_out, void *d_scratch,
                               size_t scratch_bytes, uint32_t tile_begin, uint32_t tile_count, void *stream) {
    if (tile_count == 0) return EP_ERR_BAD_ARG;
    ep_decode_job jb;
    jb.info = info;
    jb.d_stream = d_stream;
    jb.d_tile_index = d_tile_index;
    jb.d_row_scales = d_row_scales;
    jb.out_dtype = out_dtype;
    jb.d_out = d_out;
    jb.d_scratch = d_scratch;
    jb.scratch_bytes = scratch_bytes;
    jb.tile_begin = tile_begin;
    jb.tile_count = tile_count;
    return ep_decode_batch(&jb, 1, stream);
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
    jb.tile_begin = 0;
    jb.tile_count = 0;
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

// ---- decode without a caller-provided scratch buffer ----------------------------------------------------
// For callers that cannot allocate device memory when they need to decode (they were given input and
// output buffers by a framework that owns the allocator, or an allocation would stall the device in the
// middle of serving).  The large-table path then builds its tables in this fixed area instead of in
// caller scratch.  One area per device, shared by every call: calls that overlap on the GPU race on it.
namespace {

constexpr size_t kStaticTableBytes = size_t(EP_NUM_TABLES) * (size_t(1) << EP_STATIC_MAX_B) * 4u;   // 557 056
static __device__ __align__(256) unsigned char g_ep_static_tables[kStaticTableBytes];

// In host code `g_ep_static_tables` is only a handle for the runtime, not an address a kernel could use:
// the device address is asked for once per device, with that device current.
void *g_static_tables_addr[64] = {};

int static_tables_address(void **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EP_ERR_CUDA;
    if (dev < 0 || dev >= 64) return EP_ERR_UNSUPPORTED;
    if (!g_static_tables_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_ep_static_tables) != cudaSuccess || !p) return EP_ERR_CUDA;
        g_static_tables_addr[dev] = p;
    }
    *out = g_static_tables_addr[dev];
    return EP_OK;
}

}  // namespace

extern "C" int ep_decode_tensor_static(const ep_info *info, const void *d_stream, const void *d_tile_index,
                                       const float *d_row_scales, int32_t out_dtype, void *d_out, void *stream) {
    if (!info) return EP_ERR_BAD_ARG;
    void *tables = nullptr;
    size_t bytes = 0;
    if (ep_decode_scratch_bytes(info) != 0) {
        if (info->b > EP_STATIC_MAX_B) return EP_ERR_STATIC_LIMIT;   // tables of 2^b slots would not fit the built-in area
        const int rc = static_tables_address(&tables);
        if (rc) return rc;
        bytes = kStaticTableBytes;
    }
    return ep_decode_tensor(info, d_stream, d_tile_index, d_row_scales, out_dtype, d_out, tables, bytes, stream);
}
