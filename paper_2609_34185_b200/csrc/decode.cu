// Fused EntroPack decode for sm_100a (paper Sec. 3.7): tiled 32-state rANS symbol decode (Eq. 18),
// arithmetic inverse of the field representation (Eq. 5), multiplication by the fp32 row scale and
// rounding to the output type (Eq. 19), written straight to the weight tensor.  No symbol tensor,
// no codebook, no tensor cores (the path is not a contraction).
//
// Mapping: one warp per tile, one rANS state per lane (the paper's layout).  A CTA of 32 warps builds (or
// copies) the sixteen slot -> (frequency, offset, value) lookup tables of the coordinate fields once in
// shared memory and then streams tiles through them.  A lookup entry is one word
//     [31:21] f      [20:11] code     [10:0] u - F
// where `code` is the symbol's coordinate relative to an even base zlo (z - zlo; 2m - zlo for the m
// field).  f < 2^11 always: a coordinate table with a single symbol at b = 11 (f = 2^11) goes to the
// large-table path.  (entry & 0x1FF800) | 0x45800000 is the fp32 number 4096 + code (| 0x400 adds the
// half of coset 1), so one subtraction of 4096 - zlo yields the lattice coordinate p exactly, and one fp32
// multiply by the row scale gives the product of Eq. 19 with the same operands and rounding as the
// definition.  The coset symbol has two values only: it is decoded by comparing the slot with the
// frequency of coset 0, without a table.
//
// Payload words reach the lanes through a per-tile ring in shared memory, filled 512 bytes at a time by
// cp.async (16 bytes per lane, source clamped to the end of the payload) ahead of the read cursor; the
// first 512 bytes of the ring are mirrored behind its end so that the nine steps of a group never have
// to wrap an address.  (With b <= 11 a lane takes at most seven words in nine steps: a step shortens the
// state by at most eleven bits, a word adds sixteen.)
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "stream.hpp"

namespace {

// Tiles a warp decodes side by side (1 to 4) and warps per CTA.  The loop below is written for any number of
// chains per warp, their instructions interleaved line by line; measured on B200 (8192 x 8192 at 4 bpp to FP16 /
// the 372 M-parameter layer at 3.5 bpp to BF16, Gparams/s): 32 warps x 1 chain 985 / 1171, 24 x 2 940 / 1104,
// 16 x 3 781 / 889, 12 x 4 677 / 744.  The loop is bound by the issue slots, the ALU pipe and the shared-memory
// pipe together (each about 70 % busy), not by the latency of one chain: what counts is the number of warps.
#ifndef EP_CHAINS
#define EP_CHAINS 1
#endif
#ifndef EP_WARPS
#define EP_WARPS (EP_CHAINS == 1 ? 32 : 48 / EP_CHAINS)
#endif
constexpr uint32_t kChains = EP_CHAINS;
constexpr int kWarps = EP_WARPS;                             // warps per CTA (one CTA per SM)
constexpr int kThreads = kWarps * 32;
constexpr uint32_t kTilesPerRound = kWarps * kChains;        // 48 tiles per CTA at a time
static_assert(kTilesPerRound == ep::kDecodeTilesPerCta, "tile-size suggestions assume this many tiles per CTA");
constexpr uint32_t kLutEntries = 2048;                       // 2^11 slots per table
constexpr uint32_t kLutStride = kLutEntries * 4;             // bytes per table in shared memory
constexpr uint32_t kCosetStride = 8 * kLutStride;            // the eight tables of coset 1 follow those of coset 0
constexpr uint32_t kLutBytes = 16 * kLutStride;              // 131072
// Payload ring of a chain: three chunks of 512 bytes (one cp.async round of a warp, 16 bytes per lane) plus a mirror
// of its first 512 bytes.  (Measured and dropped: 64 rings of four 256-byte chunks for two tiles per warp at 32 warps.)
constexpr uint32_t kChunk = 512, kRingSlots = 3;
constexpr uint32_t kRingBytes = kRingSlots * kChunk;         // 1536
constexpr uint32_t kRingMirror = 512;                        // >= 7 words * 32 lanes * 2 bytes + one lane span (62)
constexpr uint32_t kRingStride = kRingBytes + kRingMirror;   // 2048 per chain
constexpr uint32_t kCtxBytes = 32 + 32 * kChains;            // per warp: what the rare paths of the hot loop need
constexpr uint32_t kRingBase = kLutBytes;
constexpr uint32_t kCtxBase = kRingBase + kWarps * kChains * kRingStride;
// 2^12-slot streams: per table, the entries of the kHotSpan coordinate values around zero are kept in shared memory
// (the rest is read from global memory); this fills what the tables, rings and context blocks of the 32-warp build
// leave of the 227 KB
constexpr uint32_t kHotSpan = 528;                           // coordinate codes per table in the hot window
constexpr uint32_t kHotBytes = 16 * kHotSpan * 4;            // 33792
constexpr uint32_t kColdCodes = 4096;                        // codes per table in the complete entry array (global memory)
constexpr uint32_t kColdBytes = 16 * kColdCodes * 4;         // 262144
constexpr uint32_t kHotBase = kCtxBase + kWarps * kCtxBytes;
constexpr bool kTwoLevelInLoop = EP_CHAINS == 1 && kHotBase + kHotBytes <= 232448;
constexpr uint32_t kSmemBytes = kHotBase + (kTwoLevelInLoop ? kHotBytes : 0);   // 232448 in the default build
static_assert(kSmemBytes <= 232448, "more shared memory than an sm_100 CTA can have");
constexpr uint32_t kCodeMask = 0x001FF800u;                  // 10-bit code field
constexpr uint32_t kExp4096 = 0x45800000u;                   // fp32 bit pattern of 4096.0
constexpr uint32_t kOwnSlots = 16;                           // table build: slots of a symbol that its own lane writes
constexpr uint32_t kEntryUnused = 1u << 21;                  // f = 1: what a slot no symbol owns holds (damaged tables)

// per-warp context block (byte offsets); chain c has its part at kCtxChain + c * kCtxChainStride
constexpr uint32_t kCtxScales = 0;         // u64 row scales
constexpr uint32_t kCtxRowBytes = 8;       // u32 output bytes per row
constexpr uint32_t kCtxRowMax = 12;        // u32 last row index
constexpr uint32_t kCtxMul21 = 16;         // u32 2^21 and
constexpr uint32_t kCtxMul11 = 20;         // u32 2^11: multipliers the hot loop must not see as constants (see EP_STEP)
constexpr uint32_t kCtxRowRcp = 24;        // u32 ceil(2^32 / bytes per row)
constexpr uint32_t kCtxChain = 32, kCtxChainStride = 32;
constexpr uint32_t kCcSrc = 0;             // u64 global address of lane 0's 16 bytes of the next chunk to request
constexpr uint32_t kCcRem = 8;             // s32 payload bytes from there to the end of the payload (may be <= 0)
constexpr uint32_t kCcDst = 12;            // u32 ring address of lane 0's 16 bytes of that chunk's slot
constexpr uint32_t kCcRing = 16;           // u32 ring base (shared-memory address)
constexpr uint32_t kCcWbase = 20;          // u32 ring address of byte position 0 (cursor address minus position)
constexpr uint32_t kCcEndo = 24;           // u32 output byte offset after the tile's last block

__device__ unsigned int g_ep_status = 0;

struct JobParams {
    const uint8_t *stream;        // blob base (device)
    const uint32_t *tile_index;   // n_tiles records of 33 words + 1 final word
    const float *scales;
    void *out;
    const uint32_t *lut_image;    // 128 KB table image from ep_prepare_tables / the table-build launch, or null: build the
                                  // tables here (b <= 11 only)
    const uint32_t *cold;         // b = 12: entries of all codes of the sixteen coordinate tables, and
    uint32_t hs2;                 //         twice the first code of the hot window
    uint32_t off_freq;            // byte offset of the u16 frequency arrays inside the blob
    uint32_t off_payload;
    uint32_t total_words;
    uint32_t n_vec;
    uint32_t per_row;             // C / 8
    uint32_t V, n_tiles, b;       // n_tiles: tiles of the whole tensor
    uint32_t tile0, tile_cnt;     // the tiles this launch decodes: [tile0, tile0 + tile_cnt)
    int32_t zlo;                  // even, <= -2
    uint32_t rounds;              // ceil(tile_cnt / 48): in one round the warps of a CTA take 48 consecutive tiles
    uint32_t round_cost;          // work of one round in groups of 32 vectors (ceil(V / 32))
    uint32_t cost_begin;          // sum of rounds * round_cost over the jobs before this one
    uint32_t row_bytes;           // output bytes per row
    uint32_t row_rcp;             // ceil(2^32 / row_bytes)
    uint32_t row_max;             // index of the last row
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
__device__ __forceinline__ void sts64(uint32_t addr, uint64_t v) {
    asm volatile("st.shared.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
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
// Warp t - 1 fills coordinate table t (t = 1..16; the coset table t = 0 needs none).  Symbols are taken 32 at
// a time: a warp scan gives each lane its symbol's first slot, every lane writes the first sixteen slots of
// its own symbol, and the few symbols with more slots than that are then filled by the whole warp, one
// after the other (that loop is serial: its length, not the number of stores, is what the build time
// depends on).  `base` receives the 2048 entries: a shared-memory address here, see ep_prepare_tables_kernel
// for the same routine writing a table image to global memory.
template <class Store>
__device__ __forceinline__ void build_one_table(const JobParams &J, uint32_t t, uint32_t lane, Store put) {
    const uint32_t K = J.tK[t];
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(J.stream + J.off_freq) + J.foff[t];
    const int32_t tmin = J.tmin[t];
    const bool is_m = ((t - 1) & 7) == 7;
    const uint32_t slots = min(1u << J.b, kLutEntries);
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
        const uint32_t code = uint32_t((is_m ? 2 * v : v) - J.zlo);
        // (a frequency of 2^11 or more is not a stream the launcher sends here: it does not fit its field; whatever the
        // device copy holds, an entry's frequency stays in 1 .. 2047, which the word bound of the ring relies on)
        const uint32_t entry = (min(f, kLutEntries - 1u) << 21) | ((code & 0x3FFu) << 11);
        if (f >= kLutEntries) atomicOr(&g_ep_status, 1u);
#pragma unroll
        for (uint32_t u = 0; u < kOwnSlots; ++u)
            if (u < f && first + u < slots) put(first + u, entry | u);
        uint32_t big = __ballot_sync(0xFFFFFFFFu, f > kOwnSlots);
        while (big) {
            const int i = __ffs(big) - 1;
            big &= big - 1;
            const uint32_t fi = __shfl_sync(0xFFFFFFFFu, f, i);
            const uint32_t Fi = __shfl_sync(0xFFFFFFFFu, first, i);
            const uint32_t ei = __shfl_sync(0xFFFFFFFFu, entry, i);
            for (uint32_t u = kOwnSlots + lane; u < fi && Fi + u < slots; u += 32) put(Fi + u, ei | u);
        }
        run += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    // frequencies of a damaged stream may sum to less than 2^b, and a table may be empty: a slot that no symbol
    // owns gets f = 1, never what an earlier job left there (the word bound of the ring relies on f >= 1)
    for (uint32_t u = min(run, slots) + lane; u < slots; u += 32) put(u, kEntryUnused);
}

__device__ __forceinline__ void build_tables_smem(const JobParams &J, uint32_t lut_addr, uint32_t warp, uint32_t lane) {
    for (uint32_t t = 1 + warp; t < EP_NUM_TABLES; t += kWarps) {
        const uint32_t base = lut_addr + (t - 1) * kLutStride;
        build_one_table(J, t, lane, [base](uint32_t slot, uint32_t e) { sts32(base + 4u * slot, e); });
    }
}

// the prepared image of the same sixteen tables: 128 KB copied by all threads of the CTA, 16 bytes each.  The
// copy is only started here; whoever reads the tables first waits for it (cp.async.wait_group, then a CTA barrier).
__device__ __forceinline__ void copy_tables_smem(const uint32_t *image, uint32_t lut_addr, bool two_level) {
    const uint64_t src = reinterpret_cast<uint64_t>(image);
    for (uint32_t o = 16u * threadIdx.x; o < kLutBytes; o += 16u * kThreads) cp_async16(lut_addr + o, src + o, 16);
    if (kTwoLevelInLoop && two_level)        // the hot part of the second level follows the image
        for (uint32_t o = 16u * threadIdx.x; o < kHotBytes; o += 16u * kThreads)
            cp_async16(lut_addr + kHotBase + o, src + kLutBytes + o, 16);
    cp_async_commit();
}

// frequencies of the two cosets as the decode uses them: u < f0 means coset 0.  A coset that never occurs
// has frequency 0 in the stream and is never selected; it is raised to 1 here only so that a damaged stream
// cannot produce a state that takes a word in every step.
struct CosetFreq { uint32_t f0, f1; };
__device__ __forceinline__ CosetFreq load_coset(const JobParams &J) {
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(J.stream + J.off_freq) + J.foff[0];
    uint32_t f0 = 0, f1 = 0;
    if (J.tmin[0] == 0) {
        f0 = __ldg(fq);
        if (J.tK[0] > 1) f1 = __ldg(fq + 1);
    } else {
        f1 = __ldg(fq);
    }
    const uint32_t M = 1u << J.b;
    CosetFreq c;
    c.f0 = min(f0, M);                 // u < f0 <=> coset 0 (f0 = 0: never)
    c.f1 = max(min(f1, M), 1u);
    return c;
}

// ---- one rANS symbol (Eq. 18) followed by renormalisation: plain version --------------------------
// x: this lane's state; wa: shared-memory byte address of the tile's word cursor (same in all lanes).
// Lanes that need a word take them in lane order: lane l reads the word popc(ballot & lanes below l)
// places after the cursor; the cursor then advances by popc(ballot) words.  Lanes without a vector
// (`act` false: the last, partly filled group of a tile) leave their state alone and take no word.
__device__ __forceinline__ void renorm_plain(uint32_t &x, uint32_t &wa, uint32_t lt, bool need) {
    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, need);
    if (need) {
        uint16_t w;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(w) : "r"(wa + 2u * __popc(bal & lt)));
        x = (x << 16) | w;
    }
    wa += 2u * __popc(bal);
}
__device__ __forceinline__ uint32_t rans_step_plain(uint32_t &x, uint32_t table_addr, uint32_t mask, uint32_t b, uint32_t &wa,
                                                    uint32_t lt, bool act) {
    uint32_t e = 0;
    bool need = false;
    if (act) {
        e = lds32(table_addr + ((x & mask) << 2));
        x = (e >> 21) * (x >> b) + (e & 0x7FFu);
        need = x < ep::kStateLow;
    }
    renorm_plain(x, wa, lt, need);
    return e;
}
// the coset symbol: 0 if the slot lies below f0, else 1
__device__ __forceinline__ uint32_t coset_step_plain(uint32_t &x, CosetFreq cf, uint32_t mask, uint32_t b, uint32_t &wa,
                                                     uint32_t lt, bool act) {
    uint32_t c = 0;
    bool need = false;
    if (act) {
        const uint32_t u = x & mask;
        c = u < cf.f0 ? 0u : 1u;
        x = (c ? cf.f1 : max(cf.f0, 1u)) * (x >> b) + (c ? u - cf.f0 : u);
        need = x < ep::kStateLow;
    }
    renorm_plain(x, wa, lt, need);
    return c;
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

// ---- one group of 32 vectors, plain version: nine symbols per lane, then Eq. 5 / Eq. 19 and the store ---
template <int DT>
__device__ __forceinline__ void decode_group_plain(uint32_t &x, uint32_t &wa, uint32_t lut_addr, CosetFreq cf, uint32_t mask,
                                                   uint32_t b, uint32_t lt, bool act, uint32_t k0_bits, float sigma,
                                                   int32_t zlo, void *dst) {
    uint32_t e[9];
    const uint32_t c = coset_step_plain(x, cf, mask, b, wa, lt, act);
    const uint32_t tab = lut_addr + c * kCosetStride;
#pragma unroll
    for (int k = 1; k <= 8; ++k) e[k] = rans_step_plain(x, tab + uint32_t(k - 1) * kLutStride, mask, b, wa, lt, act);
    if (!act) return;
    // parity of z1 + ... + z7 = xor of the codes' lowest bits (zlo is even); it is the lowest bit of z8
    const uint32_t par = (e[1] ^ e[2] ^ e[3] ^ e[4] ^ e[5] ^ e[6] ^ e[7]) & 0x800u;
    if constexpr (DT == EP_FIELDS_I32) {
        int32_t *f = reinterpret_cast<int32_t *>(dst);
        f[0] = int32_t(c);
#pragma unroll
        for (int k = 1; k <= 7; ++k) f[k] = int32_t((e[k] & kCodeMask) >> 11) + zlo;
        f[8] = (int32_t((e[8] & kCodeMask) >> 11) + zlo) >> 1;
    } else {
        // (entry & mask) | 0x45800000 | c << 10 is 4096 + code + c/2 as fp32 (one ulp here is 2^-11); subtracting
        // 4096 - zlo gives p = z + c/2 exactly
        const uint32_t cc = kExp4096 | (c << 10);
        const uint64_t kk = pack64(k0_bits, k0_bits);
        const uint64_t ss = pack64(__float_as_uint(sigma), __float_as_uint(sigma));
        uint32_t xb[8];
#pragma unroll
        for (int k = 1; k <= 7; ++k) xb[k - 1] = (e[k] & kCodeMask) | cc;
        xb[7] = (e[8] & kCodeMask) | par | cc;
        float w[8];
#pragma unroll
        for (int i = 0; i < 8; i += 2) unpack64(mul2(sub2(pack64(xb[i], xb[i + 1]), kk), ss), w[i], w[i + 1]);
        Out<DT>::store(dst, w);
    }
}

// ---- the same group with the hot loop's word addressing, for full groups of 2^11-slot streams -------------
// Every lane keeps its own word address: the words taken in the previous step by this lane and the lanes above it
// plus those taken in this step by the lanes below are one population count of a bit-select of the two ballots.
// Used where the loop around the group is C++ (the kernel that feeds the tensor cores); BF16 block returned in `blk`.
// renormalisation: lanes whose state fell below 2^15 take a word each, in lane order (the hot loop's seven instructions)
__device__ __forceinline__ void lean_renorm(uint32_t &x, uint32_t &a, uint32_t &bal, uint32_t lt) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 now, t, w;\n\t"
                 "setp.lt.u32 p, %0, 32768;\n\t"
                 "vote.sync.ballot.b32 now, p, 0xffffffff;\n\t"
                 "lop3.b32 t, %3, now, %2, 0xCA;\n\t"          // the lanes below: this step's ballot; this lane and above: the last one's
                 "popc.b32 t, t;\n\t"
                 "mad.lo.u32 %1, t, 2, %1;\n\t"
                 "ld.shared.u16 w, [%1];\n\t"
                 "@p mad.lo.u32 %0, %0, 65536, w;\n\t"
                 "mov.b32 %2, now;\n\t}"
                 : "+r"(x), "+r"(a), "+r"(bal) : "r"(lt) : "memory");
}
// one coordinate symbol (Eq. 18) from the table at shared-memory address `table`: returns the entry
__device__ __forceinline__ uint32_t lean_step(uint32_t &x, uint32_t &a, uint32_t &bal, uint32_t table, uint32_t lt) {
    uint32_t e;
    asm volatile("{\n\t.reg .b32 q, u, f, bi;\n\t"
                 "shr.u32 q, %0, 11;\n\t"
                 "mad.lo.u32 u, q, 0xFFFFE000, %2;\n\t"        // slot address 4 (x & 2047) + table = 4 x - 8192 (x >> 11) + table
                 "mad.lo.u32 u, %0, 4, u;\n\t"
                 "ld.shared.u32 %1, [u];\n\t"
                 "shr.u32 f, %1, 21;\n\t"
                 "and.b32 bi, %1, 0x7FF;\n\t"
                 "mad.lo.u32 %0, f, q, bi;\n\t}"
                 : "+r"(x), "=r"(e) : "r"(table) : "memory");
    lean_renorm(x, a, bal, lt);
    return e;
}
__device__ __forceinline__ uint4 decode_group_lean_bf16(uint32_t &x, uint32_t &wa, uint32_t lut_addr, CosetFreq cf, uint32_t lt,
                                                        uint32_t k0_bits, float sigma) {
    uint32_t a = wa, bal = 0, e[9];
    {   // the coset: slot below f0 -> 0, else 1
        const uint32_t u = x & 2047u, q = x >> 11;
        const bool c1 = u >= cf.f0;
        x = (c1 ? cf.f1 : max(cf.f0, 1u)) * q + (c1 ? u - cf.f0 : u);
        e[0] = c1 ? 1u : 0u;
        lean_renorm(x, a, bal, lt);
    }
    const uint32_t tab = lut_addr + e[0] * kCosetStride;
#pragma unroll
    for (int k = 1; k <= 8; ++k) e[k] = lean_step(x, a, bal, tab + uint32_t(k - 1) * kLutStride, lt);
    wa = __shfl_sync(0xFFFFFFFFu, a, 0) + 2u * __popc(bal);      // lane 0's address is the cursor before the last step
    const uint32_t par = (e[1] ^ e[2] ^ e[3] ^ e[4] ^ e[5] ^ e[6] ^ e[7]) & 0x800u;
    const uint32_t cc = kExp4096 | (e[0] << 10);
    const uint64_t kk = pack64(k0_bits, k0_bits);
    const uint64_t ss = pack64(__float_as_uint(sigma), __float_as_uint(sigma));
    uint32_t xb[8];
#pragma unroll
    for (int k = 1; k <= 7; ++k) xb[k - 1] = (e[k] & kCodeMask) | cc;
    xb[7] = (e[8] & kCodeMask) | par | cc;
    float w[8];
#pragma unroll
    for (int i = 0; i < 8; i += 2) unpack64(mul2(sub2(pack64(xb[i], xb[i + 1]), kk), ss), w[i], w[i + 1]);
    return make_uint4(pack_bf16(w[0], w[1]), pack_bf16(w[2], w[3]), pack_bf16(w[4], w[5]), pack_bf16(w[6], w[7]));
}

// ---- payload ring ------------------------------------------------------------------------------------
// chunk c of a tile = global bytes [a0 + CHUNK c, a0 + CHUNK (c + 1)), a0 = tile's first word rounded down to
// 16 bytes; it lives in ring slot c mod SLOTS, and a chunk in one of the slots that make up the ring's first 512
// bytes is written a second time behind the ring's end.  `room` = bytes from a0 to the end of the payload: nothing
// beyond it is read (cp.async zero-fills the rest).  The decode kernel's rings are 3 x 512 bytes; the kernel that
// feeds the tensor cores needs the shared memory for its operands and takes 4 x 256.
template <uint32_t CHUNK = kChunk, uint32_t SLOTS = kRingSlots>
__device__ __forceinline__ void ring_issue(uint32_t ring, uint64_t a0, uint32_t room, uint32_t c, uint32_t lane) {
    if (lane < CHUNK / 16u) {
        uint32_t o = CHUNK * c + 16u * lane;
        uint32_t n = 16;
        if (o + 16u > room) {
            n = o < room ? room - o : 0u;
            if (n == 0) o = 0;                   // nothing is read, but keep the address a valid one
        }
        const uint32_t slot = c % SLOTS;
        const uint32_t dst = ring + CHUNK * slot + 16u * lane;
        cp_async16(dst, a0 + o, n);
        if (slot < kRingMirror / CHUNK) cp_async16(dst + CHUNK * SLOTS, a0 + o, n);
    }
    cp_async_commit();
}

// The cursor entered a new chunk: request chunks up to SLOTS - 1 ahead of it and wait for all but the
// newest.  `threshold` = start of the chunk after the cursor's at the previous service; chunks up to
// threshold / CHUNK + SLOTS - 2 have been requested.  A group touches at most 448 + 62 bytes from its start,
// which the chunks complete after this call cover (1024 bytes from the cursor's chunk on, or 768).
template <uint32_t CHUNK = kChunk, uint32_t SLOTS = kRingSlots>
__device__ __forceinline__ void ring_service(uint32_t ring, uint64_t a0, uint32_t room, uint32_t pos, uint32_t &threshold,
                                             uint32_t lane) {
    const uint32_t cur = pos / CHUNK;
    for (uint32_t c = threshold / CHUNK + SLOTS - 1u; c < cur + SLOTS; ++c) ring_issue<CHUNK, SLOTS>(ring, a0, room, c, lane);
    cp_async_wait<1>();
    __syncwarp();
    threshold = CHUNK * (cur + 1u);
}

// what a chain needs to know about its tile
struct TileSetup {
    uint32_t x;            // this lane's state, forced into [2^15, 2^31) (a no-op for a valid stream)
    uint32_t off, end;     // first payload word of the tile and of the next one
    uint32_t v0, nv;       // first block and number of blocks
    uint64_t a0;           // global address of chunk 0
    uint32_t lead, room;   // cursor position inside chunk 0; payload bytes from a0 on
};
__device__ __forceinline__ TileSetup tile_setup(const JobParams &J, uint32_t tile, bool valid, uint32_t lane) {
    TileSetup T;
    const uint32_t *rec = J.tile_index + size_t(tile) * 33u;
    T.x = max(rec[lane] & 0x7FFFFFFFu, ep::kStateLow);
    T.off = min(rec[32], J.total_words);    // a damaged index must not move reads outside the payload
    T.end = (tile + 1 < J.n_tiles) ? rec[33 + 32] : rec[33];
    T.v0 = tile * J.V;
    T.nv = valid ? min(J.V, J.n_vec - T.v0) : 0u;
    const uint64_t pay = reinterpret_cast<uint64_t>(J.stream + J.off_payload);
    const uint64_t first = pay + 2ull * T.off;
    T.a0 = first & ~15ull;
    T.lead = uint32_t(first - T.a0);
    T.room = uint32_t(pay + 2ull * J.total_words - T.a0);     // the payload is shorter than 2 GB
    return T;
}

// Plain C++ version of the tile loop, used for the field-dump mode, for streams with b < 11 and for tensors with
// fewer than 32 blocks per row (a group may then cross several rows).
template <int DT>
__device__ __forceinline__ void decode_tile_plain(const JobParams &J, uint32_t tile, uint32_t lut_addr, CosetFreq cf,
                                                  uint32_t ring, uint32_t lane) {
    const TileSetup T = tile_setup(J, tile, true, lane);
    uint32_t x = T.x;
    const uint32_t b = J.b, mask = (1u << b) - 1u, lt = (1u << lane) - 1u;
    const uint32_t per_row = J.per_row;
    uint32_t pos = T.lead;        // byte position of the cursor relative to a0
    uint32_t threshold;           // next chunk boundary the cursor has not yet crossed
    for (uint32_t c = 0; c < kRingSlots; ++c) ring_issue(ring, T.a0, T.room, c, lane);
    cp_async_wait<1>();
    __syncwarp();
    threshold = kChunk;
    const uint32_t k0_bits = __float_as_uint(float(4096 - J.zlo));
    const uint32_t row_max = J.n_vec / per_row - 1u;
    for (uint32_t g = 0; g * 32u < T.nv; ++g) {
        if (pos >= threshold) ring_service(ring, T.a0, T.room, pos, threshold, lane);
        const uint32_t wa0 = ring + pos % kRingBytes;
        uint32_t wa = wa0;
        const uint32_t i = g * 32u + lane;
        const bool act = i < T.nv;
        const uint32_t v = T.v0 + i;
        const float sigma = (DT == EP_FIELDS_I32) ? 0.f : __ldg(J.scales + min(v / per_row, row_max));
        decode_group_plain<DT>(x, wa, lut_addr, cf, mask, b, lt, act, k0_bits, sigma, J.zlo,
                               static_cast<uint8_t *>(J.out) + size_t(v) * BlockBytes<DT>::value);
        pos += wa - wa0;
    }
    cp_async_wait<0>();          // nothing may still be landing in the ring when the next tile starts
    __syncwarp();
    // integrity: the encoder started every state at 2^15 and the tile's words end where the next tile's begin
    const bool bad = (x != ep::kStateLow) || (T.off + ((pos - T.lead) >> 1) != T.end);
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(&g_ep_status, 1u);
}

// ---- the hot loop in PTX: several tiles per warp ----------------------------------------------------------
// All groups of EP_CHAINS tiles ("chains" A, B, ...), written as one asm statement so that every branch can be
// marked warp-uniform (bra.uni), the chains' instructions can be interleaved, and the rare work - refilling a
// payload ring, moving to the next row, a tile's end - sits out of line behind ONE warp vote per loop pass.
//
// Word addresses.  Lane l of a chain keeps its own address a_l of the word it would take in the current step.
// With bal_k the ballot of the lanes that need a word after step k,
//     a_l(k) = a_l(k-1) + 2 popc((bal_k & below_l) | (bal_{k-1} & ~below_l)):
// the words taken in step k-1 by lanes l and above, plus those taken in step k by the lanes below.  The two
// masks are disjoint, so one bit-select and ONE population count per step replace the prefix count and the
// cursor advance (lane 0's address is the tile's word cursor before the step).
//
// Loop-carried per chain: x state, a word address, bal last ballot, doff byte offset of this lane's block in the
// output; inside the asm: lim = first doff at which this lane leaves its row or the tile, wthr = ring address at
// which the cursor leaves its 512-byte chunk (minus 2), ss = the row scale twice, act = lane has a block.
// A chain whose tile has ended (or that never had one) runs along with all lanes inactive: states and
// addresses stand still, nothing is stored.
//
// asm operands: chain c has x, a, bal, doff at %(4c) .. %(4c+3); then come the shared inputs, named here:
#if EP_CHAINS == 1
#define EP_LT "%4"
#define EP_LUT0 "%5"
#define EP_LUT1 "%6"
#define EP_CTX "%7"
#define EP_KK "%8"
#define EP_OUT "%9"
#define EP_F0 "%10"
#define EP_F1 "%11"
#define EP_L16 "%12"
#define EP_L2B "%13"
#define EP_HS2 "%14"
#define EP_HOTOFF "%15"
#elif EP_CHAINS == 2
#define EP_LT "%8"     /* lanes below this one (mask) */
#define EP_LUT0 "%9"   /* tables of coset 0 */
#define EP_LUT1 "%10"  /* tables of coset 1 */
#define EP_CTX "%11"   /* this warp's context block */
#define EP_KK "%12"    /* {4096 - zlo, 4096 - zlo} as fp32 pair */
#define EP_OUT "%13"   /* output base address */
#define EP_F0 "%14"    /* frequency of coset 0 */
#define EP_F1 "%15"    /* frequency of coset 1, at least 1 */
#define EP_L16 "%16"   /* 16 * lane */
#define EP_L2B "%17"   /* 2^12-slot streams: the complete second-level array (global memory), */
#define EP_HS2 "%18"   /* twice the first code of the hot window, */
#define EP_HOTOFF "%19"  /* offset of the hot part in shared memory */
#elif EP_CHAINS == 3
#define EP_LT "%12"
#define EP_LUT0 "%13"
#define EP_LUT1 "%14"
#define EP_CTX "%15"
#define EP_KK "%16"
#define EP_OUT "%17"
#define EP_F0 "%18"
#define EP_F1 "%19"
#define EP_L16 "%20"
#define EP_L2B "%21"
#define EP_HS2 "%22"
#define EP_HOTOFF "%23"
#else
#define EP_LT "%16"
#define EP_LUT0 "%17"
#define EP_LUT1 "%18"
#define EP_CTX "%19"
#define EP_KK "%20"
#define EP_OUT "%21"
#define EP_F0 "%22"
#define EP_F1 "%23"
#define EP_L16 "%24"
#define EP_L2B "%25"
#define EP_HS2 "%26"
#define EP_HOTOFF "%27"
#endif
// one macro call per chain: M(S = suffix, X, AW, BAL, DOFF, CB = byte offset of the chain's context, more...)
#define EP_CH_A(M, ...) M("A", "%0", "%1", "%2", "%3", "32", ##__VA_ARGS__)
#define EP_CH_B(M, ...) M("B", "%4", "%5", "%6", "%7", "64", ##__VA_ARGS__)
#define EP_CH_C(M, ...) M("C", "%8", "%9", "%10", "%11", "96", ##__VA_ARGS__)
#define EP_CH_D(M, ...) M("D", "%12", "%13", "%14", "%15", "128", ##__VA_ARGS__)
#if EP_CHAINS == 1
#define EP_ALL(M, ...) EP_CH_A(M, ##__VA_ARGS__)
#elif EP_CHAINS == 2
#define EP_ALL(M, ...) EP_CH_A(M, ##__VA_ARGS__) EP_CH_B(M, ##__VA_ARGS__)
#elif EP_CHAINS == 3
#define EP_ALL(M, ...) EP_CH_A(M, ##__VA_ARGS__) EP_CH_B(M, ##__VA_ARGS__) EP_CH_C(M, ##__VA_ARGS__)
#else
#define EP_ALL(M, ...) EP_CH_A(M, ##__VA_ARGS__) EP_CH_B(M, ##__VA_ARGS__) EP_CH_C(M, ##__VA_ARGS__) EP_CH_D(M, ##__VA_ARGS__)
#endif

#define EP_CM "0x1FF800"
// The loop body is written line by line: every macro below emits ONE instruction for ONE chain, and EP_ALL
// repeats it for all chains before the next line follows.  The assembler keeps this order, so a chain's next
// dependent instruction comes only after the other chains' same instruction: that distance, not the
// scheduler, is what hides the latencies inside a warp.
// Common parameters of a line: S, X, AW, BAL, DOFF, CB (see EP_CH_A); then E = name of the entry register
// (a suffix is added), OFF = byte offset of the field's table, BIN / BOUT = which register holds the previous /
// receives the new ballot: NA, NB (temporaries) or BL (the chain's loop-carried operand).
#define EP_B_NA(S, BAL) "na" S
#define EP_B_NB(S, BAL) "nb" S
#define EP_B_BL(S, BAL) BAL
// a coordinate field: table OFF / 8192 of the lane's coset (Eq. 18)
#ifdef EP_STEP_WIDE
// x * 2^21 as a 64-bit product gives x >> 11 in the high word and the slot in the top bits of the low word,
// e * 2^11 gives f in the high word: both on the multiply-add pipe instead of shifts and masks on the ALU pipe
// (the two multipliers come from memory so that the assembler does not turn the products back into shifts)
#define EP_L1(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "mul.wide.u32 xw" S ", " X ", m21;\n\t" "mov.b64 {u" S ", q" S "}, xw" S ";\n\t"
#define EP_L2(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "shr.u32 u" S ", u" S ", 19;\n\t" "add.u32 u" S ", u" S ", tab" S ";\n\t"
#define EP_L3(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "ld.shared.u32 " E S ", [u" S "+" OFF "];\n\t"
#define EP_L4(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT)
#ifdef EP_STEP_WIDEQ
#define EP_L5(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "shr.u32 f" S ", " E S ", 21;\n\t"
#else
#define EP_L5(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "mul.wide.u32 xw" S ", " E S ", m11;\n\t" "mov.b64 {bi" S ", f" S "}, xw" S ";\n\t"
#endif
#else
// slot address 4 (x & 0x7FF) + tab as 4 x - 8192 (x >> 11) + tab: two multiply-adds instead of a mask and one (the
// multiply-add pipe has room, the ALU pipe has not; measured + 0.3 % / + 0.8 % on the 8192^2 tensor / the layer)
#ifndef EP_SLOT_MASK
#define EP_L1(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "shr.u32 q" S ", " X ", 11;\n\t" "mad.lo.u32 u" S ", q" S ", 0xFFFFE000, tab" S ";\n\t"
#define EP_L2(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "mad.lo.u32 u" S ", " X ", 4, u" S ";\n\t"
#else
#define EP_L1(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "and.b32 u" S ", " X ", 0x7FF;\n\t"
#define EP_L2(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "mad.lo.u32 u" S ", u" S ", 4, tab" S ";\n\t"
#endif
#define EP_L3(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "ld.shared.u32 " E S ", [u" S "+" OFF "];\n\t"
#ifndef EP_SLOT_MASK
#define EP_L4(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT)
#elif defined(EP_Q_MULHI)
// x >> 11 as the high word of x * 2^21: on the multiply-add pipe, off the step's critical path
#define EP_L4(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "mul.hi.u32 q" S ", " X ", m21;\n\t"
#else
#define EP_L4(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "shr.u32 q" S ", " X ", 11;\n\t"
#endif
#define EP_L5(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "shr.u32 f" S ", " E S ", 21;\n\t"
#endif
#define EP_L6(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "and.b32 bi" S ", " E S ", 0x7FF;\n\t"
#define EP_L7(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "@act" S " mad.lo.u32 " X ", f" S ", q" S ", bi" S ";\n\t"
// renormalisation: lanes whose state fell below 2^15 take a word each, in lane order
#define EP_L8(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "setp.lt.and.u32 p" S ", " X ", 32768, act" S ";\n\t"
#define EP_L9(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "vote.sync.ballot.b32 " EP_B_##BOUT(S, BAL) ", p" S ", 0xffffffff;\n\t"
#define EP_L10(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) \
    "lop3.b32 t" S ", " EP_LT ", " EP_B_##BOUT(S, BAL) ", " EP_B_##BIN(S, BAL) ", 0xCA;\n\t"
#define EP_L11(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "popc.b32 t" S ", t" S ";\n\t"
#define EP_L12(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "mad.lo.u32 " AW ", t" S ", 2, " AW ";\n\t"
#define EP_L13(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "ld.shared.u16 w" S ", [" AW "];\n\t"
#define EP_L14(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT) "@p" S " mad.lo.u32 " X ", " X ", 65536, w" S ";\n\t"
#define EP_RENORM_ALL(E, OFF, BIN, BOUT)                                                             \
    EP_ALL(EP_L8, E, OFF, BIN, BOUT) EP_ALL(EP_L9, E, OFF, BIN, BOUT) EP_ALL(EP_L10, E, OFF, BIN, BOUT)  \
    EP_ALL(EP_L11, E, OFF, BIN, BOUT) EP_ALL(EP_L12, E, OFF, BIN, BOUT) EP_ALL(EP_L13, E, OFF, BIN, BOUT) \
    EP_ALL(EP_L14, E, OFF, BIN, BOUT)
#define EP_STEP_ALL(E, OFF, BIN, BOUT)                                                               \
    EP_ALL(EP_L1, E, OFF, BIN, BOUT) EP_ALL(EP_L2, E, OFF, BIN, BOUT) EP_ALL(EP_L3, E, OFF, BIN, BOUT)   \
    EP_ALL(EP_L4, E, OFF, BIN, BOUT) EP_ALL(EP_L5, E, OFF, BIN, BOUT) EP_ALL(EP_L6, E, OFF, BIN, BOUT)   \
    EP_ALL(EP_L7, E, OFF, BIN, BOUT) EP_RENORM_ALL(E, OFF, BIN, BOUT)
// the coset: slot below f0 -> coset 0 with frequency f0, else coset 1 with frequency f1 and offset f0
#define EP_C1(S, X, AW, BAL, DOFF, CB) "and.b32 u" S ", " X ", 0x7FF;\n\t"
#define EP_C2(S, X, AW, BAL, DOFF, CB) "shr.u32 q" S ", " X ", 11;\n\t"
#define EP_C3(S, X, AW, BAL, DOFF, CB) "setp.lt.u32 pc" S ", u" S ", " EP_F0 ";\n\t"
#define EP_C4(S, X, AW, BAL, DOFF, CB) "selp.b32 f" S ", f0c, " EP_F1 ", pc" S ";\n\t"
#define EP_C5(S, X, AW, BAL, DOFF, CB) "@!pc" S " sub.u32 u" S ", u" S ", " EP_F0 ";\n\t"
#define EP_C6(S, X, AW, BAL, DOFF, CB) "@act" S " mad.lo.u32 " X ", f" S ", q" S ", u" S ";\n\t"
#define EP_C7(S, X, AW, BAL, DOFF, CB) "selp.b32 tab" S ", " EP_LUT0 ", " EP_LUT1 ", pc" S ";\n\t"
#define EP_C8(S, X, AW, BAL, DOFF, CB) "selp.b32 cc" S ", c0r, c1r, pc" S ";\n\t"
#define EP_COSET_ALL                                                                                 \
    EP_ALL(EP_C1) EP_ALL(EP_C2) EP_ALL(EP_C3) EP_ALL(EP_C4) EP_ALL(EP_C5) EP_ALL(EP_C6) EP_ALL(EP_C7) EP_ALL(EP_C8) \
    EP_RENORM_ALL("", "", BL, NA)
// Eq. 5 and the product of Eq. 19 for two neighbouring weights: 4096 + code (+ 1/2) as fp32, minus 4096 - zlo, times sigma
#define EP_XA(S, X, AW, BAL, DOFF, CB, E) "lop3.b32 xa" S ", " E S ", " EP_CM ", cc" S ", 0xEA;\n\t"
#define EP_XB(S, X, AW, BAL, DOFF, CB, E) "lop3.b32 xb" S ", " E S ", " EP_CM ", cc" S ", 0xEA;\n\t"
#define EP_P1(S, X, AW, BAL, DOFF, CB) "mov.b64 pr" S ", {xa" S ", xb" S "};\n\t"
#define EP_P2(S, X, AW, BAL, DOFF, CB) "sub.rn.f32x2 pr" S ", pr" S ", " EP_KK ";\n\t"
#define EP_P3(S, X, AW, BAL, DOFF, CB) "mul.rn.f32x2 pr" S ", pr" S ", ss" S ";\n\t"
#define EP_P4(S, X, AW, BAL, DOFF, CB) "mov.b64 {wl" S ", wh" S "}, pr" S ";\n\t"
#ifdef EP_SCALAR_FP
#undef EP_P1
#undef EP_P2
#undef EP_P3
#undef EP_P4
#define EP_P1(S, X, AW, BAL, DOFF, CB) "mov.b32 wl" S ", xa" S ";\n\t" "sub.rn.f32 wl" S ", wl" S ", k0f;\n\t"
#define EP_P2(S, X, AW, BAL, DOFF, CB) "mov.b32 wh" S ", xb" S ";\n\t" "sub.rn.f32 wh" S ", wh" S ", k0f;\n\t"
#define EP_P3(S, X, AW, BAL, DOFF, CB) "mul.rn.f32 wl" S ", wl" S ", sg" S ";\n\t"
#define EP_P4(S, X, AW, BAL, DOFF, CB) "mul.rn.f32 wh" S ", wh" S ", sg" S ";\n\t"
#endif
#define EP_PAIR_ALL EP_ALL(EP_P1) EP_ALL(EP_P2) EP_ALL(EP_P3) EP_ALL(EP_P4)
// parity of z1 + ... + z7 = xor of the codes' lowest bits (bit 11 of the entries; zlo is even): the lowest bit of z8
#define EP_PAR3(S, X, AW, BAL, DOFF, CB, EA, EB, EC) "lop3.b32 par" S ", " EA S ", " EB S ", " EC S ", 0x96;\n\t"
#define EP_PARX(S, X, AW, BAL, DOFF, CB) "lop3.b32 par" S ", par" S ", 0x800, cc" S ", 0xEA;\n\t"
#define EP_X8(S, X, AW, BAL, DOFF, CB) "lop3.b32 xb" S ", e8" S ", " EP_CM ", par" S ", 0xEA;\n\t"
#define EP_ADDR(S, X, AW, BAL, DOFF, CB) "mad.wide.u32 ad" S ", " DOFF ", 1, " EP_OUT ";\n\t"

// ---- streams with 2^12 slots per table (b = 12: the paper's setting for 8 bpp targets) ------------------------
// Sixteen tables of 4096 four-byte entries would not fit shared memory, so the lookup has two levels.  Shared memory
// holds, per slot, 16 bits: twice the code of the slot's coordinate value, code = z - zlo (2m - zlo for the m field;
// the same 128 KB and strides as the one-level tables of b = 11).  The code is all Eq. 5 needs - it goes into the
// mantissa of 2^22 (bit 0 = the coset's half, bit 1 = one) - and it addresses the second level, one word per (table,
// code): f << 16 | F.  Entries of the kHotSpan codes around zero sit in shared memory, all of them in global memory.
// HOFF / COFF = byte offset of the field's table in the hot part / in the complete array.
#define EP_N1(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "and.b32 u" S ", " X ", 0xFFF;\n\t"
#define EP_N2(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "mad.lo.u32 t" S ", u" S ", 2, tab" S ";\n\t"
#define EP_N3(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "ld.shared.u16 " E S ", [t" S "+" OFF "];\n\t"
/* codes inside the hot window: entry in shared memory; the others: global memory */
#define EP_N4(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "sub.u32 w" S ", " E S ", " EP_HS2 ";\n\t"
#define EP_N5(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "setp.lt.u32 pc" S ", w" S ", 1056;\n\t"
#define EP_N6(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "mad.lo.u32 t" S ", w" S ", 2, hotc" S ";\n\t"
#define EP_N7(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "mad.wide.u32 ad" S ", " E S ", 2, lc" S ";\n\t"
#define EP_N8(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) \
    "@pc" S " ld.shared.u32 w" S ", [t" S "+" HOFF "];\n\t" "@!pc" S " ld.global.nc.u32 w" S ", [ad" S "+" COFF "];\n\t"
#define EP_N9(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "shr.u32 q" S ", " X ", 12;\n\t"
#define EP_N10(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "shr.u32 f" S ", w" S ", 16;\n\t"
#define EP_N11(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "and.b32 bi" S ", w" S ", 0xFFFF;\n\t"
#define EP_N12(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "sub.u32 bi" S ", u" S ", bi" S ";\n\t"
#define EP_N13(S, X, AW, BAL, DOFF, CB, E, OFF, BIN, BOUT, HOFF, COFF) "@act" S " mad.lo.u32 " X ", f" S ", q" S ", bi" S ";\n\t"
#define EP_STEP12_ALL(E, OFF, BIN, BOUT, HOFF, COFF)                                                             \
    EP_ALL(EP_N1, E, OFF, BIN, BOUT, HOFF, COFF) EP_ALL(EP_N2, E, OFF, BIN, BOUT, HOFF, COFF)                    \
    EP_ALL(EP_N3, E, OFF, BIN, BOUT, HOFF, COFF) EP_ALL(EP_N4, E, OFF, BIN, BOUT, HOFF, COFF)                    \
    EP_ALL(EP_N5, E, OFF, BIN, BOUT, HOFF, COFF) EP_ALL(EP_N6, E, OFF, BIN, BOUT, HOFF, COFF)                    \
    EP_ALL(EP_N7, E, OFF, BIN, BOUT, HOFF, COFF) EP_ALL(EP_N8, E, OFF, BIN, BOUT, HOFF, COFF)                    \
    EP_ALL(EP_N9, E, OFF, BIN, BOUT, HOFF, COFF) EP_ALL(EP_N10, E, OFF, BIN, BOUT, HOFF, COFF)                   \
    EP_ALL(EP_N11, E, OFF, BIN, BOUT, HOFF, COFF) EP_ALL(EP_N12, E, OFF, BIN, BOUT, HOFF, COFF)                  \
    EP_ALL(EP_N13, E, OFF, BIN, BOUT, HOFF, COFF) EP_RENORM_ALL(E, OFF, BIN, BOUT)
#define EP_C1_12(S, X, AW, BAL, DOFF, CB) "and.b32 u" S ", " X ", 0xFFF;\n\t"
#define EP_C2_12(S, X, AW, BAL, DOFF, CB) "shr.u32 q" S ", " X ", 12;\n\t"
/* per coset: 2^22 (+ 1/2) as fp32, the hot part and the complete array of its eight tables */
#define EP_C8_12(S, X, AW, BAL, DOFF, CB) "selp.b32 cc" S ", d0r, d1r, pc" S ";\n\t"
#define EP_C9_12(S, X, AW, BAL, DOFF, CB) "selp.b32 hotc" S ", hotb, hotb1, pc" S ";\n\t"
#define EP_C10_12(S, X, AW, BAL, DOFF, CB) "selp.b64 lc" S ", " EP_L2B ", l2b1, pc" S ";\n\t"
#define EP_COSET12_ALL                                                                               \
    EP_ALL(EP_C1_12) EP_ALL(EP_C2_12) EP_ALL(EP_C3) EP_ALL(EP_C4) EP_ALL(EP_C5) EP_ALL(EP_C6) EP_ALL(EP_C7)  \
    EP_ALL(EP_C8_12) EP_ALL(EP_C9_12) EP_ALL(EP_C10_12) EP_RENORM_ALL("", "", BL, NA)
// Eq. 5: 2^22 + code (+ 1/2) as fp32; z8 = 2m + parity of (z1 + ... + z7), the parity from bit 1 of the xor of the
// looked-up values (zlo is even)
#define EP_XA12(S, X, AW, BAL, DOFF, CB, E) "or.b32 xa" S ", " E S ", cc" S ";\n\t"
#define EP_XB12(S, X, AW, BAL, DOFF, CB, E) "or.b32 xb" S ", " E S ", cc" S ";\n\t"
#define EP_PARX12(S, X, AW, BAL, DOFF, CB) "lop3.b32 par" S ", par" S ", 0x2, cc" S ", 0xEA;\n\t"
#define EP_X8_12(S, X, AW, BAL, DOFF, CB) "or.b32 xb" S ", e8" S ", par" S ";\n\t"
// the nine steps and the arithmetic of one group, 2^11-slot and 2^12-slot streams
#define EP_BODY11(CVT)                                                                                                \
        EP_COSET_ALL                                                                                                  \
        EP_STEP_ALL("e1", "0", NA, NB)     EP_ALL(EP_XA, "e1")                                                        \
        EP_STEP_ALL("e2", "8192", NB, NA)  EP_ALL(EP_XB, "e2") EP_PAIR_ALL EP_ALL(CVT, "0")                           \
        EP_STEP_ALL("e3", "16384", NA, NB) EP_ALL(EP_PAR3, "e1", "e2", "e3") EP_ALL(EP_XA, "e3")                      \
        EP_STEP_ALL("e4", "24576", NB, NA) EP_ALL(EP_XB, "e4") EP_PAIR_ALL EP_ALL(CVT, "1")                           \
        EP_STEP_ALL("e5", "32768", NA, NB) EP_ALL(EP_PAR3, "par", "e4", "e5") EP_ALL(EP_XA, "e5")                     \
        EP_STEP_ALL("e6", "40960", NB, NA) EP_ALL(EP_XB, "e6") EP_PAIR_ALL EP_ALL(CVT, "2")                           \
        EP_STEP_ALL("e7", "49152", NA, NB) EP_ALL(EP_PAR3, "par", "e6", "e7") EP_ALL(EP_XA, "e7")                     \
        EP_STEP_ALL("e8", "57344", NB, BL) EP_ALL(EP_PARX) EP_ALL(EP_X8) EP_PAIR_ALL EP_ALL(CVT, "3")
#define EP_BODY12(CVT)                                                                                                \
        EP_COSET12_ALL                                                                                                \
        EP_STEP12_ALL("e1", "0", NA, NB, "0", "0")             EP_ALL(EP_XA12, "e1")                                  \
        EP_STEP12_ALL("e2", "8192", NB, NA, "2112", "16384")   EP_ALL(EP_XB12, "e2") EP_PAIR_ALL EP_ALL(CVT, "0")     \
        EP_STEP12_ALL("e3", "16384", NA, NB, "4224", "32768")  EP_ALL(EP_PAR3, "e1", "e2", "e3") EP_ALL(EP_XA12, "e3") \
        EP_STEP12_ALL("e4", "24576", NB, NA, "6336", "49152")  EP_ALL(EP_XB12, "e4") EP_PAIR_ALL EP_ALL(CVT, "1")     \
        EP_STEP12_ALL("e5", "32768", NA, NB, "8448", "65536")  EP_ALL(EP_PAR3, "par", "e4", "e5") EP_ALL(EP_XA12, "e5") \
        EP_STEP12_ALL("e6", "40960", NB, NA, "10560", "81920") EP_ALL(EP_XB12, "e6") EP_PAIR_ALL EP_ALL(CVT, "2")     \
        EP_STEP12_ALL("e7", "49152", NA, NB, "12672", "98304") EP_ALL(EP_PAR3, "par", "e6", "e7") EP_ALL(EP_XA12, "e7") \
        EP_STEP12_ALL("e8", "57344", NB, BL, "14784", "114688") EP_ALL(EP_PARX12) EP_ALL(EP_X8_12) EP_PAIR_ALL EP_ALL(CVT, "3")

// per output type: CVT(S, j, lo, hi) turns weights 2j, 2j+1 into their stored form, STORE(S) writes the block
#define EP_CVT_BF16(S, X, AW, BAL, DOFF, CB, J) "cvt.rn.bf16x2.f32 o" J S ", wh" S ", wl" S ";\n\t"
#define EP_CVT_FP16(S, X, AW, BAL, DOFF, CB, J) "cvt.rn.satfinite.f16x2.f32 o" J S ", wh" S ", wl" S ";\n\t"
#define EP_ST_16(S, X, AW, BAL, DOFF, CB) "@act" S " st.global.v4.b32 [ad" S "], {o0" S ", o1" S ", o2" S ", o3" S "};\n\t"
#define EP_CVT_E4M3(S, X, AW, BAL, DOFF, CB, J) "cvt.rn.satfinite.e4m3x2.f32 h" J S ", wh" S ", wl" S ";\n\t"
#define EP_CVT_E5M2(S, X, AW, BAL, DOFF, CB, J) "cvt.rn.satfinite.e5m2x2.f32 h" J S ", wh" S ", wl" S ";\n\t"
#define EP_ST_F8(S, X, AW, BAL, DOFF, CB)                                                    \
    "mov.b32 o0" S ", {h0" S ", h1" S "};\n\t"                           \
    "mov.b32 o1" S ", {h2" S ", h3" S "};\n\t"                           \
    "@act" S " st.global.v2.b32 [ad" S "], {o0" S ", o1" S "};\n\t"
#define EP_CVT_FP32(S, X, AW, BAL, DOFF, CB, J) "mov.b32 ia" J S ", wl" S ";\n\t" "mov.b32 ib" J S ", wh" S ";\n\t"
#define EP_ST_FP32(S, X, AW, BAL, DOFF, CB)                                                  \
    "@act" S " st.global.v4.b32 [ad" S "], {ia0" S ", ib0" S ", ia1" S ", ib1" S "};\n\t" \
    "@act" S " st.global.v4.b32 [ad" S "+16], {ia2" S ", ib2" S ", ia3" S ", ib3" S "};\n\t"
/* one-byte integers: round to nearest even into s32 (out-of-range values end at INT_MIN / INT_MAX, NaN at 0), then
   saturate and pack four at a time: cvt.pack d, a, b, c gives (c << 16) | sat(a) << 8 | sat(b) */
#define EP_CVT_I8(S, X, AW, BAL, DOFF, CB, J) "cvt.rni.s32.f32 ia" J S ", wl" S ";\n\t" "cvt.rni.s32.f32 ib" J S ", wh" S ";\n\t"
#define EP_ST_INT8(S, X, AW, BAL, DOFF, CB)                                                  \
    "cvt.pack.sat.s8.s32.b32 o2" S ", ib1" S ", ia1" S ", 0;\n\t"        \
    "cvt.pack.sat.s8.s32.b32 o0" S ", ib0" S ", ia0" S ", o2" S ";\n\t"  \
    "cvt.pack.sat.s8.s32.b32 o3" S ", ib3" S ", ia3" S ", 0;\n\t"        \
    "cvt.pack.sat.s8.s32.b32 o1" S ", ib2" S ", ia2" S ", o3" S ";\n\t"  \
    "@act" S " st.global.v2.b32 [ad" S "], {o0" S ", o1" S "};\n\t"
#define EP_ST_UINT8(S, X, AW, BAL, DOFF, CB)                                                 \
    "cvt.pack.sat.u8.s32.b32 o2" S ", ib1" S ", ia1" S ", 0;\n\t"        \
    "cvt.pack.sat.u8.s32.b32 o0" S ", ib0" S ", ia0" S ", o2" S ";\n\t"  \
    "cvt.pack.sat.u8.s32.b32 o3" S ", ib3" S ", ia3" S ", 0;\n\t"        \
    "cvt.pack.sat.u8.s32.b32 o1" S ", ib2" S ", ia2" S ", o3" S ";\n\t"  \
    "@act" S " st.global.v2.b32 [ad" S "], {o0" S ", o1" S "};\n\t"

// registers of one chain
#define EP_REGS(S, X, AW, BAL, DOFF, CB)                                                                             \
    ".reg .pred p" S ", pc" S ", act" S ";\n\t"                                                                      \
    ".reg .b32 u" S ", q" S ", f" S ", bi" S ", t" S ", w" S ", tab" S ", cc" S ", par" S ", na" S ", nb" S ";\n\t"  \
    ".reg .b32 e1" S ", e2" S ", e3" S ", e4" S ", e5" S ", e6" S ", e7" S ", e8" S ", xa" S ", xb" S ";\n\t"        \
    ".reg .b32 o0" S ", o1" S ", o2" S ", o3" S ", ia0" S ", ib0" S ", ia1" S ", ib1" S ", ia2" S ", ib2" S ", ia3" S ", ib3" S ";\n\t" \
    ".reg .b16 h0" S ", h1" S ", h2" S ", h3" S ";\n\t"                                                              \
    ".reg .f32 wl" S ", wh" S ", sg" S ";\n\t"                                                                       \
    ".reg .b32 lim" S ", wthr" S ", hotc" S ";\n\t"                                                                  \
    ".reg .b64 pr" S ", ss" S ", ad" S ", xw" S ", lc" S ";\n\t"
// before the first pass: the cursor leaves its first chunk at ring + chunk size - 2; lim = 0 sends the chain through EP_ROWS
#define EP_INIT(S, X, AW, BAL, DOFF, CB)                                 \
    "ld.shared.u32 r0, [" EP_CTX "+" CB "+16];\n\t"                      \
    "add.u32 wthr" S ", r0, 510;\n\t"                                    \
    "mov.u32 lim" S ", 0;\n\t"

#define EP_ADVANCE(S, X, AW, BAL, DOFF, CB, GROUP_BYTES) "add.u32 " DOFF ", " DOFF ", " GROUP_BYTES ";\n\t"
// go on only if no lane of the chain left its chunk or reached its lim
#define EP_CALM(S, X, AW, BAL, DOFF, CB)                                 \
    "setp.lt.and.u32 pq, " AW ", wthr" S ", pq;\n\t"                     \
    "setp.lt.and.u32 pq, " DOFF ", lim" S ", pq;\n\t"
#define EP_CALM0(S, X, AW, BAL, DOFF, CB)                                \
    "setp.lt.u32 pq, " AW ", wthr" S ";\n\t"                             \
    "setp.lt.and.u32 pq, " DOFF ", lim" S ", pq;\n\t"
#if EP_CHAINS == 1
#define EP_CALM_ALL EP_CH_A(EP_CALM0)
#elif EP_CHAINS == 2
#define EP_CALM_ALL EP_CH_A(EP_CALM0) EP_CH_B(EP_CALM)
#elif EP_CHAINS == 3
#define EP_CALM_ALL EP_CH_A(EP_CALM0) EP_CH_B(EP_CALM) EP_CH_C(EP_CALM)
#else
#define EP_CALM_ALL EP_CH_A(EP_CALM0) EP_CH_B(EP_CALM) EP_CH_C(EP_CALM) EP_CH_D(EP_CALM)
#endif

// some lane of the chain reached its lim (also run once on entry): where is each lane now?
// CB = byte offset of the chain's part of the context block.  row = doff / bytes per row by a multiply-high
// with ceil(2^32 / bytes per row), which is at most one too large.
#define EP_ROWS(S, X, AW, BAL, DOFF, CB)                                 \
    "setp.ge.u32 pr, " DOFF ", lim" S ";\n\t"                                                                  \
    "vote.sync.any.pred pr, pr, 0xffffffff;\n\t"                                                               \
    "@!pr bra.uni EP_ROWS_END_" S ";\n\t"                                                                      \
    "ld.shared.v2.u32 {r0, r1}, [" EP_CTX "+8];\n\t"    /* bytes per row, last row */                          \
    "ld.shared.u32 r2, [" EP_CTX "+" CB "+24];\n\t"     /* offset after the tile's last block */               \
    "ld.shared.u32 r5, [" EP_CTX "+24];\n\t"                                                                   \
    "mul.hi.u32 r3, " DOFF ", r5;\n\t"                                                                         \
    "mul.lo.u32 r4, r3, r0;\n\t"                                                                               \
    "setp.gt.u32 pv, r4, " DOFF ";\n\t"                                                                        \
    "@pv sub.u32 r3, r3, 1;\n\t"                                                                               \
    "mad.lo.u32 r4, r3, r0, r0;\n\t"                    /* offset at which this lane enters the next row */    \
    "min.u32 lim" S ", r4, r2;\n\t"                                                                            \
    "setp.lt.u32 act" S ", " DOFF ", r2;\n\t"                                                                  \
    "@!act" S " mov.u32 lim" S ", 0xffffffff;\n\t"      /* a lane without a block never asks again */          \
    "min.u32 r3, r3, r1;\n\t"                                                                                  \
    "ld.shared.u64 ra, [" EP_CTX "];\n\t"                                                                      \
    "mul.wide.u32 rb, r3, 4;\n\t"                                                                              \
    "add.s64 ra, ra, rb;\n\t"                                                                                  \
    "ld.global.nc.b32 r4, [ra];\n\t"                                                                           \
    "mov.b64 ss" S ", {r4, r4};\n\t"                                                                           \
    "mov.b32 sg" S ", r4;\n\t"                                                                                 \
    "EP_ROWS_END_" S ":\n\t"
#define EP_ANY_ACT(S, X, AW, BAL, DOFF, CB) "or.pred pr, pr, act" S ";\n\t"

// The chain's cursor left its 512-byte chunk (a group takes at most 448 + 62 bytes, so it is in the next one):
// request the chunk two ahead of the cursor's new one into the slot that became free, wait for all requests but
// this newest one, and move every address back by the ring's length when the cursor's chunk is the one in slot 0
// again.  The context keeps the request state ready to use: source address, bytes left, destination.
#define EP_SERVICE(S, X, AW, BAL, DOFF, CB)                              \
    "setp.ge.u32 pr, " AW ", wthr" S ";\n\t"                                                                   \
    "vote.sync.any.pred pr, pr, 0xffffffff;\n\t"                                                               \
    "@!pr bra.uni EP_SVC_END_" S ";\n\t"                                                                       \
    "shfl.sync.idx.b32 r6, " AW ", 0, 31, 0xffffffff;\n\t"                                                     \
    "popc.b32 r0, " BAL ";\n\t"                                                                                \
    "mad.lo.u32 r6, r0, 2, r6;\n\t"                     /* the cursor's address */                             \
    "add.u32 r0, wthr" S ", 2;\n\t"                     /* end of the chunk it was in */                       \
    "setp.lt.u32 pq, r6, r0;\n\t"                                                                              \
    "@pq bra.uni EP_SVC_END_" S ";\n\t"                 /* (a lane address ran ahead of the cursor: not yet) */ \
    "ld.shared.v4.u32 {r11, r12, r1, r2}, [" EP_CTX "+" CB "];\n\t"  /* source, bytes left, destination */     \
    "ld.shared.u32 r10, [" EP_CTX "+" CB "+16];\n\t"    /* ring base */                                        \
    "mov.b64 ra, {r11, r12};\n\t"                                                                              \
    "sub.s32 r3, r1, " EP_L16 ";\n\t"                                                                          \
    "min.s32 r3, r3, 16;\n\t"                           /* bytes of this lane's 16 inside the payload */       \
    "setp.gt.s32 pv, r3, 0;\n\t"                        /* none: no request (nothing valid reads them) */      \
    "mad.wide.u32 rb, " EP_L16 ", 1, ra;\n\t"                                                                  \
    "add.u32 r5, r2, " EP_L16 ";\n\t"                                                                          \
    "@pv cp.async.cg.shared.global [r5], [rb], 16, r3;\n\t"                                                    \
    "setp.eq.and.u32 pq, r2, r10, pv;\n\t"              /* slot 0 is written to the mirror as well */          \
    "@pq cp.async.cg.shared.global [r5+1536], [rb], 16, r3;\n\t"                                               \
    "cp.async.commit_group;\n\t"                                                                               \
    "add.cc.u32 r11, r11, 512;\n\t"                                                                            \
    "addc.u32 r12, r12, 0;\n\t"                                                                                \
    "sub.s32 r1, r1, 512;\n\t"                                                                                 \
    "add.u32 r2, r2, 512;\n\t"                                                                                 \
    "sub.u32 r4, r2, r10;\n\t"                                                                                 \
    "setp.ge.u32 pv, r4, 1536;\n\t"                                                                            \
    "selp.b32 r2, r10, r2, pv;\n\t"                                                                            \
    "st.shared.v4.u32 [" EP_CTX "+" CB "], {r11, r12, r1, r2};\n\t"                                            \
    "cp.async.wait_group 1;\n\t"                                                                               \
    "bar.warp.sync 0xffffffff;\n\t"                                                                            \
    "add.u32 wthr" S ", wthr" S ", 512;\n\t"            /* the cursor's chunk is the next slot's */            \
    "sub.u32 r4, wthr" S ", r10;\n\t"                                                                          \
    "setp.lt.u32 pq, r4, 2046;\n\t"                                                                            \
    "@pq bra.uni EP_SVC_END_" S ";\n\t"                                                                        \
    "sub.u32 wthr" S ", wthr" S ", 1536;\n\t"           /* past the third slot: everything back by the ring */ \
    "sub.u32 " AW ", " AW ", 1536;\n\t"                                                                        \
    "ld.shared.u32 r5, [" EP_CTX "+" CB "+20];\n\t"                                                            \
    "sub.u32 r5, r5, 1536;\n\t"                                                                                \
    "st.shared.u32 [" EP_CTX "+" CB "+20], r5;\n\t"                                                            \
    "EP_SVC_END_" S ":\n\t"

#if EP_CHAINS == 1
#define EP_LOOP_OPERANDS                                                                                              \
        : "+&r"(x[0]), "+&r"(a[0]), "+&r"(bal[0]), "+&r"(doff[0])
#elif EP_CHAINS == 2
#define EP_LOOP_OPERANDS                                                                                              \
        : "+&r"(x[0]), "+&r"(a[0]), "+&r"(bal[0]), "+&r"(doff[0]), "+&r"(x[1]), "+&r"(a[1]), "+&r"(bal[1]), "+&r"(doff[1])
#elif EP_CHAINS == 3
#define EP_LOOP_OPERANDS                                                                                              \
        : "+&r"(x[0]), "+&r"(a[0]), "+&r"(bal[0]), "+&r"(doff[0]), "+&r"(x[1]), "+&r"(a[1]), "+&r"(bal[1]), "+&r"(doff[1]), \
          "+&r"(x[2]), "+&r"(a[2]), "+&r"(bal[2]), "+&r"(doff[2])
#else
#define EP_LOOP_OPERANDS                                                                                              \
        : "+&r"(x[0]), "+&r"(a[0]), "+&r"(bal[0]), "+&r"(doff[0]), "+&r"(x[1]), "+&r"(a[1]), "+&r"(bal[1]), "+&r"(doff[1]), \
          "+&r"(x[2]), "+&r"(a[2]), "+&r"(bal[2]), "+&r"(doff[2]), "+&r"(x[3]), "+&r"(a[3]), "+&r"(bal[3]), "+&r"(doff[3])
#endif

#define EP_TILES_LOOP_ASM(BODY, CVT, STORE, GROUP_BYTES)                                                                    \
    asm volatile(                                                                                                     \
        "{\n\t"                                                                                                       \
        EP_ALL(EP_REGS)                                                                                               \
        ".reg .pred pq, pv, pr;\n\t"                                                                                  \
        ".reg .b32 r0, r1, r2, r3, r4, r5, r6, r7, r8, r9, r10, r11, r12, c0r, c1r, d0r, d1r, f0c, m21, m11, hotb, hotb1;\n\t" \
        ".reg .b64 ra, rb, l2b1;\n\t"                                                                                 \
        ".reg .f32 k0f, k1f;\n\t"                                                                                     \
        "mov.b64 {k0f, k1f}, " EP_KK ";\n\t"                                                                          \
        "mov.b32 c0r, 0x45800000;\n\t"                                                                                \
        "mov.b32 c1r, 0x45800400;\n\t"                                                                                \
        "mov.b32 d0r, 0x4A800000;\n\t"                /* 2^22, 2^22 + 1/2 (2^12-slot streams) */                    \
        "mov.b32 d1r, 0x4A800001;\n\t"                                                                                \
        "max.u32 f0c, " EP_F0 ", 1;\n\t"                /* frequency used for coset 0: never 0 */                     \
        "add.u32 hotb, " EP_LUT0 ", " EP_HOTOFF ";\n\t"   /* 2^12-slot streams: hot entries of coset 0, */              \
        "add.u32 hotb1, hotb, 16896;\n\t"                 /* of coset 1; complete array of coset 1 */                   \
        "add.s64 l2b1, " EP_L2B ", 131072;\n\t"                                                                       \
        "ld.shared.v2.u32 {m21, m11}, [" EP_CTX "+16];\n\t" /* 2^21, 2^11 */                                          \
        EP_ALL(EP_INIT)                                                                                               \
        "bra.uni EP_RARE;\n\t"                                                                                        \
        "EP_LOOP:\n\t"                                                                                                \
        BODY(CVT)                                                                                                     \
        EP_ALL(EP_ADDR) EP_ALL(STORE)                                                                                \
        EP_ALL(EP_ADVANCE, #GROUP_BYTES)                                                                              \
        /* one vote for everything rare */                                                                            \
        EP_CALM_ALL                                                                                                   \
        "vote.sync.all.pred pq, pq, 0xffffffff;\n\t"                                                                  \
        "@pq bra.uni EP_LOOP;\n\t"                                                                                    \
        "EP_RARE:\n\t"                                                                                                \
        EP_ALL(EP_ROWS)                                                                                               \
        "setp.lt.u32 pr, " EP_LT ", 0;\n\t"          /* false */                                                                                   \
        EP_ALL(EP_ANY_ACT)                                                                                            \
        "vote.sync.any.pred pr, pr, 0xffffffff;\n\t"                                                                  \
        "@!pr bra.uni EP_DONE;\n\t"                                                                                   \
        EP_ALL(EP_SERVICE)                                                                                            \
        "bra.uni EP_LOOP;\n\t"                                                                                        \
        "EP_DONE:\n\t"                                                                                                \
        "}"                                                                                                           \
        /* every read-write operand is early-clobber: the loop reads the inputs after it has updated them */         \
        EP_LOOP_OPERANDS                                                                                              \
        : "r"(lt), "r"(lut_addr), "r"(lut_addr + kCosetStride), "r"(ctx), "l"(kk), "l"(out_base), "r"(cf.f0),         \
          "r"(cf.f1), "r"(lane16), "l"(l2base), "r"(hs2), "n"(kHotBase)                                             \
        : "memory")

// kChains tiles of a tensor whose rows hold at least 32 blocks and whose tables have 2^B slots (B = 11: one-level
// tables; B = 12: two levels, see EP_M1); chain c takes tile
// `first + c`.  A chain whose slot lies past the job's last tile gets that last tile's record, only so that its
// addresses stay inside the stream, and no block at all.  The number of groups is data here, not control flow the
// compiler reasons about: every branch on it is a bra.uni on a warp vote.
// `tables_pending`: the job's lookup tables are still being written (by this CTA's own stores or copies): the
// tiles' records and first payload chunks are requested first, the CTA barrier comes after.
template <int DT, int B>
__device__ __forceinline__ void decode_tiles_fast(const JobParams &J, uint32_t first, uint32_t lut_addr, CosetFreq cf,
                                                  uint32_t ring, uint32_t ctx, uint32_t lane, bool tables_pending) {
    constexpr uint32_t BB = Out<DT>::kBlockBytes;
    const uint32_t lt = (1u << lane) - 1u, lane16 = 16u * lane;
    uint32_t x[kChains], a[kChains], bal[kChains], doff[kChains], off[kChains], end[kChains], lead[kChains];
    bool valid[kChains];
#pragma unroll
    for (uint32_t c = 0; c < kChains; ++c) {
        valid[c] = first + c < J.tile_cnt;
        const uint32_t tile = J.tile0 + min(first + c, J.tile_cnt - 1u);
        const uint32_t rg = ring + c * kRingStride, cctx = ctx + kCtxChain + c * kCtxChainStride;
        const TileSetup T = tile_setup(J, tile, valid[c], lane);
        for (uint32_t k = 0; k < kRingSlots; ++k) ring_issue(rg, T.a0, T.room, k, lane);
        // the record of the tile this chain takes in the CTA's next round (132 bytes: two lines), into L2
        if (lane < 2u && tile + kTilesPerRound < J.n_tiles) prefetch_l2(J.tile_index + size_t(tile + kTilesPerRound) * 33u + 32u * lane);
        if (lane == 0) {                 // the next request is chunk 3, into slot 0
            prefetch_l2(J.scales + min(T.v0 / J.per_row, J.row_max));      // the first row scale the loop will ask for
            sts64(cctx + kCcSrc, T.a0 + kRingBytes);
            sts32(cctx + kCcRem, T.room - kRingBytes);
            sts32(cctx + kCcDst, rg);
            sts32(cctx + kCcRing, rg);
            sts32(cctx + kCcWbase, rg);
            sts32(cctx + kCcEndo, (T.v0 + T.nv) * BB);
        }
        x[c] = T.x; a[c] = rg + T.lead; bal[c] = 0; doff[c] = (T.v0 + lane) * BB;
        off[c] = T.off; end[c] = T.end; lead[c] = T.lead;
    }
    cp_async_wait<1>();           // all but the last chain's third chunk have landed (and the table image, if any)
    __syncwarp();
    if (tables_pending) __syncthreads();
    const uint32_t k0 = __float_as_uint(float((B == 11 ? 4096 : 4194304) - J.zlo));
    const uint64_t kk = pack64(k0, k0);
    const uint64_t out_base = reinterpret_cast<uint64_t>(J.out);
    const uint64_t l2base = reinterpret_cast<uint64_t>(J.cold);
    const uint32_t hs2 = J.hs2;
    if constexpr (B == 11) {
        if constexpr (DT == EP_BF16) EP_TILES_LOOP_ASM(EP_BODY11, EP_CVT_BF16, EP_ST_16, 512);
        else if constexpr (DT == EP_FP16) EP_TILES_LOOP_ASM(EP_BODY11, EP_CVT_FP16, EP_ST_16, 512);
        else if constexpr (DT == EP_FP8_E4M3) EP_TILES_LOOP_ASM(EP_BODY11, EP_CVT_E4M3, EP_ST_F8, 256);
        else if constexpr (DT == EP_FP8_E5M2) EP_TILES_LOOP_ASM(EP_BODY11, EP_CVT_E5M2, EP_ST_F8, 256);
        else if constexpr (DT == EP_FP32) EP_TILES_LOOP_ASM(EP_BODY11, EP_CVT_FP32, EP_ST_FP32, 1024);
        else if constexpr (DT == EP_UINT8) EP_TILES_LOOP_ASM(EP_BODY11, EP_CVT_I8, EP_ST_UINT8, 256);
        else EP_TILES_LOOP_ASM(EP_BODY11, EP_CVT_I8, EP_ST_INT8, 256);
    } else {
        if constexpr (DT == EP_BF16) EP_TILES_LOOP_ASM(EP_BODY12, EP_CVT_BF16, EP_ST_16, 512);
        else if constexpr (DT == EP_FP16) EP_TILES_LOOP_ASM(EP_BODY12, EP_CVT_FP16, EP_ST_16, 512);
        else if constexpr (DT == EP_FP8_E4M3) EP_TILES_LOOP_ASM(EP_BODY12, EP_CVT_E4M3, EP_ST_F8, 256);
        else if constexpr (DT == EP_FP8_E5M2) EP_TILES_LOOP_ASM(EP_BODY12, EP_CVT_E5M2, EP_ST_F8, 256);
        else if constexpr (DT == EP_FP32) EP_TILES_LOOP_ASM(EP_BODY12, EP_CVT_FP32, EP_ST_FP32, 1024);
        else if constexpr (DT == EP_UINT8) EP_TILES_LOOP_ASM(EP_BODY12, EP_CVT_I8, EP_ST_UINT8, 256);
        else EP_TILES_LOOP_ASM(EP_BODY12, EP_CVT_I8, EP_ST_INT8, 256);
    }
    cp_async_wait<0>();           // nothing may still be landing in the rings when the next tiles start
    __syncwarp();
    // integrity: the encoder started every state at 2^15 and a tile's words end where the next tile's begin
    bool bad = false;
#pragma unroll
    for (uint32_t c = 0; c < kChains; ++c) {
        const uint32_t cur = __shfl_sync(0xFFFFFFFFu, a[c], 0) + 2u * __popc(bal[c]) -
                             lds32(ctx + kCtxChain + c * kCtxChainStride + kCcWbase);
        bad |= valid[c] && ((x[c] != ep::kStateLow) || (off[c] + ((cur - lead[c]) >> 1) != end[c]));
    }
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(&g_ep_status, 1u);
    __syncwarp();                 // the context block is rewritten by the next tiles
}

// One persistent CTA per SM.  The rounds of all jobs of the launch form one list (job after job); CTA k takes the
// rounds whose cumulative cost at their start lies in [k, k + 1) * ceil(total / gridDim.x) - a contiguous stretch,
// usually inside one job - and sets the lookup tables up again when the stretch crosses into the next job.  Everything
// that steers this (loop bounds, job changes) depends on blockIdx and kernel parameters only, so the compiler
// sees warp-uniform control flow and puts no divergence guards around the warp votes of the hot loop; in the last
// round of a job a chain past the job's last tile goes through the same code with no block to decode.
template <int DT>
__global__ void __launch_bounds__(kThreads, 1) ep_decode_smem_kernel(const __grid_constant__ BatchParams P) {
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t lut_addr = uint32_t(__cvta_generic_to_shared(smem));
    const uint32_t ring = lut_addr + kRingBase + warp * (kChains * kRingStride);
    const uint32_t ctx = lut_addr + kCtxBase + warp * kCtxBytes;
    bool tables_in_use = false;
    for (int j = 0; j < P.n_jobs; ++j) {
        const JobParams &J = P.job[j];
        // rounds r of this job with cost_begin + r * round_cost in [lo, hi), this CTA's share of the total cost
        // (recomputed per job rather than kept in registers across the decode loops)
        const uint32_t lo = P.cost_per_cta * blockIdx.x, hi = lo + P.cost_per_cta;      // below 2^31 (see the launcher)
        const uint32_t a = lo > J.cost_begin ? lo - J.cost_begin : 0u, b = hi > J.cost_begin ? hi - J.cost_begin : 0u;
        const uint32_t r0 = min((a + J.round_cost - 1u) / J.round_cost, J.rounds);
        const uint32_t r1 = min((b + J.round_cost - 1u) / J.round_cost, J.rounds);
        if (r0 >= r1) continue;
        if (tables_in_use) __syncthreads();          // every warp is done with the previous job's tables
        // the table image is requested first: the tiles' records and payload (two dependent reads of memory that no
        // cache holds yet) are on their way while it arrives
        if (J.lut_image) copy_tables_smem(J.lut_image, lut_addr, J.b == 12u);
        else build_tables_smem(J, lut_addr, warp, lane);
        const CosetFreq cf = load_coset(J);
        bool tables_pending = true;
        tables_in_use = true;
        // (a stream with 2^12 slots reaches this kernel only in the configuration of the hot loop: see the launcher)
        const bool fast = DT != EP_FIELDS_I32 && J.per_row >= 32u && (J.b == 11u || J.b == 12u) && J.V < (1u << 20);
        if (fast && lane == 0) {                     // what the hot loop's rare paths need to know about the job
            sts64(ctx + kCtxScales, reinterpret_cast<uint64_t>(J.scales));
            sts32(ctx + kCtxRowBytes, J.row_bytes);
            sts32(ctx + kCtxRowMax, J.row_max);      // the step after a tensor's last block must not read past the scales
            sts32(ctx + kCtxMul21, 1u << 21);
            sts32(ctx + kCtxMul11, 1u << 11);
            sts32(ctx + kCtxRowRcp, J.row_rcp);
        }
        __syncwarp();
        for (uint32_t r = r0; r < r1; ++r) {
            const uint32_t base = r * kTilesPerRound + kChains * warp;
            if constexpr (DT != EP_FIELDS_I32) {
                if (fast) {
                    if (kTwoLevelInLoop && J.b == 12u) {
                        if constexpr (kTwoLevelInLoop) decode_tiles_fast<DT, 12>(J, base, lut_addr, cf, ring, ctx, lane, tables_pending);
                    } else {
                        decode_tiles_fast<DT, 11>(J, base, lut_addr, cf, ring, ctx, lane, tables_pending);
                    }
                    tables_pending = false;
                    continue;
                }
            }
            if (tables_pending) {
                cp_async_wait<0>();
                __syncthreads();
                tables_pending = false;
            }
            for (uint32_t c = 0; c < kChains; ++c)
                if (base + c < J.tile_cnt) decode_tile_plain<DT>(J, J.tile0 + base + c, lut_addr, cf, ring, lane);
        }
    }
}

// ======================================================================================================
// Decode fused into a matrix product (the step the paper leaves as future work, Sec. "Limitations and future
// work": its decoder still materialises the dense tensor before the product).  First slice: y = x W^T for up
// to 32 tokens - the regime in which reading the weights dominates a linear layer -, W decoded tile by tile
// straight into the shared-memory operand of a tcgen05 matrix instruction and never written to global memory.
//
// The stream must have one tile per row of W (V = C / 8) and C a multiple of 256.  The rows are spread evenly over
// the SMs; a CTA takes its range 30 rows at a time, one row per warp: warps 0 .. 29 decode their rows group by group
// (a group = 32 blocks = 256 columns), so after every group the CTA holds a 30 x 256 slab of W - the B operand
// (N = 32 with two idle rows, K-major, 128-byte swizzle: a lane's 16-byte block is one piece of a swizzled row, so
// the stores are conflict-free).  Warps 30 and 31 decode nothing.  One lane of warp 30 brings the matching 256
// columns of x in (A operand, M = 64 rows of which the first 16 or 32 are tokens; the others read whatever shared
// memory follows and produce accumulator rows nobody stores) with four tensor copies (cp.async.bulk.tensor, the
// copy engine swizzles).  One lane of warp 31 waits until x has landed and all rows of the slab are stored and
// issues the slab's sixteen K = 16 instructions.  (A decoding warp cannot do that on the side: whoever issues falls
// behind by the time it takes, and with two slabs every warp is at most one group ahead of the slowest - measured
// 138 us for the layer below; one warp for copies and instructions together 90 us, its single instruction stream
// being the slowest in the CTA; two warps on two schedulers 84 us.)  The fp32 accumulator (64 lanes x 32 columns)
// stays in tensor memory over the whole row and is read out once per step.
//
// Shared memory: the lookup tables (128 KB), 32 payload rings of 4 x 256 + 512 bytes (48 KB), then A (16 KB: two units
// of x - a group's 256 columns of up to 16 tokens each, or half a group's of up to 32 -, refilled by the loading warp as
// soon as the instructions that read a unit are done), B (two slabs of 16 KB: the warps decode the next group while the
// tensor core reads the last one) and the mbarriers.  What bounds the token count: a group's columns of x must be in
// flight while the group is decoded (about 1 us), every CTA re-reads x from L2, and 16 KB is the landing space left.
// Every wait on an mbarrier gives up after kSpinLimit polls, raises the abort word and lets the kernel run to its
// end (wrong output, status flag set) instead of hanging.
struct GemmParams {
    JobParams J;
    const uint16_t *x;            // [T, C] bf16, row-major
    float *y;                     // [T, R] fp32, row-major
    uint32_t T, Tpad;             // tokens; rows of x that are staged (16 or 32)
    uint32_t R, C;
    uint32_t rows_per_cta;        // CTA k takes rows [k, k + 1) * rows_per_cta, 31 at a time
    uint32_t groups;              // C / 256
};

constexpr uint32_t kGemmChunk = 256, kGemmSlots = 4;     // payload ring of this kernel
constexpr uint32_t kGemmRingStride = kGemmChunk * kGemmSlots + kRingMirror;   // 1536
constexpr uint32_t kGemmA = kRingBase + 32u * kGemmRingStride;   // A operand: per stage four 64-column tiles of Tpad rows
constexpr uint32_t kGemmB = kGemmA + 16384;              // B operand: two slabs of four 64-column tiles of 32 rows
constexpr uint32_t kGemmBar = kGemmB + 32768;            // mbarriers, tensor-memory address, abort word, counter
constexpr uint32_t kGemmSmem = kGemmBar + 256;
constexpr uint32_t kSpinLimit = 1u << 18;             // attempts of about a microsecond each at most: a quarter of a second
constexpr uint32_t kGemmRows = 30;                       // rows of W per step: warps 0 .. 29 decode one each, warp 30 brings x in, warp 31 issues the matrix instructions
constexpr uint32_t kGemmIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((32u >> 3) << 17) | ((64u >> 4) << 24);   // f32 += bf16 x bf16, K-major both, N = 32, M = 64
static_assert(kGemmA % 1024 == 0, "swizzled operand tiles start on 1024-byte boundaries");
static_assert(kGemmSmem <= 232448, "more shared memory than an sm_100 CTA can have");

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// a test that never waits
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// one attempt: the thread may be suspended by the hardware for up to about a microsecond while the phase is pending
// (a busy test_wait loop of 32 waiting lanes took half of the kernel's issue slots away from the decoding warps)
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    return ok != 0;
}
// waits for the phase of the given parity to complete; false (and the abort word set) if it does not within the limit
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t abort_addr) {
    if (mbar_test(bar, parity)) return true;             // usually the phase is long complete
    if (lds32(abort_addr)) return false;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 255u) == 255u && lds32(abort_addr)) return false;
    }
    sts32(abort_addr, 1u);
    return false;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// K-major operand tile with 128-byte swizzle: rows of 128 bytes, groups of eight rows 1024 bytes apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    return uint64_t((smem_addr >> 4) & 0x3FFFu) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) |
           (uint64_t(2) << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <uint32_t TPAD>
__global__ void __launch_bounds__(kThreads, 1) ep_decode_gemm_kernel(const __grid_constant__ GemmParams P,
                                                                     const __grid_constant__ CUtensorMap x_map) {
    extern __shared__ __align__(16) uint8_t smem[];      // (the operand tiles need 1024: checked at run time, see abort word)
    const JobParams &J = P.J;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t lut_addr = uint32_t(__cvta_generic_to_shared(smem));
    const uint32_t ring = lut_addr + kRingBase + warp * kGemmRingStride;
    const uint32_t a_base = lut_addr + kGemmA, b_base = lut_addr + kGemmB;
    // A holds two units of x, a unit being half of what fits: four tiles of 64 columns x 16 rows (one group's columns), or
    // two tiles x 32 rows (half a group's).  Per unit one mbarrier "landed" and one "read"; per slab of B one "rows stored"
    // and one "read".
    constexpr uint32_t a_tile_bytes = TPAD * 128u, kUnitTiles = 8192u / a_tile_bytes, kUnitsPerGroup = 4u / kUnitTiles;
    const uint32_t bar_a = lut_addr + kGemmBar, bar_afree = bar_a + 64u, bar_mma = bar_a + 128u, bar_b = bar_a + 144u,
                   slot = bar_a + 160u, abort_addr = bar_a + 164u;
    if (tid == 0) {
        for (uint32_t i = 0; i < 2u; ++i) {
            mbar_init(bar_a + 8u * i, 1u);       // the loading lane's arrival; completes when the unit's tiles have landed
            mbar_init(bar_afree + 8u * i, 1u);   // the commit after the matrix instructions that read the unit
        }
        mbar_init(bar_mma, 1u);              // the commit after a group's matrix instructions
        mbar_init(bar_mma + 8u, 1u);
        mbar_init(bar_b, kGemmRows);         // every decoding warp, when its row of the slab is stored
        mbar_init(bar_b + 8u, kGemmRows);
        sts32(abort_addr, (lut_addr & 1023u) ? 1u : 0u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {                         // 32 columns of tensor memory: the 64 x 32 fp32 accumulator
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(32u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp >= kGemmRows) {                 // rows 30 and 31 of both slabs belong to no warp: zero (this warp's row, all its pieces)
        for (uint32_t i = lane; i < 2u * 4u * 8u; i += 32u)
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(b_base + (i >> 5) * 16384u + ((i >> 3) & 3u) * 4096u + warp * 128u + (i & 7u) * 16u), "r"(0u) : "memory");
        fence_async_smem();
    }
    copy_tables_smem(J.lut_image, lut_addr, false);
    const CosetFreq cf = load_coset(J);
    cp_async_wait<0>();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32(slot);

    const uint32_t row_begin = min(blockIdx.x * P.rows_per_cta, P.R), row_end = min(row_begin + P.rows_per_cta, P.R);
    const uint32_t steps = (row_end - row_begin + kGemmRows - 1u) / kGemmRows;
    const uint32_t q_total = steps * P.groups;               // groups this CTA hands to the tensor core
    // usually the phase is long complete: one test by the whole warp; otherwise one lane polls and the warp follows
    auto wait_warp = [&](uint32_t bar, uint32_t parity) {
        if (mbar_test(bar, parity)) return;
        if (lane == 0) mbar_wait(bar, parity, abort_addr);
        __syncwarp();
    };
    bool bad = false;
    // the end of a step (accumulator read out, next rows may overwrite it) concerns the decoding warps and the issuing
    // warp; the loading warp runs ahead of them across steps
    auto step_sync = [&]() {
        tc_fence_before();
        asm volatile("bar.sync 1, %0;" ::"n"(kThreads - 32) : "memory");
        tc_fence_after();
    };

    if (warp == kGemmRows) {
        // ---- the loading warp: one lane brings x into A, unit after unit, nothing else ----
        // tile i of the CTA's sequence = columns [64 i, 64 i + 64) of x, counted over all groups (and again from column 0 for
        // every step); the copy engine lays it out and swizzles it; rows past the last token lie outside the tensor and
        // arrive as zeros
        if (lane == 0) {
            const uint32_t tiles_per_step = 4u * P.groups;
            for (uint32_t j = 0; j < kUnitsPerGroup * q_total; ++j) {
                const uint32_t buf = j & 1u;
                // (after a wait that ran out nothing is copied any more: re-arming a barrier whose phase never completed
                // would overflow its transaction count)
                if (j >= 2u && !mbar_wait(bar_afree + 8u * buf, ((j >> 1) - 1u) & 1u, abort_addr)) break;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a + 8u * buf), "r"(8192u) : "memory");
#pragma unroll
                for (uint32_t t = 0; t < kUnitTiles; ++t)
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(a_base + buf * 8192u + t * a_tile_bytes), "l"(&x_map),
                                   "r"(((j * kUnitTiles + t) % tiles_per_step) * 64u), "r"(0u), "r"(bar_a + 8u * buf)
                                 : "memory");
            }
        }
        __syncwarp();
    } else if (warp == kGemmRows + 1u) {
        // ---- the issuing warp: one lane waits for a group's rows and, unit by unit, for x, and issues the matrix instructions ----
        for (uint32_t q = 0; q < q_total; ++q) {
            const uint32_t g = q % P.groups;
            if (lane == 0) {
                bool ready = mbar_wait(bar_b + 8u * (q & 1u), (q >> 1) & 1u, abort_addr);
                // descriptors differ in their address field only: low word + (bytes >> 4)
                const uint64_t da = umma_desc(a_base), db = umma_desc(b_base + 16384u * (q & 1u));
                const uint32_t da_hi = uint32_t(da >> 32), db_hi = uint32_t(db >> 32), da_lo = uint32_t(da), db_lo = uint32_t(db);
#pragma unroll
                for (uint32_t h = 0; h < kUnitsPerGroup; ++h) {
                    const uint32_t j = kUnitsPerGroup * q + h, buf = j & 1u;
                    ready = ready && mbar_wait(bar_a + 8u * buf, (j >> 1) & 1u, abort_addr);
                    tc_fence_after();
#pragma unroll
                    for (uint32_t t = 0; t < kUnitTiles; ++t)
#pragma unroll
                        for (uint32_t k = 0; k < 4; ++k)             // 16 columns = 32 bytes further along the swizzled rows
                            if (ready)                               // (operands that never arrived are not multiplied)
                                umma_bf16(tmem, pack64(da_lo + ((buf * 8192u + t * a_tile_bytes + 32u * k) >> 4), da_hi),
                                          pack64(db_lo + (((h * kUnitTiles + t) * 4096u + 32u * k) >> 4), db_hi), kGemmIdesc,
                                          (g | h | t | k) ? 1u : 0u);
                    umma_commit(bar_afree + 8u * buf);
                }
                umma_commit(bar_mma + 8u * (q & 1u));
            }
            __syncwarp();
            if (g + 1u == P.groups) step_sync();
        }
    } else {
        // ---- the decoding warps: one row of W each, group by group into the slabs of B ----
        const uint32_t lt = (1u << lane) - 1u;
        const uint32_t k0_bits = __float_as_uint(float(4096 - J.zlo));
        // where this lane's block of a group goes in a slab: 64-column tile lane / 8, row = warp, piece lane % 8 of the row
        const uint32_t b_dst = b_base + (lane >> 3) * 4096u + warp * 128u + (((lane & 7u) ^ (warp & 7u)) << 4);
        uint32_t q = 0;
        for (uint32_t r0 = row_begin; r0 < row_end; r0 += kGemmRows) {
            const bool active = r0 + warp < row_end;                    // the last rows of the CTA's range may be fewer than 31
            const uint32_t tile = min(r0 + warp, P.R - 1u);             // = the row of W
            const TileSetup Tl = tile_setup(J, tile, active, lane);
            uint32_t x = Tl.x, pos = Tl.lead, threshold = kGemmChunk;
            if (active) {
                for (uint32_t c = 0; c < kGemmSlots; ++c) ring_issue<kGemmChunk, kGemmSlots>(ring, Tl.a0, Tl.room, c, lane);
                cp_async_wait<1>();
                __syncwarp();
            }
            const float sigma = __ldg(J.scales + tile);
            // the row this warp takes in the next step: its record is asked for now and, a few groups on, the start of
            // its payload is brought into L2, so that the next step does not begin with two reads from DRAM in a row
            const bool has_next = r0 + kGemmRows + warp < row_end;
            const uint32_t *rec_next = J.tile_index + size_t(min(tile + kGemmRows, P.R - 1u)) * 33u;
            uint32_t off_next = 0;
            if (has_next) off_next = __ldg(rec_next + 32);
            if (has_next && lane == 0) prefetch_l2(rec_next);
            for (uint32_t g = 0; g < P.groups; ++g, ++q) {
                if (g == 2u && has_next) {
                    const uint64_t at = 2ull * min(off_next, J.total_words) + 128u * lane;      // 4 KB: the ring's first fill and more
                    if (at < 2ull * J.total_words) prefetch_l2(J.stream + J.off_payload + at);
                }
                uint4 blk = make_uint4(0u, 0u, 0u, 0u);
                if (active) {
                    if (pos >= threshold) ring_service<kGemmChunk, kGemmSlots>(ring, Tl.a0, Tl.room, pos, threshold, lane);
                    const uint32_t wa0 = ring + pos % (kGemmChunk * kGemmSlots);
                    uint32_t wa = wa0;
                    blk = decode_group_lean_bf16(x, wa, lut_addr, cf, lt, k0_bits, sigma);
                    pos += wa - wa0;
                }
                // the slab is free: the tensor core is done with the group that used it last, two groups ago
                if (q >= 2u) wait_warp(bar_mma + 8u * (q & 1u), ((q >> 1) - 1u) & 1u);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(b_dst + 16384u * (q & 1u)), "r"(blk.x), "r"(blk.y), "r"(blk.z), "r"(blk.w) : "memory");
                fence_async_smem();          // the stores above are read through the async proxy
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_b + 8u * (q & 1u)) : "memory");
            }
            // the accumulator of these rows: with M = 64, token 16 w + l is lane l < 16 of warp w's quarter; columns = rows of W
            wait_warp(bar_mma + 8u * ((q - 1u) & 1u), ((q - 1u) >> 1) & 1u);
            tc_fence_after();
            if (warp < 2u) {
                uint32_t v[32];
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                             "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, "
                             "%23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                             : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                               "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                               "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                               "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                             : "r"(tmem + ((warp * 32u) << 16)));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const uint32_t t = warp * 16u + lane;
                if (lane < 16u && t < P.T) {
                    float *dst = P.y + size_t(t) * P.R + r0;
                    const uint32_t n = min(kGemmRows, row_end - r0);
#pragma unroll
                    for (uint32_t i = 0; i < kGemmRows; ++i)
                        if (i < n) dst[i] = __uint_as_float(v[i]);
                }
            }
            cp_async_wait<0>();              // nothing may still be landing in the ring when the next row starts
            step_sync();                     // the accumulator has been read before the next rows overwrite it
            bad |= active && ((x != ep::kStateLow) || (Tl.off + ((pos - Tl.lead) >> 1) != Tl.end));
        }
    }
    const bool aborted = lds32(abort_addr) != 0;
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(&g_ep_status, 1u);
    if (aborted && tid == 0) atomicOr(&g_ep_status, 2u);
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(32u) : "memory");
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
    // table geometry from the host's ep_info, never from the device copy of the directory
    int32_t tmin[EP_NUM_TABLES];
    uint16_t tK[EP_NUM_TABLES];
    uint32_t foff[EP_NUM_TABLES]; // start of table t's frequencies, in u16 units
    // two-level tables of a 2^12-slot stream (ep_build_tables12_kernel only)
    uint16_t *image;              // 16 x 4096 slots: twice the coordinate code
    uint32_t *hot;                // 16 x kHotSpan entries: the codes hs .. hs + kHotSpan - 1
    uint32_t *cold;               // 16 x kColdCodes entries: every code
    int32_t zlo;                  // coordinate value of code 0 (even)
    uint32_t hs;                  // first code of the hot window
};

struct GBatchParams {
    GJobParams job[EP_MAX_BATCH];
    int32_t n_jobs;
};

constexpr int kGThreads = 256;
constexpr int kGWarps = kGThreads / 32;

// one CTA per (table, job): exclusive prefix sums of the frequencies in shared memory (as u16; the last
// entry 2^b <= 32768 still fits), then every slot finds its symbol by binary search.  A table without symbols
// (or whose frequencies fall short of 2^b in a damaged stream) gets index 0 with offset 0 in the slots nobody owns.
__global__ void __launch_bounds__(1024) ep_build_tables_kernel(const __grid_constant__ GBatchParams P) {
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ uint32_t part[1024];
    const GJobParams &J = P.job[blockIdx.y];
    const uint32_t t = blockIdx.x, tid = threadIdx.x;
    const uint32_t K = J.tK[t];
    const uint32_t M = 1u << J.b;
    uint32_t *lut = J.lut + (size_t(t) << J.b);
    if (K == 0) {
        for (uint32_t u = tid; u < M; u += blockDim.x) lut[u] = 0u;
        return;
    }
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(J.stream + J.off_tables + 8 * EP_NUM_TABLES) + J.foff[t];
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
        F[K] = uint16_t(min(run, M));                                // = 2^b for a valid stream
    }
    __syncthreads();
    uint32_t run = part[tid];
    for (uint32_t j = j0; j < j1; ++j) { F[j] = uint16_t(min(run, M)); run += fq[j]; }
    __syncthreads();
    for (uint32_t u = tid; u < M; u += blockDim.x) {
        uint32_t lo = 0, hi = K;                                     // largest j with F[j] <= u (F[0] = 0)
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (uint32_t(F[mid]) <= u) lo = mid; else hi = mid;
        }
        lut[u] = (lo << 16) | ((u - uint32_t(F[lo])) & 0xFFFFu);     // lo < K <= 65535
    }
}

// Two-level tables of a 2^12-slot stream (see EP_N1): one CTA per (coordinate table, job).  Prefix sums of the
// frequencies as above; then every code of the coordinate range gets its entry f << 16 | F in the complete array -
// and in the hot part, if it lies in the window of kHotSpan codes that the decode kernel keeps in shared memory -,
// and every slot finds its symbol by binary search and stores twice the symbol's code.  A code no symbol of the
// table has, and a symbol that never occurs, get f = 1 (they own no slot; the floor only keeps a damaged stream
// from producing states that take a word in every step).
__global__ void __launch_bounds__(1024) ep_build_tables12_kernel(const __grid_constant__ GBatchParams P) {
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ uint32_t part[1024];
    const GJobParams &J = P.job[blockIdx.y];
    const uint32_t t = blockIdx.x + 1u, tid = threadIdx.x;
    const uint32_t K = J.tK[t];
    constexpr uint32_t M = 4096;
    uint16_t *image = J.image + size_t(t - 1u) * M;
    uint32_t *hot = J.hot + (t - 1u) * kHotSpan;
    uint32_t *cold = J.cold + (t - 1u) * kColdCodes;
    const uint32_t unused = 1u << 16;                                 // f = 1, F = 0
    const bool is_m = ((t - 1u) & 7u) == 7u;                          // the m field: its coordinate is 2m (+ parity)
    if (K == 0) {
        for (uint32_t c = tid; c < kColdCodes; c += blockDim.x) cold[c] = unused;
        for (uint32_t c = tid; c < kHotSpan; c += blockDim.x) hot[c] = unused;
        for (uint32_t u = tid; u < M; u += blockDim.x) image[u] = 0;  // never looked up in a valid stream
        return;
    }
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(J.stream + J.off_tables + 8 * EP_NUM_TABLES) + J.foff[t];
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
        F[K] = uint16_t(min(run, M));
    }
    __syncthreads();
    uint32_t run = part[tid];
    for (uint32_t j = j0; j < j1; ++j) { F[j] = uint16_t(min(run, M)); run += fq[j]; }
    __syncthreads();
    for (uint32_t c = tid; c < kColdCodes; c += blockDim.x) {
        const int32_t z = int32_t(c) + J.zlo;                         // the coordinate value of this code
        const int32_t j = (is_m ? (z >> 1) : z) - J.tmin[t];          // (z even for the m field: the shift is exact)
        uint32_t e = unused;
        if (!(is_m && (z & 1)) && j >= 0 && uint32_t(j) < K)
            e = (min(max(uint32_t(fq[j]), 1u), M) << 16) | min(uint32_t(F[j]), M - 1u);
        cold[c] = e;
        if (c - J.hs < kHotSpan) hot[c - J.hs] = e;                   // (unsigned: a code below the window wraps)
    }
    for (uint32_t u = tid; u < M; u += blockDim.x) {
        uint32_t lo = 0, hi = K;                                     // largest j with F[j] <= u (F[0] = 0)
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (uint32_t(F[mid]) <= u) lo = mid; else hi = mid;
        }
        const int32_t z = J.tmin[t] + int32_t(lo);
        const int32_t code = (is_m ? 2 * z : z) - J.zlo;
        image[u] = uint16_t(2 * min(max(code, 0), int32_t(kColdCodes) - 1));
    }
}

// one symbol: returns its index inside table t's symbol range (0 for an idle lane); Kmax = the table's last index
__device__ __forceinline__ uint32_t grans_step(uint32_t &x, const uint32_t *table, const uint16_t *freq, uint32_t Kmax,
                                               uint32_t mask, uint32_t b, uint32_t &ptr, const uint16_t *pay, uint32_t lt,
                                               bool act, uint32_t last_word) {
    uint32_t sym = 0;
    bool need = false;
    if (act) {
        const uint32_t e = __ldg(table + (x & mask));
        sym = min(e >> 16, Kmax);                 // whatever the scratch holds, stay inside the frequency array
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
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    int j = 0;
    while (j + 1 < P.n_jobs && blockIdx.x >= P.job[j + 1].cta_begin) ++j;
    const GJobParams &J = P.job[j];
    const uint16_t *fq = reinterpret_cast<const uint16_t *>(J.stream + J.off_tables + 8 * EP_NUM_TABLES);
    const uint32_t b = J.b, mask = (1u << b) - 1u, lt = (1u << lane) - 1u;
    const uint16_t *pay = reinterpret_cast<const uint16_t *>(J.stream + J.off_payload);
    const uint32_t last_word = J.total_words ? J.total_words - 1u : 0u;
    const uint32_t cta = blockIdx.x - J.cta_begin;
    const uint32_t K0max = J.tK[0] ? J.tK[0] - 1u : 0u;
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
            fld[0] = int32_t(grans_step(x, J.lut, fq + J.foff[0], K0max, mask, b, ptr, pay, lt, act, last_word)) + J.tmin[0];
            const uint32_t t0 = 1u + 8u * uint32_t(fld[0] & 1);          // first coordinate table of this coset
#pragma unroll
            for (uint32_t k = 0; k < 8; ++k) {
                const uint32_t t = t0 + k;
                const uint32_t Kt = J.tK[t];
                fld[k + 1] = int32_t(grans_step(x, J.lut + (size_t(t) << b), fq + J.foff[t], Kt ? Kt - 1u : 0u, mask, b, ptr, pay,
                                                lt, act && Kt != 0u, last_word)) + J.tmin[t];
            }
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

// a prepared image of the sixteen shared-memory tables in global memory (ep_prepare_tables): warp w of the
// job's CTA builds table w + 1 with the routine the decode kernel uses on shared memory
__global__ void __launch_bounds__(512) ep_prepare_tables_kernel(const __grid_constant__ JobParams J, uint32_t *image) {
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t t = 1u + warp;
    if (t >= EP_NUM_TABLES) return;
    uint32_t *dst = image + (t - 1u) * kLutEntries;
    build_one_table(J, t, lane, [dst](uint32_t slot, uint32_t e) { dst[slot] = e; });
    // b < 11: the slots above 2^b are never read, but the image is copied whole
    for (uint32_t u = (1u << J.b) + lane; u < kLutEntries; u += 32) dst[u] = kEntryUnused;
}

// ---- host side -----------------------------------------------------------------------------------

// the tiles a job asks for: its range, or the whole tensor when both range fields are 0
inline uint32_t job_tile0(const ep_decode_job &jb) { return jb.tile_count ? jb.tile_begin : 0u; }
inline uint32_t job_tiles(const ep_decode_job &jb) { return jb.tile_count ? jb.tile_count : jb.info->n_tiles; }

int g_num_sms[64] = {};

int num_sms() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && g_num_sms[dev]) return g_num_sms[dev];
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64) g_num_sms[dev] = n;
    return n;
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
    if (zlo < -1024) return false;                    // 4096 - zlo stays below 8192: same fp32 exponent as 4096 + code
    for (int t = 1; t < EP_NUM_TABLES; ++t) {         // (the coset table is decoded by comparison: any frequency goes)
        if (I.table_K[t] > kLutEntries) return false;
        if (I.b == 11 && I.table_K[t] == 1) return false;   // a lone symbol has f = 2^11: one bit more than the f field
    }
    return true;
}

// table geometry of a job whose tables fit shared memory
void fill_table_params(JobParams &J, const ep_info &I) {
    J.off_freq = I.off_tables + 8u * EP_NUM_TABLES;
    J.b = I.b;
    J.zlo = int32_t(even_base(coord_range(I)));
    uint32_t acc = 0;
    for (int t = 0; t < EP_NUM_TABLES; ++t) {
        J.tmin[t] = int16_t(I.table_min[t]);
        J.tK[t] = uint16_t(I.table_K[t]);
        J.foff[t] = uint16_t(acc);
        acc += I.table_K[t];
    }
}

template <int DT>
cudaError_t launch_smem(const BatchParams &P, uint32_t grid, cudaStream_t st) {
    static bool configured[64] = {};   // the attribute is per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(ep_decode_smem_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemBytes));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    ep_decode_smem_kernel<DT><<<grid, kThreads, kSmemBytes, st>>>(P);
    return cudaGetLastError();
}

size_t large_table_bytes(const ep_info &I) { return size_t(EP_NUM_TABLES) * (size_t(1) << I.b) * 4u; }

// 2^12-slot streams whose coordinates span at most kColdCodes values decode from two-level tables in the hot loop
bool fits_two_level(const ep_info &I) {
    if (!kTwoLevelInLoop || I.b != 12) return false;
    const Range r = coord_range(I);
    const int64_t zlo = even_base(r);
    return r.any && r.hi - zlo < int64_t(kColdCodes) && zlo >= -(int64_t(1) << 20);   // 2^22 - zlo and 2^22 + code: one exponent
}
// first code of the hot window: kHotSpan codes centred on the coordinate value 0, kept inside the code range
uint32_t hot_start(const ep_info &I) {
    const Range r = coord_range(I);
    const int64_t zlo = even_base(r), codes = (r.any ? r.hi : 0) - zlo + 1;
    const int64_t last = codes > int64_t(kHotSpan) ? codes - int64_t(kHotSpan) : 0;
    int64_t hs = -zlo - int64_t(kHotSpan / 2);
    if (hs < 0) hs = 0;
    return uint32_t(hs < last ? hs : last);
}
// image, hot part, complete array; the flat tables of the large-table kernel follow at this offset
size_t two_level_bytes(const ep_info &) { return size_t(kLutBytes) + kHotBytes + kColdBytes; }
// can the hot loop serve this request?  (the field dump and narrow tensors take the plain kernels)
bool hot_loop_shape(const ep_info &I, int32_t dt) { return dt != EP_FIELDS_I32 && I.C / 8 >= 32u && I.V < (1u << 20); }

// the host-side parameters of a large-table job (geometry from `info` only); `lut` = where its tables are or go
int fill_large_job(GJobParams &J, const ep_decode_job &jb, uint32_t *lut) {
    const ep_info &I = *jb.info;
    uint32_t acc = 0;
    for (int t = 0; t < EP_NUM_TABLES; ++t) {
        if (I.table_K[t] > 65535u) return EP_ERR_UNSUPPORTED;
        J.tmin[t] = I.table_min[t];
        J.tK[t] = uint16_t(I.table_K[t]);
        J.foff[t] = acc;
        acc += I.table_K[t];
    }
    J.stream = static_cast<const uint8_t *>(jb.d_stream);
    J.tile_index = static_cast<const uint32_t *>(jb.d_tile_index);
    J.scales = jb.d_row_scales;
    J.out = jb.d_out;
    J.lut = lut;
    J.off_tables = I.off_tables;
    J.off_payload = I.off_payload;
    J.total_words = uint32_t(I.total_words);
    J.n_vec = uint32_t(uint64_t(I.R) * (I.C / 8));
    J.per_row = I.C / 8;
    J.V = I.V;
    J.n_tiles = I.n_tiles;
    J.b = I.b;
    return EP_OK;
}

// where the two-level tables of a job live inside its table buffer
void set_two_level(GJobParams &J, const ep_info &I, void *base) {
    J.image = static_cast<uint16_t *>(base);
    J.hot = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(base) + kLutBytes);
    J.cold = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(base) + kLutBytes + kHotBytes);
    J.zlo = int32_t(even_base(coord_range(I)));
    J.hs = hot_start(I);
}

cudaError_t launch_build12(const GBatchParams &P, int n_jobs, cudaStream_t st) {
    uint32_t max_K = 1;
    for (int i = 0; i < n_jobs; ++i)
        for (int t = 1; t < EP_NUM_TABLES; ++t)
            if (P.job[i].tK[t] > max_K) max_K = P.job[i].tK[t];
    const size_t smem = 2u * (size_t(max_K) + 1u);
    if (smem > 48u * 1024u) {
        const cudaError_t e = cudaFuncSetAttribute(ep_build_tables12_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
    }
    ep_build_tables12_kernel<<<dim3(EP_NUM_TABLES - 1, n_jobs), 1024, smem, st>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_build(const GBatchParams &P, int n_jobs, cudaStream_t st) {
    uint32_t max_K = 1;
    for (int i = 0; i < n_jobs; ++i)
        for (int t = 0; t < EP_NUM_TABLES; ++t)
            if (P.job[i].tK[t] > max_K) max_K = P.job[i].tK[t];
    const size_t smem = 2u * (size_t(max_K) + 1u);
    if (smem > 48u * 1024u) {
        const cudaError_t e = cudaFuncSetAttribute(ep_build_tables_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
    }
    ep_build_tables_kernel<<<dim3(EP_NUM_TABLES, n_jobs), 1024, smem, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

extern "C" size_t ep_decode_scratch_bytes(const ep_info *info) {
    if (!info) return 0;
    if (fits_smem_tables(*info)) return 0;
    return (fits_two_level(*info) ? two_level_bytes(*info) : 0) + large_table_bytes(*info);
}

extern "C" size_t ep_decode_tables_bytes(const ep_info *info) {
    if (!info) return 0;
    return fits_smem_tables(*info) ? size_t(kLutBytes) : ep_decode_scratch_bytes(info);
}

extern "C" uint32_t ep_decode_tiles_per_sm(void) { return kTilesPerRound; }

extern "C" int ep_prepare_tables(const ep_info *info, const void *d_stream, void *d_tables, size_t tables_bytes, void *stream) {
    if (!info || !d_stream || !d_tables) return EP_ERR_BAD_ARG;
    const ep_info &I = *info;
    if (I.b < 9 || I.b > 15 || (reinterpret_cast<uintptr_t>(d_stream) & 3)) return EP_ERR_BAD_ARG;
    if (tables_bytes < ep_decode_tables_bytes(info) || (reinterpret_cast<uintptr_t>(d_tables) & 255)) return EP_ERR_SCRATCH;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (fits_smem_tables(I)) {
        JobParams J;
        std::memset(&J, 0, sizeof(J));
        J.stream = static_cast<const uint8_t *>(d_stream);
        fill_table_params(J, I);
        ep_prepare_tables_kernel<<<1, 512, 0, st>>>(J, static_cast<uint32_t *>(d_tables));
        return cudaGetLastError() == cudaSuccess ? EP_OK : EP_ERR_CUDA;
    }
    GBatchParams P;
    std::memset(&P, 0, sizeof(P));
    P.n_jobs = 1;
    ep_decode_job jb;
    std::memset(&jb, 0, sizeof(jb));
    jb.info = info;
    jb.d_stream = d_stream;
    // a 2^12-slot stream gets the two-level tables of the hot loop first, then the flat tables the plain kernel
    // uses for the field dump and for narrow tensors
    uint8_t *base = static_cast<uint8_t *>(d_tables);
    const bool two = fits_two_level(I);
    const int rc = fill_large_job(P.job[0], jb, reinterpret_cast<uint32_t *>(base + (two ? two_level_bytes(I) : 0)));
    if (rc) return rc;
    if (two) {
        set_two_level(P.job[0], I, base);
        if (launch_build12(P, 1, st) != cudaSuccess) return EP_ERR_CUDA;
    }
    return launch_build(P, 1, st) == cudaSuccess ? EP_OK : EP_ERR_CUDA;
}

namespace {

template <int DT>
cudaError_t launch_glut(const GBatchParams &P, uint32_t grid, cudaStream_t st) {
    ep_decode_glut_kernel<DT><<<grid, kGThreads, 0, st>>>(P);
    return cudaGetLastError();
}

// jobs whose tables do not fit shared memory: decode from tables in global memory - the caller's prepared
// ones, or tables built into the caller's scratch by one extra launch first
int decode_large_tables(const ep_decode_job *const *jobs, int n_jobs, int32_t dt, int sms, cudaStream_t st) {
    GBatchParams P, B;      // B: the jobs whose tables have to be built
    std::memset(&P, 0, sizeof(P));
    std::memset(&B, 0, sizeof(B));
    P.n_jobs = n_jobs;
    uint32_t next = 0;
    int n_build = 0;
    for (int i = 0; i < n_jobs; ++i) {
        const ep_decode_job &jb = *jobs[i];
        const ep_info &I = *jb.info;
        // the flat tables follow the two-level ones where the buffer has both (prepared tables always, scratch
        // if it is large enough); a scratch buffer of the flat tables' size alone holds just them
        const size_t need = large_table_bytes(I), before = fits_two_level(I) ? two_level_bytes(I) : 0;
        uint32_t *lut;
        if (jb.d_tables) {
            if (reinterpret_cast<uintptr_t>(jb.d_tables) & 255) return EP_ERR_SCRATCH;
            lut = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(const_cast<void *>(jb.d_tables)) + before);
        } else {
            if (!jb.d_scratch || jb.scratch_bytes < need || (reinterpret_cast<uintptr_t>(jb.d_scratch) & 255)) return EP_ERR_SCRATCH;
            lut = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(jb.d_scratch) + (jb.scratch_bytes >= before + need ? before : 0));
        }
        GJobParams &J = P.job[i];
        const int rc = fill_large_job(J, jb, lut);
        if (rc) return rc;
        J.tile0 = job_tile0(jb);
        J.tile_cnt = job_tiles(jb);
        const uint64_t want = (uint64_t(J.tile_cnt) + kGWarps - 1) / kGWarps;
        const uint64_t cap = uint64_t(sms) * 8u;
        J.cta_begin = next;
        J.cta_count = uint32_t(want < cap ? want : cap);
        next += J.cta_count;
        if (!jb.d_tables) B.job[n_build++] = J;
    }
    if (n_build) {
        B.n_jobs = n_build;
        if (launch_build(B, n_build, st) != cudaSuccess) return EP_ERR_CUDA;
    }
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
        else if (fits_two_level(I) && hot_loop_shape(I, dt) &&
                 (jb.d_tables || (jb.d_scratch && jb.scratch_bytes >= two_level_bytes(I)))) { fast[n_jobs++] = &jb; }
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
    GBatchParams B12;               // two-level tables that have to be built into scratch first
    std::memset(&B12, 0, sizeof(B12));
    int n_build12 = 0;
    // persistent CTAs, one per SM (fewer if the launch has fewer rounds than SMs); the kernel splits the
    // cost-weighted list of all rounds evenly over them
    uint64_t rounds_total = 0, cost = 0;
    for (int i = 0; i < n_jobs; ++i) {
        const ep_decode_job &jb = *fast[i];
        const ep_info &I = *jb.info;
        JobParams &J = P.job[i];
        const uint32_t my_tiles = job_tiles(jb);
        if (jb.d_tables && (reinterpret_cast<uintptr_t>(jb.d_tables) & 255)) return EP_ERR_SCRATCH;
        J.stream = static_cast<const uint8_t *>(jb.d_stream);
        J.tile_index = static_cast<const uint32_t *>(jb.d_tile_index);
        J.scales = jb.d_row_scales;
        J.out = jb.d_out;
        J.lut_image = static_cast<const uint32_t *>(jb.d_tables);
        if (I.b == 12) {            // two-level tables: prepared, or built into the caller's scratch by a launch before this one
            void *base = const_cast<void *>(jb.d_tables);
            if (!base) {
                if (reinterpret_cast<uintptr_t>(jb.d_scratch) & 255) return EP_ERR_SCRATCH;
                base = jb.d_scratch;
                GJobParams &G = B12.job[n_build12++];
                const int rc = fill_large_job(G, jb, nullptr);
                if (rc) return rc;
                set_two_level(G, I, base);
            }
            J.lut_image = static_cast<const uint32_t *>(base);
            J.cold = reinterpret_cast<const uint32_t *>(static_cast<const uint8_t *>(base) + kLutBytes + kHotBytes);
            J.hs2 = 2u * hot_start(I);
        }
        J.off_payload = I.off_payload;
        J.total_words = uint32_t(I.total_words);
        J.n_vec = uint32_t(uint64_t(I.R) * (I.C / 8));
        J.per_row = I.C / 8;
        J.V = I.V;
        J.n_tiles = I.n_tiles;
        J.tile0 = job_tile0(jb);
        J.tile_cnt = my_tiles;
        fill_table_params(J, I);
        const uint32_t block_bytes = dt == EP_FIELDS_I32 ? 36u : dt == EP_FP32 ? 32u : (dt == EP_BF16 || dt == EP_FP16) ? 16u : 8u;
        J.row_bytes = J.per_row * block_bytes;
        J.row_rcp = uint32_t(0xFFFFFFFFu / J.row_bytes + 1u);
        J.row_max = I.R - 1u;
        J.rounds = (my_tiles + kTilesPerRound - 1u) / kTilesPerRound;
        J.round_cost = (I.V + 31u) / 32u;
        J.cost_begin = uint32_t(cost);
        cost += uint64_t(J.rounds) * J.round_cost;
        rounds_total += J.rounds;
    }
    if (n_build12) {
        B12.n_jobs = n_build12;
        if (launch_build12(B12, n_build12, st) != cudaSuccess) return EP_ERR_CUDA;
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

namespace {
ep_decode_job one_job(const ep_info *info, const void *d_stream, const void *d_tile_index, const float *d_row_scales,
                      int32_t out_dtype, void *d_out, void *d_scratch, size_t scratch_bytes) {
    ep_decode_job jb;
    std::memset(&jb, 0, sizeof(jb));
    jb.info = info;
    jb.d_stream = d_stream;
    jb.d_tile_index = d_tile_index;
    jb.d_row_scales = d_row_scales;
    jb.out_dtype = out_dtype;
    jb.d_out = d_out;
    jb.d_scratch = d_scratch;
    jb.scratch_bytes = scratch_bytes;
    return jb;
}
}  // namespace

extern "C" int ep_decode_tiles(const ep_info *info, const void *d_stream, const void *d_tile_index,
                               const float *d_row_scales, int32_t out_dtype, void *d_out, void *d_scratch,
                               size_t scratch_bytes, uint32_t tile_begin, uint32_t tile_count, void *stream) {
    if (tile_count == 0) return EP_ERR_BAD_ARG;
    ep_decode_job jb = one_job(info, d_stream, d_tile_index, d_row_scales, out_dtype, d_out, d_scratch, scratch_bytes);
    jb.tile_begin = tile_begin;
    jb.tile_count = tile_count;
    return ep_decode_batch(&jb, 1, stream);
}

extern "C" int ep_decode_tensor(const ep_info *info, const void *d_stream, const void *d_tile_index,
                                const float *d_row_scales, int32_t out_dtype, void *d_out, void *d_scratch,
                                size_t scratch_bytes, void *stream) {
    const ep_decode_job jb = one_job(info, d_stream, d_tile_index, d_row_scales, out_dtype, d_out, d_scratch, scratch_bytes);
    return ep_decode_batch(&jb, 1, stream);
}

namespace {
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                   const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
}

extern "C" int ep_decode_gemm(const ep_info *info, const void *d_stream, const void *d_tile_index, const float *d_row_scales,
                              const void *d_tables, const void *d_x, uint32_t T, float *d_y, void *stream) {
    if (!info || !d_stream || !d_tile_index || !d_row_scales || !d_tables || !d_x || !d_y || T == 0) return EP_ERR_BAD_ARG;
    const ep_info &I = *info;
    if (I.C == 0 || I.C % 8 || I.R == 0 || I.V == 0 || I.b < 9 || I.b > 15 || I.J != ep::kStates) return EP_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_stream) & 3) || (reinterpret_cast<uintptr_t>(d_tile_index) & 3) ||
        (reinterpret_cast<uintptr_t>(d_x) & 15) || (reinterpret_cast<uintptr_t>(d_y) & 15))
        return EP_ERR_BAD_ARG;
    if (reinterpret_cast<uintptr_t>(d_tables) & 255) return EP_ERR_SCRATCH;
    if (I.table_K[0] == 0 || I.table_min[0] < 0 || int64_t(I.table_min[0]) + I.table_K[0] > 2) return EP_ERR_BAD_STREAM;
    // one tile per row, whole groups per row, 32 rows per CTA, tables in shared memory, 32 warps of one tile each
    if (kChains != 1 || kWarps != 32 || I.b != 11 || !fits_smem_tables(I) || I.V != I.C / 8 || I.C % 256 || T > 32 ||
        I.total_words >= (1ull << 30) || uint64_t(I.R) * I.C >= (1ull << 32))
        return EP_ERR_UNSUPPORTED;
    const int sms = num_sms();
    if (sms <= 0) return EP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GemmParams P;
    std::memset(&P, 0, sizeof(P));
    JobParams &J = P.J;
    J.stream = static_cast<const uint8_t *>(d_stream);
    J.tile_index = static_cast<const uint32_t *>(d_tile_index);
    J.scales = d_row_scales;
    J.lut_image = static_cast<const uint32_t *>(d_tables);
    J.off_payload = I.off_payload;
    J.total_words = uint32_t(I.total_words);
    J.n_vec = uint32_t(uint64_t(I.R) * (I.C / 8));
    J.per_row = I.C / 8;
    J.V = I.V;
    J.n_tiles = I.n_tiles;
    J.tile_cnt = I.n_tiles;
    J.row_max = I.R - 1u;
    fill_table_params(J, I);
    P.x = static_cast<const uint16_t *>(d_x);
    P.y = d_y;
    P.T = T;
    P.Tpad = T <= 16 ? 16u : 32u;
    P.R = I.R;
    P.C = I.C;
    // rows spread evenly over the SMs (a CTA takes its range 31 rows at a time; the last, shorter step runs with fewer
    // warps and ends sooner than a full one)
    P.rows_per_cta = (I.R + uint32_t(sms) - 1u) / uint32_t(sms);
    P.groups = I.C / 256u;
    if (I.n_tiles != I.R) return EP_ERR_BAD_ARG;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EP_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        if (cudaFuncSetAttribute(ep_decode_gemm_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmem)) != cudaSuccess ||
            cudaFuncSetAttribute(ep_decode_gemm_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmem)) != cudaSuccess)
            return EP_ERR_CUDA;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const uint32_t grid = (I.R + P.rows_per_cta - 1u) / P.rows_per_cta;
    // x as a two-dimensional tensor for the copy engine: boxes of 64 columns (128 bytes, the swizzle span) x Tpad rows
    static EncodeTiledFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
            qres != cudaDriverEntryPointSuccess)
            return EP_ERR_CUDA;
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    CUtensorMap x_map;
    const cuuint64_t dims[2] = {I.C, T}, strides[1] = {cuuint64_t(I.C) * 2u};
    const cuuint32_t box[2] = {64u, P.Tpad}, estr[2] = {1u, 1u};
    if (encode(&x_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(d_x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return EP_ERR_CUDA;
    if (P.Tpad == 16u) ep_decode_gemm_kernel<16><<<grid, kThreads, kGemmSmem, st>>>(P, x_map);
    else ep_decode_gemm_kernel<32><<<grid, kThreads, kGemmSmem, st>>>(P, x_map);
    return cudaGetLastError() == cudaSuccess ? EP_OK : EP_ERR_CUDA;
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
