// CUDA back end of the EntroPack encoder (paper Sec. 3.2-3.6): row RMS, E8 quantisation with field
// histograms, row-scale refit and tiled 32-state rANS encoding run on the GPU; the few-kilobyte steps
// (frequency normalisation, C_CE, the stored-size estimate, the bisection itself) stay on the host and
// are shared with the host back end, so both produce the same bytes for the same input.
//
// Every floating-point step uses the same operations in the same order as the host code: IEEE
// single-precision division and subtraction, round-to-nearest-even, double-precision sums in index
// order written with explicit add / multiply intrinsics so that nothing is fused.
#include <cuda_runtime.h>

#include <mutex>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "encoder_core.hpp"

namespace ep {
int check_encode_args(uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts &o);
}

namespace {

using namespace ep;

constexpr int kHistBins = 8192;          // per table, values -4096 .. 4095
constexpr int kHistOrigin = -4096;
constexpr int kLocalBins = 512;          // shared-memory window per table, values -256 .. 255
constexpr int kLocalOrigin = -256;
constexpr uint32_t kMaxTableSymbols = 40960;   // sum of K over the 17 tables that the tile encoder keeps in shared memory

// ---- rows whose sums run in index order ---------------------------------------------------------------
// The row RMS (Sec. 3.2) and the refit of Eq. 13 sum over a row in double precision in index order, as the host code
// does: one serial chain of additions per row, which no reduction tree reproduces bit for bit.  One thread per row
// reading its own row leaves the GPU waiting for memory (8192 rows = 256 warps with a few KB in flight each: 0.29 ms
// for the RMS of an 8192 x 8192 tensor).  So a CTA takes kRowsPerCta rows: all its threads stream the rows through
// shared memory with cp.async, kRowStages chunks ahead, and kRowsPerCta lanes of its first warp run the chains.
constexpr uint32_t kRowsPerCta = 8, kRowStages = 4, kRowThreads = 256;
constexpr uint32_t kRmsChunk = 256;                 // floats per row and chunk
constexpr uint32_t kRmsStride = kRmsChunk + 4;      // padded: the eight lanes read different banks

__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(uint32_t(__cvta_generic_to_shared(smem_dst))), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit_group() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__global__ void __launch_bounds__(kRowThreads) row_rms_kernel(const float *__restrict__ W, uint32_t R, uint32_t C, float *__restrict__ mu) {
    __shared__ __align__(16) float buf[kRowStages][kRowsPerCta][kRmsStride];
    const uint32_t tid = threadIdx.x, row0 = blockIdx.x * kRowsPerCta;
    const uint32_t chunks = (C + kRmsChunk - 1) / kRmsChunk;
    // chunk c of the CTA's rows: kRowsPerCta x 64 pieces of 16 bytes, two per thread (rows start 16-byte aligned: C % 8 == 0)
    auto issue = [&](uint32_t c) {
        if (c < chunks) {
            for (uint32_t i = tid; i < kRowsPerCta * (kRmsChunk / 4); i += kRowThreads) {
                const uint32_t r = i / (kRmsChunk / 4), j = i % (kRmsChunk / 4), col = c * kRmsChunk + 4 * j;
                if (row0 + r < R && col < C) cp_async_16(&buf[c % kRowStages][r][4 * j], W + size_t(row0 + r) * C + col);
            }
        }
        cp_async_commit_group();
    };
    for (uint32_t c = 0; c + 1 < kRowStages; ++c) issue(c);
    double acc = 0.0;
    for (uint32_t c = 0; c < chunks; ++c) {
        issue(c + kRowStages - 1);
        cp_async_wait_group<kRowStages - 1>();
        __syncthreads();
        if (tid < kRowsPerCta && row0 + tid < R) {
            const uint32_t n4 = (min(kRmsChunk, C - c * kRmsChunk)) / 4;
            const float4 *x = reinterpret_cast<const float4 *>(&buf[c % kRowStages][tid][0]);
            for (uint32_t j = 0; j < n4; ++j) {
                const float4 v = x[j];
                acc = __dadd_rn(acc, __dmul_rn(double(v.x), double(v.x)));
                acc = __dadd_rn(acc, __dmul_rn(double(v.y), double(v.y)));
                acc = __dadd_rn(acc, __dmul_rn(double(v.z), double(v.z)));
                acc = __dadd_rn(acc, __dmul_rn(double(v.w), double(v.w)));
            }
        }
        __syncthreads();                     // the stage may be overwritten by the next issue
    }
    if (tid < kRowsPerCta && row0 + tid < R) {
        double m = __dsqrt_rn(__ddiv_rn(acc, double(C)));
        if (!(m > 1e-12)) m = 1e-12;
        mu[row0 + tid] = __double2float_rn(m);
    }
}

// Eq. 3 on one 8-vector: integer point and fp32 residuals of that point
struct D8 {
    int32_t z[8];
    float res[8];
};
__device__ __forceinline__ void nearest_d8(const float *y, D8 &o) {
    int32_t sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float f = rintf(y[i]);                 // ties to even
        o.z[i] = int32_t(f);
        o.res[i] = __fsub_rn(y[i], f);
        sum += o.z[i];
    }
    if (sum & 1) {
        int at = 0;
        float big = fabsf(o.res[0]);
#pragma unroll
        for (int i = 1; i < 8; ++i) {
            const float a = fabsf(o.res[i]);
            if (a > big) { big = a; at = i; }        // first coordinate of largest residual
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i == at) {
                o.z[i] += (o.res[i] >= 0.0f) ? 1 : -1;   // sign(0) = +1
                o.res[i] = __fsub_rn(y[i], float(o.z[i]));
            }
    }
}

// Eq. 2 + Eq. 4 on one block of eight weights; returns false if a coordinate leaves the histogram range
__device__ __forceinline__ bool quantise_block(const float *x, float mu, float s, int32_t *fld) {
    float y[8], yh[8];
    bool ok = true;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        y[i] = __fdiv_rn(__fdiv_rn(x[i], mu), s);
        yh[i] = __fsub_rn(y[i], 0.5f);
        ok = ok && (fabsf(y[i]) < 4000.0f);
    }
    if (!ok) return false;
    D8 a, h;
    nearest_d8(y, a);
    nearest_d8(yh, h);
    double da = 0.0, dh = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        da = __dadd_rn(da, __dmul_rn(double(a.res[i]), double(a.res[i])));
        dh = __dadd_rn(dh, __dmul_rn(double(h.res[i]), double(h.res[i])));
    }
    const bool half = dh < da;                       // the half coset only when strictly closer
    fld[0] = half ? 1 : 0;
    int32_t s7 = 0;
#pragma unroll
    for (int i = 0; i < 7; ++i) {
        fld[1 + i] = half ? h.z[i] : a.z[i];
        s7 += fld[1 + i];
    }
    const int32_t z8 = half ? h.z[7] : a.z[7];
    fld[8] = (z8 - (s7 & 1)) >> 1;
    return true;
}

// Quantise blocks of the listed rows (rows == nullptr: all rows) at scale s; store the fields (fields != nullptr)
// and count them: a shared-memory window per CTA for values near zero, global atomics for the rest.
__global__ void __launch_bounds__(256) quantise_count_kernel(const float *__restrict__ W, uint32_t C, const float *__restrict__ mu,
                                                             const uint32_t *__restrict__ rows, uint64_t n_blocks8, float s,
                                                             int16_t *__restrict__ fields, uint32_t *__restrict__ hist,
                                                             int *__restrict__ overflow) {
    __shared__ uint32_t local[EP_NUM_TABLES * kLocalBins];
    for (uint32_t i = threadIdx.x; i < EP_NUM_TABLES * kLocalBins; i += blockDim.x) local[i] = 0;
    __syncthreads();
    const uint32_t per_row = C / 8;
    for (uint64_t v = uint64_t(blockIdx.x) * blockDim.x + threadIdx.x; v < n_blocks8; v += uint64_t(gridDim.x) * blockDim.x) {
        const uint64_t i = v / per_row;
        const uint32_t col = uint32_t(v - i * per_row);
        const uint64_t r = rows ? rows[i] : i;
        const float4 *src = reinterpret_cast<const float4 *>(W + r * C + 8ull * col);
        const float4 lo = src[0], hi = src[1];
        const float x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        int32_t fld[9];
        if (!quantise_block(x, mu[r], s, fld)) { *overflow = 1; continue; }
        if (fields) {
#pragma unroll
            for (int k = 0; k < 9; ++k) fields[v * 9 + k] = int16_t(fld[k]);
        }
#pragma unroll
        for (int k = 0; k < 9; ++k) {
            const int t = k == 0 ? 0 : 1 + 8 * fld[0] + (k - 1);
            const int32_t val = fld[k];
            if (val >= kLocalOrigin && val < kLocalOrigin + kLocalBins) atomicAdd(&local[t * kLocalBins + (val - kLocalOrigin)], 1u);
            else if (val >= kHistOrigin && val < kHistOrigin + kHistBins) atomicAdd(&hist[t * kHistBins + (val - kHistOrigin)], 1u);
            else *overflow = 1;
        }
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < EP_NUM_TABLES * kLocalBins; i += blockDim.x) {
        const uint32_t c = local[i];
        if (c) {
            const uint32_t t = i / kLocalBins, j = i % kLocalBins;
            atomicAdd(&hist[t * kHistBins + (int(j) + kLocalOrigin - kHistOrigin)], c);
        }
    }
}

// Eq. 13: the two sums of a row in double in index order.  One block = 8 weights and its nine fields.
__device__ __forceinline__ void refit_block(const float *xv, const int16_t *qv, double &xp, double &pp) {
    const double half = 0.5 * double(qv[0]);
    int32_t s7 = 0;
#pragma unroll
    for (int j = 0; j < 7; ++j) {
        const double p = __dadd_rn(double(qv[1 + j]), half);
        xp = __dadd_rn(xp, __dmul_rn(double(xv[j]), p));
        pp = __dadd_rn(pp, __dmul_rn(p, p));
        s7 += qv[1 + j];
    }
    const double p8 = __dadd_rn(double(2 * qv[8] + (s7 & 1)), half);   // Eq. 5
    xp = __dadd_rn(xp, __dmul_rn(double(xv[7]), p8));
    pp = __dadd_rn(pp, __dmul_rn(p8, p8));
}
__device__ __forceinline__ float refit_result(double xp, double pp, float s, float mu) {
    double sg;
    if (pp > 0.0) {
        sg = __ddiv_rn(xp, pp);
        if (!(sg > 1e-12)) sg = 1e-12;
    } else {
        sg = __dmul_rn(double(s), double(mu));
    }
    return __double2float_rn(sg);
}

// rows streamed through shared memory (see row_rms_kernel); needs 16-byte aligned field rows: C a multiple of 64
constexpr uint32_t kRefitBlocks = 16;                              // blocks per row and chunk
constexpr uint32_t kRefitWStride = kRefitBlocks * 8 + 4;           // floats, padded
constexpr uint32_t kRefitQStride = kRefitBlocks * 9 + 8;           // int16, padded, a multiple of 8
__global__ void __launch_bounds__(kRowThreads) refit_kernel(const float *__restrict__ W, uint32_t R, uint32_t C,
                                                            const int16_t *__restrict__ fields, float s,
                                                            const float *__restrict__ mu, float *__restrict__ sigma) {
    __shared__ __align__(16) float wbuf[kRowStages][kRowsPerCta][kRefitWStride];
    __shared__ __align__(16) int16_t qbuf[kRowStages][kRowsPerCta][kRefitQStride];
    const uint32_t tid = threadIdx.x, row0 = blockIdx.x * kRowsPerCta, per_row = C / 8;
    const uint32_t chunks = (per_row + kRefitBlocks - 1) / kRefitBlocks;
    // chunk c of the CTA's rows: per row up to 32 pieces of weights and 18 of fields, 16 bytes each
    constexpr uint32_t kWPieces = kRefitBlocks * 2, kQPieces = kRefitBlocks * 18 / 16, kPieces = kWPieces + kQPieces;
    auto issue = [&](uint32_t c) {
        if (c < chunks) {
            const uint32_t nb = min(kRefitBlocks, per_row - c * kRefitBlocks);     // blocks in this chunk: 16, or 8 at a row's end
            for (uint32_t i = tid; i < kRowsPerCta * kPieces; i += kRowThreads) {
                const uint32_t r = i / kPieces, j = i % kPieces;
                if (row0 + r >= R) continue;
                if (j < kWPieces) {
                    if (j < 2 * nb) cp_async_16(&wbuf[c % kRowStages][r][4 * j], W + size_t(row0 + r) * C + size_t(c) * kRefitBlocks * 8 + 4 * j);
                } else {
                    const uint32_t k = j - kWPieces;
                    if (16 * k < 18 * nb)
                        cp_async_16(&qbuf[c % kRowStages][r][8 * k], fields + (size_t(row0 + r) * per_row + size_t(c) * kRefitBlocks) * 9 + 8 * k);
                }
            }
        }
        cp_async_commit_group();
    };
    for (uint32_t c = 0; c + 1 < kRowStages; ++c) issue(c);
    double xp = 0.0, pp = 0.0;
    for (uint32_t c = 0; c < chunks; ++c) {
        issue(c + kRowStages - 1);
        cp_async_wait_group<kRowStages - 1>();
        __syncthreads();
        if (tid < kRowsPerCta && row0 + tid < R) {
            const uint32_t nb = min(kRefitBlocks, per_row - c * kRefitBlocks);
            const float *xw = &wbuf[c % kRowStages][tid][0];
            const int16_t *q = &qbuf[c % kRowStages][tid][0];
            for (uint32_t v = 0; v < nb; ++v) refit_block(xw + 8 * v, q + 9 * v, xp, pp);
        }
        __syncthreads();                     // the stage may be overwritten by the next issue
    }
    if (tid < kRowsPerCta && row0 + tid < R) sigma[row0 + tid] = refit_result(xp, pp, s, mu[row0 + tid]);
}

// the same for any C: one thread per row reading its own row
__global__ void refit_rows_kernel(const float *__restrict__ W, uint32_t R, uint32_t C, const int16_t *__restrict__ fields, float s,
                                  const float *__restrict__ mu, float *__restrict__ sigma) {
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= R) return;
    const uint32_t per_row = C / 8;
    const float *x = W + size_t(r) * C;
    const int16_t *q = fields + size_t(r) * per_row * 9;
    double xp = 0.0, pp = 0.0;
    for (uint32_t v = 0; v < per_row; ++v) {
        float xv[8];
        int16_t qv[9];
#pragma unroll
        for (int j = 0; j < 8; ++j) xv[j] = __ldg(x + 8 * v + j);
#pragma unroll
        for (int j = 0; j < 9; ++j) qv[j] = q[9 * v + j];
        refit_block(xv, qv, xp, pp);
    }
    sigma[r] = refit_result(xp, pp, s, mu[r]);
}

struct EncodeTables {
    int32_t tmin[EP_NUM_TABLES];
    uint32_t off[EP_NUM_TABLES];     // start of table t inside the (f, F) array
    uint32_t total;                  // sum of K
};

// Sec. 3.6 / App. "Tiled rANS implementation": one warp per tile, one state per lane.  The decoder reads,
// per (group, field), the words of the needy lanes in ascending lane order; the encoder walks groups and
// fields backwards and fills the tile's word area from its end, writing each step's words as one block in
// ascending lane order, which is the order the reversed word list of a sequential encoder would have.
__global__ void __launch_bounds__(256) tile_encode_kernel(const int16_t *__restrict__ fields, uint32_t n_vec, uint32_t V,
                                                          uint32_t n_tiles, uint32_t b, EncodeTables T,
                                                          const uint32_t *__restrict__ fF, uint16_t *__restrict__ scratch,
                                                          uint32_t cap, uint32_t *__restrict__ states,
                                                          uint32_t *__restrict__ counts) {
    extern __shared__ uint32_t tab[];    // per symbol: f | F << 16
    for (uint32_t i = threadIdx.x; i < T.total; i += blockDim.x) tab[i] = fF[i];
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t tile = blockIdx.x * (blockDim.x >> 5) + warp;
    if (tile >= n_tiles) return;
    const uint32_t v0 = tile * V;
    const uint32_t nv = min(V, n_vec - v0);
    const uint32_t lt = (1u << lane) - 1u;
    uint16_t *area = scratch + size_t(tile) * cap;
    uint32_t end = cap;                  // words [end, cap) of the area are written
    uint32_t x = kStateLow;
    const uint32_t groups = (nv + 31u) >> 5;
    for (uint32_t g = groups; g-- > 0;) {
        const uint32_t i = g * 32u + lane;
        const bool act = i < nv;
        const int16_t *q = fields + size_t(v0 + (act ? i : 0u)) * 9u;
        const int c = act ? int(q[0]) : 0;
        for (int k = 8; k >= 0; --k) {
            uint32_t f = 1, F = 0;
            bool emit = false;
            if (act) {
                const int t = k == 0 ? 0 : 1 + 8 * c + (k - 1);
                const uint32_t sym = uint32_t(int32_t(q[k]) - T.tmin[t]);
                const uint32_t e = tab[min(T.off[t] + sym, T.total - 1u)];   // in range by construction; clamped anyway
                f = e & 0xFFFFu;
                F = e >> 16;
                emit = x >= (f << (31u - b));         // f * 2^(31-b) <= 2^31 fits 32 bits
            }
            const uint32_t bal = __ballot_sync(0xFFFFFFFFu, emit);
            const uint32_t n = __popc(bal);
            if (n > end) { end = 0; break; }          // cannot happen: at most one word per symbol fits the area
            end -= n;
            if (emit) {
                area[end + __popc(bal & lt)] = uint16_t(x);
                x >>= 16;
            }
            if (act) x = ((x / f) << b) + (x % f) + F;   // Eq. 17
        }
    }
    states[size_t(tile) * 32u + lane] = x;
    if (lane == 0) counts[tile] = cap - end;
}

// move every tile's words from the end of its area to its place in the payload
__global__ void compact_kernel(const uint16_t *__restrict__ scratch, uint32_t cap, const uint32_t *__restrict__ counts,
                               const uint32_t *__restrict__ offsets, uint32_t n_tiles, uint16_t *__restrict__ payload) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t tile = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (tile >= n_tiles) return;
    const uint32_t n = counts[tile];
    const uint16_t *src = scratch + size_t(tile) * cap + (cap - n);
    uint16_t *dst = payload + offsets[tile];
    for (uint32_t i = lane; i < n; i += 32u) dst[i] = src[i];
}

size_t align_up(size_t v) { return (v + 255) & ~size_t(255); }

struct Workspace {
    float *mu, *sigma;
    uint32_t *rows, *hist, *states, *counts, *offsets, *fF;
    int *overflow;
    int16_t *fields;
    uint16_t *scratch, *payload;
    size_t bytes;
};

Workspace carve(uint8_t *base, uint32_t R, uint32_t C, uint32_t V) {
    const uint64_t nvec = uint64_t(R) * (C / 8);
    const uint64_t n_tiles = (nvec + V - 1) / V;
    const uint64_t cap = 9ull * V;
    size_t at = 0;
    auto take = [&](size_t n) { uint8_t *p = base ? base + at : nullptr; at += align_up(n); return p; };
    Workspace w{};
    w.mu = reinterpret_cast<float *>(take(4ull * R));
    w.sigma = reinterpret_cast<float *>(take(4ull * R));
    w.rows = reinterpret_cast<uint32_t *>(take(4ull * R));
    w.hist = reinterpret_cast<uint32_t *>(take(4ull * EP_NUM_TABLES * kHistBins));
    w.overflow = reinterpret_cast<int *>(take(4));
    w.fF = reinterpret_cast<uint32_t *>(take(4ull * kMaxTableSymbols));
    w.states = reinterpret_cast<uint32_t *>(take(128ull * n_tiles));
    w.counts = reinterpret_cast<uint32_t *>(take(4ull * n_tiles));
    w.offsets = reinterpret_cast<uint32_t *>(take(4ull * (n_tiles + 1)));
    w.fields = reinterpret_cast<int16_t *>(take(18ull * nvec));
    w.scratch = reinterpret_cast<uint16_t *>(take(2ull * cap * n_tiles));
    w.payload = reinterpret_cast<uint16_t *>(take(2ull * cap * n_tiles));
    w.bytes = at;
    return w;
}

#define EP_CUDA(call)                                \
    do {                                             \
        if ((call) != cudaSuccess) return EP_ERR_CUDA; \
    } while (0)

// Page-locked host memory: for finished blobs and for the histograms that come back after every counting pass.
// Locking memory costs milliseconds, so each of the two uses keeps the buffer it last gave back (one at most, the
// larger one when two compete) for the next request that fits into it.
struct PinnedSlot {
    std::mutex lock;
    uint8_t *spare = nullptr;
    size_t spare_cap = 0;

    uint8_t *acquire(size_t n, size_t headroom, size_t *cap) {
        {
            std::lock_guard<std::mutex> hold(lock);
            if (spare && spare_cap >= n) {
                uint8_t *p = spare;
                *cap = spare_cap;
                spare = nullptr;
                spare_cap = 0;
                return p;
            }
        }
        const size_t want = n + headroom;
        void *p = nullptr;
        if (cudaHostAlloc(&p, want, cudaHostAllocDefault) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        *cap = want;
        return static_cast<uint8_t *>(p);
    }
    void release(uint8_t *p, size_t cap) {
        uint8_t *drop = p;
        {
            std::lock_guard<std::mutex> hold(lock);
            if (cap > spare_cap) {               // keep the larger of the two
                drop = spare;
                spare = p;
                spare_cap = cap;
            }
        }
        if (drop) cudaFreeHost(drop);
    }
};
PinnedSlot g_blob_slot, g_hist_slot;

// headroom for blobs: the next tensor of a model is rarely the same size
uint8_t *pinned_acquire(size_t n, size_t *cap) { return g_blob_slot.acquire(n, n / 8 + 4096, cap); }
void pinned_release(uint8_t *p, size_t cap) { g_blob_slot.release(p, cap); }

class DeviceBackend final : public EncodeBackend {
public:
    DeviceBackend(const float *dW, uint32_t R, uint32_t C, uint32_t V, uint8_t *ws, cudaStream_t st)
        : W_(dW), R_(R), C_(C), V_(V), w_(carve(ws, R, C, V)), st_(st) {
        hist_ = reinterpret_cast<uint32_t *>(g_hist_slot.acquire(kHistBytes, 0, &hist_cap_));
        if (!hist_) throw std::bad_alloc();
    }
    ~DeviceBackend() override { if (hist_) g_hist_slot.release(reinterpret_cast<uint8_t *>(hist_), hist_cap_); }

    int prepare(const std::vector<uint32_t> &sample) override {
        n_sample_ = uint32_t(sample.size());
        EP_CUDA(cudaMemcpyAsync(w_.rows, sample.data(), 4ull * n_sample_, cudaMemcpyHostToDevice, st_));
        row_rms_kernel<<<(R_ + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, st_>>>(W_, R_, C_, w_.mu);
        EP_CUDA(cudaGetLastError());
        return EP_OK;
    }
    int count_sample(float s, Model &m) override { return count(w_.rows, n_sample_, s, nullptr, m); }
    int count_full(float s, Model &m) override { return count(nullptr, R_, s, w_.fields, m); }

    int finish(float s, int b, uint32_t V, const Model &m, ep_blob *out) override {
        const uint64_t nvec = uint64_t(R_) * (C_ / 8);
        const uint32_t n_tiles = uint32_t((nvec + V - 1) / V);
        const uint32_t cap = 9u * V;
        if (C_ % 64 == 0 && (reinterpret_cast<uintptr_t>(w_.fields) & 15) == 0)
            refit_kernel<<<(R_ + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, st_>>>(W_, R_, C_, w_.fields, s, w_.mu, w_.sigma);
        else
            refit_rows_kernel<<<(R_ + 63) / 64, 64, 0, st_>>>(W_, R_, C_, w_.fields, s, w_.mu, w_.sigma);
        EP_CUDA(cudaGetLastError());
        EncodeTables T{};
        std::vector<uint32_t> fF;
        for (int t = 0; t < EP_NUM_TABLES; ++t) {
            T.tmin[t] = m.t[t].lo;
            T.off[t] = uint32_t(fF.size());
            for (uint32_t j = 0; j < m.t[t].K(); ++j) fF.push_back(m.t[t].f[j] | (m.t[t].F[j] << 16));
        }
        T.total = uint32_t(fF.size());
        if (T.total > kMaxTableSymbols) return EP_ERR_UNSUPPORTED;
        EP_CUDA(cudaMemcpyAsync(w_.fF, fF.data(), 4ull * fF.size(), cudaMemcpyHostToDevice, st_));
        const size_t smem = 4ull * T.total;
        if (smem > 48u * 1024u)
            EP_CUDA(cudaFuncSetAttribute(tile_encode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        tile_encode_kernel<<<(n_tiles + 7) / 8, 256, smem, st_>>>(w_.fields, uint32_t(nvec), V, n_tiles, uint32_t(b), T, w_.fF,
                                                                  w_.scratch, cap, w_.states, w_.counts);
        EP_CUDA(cudaGetLastError());
        std::vector<uint32_t> counts(n_tiles), offsets(n_tiles + 1, 0);
        EP_CUDA(cudaMemcpyAsync(counts.data(), w_.counts, 4ull * n_tiles, cudaMemcpyDeviceToHost, st_));
        EP_CUDA(cudaStreamSynchronize(st_));
        uint64_t total = 0;
        for (uint32_t t = 0; t < n_tiles; ++t) { offsets[t] = uint32_t(total); total += counts[t]; }
        offsets[n_tiles] = uint32_t(total);
        if (total >= (1ull << 31)) return EP_ERR_UNSUPPORTED;
        EP_CUDA(cudaMemcpyAsync(w_.offsets, offsets.data(), 4ull * (n_tiles + 1), cudaMemcpyHostToDevice, st_));
        compact_kernel<<<(n_tiles + 7) / 8, 256, 0, st_>>>(w_.scratch, cap, w_.counts, w_.offsets, n_tiles, w_.payload);
        EP_CUDA(cudaGetLastError());
        std::vector<uint32_t> states(size_t(n_tiles) * 32);
        std::vector<float> sigma(R_);
        EP_CUDA(cudaMemcpyAsync(states.data(), w_.states, 128ull * n_tiles, cudaMemcpyDeviceToHost, st_));
        EP_CUDA(cudaMemcpyAsync(sigma.data(), w_.sigma, 4ull * R_, cudaMemcpyDeviceToHost, st_));
        EP_CUDA(cudaStreamSynchronize(st_));
        // everything but the payload is laid out on the host; the compacted payload is copied straight into its place
        uint64_t payload_at = 0;
        out->acquire = pinned_acquire;
        out->release = pinned_release;
        const int rc = assemble_blob(m, R_, C_, b, V, sigma.data(), s, states.data(), nullptr, counts.data(), out, &payload_at);
        if (rc) return rc;
        if (total) {
            EP_CUDA(cudaMemcpyAsync(out->data() + payload_at, w_.payload, 2ull * total, cudaMemcpyDeviceToHost, st_));
            EP_CUDA(cudaStreamSynchronize(st_));
        }
        return EP_OK;
    }

private:
    int count(const uint32_t *rows, uint32_t n_rows, float s, int16_t *fields, Model &m) {
        EP_CUDA(cudaMemsetAsync(w_.hist, 0, 4ull * EP_NUM_TABLES * kHistBins, st_));
        EP_CUDA(cudaMemsetAsync(w_.overflow, 0, 4, st_));
        const uint64_t n = uint64_t(n_rows) * (C_ / 8);
        const uint64_t want = (n + 255) / 256;
        const uint32_t grid = uint32_t(std::min<uint64_t>(want, 148u * 16u));
        quantise_count_kernel<<<grid, 256, 0, st_>>>(W_, C_, w_.mu, rows, n, s, fields, w_.hist, w_.overflow);
        EP_CUDA(cudaGetLastError());
        int overflow = 0;
        EP_CUDA(cudaMemcpyAsync(hist_, w_.hist, kHistBytes, cudaMemcpyDeviceToHost, st_));
        EP_CUDA(cudaMemcpyAsync(&overflow, w_.overflow, 4, cudaMemcpyDeviceToHost, st_));
        EP_CUDA(cudaStreamSynchronize(st_));
        if (overflow) return EP_ERR_UNSUPPORTED;     // a coordinate beyond +-4095: use the host encoder
        m.from_histograms(hist_, kHistBins, kHistOrigin);
        return EP_OK;
    }

    const float *W_;
    uint32_t R_, C_, V_;
    Workspace w_;
    cudaStream_t st_;
    static constexpr size_t kHistBytes = 4ull * EP_NUM_TABLES * kHistBins;
    uint32_t *hist_ = nullptr;       // page-locked: the copy back after each counting pass is a plain DMA
    size_t hist_cap_ = 0;
    uint32_t n_sample_ = 0;
};

uint32_t tile_vectors_of(const ep_encode_opts &o, double target_bpp) {
    return o.tile_vectors ? o.tile_vectors : ep_default_tile_vectors(target_bpp);
}

}  // namespace

extern "C" size_t ep_encode_device_workspace_bytes(uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts *opts_in) {
    ep_encode_opts o;
    if (opts_in) o = *opts_in; else ep_encode_opts_default(&o);
    if (ep::check_encode_args(R, C, target_bpp, o)) return 0;
    return carve(nullptr, R, C, tile_vectors_of(o, target_bpp)).bytes;
}

extern "C" int ep_encode_device(const float *d_W, uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts *opts_in,
                                void *d_workspace, size_t workspace_bytes, void *stream, ep_blob **out) {
    if (!d_W || !out || !d_workspace) return EP_ERR_BAD_ARG;
    ep_encode_opts o;
    if (opts_in) o = *opts_in; else ep_encode_opts_default(&o);
    const int bad = ep::check_encode_args(R, C, target_bpp, o);
    if (bad) return bad;
    if ((reinterpret_cast<uintptr_t>(d_W) & 15) || (reinterpret_cast<uintptr_t>(d_workspace) & 255)) return EP_ERR_BAD_ARG;
    const uint32_t V = tile_vectors_of(o, target_bpp);
    if (uint64_t(V) * 9u >= (1ull << 31)) return EP_ERR_UNSUPPORTED;
    if (workspace_bytes < carve(nullptr, R, C, V).bytes) return EP_ERR_SCRATCH;
    try {
        DeviceBackend be(d_W, R, C, V, static_cast<uint8_t *>(d_workspace), static_cast<cudaStream_t>(stream));
        return ep::run_encode(be, R, C, target_bpp, o, out);
    } catch (const std::bad_alloc &) {
        return EP_ERR_NOMEM;
    } catch (...) {
        return EP_ERR_UNSUPPORTED;
    }
}
