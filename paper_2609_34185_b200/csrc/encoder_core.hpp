// Shared pieces of the EntroPack encoder: the seventeen-table model, the stored-size estimate,
// the row sampler, blob assembly, and the search driver (Algorithm 1 plus the full-tensor rate
// correction) that runs on top of either back end - host threads (encoder.cpp) or CUDA kernels
// (encode_gpu.cu).  Both back ends produce byte-identical streams for the same input.
#pragma once
#include <cstdint>
#include <memory>
#include <new>
#include <utility>
#include <vector>

#include "stream.hpp"

// allocator whose resize() leaves new bytes uninitialised (a blob of tens of MB is written exactly once)
template <class T>
struct ep_no_init_allocator : std::allocator<T> {
    template <class U> struct rebind { using other = ep_no_init_allocator<U>; };
    ep_no_init_allocator() = default;
    template <class U> ep_no_init_allocator(const ep_no_init_allocator<U> &) {}
    template <class U> void construct(U *p) { ::new (static_cast<void *>(p)) U; }
    template <class U, class... A> void construct(U *p, A &&...a) { ::new (static_cast<void *>(p)) U(std::forward<A>(a)...); }
};

// Host storage of a stored representation.  By default ordinary heap memory; a back end may install its
// own source (the GPU back end: page-locked memory, which the device copies into at full bus speed and
// which a later upload reads at full speed too) before the blob is assembled.
struct ep_blob {
    std::vector<uint8_t, ep_no_init_allocator<uint8_t>> heap;
    uint8_t *ext = nullptr;                                  // storage obtained through `acquire`
    size_t ext_size = 0, ext_cap = 0;
    uint8_t *(*acquire)(size_t n, size_t *cap) = nullptr;    // nullptr on failure
    void (*release)(uint8_t *p, size_t cap) = nullptr;
    ep_encode_report report{};

    ep_blob() = default;
    ep_blob(const ep_blob &) = delete;
    ep_blob &operator=(const ep_blob &) = delete;
    ~ep_blob() { if (ext && release) release(ext, ext_cap); }
    // n bytes of uninitialised storage (replaces what the blob held); nullptr if the source has none
    uint8_t *allocate(size_t n) {
        if (acquire) {
            if (ext && release) release(ext, ext_cap);
            ext_size = ext_cap = 0;
            ext = acquire(n, &ext_cap);
            if (!ext) return nullptr;
            ext_size = n;
            return ext;
        }
        heap.resize(n);
        return heap.data();
    }
    const uint8_t *data() const { return ext ? ext : heap.data(); }
    uint8_t *data() { return ext ? ext : heap.data(); }
    size_t size() const { return ext ? ext_size : heap.size(); }
};

namespace ep {

constexpr double kEta = 1e-12;

int resolve_threads(int requested);

// ---- Sec. 3.3: the seventeen categorical tables -------------------------------------------------
struct Table {
    int32_t lo = 0;
    std::vector<uint64_t> n;   // counts over [lo, lo + K)
    std::vector<uint32_t> f;   // b-bit frequencies
    std::vector<uint32_t> F;   // exclusive prefix sums, K + 1 entries
    uint64_t total = 0;
    uint32_t K() const { return uint32_t(n.size()); }
    uint32_t observed() const;
};

struct Model {
    Table t[EP_NUM_TABLES];
    void count(const int32_t *fields, uint64_t nvec, int threads);          // from (c, z1..z7, m) tuples
    // from dense histograms hist[t][value - origin], `bins` bins per table (zero bins outside the observed range)
    void from_histograms(const uint32_t *hist, uint32_t bins, int32_t origin);
    void normalise(int b);                                                   // integer frequencies summing to 2^b
    double cross_entropy_bits(int b) const;                                  // Eq. 8
    uint64_t section_bytes() const;
    uint32_t worst_observed() const;                                         // largest alphabet over all tables
    uint32_t worst_coordinate_observed() const;                              // A_max: over the 16 coordinate tables
};

// Eq. 10-11: estimated stored bits of nvec vectors in `rows` rows under model m
double estimate_bits(const Model &m, int b, uint64_t nvec, uint64_t rows, uint32_t V, double retained, double *cce_out);

// App. "Scale-search settings": complete rows, shape-dependent seed, sorted
std::vector<uint32_t> sample_rows(uint32_t R, uint32_t C, uint32_t budget_vectors);

// header + tables + scales + tile index + payload; `states` holds 32 words per tile, tile t's payload is
// tile_words[t] .. + tile_len[t].  With tile_words == nullptr the payload section is left unwritten for the
// caller to fill in place: it starts at out->bytes.data() + *payload_offset and holds the tiles back to back.
int assemble_blob(const Model &m, uint32_t R, uint32_t C, int b, uint32_t V, const float *sigma, float s_info,
                  const uint32_t *states, const uint16_t *const *tile_words, const uint32_t *tile_len, ep_blob *out,
                  uint64_t *payload_offset = nullptr);

// What a back end must provide.  Each call returns an ep_status.
struct EncodeBackend {
    virtual ~EncodeBackend() {}
    virtual int prepare(const std::vector<uint32_t> &sample) = 0;   // row RMS; remember the row sample
    virtual int count_sample(float s, Model &m) = 0;                // quantise the sample at s, count its fields
    virtual int count_full(float s, Model &m) = 0;                  // quantise the whole tensor at s (kept), count
    // refit the row scales of the kept quantisation (Eq. 13), encode the tiles under the normalised
    // full-tensor model m and assemble the blob
    virtual int finish(float s, int b, uint32_t V, const Model &m, ep_blob *out) = 0;
    // per-row rate-distortion refinement of the kept quantisation (Sec. 3.5, Alg. 2); on success `m` holds the
    // counts of the refined fields and finish() uses the refined row scales.  Optional.
    virtual int refine(float /*s*/, int /*b*/, uint32_t /*V*/, const ep_encode_opts & /*o*/, Model & /*m*/) { return EP_ERR_UNSUPPORTED; }
};

// the K nested candidate ratios of Alg. 2: 1 first, then log-midpoints of the widest remaining interval of [0.70, 1.45]
std::vector<double> rdo_ratios(int K);

// Algorithm 1, the rate-correction stage and the final packing over a back end.
int run_encode(EncodeBackend &be, uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts &o, ep_blob **out);

}  // namespace ep
