// Parsing and structural validation of the stored representation (host side).
#include "stream.hpp"

#include <cmath>

namespace ep {

int parse_info(const void *blob_v, size_t n, ep_info *out) {
    if (!blob_v || !out) return EP_ERR_BAD_ARG;
    const uint8_t *blob = static_cast<const uint8_t *>(blob_v);
    if (n < kHeaderBytes) return EP_ERR_BAD_STREAM;
    if (load_le<uint32_t>(blob) != kMagic || load_le<uint16_t>(blob + 4) != 1) return EP_ERR_BAD_STREAM;
    ep_info I{};
    I.b = blob[6];
    I.J = blob[7];
    I.R = load_le<uint32_t>(blob + 8);
    I.C = load_le<uint32_t>(blob + 12);
    I.V = load_le<uint32_t>(blob + 16);
    I.n_tiles = load_le<uint32_t>(blob + 20);
    I.s = load_le<float>(blob + 24);
    I.coord_min = load_le<int16_t>(blob + 28);
    I.coord_max = load_le<int16_t>(blob + 30);
    I.off_tables = load_le<uint32_t>(blob + 32);
    I.off_scales = load_le<uint32_t>(blob + 36);
    I.off_tiles = load_le<uint32_t>(blob + 40);
    I.off_payload = load_le<uint32_t>(blob + 44);
    I.total_bytes = load_le<uint64_t>(blob + 48);
    I.total_words = load_le<uint32_t>(blob + 56);
    if (I.J != kStates || I.b < 9 || I.b > 15) return EP_ERR_BAD_STREAM;
    if (I.R == 0 || I.C == 0 || I.C % 8 != 0 || I.V == 0) return EP_ERR_BAD_STREAM;
    const uint64_t nvec = uint64_t(I.R) * (I.C / 8);
    if (nvec >= (1ull << 32)) return EP_ERR_BAD_STREAM;
    if ((nvec + I.V - 1) / I.V != I.n_tiles) return EP_ERR_BAD_STREAM;
    if (I.total_bytes != n || I.off_tables != kHeaderBytes) return EP_ERR_BAD_STREAM;
    if (n < kHeaderBytes + 8ull * EP_NUM_TABLES) return EP_ERR_BAD_STREAM;
    const uint8_t *dir = blob + I.off_tables;
    for (int t = 0; t < EP_NUM_TABLES; ++t) {
        I.table_min[t] = load_le<int32_t>(dir + 4 * t);
        I.table_K[t] = load_le<uint32_t>(dir + 4 * EP_NUM_TABLES + 4 * t);
        if (I.table_K[t] > (1u << 16)) return EP_ERR_BAD_STREAM;
    }
    const uint64_t tb = table_section_bytes(I.table_K);
    if (I.off_scales != I.off_tables + tb) return EP_ERR_BAD_STREAM;
    if (I.off_tiles != uint64_t(I.off_scales) + 4ull * I.R) return EP_ERR_BAD_STREAM;
    if (I.off_payload != uint64_t(I.off_tiles) + uint64_t(kTileRecordBytes) * I.n_tiles + 4ull) return EP_ERR_BAD_STREAM;
    if (I.total_bytes != uint64_t(I.off_payload) + 2ull * I.total_words) return EP_ERR_BAD_STREAM;
    *out = I;
    return EP_OK;
}

}  // namespace ep

extern "C" int ep_blob_info(const void *blob, size_t n, ep_info *out) { return ep::parse_info(blob, n, out); }

extern "C" int ep_validate(const void *blob_v, size_t n) {
    using namespace ep;
    ep_info I;
    int rc = parse_info(blob_v, n, &I);
    if (rc) return rc;
    const uint8_t *blob = static_cast<const uint8_t *>(blob_v);
    // every used table sums to 2^b; the coset table and, per observed coset, its coordinate tables exist
    const uint8_t *fq = blob + I.off_tables + 8 * EP_NUM_TABLES;
    bool used[EP_NUM_TABLES];
    for (int t = 0; t < EP_NUM_TABLES; ++t) {
        uint64_t sum = 0;
        for (uint32_t j = 0; j < I.table_K[t]; ++j) sum += load_le<uint16_t>(fq + 2ull * j);
        fq += 2ull * I.table_K[t];
        used[t] = I.table_K[t] != 0;
        if (used[t] && sum != (1ull << I.b)) return EP_ERR_BAD_STREAM;
    }
    if (!used[0]) return EP_ERR_BAD_STREAM;
    {   // coset symbols must be 0/1 and each coset with positive frequency needs all eight tables
        if (I.table_min[0] < 0 || int64_t(I.table_min[0]) + I.table_K[0] > 2) return EP_ERR_BAD_STREAM;
        const uint8_t *f0 = blob + I.off_tables + 8 * EP_NUM_TABLES;
        for (uint32_t j = 0; j < I.table_K[0]; ++j) {
            if (load_le<uint16_t>(f0 + 2 * j) == 0) continue;
            const int c = I.table_min[0] + int(j);
            for (int k = 1; k <= 8; ++k)
                if (!used[table_id(c, k)]) return EP_ERR_BAD_STREAM;
        }
    }
    // tile records: states in range, offsets monotone, final boundary = total words
    const uint8_t *ti = blob + I.off_tiles;
    uint32_t prev = 0;
    for (uint32_t t = 0; t < I.n_tiles; ++t) {
        const uint8_t *rec = ti + uint64_t(kTileRecordBytes) * t;
        for (uint32_t l = 0; l < kStates; ++l) {
            const uint32_t x = load_le<uint32_t>(rec + 4 * l);
            if (x < kStateLow || x >= (1u << 31)) return EP_ERR_BAD_STREAM;
        }
        const uint32_t off = load_le<uint32_t>(rec + 4 * kStates);
        if ((t == 0 && off != 0) || off < prev || off > I.total_words) return EP_ERR_BAD_STREAM;
        prev = off;
    }
    const uint32_t fin = load_le<uint32_t>(ti + uint64_t(kTileRecordBytes) * I.n_tiles);
    if (fin != I.total_words || fin < prev) return EP_ERR_BAD_STREAM;
    return EP_OK;
}

extern "C" const char *ep_strerror(int status) {
    switch (status) {
    case EP_OK: return "ok";
    case EP_ERR_BAD_ARG: return "bad argument";
    case EP_ERR_BAD_STREAM: return "malformed or inconsistent compressed stream";
    case EP_ERR_UNSUPPORTED: return "unsupported request";
    case EP_ERR_CUDA: return "CUDA runtime error";
    case EP_ERR_NOMEM: return "out of host memory";
    case EP_ERR_SCRATCH: return "scratch buffer missing, misaligned or too small";
    case EP_ERR_STATIC_LIMIT: return "stream needs lookup tables larger than the built-in area (b above EP_STATIC_MAX_B)";
    default: return "unknown status";
    }
}

extern "C" uint32_t ep_default_tile_vectors(double target_bpp) {
    // the paper's defaults: 32768 / 16384 / 8192 / 4096 symbols at 2 / 4 / 7 / 8 bpp; V = max(32, S/9)
    const uint32_t S = target_bpp < 3.0 ? 32768u : target_bpp < 5.5 ? 16384u : target_bpp < 7.5 ? 8192u : 4096u;
    const uint32_t V = S / 9u;
    return V < 32u ? 32u : V;
}

extern "C" uint32_t ep_suggest_tile_vectors(uint32_t R, uint32_t C, double target_bpp, uint32_t decode_slots) {
    const uint32_t vmax = ep_default_tile_vectors(target_bpp);
    const uint64_t nvec = uint64_t(R) * (C / 8);
    if (decode_slots == 0 || nvec == 0) return vmax;
    // a small tensor cannot fill the decoder anyway: never let metadata grow beyond about 4x the default's share
    // (a quarter of the default, rounded down to whole groups of 32 vectors)
    const uint64_t floor_v = (vmax / 4) / 32 * 32 > 32 ? (vmax / 4) / 32 * 32 : 32;
    // fewest rounds whose tiles are not larger than the default; tile sizes are multiples of 32 vectors (whole
    // groups of 32 rANS states, no partly filled last group) whenever that still fits
    for (uint64_t rounds = 1;; ++rounds) {
        const uint64_t tiles = rounds * decode_slots;
        uint64_t V = (nvec + tiles - 1) / tiles;
        if (V > vmax) continue;
        const uint64_t V32 = (V + 31) & ~uint64_t(31);
        if (V32 <= vmax) V = V32;
        return uint32_t(V < floor_v ? floor_v : V);
    }
}

extern "C" uint32_t ep_suggest_tile_vectors_batch(const uint32_t *R, const uint32_t *C, uint32_t n, double target_bpp,
                                                  uint32_t decode_ctas) {
    const uint32_t vmax = ep_default_tile_vectors(target_bpp);
    if (!R || !C || n == 0 || decode_ctas == 0) return vmax;
    // One launch decodes all n tensors: a CTA takes 48 tiles per round, the rounds of all tensors are split evenly
    // over the CTAs, so the launch lasts ceil(rounds / CTAs) rounds of ceil(V / 32) groups each (plus a small
    // fixed cost per round: tile set-up and the last, partly idle steps).  Take the multiple of 32 that makes this
    // shortest; on ties the larger tile (less metadata).  Never below a quarter of the paper's default.
    const uint32_t lo = (vmax / 4u) / 32u * 32u > 32u ? (vmax / 4u) / 32u * 32u : 32u;   // as in ep_suggest_tile_vectors
    uint32_t best_v = vmax;
    uint64_t best_cost = ~0ull;
    for (uint32_t V = lo; V <= vmax; V += 32u) {
        uint64_t rounds = 0;
        for (uint32_t i = 0; i < n; ++i) {
            const uint64_t nvec = uint64_t(R[i]) * (C[i] / 8u);
            const uint64_t tiles = (nvec + V - 1u) / V;
            rounds += (tiles + ep::kDecodeTilesPerCta - 1u) / ep::kDecodeTilesPerCta;
        }
        const uint64_t cost = ((rounds + decode_ctas - 1u) / decode_ctas) * (V / 32u + 2u);
        if (cost <= best_cost) { best_cost = cost; best_v = V; }
    }
    return best_v;
}

extern "C" int ep_version(void) { return 1; }
