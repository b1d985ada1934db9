// Host-side EntroPack encoder (paper Sec. 3.2-3.6): row normalisation, E8 nearest-point
// quantisation, field representation, coset-conditioned model, sampled storage estimate,
// geometric scale search with precision escalation (Algorithm 1), row-scale refit (Eq. 13),
// final tables and tiled 32-state rANS encoding (Eq. 17).
//
// Numerical conventions (they decide which lattice point and which scale are chosen, so they are
// part of the format's encoder contract):
//   * row RMS: squares accumulated in double in index order, one rounding to fp32;
//   * quantiser input: two fp32 divisions, (x / mu) / s, with s rounded once to fp32;
//   * coordinate rounding ties to even; parity fix on the first coordinate of largest |residual|,
//     sign(0) = +1; the half coset is taken only when strictly closer (distances: fp32 residuals
//     of the final candidates, squares summed in double in index order);
//   * frequencies: f = max(1, floor(n 2^b / total)); deficit to the largest f (lowest index),
//     excess taken from the current largest f;
//   * C_CE summed over tables 0..16 and symbols in ascending order, in double.
// This file must be compiled without floating-point contraction.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <functional>
#include <new>
#include <thread>
#include <vector>

#include "encoder_core.hpp"

namespace ep {

// ---- small thread helper: static contiguous partition of [0, n) -------------------------------
void parallel_for(uint64_t n, int threads, const std::function<void(uint64_t, uint64_t, int)> &body) {
    if (threads <= 1 || n < 2) { body(0, n, 0); return; }
    const uint64_t parts = std::min<uint64_t>(uint64_t(threads), n);
    std::vector<std::thread> pool;
    pool.reserve(parts);
    for (uint64_t p = 0; p < parts; ++p) {
        const uint64_t lo = n * p / parts, hi = n * (p + 1) / parts;
        pool.emplace_back([=, &body] { body(lo, hi, int(p)); });
    }
    for (auto &t : pool) t.join();
}

int resolve_threads(int requested) {
    if (requested > 0) return requested;
    const unsigned hw = std::thread::hardware_concurrency();
    return hw ? int(hw) : 1;
}

// ---- Sec. 3.3: the seventeen categorical tables -------------------------------------------------
uint32_t Table::observed() const {
    uint32_t o = 0;
    for (uint64_t c : n) o += c != 0;
    return o;
}

// counts from field tuples; threads reduce private (min, max) first, then private histograms
void Model::count(const int32_t *fld, uint64_t nvec, int threads) {
    struct Range { int64_t lo[EP_NUM_TABLES], hi[EP_NUM_TABLES]; bool any[EP_NUM_TABLES]; };
    const int T = std::max(1, threads);
    std::vector<Range> rg(T);
    for (auto &r : rg) for (int i = 0; i < EP_NUM_TABLES; ++i) { r.any[i] = false; r.lo[i] = r.hi[i] = 0; }
    parallel_for(nvec, T, [&](uint64_t a, uint64_t b, int id) {
        Range &r = rg[id];
        for (uint64_t v = a; v < b; ++v) {
            const int32_t *q = fld + 9 * v;
            for (int k = 0; k < 9; ++k) {
                const int ti = table_id(q[0], k);
                if (!r.any[ti]) { r.any[ti] = true; r.lo[ti] = r.hi[ti] = q[k]; }
                else { r.lo[ti] = std::min<int64_t>(r.lo[ti], q[k]); r.hi[ti] = std::max<int64_t>(r.hi[ti], q[k]); }
            }
        }
    });
    for (int i = 0; i < EP_NUM_TABLES; ++i) {
        bool any = false;
        int64_t lo = 0, hi = 0;
        for (auto &r : rg) if (r.any[i]) {
            if (!any) { lo = r.lo[i]; hi = r.hi[i]; any = true; }
            else { lo = std::min(lo, r.lo[i]); hi = std::max(hi, r.hi[i]); }
        }
        t[i] = Table();
        if (any) { t[i].lo = int32_t(lo); t[i].n.assign(size_t(hi - lo + 1), 0); }
    }
    std::vector<std::vector<uint64_t>> priv(size_t(T) * EP_NUM_TABLES);
    parallel_for(nvec, T, [&](uint64_t a, uint64_t b, int id) {
        std::vector<uint64_t> *h = &priv[size_t(id) * EP_NUM_TABLES];
        for (int i = 0; i < EP_NUM_TABLES; ++i) h[i].assign(t[i].n.size(), 0);
        for (uint64_t v = a; v < b; ++v) {
            const int32_t *q = fld + 9 * v;
            for (int k = 0; k < 9; ++k) {
                const int ti = table_id(q[0], k);
                h[ti][size_t(q[k] - t[ti].lo)]++;
            }
        }
    });
    for (int id = 0; id < T; ++id)
        for (int i = 0; i < EP_NUM_TABLES; ++i) {
            const auto &h = priv[size_t(id) * EP_NUM_TABLES + i];
            for (size_t j = 0; j < h.size(); ++j) { t[i].n[j] += h[j]; t[i].total += h[j]; }
        }
}

void Model::from_histograms(const uint32_t *hist, uint32_t bins, int32_t origin) {
    for (int i = 0; i < EP_NUM_TABLES; ++i) {
        const uint32_t *h = hist + size_t(i) * bins;
        uint32_t first = bins, last = 0;
        for (uint32_t j = 0; j < bins; ++j)
            if (h[j]) { if (first == bins) first = j; last = j; }
        t[i] = Table();
        if (first == bins) continue;
        t[i].lo = origin + int32_t(first);
        t[i].n.assign(h + first, h + last + 1);
        for (uint64_t c : t[i].n) t[i].total += c;
    }
}

// integer frequencies summing to 2^b, every observed symbol >= 1
void Model::normalise(int b) {
    const uint64_t M = 1ull << b;
    for (auto &tb : t) {
        const uint32_t K = tb.K();
        tb.f.assign(K, 0);
        tb.F.assign(K + 1, 0);
        if (!K || !tb.total) continue;
        uint64_t sum = 0;
        for (uint32_t j = 0; j < K; ++j) {
            if (!tb.n[j]) continue;
            const uint64_t q = tb.n[j] * M / tb.total;
            tb.f[j] = uint32_t(std::max<uint64_t>(q, 1));
            sum += tb.f[j];
        }
        auto largest = [&] { return uint32_t(std::max_element(tb.f.begin(), tb.f.end()) - tb.f.begin()); };
        if (sum < M) tb.f[largest()] += uint32_t(M - sum);
        while (sum > M) {
            const uint32_t j = largest();
            const uint64_t take = std::min<uint64_t>(sum - M, uint64_t(tb.f[j]) - 1);
            if (take == 0) break;   // over 2^b observed symbols: callers check worst_observed() before relying on the sum
            tb.f[j] -= uint32_t(take);
            sum -= take;
        }
        for (uint32_t j = 0; j < K; ++j) tb.F[j + 1] = tb.F[j] + tb.f[j];
    }
}

// Eq. 8
double Model::cross_entropy_bits(int b) const {
    double acc = 0.0;
    for (const auto &tb : t)
        for (uint32_t j = 0; j < tb.K(); ++j)
            if (tb.n[j]) acc += double(tb.n[j]) * (double(b) - std::log2(double(tb.f[j])));
    return acc;
}

uint64_t Model::section_bytes() const {
    uint32_t K[EP_NUM_TABLES];
    for (int i = 0; i < EP_NUM_TABLES; ++i) K[i] = t[i].K();
    return table_section_bytes(K);
}

uint32_t Model::worst_observed() const {
    uint32_t w = 0;
    for (const auto &tb : t) w = std::max(w, tb.observed());
    return w;
}

uint32_t Model::worst_coordinate_observed() const {
    uint32_t w = 0;
    for (int i = 1; i < EP_NUM_TABLES; ++i) w = std::max(w, t[i].observed());
    return w;
}

// Eq. 10-11: estimated stored bits of nvec vectors in `rows` rows under model m
double estimate_bits(const Model &m, int b, uint64_t nvec, uint64_t rows, uint32_t V, double retained, double *cce_out) {
    const double cce = m.cross_entropy_bits(b);
    const uint64_t n_tile = (nvec + V - 1) / V;
    const double left = std::max(0.0, cce - retained * double(kStates) * double(n_tile));
    const double payload = 16.0 * std::ceil(left / 16.0);
    const double restart = double(n_tile) * (32.0 * kStates + 32.0) + 32.0;
    const double tables = 8.0 * double(m.section_bytes());
    const double scales = 32.0 * double(rows);
    const double other = 8.0 * kHeaderBytes;
    if (cce_out) *cce_out = cce;
    return payload + restart + tables + scales + other;
}

// ---- App. "Scale-search settings": the fixed row sample -----------------------------------------
static inline uint64_t splitmix64(uint64_t &state) {
    uint64_t z = (state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

std::vector<uint32_t> sample_rows(uint32_t R, uint32_t C, uint32_t budget_vectors) {
    const uint32_t per_row = C / 8;
    uint32_t n = std::max<uint32_t>(1, budget_vectors / per_row);
    n = std::min(n, R);
    std::vector<uint32_t> idx(R);
    for (uint32_t i = 0; i < R; ++i) idx[i] = i;
    uint64_t st = (uint64_t(R) << 32) + uint64_t(C);
    for (uint32_t i = 0; i < n; ++i) {
        const uint32_t j = i + uint32_t(splitmix64(st) % uint64_t(R - i));
        std::swap(idx[i], idx[j]);
    }
    idx.resize(n);
    std::sort(idx.begin(), idx.end());
    return idx;
}

// header + tables + scales + tile index + payload
int assemble_blob(const Model &m, uint32_t R, uint32_t C, int b, uint32_t V, const float *sigma, float s_info,
                  const uint32_t *states, const uint16_t *const *tile_words, const uint32_t *tile_len, ep_blob *out,
                  uint64_t *payload_offset) {
    const uint64_t nvec = uint64_t(R) * (C / 8);
    const uint32_t n_tiles = uint32_t((nvec + V - 1) / V);
    uint64_t total_words = 0;
    for (uint32_t t = 0; t < n_tiles; ++t) total_words += tile_len[t];
    // coordinate range of z_1..z_8 (z_8 = 2m + parity spans [2 m_lo, 2 m_hi + 1])
    bool any = false;
    int64_t cmin = 0, cmax = 0;
    for (int c = 0; c < 2; ++c)
        for (int k = 1; k <= 8; ++k) {
            const Table &tb = m.t[table_id(c, k)];
            if (!tb.K()) continue;
            int64_t lo = tb.lo, hi = int64_t(tb.lo) + tb.K() - 1;
            if (k == 8) { lo *= 2; hi = 2 * hi + 1; }
            if (!any) { cmin = lo; cmax = hi; any = true; }
            else { cmin = std::min(cmin, lo); cmax = std::max(cmax, hi); }
        }
    cmin = std::max<int64_t>(cmin, -32768);
    cmax = std::min<int64_t>(cmax, 32767);
    const uint64_t tb_bytes = m.section_bytes();
    const uint64_t off_tables = kHeaderBytes, off_scales = off_tables + tb_bytes, off_tiles = off_scales + 4ull * R;
    const uint64_t off_payload = off_tiles + uint64_t(kTileRecordBytes) * n_tiles + 4, total = off_payload + 2 * total_words;
    if (total >= (1ull << 32)) return EP_ERR_UNSUPPORTED;   // section offsets are 32-bit
    uint8_t *p = out->allocate(size_t(total));   // uninitialised: everything before the payload is zeroed here,
    if (!p) return EP_ERR_NOMEM;                 // the payload is written whole below or by the caller
    std::memset(p, 0, size_t(off_payload));
    if (payload_offset) *payload_offset = off_payload;
    store_le<uint32_t>(p, kMagic);
    store_le<uint16_t>(p + 4, 1);
    p[6] = uint8_t(b);
    p[7] = uint8_t(kStates);
    store_le<uint32_t>(p + 8, R);
    store_le<uint32_t>(p + 12, C);
    store_le<uint32_t>(p + 16, V);
    store_le<uint32_t>(p + 20, n_tiles);
    store_le<float>(p + 24, s_info);
    store_le<int16_t>(p + 28, int16_t(cmin));
    store_le<int16_t>(p + 30, int16_t(cmax));
    store_le<uint32_t>(p + 32, uint32_t(off_tables));
    store_le<uint32_t>(p + 36, uint32_t(off_scales));
    store_le<uint32_t>(p + 40, uint32_t(off_tiles));
    store_le<uint32_t>(p + 44, uint32_t(off_payload));
    store_le<uint64_t>(p + 48, total);
    store_le<uint32_t>(p + 56, uint32_t(total_words));
    uint8_t *dir = p + off_tables;
    uint8_t *fq = dir + 8 * EP_NUM_TABLES;
    for (int i = 0; i < EP_NUM_TABLES; ++i) {
        store_le<int32_t>(dir + 4 * i, m.t[i].lo);
        store_le<uint32_t>(dir + 4 * EP_NUM_TABLES + 4 * i, m.t[i].K());
        for (uint32_t j = 0; j < m.t[i].K(); ++j, fq += 2) store_le<uint16_t>(fq, uint16_t(m.t[i].f[j]));
    }
    std::memcpy(p + off_scales, sigma, 4ull * R);
    uint64_t at = 0;
    for (uint32_t t = 0; t < n_tiles; ++t) {
        uint8_t *rec = p + off_tiles + uint64_t(kTileRecordBytes) * t;
        std::memcpy(rec, states + size_t(t) * kStates, 4 * kStates);
        store_le<uint32_t>(rec + 4 * kStates, uint32_t(at));
        if (tile_words && tile_len[t]) std::memcpy(p + off_payload + 2 * at, tile_words[t], 2ull * tile_len[t]);
        at += tile_len[t];
    }
    store_le<uint32_t>(p + off_tiles + uint64_t(kTileRecordBytes) * n_tiles, uint32_t(at));
    return EP_OK;
}

// ---- Sec. 3.5 / Alg. 2: candidate ratios ---------------------------------------------------------------
std::vector<double> rdo_ratios(int K) {
    std::vector<double> cut = {std::log(0.70), 0.0, std::log(1.45)};   // sorted log-points, the two bounds included
    std::vector<double> rho = {1.0};
    while (int(rho.size()) < K) {
        size_t at = 0;
        double widest = -1.0;
        for (size_t j = 0; j + 1 < cut.size(); ++j)
            if (cut[j + 1] - cut[j] > widest) { widest = cut[j + 1] - cut[j]; at = j; }   // first one on ties
        const double mid = 0.5 * (cut[at] + cut[at + 1]);
        cut.insert(cut.begin() + long(at) + 1, mid);
        rho.push_back(std::exp(mid));
    }
    return rho;
}

// ---- Algorithm 1 + rate correction + packing, over a back end ---------------------------------------
int run_encode(EncodeBackend &be, uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts &o, ep_blob **out) {
    const uint64_t nvec = uint64_t(R) * (C / 8);
    const uint32_t V = o.tile_vectors ? o.tile_vectors : ep_default_tile_vectors(target_bpp);
    int b = o.b_start ? o.b_start : (target_bpp <= 7.0 ? 11 : 12);
    b = std::min(b, o.b_max);
    const std::vector<uint32_t> rows = sample_rows(R, C, o.sample_vectors);
    const uint64_t svec = uint64_t(rows.size()) * (C / 8);
    int rc = be.prepare(rows);
    if (rc) return rc;
    float s = 0.0f;
    double last_rate = 0.0;
    Model full;
    for (;; ++b) {
        double lo = o.bracket_lo, hi = o.bracket_hi;
        for (int it = 0; it < o.search_steps; ++it) {
            const double mid = std::sqrt(lo * hi);
            Model m;
            if ((rc = be.count_sample(float(mid), m))) return rc;
            // more observed symbols than 2^b slots: no b-bit table exists for this scale; treat it as too fine
            // (rate above the target).  If the scale found this way still overflows on the full tensor, b goes up.
            if (m.worst_observed() > (1u << b)) { lo = mid; continue; }
            m.normalise(b);
            const double bits = estimate_bits(m, b, svec, rows.size(), V, o.retained_bits, nullptr);
            last_rate = bits / (8.0 * double(svec));
            if (last_rate > target_bpp) lo = mid; else hi = mid;
        }
        s = float(std::sqrt(lo * hi));
        bool fits = false;
        for (;;) {
            if ((rc = be.count_full(s, full))) return rc;
            if (full.worst_observed() <= (1u << b)) { fits = true; break; }
            if (b < o.b_max) break;
            s = float(1.05 * double(s) * double(full.worst_coordinate_observed()) / double(1u << b));
        }
        if (fits) break;
    }
    // Beyond Algorithm 1: steer s with the full-tensor estimate (Eq. 10-11), first by the one-bit-per-doubling
    // law (Eq. 9), then by the measured slope.  The sampled tables miss rare symbols of the full tensor, which
    // costs rate on heavy tails.
    struct { double log_s, rate; bool valid; } last{0.0, 0.0, false};
    for (int step = 0; step < o.polish_steps; ++step) {
        Model m = full;
        m.normalise(b);
        const double est = estimate_bits(m, b, nvec, R, V, o.polish_retained_bits, nullptr) / (double(R) * double(C));
        if (std::fabs(est - target_bpp) <= 0.002 * target_bpp) break;
        // rate lost per doubling of s: 1 bit by Eq. 9 for the first move, afterwards the secant slope
        const double log_s = std::log2(double(s));
        double per_doubling = 1.0;
        if (last.valid && log_s != last.log_s) {
            per_doubling = -(est - last.rate) / (log_s - last.log_s);
            if (!(per_doubling >= 0.5)) per_doubling = 0.5;
            if (per_doubling > 4.0) per_doubling = 4.0;
        }
        last = {log_s, est, true};
        const float before = s;
        double moved = std::exp2(log_s + (est - target_bpp) / per_doubling);
        if (!(moved >= o.bracket_lo)) moved = o.bracket_lo;   // never leave the search bracket
        if (moved > o.bracket_hi) moved = o.bracket_hi;
        s = float(moved);
        if (s == before) break;
        if ((rc = be.count_full(s, full))) return rc;
        if (full.worst_observed() > (1u << b)) {   // the finer scale overflows the tables: undo and stop
            s = before;
            if ((rc = be.count_full(s, full))) return rc;
            break;
        }
    }
    if (o.rdo_candidates > 1 && (rc = be.refine(s, b, V, o, full))) return rc;
    full.normalise(b);
    ep_blob *blob = new ep_blob();
    rc = be.finish(s, b, V, full, blob);
    if (rc) { delete blob; return rc; }
    blob->report.s = double(s);
    blob->report.b = b;
    blob->report.bytes = blob->size();
    blob->report.stored_bpp = 8.0 * double(blob->size()) / (double(R) * double(C));
    blob->report.est_bpp_sample = last_rate;
    blob->report.cce_bits = full.cross_entropy_bits(b);
    blob->report.sample_rows = uint32_t(rows.size());
    *out = blob;
    return EP_OK;
}

namespace {

// ---- Sec. 3.2 ----------------------------------------------------------------------------------
float row_rms(const float *x, uint32_t C) {
    double acc = 0.0;
    for (uint32_t j = 0; j < C; ++j) { const double v = x[j]; acc += v * v; }
    double mu = std::sqrt(acc / double(C));
    if (!(mu > kEta)) mu = kEta;
    return float(mu);
}

// round to nearest integer, ties to even (default rounding mode); |y| < 2^22 uses the exact
// add-and-subtract of 1.5 * 2^23, anything larger is handed to the library routine.
inline float round_even(float y) {
    if (std::fabs(y) < 4194304.0f) {
        volatile float t = y + 12582912.0f;
        return t - 12582912.0f;
    }
    return std::nearbyintf(y);
}

// Eq. 3 on one 8-vector; returns the integer point and keeps the fp32 residuals of that point.
struct D8 {
    int32_t z[8];
    float res[8];
};
inline void nearest_d8(const float *y, D8 &o) {
    int32_t sum = 0;
    for (int i = 0; i < 8; ++i) {
        const float f = round_even(y[i]);
        o.z[i] = int32_t(f);
        o.res[i] = y[i] - f;
        sum += o.z[i];
    }
    if (sum & 1) {
        int at = 0;
        float big = std::fabs(o.res[0]);
        for (int i = 1; i < 8; ++i) {
            const float a = std::fabs(o.res[i]);
            if (a > big) { big = a; at = i; }
        }
        const int step = (o.res[at] >= 0.0f) ? 1 : -1;
        o.z[at] += step;
        o.res[at] = y[at] - float(o.z[at]);
    }
}

// Eq. 2 + Eq. 4: quantise one block x[0..8) of a row with RMS mu at scale s; writes (c, z1..z7, m).
inline void quantise_block(const float *x, float mu, float s, int32_t *fld) {
    float y[8], yh[8];
    for (int i = 0; i < 8; ++i) {
        const float X = x[i] / mu;
        y[i] = X / s;
        yh[i] = y[i] - 0.5f;
    }
    D8 a, h;
    nearest_d8(y, a);
    nearest_d8(yh, h);
    double da = 0.0, dh = 0.0;
    for (int i = 0; i < 8; ++i) {
        da += double(a.res[i]) * double(a.res[i]);
        dh += double(h.res[i]) * double(h.res[i]);
    }
    const D8 &w = (dh < da) ? h : a;
    fld[0] = (dh < da) ? 1 : 0;
    int32_t s7 = 0;
    for (int i = 0; i < 7; ++i) { fld[1 + i] = w.z[i]; s7 += w.z[i]; }
    const int32_t pi = s7 & 1;              // two's complement: (sum mod 2) in {0, 1}
    fld[8] = (w.z[7] - pi) >> 1;            // exact: z8 - pi is even
}

void quantise_rows(const float *W, uint32_t C, const float *mu, const uint32_t *rows, uint64_t n_rows, float s,
                   int32_t *fields, int threads) {
    const uint32_t per_row = C / 8;
    parallel_for(n_rows, threads, [&](uint64_t lo, uint64_t hi, int) {
        for (uint64_t i = lo; i < hi; ++i) {
            const uint64_t r = rows ? rows[i] : i;
            const float *x = W + r * C;
            int32_t *f = fields + i * per_row * 9;
            for (uint32_t v = 0; v < per_row; ++v) quantise_block(x + 8 * v, mu[r], s, f + 9 * v);
        }
    });
}

// ---- Sec. 3.6 / App. "Tiled rANS implementation": one tile -------------------------------------
// The decoder visits (group of 32 vectors, field 0..8, lane 0..31); the encoder walks that order
// backwards, emits a word before the update whenever xi >= f * 2^(31-b), and finally reverses the
// tile's words.
void encode_tile(const int32_t *fld, uint32_t nv, const Model &m, int b, uint32_t *states, std::vector<uint16_t> &words) {
    uint32_t xi[kStates];
    for (auto &x : xi) x = kStateLow;
    words.clear();
    words.reserve(size_t(nv) * 5);
    const uint32_t groups = (nv + kStates - 1) / kStates;
    for (uint32_t g = groups; g-- > 0;) {
        const uint32_t lanes = std::min<uint32_t>(kStates, nv - g * kStates);
        for (int k = 8; k >= 0; --k)
            for (uint32_t l = lanes; l-- > 0;) {
                const int32_t *q = fld + 9ull * (uint64_t(g) * kStates + l);
                const Table &tb = m.t[table_id(q[0], k)];
                const uint32_t sym = uint32_t(q[k] - tb.lo);
                const uint32_t f = tb.f[sym], F = tb.F[sym];
                uint32_t x = xi[l];
                if (uint64_t(x) >= (uint64_t(f) << (31 - b))) { words.push_back(uint16_t(x)); x >>= 16; }
                xi[l] = ((x / f) << b) + (x % f) + F;
            }
    }
    std::reverse(words.begin(), words.end());
    std::copy(xi, xi + kStates, states);
}

// tile coding of given fields under a normalised model, then assembly
int pack_fields_host(const int32_t *fields, uint32_t R, uint32_t C, int b, uint32_t V, const Model &m, const float *sigma,
                     float s_info, int threads, ep_blob *out) {
    const uint64_t nvec = uint64_t(R) * (C / 8);
    const uint32_t n_tiles = uint32_t((nvec + V - 1) / V);
    std::vector<std::vector<uint16_t>> words(n_tiles);
    std::vector<uint32_t> states(size_t(n_tiles) * kStates);
    parallel_for(n_tiles, threads, [&](uint64_t lo, uint64_t hi, int) {
        for (uint64_t t = lo; t < hi; ++t) {
            const uint64_t v0 = t * V;
            const uint32_t nv = uint32_t(std::min<uint64_t>(V, nvec - v0));
            encode_tile(fields + 9 * v0, nv, m, b, &states[t * kStates], words[t]);
        }
    });
    std::vector<const uint16_t *> ptr(n_tiles);
    std::vector<uint32_t> len(n_tiles);
    for (uint32_t t = 0; t < n_tiles; ++t) { ptr[t] = words[t].data(); len[t] = uint32_t(words[t].size()); }
    return assemble_blob(m, R, C, b, V, sigma, s_info, states.data(), ptr.data(), len.data(), out);
}

// Eq. 13
void refit(const float *W, uint32_t R, uint32_t C, const int32_t *fields, float s, const float *mu, float *sigma, int threads) {
    const uint32_t per_row = C / 8;
    parallel_for(R, threads, [&](uint64_t lo, uint64_t hi, int) {
        for (uint64_t r = lo; r < hi; ++r) {
            double xp = 0.0, pp = 0.0;
            const float *x = W + r * C;
            for (uint32_t v = 0; v < per_row; ++v) {
                const int32_t *q = fields + 9 * (r * per_row + v);
                const double half = 0.5 * double(q[0]);
                int32_t s7 = 0;
                for (int j = 0; j < 7; ++j) {
                    const double p = double(q[1 + j]) + half;
                    xp += double(x[8 * v + j]) * p;
                    pp += p * p;
                    s7 += q[1 + j];
                }
                const double p8 = double(2 * q[8] + (s7 & 1)) + half;   // Eq. 5
                xp += double(x[8 * v + 7]) * p8;
                pp += p8 * p8;
            }
            double sg;
            if (pp > 0.0) { sg = xp / pp; if (!(sg > kEta)) sg = kEta; }
            else sg = double(s) * double(mu[r]);
            sigma[r] = float(sg);
        }
    });
}


// ---- the host back end: everything on CPU threads ------------------------------------------------------
class HostBackend final : public EncodeBackend {
public:
    HostBackend(const float *W, uint32_t R, uint32_t C, int threads) : W_(W), R_(R), C_(C), threads_(threads) {}

    int prepare(const std::vector<uint32_t> &sample) override {
        rows_ = sample;
        mu_.resize(R_);
        parallel_for(R_, threads_, [&](uint64_t lo, uint64_t hi, int) {
            for (uint64_t r = lo; r < hi; ++r) mu_[r] = row_rms(W_ + r * C_, C_);
        });
        sfields_.resize(size_t(rows_.size()) * (C_ / 8) * 9);
        fields_.resize(size_t(R_) * (C_ / 8) * 9);
        return EP_OK;
    }
    int count_sample(float s, Model &m) override {
        quantise_rows(W_, C_, mu_.data(), rows_.data(), rows_.size(), s, sfields_.data(), threads_);
        m.count(sfields_.data(), uint64_t(rows_.size()) * (C_ / 8), threads_);
        return EP_OK;
    }
    int count_full(float s, Model &m) override {
        quantise_rows(W_, C_, mu_.data(), nullptr, R_, s, fields_.data(), threads_);
        m.count(fields_.data(), uint64_t(R_) * (C_ / 8), threads_);
        return EP_OK;
    }
    int finish(float s, int b, uint32_t V, const Model &m, ep_blob *out) override {
        std::vector<float> sigma(R_);
        if (refined_sigma_.empty()) refit(W_, R_, C_, fields_.data(), s, mu_.data(), sigma.data(), threads_);
        else sigma = refined_sigma_;
        return pack_fields_host(fields_.data(), R_, C_, b, V, m, sigma.data(), s, threads_, out);
    }

    // Sec. 3.5 / Alg. 2.  Candidate k quantises every row at rho_k * s and refits its scale (Eq. 13); D is the
    // row's squared error with the stored fp32 scale.  Each sweep fits one shared model to the rows' current
    // choices (every value of the range spanned by all candidates gets half a count more), prices every
    // candidate (Eq. 14), sets the budget of Eq. 15 from the baseline's and the mixture's estimated bytes, and
    // picks per row argmin D + lambda R (Eq. 16) with the smallest common lambda found that meets the budget.
    int refine(float s, int b, uint32_t V, const ep_encode_opts &o, Model &m) override {
        const int K = o.rdo_candidates;
        const uint32_t per_row = C_ / 8;
        const uint64_t nvec = uint64_t(R_) * per_row;
        const std::vector<double> rho = rdo_ratios(K);
        struct Candidate { std::vector<int32_t> fields; std::vector<float> sigma; };
        std::vector<Candidate> cand(K);
        std::vector<double> D(size_t(R_) * K), cost(size_t(R_) * K);
        for (int k = 0; k < K; ++k) {
            Candidate &c = cand[k];
            c.sigma.resize(R_);
            if (k == 0) {
                c.fields = fields_;
                refit(W_, R_, C_, c.fields.data(), s, mu_.data(), c.sigma.data(), threads_);
            } else {
                const float sk = float(rho[k] * double(s));
                c.fields.resize(size_t(nvec) * 9);
                quantise_rows(W_, C_, mu_.data(), nullptr, R_, sk, c.fields.data(), threads_);
                refit(W_, R_, C_, c.fields.data(), sk, mu_.data(), c.sigma.data(), threads_);
            }
            parallel_for(R_, threads_, [&](uint64_t lo, uint64_t hi, int) {
                for (uint64_t r = lo; r < hi; ++r) {
                    double err = 0.0;
                    const double sg = double(c.sigma[r]);
                    for (uint32_t v = 0; v < per_row; ++v) {
                        const int32_t *q = c.fields.data() + 9 * (r * per_row + v);
                        int32_t s7 = 0, two_p[8];
                        for (int j = 0; j < 7; ++j) { two_p[j] = 2 * q[1 + j] + q[0]; s7 += q[1 + j]; }
                        two_p[7] = 2 * (2 * q[8] + (s7 & 1)) + q[0];
                        for (int j = 0; j < 8; ++j) {
                            const double d = double(W_[r * C_ + 8 * v + j]) - sg * (0.5 * double(two_p[j]));
                            err += d * d;
                        }
                    }
                    D[r * K + k] = err;
                }
            });
        }
        // value range of every table over all candidates
        int64_t lo[EP_NUM_TABLES], hi[EP_NUM_TABLES];
        bool used[EP_NUM_TABLES] = {};
        for (const Candidate &c : cand)
            for (uint64_t v = 0; v < nvec; ++v) {
                const int32_t *q = c.fields.data() + 9 * v;
                for (int j = 0; j < 9; ++j) {
                    const int t = table_id(q[0], j);
                    if (!used[t]) { used[t] = true; lo[t] = hi[t] = q[j]; }
                    else { lo[t] = std::min<int64_t>(lo[t], q[j]); hi[t] = std::max<int64_t>(hi[t], q[j]); }
                }
            }
        std::vector<double> price[EP_NUM_TABLES];      // -log2 of the smoothed probability
        std::vector<uint64_t> seen[EP_NUM_TABLES];
        for (int t = 0; t < EP_NUM_TABLES; ++t)
            if (used[t]) { price[t].resize(size_t(hi[t] - lo[t] + 1)); seen[t].resize(price[t].size()); }
        auto choose = [&](double lambda, std::vector<int> &pick) {   // kappa_lambda and L(lambda)
            double L = 0.0;
            for (uint32_t r = 0; r < R_; ++r) {
                int best = 0;
                double bv = D[size_t(r) * K] + lambda * cost[size_t(r) * K];
                for (int k = 1; k < K; ++k) {
                    const double v = D[size_t(r) * K + k] + lambda * cost[size_t(r) * K + k];
                    if (v < bv) { bv = v; best = k; }
                }
                pick[r] = best;
                L += cost[size_t(r) * K + best];
            }
            return L;
        };
        auto gather = [&](const std::vector<int> &pick, std::vector<int32_t> &dst) {
            for (uint32_t r = 0; r < R_; ++r)
                std::copy_n(cand[pick[r]].fields.begin() + long(9 * uint64_t(r) * per_row), 9 * per_row,
                            dst.begin() + long(9 * uint64_t(r) * per_row));
        };
        Model base;
        base.count(cand[0].fields.data(), nvec, threads_);
        base.normalise(b);
        const double B = estimate_bits(base, b, nvec, R_, V, o.retained_bits, nullptr) / 8.0;
        std::vector<int> sel(R_, 0), hat(R_), trial(R_);
        std::vector<int32_t> mix(size_t(nvec) * 9);
        for (int sweep = 0; sweep < o.rdo_sweeps; ++sweep) {
            gather(sel, mix);
            uint64_t total[EP_NUM_TABLES] = {};
            for (int t = 0; t < EP_NUM_TABLES; ++t) std::fill(seen[t].begin(), seen[t].end(), 0);
            for (uint64_t v = 0; v < nvec; ++v) {
                const int32_t *q = mix.data() + 9 * v;
                for (int j = 0; j < 9; ++j) { const int t = table_id(q[0], j); seen[t][size_t(q[j] - lo[t])]++; total[t]++; }
            }
            for (int t = 0; t < EP_NUM_TABLES; ++t) {
                if (!used[t]) continue;
                const double den = double(total[t]) + 0.5 * double(price[t].size());
                for (size_t z = 0; z < price[t].size(); ++z) price[t][z] = -std::log2((double(seen[t][z]) + 0.5) / den);
            }
            parallel_for(R_, threads_, [&](uint64_t a, uint64_t e, int) {
                for (uint64_t r = a; r < e; ++r)
                    for (int k = 0; k < K; ++k) {
                        double bits = 0.0;
                        for (uint32_t v = 0; v < per_row; ++v) {
                            const int32_t *q = cand[k].fields.data() + 9 * (r * per_row + v);
                            for (int j = 0; j < 9; ++j) { const int t = table_id(q[0], j); bits += price[t][size_t(q[j] - lo[t])]; }
                        }
                        cost[r * K + k] = bits;
                    }
            });
            Model mm;
            mm.count(mix.data(), nvec, threads_);
            if (mm.worst_observed() > (1u << b)) break;
            mm.normalise(b);
            const double Bmix = estimate_bits(mm, b, nvec, R_, V, o.retained_bits, nullptr) / 8.0;
            double cur = 0.0, dcur = 0.0;
            for (uint32_t r = 0; r < R_; ++r) { cur += cost[size_t(r) * K + sel[r]]; dcur += D[size_t(r) * K + sel[r]]; }
            const double budget = cur + 8.0 * (B - Bmix);
            if (choose(0.0, hat) > budget) {
                double lam_lo = 0.0, lam_hi = (cur > 0.0 && dcur > 0.0) ? dcur / cur : 1e-12;
                bool bracketed = false;
                for (int d = 0; d < 64; ++d) {
                    if (choose(lam_hi, trial) <= budget) { bracketed = true; break; }
                    lam_lo = lam_hi;
                    lam_hi *= 2.0;
                }
                if (bracketed) {
                    hat = trial;
                    for (int it = 0; it < 20; ++it) {
                        const double lam = lam_lo == 0.0 ? 0.5 * lam_hi : std::sqrt(lam_lo * lam_hi);
                        if (choose(lam, trial) > budget) lam_lo = lam;
                        else { lam_hi = lam; hat = trial; }
                    }
                } else {
                    hat = sel;       // no penalty meets the budget: keep the current selection
                }
            }
            sel = hat;
        }
        gather(sel, mix);
        Model refined;
        refined.count(mix.data(), nvec, threads_);
        if (refined.worst_observed() <= (1u << b)) {     // otherwise the baseline stays
            fields_.swap(mix);
            refined_sigma_.resize(R_);
            for (uint32_t r = 0; r < R_; ++r) refined_sigma_[r] = cand[sel[r]].sigma[r];
            m = refined;
        }
        return EP_OK;
    }

private:
    const float *W_;
    uint32_t R_, C_;
    int threads_;
    std::vector<uint32_t> rows_;
    std::vector<float> mu_;
    std::vector<int32_t> sfields_, fields_;
    std::vector<float> refined_sigma_;
};

}  // namespace
}  // namespace ep

// ---- C ABI -----------------------------------------------------------------------------------------

extern "C" void ep_encode_opts_default(ep_encode_opts *o) {
    if (!o) return;
    o->bracket_lo = 1e-3;
    o->bracket_hi = 8.0;
    o->search_steps = 12;
    o->sample_vectors = 1u << 18;
    o->tile_vectors = 0;
    o->b_start = 0;
    o->b_max = 15;
    o->retained_bits = 16.0;
    o->polish_steps = 3;
    o->polish_retained_bits = 8.0;
    o->threads = 0;
    o->rdo_candidates = 1;
    o->rdo_sweeps = 1;
}

namespace ep {
int check_encode_args(uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts &o) {
    if (R == 0 || C == 0 || C % 8 != 0 || !(target_bpp > 0.0)) return EP_ERR_BAD_ARG;
    if (uint64_t(R) * (C / 8) >= (1ull << 32)) return EP_ERR_BAD_ARG;
    if (!(o.bracket_lo > 0.0) || !(o.bracket_hi > o.bracket_lo) || o.search_steps < 0 || o.polish_steps < 0 || o.rdo_candidates < 1 || o.rdo_candidates > 64 || o.rdo_sweeps < 0 || o.b_max > 15 ||
        o.b_max < 9 || (o.b_start != 0 && (o.b_start < 9 || o.b_start > o.b_max)))
        return EP_ERR_BAD_ARG;
    return EP_OK;
}
}  // namespace ep

extern "C" int ep_encode(const float *W, uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts *opts_in,
                         ep_blob **out) {
    using namespace ep;
    if (!W || !out) return EP_ERR_BAD_ARG;
    ep_encode_opts o;
    if (opts_in) o = *opts_in; else ep_encode_opts_default(&o);
    const int bad = check_encode_args(R, C, target_bpp, o);
    if (bad) return bad;
    try {
        HostBackend be(W, R, C, resolve_threads(o.threads));
        return run_encode(be, R, C, target_bpp, o, out);
    } catch (const std::bad_alloc &) {
        return EP_ERR_NOMEM;
    } catch (...) {
        return EP_ERR_UNSUPPORTED;
    }
}

extern "C" int ep_pack_fields(const int32_t *fields, uint32_t R, uint32_t C, int32_t b, uint32_t V,
                              const float *row_scales, float s_info, int32_t threads, ep_blob **out) {
    using namespace ep;
    if (!fields || !row_scales || !out || R == 0 || C == 0 || C % 8 != 0 || V == 0 || b < 9 || b > 15) return EP_ERR_BAD_ARG;
    const uint64_t nvec = uint64_t(R) * (C / 8);
    if (nvec >= (1ull << 32)) return EP_ERR_BAD_ARG;
    for (uint64_t v = 0; v < nvec; ++v)
        if (fields[9 * v] != 0 && fields[9 * v] != 1) return EP_ERR_BAD_ARG;
    try {
        const int T = resolve_threads(threads);
        Model m;
        m.count(fields, nvec, T);
        if (m.worst_observed() > (1u << b)) return EP_ERR_UNSUPPORTED;
        m.normalise(b);
        ep_blob *blob = new ep_blob();
        const int rc = pack_fields_host(fields, R, C, b, V, m, row_scales, s_info, T, blob);
        if (rc) { delete blob; return rc; }
        blob->report.s = double(s_info);
        blob->report.b = b;
        blob->report.bytes = blob->size();
        blob->report.stored_bpp = 8.0 * double(blob->size()) / (double(R) * double(C));
        blob->report.cce_bits = m.cross_entropy_bits(b);
        *out = blob;
        return EP_OK;
    } catch (const std::bad_alloc &) {
        return EP_ERR_NOMEM;
    } catch (...) {
        return EP_ERR_UNSUPPORTED;
    }
}

extern "C" const void *ep_blob_data(const ep_blob *b) { return b ? b->data() : nullptr; }
extern "C" size_t ep_blob_bytes(const ep_blob *b) { return b ? b->size() : 0; }
extern "C" int ep_blob_report(const ep_blob *b, ep_encode_report *out) {
    if (!b || !out) return EP_ERR_BAD_ARG;
    *out = b->report;
    return EP_OK;
}
extern "C" void ep_blob_free(ep_blob *b) { delete b; }
