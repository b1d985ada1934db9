// Stored-representation layout helpers shared by the host encoder, the validator and the
// decode launcher of the library.  Byte layout: see include/entropack.h.
#pragma once
#include <cstdint>
#include <cstring>

#include "entropack.h"

namespace ep {

constexpr uint32_t kMagic = 0x314B5045u;  // "EPK1"
constexpr uint32_t kHeaderBytes = 64;
constexpr uint32_t kStates = 32;          // J
constexpr uint32_t kTileRecordBytes = 4 * kStates + 4;
constexpr uint32_t kStateLow = 1u << 15;  // states live in [2^15, 2^31)
#ifndef EP_TILES_PER_CTA
#define EP_TILES_PER_CTA 32
#endif
constexpr uint32_t kDecodeTilesPerCta = EP_TILES_PER_CTA;  // tiles one CTA of the decode kernel works on at a time (one per warp)

template <class T>
inline T load_le(const uint8_t *p) {
    T v;
    std::memcpy(&v, p, sizeof(T));  // little-endian hosts only (x86-64, aarch64)
    return v;
}
template <class T>
inline void store_le(uint8_t *p, T v) {
    std::memcpy(p, &v, sizeof(T));
}

// table id of field k (0 = coset, 1..7 = z_k, 8 = m) under coset c
inline int table_id(int c, int k) { return k == 0 ? 0 : 1 + 8 * c + (k - 1); }

inline uint64_t table_section_bytes(const uint32_t K[EP_NUM_TABLES]) {
    uint64_t k = 0;
    for (int t = 0; t < EP_NUM_TABLES; ++t) k += K[t];
    return (8ull * EP_NUM_TABLES + 2ull * k + 3ull) & ~3ull;
}

int parse_info(const void *blob, size_t n, ep_info *out);

}  // namespace ep
