// Host-side GF(2) arithmetic for CRC32C and the constant tables the kernels use.
//
// A CRC register value v stands for a polynomial over GF(2) of degree < 32 in the reflected
// convention (bit 31 = x^0 ... bit 0 = x^31).  Advancing the register over n zero bytes
// multiplies it by x^(8n) modulo the CRC polynomial; every table below is such a product
// for a fixed n, indexed by one byte or one nibble of the register.
#pragma once
#include <cstdint>

namespace wm {

constexpr uint32_t kPolyReflected = 0x82F63B78u;   // CRC32C (Castagnoli), the checksum of the wire format
constexpr uint32_t kPolyZlib = 0xEDB88320u;        // CRC-32 of zlib, an option of the checksum call only

// Byte offsets inside the shared-memory table image.  The image is placed at an address that
// is a multiple of 64 KiB inside the shared window, so that "table base | value << 8 | lane
// slot" can be put together with one byte permute.
//   A01: entry b at b*256: 32 lane copies of G[0][b] (bytes 0..127), then of G[1][b]
//   A23: the same for G[2], G[3]
//   NK : four 4 KiB arrays, array j = nibbles 2j and 2j+1 of the lane-finish table:
//        entry v at v*256: NK[lane][2j][v] for the 32 lanes, then NK[lane][2j+1][v]
constexpr uint32_t kImgA01 = 0x00000, kImgA23 = 0x10000, kImgNK = 0x20000, kImgBytes = 0x24000;

// Tables shared by all kernels; one copy lives in device memory per device.
struct Tables {
    uint32_t image[kImgBytes / 4];   // the shared-memory image described above
    uint32_t NW[8][8][16];           // NW[w][n][v] = (v << 4n) advanced over 2048 (7 - w) bytes
    uint32_t HT[4][256];             // HT[k][b] = (b << 8k) advanced over 16384 bytes (one tile)
    uint32_t T0[256];                // T0[b]    = b advanced over one byte (the classic table)
};

inline uint32_t times_x(uint32_t v, uint32_t poly) { return (v >> 1) ^ ((v & 1u) ? poly : 0u); }

inline uint32_t mulmod(uint32_t a, uint32_t b, uint32_t poly = kPolyReflected)
{
    uint32_t r = 0;
    for (int i = 0; i < 32; i++) {
        if (a & 0x80000000u) r ^= b;
        a <<= 1;
        b = times_x(b, poly);
    }
    return r;
}

// x^(8 n) mod P
inline uint32_t x_pow_bytes(uint64_t n, uint32_t poly = kPolyReflected)
{
    uint32_t result = 0x80000000u, base = 0x00800000u;
    while (n) {
        if (n & 1u) result = mulmod(result, base, poly);
        base = mulmod(base, base, poly);
        n >>= 1;
    }
    return result;
}

inline void build_tables(Tables& t, uint32_t poly = kPolyReflected)
{
    const uint32_t k128 = x_pow_bytes(128, poly), kTile = x_pow_bytes(16384, poly), k1 = x_pow_bytes(1, poly);
    // G[k][b] = (b << 8k) advanced over 128 bytes (one row stride of the word-strided chain)
    for (uint32_t k = 0; k < 4; k++)
        for (uint32_t b = 0; b < 256; b++) {
            const uint32_t g = mulmod(b << (8 * k), k128, poly);
            uint32_t* dst = t.image + ((k < 2 ? kImgA01 : kImgA23) + b * 256 + (k & 1) * 128) / 4;
            for (uint32_t l = 0; l < 32; l++) dst[l] = g;
            t.HT[k][b] = mulmod(b << (8 * k), kTile, poly);
        }
    for (uint32_t b = 0; b < 256; b++) t.T0[b] = mulmod(b, k1, poly);
    // NK[l][n][v] = (v << 4n) advanced over 128 - 4l bytes (a lane's place inside its row)
    for (uint32_t l = 0; l < 32; l++) {
        const uint32_t kl = x_pow_bytes(128 - 4 * l, poly);
        for (uint32_t n = 0; n < 8; n++)
            for (uint32_t v = 0; v < 16; v++)
                t.image[(kImgNK + (n / 2) * 0x1000 + v * 256 + (n & 1) * 128) / 4 + l] = mulmod(v << (4 * n), kl, poly);
    }
    for (uint32_t w = 0; w < 8; w++) {
        const uint32_t kw = x_pow_bytes(2048u * (7 - w), poly);
        for (uint32_t n = 0; n < 8; n++)
            for (uint32_t v = 0; v < 16; v++) t.NW[w][n][v] = mulmod(v << (4 * n), kw, poly);
    }
}

}  // namespace wm
