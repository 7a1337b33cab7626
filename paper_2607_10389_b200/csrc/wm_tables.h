// Host-side GF(2) arithmetic for CRC32C and the constant tables the kernels use.
//
// A CRC register value v stands for a polynomial over GF(2) of degree < 32 in the reflected
// convention (bit 31 = x^0 ... bit 0 = x^31).  Advancing the register over n zero bytes
// multiplies it by x^(8n) modulo the CRC32C polynomial; every table below is such a product
// for a fixed n, indexed by one byte or one nibble of the register.
#pragma once
#include <cstdint>

namespace wm {

constexpr uint32_t kPolyReflected = 0x82F63B78u;

// Tables shared by all kernels; one copy lives in device memory per device.
struct Tables {
    uint32_t G[4][256];       // G[k][b]  = (b << 8k) advanced over 128 bytes (one row stride)
    uint32_t NK[32][8][16];   // NK[l][n][v] = (v << 4n) advanced over 128 - 4l bytes (lane finish)
    uint32_t NW[8][8][16];    // NW[w][n][v] = (v << 4n) advanced over 2048 (7 - w) bytes (warp position)
    uint32_t HT[4][256];      // HT[k][b] = (b << 8k) advanced over 16384 bytes (one tile)
    uint32_t T0[256];         // T0[b]    = b advanced over one byte (the classic table)
};

inline uint32_t times_x(uint32_t v) { return (v >> 1) ^ ((v & 1u) ? kPolyReflected : 0u); }

inline uint32_t mulmod(uint32_t a, uint32_t b)
{
    uint32_t r = 0;
    for (int i = 0; i < 32; i++) {
        if (a & 0x80000000u) r ^= b;
        a <<= 1;
        b = times_x(b);
    }
    return r;
}

// x^(8 n) mod P
inline uint32_t x_pow_bytes(uint64_t n)
{
    uint32_t result = 0x80000000u, base = 0x00800000u;
    while (n) {
        if (n & 1u) result = mulmod(result, base);
        base = mulmod(base, base);
        n >>= 1;
    }
    return result;
}

inline void build_tables(Tables& t)
{
    const uint32_t k128 = x_pow_bytes(128), kTile = x_pow_bytes(16384), k1 = x_pow_bytes(1);
    for (uint32_t k = 0; k < 4; k++)
        for (uint32_t b = 0; b < 256; b++) {
            t.G[k][b] = mulmod(b << (8 * k), k128);
            t.HT[k][b] = mulmod(b << (8 * k), kTile);
        }
    for (uint32_t b = 0; b < 256; b++) t.T0[b] = mulmod(b, k1);
    for (uint32_t l = 0; l < 32; l++) {
        const uint32_t kl = x_pow_bytes(128 - 4 * l);
        for (uint32_t n = 0; n < 8; n++)
            for (uint32_t v = 0; v < 16; v++) t.NK[l][n][v] = mulmod(v << (4 * n), kl);
    }
    for (uint32_t w = 0; w < 8; w++) {
        const uint32_t kw = x_pow_bytes(2048u * (7 - w));
        for (uint32_t n = 0; n < 8; n++)
            for (uint32_t v = 0; v < 16; v++) t.NW[w][n][v] = mulmod(v << (4 * n), kw);
    }
}

}  // namespace wm
