/* Second opinion for the CRC32C pins, and a strong CPU baseline for the checksum step: the
 * x86 SSE4.2 `crc32` instruction implements the Castagnoli polynomial in hardware.  Not part
 * of the oracle proper (nothing in wm_oracle.c uses it); built only where the host has SSE4.2.
 * TEST INFRASTRUCTURE ONLY, like everything in this directory. */
#include <nmmintrin.h>
#include <stdint.h>
#include <string.h>

/* one byte per instruction: the plainest use, for the pins */
uint32_t hw_crc32c(const uint8_t* p, uint64_t n)
{
    uint32_t crc = 0xFFFFFFFFu;
    for (uint64_t i = 0; i < n; i++) crc = _mm_crc32_u8(crc, p[i]);
    return crc ^ 0xFFFFFFFFu;
}

/* eight bytes per instruction, one dependent chain: what a careful single-threaded CPU
 * implementation without carry-less multiplication reaches */
uint32_t hw_crc32c_u64(const uint8_t* p, uint64_t n)
{
    uint64_t crc = 0xFFFFFFFFu;
    while (n >= 8) {
        uint64_t w;
        memcpy(&w, p, 8);
        crc = _mm_crc32_u64(crc, w);
        p += 8;
        n -= 8;
    }
    uint32_t c = (uint32_t)crc;
    while (n--) c = _mm_crc32_u8(c, *p++);
    return c ^ 0xFFFFFFFFu;
}
