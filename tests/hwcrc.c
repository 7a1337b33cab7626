/* Second opinion for the CRC32C pins: the x86 SSE4.2 `crc32` instruction implements the
 * Castagnoli polynomial in hardware.  Built only by the CPU tests, only where the host
 * has SSE4.2. */
#include <nmmintrin.h>
#include <stdint.h>

uint32_t hw_crc32c(const uint8_t* p, uint64_t n)
{
    uint32_t crc = 0xFFFFFFFFu;
    for (uint64_t i = 0; i < n; i++) crc = _mm_crc32_u8(crc, p[i]);
    return crc ^ 0xFFFFFFFFu;
}
