/*
 * CPU oracle for the exact-state session mover's data path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded
 * statement of what the path computes.  It shares no code, header, table or
 * constant generator with the CUDA library and must never be reached from the
 * product path: only the tests, the smoke check and the benchmark's CPU
 * baseline leg may call it.
 *
 * What it follows:
 *   - per-chunk CRC and its GF(2) combination: the paper's verification plane
 *     (Section 6.5: per-chunk CRC overlapped with receive, "GF(2)-combined";
 *     Section 4.1: transfer, CRC-verify, rehydrate).  The polynomial is CRC32C
 *     (Castagnoli), pinned by its check value 0xE3069283.
 *   - dirty chunks of a pre-copy round: Appendix G (round 0 ships every chunk,
 *     later rounds ship the chunks that changed) and Section 3.3 (the dirty
 *     fraction per generation step).
 *   - lossless codec inside the verified envelope: Section 6.4 (bf16 plane
 *     split, the exponent plane carries the redundancy, every round trip
 *     bit-exact, receipts bind to the decoded bytes).  The paper fixes these
 *     properties, not a byte layout; the WM1 layout implemented here is this
 *     repository's own and is written out in wmo_encode()'s comment.
 *   - commit only on a matching fingerprint: Section 4.1 (Sufficiency) and
 *     Table 1 (migrate stages into a shadow slot; commit re-verifies).
 *
 * Pin status: CRC, combine and dirty mask are pinned to published check values,
 * a hardware CRC instruction, zlib's combine identity and brute force.  The
 * encoder's byte layout is new, so no outside implementation exists for it:
 * "parity unpinned" against the outside world; it is pinned by hand-built
 * tiles, a size law recomputed independently, and the round trip.  The same
 * holds for the ENT tiles of the entropy option ("parity unpinned" against the
 * outside world): hand-derived streams, Kraft equality, Shannon's bound, the
 * size law and the choice among the three forms recomputed independently.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define WMO_TILE 16384u          /* bytes per tile                       */
#define WMO_GROUP_ELEMS 256u     /* bf16 elements per group (512 bytes)  */
#define WMO_GROUPS_PER_TILE 32u
#define WMO_HEADER 64u

enum {
    WMO_OK = 0, WMO_ERR_ARG = -1, WMO_ERR_CAPACITY = -2, WMO_ERR_FORMAT = -3,
    WMO_ERR_META_CRC = -4, WMO_ERR_STRUCT = -5, WMO_ERR_DESC = -6,
    WMO_ERR_CHUNK_CRC = -7, WMO_ERR_STALE = -8, WMO_ERR_CACHE_CRC = -9
};

typedef struct {
    int32_t  status;
    uint32_t first_bad_chunk;
    uint32_t n_bad_chunks;
    uint32_t n_present;
    uint64_t wire_len;
    uint64_t payload_bytes;
    uint32_t cache_crc;
    uint32_t reserved;
} wmo_result;

/* ------------------------------------------------------------------ CRC --- */

#define WMO_POLY_CRC32C 0x82F63B78u   /* reflected form of 0x1EDC6F41 */

/* The definition: reflected CRC-32, init all ones, one bit at a time (LSB of each
 * byte first), final complement.  `poly` is the reflected polynomial, so the
 * zlib/IEEE variant (0xEDB88320) can be checked against Python's zlib. */
uint32_t wmo_crc_bitwise(const uint8_t* p, uint64_t n, uint32_t poly)
{
    uint32_t crc = 0xFFFFFFFFu;
    for (uint64_t i = 0; i < n; i++) {
        crc ^= p[i];
        for (int k = 0; k < 8; k++)
            crc = (crc >> 1) ^ ((crc & 1u) ? poly : 0u);
    }
    return crc ^ 0xFFFFFFFFu;
}

/* Same function through the classic one-byte table (built from the bit loop).  The functions
 * of this file keep no state between calls and may be called from several threads at once (the
 * tests run chunk ranges on a thread pool); the table is the one thing shared, and it is built
 * when the library is loaded, before any caller exists. */
static uint32_t g_tab[256];
__attribute__((constructor)) static void build_tab(void)
{
    for (uint32_t b = 0; b < 256; b++) {
        uint32_t v = b;
        for (int k = 0; k < 8; k++)
            v = (v >> 1) ^ ((v & 1u) ? WMO_POLY_CRC32C : 0u);
        g_tab[b] = v;
    }
}

uint32_t wmo_crc32c(const uint8_t* p, uint64_t n)
{
    uint32_t crc = 0xFFFFFFFFu;
    for (uint64_t i = 0; i < n; i++)
        crc = g_tab[(crc ^ p[i]) & 0xFFu] ^ (crc >> 8);
    return crc ^ 0xFFFFFFFFu;
}

/* Product of two residues modulo the CRC32C polynomial.  A 32-bit value stands
 * for a polynomial of degree < 32 with bit 31 = x^0 ... bit 0 = x^31 (the
 * reflected convention), so "times x" is a right shift with feedback. */
static uint32_t gf2_mulmod(uint32_t a, uint32_t b)
{
    uint32_t r = 0;
    for (int i = 0; i < 32; i++) {
        if (a & 0x80000000u) r ^= b;
        a <<= 1;
        b = (b >> 1) ^ ((b & 1u) ? WMO_POLY_CRC32C : 0u);
    }
    return r;
}

/* x^(8*nbytes) mod P by square and multiply. */
static uint32_t gf2_x_pow_8n(uint64_t nbytes)
{
    uint32_t result = 0x80000000u;      /* x^0 */
    uint32_t base = 0x00800000u;        /* x^8 */
    while (nbytes) {
        if (nbytes & 1u) result = gf2_mulmod(result, base);
        base = gf2_mulmod(base, base);
        nbytes >>= 1;
    }
    return result;
}

/* crc(A||B) from crc(A), crc(B) and len(B): crc(A) * x^(8 len(B)) + crc(B).  The
 * all-ones init and the final complement cancel between the three terms. */
uint32_t wmo_crc_combine(uint32_t crc_a, uint32_t crc_b, uint64_t len_b)
{
    return gf2_mulmod(crc_a, gf2_x_pow_8n(len_b)) ^ crc_b;
}

/* ------------------------------------------------------------ geometry --- */

uint64_t wmo_num_chunks(uint64_t nbytes, uint32_t chunk_bytes)
{
    return (nbytes + chunk_bytes - 1) / chunk_bytes;
}

uint64_t wmo_num_tiles(uint64_t nbytes)
{
    return (nbytes + WMO_TILE - 1) / WMO_TILE;
}

uint64_t wmo_meta_end(uint64_t nbytes, uint32_t chunk_bytes)
{
    uint64_t m = WMO_HEADER + 16u * wmo_num_chunks(nbytes, chunk_bytes) + 2u * wmo_num_tiles(nbytes);
    return (m + 31u) & ~(uint64_t)31u;
}

uint64_t wmo_wire_bound(uint64_t nbytes, uint32_t chunk_bytes)
{
    return wmo_meta_end(nbytes, chunk_bytes) + nbytes;
}

static int args_ok(uint64_t nbytes, uint32_t chunk_bytes)
{
    if (nbytes == 0 || chunk_bytes == 0) return 0;
    if (chunk_bytes % WMO_TILE != 0 || chunk_bytes > (1u << 30)) return 0;
    if (wmo_num_tiles(nbytes) > 0xFFFFFFFFull) return 0;
    return 1;
}

static uint64_t chunk_len(uint64_t nbytes, uint32_t chunk_bytes, uint64_t c)
{
    uint64_t lo = c * chunk_bytes;
    uint64_t hi = lo + chunk_bytes;
    return (hi > nbytes ? nbytes : hi) - lo;
}

/* ------------------------------------------------- checksum / dirty mask --- */

int wmo_checksum(const uint8_t* cache, uint64_t nbytes, uint32_t chunk_bytes, uint32_t* crc_out)
{
    if (!cache || !crc_out || !args_ok(nbytes, chunk_bytes)) return WMO_ERR_ARG;
    uint64_t nc = wmo_num_chunks(nbytes, chunk_bytes);
    for (uint64_t c = 0; c < nc; c++)
        crc_out[c] = wmo_crc32c(cache + c * chunk_bytes, chunk_len(nbytes, chunk_bytes, c));
    return WMO_OK;
}

/* A chunk is dirty iff any of its bytes differs from the previous snapshot. */
int wmo_dirty_diff(const uint8_t* cache, const uint8_t* prev, uint64_t nbytes, uint32_t chunk_bytes,
                   uint8_t* dirty_out, uint32_t* dirty_idx_out, uint32_t* n_dirty_out)
{
    if (!cache || !prev || !dirty_out || !n_dirty_out || !args_ok(nbytes, chunk_bytes)) return WMO_ERR_ARG;
    uint64_t nc = wmo_num_chunks(nbytes, chunk_bytes);
    uint32_t n = 0;
    for (uint64_t c = 0; c < nc; c++) {
        uint64_t len = chunk_len(nbytes, chunk_bytes, c);
        uint8_t d = 0;
        for (uint64_t i = 0; i < len; i++)
            if (cache[c * chunk_bytes + i] != prev[c * chunk_bytes + i]) { d = 1; break; }
        dirty_out[c] = d;
        if (d) { if (dirty_idx_out) dirty_idx_out[n] = (uint32_t)c; n++; }
    }
    *n_dirty_out = n;
    return WMO_OK;
}

/* --------------------------------------------------------------- encode --- */

static void put16(uint8_t* p, uint32_t v) { p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); }
static void put32(uint8_t* p, uint32_t v) { for (int i = 0; i < 4; i++) p[i] = (uint8_t)(v >> (8 * i)); }
static void put64(uint8_t* p, uint64_t v) { for (int i = 0; i < 8; i++) p[i] = (uint8_t)(v >> (8 * i)); }
static uint32_t get16(const uint8_t* p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8); }
static uint32_t get32(const uint8_t* p) { uint32_t v = 0; for (int i = 0; i < 4; i++) v |= (uint32_t)p[i] << (8 * i); return v; }
static uint64_t get64(const uint8_t* p) { uint64_t v = 0; for (int i = 0; i < 8; i++) v |= (uint64_t)p[i] << (8 * i); return v; }

/* ---------------------------------------------------------------- XXH64 ---
 * The 64-bit xxHash of a byte string (the published algorithm, all arithmetic modulo 2^64,
 * input read little-endian), as an alternative chunk checksum.  Four accumulators take the
 * input in 32-byte stripes, lane k getting bytes [8k, 8k+8) of every stripe; they are merged,
 * the length is added, the tail goes in 8, 4 and 1 bytes at a time, and an avalanche ends it.
 */
#define XP1 0x9E3779B185EBCA87ull
#define XP2 0xC2B2AE3D27D4EB4Full
#define XP3 0x165667B19E3779F9ull
#define XP4 0x85EBCA77C2B2AE63ull
#define XP5 0x27D4EB2F165667C5ull

static uint64_t xrotl(uint64_t v, int r) { return (v << r) | (v >> (64 - r)); }
static uint64_t xround(uint64_t acc, uint64_t in) { return xrotl(acc + in * XP2, 31) * XP1; }
static uint64_t xmerge(uint64_t h, uint64_t v) { return (h ^ xround(0, v)) * XP1 + XP4; }

uint64_t wmo_xxh64(const uint8_t* p, uint64_t n, uint64_t seed)
{
    const uint8_t* end = p + n;
    uint64_t h;
    if (n >= 32) {
        uint64_t v1 = seed + XP1 + XP2, v2 = seed + XP2, v3 = seed, v4 = seed - XP1;
        while ((uint64_t)(end - p) >= 32) {
            v1 = xround(v1, get64(p));
            v2 = xround(v2, get64(p + 8));
            v3 = xround(v3, get64(p + 16));
            v4 = xround(v4, get64(p + 24));
            p += 32;
        }
        h = xrotl(v1, 1) + xrotl(v2, 7) + xrotl(v3, 12) + xrotl(v4, 18);
        h = xmerge(h, v1); h = xmerge(h, v2); h = xmerge(h, v3); h = xmerge(h, v4);
    } else {
        h = seed + XP5;
    }
    h += n;
    while ((uint64_t)(end - p) >= 8) { h = xrotl(h ^ xround(0, get64(p)), 27) * XP1 + XP4; p += 8; }
    if ((uint64_t)(end - p) >= 4) { h = xrotl(h ^ ((uint64_t)get32(p) * XP1), 23) * XP2 + XP3; p += 4; }
    while (p < end) { h = xrotl(h ^ ((uint64_t)*p * XP5), 11) * XP1; p++; }
    h ^= h >> 33; h *= XP2; h ^= h >> 29; h *= XP3; h ^= h >> 32;
    return h;
}

/* XXH64 of every chunk, as wmo_checksum does for the CRC. */
int wmo_checksum_xxh64(const uint8_t* cache, uint64_t nbytes, uint32_t chunk_bytes, uint64_t seed, uint64_t* out)
{
    if (!cache || !out || !args_ok(nbytes, chunk_bytes)) return WMO_ERR_ARG;
    uint64_t nc = wmo_num_chunks(nbytes, chunk_bytes);
    for (uint64_t c = 0; c < nc; c++) out[c] = wmo_xxh64(cache + c * chunk_bytes, chunk_len(nbytes, chunk_bytes, c), seed);
    return WMO_OK;
}

/* Position of element e (0..255, memory order) inside its group's coded order.
 * The group's 512 bytes are four rows of 128 bytes; element e sits in row
 * r = e / 64 at 32-bit word l = (e % 64) / 2, half h = e % 2.  Coded order takes
 * the same word of all four rows together: k = 8 l + 2 r + h. */
static uint32_t coded_pos(uint32_t e)
{
    uint32_t r = e / 64u, l = (e % 64u) / 2u, h = e % 2u;
    return 8u * l + 2u * r + h;
}

static uint32_t desc_check(uint32_t base, uint32_t w)
{
    return ((base & 0xFu) ^ (base >> 4) ^ w ^ 0x5u) & 0xFu;
}

/* Encode one full tile (16384 bytes = 8192 bf16 elements, 32 groups of 256).
 * Returns the encoded length and the tile-table entry.
 *
 * Per element v (little-endian u16): E = (v >> 7) & 0xFF is the bf16 exponent,
 * SM = ((v & 0x7F) << 1) | (v >> 15) is mantissa and sign (rotl16(v,1) split into
 * its high and low byte).  Per group: base = min E, range = max E - base,
 * w = bit length of range (0..8).  S = sum of w over the 32 groups.
 *   S <= 253: PACK tile of 8256 + 32 S bytes (< 16384):
 *       desc[32]  u16 each: base | w << 8 | chk << 12
 *       SM[8192]  byte 256 g + k = SM of the element with coded position k in group g
 *       Epack_g   32 w_g bytes holding d = E - base, split into bit planes.  w = 8: one
 *                 plane of 8 bits per element.  Otherwise the planes present are, in this
 *                 order, a 4-bit plane (128 bytes) if w & 4, a 2-bit plane (64 bytes) if
 *                 w & 2, a 1-bit plane (32 bytes) if w & 1; they take consecutive bits of d
 *                 starting at bit 0 (w = 7: bits 0-3, 4-5, 6; w = 5: bits 0-3, 4).  Inside a
 *                 p-bit plane, viewed as an LSB-first bit string, the element with coded
 *                 position k occupies bits [k p, (k+1) p).
 *   else: RAW tile, the 16384 bytes verbatim.
 */

/* Bit planes of a group of width w, in stored order: plane sizes in bits per element. */
static int plane_widths(uint32_t w, uint32_t p[3])
{
    int n = 0;
    if (w == 8u) { p[n++] = 8u; return n; }
    if (w & 4u) p[n++] = 4u;
    if (w & 2u) p[n++] = 2u;
    if (w & 1u) p[n++] = 1u;
    return n;
}

/* ------------------------------------------------- ENT tiles (option) ---
 * Entropy-coded exponents (the variant of the codec the paper measured codes the exponent
 * plane with an entropy coder; Section 6.4).  An image that sets header flags bit 2 stores a
 * full tile as an ENT tile, a PACK tile or raw, whichever is shortest; the sign-mantissa plane
 * of an ENT tile is the one of a PACK tile.
 *
 * A tile is eight shares of 16 rows (row = 128 bytes = 64 elements).  Share s has 32 strands;
 * strand l holds the 32 elements at 32-bit word l of the share's rows, row after row, low half
 * first: element i of the strand is tile element 64 (16 s + i / 2) + 2 l + i % 2.
 *
 *   anchor_s = (sum of the share's 1024 exponents + 512) >> 10      (the rounded mean)
 *   u = E - anchor_s is coded with a fixed prefix code; the bits of a codeword are listed in
 *   the order they are written, and a strand is an LSB-first bit string:
 *        u:   0    +1    -1    -2     +2     -3     -4      -5       +3        -6
 *      bits:  00   10    01    1100   1110   1101   11110   111110   1111110   11111110
 *      any other u: 11111111 followed by the eight bits of E itself, low bit first (16 bits)
 *   (as numbers, first bit = bit 0: 0, 1, 2, 3, 7, 11, 15, 31, 63, 127, 255 | E << 8).
 *
 * A strand's bit string is its 32 codewords one after the other (64 to 512 bits).  A share's
 * stream is its 32 strands' strings one after the other, strand 0 first, with no gaps, written
 * LSB-first into 32-bit little-endian words and zero-filled to a whole word.  The length of
 * every strand, minus 64, is stored in one byte, so that a reader can start on all strands at
 * once; a tile with a strand longer than 319 bits is not stored in this form.
 *
 *   ENT tile:  anchor[8] u8 | words[8] u16 (32-bit words in each share's stream) | 40 zero bytes
 *              SM[8192] as in a PACK tile | bits[8][32] u8 (strand lengths - 64) |
 *              the eight streams | zero fill to a multiple of 32
 *   entry = 0x8000 | length / 32 (the length is below 16384 whenever the form is used).
 */
static const int      ent_sym[10]  = {0, 1, -1, -2, 2, -3, -4, -5, 3, -6};
static const uint32_t ent_len[10]  = {2, 2, 2, 4, 4, 4, 5, 6, 7, 8};
static const uint32_t ent_bits[10] = {0, 1, 2, 3, 7, 11, 15, 31, 63, 127};

#define WMO_ENT_FIXED (64u + 8192u + 256u)      /* header, sign-mantissa plane, strand lengths */
#define WMO_ENT_MAX_STRAND 319u

static uint32_t ent_elem(uint32_t share, uint32_t strand, uint32_t i)
{
    return 64u * (16u * share + i / 2u) + 2u * strand + i % 2u;
}

static void ent_codeword(uint32_t E, uint32_t anchor, uint32_t* bits, uint32_t* len)
{
    int u = (int)E - (int)anchor;
    for (int k = 0; k < 10; k++)
        if (u == ent_sym[k]) { *bits = ent_bits[k]; *len = ent_len[k]; return; }
    *bits = 255u | (E << 8);
    *len = 16u;
}

/* `n` bits (n <= 32) from bit `at` on of the LSB-first bit string `p` of `nbits` bits; bits
 * beyond the end read as zero. */
static uint32_t get_bits(const uint8_t* p, uint64_t nbits, uint64_t at, uint32_t n)
{
    uint64_t v = 0, first = at / 8u, nbytes = nbits / 8u;       /* (nbits is a whole number of bytes) */
    for (uint32_t k = 0; k < 5; k++)
        if (first + k < nbytes) v |= (uint64_t)p[first + k] << (8u * k);
    v >>= at % 8u;
    return (uint32_t)(n >= 32u ? v : v & ((1ull << n) - 1ull));
}

/* Length and symbol of the codeword at the low end of `buf` (16 bits suffice).  Returns the
 * length; *E receives the exponent. */
static uint32_t ent_parse(uint32_t buf, uint32_t anchor, uint32_t* E)
{
    for (int k = 0; k < 10; k++)
        if ((buf & ((1u << ent_len[k]) - 1u)) == ent_bits[k]) {
            *E = (uint32_t)((int)anchor + ent_sym[k]) & 0xFFu;
            return ent_len[k];
        }
    *E = (buf >> 8) & 0xFFu;
    return 16u;
}

/* Encode the exponents of one tile as ENT streams.  Returns the tile's length in bytes (a
 * multiple of 32), or WMO_TILE when the form cannot hold the tile (a strand of more than 319 bits)
 * or is not shorter than the tile itself; `out` is then not to be used.  `out` must hold
 * 2 * WMO_TILE bytes. */
static uint32_t encode_ent_tile(const uint8_t* src, uint8_t* out)
{
    memset(out, 0, 2 * WMO_TILE);
    uint8_t* stream = out + WMO_ENT_FIXED;
    uint32_t words_total = 0;
    for (uint32_t s = 0; s < 8; s++) {
        uint32_t sum = 0;
        for (uint32_t e = 0; e < 1024; e++) sum += (get16(src + 2u * (1024u * s + e)) >> 7) & 0xFFu;
        uint32_t anchor = (sum + 512u) >> 10;
        out[s] = (uint8_t)anchor;
        uint64_t at = 0;                         /* bits of the share's stream written so far */
        uint8_t* sp = stream + 4u * words_total;
        for (uint32_t l = 0; l < 32; l++) {
            uint64_t start = at;
            for (uint32_t i = 0; i < 32; i++) {
                uint32_t E = (get16(src + 2u * ent_elem(s, l, i)) >> 7) & 0xFFu, cw, len;
                ent_codeword(E, anchor, &cw, &len);
                for (uint32_t b = 0; b < len; b++, at++)
                    if ((cw >> b) & 1u) sp[at / 8u] |= (uint8_t)(1u << (at % 8u));
            }
            if (at - start > WMO_ENT_MAX_STRAND) return WMO_TILE;
            out[64u + 8192u + 32u * s + l] = (uint8_t)(at - start - 64u);
        }
        uint32_t words = (uint32_t)((at + 31u) / 32u);
        put16(out + 8 + 2u * s, words);
        words_total += words;
        if (WMO_ENT_FIXED + 4u * words_total >= WMO_TILE) return WMO_TILE;
    }
    uint32_t len = (WMO_ENT_FIXED + 4u * words_total + 31u) & ~31u;
    /* sign-mantissa plane: the PACK tile's */
    for (uint32_t g = 0; g < WMO_GROUPS_PER_TILE; g++)
        for (uint32_t e = 0; e < WMO_GROUP_ELEMS; e++) {
            uint32_t v = get16(src + 2u * (g * WMO_GROUP_ELEMS + e));
            out[64u + 256u * g + coded_pos(e)] = (uint8_t)(((v & 0x7Fu) << 1) | (v >> 15));
        }
    return len < WMO_TILE ? len : WMO_TILE;
}

/* Header of an ENT tile against its table entry: every share's word count within what 32
 * strands of 64 to 319 bits can need, and the length they add up to.  Returns 0 when it fits. */
static int ent_header_bad(const uint8_t* in, uint32_t entry)
{
    uint32_t total = 0;
    for (uint32_t s = 0; s < 8; s++) {
        uint32_t c = get16(in + 8 + 2u * s);
        if (c < 64u || c > 319u) return 1;
        total += c;
    }
    return ((WMO_ENT_FIXED + 4u * total + 31u) / 32u) != (entry & 0x7FFFu);
}

/* Read the eight streams of an ENT tile whose header fits (`entry`: its tile-table entry).  With
 * dst != NULL the tile is written there.  Returns 0 when every byte of the tile is accounted for:
 * the strand lengths of every share add up to its word count, every strand's 32 codewords take
 * exactly its length, the fill bits of every stream's last word are zero, every anchor is the
 * rounded mean of the exponents its share decodes to (what the encoder writes), the 40 spare
 * header bytes and the fill behind the last stream are zero; 1 otherwise.  With these no bit of
 * an ENT tile can change without the tile being refused or the decoded bytes changing. */
static int decode_ent_tile(const uint8_t* in, uint8_t* dst, uint32_t entry)
{
    const uint8_t* stream = in + WMO_ENT_FIXED;
    int bad = 0;
    uint32_t words_total = 0;
    for (uint32_t i = 24; i < 64; i++)
        if (in[i]) bad = 1;
    for (uint32_t s = 0; s < 8; s++) {
        uint32_t anchor = in[s], words = get16(in + 8 + 2u * s), esum = 0;
        uint64_t nbits = 32ull * words, at = 0;
        for (uint32_t l = 0; l < 32; l++) {
            uint64_t want = 64u + in[64u + 8192u + 32u * s + l], start = at;
            uint64_t p = at;
            for (uint32_t i = 0; i < 32; i++) {
                uint32_t E, len = ent_parse(get_bits(stream, nbits, p, 16), anchor, &E);
                p += len;
                esum += E;
                if (dst) {
                    uint32_t e = ent_elem(s, l, i);
                    uint32_t SM = in[64u + 256u * (e / 256u) + coded_pos(e % 256u)];
                    put16(dst + 2u * e, ((SM & 1u) << 15) | (E << 7) | (SM >> 1));
                }
            }
            if (p - start != want) bad = 1;      /* the codewords take exactly the length that is written down */
            at = start + want;                   /* the next strand starts where the lengths say */
        }
        if ((at + 31u) / 32u != words) bad = 1;
        for (uint64_t b = at; b < nbits; b++)    /* the fill bits of the stream's last word are zero */
            if (get_bits(stream, nbits, b, 1)) bad = 1;
        if (((esum + 512u) >> 10) != anchor) bad = 1;
        stream += 4u * words;
        words_total += words;
    }
    for (uint32_t i = WMO_ENT_FIXED + 4u * words_total; i < 32u * (entry & 0x7FFFu); i++)
        if (in[i]) bad = 1;
    return bad;
}

#define WMO_OPT_ZERO_TILES 1   /* encoder options */
#define WMO_OPT_ENTROPY 2
#define WMO_OPT_ENT_ONLY 4

static uint32_t encode_full_tile(const uint8_t* src, uint8_t* out, uint32_t* entry, int options)
{
    uint32_t base[WMO_GROUPS_PER_TILE], w[WMO_GROUPS_PER_TILE], S = 0;
    /* option: a tile whose 16384 bytes are all zero (unused allocation) has entry 1 and no payload */
    if (options & WMO_OPT_ZERO_TILES) {
        uint32_t any = 0;
        for (uint32_t i = 0; i < WMO_TILE; i++) any |= src[i];
        if (!any) { *entry = 1u; return 0; }
        /* the same option: a tile whose 8192 elements all hold one (non-zero) value is entry 2 and
         * 32 bytes of payload, the value first (little-endian u16), then 30 zero bytes */
        uint32_t v0 = get16(src), same = 1;
        for (uint32_t e = 1; e < 8192u; e++) if (get16(src + 2u * e) != v0) { same = 0; break; }
        if (same) { memset(out, 0, 32); put16(out, v0); *entry = 2u; return 32u; }
    }
    /* option: entropy-coded exponents.  The tile is stored in the shortest of the three forms
     * (ENT, PACK, raw); on equal lengths PACK goes before ENT and a coded form before raw, so
     * an image with the option is never longer than one without.  (WMO_OPT_ENT_ONLY, a switch
     * of this oracle alone, leaves PACK out: the tests use it to pin the ENT coder by itself.) */
    uint8_t ent_buf[2 * WMO_TILE];
    uint32_t ent_len = WMO_TILE;
    if (options & WMO_OPT_ENTROPY) {
        ent_len = encode_ent_tile(src, ent_buf);
        if (options & WMO_OPT_ENT_ONLY) {
            if (ent_len < WMO_TILE) { memcpy(out, ent_buf, ent_len); *entry = 0x8000u | (ent_len / 32u); return ent_len; }
            memcpy(out, src, WMO_TILE);
            *entry = 512u;
            return WMO_TILE;
        }
    }
    for (uint32_t g = 0; g < WMO_GROUPS_PER_TILE; g++) {
        uint32_t mn = 255, mx = 0;
        for (uint32_t e = 0; e < WMO_GROUP_ELEMS; e++) {
            uint32_t v = get16(src + 2u * (g * WMO_GROUP_ELEMS + e));
            uint32_t E = (v >> 7) & 0xFFu;
            if (E < mn) mn = E;
            if (E > mx) mx = E;
        }
        uint32_t range = mx - mn, bits = 0;
        while (range) { bits++; range >>= 1; }
        base[g] = mn; w[g] = bits; S += bits;
    }
    {
        uint32_t pack_len = S <= 253u ? 8256u + 32u * S : WMO_TILE;
        if (ent_len < pack_len) { memcpy(out, ent_buf, ent_len); *entry = 0x8000u | (ent_len / 32u); return ent_len; }
    }
    if (S > 253u) {
        memcpy(out, src, WMO_TILE);
        *entry = 512u;
        return WMO_TILE;
    }
    uint32_t len = 8256u + 32u * S;
    memset(out, 0, len);
    uint8_t* sm = out + 64;
    uint8_t* ep = out + 64 + 8192;
    for (uint32_t g = 0; g < WMO_GROUPS_PER_TILE; g++) {
        put16(out + 2u * g, base[g] | (w[g] << 8) | (desc_check(base[g], w[g]) << 12));
        for (uint32_t e = 0; e < WMO_GROUP_ELEMS; e++) {
            uint32_t v = get16(src + 2u * (g * WMO_GROUP_ELEMS + e));
            uint32_t E = (v >> 7) & 0xFFu;
            uint32_t SM = ((v & 0x7Fu) << 1) | (v >> 15);
            uint32_t k = coded_pos(e);
            sm[256u * g + k] = (uint8_t)SM;
            uint32_t d = E - base[g];
            uint32_t pw[3], lo = 0;                  /* lo: first bit of d the plane takes */
            int np = plane_widths(w[g], pw);
            uint8_t* plane = ep;
            for (int q = 0; q < np; q++) {
                for (uint32_t j = 0; j < pw[q]; j++) {
                    uint32_t bit = k * pw[q] + j;
                    if ((d >> (lo + j)) & 1u) plane[bit / 8u] |= (uint8_t)(1u << (bit % 8u));
                }
                lo += pw[q];
                plane += 32u * pw[q];
            }
        }
        ep += 32u * w[g];
    }
    *entry = 258u + S;
    return len;
}

/* WM1 wire image (all integers little-endian):
 *
 *   header[64] | chunk_dir[16 n_chunks] | tile_tab[2 n_tiles] | zero pad to a
 *   multiple of 32 (= meta_end) | payload
 *
 *   header:  0 "WMV1"   4 u16 version=1   6 u16 flags (bit0: a dirty mask was given;
 *            bit1: ZERO tile option; bit2: ENT tiles may occur)
 *            8 u64 nbytes   16 u32 chunk_bytes   20 u32 tile_bytes=16384
 *           24 u32 n_chunks 28 u32 n_present     32 u64 payload_bytes
 *           40 u64 wire_len 48 u32 cache_crc     52 u32 meta_crc   56 8 zero bytes
 *   chunk_dir[c]: u64 payload_off | u32 enc_len | u32 crc
 *   tile_tab[t] : 0 absent | 1 ZERO full tile (all bytes zero, no payload) |
 *                 2 CONST full tile (all 8192 elements equal and not zero; payload = the
 *                 value, u16, and 30 zero bytes; entries 1 and 2 only with flags bit1) |
 *                 258..511 PACK of 32*value bytes | 512 RAW full tile |
 *                 0x8000 | n, n = 259..511: ENT of 32 n bytes | 0xFFFF RAW partial tail tile
 *   payload: encoded tiles of present chunks in ascending order, no padding.
 *
 * cache_crc is the CRC32C of the whole cache, obtained by combining the directory
 * CRCs (for an absent chunk the caller's crc_inout[c] is trusted).  meta_crc is the
 * CRC32C of wire[0, meta_end) with its own four bytes taken as zero.
 *
 * `dirty` may be NULL (every chunk present).  crc_inout[c] is written for present
 * chunks and read for absent ones.  Returns the status also stored in *res.
 */
#define WMO_FLAG_MASKED 1u       /* header flags: a dirty mask was given             */
#define WMO_FLAG_ZERO_TILES 2u   /* header flags: all-zero tiles are table entries   */
#define WMO_FLAG_ENTROPY 4u      /* header flags: ENT tiles may occur                */

int wmo_encode_opt(const uint8_t* cache, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
                   uint32_t* crc_inout, uint8_t* wire, uint64_t wire_cap, int options, wmo_result* res);

int wmo_encode(const uint8_t* cache, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
               uint32_t* crc_inout, uint8_t* wire, uint64_t wire_cap, wmo_result* res)
{
    return wmo_encode_opt(cache, nbytes, chunk_bytes, dirty, crc_inout, wire, wire_cap, 0, res);
}

/* options: WMO_OPT_ZERO_TILES (tile table entry 1; header flags bit 1), WMO_OPT_ENTROPY (ENT tiles
 * where they are shorter than PACK tiles; header flags bit 2). */
int wmo_encode_opt(const uint8_t* cache, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
                   uint32_t* crc_inout, uint8_t* wire, uint64_t wire_cap, int options, wmo_result* res)
{
    if (!cache || !crc_inout || !wire || !res || !args_ok(nbytes, chunk_bytes)) return WMO_ERR_ARG;
    uint64_t nc = wmo_num_chunks(nbytes, chunk_bytes), nt = wmo_num_tiles(nbytes);
    uint64_t meta_end = wmo_meta_end(nbytes, chunk_bytes);
    if (wire_cap < meta_end) return WMO_ERR_ARG;
    memset(res, 0, sizeof *res);
    memset(wire, 0, meta_end);

    uint8_t* dir = wire + WMO_HEADER;
    uint8_t* tab = dir + 16u * nc;
    uint8_t* tile_buf = (uint8_t*)malloc(2 * WMO_TILE);     /* an ENT attempt may run past the tile size */
    uint64_t off = 0;              /* payload bytes emitted so far */
    uint32_t n_present = 0, cache_crc = 0;
    int overflow = 0;

    for (uint64_t c = 0; c < nc; c++) {
        uint64_t clen = chunk_len(nbytes, chunk_bytes, c);
        const uint8_t* cp = cache + c * chunk_bytes;
        int present = dirty ? (dirty[c] != 0) : 1;
        uint64_t enc_len = 0;
        if (present) {
            n_present++;
            crc_inout[c] = wmo_crc32c(cp, clen);
            for (uint64_t o = 0; o < clen; o += WMO_TILE) {
                uint64_t t = (c * chunk_bytes + o) / WMO_TILE;
                uint64_t tlen = clen - o < WMO_TILE ? clen - o : WMO_TILE;
                uint32_t entry, elen;
                if (tlen < WMO_TILE) { memcpy(tile_buf, cp + o, tlen); entry = 0xFFFFu; elen = (uint32_t)tlen; }
                else elen = encode_full_tile(cp + o, tile_buf, &entry, options);
                put16(tab + 2u * t, entry);
                if (!overflow && meta_end + off + enc_len + elen <= wire_cap)
                    memcpy(wire + meta_end + off + enc_len, tile_buf, elen);
                else
                    overflow = 1;
                enc_len += elen;
            }
        }
        put64(dir + 16u * c, off);
        put32(dir + 16u * c + 8, (uint32_t)enc_len);
        put32(dir + 16u * c + 12, crc_inout[c]);
        cache_crc = (c == 0) ? crc_inout[c] : wmo_crc_combine(cache_crc, crc_inout[c], clen);
        off += enc_len;
    }
    free(tile_buf);

    memcpy(wire, "WMV1", 4);
    put16(wire + 4, 1);
    put16(wire + 6, (dirty ? WMO_FLAG_MASKED : 0u) | ((options & WMO_OPT_ZERO_TILES) ? WMO_FLAG_ZERO_TILES : 0u) |
                        ((options & WMO_OPT_ENTROPY) ? WMO_FLAG_ENTROPY : 0u));
    put64(wire + 8, nbytes);
    put32(wire + 16, chunk_bytes);
    put32(wire + 20, WMO_TILE);
    put32(wire + 24, (uint32_t)nc);
    put32(wire + 28, n_present);
    put64(wire + 32, off);
    put64(wire + 40, meta_end + off);
    put32(wire + 48, cache_crc);
    put32(wire + 52, 0);
    put32(wire + 52, wmo_crc32c(wire, meta_end));
    (void)nt;

    res->status = overflow ? WMO_ERR_CAPACITY : WMO_OK;
    res->n_present = n_present;
    res->wire_len = meta_end + off;
    res->payload_bytes = off;
    res->cache_crc = cache_crc;
    return res->status;
}

/* -------------------------------------------------------- decode+verify --- */

static void fail(wmo_result* res, int status, uint32_t first, uint32_t count)
{
    res->status = status; res->first_bad_chunk = first; res->n_bad_chunks = count;
}

/* Decode one PACK tile whose descriptors were already validated. */
static void decode_pack_tile(const uint8_t* in, uint8_t* dst)
{
    const uint8_t* sm = in + 64;
    const uint8_t* ep = in + 64 + 8192;
    for (uint32_t g = 0; g < WMO_GROUPS_PER_TILE; g++) {
        uint32_t desc = get16(in + 2u * g);
        uint32_t base = desc & 0xFFu, w = (desc >> 8) & 0xFu;
        for (uint32_t e = 0; e < WMO_GROUP_ELEMS; e++) {
            uint32_t k = coded_pos(e), d = 0;
            uint32_t pw[3], lo = 0;
            int np = plane_widths(w, pw);
            const uint8_t* plane = ep;
            for (int q = 0; q < np; q++) {
                for (uint32_t j = 0; j < pw[q]; j++) {
                    uint32_t bit = k * pw[q] + j;
                    d |= (uint32_t)((plane[bit / 8u] >> (bit % 8u)) & 1u) << (lo + j);
                }
                lo += pw[q];
                plane += 32u * pw[q];
            }
            uint32_t E = (base + d) & 0xFFu;
            uint32_t SM = sm[256u * g + k];
            uint32_t v = ((SM & 1u) << 15) | (E << 7) | (SM >> 1);
            put16(dst + 2u * (g * WMO_GROUP_ELEMS + e), v);
        }
        ep += 32u * w;
    }
}

/* Checks, in this order; the first failing step gives the status:
 *  1 header fields against the call's arguments and wire_len        -> FORMAT
 *  2 meta_crc                                                       -> META_CRC
 *  3 directory / tile-table structure                               -> STRUCT
 *  4 every PACK tile, in tile order: descriptors (w <= 8, check nibble) -> DESC,
 *    then 258 + sum w equals the tile entry                         -> STRUCT;
 *    every ENT tile: stream counts in range and adding up to the entry -> STRUCT,
 *    then each stream used up exactly by its 1024 codewords, fill bits zero, anchors the
 *    rounded means of what they decode, spare header bytes and end fill zero -> DESC;
 *    every CONST tile: the 30 bytes behind the value zero            -> DESC
 *    (status of the lowest failing tile; n_bad_chunks = chunks with a failing tile)
 *  5 decode; CRC32C of each decoded chunk equals its directory CRC  -> CHUNK_CRC
 *  6 absent chunk: dst_crc_inout[c] equals its directory CRC        -> STALE
 *  7 combination of all directory CRCs equals cache_crc             -> CACHE_CRC
 *  8 only then dst_crc_inout[c] <- crc for present chunks; status OK.
 * first_bad_chunk is the lowest chunk failing the failing step.  On any failure the
 * contents of dst are unspecified (bounded to [dst, dst+nbytes)) and dst_crc_inout
 * is unchanged; the caller must not install dst.
 */
int wmo_decode_verify_opt(const uint8_t* wire, uint64_t wire_len, uint8_t* dst, uint64_t nbytes,
                          uint32_t chunk_bytes, uint32_t* dst_crc_inout, int expect_entropy, wmo_result* res);

int wmo_decode_verify(const uint8_t* wire, uint64_t wire_len, uint8_t* dst, uint64_t nbytes,
                      uint32_t chunk_bytes, uint32_t* dst_crc_inout, wmo_result* res)
{
    return wmo_decode_verify_opt(wire, wire_len, dst, nbytes, chunk_bytes, dst_crc_inout, -1, res);
}

/* expect_entropy: -1 accepts both kinds of image; 0 / 1: a receiver that was told which codec
 * option the sender uses treats an image of the other kind as a format error (step 1). */
int wmo_decode_verify_opt(const uint8_t* wire, uint64_t wire_len, uint8_t* dst, uint64_t nbytes,
                          uint32_t chunk_bytes, uint32_t* dst_crc_inout, int expect_entropy, wmo_result* res)
{
    if (!wire || !dst || !dst_crc_inout || !res || !args_ok(nbytes, chunk_bytes)) return WMO_ERR_ARG;
    memset(res, 0, sizeof *res);
    uint64_t nc = wmo_num_chunks(nbytes, chunk_bytes), nt = wmo_num_tiles(nbytes);
    uint64_t meta_end = wmo_meta_end(nbytes, chunk_bytes);

    /* 1 */
    if (wire_len < WMO_HEADER || memcmp(wire, "WMV1", 4) != 0 || get16(wire + 4) != 1 ||
        get16(wire + 6) > 7 || (expect_entropy >= 0 && (int)((get16(wire + 6) >> 2) & 1u) != expect_entropy) ||
        get64(wire + 8) != nbytes || get32(wire + 16) != chunk_bytes ||
        get32(wire + 20) != WMO_TILE || get32(wire + 24) != nc || get64(wire + 40) != wire_len ||
        wire_len < meta_end || get64(wire + 32) != wire_len - meta_end) {
        fail(res, WMO_ERR_FORMAT, 0, 0);
        return res->status;
    }
    uint64_t payload_bytes = get64(wire + 32);
    int zero_ok = (get16(wire + 6) & 2u) != 0;      /* entry 1 is legal only in an image that declares the option */
    int ent_on = (get16(wire + 6) & 4u) != 0;       /* ENT entries only in an image that declares the option */
    uint32_t n_present_hdr = get32(wire + 28);
    uint32_t cache_crc_hdr = get32(wire + 48);
    res->wire_len = wire_len; res->payload_bytes = payload_bytes;
    res->n_present = n_present_hdr; res->cache_crc = cache_crc_hdr;

    /* 2 */
    {
        uint8_t* meta = (uint8_t*)malloc(meta_end);
        memcpy(meta, wire, meta_end);
        put32(meta + 52, 0);
        uint32_t got = wmo_crc32c(meta, meta_end);
        free(meta);
        if (got != get32(wire + 52)) { fail(res, WMO_ERR_META_CRC, 0, 0); return res->status; }
    }

    const uint8_t* dir = wire + WMO_HEADER;
    const uint8_t* tab = dir + 16u * nc;
    const uint8_t* payload = wire + meta_end;

    /* 3 */
    {
        uint64_t run = 0; uint32_t present = 0, bad = 0, first = 0;
        for (uint64_t c = 0; c < nc; c++) {
            uint64_t clen = chunk_len(nbytes, chunk_bytes, c);
            uint64_t poff = get64(dir + 16u * c);
            uint32_t elen = get32(dir + 16u * c + 8);
            uint64_t t0 = c * (uint64_t)chunk_bytes / WMO_TILE, ntc = (clen + WMO_TILE - 1) / WMO_TILE;
            int ok = (poff == run);
            uint64_t sum = 0; int any = 0, all = 1;
            for (uint64_t i = 0; i < ntc; i++) {
                uint32_t e = get16(tab + 2u * (t0 + i));
                uint64_t tlen = clen - i * WMO_TILE < WMO_TILE ? clen - i * WMO_TILE : WMO_TILE;
                if (e == 0) { all = 0; continue; }
                any = 1;
                if (tlen < WMO_TILE) { if (e != 0xFFFFu) ok = 0; sum += tlen; }
                else if (e == 1u && zero_ok) sum += 0;     /* ZERO tile: full tiles only, no payload */
                else if (e == 2u && zero_ok) sum += 32u;   /* CONST tile: the value in 32 bytes of payload */
                else if (e >= 258u && e <= 512u) sum += 32u * (uint64_t)e;
                else if (ent_on && e >= (0x8000u | 259u) && e <= (0x8000u | 511u)) sum += 32u * (uint64_t)(e & 0x7FFFu);
                else ok = 0;
            }
            if (any && !all) ok = 0;                   /* a chunk is present as a whole or not at all */
            if (any) present++;
            if (sum != elen) ok = 0;
            if (!ok) { if (!bad) first = (uint32_t)c; bad++; }
            run += elen;
        }
        if (!bad && (run != payload_bytes || present != n_present_hdr)) { bad = 1; first = 0; }
        if (bad) { fail(res, WMO_ERR_STRUCT, first, bad); return res->status; }
    }

    /* 4 */
    {
        int status = WMO_OK; uint32_t first = 0, bad = 0;
        for (uint64_t c = 0; c < nc; c++) {
            uint64_t clen = chunk_len(nbytes, chunk_bytes, c);
            uint64_t t0 = c * (uint64_t)chunk_bytes / WMO_TILE, ntc = (clen + WMO_TILE - 1) / WMO_TILE;
            uint64_t off = get64(dir + 16u * c);
            int chunk_bad = 0;
            for (uint64_t i = 0; i < ntc; i++) {
                uint32_t e = get16(tab + 2u * (t0 + i));
                if (e == 0) break;
                uint64_t tlen = (e == 0xFFFFu) ? clen - i * WMO_TILE : (e == 1u) ? 0 : (e == 2u) ? 32u : 32u * (uint64_t)(e & 0x7FFFu);
                if (e != 0xFFFFu && (e & 0x8000u)) {
                    /* ENT tile: the header against the entry -> STRUCT, then every stream must be used up exactly -> DESC */
                    int tile_status = WMO_OK;
                    if (ent_header_bad(payload + off, e)) tile_status = WMO_ERR_STRUCT;
                    else if (decode_ent_tile(payload + off, NULL, e)) tile_status = WMO_ERR_DESC;
                    if (tile_status != WMO_OK) {
                        chunk_bad = 1;
                        if (status == WMO_OK) status = tile_status;
                    }
                } else if (e == 2u) {
                    /* CONST tile: the 30 bytes behind the value are zero -> DESC */
                    for (uint32_t k = 2; k < 32; k++)
                        if (payload[off + k]) { chunk_bad = 1; if (status == WMO_OK) status = WMO_ERR_DESC; break; }
                } else if (e >= 258u && e <= 511u) {
                    const uint8_t* in = payload + off;
                    int tile_status = WMO_OK; uint32_t S = 0;
                    for (uint32_t g = 0; g < WMO_GROUPS_PER_TILE; g++) {
                        uint32_t desc = get16(in + 2u * g);
                        uint32_t base = desc & 0xFFu, w = (desc >> 8) & 0xFu, chk = desc >> 12;
                        if (w > 8u || chk != desc_check(base, w)) tile_status = WMO_ERR_DESC;
                        S += w;
                    }
                    if (tile_status == WMO_OK && 258u + S != e) tile_status = WMO_ERR_STRUCT;
                    if (tile_status != WMO_OK) {
                        chunk_bad = 1;
                        if (status == WMO_OK) status = tile_status;
                    }
                }
                off += tlen;
            }
            if (chunk_bad) { if (!bad) first = (uint32_t)c; bad++; }
        }
        if (bad) { fail(res, status, first, bad); return res->status; }
    }

    /* 5 */
    {
        uint32_t first = 0, bad = 0;
        for (uint64_t c = 0; c < nc; c++) {
            uint64_t clen = chunk_len(nbytes, chunk_bytes, c);
            uint64_t t0 = c * (uint64_t)chunk_bytes / WMO_TILE, ntc = (clen + WMO_TILE - 1) / WMO_TILE;
            uint64_t off = get64(dir + 16u * c);
            if (get16(tab + 2u * t0) == 0) continue;
            uint8_t* out = dst + c * (uint64_t)chunk_bytes;
            for (uint64_t i = 0; i < ntc; i++) {
                uint32_t e = get16(tab + 2u * (t0 + i));
                uint64_t tlen = (e == 0xFFFFu) ? clen - i * WMO_TILE : (e == 1u) ? 0 : (e == 2u) ? 32u : 32u * (uint64_t)(e & 0x7FFFu);
                if (e == 1u) memset(out + i * WMO_TILE, 0, WMO_TILE);
                else if (e == 2u) { for (uint32_t k = 0; k < 8192u; k++) memcpy(out + i * WMO_TILE + 2u * k, payload + off, 2); }
                else if (e != 0xFFFFu && (e & 0x8000u)) decode_ent_tile(payload + off, out + i * WMO_TILE, e);
                else if (e == 512u || e == 0xFFFFu) memcpy(out + i * WMO_TILE, payload + off, tlen);
                else decode_pack_tile(payload + off, out + i * WMO_TILE);
                off += tlen;
            }
            if (wmo_crc32c(out, clen) != get32(dir + 16u * c + 12)) { if (!bad) first = (uint32_t)c; bad++; }
        }
        if (bad) { fail(res, WMO_ERR_CHUNK_CRC, first, bad); return res->status; }
    }

    /* 6 */
    {
        uint32_t first = 0, bad = 0;
        for (uint64_t c = 0; c < nc; c++) {
            uint64_t t0 = c * (uint64_t)chunk_bytes / WMO_TILE;
            if (get16(tab + 2u * t0) != 0) continue;
            if (dst_crc_inout[c] != get32(dir + 16u * c + 12)) { if (!bad) first = (uint32_t)c; bad++; }
        }
        if (bad) { fail(res, WMO_ERR_STALE, first, bad); return res->status; }
    }

    /* 7 */
    {
        uint32_t acc = 0;
        for (uint64_t c = 0; c < nc; c++) {
            uint32_t crc = get32(dir + 16u * c + 12);
            acc = (c == 0) ? crc : wmo_crc_combine(acc, crc, chunk_len(nbytes, chunk_bytes, c));
        }
        if (acc != cache_crc_hdr) { fail(res, WMO_ERR_CACHE_CRC, 0, 0); return res->status; }
    }

    /* 8 */
    for (uint64_t c = 0; c < nc; c++) {
        uint64_t t0 = c * (uint64_t)chunk_bytes / WMO_TILE;
        if (get16(tab + 2u * t0) != 0) dst_crc_inout[c] = get32(dir + 16u * c + 12);
    }
    (void)nt;
    res->status = WMO_OK;
    return WMO_OK;
}
