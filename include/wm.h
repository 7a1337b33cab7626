/*
 * wm.h - C ABI of the B200 data path of an exact-state session mover.
 *
 * The library turns a GPU-resident bf16 attention cache into a verified wire image and
 * back: per-chunk checksums, a dirty-chunk diff against the previous snapshot, a lossless
 * encode into one contiguous buffer, and a decode that re-fingerprints the decoded bytes
 * so that the destination is bit-identical to the source or is not installed.
 *
 * Conventions for every call
 *   - Pointers marked [dev] are device memory owned by the caller; the library allocates
 *     nothing per call and keeps no per-session state.  Constant tables are uploaded once
 *     per device on first use (that first call may synchronise the device).
 *   - `stream` is a cudaStream_t passed as void*.  All work is enqueued on it; no call
 *     synchronises.  Data-dependent outcomes arrive in `*result` [dev] on the stream.
 *   - The return value is host-side and synchronous: WM_ERR_ARG for a bad argument
 *     (null pointer, nbytes == 0, chunk_bytes not a multiple of 16384 or above 2^30, a
 *     cache / wire / dst pointer that is not 16-byte aligned, a workspace that is too
 *     small or not 16-byte aligned, wire_cap below the metadata size), WM_ERR_CUDA for
 *     a launch failure, else WM_OK.
 *   - Calls that share a workspace must be ordered on one stream (or by events).
 *   - A call enqueues a short chain of kernels; all but the first are launched with
 *     programmatic stream serialization (they may start while their predecessor drains and
 *     wait inside before touching its results).  Work enqueued by the caller before or after
 *     a call keeps ordinary stream order.
 *   - All integers in the wire image are little-endian.  Tile = 16384 bytes, group = 256
 *     bf16 elements; n_chunks = ceil(nbytes / chunk_bytes), n_tiles = ceil(nbytes / 16384).
 */
#ifndef WM_H
#define WM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define WM_TILE_BYTES 16384u

typedef enum {
    WM_OK = 0,
    WM_ERR_ARG = -1,        /* host-side argument check                                  */
    WM_ERR_CAPACITY = -2,   /* encode: wire image does not fit wire_cap                  */
    WM_ERR_FORMAT = -3,     /* decode: header does not match the call                    */
    WM_ERR_META_CRC = -4,   /* decode: header / directory / tile table damaged           */
    WM_ERR_STRUCT = -5,     /* decode: directory and tile table disagree                 */
    WM_ERR_DESC = -6,       /* decode: a group descriptor is invalid                     */
    WM_ERR_CHUNK_CRC = -7,  /* decode: a decoded chunk does not have the source's CRC    */
    WM_ERR_STALE = -8,      /* decode: a chunk not shipped differs at the destination    */
    WM_ERR_CACHE_CRC = -9,  /* decode: directory CRCs do not combine to the cache CRC    */
    WM_ERR_TIMEOUT = -10,   /* a bounded device-side wait ran out (see wm_wait_budget_ms) */
    WM_ERR_CUDA = -11       /* CUDA runtime error on launch                              */
} wm_status;

/* Outcome of wm_encode / wm_decode_verify, written on the stream.  40 bytes. */
typedef struct {
    int32_t  status;           /* wm_status                                              */
    uint32_t first_bad_chunk;  /* lowest chunk failing the failing check (decode)        */
    uint32_t n_bad_chunks;     /* chunks failing that check (decode)                     */
    uint32_t n_present;        /* chunks carried by the wire image                       */
    uint64_t wire_len;         /* bytes of the wire image (encode: needed size)          */
    uint64_t payload_bytes;    /* wire_len minus metadata                                */
    uint32_t cache_crc;        /* CRC32C of the whole cache                              */
    uint32_t reserved;
} wm_result;

/* Geometry helpers (pure host arithmetic). */
uint64_t wm_num_chunks(uint64_t nbytes, uint32_t chunk_bytes);
uint64_t wm_num_tiles(uint64_t nbytes);
/* Size of header + chunk directory + tile table, rounded up to 32 bytes. */
uint64_t wm_meta_bytes(uint64_t nbytes, uint32_t chunk_bytes);
/* Worst-case wire size (every tile stored raw): wm_meta_bytes + nbytes. */
uint64_t wm_wire_bound(uint64_t nbytes, uint32_t chunk_bytes);
/* Scratch the calls below need for this geometry (one size fits all four). */
uint64_t wm_workspace_bytes(uint64_t nbytes, uint32_t chunk_bytes);

/*
 * wm_wait_budget_ms - upper bound of every device-side wait, in milliseconds.
 * Paper: fail-closed behaviour (Section 4.1: a move either completes verified or installs nothing).
 * The kernels wait in three places: for a bulk copy into shared memory, for the placement
 * scanner (encode: a tile's offset), and the scanner for the tiles' lengths.  Each wait is bounded
 * by time on the GPU's own clock, not by a number of polls, so a kernel that shares the GPU with
 * other work and is descheduled for a while is not mistaken for a failure, and a real failure
 * never turns into a hang: when the budget has passed the kernel gives up, withdraws the
 * remaining work, returns, and the call reports WM_ERR_TIMEOUT (the CUDA context stays usable and
 * the next call on the same workspace starts clean).  Default 2000 ms; process-wide, read by each
 * call when it is issued; 0 is taken as 1.
 */
void wm_wait_budget_ms(uint32_t ms);

/*
 * wm_workspace_status - device-side outcome of the last call that used this workspace.
 * wm_encode and the wm_decode_verify family report through their result record; wm_checksum,
 * wm_checksum_poly and wm_dirty_diff have none.  Their only device-side failure is a wait that
 * ran out (or, WM_ERR_CUDA, a kernel that did not get its shared memory); then the checksum calls
 * fill crc_out with zeros instead of delivering digests of data that never arrived, and this call
 * says why.  wm_dirty_diff has no device-side wait and always leaves WM_OK here.
 * Synchronous: copies one word from the workspace on `stream` and waits for the stream.
 *   workspace [dev] a workspace a call was issued with on `stream`; NULL: the built-in scratch
 *             of wm_checksum_noalloc on the current device
 * Returns WM_OK, WM_ERR_TIMEOUT, WM_ERR_CUDA (also when the copy itself fails), or, after a codec
 * call, what its result record says of WM_ERR_CAPACITY / WM_ERR_ARG.
 */
wm_status wm_workspace_status(const void* workspace, void* stream);

/*
 * wm_inject_stall - test hook for the give-up paths (the paper has no counterpart).
 * While on, calls issued by this process leave out what their bounded waits wait for: the encode
 * kernel's scanner returns at once (no tile ever gets its offset), the checksum and decode kernels
 * do not start their bulk copies.  Every wait then runs out after wm_wait_budget_ms and the call
 * ends in WM_ERR_TIMEOUT without a fault or a hang, which is what tests need to see the timeout
 * handling run (set a budget of a few tens of milliseconds first).  Off by default; never turn
 * it on in production.
 */
void wm_inject_stall(int on);

/*
 * wm_checksum - CRC32C of every chunk of the flat cache.
 * Paper: the verification plane (Section 6.5: per-chunk CRC, GF(2)-combined) and the
 * transfer / CRC-verify / rehydrate primitive (Section 4.1).  The polynomial is CRC32C
 * (reflected 0x82F63B78, init and final xor all ones; "123456789" -> 0xE3069283).
 *   cache     [dev] nbytes bytes, 16-byte aligned, read only
 *   crc_out   [dev] u32[n_chunks]; crc_out[c] = CRC32C(cache[c*chunk_bytes, min((c+1)*chunk_bytes, nbytes)))
 *   workspace [dev] wm_workspace_bytes() bytes, 16-byte aligned
 */
wm_status wm_checksum(const void* cache, uint64_t nbytes, uint32_t chunk_bytes,
                      uint32_t* crc_out, void* workspace, uint64_t workspace_bytes, void* stream);

/*
 * wm_checksum_poly - wm_checksum with the CRC polynomial as an argument.
 * Paper: the verification plane (Section 6.5) measures its chunk CRC with zlib's CRC-32 on the
 * CPU side, while the wire format of this library fixes CRC32C.  This call offers both for the
 * checksum step alone; wm_encode and wm_decode_verify always use CRC32C.
 *   polynomial  WM_POLY_CRC32C (the same as wm_checksum) or WM_POLY_ZLIB (reflected 0xEDB88320,
 *               init and final xor all ones; "123456789" -> 0xCBF43926, what zlib's crc32 returns);
 *               anything else returns WM_ERR_ARG and launches nothing
 * All other arguments, layouts and errors are those of wm_checksum.  The first WM_POLY_ZLIB
 * call on a device allocates and uploads that polynomial's tables (synchronous, once).
 */
#define WM_POLY_CRC32C 0
#define WM_POLY_ZLIB 1
wm_status wm_checksum_poly(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, int polynomial,
                           uint32_t* crc_out, void* workspace, uint64_t workspace_bytes, void* stream);

/*
 * wm_checksum_xxh64 - the 64-bit xxHash (XXH64) of every chunk, a checksum option beside the CRC.
 * Paper: the verification plane fingerprints chunks (Section 6.5); a non-cryptographic 64-bit hash
 * is the usual alternative where 32 bits are felt to be too few.  The values are those of the
 * published algorithm (seed 0, empty input: 0xEF46DB3751D8E999; "123456789": 0x8CB841DB40E6AE83).
 *   cache     [dev] nbytes bytes, 16-byte aligned, read only
 *   seed      the hash's seed, the same for every chunk
 *   hash_out  [dev] u64[n_chunks]; hash_out[c] = XXH64(cache[c*chunk_bytes, min((c+1)*chunk_bytes, nbytes)), seed)
 * No workspace.  Unlike a CRC, hashes of pieces cannot be combined, so there is no whole-cache
 * value and wm_encode / wm_decode_verify do not use this hash.  WM_ERR_ARG on a bad geometry.
 */
wm_status wm_checksum_xxh64(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, uint64_t seed,
                            uint64_t* hash_out, void* stream);

/*
 * wm_dirty_diff - which chunks changed since the previous snapshot.
 * Paper: live pre-copy (Appendix G: round 0 ships every chunk, each later round the dirty
 * ones) and the measured dirty fraction per generation step (Section 3.3).  The compare is
 * exact (byte for byte), not a comparison of checksums.
 *   cache, prev   [dev] nbytes bytes each, 16-byte aligned, read only
 *   dirty_out     [dev] u8[n_chunks]: 1 iff any byte of the chunk differs, else 0
 *   dirty_idx_out [dev] u32[n_chunks] or NULL: ascending indices of dirty chunks in the
 *                 first *n_dirty_out entries (the rest is left untouched)
 *   n_dirty_out   [dev] u32: number of dirty chunks
 */
wm_status wm_dirty_diff(const void* cache, const void* prev, uint64_t nbytes, uint32_t chunk_bytes,
                        uint8_t* dirty_out, uint32_t* dirty_idx_out, uint32_t* n_dirty_out,
                        void* workspace, uint64_t workspace_bytes, void* stream);

/*
 * wm_encode - checksum + lossless encode into one contiguous wire image (format WM1).
 * Paper: the lossless codec inside the verified envelope (Section 6.4: bf16 plane split, the
 * exponent plane carries the redundancy, every round trip bit-exact, receipts bind to the
 * decoded bytes).  The paper fixes those properties, not a layout; WM1 is this library's:
 *
 *   header[64] | chunk_dir[16*n_chunks] | tile_tab[2*n_tiles] | zero pad to 32 | payload
 *   header: 0 "WMV1" | 4 u16 version=1 | 6 u16 flags (bit0: a dirty mask was given; bit1:
 *           the ZERO tile option, see wm_zero_tiles_enable; bit2: ENT tiles may occur, see
 *           wm_entropy_enable) |
 *           8 u64 nbytes | 16 u32 chunk_bytes | 20 u32 tile_bytes=16384 | 24 u32 n_chunks |
 *           28 u32 n_present | 32 u64 payload_bytes | 40 u64 wire_len | 48 u32 cache_crc |
 *           52 u32 meta_crc (CRC32C of the metadata with this field as zero) | 56 zero[8]
 *   chunk_dir[c]: u64 payload_off | u32 enc_len | u32 crc
 *   tile_tab[t] (u16): 0 tile of an absent chunk | 1 ZERO tile: a full tile whose bytes are
 *           all zero, no payload (only in images with flags bit1) | 2 CONST tile: a full tile whose 8192
 *           elements all hold one non-zero value; payload = that value (u16) and 30 zero bytes
 *           (only in images with flags bit1) | 258..511 PACK tile of 32*value bytes
 *           | 512 RAW full tile | 0x8000 | n, n = 259..511: ENT tile of
 *           32*n bytes (only with flags bit2) | 0xFFFF RAW partial tail tile (nbytes mod 16384 bytes)
 *   payload: encoded tiles of present chunks in ascending order, no padding
 *   PACK tile (32 groups of 256 elements): desc[32] u16 (base | w<<8 | chk<<12,
 *           chk = (base&15) ^ (base>>4) ^ w ^ 5) | SM[8192] | Epack_0 .. Epack_31.
 *           Element v (u16): E = (v>>7)&0xFF, SM = ((v&0x7F)<<1) | (v>>15).  Per group
 *           base = min E, w = bit length of (max E - base); a tile packs iff sum w <= 253
 *           (length 8256 + 32*sum w), else it is stored raw.  Inside a group, element e
 *           (memory order) has coded position k = 8*((e%64)/2) + 2*(e/64) + (e%2); SM[256 g + k]
 *           is its SM byte.  Epack_g (32 w bytes) stores d = E - base as bit planes, in this
 *           order, each present iff w has that bit: for w < 8 a 4-bit plane (128 bytes), a
 *           2-bit plane (64 bytes), a 1-bit plane (32 bytes); for w = 8 one 8-bit plane (256
 *           bytes).  The planes take consecutive bits of d from bit 0 upwards (w = 7: bits
 *           0..3, 4..5, 6); element k sits at bits [k p, (k+1) p) of its p-bit plane, LSB first.
 *           The payload is limited to 32 GiB (WM_ERR_ARG beyond that).
 *
 *   dirty     [dev] u8[n_chunks] or NULL (NULL = every chunk present: the fused
 *             checksum+encode of a full move)
 *   crc_inout [dev] u32[n_chunks]: written for present chunks, read (trusted) for absent ones
 *   wire      [dev] wire_cap bytes, 16-byte aligned; bytes beyond result->wire_len are unspecified
 *   result    [dev] status WM_OK, WM_ERR_CAPACITY (nothing is written past wire_cap;
 *             wire_len still reports the needed size) or WM_ERR_TIMEOUT
 * The image is canonical: equal inputs give equal bytes in [0, wire_len).
 */
wm_status wm_encode(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
                    uint32_t* crc_inout, void* wire, uint64_t wire_cap,
                    void* workspace, uint64_t workspace_bytes, wm_result* result, void* stream);

/*
 * wm_decode_verify - decode a wire image into the shadow buffer and verify it.
 * Paper: commit only on a matching fingerprint (Section 4.1, Sufficiency: a torn state can
 * never be installed; Table 1: migrate stages into a shadow slot, commit re-verifies).
 * Checks, in this order; the first failing step gives result->status:
 *   1 header fields equal the call's arguments and wire_len        WM_ERR_FORMAT
 *   2 meta_crc                                                     WM_ERR_META_CRC
 *   3 directory and tile table are consistent                      WM_ERR_STRUCT
 *   4 coded tiles in tile order; the status is that of the lowest failing tile.  PACK tile:
 *     descriptors valid (WM_ERR_DESC), then 258 + sum w equals the tile entry (WM_ERR_STRUCT).
 *     ENT tile (images with flags bit2): the eight word counts within 64..319 and adding up
 *     to the entry (WM_ERR_STRUCT), then every share's strand lengths adding up to its word
 *     count, every strand's 32 codewords taking exactly its length, the fill bits of every
 *     stream's last word zero, every anchor the rounded mean of the exponents its share decodes
 *     to, the header's 40 spare bytes and the fill behind the last stream zero (WM_ERR_DESC).  CONST tile (images with flags bit1): the 30 bytes behind the value zero
 *     (WM_ERR_DESC).  No byte of a coded tile is left unaccounted for
 *   5 CRC32C of every decoded chunk equals its directory CRC       WM_ERR_CHUNK_CRC
 *   6 absent chunk: dst_crc_inout[c] equals its directory CRC      WM_ERR_STALE
 *   7 the directory CRCs combine to header.cache_crc               WM_ERR_CACHE_CRC
 *   8 only then dst_crc_inout[c] <- crc for present chunks, status WM_OK
 * A bounded device-side wait that ran out (a bulk copy that did not arrive within
 * wm_wait_budget_ms) gives WM_ERR_TIMEOUT ahead of steps 4..7: the kernels failed, nothing can be
 * said about the image, nothing is installed.
 *   dst           [dev] nbytes bytes, 16-byte aligned: the SHADOW slot.  Present chunks are
 *                 written, absent chunks are left as they are.  On any failure its content is
 *                 unspecified (never written outside [dst, dst+nbytes)) and dst_crc_inout is
 *                 unchanged: the caller installs (swaps in) dst only on WM_OK.
 *   dst_crc_inout [dev] u32[n_chunks]: the receiver's CRC vector for the content of dst
 */
wm_status wm_decode_verify(const void* wire, uint64_t wire_len, void* dst, uint64_t nbytes,
                           uint32_t chunk_bytes, uint32_t* dst_crc_inout,
                           void* workspace, uint64_t workspace_bytes, wm_result* result, void* stream);

/*
 * wm_decode_verify_strict - verify first, write afterwards.
 * Paper: the all-or-nothing guarantee of a move (Section 1; Section 4.1: a torn state can never
 * be installed).  wm_decode_verify gives that guarantee
 * through the caller's shadow buffer; this call gives it for a buffer that is decoded into in
 * place (the live cache of a pre-copy round): a first pass unpacks and checksums the image
 * without storing a byte, the verdict is taken with all of wm_decode_verify's checks, and only
 * after WM_OK does a second pass unpack again and store.  On any failure dst and
 * dst_crc_inout are left exactly as they were.  Same arguments and result as
 * wm_decode_verify; the image is read twice, so the call takes about 1.7 times as long.  The
 * wire image must not change between the two passes (it is the caller's buffer on the
 * caller's stream).
 */
wm_status wm_decode_verify_strict(const void* wire, uint64_t wire_len, void* dst, uint64_t nbytes,
                                  uint32_t chunk_bytes, uint32_t* dst_crc_inout,
                                  void* workspace, uint64_t workspace_bytes, wm_result* result, void* stream);

/*
 * wm_zero_tiles_enable - encoder option: ship unused (all-zero) memory as table entries.
 * Paper: at least 19.4 % of the movable set is an allocation that no step writes or reads
 * (Section 3.3).  Read here as zero-filled memory: with the option on, a full tile of a
 * present chunk whose 16384 bytes are all zero gets tile_tab entry 1 and no payload bytes
 * (without it such a tile packs to 8256 bytes), and header flags bit1 is set.  Only the
 * all-zero byte pattern qualifies for entry 1 (minus zero and denormals are data).  A full tile
 * whose 8192 elements all hold one other value (a mask fill such as -Inf, say) gets entry 2 and
 * 32 bytes of payload: the value, little-endian, and 30 zero bytes.  The decoder accepts
 * entries 1 and 2 in images that declare the option, writes the zeros or the value, and
 * checksums them like any decoded tile.  Process-wide switch, off by default (the detection costs the encoder about
 * 3 % on caches without such tiles); applies to wm_encode and wm_encode_leaves.
 */
void wm_zero_tiles_enable(int on);

/*
 * wm_entropy_enable - codec option: entropy-coded exponents (ENT tiles beside PACK tiles).
 * Paper: the codec it measured entropy-codes the exponent plane inside the verified envelope
 * (Section 6.4); the bit-plane packing of the default format stops at a fixed number of bits
 * per group.  With the option on, wm_encode / wm_encode_leaves store every full tile of a present
 * chunk in the shortest of three forms, an ENT tile, a PACK tile or raw (PACK on a tie, a coded
 * form before raw), and set header flags bit 2: such an image is never longer than one without
 * the option.  The wm_decode_verify family then expects such images; a decode call whose option
 * differs from the image's flag returns WM_ERR_FORMAT.  The zero-tile option combines with this
 * one.  Process-wide, off by default; set it on both ends of a move before the calls are issued
 * (or use the calls that take their options as an argument).
 *
 * ENT tile (entry 0x8000 | length / 32 in the tile table; the length is below 16384):
 *   a tile is eight shares of 16 rows (row = 128 bytes); share s has 32 strands, strand l = the 32
 *   elements at 32-bit word l of the share's rows, row after row, low half first.
 *   anchor_s = (sum of the share's 1024 exponents + 512) >> 10.  u = E - anchor_s is coded
 *       u:    0   +1   -1   -2    +2    -3    -4     -5      +3       -6        other
 *       bits: 00  10   01   1100  1110  1101  11110  111110  1111110  11111110  11111111 + E (8 bits, low first)
 *   (in writing order).  A strand's bit string is its 32 codewords one after the other (64 to 512
 *   bits).  A share's stream is its 32 strands' strings one after the other, strand 0 first,
 *   without gaps, written LSB-first into 32-bit little-endian words and zero-filled to a whole
 *   word.  Every strand's length minus 64 is stored in a byte, so that a reader can start on
 *   all 32 strands of a share at once (lane l of a warp decodes strand l from the bit where the
 *   lengths before it add up to); a tile with a strand longer than 319 bits is not stored in
 *   this form.
 *   Layout: anchor[8] u8 | words[8] u16 (32-bit words per stream) | 40 zero bytes | SM[8192] as in
 *   a PACK tile | bits[8][32] u8 (strand lengths - 64) | the eight streams | zero fill to a
 *   multiple of 32 bytes.
 * Decode checks (step 4): word counts within 64..319 and adding up to the entry (else
 * WM_ERR_STRUCT); a share's strand lengths adding up to its word count, every strand's 32
 * codewords taking exactly its length, the fill bits of every stream's last word, the 40 spare
 * header bytes and the fill behind the last stream zero, every anchor equal to the formula above
 * applied to what its share decodes to (else WM_ERR_DESC).
 */
void wm_entropy_enable(int on);

/*
 * Leaf mode - the cache as the engine holds it: a list of tensors, not one buffer.
 * Paper: the mover flattens the live cache before the transfer and rehydrates it after
 * (Section 1 and Section 4.1: flatten, transfer, CRC-verify, rehydrate; Section 5: the movable
 * set is 420 tensors, 450 leaves with the control flags).  These two calls read the leaves
 * where they are and write the decoded bytes where they belong, which removes the flatten copy
 * before wm_encode and the rehydrate copy after wm_decode_verify (each a read and a write of
 * the whole cache).  The logical cache is the concatenation of the leaves in table order;
 * chunks, tiles and the wire image are exactly those of that concatenation, so the image is
 * byte for byte what wm_encode produces from the flattened buffer, and either decode call
 * accepts it.
 *   leaves    [dev] n_leaves entries (1..4096), read on the stream.  Every ptr is 16-byte
 *             aligned device memory; every nbytes is positive (any value: a two-byte flag
 *             between two tensors is fine) and the sizes add up to nbytes.  A table that
 *             breaks these rules gives result->status WM_ERR_ARG and nothing is read or
 *             written through it.
 * The 16 KiB tile grid lies over the concatenation, so a tile may begin anywhere inside a leaf.
 * A tile that lies inside one leaf moves by the same bulk copy as in the flat calls (from the
 * 16-byte boundary below its first byte, the kernel shifts by the remainder; decoded tiles whose
 * destination is not four-byte aligned take halfword or byte stores, which is slower: put odd-sized
 * leaves last where the order is yours to choose).  A tile that crosses a leaf boundary, at most
 * two per leaf, is read and written byte by byte through the table.  No byte outside the leaves
 * is ever read or written.
 * Everything else is as in wm_encode / wm_decode_verify.
 */
typedef struct {
    const void* ptr;     /* [dev] first byte of the leaf */
    uint64_t    nbytes;
} wm_leaf;

wm_status wm_encode_leaves(const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes,
                           const uint8_t* dirty, uint32_t* crc_inout, void* wire, uint64_t wire_cap,
                           void* workspace, uint64_t workspace_bytes, wm_result* result, void* stream);

wm_status wm_decode_verify_leaves(const void* wire, uint64_t wire_len, const wm_leaf* dst_leaves, uint32_t n_leaves,
                                  uint64_t nbytes, uint32_t chunk_bytes, uint32_t* dst_crc_inout,
                                  void* workspace, uint64_t workspace_bytes, wm_result* result, void* stream);

/*
 * wm_encode_opt / wm_decode_verify_opt - the codec calls with their options as an argument.
 * The switches above are process-wide defaults for the plain calls; these two take the options
 * per call and read nothing process-wide, so calls with different options can be issued from
 * different threads and streams of one process.  Exactly one of (cache, leaves) and of (dst,
 * dst_leaves) is non-NULL: the flat form or the leaf form (n_leaves is ignored in the flat form).
 *   options  WM_OPT_ZERO_TILES (encode: the zero-tile option; it combines with WM_OPT_ENTROPY)
 *            WM_OPT_ENTROPY    (encode: write ENT tiles; decode: expect an image with ENT tiles)
 *            WM_OPT_STRICT     (decode only: store nothing before every check has passed)
 *            WM_OPT_BLOCKS(n)  (n = 2..255 for encode, 1..255 for decode; 0 or absent: one block per SM):
 *                              the main kernel runs on at most n thread blocks, each of which
 *                              takes a whole SM.  For callers that share the GPU with other work
 *                              (a generating session during pre-copy, Appendix G; the two
 *                              streams of a pre-copy loop): the mover then leaves the other SMs
 *                              alone.  Tiles are claimed by ticket, so the image and every result
 *                              are the same for every n; only the time changes.
 *            any other bit: WM_ERR_ARG, nothing is launched
 * Everything else (arguments, layouts, statuses, what the result record holds) is as in
 * wm_encode / wm_encode_leaves and wm_decode_verify / wm_decode_verify_leaves / _strict.
 */
#define WM_OPT_ZERO_TILES 1u
#define WM_OPT_ENTROPY 2u
#define WM_OPT_STRICT 4u
#define WM_OPT_BLOCKS_MASK 0xFF00u
#define WM_OPT_BLOCKS(n) (((uint32_t)(n) & 0xFFu) << 8)
wm_status wm_encode_opt(const void* cache, const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes,
                        const uint8_t* dirty, uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace,
                        uint64_t workspace_bytes, uint32_t options, wm_result* result, void* stream);
wm_status wm_decode_verify_opt(const void* wire, uint64_t wire_len, void* dst, const wm_leaf* dst_leaves, uint32_t n_leaves,
                               uint64_t nbytes, uint32_t chunk_bytes, uint32_t* dst_crc_inout, void* workspace,
                               uint64_t workspace_bytes, uint32_t options, wm_result* result, void* stream);

/*
 * wm_checksum_noalloc - wm_checksum for callers that cannot allocate device memory.
 * The paper has no counterpart to this call; it exists for hosts that may not call cudaMalloc
 * at the point where they need a checksum: code running under an allocator that has been
 * frozen for the life of a serving process, plug-ins that are handed a stream and buffers but
 * no allocation rights, and start-up or recovery paths that must not touch the device heap.  Same result as wm_checksum, bit for bit, but the scratch memory and
 * the constant tables sit in arrays built into the library image (about 1.2 MiB that every
 * GPU loading the library keeps until the process exits), so the call takes no workspace.
 *   - Limit: nbytes <= WM_NOALLOC_MAX_BYTES (4 GiB); larger inputs return WM_ERR_ARG and
 *     nothing is launched.  All other argument rules are those of wm_checksum.
 *   - The first call on a device looks up the arrays' device addresses and uploads the
 *     tables (a synchronous copy).  Make that first call before any stream capture.
 *   - The call itself allocates nothing: no cudaMalloc, cudaFree or allocating library call.
 *   - There is one scratch array per device and every call uses it.  It keeps the previous
 *     call's contents (the part that must start at zero is cleared on the stream), and two
 *     calls whose kernels overlap on the GPU (different streams, no ordering) race on it:
 *     order such calls on one stream or with events.
 */
#define WM_NOALLOC_MAX_BYTES (4ull << 30)
#define WM_NOALLOC_SCRATCH_BYTES ((1u << 20) + 4096u)
wm_status wm_checksum_noalloc(const void* cache, uint64_t nbytes, uint32_t chunk_bytes,
                              uint32_t* crc_out, void* stream);

/* Number of kernels the last call on this host thread enqueued (for launch accounting). */
uint32_t wm_last_launch_count(void);

/*
 * Measurement aid (not part of the paper's method).  When enabled, every call records a CUDA
 * event pair on the caller's stream around its main kernel: kind 0 = checksum tile digests,
 * 1 = dirty diff compare, 2 = encode, 3 = decode.  wm_timing_read_ms waits for the most
 * recent pair of that kind on the current device and returns its elapsed milliseconds
 * (WM_ERR_CUDA if no such call was made while timing was enabled).  Process-wide switch.
 */
void wm_timing_enable(int on);
int wm_timing_read_ms(int kind, float* ms);

#ifdef __cplusplus
}
#endif
#endif /* WM_H */
