// wm_encode: placement (tickets, scanner warp), the single-pass fused checksum + encode kernel
// with its variants (mask, leaves, zero / constant tiles, entropy option), and its finish kernel.
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

// ------------------------------------------------------------------ wm_encode

// Clears the control block and the placement words, zero-fills the padding behind the tile
// table.  With a dirty mask the main kernel claims the tiles of the present chunks only, so
// here the table entries of all tiles start at 0 (absent) and the first block lists the present
// chunks in ascending order (ws.plist; every thread a run of consecutive chunks, one prefix over
// the threads' counts) and leaves the number of tiles to claim in the control block.
__global__ void __launch_bounds__(1024)
k_encode_init(Geo g, Ws ws, unsigned char* wire, const uint8_t* __restrict__ dirty)
{
    grid_dep_launch();
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t t = i; t < g.n_tiles; t += stride) ws.lbk[t] = 0u;
    if (i < sizeof(Ctrl) / 4) reinterpret_cast<uint32_t*>(ws.ctrl)[i] = 0u;
    // zero padding between the tile table and the payload
    const uint64_t tab_end = 64ull + 16ull * g.n_chunks + 2ull * g.n_tiles;
    if (i < g.meta_end - tab_end) wire[tab_end + i] = 0;
    __syncthreads();                                   // the control block is cleared before anything is written into it
    if (!dirty) {
        if (i == 0) ws.ctrl->n_tickets = g.n_tiles;
        return;
    }
    uint16_t* tile_tab = reinterpret_cast<uint16_t*>(wire + 64 + 16ull * g.n_chunks);
    for (uint64_t t = i; t < g.n_tiles; t += stride) tile_tab[t] = 0;
    if (blockIdx.x != 0) return;
    __shared__ uint32_t s_part[33];
    const uint32_t per = (g.n_chunks + 1023u) / 1024u;
    const uint32_t c0 = min(threadIdx.x * per, g.n_chunks), c1 = min(c0 + per, g.n_chunks);
    uint32_t mine = 0;
    for (uint32_t c = c0; c < c1; c++) mine += dirty[c] != 0 ? 1u : 0u;
    uint32_t n_listed;
    uint32_t at = block_prefix(mine, s_part, n_listed);
    for (uint32_t c = c0; c < c1; c++)
        if (dirty[c] != 0) ws.plist[at++] = c;
    if (threadIdx.x == 0) {
        // every present chunk has tiles_per_chunk tiles, except the cache's last chunk
        const uint32_t np = n_listed;
        uint32_t nt = np * g.tiles_per_chunk;
        if (np && dirty[g.n_chunks - 1]) nt -= g.tiles_per_chunk - (g.n_tiles - (g.n_chunks - 1) * g.tiles_per_chunk);
        ws.ctrl->n_list = np;
        ws.ctrl->n_tickets = nt;
    }
}

constexpr uint32_t kFlagA = 1u << 30, kFlagP = 2u << 30, kValMask = (1u << 30) - 1u;
constexpr uint32_t kUnit = 32;              // placement words count in units of 32 bytes

// Placement of the encoded tiles: a chained scan with one dedicated scanner warp.
//
// lbk[t] starts at 0.  The team that encodes tile t publishes kFlagA | len(t)/32 as soon as the
// length is known.  One scanner warp (alone in the block that wins a lock at kernel start, so
// that it has an SM's issue slots to itself) walks the array in order, 512 entries per poll,
// turns every leading run of published lengths into kFlagP | (exclusive prefix)/32, and moves
// on.  The owner of tile t then reads its offset back from lbk[t].  Every encoded length that
// another tile has to add is a multiple of 32 (only the cache's last tile can be ragged, and
// nothing follows it); 30 bits of 32-byte units cover 32 GiB of payload.
//
// Several hundred tiles are in flight at any time and publish at about the same moment;
// letting each of them walk back to the nearest finished prefix made the walk, not the data,
// the bottleneck, and assigning tiles statically made every round wait for its slowest team.
// The scanner is running by construction (it won the lock), tiles are claimed in ticket
// order, and a team publishes the length of a claimed tile without waiting for anyone, so the
// owners' waits depend only on running code; they are bounded all the same, by time (the call's
// wait budget), and end in WM_ERR_TIMEOUT.
__device__ __forceinline__ void st_relaxed_u32(uint32_t* p, uint32_t v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint32_t next_ticket(Ctrl* ctrl)
{
    return atomicAdd(&ctrl->ticket, 1u);
}

// Owner side: exclusive prefix (bytes) of tile t (one lane spins, for at most `budget_ns`; the
// poison flag and the clock are looked at every 64 polls).
__device__ __forceinline__ unsigned long long wait_prefix(const uint32_t* lbk, uint32_t t, Ctrl* ctrl, uint32_t budget_ns)
{
    const uint32_t t0 = now_ns();
    for (uint32_t polls = 0;; polls++) {
        const uint32_t v = ld_relaxed_u32(lbk + t);
        if ((v >> 30) == 2u) return (unsigned long long)(v & kValMask) * kUnit;
        if ((polls & 63u) == 63u && (ld_volatile_u32(&ctrl->poison) || now_ns() - t0 > budget_ns)) break;
    }
    give_up(ctrl);
    return 0;
}

// Scanner side (one full warp).  A poll copies 512 consecutive entries into shared memory with
// coalesced asynchronous 16-byte copies (one round trip to L2, no registers held meanwhile);
// lane l then owns entries 16 l .. 16 l + 15 of the window.
constexpr int kScanPerLane = 16;
__device__ void scan_tile_lengths(uint32_t* lbk, uint32_t n_tiles, uint32_t lane, Ctrl* ctrl, uint32_t* win,
                                  uint32_t budget_ns)
{
    uint64_t f = 0;                 // first unresolved entry
    uint64_t base = 0;              // units before f
    uint32_t spins = 0;             // polls in a row that resolved nothing
    uint32_t t0 = 0;                // the clock when that run of empty polls began
    while (f < n_tiles) {
        const uint64_t w0 = f & ~3ull;                    // 16-byte aligned window start
        const uint32_t skip = (uint32_t)(f - w0);         // entries before f (already resolved)
#pragma unroll
        for (int q = 0; q < 4; q++) {
            const uint32_t slot = 4u * (lane + 32u * q);
            if (w0 + slot < n_tiles) {                    // n_tiles entries are padded to a multiple of 4
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(win + slot);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(lbk + w0 + slot) : "memory");
            } else {
                *reinterpret_cast<uint4*>(win + slot) = make_uint4(0, 0, 0, 0);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
        uint32_t v[kScanPerLane];
#pragma unroll
        for (int q = 0; q < 4; q++) {
            const uint4 x = *reinterpret_cast<const uint4*>(win + kScanPerLane * lane + 4 * q);
            v[4 * q] = x.x; v[4 * q + 1] = x.y; v[4 * q + 2] = x.z; v[4 * q + 3] = x.w;
        }
        __syncwarp();
        // leading published entries of this lane (entries before f count as published, value 0)
        uint32_t r = 0, sum = 0;
#pragma unroll
        for (int j = 0; j < kScanPerLane; j++) {
            const uint32_t rel = kScanPerLane * lane + j;
            const bool old = rel < skip;
            const bool in = w0 + rel < n_tiles;
            if (r == (uint32_t)j && in && (old || (v[j] >> 30) == 1u)) { r++; if (!old) sum += v[j] & kValMask; }
        }
        const uint32_t fm = __ballot_sync(0xFFFFFFFFu, r == (uint32_t)kScanPerLane);
        const uint32_t lead = (fm == 0xFFFFFFFFu) ? 32u : (uint32_t)(__ffs(~fm) - 1);   // leading full lanes
        const uint32_t contrib = lane <= lead ? sum : 0u;
        uint32_t incl = contrib;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= (uint32_t)d) incl += o;
        }
        const uint32_t cnt = lane < lead ? (uint32_t)kScanPerLane : (lane == lead ? r : 0u);
        uint64_t run = base + (incl - contrib);
#pragma unroll
        for (int j = 0; j < kScanPerLane; j++) {
            const uint32_t rel = kScanPerLane * lane + j;
            if ((uint32_t)j < cnt && rel >= skip) {
                st_relaxed_u32(lbk + w0 + rel, kFlagP | (uint32_t)run);
                run += v[j] & kValMask;
            }
        }
        const uint32_t r_lead = __shfl_sync(0xFFFFFFFFu, r, lead & 31u);
        const uint32_t k_all = (uint32_t)kScanPerLane * lead + (lead < 32u ? r_lead : 0u);   // includes `skip`
        const uint32_t k = k_all > skip ? k_all - skip : 0u;
        base += __shfl_sync(0xFFFFFFFFu, incl, 31);
        f += k;
        if (k == 0) {
            // nothing new: the owners are behind.  Every 64 such polls in a row the scanner looks at the
            // poison flag and at the clock; it gives up when no length has come in for the whole budget.
            if (spins == 0u) t0 = now_ns();
            if ((++spins & 63u) == 0u) {
                const bool stop = ld_volatile_u32(&ctrl->poison) != 0u || now_ns() - t0 > budget_ns;
                if (__any_sync(0xFFFFFFFFu, stop)) {
                    if (lane == 0) give_up(ctrl);
                    return;
                }
            }
        } else {
            spins = 0;
        }
    }
}

__device__ __forceinline__ uint32_t desc_of(uint32_t base, uint32_t w)
{
    return base | (w << 8) | ((((base & 15u) ^ (base >> 4) ^ w ^ 5u) & 15u) << 12);
}

struct EncTeamCtl {
    uint32_t wtab[8][32];   // per group: base | w << 8 (| the all-zero mark on a warp's first entry) (a ring of
                            // slots: one per tile in flight and spares, so that a slot is rewritten
                            // long after its last read)
    uint32_t wdig[8][8];    // per warp: its contribution to the tile digest
    uint32_t spare8[8];     // (unused)
    uint32_t ssum[8];       // sum of the 32 widths of the slot's tile (set by the publishing warp), or a mark:
                            // zero tile, constant tile, kSumEnt | words of the streams for a tile stored in ENT form
    uint32_t etab[8][8];    // entropy option, per warp: anchor | words of its stream << 8 (0xFFFF: a strand too long for the form)
    uint32_t next[2];       // ticket claimed in this step (>= n_tiles: none left), by step parity
    uint32_t pad[2];
    unsigned long long excl[2];   // offset of the tile packed in the next step, by step parity
    unsigned long long mbar;      // completion of the bulk copy into the team's stage
    unsigned long long pad2;
    unsigned long long nptr[2];   // leaf mode: address (k_leaf_map) of the tile in next[], by step parity
    uint32_t kring[8];            // with a mask: the ticket of the tile in each ring slot (placement runs over tickets)
    unsigned char sbits[4][256];  // entropy option: every strand's bit length - 64, from the measuring step to the
                                  // packing step three steps on (slot: step mod 4, as in tensor memory)
};
static_assert(sizeof(EncTeamCtl) % 16 == 0, "team control block keeps 16-byte alignment");

__device__ __forceinline__ uint32_t tile_left(const Geo& g, uint32_t t)      // bytes of a ragged tile
{
    return (uint32_t)(g.nbytes - (uint64_t)t * kTile);
}

__device__ __forceinline__ void stg_u8(void* p, uint32_t v)
{
    asm volatile("st.global.cs.u8 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void stg_u16(void* p, uint32_t v)
{
    asm volatile("st.global.cs.u16 [%0], %1;" ::"l"(p), "h"((unsigned short)v) : "memory");
}
__device__ __forceinline__ void stg_v2(void* p, uint32_t a, uint32_t b)
{
    asm volatile("st.global.cs.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(a), "r"(b) : "memory");
}

// Write the bit planes of one group straight to the wire image.  The lane holds the eight
// exponent bytes of its elements (e4a, e4b, coded order); after the base is subtracted each
// is < 2^W.  W = 8 is stored as it is; otherwise a 4-bit, a 2-bit and a 1-bit plane (those
// whose bit is set in W) take consecutive bits of the deltas from bit 0.  In every plane lane
// l owns an aligned 4 / 2 / 1-byte unit at l times that size, so each warp store covers one
// contiguous, sector-aligned run of 128 / 64 / 32 bytes and nothing needs staging.
//   nibbles : v | v >> 4 puts two 4-bit values side by side in bytes 0 and 2 of each word
//   2 bits  : (t * 0x01041040) >> 24 gathers the four 2-bit fields of a word into one byte
//   1 bit   : (t * 0x01020408) >> 24 gathers the four bits of a word into one nibble
// (the partial products of both multiplications land on distinct bits, so no carry occurs).
template <int W>
__device__ __forceinline__ void pack_group_planes(uint32_t e4a, uint32_t e4b, uint32_t base, unsigned char* rec,
                                                  uint32_t lane)
{
    const uint32_t b4 = base * 0x01010101u;
    uint32_t da = e4a - b4, db = e4b - b4;
    if (W == 8) {
        stg_v2(rec + 8 * lane, da, db);
        return;
    }
    unsigned char* p = rec;
    if (W & 4) {
        const uint32_t na = (W == 4) ? da : (da & 0x0F0F0F0Fu), nb = (W == 4) ? db : (db & 0x0F0F0F0Fu);
        const uint32_t va = na | (na >> 4), vb = nb | (nb >> 4);
        st_stream_u32(p + 4 * lane, __byte_perm(va, vb, 0x6420));
        p += 128;
        da >>= 4; db >>= 4;
    }
    if (W & 2) {
        const uint32_t pa = (da & 0x03030303u) * 0x01041040u, pb = (db & 0x03030303u) * 0x01041040u;
        stg_u16(p + 2 * lane, __byte_perm(pa, pb, 0x0073));
        p += 64;
        da >>= 2; db >>= 2;
    }
    if (W & 1) {
        const uint32_t pa = (da & 0x01010101u) * 0x01020408u, pb = (db & 0x01010101u) * 0x01020408u;
        const uint32_t x = __byte_perm(pa, pb, 0x0073);          // byte 0: a's nibble, byte 1: b's nibble
        stg_u8(p + lane, x | (x >> 4));
    }
}


// ---- ENT tiles: entropy-coded exponents (an encoder option; header flags bit 2) --------------
// A warp's 2 KiB of a tile (16 rows) is one share; lane l's 32 elements (its 16 words, low half
// first) are strand l.  Every exponent is coded as u = E - anchor with a fixed prefix code, the
// anchor being the rounded mean of the share's exponents; a strand is the LSB-first bit string of
// its 32 codewords, and the 32 strands of a share lie one behind the other in the share's
// stream, their lengths written down in a byte each, so that every lane of the reading warp
// finds the start of its strand with one prefix sum and nobody waits for anybody.
//   u        -6  -5  -4  -3  -2  -1   0   1   2   3   other
//   length    8   6   5   4   4   2   2   2   4   7   16 (eight ones, then E itself)
//   bits    127  31  15  11   3   2   0   1   7  63   255 | E << 8        (first bit = bit 0)
// ent_slot: 0..9 for u = -6..3, 10 for everything else.
__device__ __forceinline__ uint32_t ent_slot(uint32_t E, uint32_t anchor)
{
    return min(E - anchor + 6u, 10u);
}
// Both tables are byte look-ups done with permutes (no branches: the lanes of a warp hold
// different slots): slots 0..7 from one pair of words, 8..10 from a third.
__device__ __forceinline__ uint32_t ent_lut(uint32_t lo, uint32_t hi, uint32_t top, uint32_t slot)
{
    const uint32_t a = __byte_perm(lo, hi, slot), b = __byte_perm(top, 0u, slot & 7u);
    return (slot < 8u ? a : b) & 0xFFu;
}
__device__ __forceinline__ uint32_t ent_length(uint32_t slot)
{
    return ent_lut(0x04050608u, 0x02020204u, 0x00100704u, slot);      // 8 6 5 4 | 4 2 2 2 | 4 7 16
}
__device__ __forceinline__ uint32_t ent_word(uint32_t slot, uint32_t E)
{
    const uint32_t w = ent_lut(0x0B0F1F7Fu, 0x01000203u, 0x00FF3F07u, slot);       // 127 31 15 11 | 3 2 0 1 | 7 63 255
    return w | (slot == 10u ? E << 8 : 0u);
}
// Bytes of an ENT tile whose eight streams hold `words` 32-bit words in all (a multiple of 32;
// 16384 or more means that the tile takes another form): header, sign-mantissa plane, strand
// lengths, streams.
__device__ __forceinline__ uint32_t ent_tile_bytes(uint32_t words)
{
    return (8512u + 4u * words + 31u) & ~31u;
}
// Decoder side.  A codeword is s ones and a zero (s < 8; eight ones: the escape), followed for
// s = 0 and s = 2 by one more bit x:  s = 0: u = -x;  1: +1;  2: -2 - x;  3: +2;  4..7: -4, -5, +3, -6.
// ent_ones: s, capped at 8, of the codeword at the low end of `buf` (zero beyond the valid bits).
__device__ __forceinline__ uint32_t ent_ones(uint32_t buf)
{
    return min((uint32_t)__ffs(~buf) - 1u, 8u);
}
__device__ __forceinline__ uint32_t ent_parse_length(uint32_t s)
{
    const uint32_t l = __byte_perm(0x04040202u, 0x08070605u, s & 7u) & 0xFFu;       // 2 2 4 4 | 5 6 7 8
    return s == 8u ? 16u : l;
}
__device__ __forceinline__ uint32_t ent_parse_value(uint32_t buf, uint32_t s, uint32_t anchor)
{
    const uint32_t base = __byte_perm(0x02FE0100u, 0xFA03FBFCu, s & 7u);            // 0 +1 -2 +2 | -4 -5 +3 -6
    const uint32_t x = ((s & 5u) == 0u) ? (buf >> (s + 1u)) & 1u : 0u;
    return s == 8u ? (buf >> 8) & 0xFFu : (anchor + base - x) & 0xFFu;
}

// Single-pass fused checksum + encode.  Each team keeps four tiles in flight:
//     X  measured three steps ago, packed and written to the wire image in this step
//     V, W  measured two / one steps ago, waiting for their offsets
//     Y  checksummed and measured in this step (its length is published right after the next barrier)
// The team owns one 16 KiB stage in shared memory that bulk copies (TMA) fill, one tile per
// step, each copy started a whole step before its tile is needed.  A measured tile's words
// (16 registers per lane) are parked in tensor memory until its offset is known, so a tile is
// read from memory once and nothing waits in registers.  Per step:
//     take Y's words from the stage | team barrier | publish len(W), the tile measured a step
//     ago | start the copy of the next Y | digest + exponent ranges of Y | park Y | fetch X |
//     pack X straight into the wire image
// Meanwhile two round trips to L2 are in flight whose answers are needed a step later: the
// ticket of the tile to measure two steps on and the offset of the tile to pack next.  These and
// the other single-lane chores of a step sit on different warps: the team passes one barrier per
// tile, so it runs at the pace of the warp that has the most to do.
// Template switches: MASKED (a dirty mask was given), LEAVES (the cache is a table of tensors;
// tickets are claimed one step further ahead so that a tile's address can be looked up on the
// way), ZEROS (the zero / constant tile option), ENT (the entropy option: the measuring step also
// adds up codeword lengths, the tile takes the shorter of the two coded forms, and for the ENT
// form the packing step writes the strands' lengths and the share's stream of words instead of bit planes).
// Packed data goes from registers to the wire image directly: in every region of a PACK tile
// a lane owns an aligned unit at a lane-strided place, so each warp store is one contiguous
// sector-aligned run.  Claiming a tile before the previous offset is known means that, if the
// scanner is late, this team waits while that tile's length is not out yet; with three steps
// of slack that is rare, and it only delays: the teams that hold earlier tiles never depend
// on this one.
// A tile as a team passes it round: its number in the low 22 bits, kQFirst when it is the first
// tile of its chunk, kQPresent when its chunk is encoded; kQNone: no tile.  Leaf mode adds, in
// bits 22-25, how many bytes above a 16-byte boundary the tile starts.  (The codec takes caches
// of at most 2^21 tiles, so a number never reaches kQNone or the other fields.)
constexpr uint32_t kQPresent = 1u << 31, kQFirst = 1u << 30, kQTile = (1u << 22) - 1u, kQNone = kQTile;
constexpr uint32_t kQOffShift = 22;
// Marks in a team's width table: on a warp's first entry, all 2 KiB of the warp's rows are zero;
// as the sum of the widths, the tile is all zero.
// kWarpConst: all 1024 elements of the warp's rows hold one value (its sign-mantissa byte rides in
// bits 16-23 of the entry, the exponent is the base); kSumConstTile: the tile holds one value.
constexpr uint32_t kWarpAllZero = 0x8000u, kWarpConst = 0x4000u, kSumZeroTile = 0xFFFFu, kSumConstTile = 0xFFFEu;
// The tile is stored in ENT form (shorter than its bit planes and than raw); low half: words of its streams.
constexpr uint32_t kSumEnt = 0x10000u;

// The tile behind ticket k.  Without a mask tickets are tile numbers.  With one, only the tiles of
// present chunks are claimed: ticket k is tile k mod tiles_per_chunk of the (k / tiles_per_chunk)-th
// present chunk (plist, ascending, written by k_encode_init), so placement runs over tickets and a
// sparse mask costs nothing for what it leaves out.
template <bool MASKED>
__device__ __forceinline__ uint32_t describe_tile(const Geo& g, const uint32_t* __restrict__ plist, uint32_t n_tickets, uint32_t k)
{
    if (k >= n_tickets) return kQNone;
    uint32_t t = k;
    bool first = first_in_chunk(g, k);
    if (MASKED) {
        const uint32_t j = chunk_of(g, k);
        t = plist[j] * g.tiles_per_chunk + (k - j * g.tiles_per_chunk);
    }
    return t | kQPresent | (first ? kQFirst : 0u);
}

template <int TEAMS, bool MASKED, bool LEAVES, bool ZEROS, bool ENT = false>
__global__ void __launch_bounds__(TEAMS * 256, 1)
k_encode(const unsigned char* __restrict__ cache, Geo g, const uint8_t* __restrict__ dirty,
         unsigned char* __restrict__ wire, uint64_t wire_cap, Ws ws, const Tables* __restrict__ tab)
{
    extern __shared__ __align__(16) unsigned char smem[];
    // The first block to get here becomes the scanner: one warp of it, alone on its SM (a warp
    // that shares its scheduler with busy ones gets too few issue slots to keep up).
    __shared__ uint32_t s_scanner;
    __shared__ uint32_t s_tmem;
    Smem S = setup_smem(smem, tab);
    grid_dep_wait();                   // from here on the control block and the length table are ready
    grid_dep_launch();
    if (LEAVES && (ld_volatile_u32(&ws.ctrl->err) & 8u)) return;      // the leaf table was rejected
    if (threadIdx.x == 0) s_scanner = atomicCAS(&ws.ctrl->scan_lock, 0u, 1u) == 0u;
    __syncthreads();
    if (s_scanner) {
        uint32_t* win = reinterpret_cast<uint32_t*>(S.take(2048));      // 512 entries
        // (test hook: with the scanner left out no offset is ever handed out, and the owners' waits run out)
        if (threadIdx.x < 32 && win && !(g.inject & kInjectNoScanner)) scan_tile_lengths(ws.lbk, MASKED ? ld_volatile_u32(&ws.ctrl->n_tickets) : g.n_tiles, threadIdx.x, ws.ctrl, win, g.wait_ns);
        return;
    }
    const uint32_t team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads;
    const uint32_t warp = tt / 32, lane = tt % 32;
    unsigned char* stage = nullptr;
    // (leaf mode: a tile may start off a 16-byte boundary; its copy then starts at the boundary
    // below and is 16 bytes longer, so the stage is too)
    constexpr uint32_t kStage = LEAVES ? kTile + 16u : kTile;
    for (int i = 0; i < TEAMS; i++) {          // every thread carves the same blocks in the same order
        unsigned char* p = S.take(kStage);
        if ((uint32_t)i == team) stage = p;
    }
    EncTeamCtl* tc = reinterpret_cast<EncTeamCtl*>(S.take(TEAMS * sizeof(EncTeamCtl)));
    // ENT: codeword length and codeword by k = E - anchor + 256 (1..511), so that a look-up is the
    // exponent added to an address the share works out once (no slot arithmetic per element); the
    // escape's codeword reads 0xFFFF (the packing step lets the exponent through its high byte)
    unsigned char* const t_lenE = ENT ? S.take(512) : nullptr;
    unsigned short* const t_cwE = ENT ? reinterpret_cast<unsigned short*>(S.take(1024)) : nullptr;
    if (!S.ok) { if (threadIdx.x == 0) atomicOr(&ws.ctrl->err, 4u); return; }
    tc += team;
    if (ENT && threadIdx.x < 512u) {
        const int u = (int)threadIdx.x - 256;
        const uint32_t slot = (u >= -6 && u <= 3) ? (uint32_t)(u + 6) : 10u;
        t_lenE[threadIdx.x] = (unsigned char)ent_length(slot);
        t_cwE[threadIdx.x] = (unsigned short)(slot == 10u ? 0xFFFFu : ent_word(slot, 0u));
    }
    const uint32_t lenE_s = ENT ? (uint32_t)__cvta_generic_to_shared(t_lenE) + 256u : 0u;
    const uint32_t cwE_s = ENT ? (uint32_t)__cvta_generic_to_shared(t_cwE) + 512u : 0u;

    // Tensor memory for the tiles in flight: allocated by the block's first warp, the address
    // goes round through shared memory.  Warp w of the block owns lanes 32 (w % 4) .. + 31 and
    // 64 columns from 64 (w / 4): four slots of 16 columns, one per tile in flight.
    if (threadIdx.x < 32) tmem_alloc_all(&s_tmem);
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    const uint32_t wc = threadIdx.x / 32;
    const uint32_t tmem_warp = s_tmem + ((32u * (wc & 3u)) << 16) + 64u * (wc >> 2);

    unsigned char* const dir = wire + 64;
    uint16_t* const tile_tab = reinterpret_cast<uint16_t*>(wire + 64 + 16ull * g.n_chunks);
    unsigned char* const payload = wire + g.meta_end;
    const uint64_t room = wire_cap - g.meta_end;                 // payload bytes that fit
    const uint64_t pol_once = l2_policy_evict_first();           // every tile is read once
    const uint32_t* const my_words = reinterpret_cast<const uint32_t*>(stage) + warp * 512u + lane;
    const uint32_t sm_off = 64u + 1024u * warp + 8u * lane;      // this lane's place in a group's sign-mantissa run
    const bool leader = (tt == 0);
    uint32_t phase = 0;                // parity of the stage's next completion

    auto is_tile = [](uint32_t q) { return (q & kQTile) != kQNone; };
    auto is_hot = [&](uint32_t q) { return q >= kQPresent && (q & kQTile) < g.n_full_tiles; };   // present and full
    // (the placement words are indexed by ticket: with a mask that is the ring slot's ticket, else the tile number)
    const uint32_t n_tickets = MASKED ? ld_volatile_u32(&ws.ctrl->n_tickets) : g.n_tiles;
    auto place_of = [&](uint32_t slot, uint32_t t) { return MASKED ? tc->kring[slot] : t; };
    auto publish_len = [&](uint32_t slot, uint32_t t, uint32_t len) { st_relaxed_u32(ws.lbk + place_of(slot, t), kFlagA | (len / kUnit)); };
    // where tile t lives: its address in the flat cache, or (leaf mode) the address that k_leaf_map wrote
    auto tile_src = [&](uint32_t t) -> unsigned long long {
        return LEAVES ? ws.tptr[t] : reinterpret_cast<unsigned long long>(cache + (uint64_t)t * kTile);
    };
    // One thread of the team, after the barrier that frees the stage.  Leaf mode: a tile may start
    // off a 16-byte boundary; the copy then starts at the boundary below and takes 16 bytes more
    // (k_leaf_map saw to it that they belong to the leaf); the readers shift by the remainder.
    auto start_copy = [&](uint32_t q, unsigned long long src) {
        if (!is_hot(q)) return;
        const unsigned long long a = LEAVES ? src & ~15ull : src;
        bulk_load(stage, reinterpret_cast<const void*>(a), (LEAVES && a != src) ? kTile + 16u : kTile, &tc->mbar, pol_once);
    };
    // leaf mode, handing a claimed tile on: its word carries the start's remainder
    auto with_mark = [](uint32_t q, unsigned long long addr) {
        return (!LEAVES || (q & kQTile) == kQNone) ? q : q | (((uint32_t)addr & 15u) << kQOffShift);
    };

    // Tiles in flight, oldest first: X (packed in this step), V, W (waiting for their offsets),
    // Y (measured in this step).  Ring slots of the widths: X = sl, V = sl+1, W = sl+2, Y = sl+3
    // (mod 8); tensor memory slots: Y = step mod 4, X = (step + 1) mod 4 (where it was put three
    // steps ago).
    uint32_t qX = kQNone, qV = kQNone, qW = kQNone, qY = kQNone;
    uint32_t sl = 0;
    uint32_t par = 0;                  // step parity (selects next[] / excl[])
    uint32_t step = 0;
    uint32_t d[kWordsPerLane];
    bool claiming = false;             // leader: the last ticket it claimed was a tile

    // ---- prologue: the tiles of the first two steps are claimed, the first one's copy started.
    // Leaf mode claims one step further ahead: a tile's address is looked up in the step between
    // its claim and its hand-over, so that the leader never waits for that answer either.
    uint32_t qA = kQNone;              // leader, leaf mode: claimed and described, address on its way
    uint32_t kA = 0;                   // ... and its ticket
    // With a mask (flat cache) a ticket's tile is found through the list of present chunks.  That
    // look-up too is started in the step after the claim and used at that step's end, so a ticket
    // is handed over one step later than without a mask and the leader claims one step further ahead.
    constexpr bool kLateList = MASKED && !LEAVES;
    bool haveA = false;                // leader, kLateList: ticket kA is a tile and waits for its chunk number
    if (leader) {
        mbar_init(&tc->mbar, 1);
        const uint32_t k0 = next_ticket(ws.ctrl);
        const uint32_t q0 = describe_tile<MASKED>(g, ws.plist, n_tickets, k0);
        const uint32_t k1 = is_tile(q0) ? next_ticket(ws.ctrl) : 0xFFFFFFFFu;
        const uint32_t q1 = is_tile(q0) ? describe_tile<MASKED>(g, ws.plist, n_tickets, k1) : kQNone;
        claiming = is_tile(q1);
        if (MASKED) { tc->kring[3] = k0; tc->kring[4] = k1; }      // the slots in which they will be measured
        tc->next[0] = q0;
        tc->next[1] = q1;
        tc->excl[0] = 0ull;
        tc->excl[1] = 0ull;
        if (LEAVES) {
            tc->nptr[0] = is_tile(q0) ? tile_src(q0 & kQTile) : 0ull;
            tc->nptr[1] = is_tile(q1) ? tile_src(q1 & kQTile) : 0ull;
            tc->next[0] = with_mark(q0, tc->nptr[0]);
            tc->next[1] = with_mark(q1, tc->nptr[1]);
            if (claiming) { kA = next_ticket(ws.ctrl); qA = describe_tile<MASKED>(g, ws.plist, n_tickets, kA); claiming = is_tile(qA); }
        }
        if (kLateList && claiming) { kA = next_ticket(ws.ctrl); claiming = haveA = kA < n_tickets; }
    }
    team_bar(team);
    qY = tc->next[0];
    if (leader) start_copy(qY, LEAVES ? tc->nptr[0] : tile_src(qY & kQTile));

    uint32_t trouble = 0;              // sticky: the image does not fit
    while (((qX & qV & qW & qY) & kQTile) != kQNone) {
        const bool hotY = is_hot(qY);
        if (hotY) {
            wait_for_copy<!ENT>(&tc->mbar, phase, g.wait_ns, ws.ctrl);
            phase ^= 1u;
            // leaf mode: a tile that was copied from the 16-byte boundary below it starts that many
            // bytes into the stage: whole words from a quarter of that on, each put together from two
            // neighbours when the remainder is no multiple of four
            const uint32_t off = LEAVES ? (qY >> kQOffShift) & 15u : 0u;
            const uint32_t sh = (off & 3u) * 8u;
            const uint32_t* const p = my_words + (off >> 2);
            if (LEAVES && sh) {
#pragma unroll
                for (int i = 0; i < 16; i++) d[i] = __funnelshift_r(p[i * 32], p[i * 32 + 1], sh);
            } else {
#pragma unroll
                for (int i = 0; i < 16; i++) d[i] = p[i * 32];
            }
        }
        team_bar(team);                   // stage free; what the leader left at the end of the last step is visible
        const uint32_t qN = tc->next[par ^ 1u];
        const unsigned long long exclX = tc->excl[par ^ 1u];
        // The tile measured in the last step (W now): its 32 widths are complete behind the barrier.
        // One warp that has no other single-lane chore adds them up and publishes the tile's length
        // (half a step later than the last-arriving warp could have, which the three steps of slack
        // before the tile is packed absorb; but no warp waits for a counter in the measuring step
        // and the sum is off the path of whichever warp was slowest there).
        if (warp == 6u && is_hot(qW)) {
            const uint32_t slW = (sl + 2u) & 7u;
            const uint32_t wt = tc->wtab[slW][lane];
            const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, (wt >> 8) & 15u);
            // entropy option: the ENT form is taken when it is shorter than the planes and than raw
            uint32_t ent_words = 0;
            if (ENT) ent_words = __reduce_add_sync(0xFFFFFFFFu, lane < 8u ? tc->etab[slW][lane] >> 8 : 0u);
            const uint32_t plane_len = total <= 253u ? 8256u + 32u * total : kTile;
            const bool ent_tile = ENT && ent_tile_bytes(ent_words) < plane_len;
            // unused memory (every warp's first entry carries the mark): no payload
            // (one value throughout: every warp's first entry carries the mark and they are all alike;
            // a tile of zeros has no payload, any other value 32 bytes)
            const uint32_t wt0 = __shfl_sync(0xFFFFFFFFu, wt, 0);
            const bool const_tile = ZEROS && __all_sync(0xFFFFFFFFu, (lane & 3u) != 0u || ((wt & kWarpConst) != 0u && wt == wt0));
            const bool zero_tile = const_tile && (wt0 & kWarpAllZero) != 0u;
            if (lane == 0) {
                tc->ssum[slW] = zero_tile ? kSumZeroTile : const_tile ? kSumConstTile : ent_tile ? kSumEnt | ent_words : total;
                publish_len(slW, qW & kQTile, zero_tile ? 0u : const_tile ? 32u : ent_tile ? ent_tile_bytes(ent_words) : plane_len);
            }
        }
        // The team's single-lane chores are spread over its warps, because the team waits for
        // whichever warp has the most to do.  Warp 2 starts the copy of the next tile (it has the
        // whole step to arrive).  Two round trips to L2 are started now and used at the end of the
        // step: the ticket of the tile to measure two steps on (warp 0, the leader) and the offset
        // of the tile to pack in the next step (warp 3).  Warp 1 notes what is left about X.
        uint32_t pv = 0, tk = 0xFFFFFFFFu;
        unsigned long long pA = 0;
        if (tt == 64u) start_copy(qN, LEAVES ? tc->nptr[par ^ 1u] : tile_src(qN & kQTile));
        if (tt == 96u && is_tile(qV)) pv = ld_relaxed_u32(ws.lbk + place_of((sl + 1u) & 7u, qV & kQTile));
        uint32_t plA = 0;
        if (leader) {
            if (claiming) tk = next_ticket(ws.ctrl);
            if (LEAVES && is_tile(qA)) pA = tile_src(qA & kQTile);
            if (kLateList && haveA) plA = __ldg(ws.plist + chunk_of(g, kA));
        }

        // ---- Y: digest, exponent ranges, length out, words parked
        const uint32_t slY = (sl + 3u) & 7u;
        const uint32_t tYn = qY & kQTile;
        if (hotY) {
            const uint32_t v = tile_digest_part(S, d, (qY & kQFirst) != 0, warp, lane);
            // From here on the words are kept rotated left by one bit: each half then reads
            // [E | mantissa | a sign bit], E in its high byte (the two sign bits of a word
            // land in each other's half; the packing step puts them right).
#pragma unroll
            for (int i = 0; i < 16; i++) d[i] = __funnelshift_l(d[i], d[i], 1);
            uint32_t gw[4];               // per group: base | width << 8
            uint32_t ent_w = 0;           // entropy option: anchor | words << 8 of this warp's share
            if (ENT) {
                // the share's anchor (rounded mean of its 1024 exponents: bytes 1 and 3 of a rotated
                // word), every strand's length in bits and the words the share's stream needs
                uint32_t acc = 0;
#pragma unroll
                for (int i = 0; i < 16; i++) acc = __dp4a(d[i], 0x01000100u, acc);       // bytes 1 and 3
                const uint32_t anchor = (__reduce_add_sync(0xFFFFFFFFu, acc) + 512u) >> 10;
                uint32_t bits = 0;
                const uint32_t lb = lenE_s - anchor;
#pragma unroll
                for (int i = 0; i < 16; i++)
                    bits += lds_tab_u8(lb + __byte_perm(d[i], 0u, 0x4441)) + lds_tab_u8(lb + (d[i] >> 24));
                // (a strand the length byte cannot hold, above 319 bits, keeps the tile out of the form:
                // the count is then so large that the form is never the shortest)
                const uint32_t share_bits = __reduce_add_sync(0xFFFFFFFFu, bits);
                const bool too_long = __any_sync(0xFFFFFFFFu, bits > 319u);
                tc->sbits[step & 3u][32u * warp + lane] = (unsigned char)(bits - 64u);
                ent_w = anchor | ((too_long ? 0xFFFFu : (share_bits + 31u) >> 5) << 8);
            }
            {
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const uint32_t a0 = d[4 * j], a1 = d[4 * j + 1], a2 = d[4 * j + 2], a3 = d[4 * j + 3];
                uint32_t mn = min_u16x2(min_u16x2(a0, a1), min_u16x2(a2, a3));
                uint32_t mx = max_u16x2(max_u16x2(a0, a1), max_u16x2(a2, a3));
                // both halves get the smaller (larger) of the two, so that the word as a whole
                // orders like its halves and one warp reduction per bound does
                mn = min_u16x2(mn, __byte_perm(mn, mn, 0x1032));
                mx = max_u16x2(mx, __byte_perm(mx, mx, 0x1032));
                const uint32_t emin = (__reduce_min_sync(0xFFFFFFFFu, mn) >> 8) & 0xFFu;
                const uint32_t emax = (__reduce_max_sync(0xFFFFFFFFu, mx) >> 8) & 0xFFu;
                gw[j] = emin | ((32u - __clz(emax - emin)) << 8);
            }
            }
            // Option ZEROS.  Unused memory: when all four groups have exponent 0 throughout (rare in live data)
            // look at the words themselves; a warp whose 2 KiB are all zero marks its first entry.
            // The same for any one value (a mask fill, say): all four groups have one exponent and width
            // 0; then every word must equal the warp's first, and that word's two halves each other.
            if (ZEROS && gw[0] < 256u && gw[1] == gw[0] && gw[2] == gw[0] && gw[3] == gw[0]) {
                const uint32_t first = __shfl_sync(0xFFFFFFFFu, d[0], 0);
                uint32_t diff = (first >> 16) ^ (first & 0xFFFFu);
#pragma unroll
                for (int i = 0; i < 16; i++) diff |= d[i] ^ first;
                if (!__any_sync(0xFFFFFFFFu, diff != 0u))
                    gw[0] |= kWarpConst | ((first & 0xFFu) << 16) | (first == 0u ? kWarpAllZero : 0u);
            }
            // one lane leaves the warp's results; the tile's length is added up and published right
            // after the next barrier, when all eight warps' widths are there (see the top of the step)
            if (lane == 0) {
                tc->wdig[slY][warp] = v;
                *reinterpret_cast<uint4*>(&tc->wtab[slY][4 * warp]) = make_uint4(gw[0], gw[1], gw[2], gw[3]);
                if (ENT) tc->etab[slY][warp] = ent_w;
            }
            tmem_store16(tmem_warp + 16u * (step & 3u), d);
        } else if (is_tile(qY)) {
            // rare: a tile of an absent chunk (length 0) or the ragged last tile (stored raw)
            const bool present = qY >= kQPresent;
            if (tt == 0) publish_len(slY, tYn, present ? tile_left(g, tYn) : 0u);
            if (present) {
                // (leaf mode: the ragged tile has a slot of its own in the side buffer)
                load_tile_words_guarded(reinterpret_cast<const unsigned char*>(tile_src(tYn)), tile_left(g, tYn), (qY & kQFirst) != 0, warp, lane, d);
                const uint32_t v = tile_digest_part(S, d, false, warp, lane);
                if (lane == 0) tc->wdig[slY][warp] = v;
            }
        }

        // ---- X: its words back from tensor memory, packed straight into the wire image
        const uint32_t tXn = qX & kQTile;
        if (is_hot(qX)) {
            tmem_load16(tmem_warp + 16u * ((step + 1u) & 3u), d);
            const uint32_t Smark = tc->ssum[sl];
            const bool ent_form = ENT && (Smark & kSumEnt) != 0u;
            const uint32_t Ssum = ent_form ? Smark & 0xFFFFu : Smark;       // words of the streams, or the sum of the widths
            const bool packs = !ent_form && Ssum <= 253u;
            // (a tile of all-zero bytes, marked in ssum, is its table entry and nothing else)
            const uint32_t enc_len = ent_form ? ent_tile_bytes(Ssum)
                                         : packs ? 8256u + 32u * Ssum : (ZEROS && Ssum == kSumZeroTile) ? 0u
                                         : (ZEROS && Ssum == kSumConstTile) ? 32u : kTile;
            unsigned char* const dst = payload + exclX;
            if (exclX + enc_len > room) {
                trouble |= 1u;
            } else if (ent_form) {
                // header: anchors, word counts, 40 zero bytes; zero fill behind the last stream
                if (warp == 5) {
                    if (lane < 8u) {
                        const uint32_t wt = tc->etab[sl][lane];
                        stg_u8(dst + lane, wt & 0xFFu);
                        stg_u16(dst + 8u + 2u * lane, wt >> 8);
                    } else if (lane < 18u) {
                        st_stream_u32(dst + 24u + 4u * (lane - 8u), 0u);
                    }
                    if (4u * lane < enc_len - 8512u - 4u * Ssum) st_stream_u32(dst + 8512u + 4u * Ssum + 4u * lane, 0u);
                }
                unsigned char* const sm_dst = dst + sm_off;
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint32_t sa = __byte_perm(d[4 * j], d[4 * j + 1], 0x6420), sb = __byte_perm(d[4 * j + 2], d[4 * j + 3], 0x6420);
                    const uint32_t ya = __byte_perm(sa, sa, 0x2301), yb = __byte_perm(sb, sb, 0x2301);
                    stg_v2(sm_dst + 256 * j, (sa & 0xFEFEFEFEu) | (ya & 0x01010101u), (sb & 0xFEFEFEFEu) | (yb & 0x01010101u));
                }
                // This share's stream starts behind the streams of the warps before it; inside it the
                // strands follow one another bit by bit, so lane l starts where the lengths of the
                // lanes before it (measured three steps ago) add up to.
                const uint32_t before = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? tc->etab[sl][lane] >> 8 : 0u);
                const uint32_t anchor = tc->etab[sl][warp] & 0xFFu;
                const uint32_t nb8 = tc->sbits[(step + 1u) & 3u][32u * warp + lane];
                stg_u8(dst + 8256u + 32u * warp + lane, nb8);
                uint32_t incl = 64u + nb8;
#pragma unroll
                for (int k = 1; k < 32; k <<= 1) {
                    const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, k);
                    if (lane >= (uint32_t)k) incl += o;
                }
                const uint32_t start = incl - 64u - nb8;
                unsigned char* const w_dst = dst + 8512u + 4u * before;
                // acc: the stream's bits from the last word boundary on, n of them valid (the first n
                // of the lane's first word belong to the lane before it).  Two codewords are joined
                // first (32 bits at most) and go in together; both shifts are multiplications by a
                // power of two from the table or from n (one multiply-add each, on the pipe that has
                // little else to do here, where the shifts and ORs would queue up with everything
                // else).  Words go out as they fill up, except the lane's first one, which is held
                // back until the lane before has handed over the bits it left in it.
                unsigned long long acc = 0;
                uint32_t n = start & 31u, wp = start >> 5, w_first = 0;
                bool have_first = false;
                const uint32_t lb = lenE_s - anchor, cb = cwE_s - 2u * anchor;
#pragma unroll
                for (int i = 0; i < 16; i++) {
                    const uint32_t E0 = __byte_perm(d[i], 0u, 0x4441), E1 = d[i] >> 24;
                    const uint32_t len0 = lds_tab_u8(lb + E0), len1 = lds_tab_u8(lb + E1);
                    // (the table's escape entry is 0xFFFF: the AND lets the exponent through there only)
                    const uint32_t c0 = lds_tab_u16(cb + 2u * E0) & __byte_perm(E0, 0xFFu, 0x4404);
                    const uint32_t c1 = lds_tab_u16(cb + 2u * E1) & __byte_perm(E1, 0xFFu, 0x4404);
                    const uint32_t pair = c1 * (1u << len0) + c0;
                    asm("mad.wide.u32 %0, %1, %2, %0;" : "+l"(acc) : "r"(pair), "r"(1u << n));
                    n += len0 + len1;
                    if (n >= 32u) {                        // (two codewords are 32 bits at most: one word per pair)
                        const uint32_t word = (uint32_t)acc;
                        if (have_first) st_stream_u32(w_dst + 4u * wp, word); else w_first = word;
                        have_first = true;
                        acc >>= 32;
                        n -= 32u;
                        wp++;
                    }
                }
                // (a strand is 64 bits at least, so every lane has crossed a word boundary by now)
                const uint32_t tail = (uint32_t)acc;                   // n bits of the next word, 0 when n == 0
                const uint32_t from_below = __shfl_up_sync(0xFFFFFFFFu, tail, 1);
                st_stream_u32(w_dst + 4u * (start >> 5), w_first | (lane ? from_below : 0u));
                if (lane == 31u && n) st_stream_u32(w_dst + 4u * wp, tail);
            } else if (packs) {
                if (warp == 5) {           // (any one warp: not one that has a single-lane chore)
                    const uint32_t wt = tc->wtab[sl][lane];
                    stg_u16(dst + 2 * lane, desc_of(wt & 0xFFu, (wt >> 8) & 15u));
                }
                unsigned char* const sm_dst = dst + sm_off;
                unsigned char* const pl_dst = dst + 8256;
                // widths of all 32 groups (one per lane): 32-byte units before this warp's first group
                const uint32_t wall = (tc->wtab[sl][lane] >> 8) & 15u;
                uint32_t before = __reduce_add_sync(0xFFFFFFFFu, lane < 4u * warp ? wall : 0u);
                const uint4 g4 = *reinterpret_cast<const uint4*>(&tc->wtab[sl][4 * warp]);
                const uint32_t gq[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint32_t wtg = gq[j];
                    const uint32_t base = wtg & 0xFFu, wd = (wtg >> 8) & 15u;
                    // bytes 0 and 2 of a rotated word: mantissa << 1 | the other element's sign;
                    // bytes 1 and 3: the exponents.  Gather, then swap bit 0 inside byte pairs.
                    const uint32_t sa = __byte_perm(d[4 * j], d[4 * j + 1], 0x6420), sb = __byte_perm(d[4 * j + 2], d[4 * j + 3], 0x6420);
                    const uint32_t ya = __byte_perm(sa, sa, 0x2301), yb = __byte_perm(sb, sb, 0x2301);
                    stg_v2(sm_dst + 256 * j, (sa & 0xFEFEFEFEu) | (ya & 0x01010101u), (sb & 0xFEFEFEFEu) | (yb & 0x01010101u));
                    const uint32_t e4a = __byte_perm(d[4 * j], d[4 * j + 1], 0x7531), e4b = __byte_perm(d[4 * j + 2], d[4 * j + 3], 0x7531);
                    unsigned char* rec = pl_dst + 32u * before;
                    before += wd;
                    if (wd == 4u) pack_group_planes<4>(e4a, e4b, base, rec, lane);      // by far the most frequent width
                    else switch (wd) {     // uniform across the warp
                        case 1: pack_group_planes<1>(e4a, e4b, base, rec, lane); break;
                        case 2: pack_group_planes<2>(e4a, e4b, base, rec, lane); break;
                        case 3: pack_group_planes<3>(e4a, e4b, base, rec, lane); break;
                        case 5: pack_group_planes<5>(e4a, e4b, base, rec, lane); break;
                        case 6: pack_group_planes<6>(e4a, e4b, base, rec, lane); break;
                        case 7: pack_group_planes<7>(e4a, e4b, base, rec, lane); break;
                        case 8: pack_group_planes<8>(e4a, e4b, base, rec, lane); break;
                        default: break;
                    }
                }
            } else if (ZEROS && Ssum == kSumConstTile) {
                // the value (any word's low half, rotated back), then 30 zero bytes
                if (warp == 5 && lane < 8u) st_stream_u32(dst + 4u * lane, lane == 0u ? __funnelshift_r(d[0], d[0], 1) & 0xFFFFu : 0u);
            } else if (enc_len) {
                unsigned char* q = dst + warp * 2048u + lane * 4u;
#pragma unroll
                for (int i = 0; i < 16; i++) st_stream_u32(q + i * 128, __funnelshift_r(d[i], d[i], 1));
            }
        } else if (qX >= kQPresent) {
            // rare: the ragged last tile, stored raw
            const uint32_t enc_len = tile_left(g, tXn);
            if (exclX + enc_len > room) {
                trouble |= 1u;
            } else {
                const unsigned char* src = reinterpret_cast<const unsigned char*>(tile_src(tXn));
                unsigned char* dst = payload + exclX;
                for (uint32_t i = tt; i < enc_len; i += kTeamThreads) dst[i] = src[i];
            }
        }

        // What is left to note about X is done by two other warps' first lanes (the leader's
        // warp is the one the team waits for): the digest by warp 1; the table entry, where its
        // chunk starts and the total by warp 7 (not warp 4: warps w and w + 4 issue through the same
        // scheduler, and warp 4 would share the end of the step with the leader's hand-over).
        if (tt == 32u && qX >= kQPresent && is_tile(qX)) ws.dig[tXn] = xor8(tc->wdig[sl]);
        if (tt == 224u && is_tile(qX)) {
            uint32_t entry = 0, enc_len = 0;
            if (qX >= kQPresent) {
                if (tXn < g.n_full_tiles) {
                    const uint32_t Ssum = tc->ssum[sl];
                    if (ENT && (Ssum & kSumEnt)) {
                        enc_len = ent_tile_bytes(Ssum & 0xFFFFu);
                        entry = 0x8000u | (enc_len / 32u);
                    } else {
                        entry = Ssum <= 253u ? 258u + Ssum : (ZEROS && Ssum == kSumZeroTile) ? 1u : (ZEROS && Ssum == kSumConstTile) ? 2u : 512u;
                        enc_len = (ZEROS && entry <= 2u) ? 32u * (entry - 1u) : 32u * entry;
                    }
                } else {
                    entry = 0xFFFFu;
                    enc_len = tile_left(g, tXn);
                }
            }
            tile_tab[tXn] = (uint16_t)entry;
            if (qX & kQFirst) *reinterpret_cast<unsigned long long*>(dir + 16ull * chunk_of(g, tXn)) = exclX;
            if (place_of(sl, tXn) + 1 == n_tickets) ws.ctrl->payload_total = exclX + enc_len;
        }
        if (leader && kLateList) {     // hand over the ticket whose chunk number arrived during this step
            uint32_t qn = kQNone;
            if (haveA) {
                const uint32_t j = chunk_of(g, kA);
                qn = (plA * g.tiles_per_chunk + (kA - j * g.tiles_per_chunk)) | kQPresent | (first_in_chunk(g, kA) ? kQFirst : 0u);
            }
            tc->next[par] = qn;
            tc->kring[(sl + 5u) & 7u] = kA;
            haveA = claiming && tk < n_tickets;
            claiming = haveA;
            kA = tk;
        } else if (leader) {
            uint32_t qn2 = kQNone;
            if (claiming) { qn2 = describe_tile<MASKED>(g, ws.plist, n_tickets, tk); claiming = is_tile(qn2); }
            // (the tile handed over now is measured two steps on, in ring slot sl + 5)
            if (LEAVES) {              // hand over the tile whose address arrived during this step
                tc->next[par] = with_mark(qA, pA);
                tc->nptr[par] = pA;
                if (MASKED) tc->kring[(sl + 5u) & 7u] = kA;
                qA = qn2;
                kA = tk;
            } else {
                tc->next[par] = qn2;
                if (MASKED) tc->kring[(sl + 5u) & 7u] = tk;
            }
        }
        if (tt == 96u) {
            unsigned long long e = 0;
            if (is_tile(qV))
                e = (pv >> 30) == 2u ? (unsigned long long)(pv & kValMask) * kUnit : wait_prefix(ws.lbk, place_of((sl + 1u) & 7u, qV & kQTile), ws.ctrl, g.wait_ns);
            tc->excl[par] = e;
        }
        qX = qV; qV = qW; qW = qY; qY = qN;
        sl = (sl + 1u) & 7u;
        par ^= 1u;
        step++;
    }
    if ((trouble & 1u) && lane == 0) atomicOr(&ws.ctrl->err, 1u);
    // every warp is done with its tensor memory: hand it back before the block exits
    tmem_wait_stores();
    tmem_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) tmem_free_all(s_tmem);
}

// Directory (enc_len, crc), chunk CRCs, present count; the last block to finish combines the
// chunk CRCs into the cache CRC and writes the header (meta_crc left zero).
__global__ void __launch_bounds__(1024)
k_encode_finish(const unsigned char* __restrict__ cache, Geo g, const uint8_t* __restrict__ dirty,
                uint32_t* __restrict__ crc_inout, unsigned char* __restrict__ wire, Ws ws,
                const Tables* __restrict__ tab, const __grid_constant__ ChunkPowers cp, uint32_t option_flags)
{
    __shared__ uint32_t sHT[1024];
    __shared__ uint32_t sT0[256];
    __shared__ FinishStage stage;
    __shared__ uint32_t s_acc;
    __shared__ bool s_last;
    load_ht_t0(sHT, sT0, tab);
    grid_dep_wait();
    grid_dep_launch();
    const uint32_t c0 = blockIdx.x * g.finish_cb;
    stage_chunk_digests(g, stage, ws.dig, c0);
    unsigned char* dir = wire + 64;
    const unsigned long long total = ws.ctrl->payload_total;
    // only finish_cb threads of a block fold chunks (the lookups of a full block would queue up
    // on one SM's shared memory)
    const uint32_t c = c0 + threadIdx.x;
    uint32_t present = 0, term = 0;
    const bool dead = (ld_volatile_u32(&ws.ctrl->err) & 8u) != 0;      // leaf mode: the table was rejected
    if (!dead && threadIdx.x < g.finish_cb && c < g.n_chunks) {
        present = (!dirty || dirty[c]) ? 1u : 0u;
        uint32_t crc;
        if (present) {
            crc = chunk_crc_staged(g, sHT, sT0, stage, ws.dig, chunk_first_byte(g, ws, cache, c), c, threadIdx.x);
            crc_inout[c] = crc;
        } else {
            crc = crc_inout[c];
        }
        // Where the chunk's payload starts: a present chunk's offset was written by the team that
        // placed its first tile; an absent chunk (the main kernel never saw it) starts where the next
        // present chunk does, or at the end of the payload.
        const uint32_t n_list = dirty ? ld_volatile_u32(&ws.ctrl->n_list) : 0u;
        auto starts_at = [&](uint32_t cc) -> unsigned long long {
            if (cc >= g.n_chunks) return total;
            if (!dirty || dirty[cc]) return *reinterpret_cast<const unsigned long long*>(dir + 16ull * cc);
            uint32_t lo = 0, hi = n_list;              // the first listed chunk above cc
            while (lo < hi) {
                const uint32_t mid = (lo + hi) / 2;
                if (ws.plist[mid] < cc) lo = mid + 1; else hi = mid;
            }
            return lo < n_list ? *reinterpret_cast<const unsigned long long*>(dir + 16ull * ws.plist[lo]) : total;
        };
        const unsigned long long po = starts_at(c), nx = starts_at(c + 1);
        if (!present) *reinterpret_cast<unsigned long long*>(dir + 16ull * c) = po;
        *reinterpret_cast<uint32_t*>(dir + 16ull * c + 8) = (uint32_t)(nx - po);
        *reinterpret_cast<uint32_t*>(dir + 16ull * c + 12) = crc;
        term = cache_crc_term(g, cp, crc, c);
    }
    accumulate_cache_crc(ws.ctrl, term, &s_acc);
    const uint32_t cnt = __syncthreads_count(present);
    if (threadIdx.x == 0) {
        if (cnt) atomicAdd(&ws.ctrl->n_present, cnt);
        __threadfence();
        s_last = atomicAdd(&ws.ctrl->done_a, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last || threadIdx.x != 0) return;
    __threadfence();
    const uint32_t cache_crc = ld_volatile_u32(&ws.ctrl->cache_acc);
    const uint32_t n_present = ld_volatile_u32(&ws.ctrl->n_present);
    uint32_t* h = reinterpret_cast<uint32_t*>(wire);
    h[0] = 0x31564D57u;                                  // "WMV1"
    h[1] = 1u | ((dirty ? 1u : 0u) << 16) | (option_flags << 16);      // version, flags (bit 1 zero tiles, bit 2 ENT tiles)
    h[2] = (uint32_t)g.nbytes; h[3] = (uint32_t)(g.nbytes >> 32);
    h[4] = g.chunk_bytes; h[5] = kTile; h[6] = g.n_chunks; h[7] = n_present;
    h[8] = (uint32_t)total; h[9] = (uint32_t)(total >> 32);
    const unsigned long long wl = g.meta_end + total;
    h[10] = (uint32_t)wl; h[11] = (uint32_t)(wl >> 32);
    h[12] = cache_crc; h[13] = 0u; h[14] = 0u; h[15] = 0u;
    ws.ctrl->hdr_cache_crc = cache_crc;
    ws.ctrl->hdr_n_present = n_present;
    ws.ctrl->payload_total = total;
}

}  // namespace wm
