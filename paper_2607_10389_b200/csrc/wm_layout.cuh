// Geometry of a call, the control block and the workspace layout, and the pieces every kernel
// chain shares: chunk arithmetic, the tile digest, the finish kernels' staging and CRC folds.
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

// ------------------------------------------------------------------ geometry / workspace

struct Geo {
    uint64_t nbytes;
    uint64_t meta_end;
    uint32_t chunk_bytes;
    uint32_t tiles_per_chunk;
    uint32_t n_chunks;
    uint32_t n_tiles;
    uint32_t tail_len;        // nbytes mod 16384 (0: the last tile is full)
    uint32_t last_chunk_len;  // bytes of the last chunk
    uint32_t k_tail;          // x^(8 tail_len)
    uint32_t k_chunk;         // x^(8 chunk_bytes)
    uint32_t k_last_chunk;    // x^(8 last_chunk_len)
    uint32_t n_meta_slices;   // ceil(meta_end / 16384)
    uint32_t tpc_shift;       // log2(tiles_per_chunk) when that is a power of two, else 32
    uint32_t n_full_tiles;    // tiles of exactly 16384 bytes
    uint32_t finish_cb;       // chunks handled by one block of the finish kernels
    uint32_t poly;            // reflected CRC polynomial of the k_* powers (CRC32C except in wm_checksum_poly)
    uint32_t inject;          // test hook (wm_inject_stall): kInject* bits, 0 in normal operation
    uint32_t wait_ns;         // budget of every device-side wait (wm_wait_budget_ms; at most 4 s, see now_ns)
};
// Geo::inject.  What a bounded wait waits for is left out, so that the wait runs out and the
// give-up path can be tested without a fault: the scanner warp returns at once (encode), the bulk
// copies into the stages are not issued (checksum, decode).
constexpr uint32_t kInjectNoScanner = 1u, kInjectNoCopy = 2u;

// Powers of k_chunk = x^(8 chunk_bytes), by 7-bit digit of the exponent: k_chunk^e is the product
// of d0[e & 127], d1[(e >> 7) & 127], d2[(e >> 14) & 127] and, beyond 2^21 chunks, of the
// squares hi[j] = k_chunk^(2^(21+j)) that the remaining bits select.  Built on the host once per
// geometry and handed to the finish kernels as an argument.
struct ChunkPowers {
    uint32_t d0[128], d1[128], d2[128];
    uint32_t hi[11];
    uint32_t pad;
};

struct Ctrl {                 // first 256 bytes of the workspace
    uint32_t ticket;
    uint32_t poison;
    uint32_t err;             // bit0 capacity, bit1 timeout, bit2 shared memory carve failed, bit3 leaf table refused
    uint32_t done_a;
    uint32_t done_b;
    uint32_t n_present;
    uint32_t scan_lock;
    uint32_t gate;            // decode: status of an earlier failing step (0 = none)
    uint32_t bad3_first, bad3_count;
    uint32_t bad4_first, bad4_count;
    uint32_t bad5_first, bad5_count;
    uint32_t bad6_first, bad6_count;
    unsigned long long bad4_key;   // lowest failing tile * 2 + (1 if STRUCT)
    unsigned long long payload_total;
    uint32_t hdr_n_present, hdr_cache_crc;
    uint32_t cache_acc;       // XOR of the chunks' terms of the whole-cache CRC
    uint32_t has_pack;        // decode of an image with the entropy option: it holds PACK tiles too
    uint32_t n_walked;        // leaf mode: tiles that go through the side buffer (see k_leaf_map)
    uint32_t n_list;          // masked images: present chunks listed in plist
    uint32_t n_tickets;       // tiles the main kernel has to claim (masked: those of the listed chunks only)
    uint32_t off_bad;         // decode: some chunk's payload_off is not its predecessor's plus that one's enc_len
    uint32_t pad[36];
};
static_assert(sizeof(Ctrl) == 256, "control block is 256 bytes");

// Give up: the call has failed.  The error word says why (bit 1: a wait ran out), waits end early
// once the poison flag is up, and the ticket counter jumps past every tile, so that nobody claims
// another one (claiming itself never has to look at a flag).
__device__ __forceinline__ void give_up(Ctrl* ctrl)
{
    atomicOr(&ctrl->err, 2u);
    atomicExch(&ctrl->poison, 1u);
    atomicMax(&ctrl->ticket, 0x7FFF0000u);
}

// Wait for a bulk copy into a stage: the phase of `bar` with the given parity, for at most
// `budget_ns`.  A copy is started a whole step before it is needed, so the first try nearly
// always succeeds, and everything else happens only after a try has come back empty: the clock is
// read, and when the budget has passed the thread gives up for the whole call, then gives the
// copy one more budget to land (so that the block, and with it the stage, does not go away under
// a copy still in flight) and returns false.  A thread that comes here after the call has been
// given up makes its one try and no more.  `no_second`: test hook, no copy is in flight.
// What follows a first try that came back empty.
__device__ __forceinline__ bool wait_for_copy_rest(uint32_t b, uint32_t parity, uint32_t budget_ns, Ctrl* ctrl, bool no_second)
{
    if (*reinterpret_cast<volatile uint32_t*>(&ctrl->err) & 2u) return false;
    uint32_t t0 = now_ns();
    do {
        if (mbar_try(b, parity)) return true;
    } while (now_ns() - t0 <= budget_ns);
    give_up(ctrl);
    if (no_second) return false;
    t0 = now_ns();
    do {
        if (mbar_try(b, parity)) break;
    } while (now_ns() - t0 <= budget_ns);
    return false;
}
__device__ __noinline__ bool wait_for_copy_rest_call(uint32_t b, uint32_t parity, uint32_t budget_ns, Ctrl* ctrl, bool no_second)
{
    return wait_for_copy_rest(b, parity, budget_ns, ctrl, no_second);
}
// OUT_OF_LINE: the rest is a call.  Which form is faster differs from kernel to kernel (it decides
// how the compiler lays out the hot loop around it); each kernel takes the one measured better.
template <bool OUT_OF_LINE>
__device__ __forceinline__ bool wait_for_copy_at(uint32_t b, uint32_t parity, uint32_t budget_ns, Ctrl* ctrl,
                                                 bool no_second = false)        // b: the barrier's shared-window address
{
    if (mbar_try(b, parity)) return true;
    return OUT_OF_LINE ? wait_for_copy_rest_call(b, parity, budget_ns, ctrl, no_second)
                       : wait_for_copy_rest(b, parity, budget_ns, ctrl, no_second);
}
template <bool OUT_OF_LINE>
__device__ __forceinline__ bool wait_for_copy(unsigned long long* bar, uint32_t parity, uint32_t budget_ns, Ctrl* ctrl,
                                              bool no_second = false)
{
    return wait_for_copy_at<OUT_OF_LINE>((uint32_t)__cvta_generic_to_shared(bar), parity, budget_ns, ctrl, no_second);
}

struct Ws {
    Ctrl* ctrl;
    uint32_t* lbk;               // [n_tiles] placement look-back words
    uint32_t* dig;               // [n_tiles] tile digests
    uint32_t* rel;               // [n_tiles] decode: tile offset inside its chunk's payload
    uint32_t* cflag;             // [n_chunks] bit0 present, bit1..: failed step 3/4/5/6
    uint32_t* ccrc;              // [n_chunks]
    uint32_t* mdig;              // [n_meta_slices]
    unsigned long long* tptr;    // [n_tiles] leaf mode: the address of each tile of the logical cache (see k_leaf_map)
    unsigned long long* lstart;  // [kMaxLeaves + 1] leaf mode: logical offset at which each leaf starts
    uint32_t* plist;             // [n_chunks] masked images: the present chunks (encode: ascending; decode: any order)
    uint32_t* wlist;             // [kMaxWalked] leaf mode: the tiles that go through the side buffer
    unsigned char* side;         // [min(n_tiles, kMaxWalked)][16384] leaf mode: their slots
};
constexpr uint32_t kMaxLeaves = 4096;
constexpr uint32_t kMaxWalked = 2048;        // 32 MiB of side buffer at most

constexpr uint32_t CF_PRESENT = 1, CF_BAD3 = 2, CF_BAD4 = 4, CF_BAD5 = 8, CF_BAD6 = 16;

static inline uint64_t align16(uint64_t v) { return (v + 15) & ~(uint64_t)15; }

struct WsLayout {
    uint64_t state, dig, rel, cflag, ccrc, mdig, tptr, lstart, plist, wlist, side, total;
};

static WsLayout ws_layout(const Geo& g)
{
    WsLayout L;
    uint64_t o = sizeof(Ctrl);
    L.state = o; o = align16(o + 8ull * g.n_tiles);
    L.dig = o;   o = align16(o + 4ull * g.n_tiles);
    L.rel = o;   o = align16(o + 4ull * g.n_tiles);
    L.cflag = o; o = align16(o + 4ull * g.n_chunks);
    L.ccrc = o;  o = align16(o + 4ull * g.n_chunks);
    L.mdig = o;  o = align16(o + 4ull * g.n_meta_slices);
    L.tptr = o;  o = align16(o + 8ull * g.n_tiles);
    L.lstart = o; o = align16(o + 8ull * (kMaxLeaves + 1));
    L.plist = o; o = align16(o + 4ull * g.n_chunks);
    L.wlist = o; o = align16(o + 4ull * kMaxWalked);
    L.side = o; o = align16(o + (uint64_t)kTile * (g.n_tiles < kMaxWalked ? g.n_tiles : kMaxWalked));
    L.total = o;
    return L;
}

static Ws ws_carve(void* base, const Geo& g)
{
    WsLayout L = ws_layout(g);
    unsigned char* b = static_cast<unsigned char*>(base);
    Ws w;
    w.ctrl = reinterpret_cast<Ctrl*>(b);
    w.lbk = reinterpret_cast<uint32_t*>(b + L.state);
    w.dig = reinterpret_cast<uint32_t*>(b + L.dig);
    w.rel = reinterpret_cast<uint32_t*>(b + L.rel);
    w.cflag = reinterpret_cast<uint32_t*>(b + L.cflag);
    w.ccrc = reinterpret_cast<uint32_t*>(b + L.ccrc);
    w.mdig = reinterpret_cast<uint32_t*>(b + L.mdig);
    w.tptr = reinterpret_cast<unsigned long long*>(b + L.tptr);
    w.lstart = reinterpret_cast<unsigned long long*>(b + L.lstart);
    w.plist = reinterpret_cast<uint32_t*>(b + L.plist);
    w.wlist = reinterpret_cast<uint32_t*>(b + L.wlist);
    w.side = b + L.side;
    return w;
}

// Payload offsets travel between blocks as 30-bit counts of 32-byte units, and the payload is
// never longer than the cache, so the codec entry points take caches up to 32 GiB.
constexpr uint64_t kMaxCodecBytes = 32ull << 30;

constexpr uint32_t kFinishDigests = 8192;    // tile digests a finish block stages in shared memory
constexpr uint32_t kFinishChunks = 128;      // at most this many chunks per finish block

// Process-wide settings every call reads when it is issued (atomics: calls come from any thread).
static std::atomic<uint32_t> g_wait_ns{2000u * 1000u * 1000u};         // wm_wait_budget_ms
static std::atomic<uint32_t> g_inject{0};                               // wm_inject_stall

static bool make_geo_fixed(uint64_t nbytes, uint32_t chunk_bytes, Geo& g);
static bool make_geo(uint64_t nbytes, uint32_t chunk_bytes, Geo& g)
{
    if (!make_geo_fixed(nbytes, chunk_bytes, g)) return false;
    g.wait_ns = g_wait_ns.load(std::memory_order_relaxed);
    g.inject = g_inject.load(std::memory_order_relaxed);
    return true;
}

static bool make_geo_fixed(uint64_t nbytes, uint32_t chunk_bytes, Geo& g)
{
    if (nbytes == 0 || chunk_bytes == 0 || chunk_bytes % kTile != 0 || chunk_bytes > (1u << 30)) return false;
    uint64_t nt = (nbytes + kTile - 1) / kTile;
    if (nt > 0xFFFFFFFFull) return false;
    // the powers below cost a few microseconds of host time: keep the last geometry per thread
    static thread_local Geo last;
    static thread_local bool have_last = false;
    if (have_last && last.nbytes == nbytes && last.chunk_bytes == chunk_bytes) { g = last; return true; }
    have_last = false;
    g.inject = 0;
    g.wait_ns = 0;
    g.nbytes = nbytes;
    g.chunk_bytes = chunk_bytes;
    g.tiles_per_chunk = chunk_bytes / kTile;
    g.n_chunks = (uint32_t)((nbytes + chunk_bytes - 1) / chunk_bytes);
    g.n_tiles = (uint32_t)nt;
    g.meta_end = (64ull + 16ull * g.n_chunks + 2ull * g.n_tiles + 31ull) & ~31ull;
    g.tail_len = (uint32_t)(nbytes % kTile);
    g.last_chunk_len = (uint32_t)(nbytes - (uint64_t)(g.n_chunks - 1) * chunk_bytes);
    g.k_tail = x_pow_bytes(g.tail_len);
    g.k_chunk = x_pow_bytes(chunk_bytes);
    g.k_last_chunk = x_pow_bytes(g.last_chunk_len);
    g.n_meta_slices = (uint32_t)((g.meta_end + kTile - 1) / kTile);
    g.n_full_tiles = (uint32_t)(nbytes / kTile);
    g.tpc_shift = 32;
    for (uint32_t k = 0; k < 32; k++)
        if (g.tiles_per_chunk == (1u << k)) g.tpc_shift = k;
    uint32_t cb = kFinishDigests / g.tiles_per_chunk;
    g.finish_cb = cb > kFinishChunks ? kFinishChunks : (cb ? cb : 1u);
    g.poly = kPolyReflected;
    last = g;
    have_last = true;
    return true;
}

// The powers for g (kept per thread for the last chunk size: about 400 products to build).
static const ChunkPowers& chunk_powers(const Geo& g)
{
    static thread_local ChunkPowers cp;
    static thread_local uint32_t for_k = 0;
    static thread_local bool have = false;
    if (have && for_k == g.k_chunk) return cp;
    uint32_t step = g.k_chunk;
    uint32_t* digit[3] = {cp.d0, cp.d1, cp.d2};
    for (int d = 0; d < 3; d++) {
        uint32_t v = 0x80000000u;                       // the polynomial 1
        for (int i = 0; i < 128; i++) { digit[d][i] = v; v = mulmod(v, step); }
        step = v;                                       // step^128
    }
    for (int j = 0; j < 11; j++) { cp.hi[j] = step; step = mulmod(step, step); }
    cp.pad = 0;
    for_k = g.k_chunk;
    have = true;
    return cp;
}

__device__ __forceinline__ uint32_t chunk_of(const Geo& g, uint32_t t)
{
    return g.tpc_shift < 32 ? t >> g.tpc_shift : t / g.tiles_per_chunk;
}
__device__ __forceinline__ bool first_in_chunk(const Geo& g, uint32_t t)
{
    return g.tpc_shift < 32 ? (t & (g.tiles_per_chunk - 1u)) == 0u : (t % g.tiles_per_chunk) == 0u;
}

__device__ __forceinline__ uint64_t chunk_len_dev(const Geo& g, uint32_t c)
{
    return (c + 1 == g.n_chunks) ? g.last_chunk_len : g.chunk_bytes;
}

// A warp's contribution to the digest of the team's tile, from the 16 words each lane holds
// (same value in every lane).  `init_fold`: complement the tile's first word, which folds the
// CRC's all-ones start value into the first tile of a chunk.
__device__ __forceinline__ uint32_t tile_digest_part(const Smem& S, uint32_t (&w)[kWordsPerLane], bool init_fold,
                                                     uint32_t warp, uint32_t lane)
{
    const uint32_t m = (init_fold && warp == 0 && lane == 0) ? 0xFFFFFFFFu : 0u;
    w[0] ^= m;
    const uint32_t d = warp_block_digest(S, w);
    w[0] ^= m;
    return warp_place(S, d, warp, lane);
}

__device__ __forceinline__ uint32_t xor8(const uint32_t* p)
{
    return p[0] ^ p[1] ^ p[2] ^ p[3] ^ p[4] ^ p[5] ^ p[6] ^ p[7];
}

// First byte of chunk c: in the flat buffer, or (leaf mode, flat == nullptr) where the chunk's
// first tile is (for the only chunk ever asked for, the ragged last one, that is its slot in the
// side buffer).  Only chunks shorter than four bytes are read through it.
__device__ __forceinline__ const unsigned char* chunk_first_byte(const Geo& g, const Ws& ws, const unsigned char* flat, uint32_t c)
{
    if (flat) return flat + (uint64_t)c * g.chunk_bytes;
    return chunk_len_dev(g, c) < 4 ? reinterpret_cast<const unsigned char*>(ws.tptr[(uint64_t)c * g.tiles_per_chunk]) : nullptr;
}

// CRC32C of chunk c from its tiles' digests (Horner over tiles; the all-ones init was folded
// into the first tile's digest, the final complement is applied here).  `bytes`: the chunk's
// first byte (read only when the chunk is shorter than four bytes).
__device__ uint32_t chunk_crc_from_digests(const Geo& g, const uint32_t* HT, const uint32_t* T0,
                                           const uint32_t* dig, const unsigned char* bytes, uint32_t c)
{
    const uint64_t clen = chunk_len_dev(g, c);
    if (clen < 4) return crc_bytewise(T0, bytes, (uint32_t)clen);
    const uint32_t t0 = c * g.tiles_per_chunk;
    const uint32_t ntc = (uint32_t)((clen + kTile - 1) / kTile);
    const bool ragged = (clen % kTile) != 0;
    uint32_t st = 0;
    uint32_t i = 0;
    // full tiles, eight at a time: the digests are fetched first (independent loads), then folded
    const uint32_t n_plain = ragged ? ntc - 1 : ntc;
    if ((t0 & 3u) == 0) {
        for (; i + 8 <= n_plain; i += 8) {
            const uint4 a = __ldcg(reinterpret_cast<const uint4*>(dig + t0 + i));
            const uint4 b = __ldcg(reinterpret_cast<const uint4*>(dig + t0 + i + 4));
            st = advance_tile(HT, st) ^ a.x; st = advance_tile(HT, st) ^ a.y;
            st = advance_tile(HT, st) ^ a.z; st = advance_tile(HT, st) ^ a.w;
            st = advance_tile(HT, st) ^ b.x; st = advance_tile(HT, st) ^ b.y;
            st = advance_tile(HT, st) ^ b.z; st = advance_tile(HT, st) ^ b.w;
        }
    }
    for (; i < ntc; i++) {
        if (i + 1 == ntc && ragged) st = mulmod_dev(st, g.k_tail, g.poly);
        else st = advance_tile(HT, st);
        st ^= __ldcg(dig + t0 + i);
    }
    return ~st;
}

__device__ __forceinline__ void load_ht_t0(uint32_t* sHT, uint32_t* sT0, const Tables* tab)
{
    for (uint32_t i = threadIdx.x; i < 1024; i += blockDim.x) sHT[i] = (&tab->HT[0][0])[i];
    for (uint32_t i = threadIdx.x; i < 256; i += blockDim.x) sT0[i] = tab->T0[i];
    __syncthreads();
}

// Finish blocks: a block owns g.finish_cb consecutive chunks.  Their tiles' digests are one
// contiguous run, copied to shared memory with coalesced loads (one round trip to L2 for the
// block instead of one per few digests of a serial fold); thread i then folds chunk c0 + i out
// of shared memory.  A chunk's digests sit at stride tiles_per_chunk + 1 so that the threads'
// reads fall on different banks.  Chunks with more tiles than the stage holds are folded
// from global memory.  Block-wide: every thread calls; ends with a block barrier.
struct FinishStage {
    uint32_t dig[kFinishDigests + kFinishChunks];
};

__device__ void stage_chunk_digests(const Geo& g, FinishStage& st, const uint32_t* __restrict__ dig, uint32_t c0)
{
    const uint32_t tpc = g.tiles_per_chunk;
    if (tpc <= kFinishDigests) {
        const uint64_t t0 = (uint64_t)c0 * tpc;
        uint64_t t1 = t0 + (uint64_t)g.finish_cb * tpc;
        if (t1 > g.n_tiles) t1 = g.n_tiles;
        for (uint32_t i = threadIdx.x; t0 + i < t1; i += blockDim.x) {
            const uint32_t ch = g.tpc_shift < 32 ? i >> g.tpc_shift : i / tpc;
            st.dig[i + ch] = __ldcg(dig + t0 + i);          // ch * (tpc + 1) + (i - ch * tpc)
        }
    }
    __syncthreads();
}

// CRC32C of chunk c = c0 + i from the staged digests (Horner over tiles; the all-ones start
// value was folded into the first tile's digest, the final complement is applied here).
__device__ uint32_t chunk_crc_staged(const Geo& g, const uint32_t* HT, const uint32_t* T0, const FinishStage& st,
                                     const uint32_t* dig, const unsigned char* bytes, uint32_t c, uint32_t i)
{
    if (g.tiles_per_chunk > kFinishDigests) return chunk_crc_from_digests(g, HT, T0, dig, bytes, c);
    const uint64_t clen = chunk_len_dev(g, c);
    if (clen < 4) return crc_bytewise(T0, bytes, (uint32_t)clen);
    const uint32_t ntc = (uint32_t)((clen + kTile - 1) / kTile);
    const bool ragged = (clen % kTile) != 0;
    const uint32_t* d = st.dig + (size_t)i * (g.tiles_per_chunk + 1u);
    uint32_t s = 0;
    const uint32_t n_plain = ragged ? ntc - 1 : ntc;
    for (uint32_t k = 0; k < n_plain; k++) s = advance_tile(HT, s) ^ d[k];
    if (ragged) s = mulmod_dev(s, g.k_tail, g.poly) ^ d[ntc - 1];
    return ~s;
}

// Chunk c's term of the whole-cache CRC: crc(A || B) = crc(A) x^(8 len B) + crc(B), so the CRC
// of all chunks in a row is the sum over chunks of crc_c times x^(8 * bytes after chunk c).
// Every chunk but the last has the same length: the factor is k_last_chunk * k_chunk^e with
// e = number of full chunks after c.
__device__ uint32_t cache_crc_term(const Geo& g, const ChunkPowers& cp, uint32_t crc, uint32_t c)
{
    if (c + 1 == g.n_chunks) return crc;
    uint32_t e = g.n_chunks - 2u - c;
    uint32_t f = mulmod_dev(crc, g.k_last_chunk);
    if (e & 127u) f = mulmod_dev(f, cp.d0[e & 127u]);
    if ((e >> 7) & 127u) f = mulmod_dev(f, cp.d1[(e >> 7) & 127u]);
    if ((e >> 14) & 127u) f = mulmod_dev(f, cp.d2[(e >> 14) & 127u]);
    e >>= 21;
    for (uint32_t j = 0; e; j++, e >>= 1)
        if (e & 1u) f = mulmod_dev(f, cp.hi[j]);
    return f;
}

// XOR the threads' terms into ctrl->cache_acc (block-wide; one atomic per block).
__device__ void accumulate_cache_crc(Ctrl* ctrl, uint32_t term, uint32_t* s_acc)
{
    if (threadIdx.x == 0) *s_acc = 0;
    __syncthreads();
    const uint32_t w = __reduce_xor_sync(0xFFFFFFFFu, term);
    if ((threadIdx.x & 31u) == 0 && w) atomicXor(s_acc, w);
    __syncthreads();
    if (threadIdx.x == 0 && *s_acc) atomicXor(&ctrl->cache_acc, *s_acc);
}

}  // namespace wm
