// CUDA kernels (sm_100a) and C ABI of the session mover's data path.
//
// Kernel map (every call enqueues a short chain on the caller's stream, no host sync):
//   wm_checksum      : k_tile_digests -> k_checksum_finish
//   wm_dirty_diff    : k_diff_init -> k_diff -> k_diff_compact
//   wm_encode        : k_encode_init -> k_encode (single pass; teams publish tile lengths, one
//                      scanner warp turns them into payload offsets) -> k_encode_finish (directory, cache CRC, header)
//                      -> k_meta_crc (metadata CRC, result)
//   wm_decode_verify : k_decode_init -> k_decode_check (header, metadata CRC, structure: the gate)
//                      -> k_decode (unpack + CRC of decoded bytes) -> k_decode_finish
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>

#include <cuda_runtime.h>

#include "../../include/wm.h"
#include "wm_device.cuh"

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
};

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
    uint32_t err;             // bit0 capacity, bit1 timeout
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
    uint32_t pad[40];
};
static_assert(sizeof(Ctrl) == 256, "control block is 256 bytes");

struct Ws {
    Ctrl* ctrl;
    uint32_t* lbk;               // [n_tiles] placement look-back words
    uint32_t* dig;               // [n_tiles] tile digests
    uint32_t* rel;               // [n_tiles] decode: tile offset inside its chunk's payload
    uint32_t* cflag;             // [n_chunks] bit0 present, bit1..: failed step 3/4/5/6
    uint32_t* ccrc;              // [n_chunks]
    uint32_t* mdig;              // [n_meta_slices]
    unsigned char** tptr;        // [n_tiles] leaf mode: where each tile of the logical cache lives
};

constexpr uint32_t CF_PRESENT = 1, CF_BAD3 = 2, CF_BAD4 = 4, CF_BAD5 = 8, CF_BAD6 = 16;

static inline uint64_t align16(uint64_t v) { return (v + 15) & ~(uint64_t)15; }

struct WsLayout {
    uint64_t state, dig, rel, cflag, ccrc, mdig, tptr, total;
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
    w.tptr = reinterpret_cast<unsigned char**>(b + L.tptr);
    return w;
}

// Payload offsets travel between blocks as 30-bit counts of 32-byte units, and the payload is
// never longer than the cache, so the codec entry points take caches up to 32 GiB.
constexpr uint64_t kMaxCodecBytes = 32ull << 30;

constexpr uint32_t kFinishDigests = 8192;    // tile digests a finish block stages in shared memory
constexpr uint32_t kFinishChunks = 128;      // at most this many chunks per finish block

static bool make_geo(uint64_t nbytes, uint32_t chunk_bytes, Geo& g)
{
    if (nbytes == 0 || chunk_bytes == 0 || chunk_bytes % kTile != 0 || chunk_bytes > (1u << 30)) return false;
    uint64_t nt = (nbytes + kTile - 1) / kTile;
    if (nt > 0xFFFFFFFFull) return false;
    // the powers below cost a few microseconds of host time: keep the last geometry per thread
    static thread_local Geo last;
    static thread_local bool have_last = false;
    if (have_last && last.nbytes == nbytes && last.chunk_bytes == chunk_bytes) { g = last; return true; }
    have_last = false;
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
// first tile lives.  Only chunks shorter than four bytes are ever read through it.
__device__ __forceinline__ const unsigned char* chunk_first_byte(const Geo& g, const Ws& ws, const unsigned char* flat, uint32_t c)
{
    if (flat) return flat + (uint64_t)c * g.chunk_bytes;
    return chunk_len_dev(g, c) < 4 ? ws.tptr[(uint64_t)c * g.tiles_per_chunk] : nullptr;
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

// ------------------------------------------------------------------ wm_checksum

// Tile digests of the whole cache: static striding over tiles.  Each team owns one 16 KiB stage
// that bulk copies (TMA) fill; the team takes its 16 words per lane out of the stage, hands
// the stage to the copy of its next tile and digests from registers meanwhile.
struct DigTeamCtl {
    uint32_t wdig[2][8];
    unsigned long long mbar;
    unsigned long long pad;
};
static_assert(sizeof(DigTeamCtl) % 16 == 0, "team control block keeps 16-byte alignment");

template <int TEAMS>
__global__ void __launch_bounds__(TEAMS * 256, 1)
k_tile_digests(const unsigned char* __restrict__ cache, Geo g, Ws ws, const Tables* __restrict__ tab)
{
    grid_dep_launch();
    extern __shared__ __align__(16) unsigned char smem[];
    Smem S = setup_smem(smem, tab);
    const uint32_t team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads;
    const uint32_t warp = tt / 32, lane = tt % 32;
    unsigned char* stage = nullptr;
    for (int i = 0; i < TEAMS; i++) {          // every thread carves the same blocks in the same order
        unsigned char* p = S.take(kTile);
        if ((uint32_t)i == team) stage = p;
    }
    DigTeamCtl* tc = reinterpret_cast<DigTeamCtl*>(S.take(TEAMS * sizeof(DigTeamCtl)));
    if (!S.ok) { if (threadIdx.x == 0) atomicOr(&ws.ctrl->err, 4u); return; }
    tc += team;
    const uint64_t stride = (uint64_t)gridDim.x * TEAMS;
    const uint64_t pol = l2_policy_evict_first();
    auto full = [&](uint64_t tile) { return tile < g.n_tiles && g.nbytes - tile * kTile >= kTile; };
    auto start_copy = [&](uint64_t tile) {     // thread 0 only
        if (full(tile)) bulk_load(stage, cache + tile * kTile, kTile, &tc->mbar, pol);
    };

    uint64_t t = (uint64_t)blockIdx.x * TEAMS + team;
    if (tt == 64u) { mbar_init(&tc->mbar, 1); start_copy(t); }
    team_bar(team);
    uint32_t phase = 0, par = 0;
    uint64_t t_done = ~0ull;                     // tile whose digest parts wait in wdig[par ^ 1]
    // One team barrier per tile.  The single-lane chores sit on different warps (the team waits
    // for whichever warp has the most to do): warp 2 starts the next copy, warp 1 folds and
    // stores the previous tile's digest once the barrier has made its parts complete.
    for (; t < g.n_tiles; t += stride) {
        const bool first = first_in_chunk(g, (uint32_t)t);
        uint32_t d[kWordsPerLane];
        bool fold = first;
        if (full(t)) {
            if (!mbar_wait(&tc->mbar, phase) && lane == 0) atomicOr(&ws.ctrl->err, 2u);
            phase ^= 1u;
            read_staged_words(stage, warp, lane, d);
        } else {
            load_tile_words_guarded(cache + t * kTile, (uint32_t)(g.nbytes - t * kTile), first, warp, lane, d);
            fold = false;
        }
        team_bar(team);                          // stage free; the previous tile's digest parts complete
        if (tt == 64u) start_copy(t + stride);
        if (tt == 32u && t_done != ~0ull) ws.dig[t_done] = xor8(tc->wdig[par ^ 1u]);
        const uint32_t v = tile_digest_part(S, d, fold, warp, lane);
        if (lane == 0) tc->wdig[par][warp] = v;
        t_done = t;
        par ^= 1u;
    }
    team_bar(team);
    if (tt == 32u && t_done != ~0ull) ws.dig[t_done] = xor8(tc->wdig[par ^ 1u]);
}

__global__ void __launch_bounds__(1024)
k_checksum_finish(const unsigned char* __restrict__ cache, Geo g, Ws ws, const Tables* __restrict__ tab,
                  uint32_t* __restrict__ crc_out)
{
    __shared__ uint32_t sHT[1024];
    __shared__ uint32_t sT0[256];
    __shared__ FinishStage stage;
    load_ht_t0(sHT, sT0, tab);
    grid_dep_wait();
    const uint32_t c0 = blockIdx.x * g.finish_cb;
    stage_chunk_digests(g, stage, ws.dig, c0);
    const uint32_t c = c0 + threadIdx.x;
    if (threadIdx.x < g.finish_cb && c < g.n_chunks)
        crc_out[c] = chunk_crc_staged(g, sHT, sT0, stage, ws.dig, cache + (uint64_t)c * g.chunk_bytes, c, threadIdx.x);
}

// ------------------------------------------------------------------ wm_dirty_diff

__global__ void k_diff_init(Ws ws)
{
    grid_dep_launch();
    if (threadIdx.x == 0 && blockIdx.x == 0) { ws.ctrl->ticket = 0; ws.ctrl->n_present = 0; }
}

// One block per chunk at a time (ticketed); the chunk is scanned in 32 KiB steps and dropped
// at the first step that shows a difference.
__global__ void __launch_bounds__(256)
k_diff(const unsigned char* __restrict__ cache, const unsigned char* __restrict__ prev, Geo g, Ws ws,
       uint8_t* __restrict__ dirty_out)
{
    __shared__ uint32_t s_chunk;
    constexpr uint32_t kStep = 256 * 16 * 8;      // bytes per block step
    grid_dep_wait();
    grid_dep_launch();
    while (true) {
        __syncthreads();
        if (threadIdx.x == 0) s_chunk = atomicAdd(&ws.ctrl->ticket, 1u);
        __syncthreads();
        const uint32_t c = s_chunk;
        if (c >= g.n_chunks) break;
        const uint64_t base = (uint64_t)c * g.chunk_bytes;
        const uint64_t clen = chunk_len_dev(g, c);
        const uint64_t vec_len = clen & ~(uint64_t)15;
        int any = 0;
        for (uint64_t o = 0; o < vec_len; o += kStep) {
            uint4 a[8], b[8];
#pragma unroll
            for (int k = 0; k < 8; k++) {
                uint64_t p = o + ((uint64_t)k * 256 + threadIdx.x) * 16;
                if (p < vec_len) {
                    a[k] = __ldcs(reinterpret_cast<const uint4*>(cache + base + p));
                    b[k] = __ldcs(reinterpret_cast<const uint4*>(prev + base + p));
                } else {
                    a[k] = make_uint4(0, 0, 0, 0); b[k] = a[k];
                }
            }
            uint32_t d = 0;
#pragma unroll
            for (int k = 0; k < 8; k++)
                d |= (a[k].x ^ b[k].x) | (a[k].y ^ b[k].y) | (a[k].z ^ b[k].z) | (a[k].w ^ b[k].w);
            any = __syncthreads_or(d != 0);
            if (any) break;
        }
        if (!any && vec_len < clen) {             // ragged tail of the last chunk, < 16 bytes
            uint32_t d = 0;
            if (threadIdx.x < clen - vec_len)
                d = cache[base + vec_len + threadIdx.x] != prev[base + vec_len + threadIdx.x];
            any = __syncthreads_or(d);
        }
        if (threadIdx.x == 0) dirty_out[c] = any ? 1 : 0;
    }
}

// Ascending index list of dirty chunks and their count (one block, ballot + popc scan).
__global__ void __launch_bounds__(1024)
k_diff_compact(Geo g, const uint8_t* __restrict__ dirty, uint32_t* __restrict__ idx_out, uint32_t* __restrict__ n_out)
{
    __shared__ uint32_t s_warp[32];
    __shared__ uint32_t s_carry;
    const uint32_t lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    grid_dep_wait();
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (uint32_t base = 0; base < g.n_chunks; base += 1024) {
        const uint32_t c = base + threadIdx.x;
        const bool d = c < g.n_chunks && dirty[c] != 0;
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, d);
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        uint32_t before = s_carry;
        for (uint32_t w2 = 0; w2 < warp; w2++) before += s_warp[w2];
        if (d && idx_out) idx_out[before + __popc(bal & ((1u << lane) - 1u))] = c;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t tot = 0;
            for (int w2 = 0; w2 < 32; w2++) tot += s_warp[w2];
            s_carry += tot;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) *n_out = s_carry;
}

// ------------------------------------------------------------------ leaf tables

// Leaf mode: the logical cache is the concatenation of `n` leaves (tensors).  Every leaf but
// the last is a whole number of tiles, so a tile never straddles two leaves and all that the
// main kernels need is where each tile lives: tptr[t].  Every block recomputes the leaves'
// first tiles in shared memory (at most 4096 leaves), then the blocks share the tiles.
// A table that breaks the rules (a leaf that is empty, misaligned or not a whole number of
// tiles before the last, or sizes that do not add up to nbytes) raises error bit 8; in decode
// mode it also closes the gate and writes the result record.
constexpr uint32_t kMaxLeaves = 4096;
__global__ void __launch_bounds__(1024)
k_leaf_map(const wm_leaf* __restrict__ leaves, uint32_t n, Geo g, Ws ws, wm_result* result, int decode)
{
    __shared__ uint32_t s_start[kMaxLeaves + 1];       // first tile of each leaf; [n] = total tiles
    __shared__ uint32_t s_wsum[32];
    __shared__ uint32_t s_bad;
    const uint32_t lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    grid_dep_wait();
    grid_dep_launch();
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    // thread i owns leaves 4i .. 4i+3
    uint32_t cnt[4], bad = 0;
    unsigned long long bytes = 0;
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const uint32_t i = 4 * threadIdx.x + k;
        cnt[k] = 0;
        if (i < n) {
            const unsigned long long nb = leaves[i].nbytes;
            const unsigned long long p = reinterpret_cast<unsigned long long>(leaves[i].ptr);
            if (nb == 0 || (p & 15ull) != 0 || (i + 1 < n && nb % kTile != 0)) bad = 1;
            bytes += nb;
            cnt[k] = (uint32_t)((nb + kTile - 1) / kTile);
        }
    }
    const uint32_t mine = cnt[0] + cnt[1] + cnt[2] + cnt[3];
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= (uint32_t)d) incl += o;
    }
    if (lane == 31) s_wsum[warp] = incl;
    // total bytes: the sum is exact modulo 2^64, which is all the comparison below needs
    unsigned long long tot = bytes;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) tot += __shfl_xor_sync(0xFFFFFFFFu, tot, d);
    __shared__ unsigned long long s_bytes[32];
    if (lane == 0) s_bytes[warp] = tot;
    if (bad) s_bad = 1;
    __syncthreads();
    uint32_t before = 0;
    for (uint32_t w2 = 0; w2 < warp; w2++) before += s_wsum[w2];
    uint32_t run = before + incl - mine;
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const uint32_t i = 4 * threadIdx.x + k;
        if (i < n) s_start[i] = run;
        run += cnt[k];
    }
    if (threadIdx.x == 0) {
        unsigned long long all = 0;
        for (int w2 = 0; w2 < 32; w2++) all += s_bytes[w2];
        if (all != g.nbytes) s_bad = 1;
    }
    __syncthreads();
    if (threadIdx.x == 0) s_start[n] = g.n_tiles;
    __syncthreads();
    if (s_bad) {
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            atomicOr(&ws.ctrl->err, 8u);
            if (decode) {
                ws.ctrl->gate = (uint32_t)WM_ERR_ARG;
                wm_result r;
                memset(&r, 0, sizeof r);
                r.status = WM_ERR_ARG;
                *result = r;
            }
        }
        return;
    }
    for (uint32_t t = blockIdx.x * blockDim.x + threadIdx.x; t < g.n_tiles; t += gridDim.x * blockDim.x) {
        uint32_t lo = 0, hi = n;                       // the leaf with start[lo] <= t < start[lo + 1]
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) / 2;
            if (s_start[mid] <= t) lo = mid; else hi = mid;
        }
        ws.tptr[t] = const_cast<unsigned char*>(static_cast<const unsigned char*>(leaves[lo].ptr)) + (uint64_t)(t - s_start[lo]) * kTile;
    }
}

// ------------------------------------------------------------------ wm_encode

__global__ void k_encode_init(Geo g, Ws ws, unsigned char* wire)
{
    grid_dep_launch();
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t t = i; t < g.n_tiles; t += stride) ws.lbk[t] = 0u;
    if (i < sizeof(Ctrl) / 4) reinterpret_cast<uint32_t*>(ws.ctrl)[i] = 0u;
    // zero padding between the tile table and the payload
    const uint64_t tab_end = 64ull + 16ull * g.n_chunks + 2ull * g.n_tiles;
    if (i < g.meta_end - tab_end) wire[tab_end + i] = 0;
}

constexpr uint32_t kFlagA = 1u << 30, kFlagP = 2u << 30, kValMask = (1u << 30) - 1u;
constexpr uint32_t kSpinLimit = 1u << 20;
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
// owners' waits depend only on running code; they are bounded all the same and end in
// WM_ERR_TIMEOUT.
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

// Give up: waits end early once the flag is up, and the ticket counter jumps past every tile,
// so that nobody claims another one (claiming itself never has to look at the flag).
__device__ __forceinline__ void raise_poison(Ctrl* ctrl)
{
    atomicExch(&ctrl->poison, 1u);
    atomicMax(&ctrl->ticket, 0x7FFF0000u);
}
__device__ __forceinline__ uint32_t next_ticket(Ctrl* ctrl)
{
    return atomicAdd(&ctrl->ticket, 1u);
}

// Owner side: exclusive prefix (bytes) of tile t (one lane spins; bounded).
__device__ __forceinline__ unsigned long long wait_prefix(const uint32_t* lbk, uint32_t t, Ctrl* ctrl)
{
    for (uint32_t polls = 0; polls < kSpinLimit; polls++) {
        const uint32_t v = ld_relaxed_u32(lbk + t);
        if ((v >> 30) == 2u) return (unsigned long long)(v & kValMask) * kUnit;
        if ((polls & 1023u) == 1023u && ld_volatile_u32(&ctrl->poison)) break;
    }
    atomicOr(&ctrl->err, 2u);
    raise_poison(ctrl);
    return 0;
}

// Scanner side (one full warp).  A poll copies 512 consecutive entries into shared memory with
// coalesced asynchronous 16-byte copies (one round trip to L2, no registers held meanwhile);
// lane l then owns entries 16 l .. 16 l + 15 of the window.
constexpr int kScanPerLane = 16;
__device__ void scan_tile_lengths(uint32_t* lbk, uint32_t n_tiles, uint32_t lane, Ctrl* ctrl, uint32_t* win)
{
    uint64_t f = 0;                 // first unresolved entry
    uint64_t base = 0;              // units before f
    uint32_t spins = 0;
#ifdef WM_DEBUG_COUNTERS
    uint32_t dbg_iters = 0, dbg_empty = 0;
#endif
    while (f < n_tiles) {
#ifdef WM_DEBUG_COUNTERS
        dbg_iters++;
#endif
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
#ifdef WM_DEBUG_COUNTERS
        if (k == 0) dbg_empty++;
#endif
        if (k == 0) {
            if (++spins > kSpinLimit || ((spins & 1023u) == 1023u && ld_volatile_u32(&ctrl->poison))) {
                if (lane == 0) { atomicOr(&ctrl->err, 2u); raise_poison(ctrl); }
                return;
            }
        } else {
            spins = 0;
        }
    }
#ifdef WM_DEBUG_COUNTERS
    if (lane == 0) { ctrl->pad[0] = dbg_iters; ctrl->pad[1] = dbg_empty; }
#endif
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
    uint32_t wsum[8];       // sum of widths so far | warps arrived << 16 (the last warp publishes)
    uint32_t ssum[8];       // sum of the 32 widths of the slot's tile (set by that last warp), or a mark:
                            // zero tile, constant tile, kSumEnt | halfwords for a tile stored in ENT form
    uint32_t etab[8][8];    // entropy option, per warp: anchor | halfwords of its stream << 8
    uint32_t next[2];       // ticket claimed in this step (>= n_tiles: none left), by step parity
    uint32_t pad[2];
    unsigned long long excl[2];   // offset of the tile packed in the next step, by step parity
    unsigned long long mbar;      // completion of the bulk copy into the team's stage
    unsigned long long pad2;
    const unsigned char* nptr[2]; // leaf mode: where the tile in next[] lives, by step parity
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
// anchor being the rounded mean of the share's exponents; a strand is an LSB-first bit string
// cut into halfwords, and the 32 strands of a share are interleaved in the order a reader
// needs them: at step i every strand whose codeword i is not complete in what it has taken so
// far takes the stream's next halfword, strands in ascending order.
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
// Bytes of an ENT tile whose eight streams hold `halfwords` halfwords in all (a multiple of 32;
// 16384 or more means that the tile is stored raw instead).
__device__ __forceinline__ uint32_t ent_tile_bytes(uint32_t halfwords)
{
    return (8256u + 2u * halfwords + 31u) & ~31u;
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
//     Y  checksummed and measured in this step (its length is published at once)
// The team owns one 16 KiB stage in shared memory that bulk copies (TMA) fill, one tile per
// step, each copy started a whole step before its tile is needed.  A measured tile's words
// (16 registers per lane) are parked in tensor memory until its offset is known, so a tile is
// read from memory once and nothing waits in registers.  Per step:
//     take Y's words from the stage | team barrier | start the copy of the next Y |
//     digest + exponent ranges of Y, publish len(Y) | park Y | fetch X | pack X straight into
//     the wire image
// Meanwhile two round trips to L2 are in flight whose answers are needed a step later: the
// ticket of the tile to measure two steps on and the offset of the tile to pack next.  These and
// the other single-lane chores of a step sit on different warps: the team passes one barrier per
// tile, so it runs at the pace of the warp that has the most to do.
// Template switches: MASKED (a dirty mask was given), LEAVES (the cache is a table of tensors;
// tickets are claimed one step further ahead so that a tile's address can be looked up on the
// way), ZEROS (the zero-tile option), ENT (the entropy option: the measuring step adds up codeword
// lengths instead of taking exponent ranges, the packing step writes the share's interleaved
// stream of halfwords instead of bit planes).
// Packed data goes from registers to the wire image directly: in every region of a PACK tile
// a lane owns an aligned unit at a lane-strided place, so each warp store is one contiguous
// sector-aligned run.  Claiming a tile before the previous offset is known means that, if the
// scanner is late, this team waits while that tile's length is not out yet; with three steps
// of slack that is rare, and it only delays: the teams that hold earlier tiles never depend
// on this one.
// A tile as a team passes it round: its number in the low 30 bits, kQFirst when it is the first
// tile of its chunk, kQPresent when its chunk is encoded; kQNone: no tile.  (The codec takes
// caches of at most 2^21 tiles, so a number never reaches the flag bits.)
constexpr uint32_t kQPresent = 1u << 31, kQFirst = 1u << 30, kQTile = (1u << 30) - 1u, kQNone = kQTile;
// Marks in a team's width table: on a warp's first entry, all 2 KiB of the warp's rows are zero;
// as the sum of the widths, the tile is all zero.
// kWarpConst: all 1024 elements of the warp's rows hold one value (its sign-mantissa byte rides in
// bits 16-23 of the entry, the exponent is the base); kSumConstTile: the tile holds one value.
constexpr uint32_t kWarpAllZero = 0x8000u, kWarpConst = 0x4000u, kSumZeroTile = 0xFFFFu, kSumConstTile = 0xFFFEu;
// The tile is stored in ENT form (shorter than its bit planes and than raw); low half: halfwords.
constexpr uint32_t kSumEnt = 0x10000u;

template <bool MASKED>
__device__ __forceinline__ uint32_t describe_tile(const Geo& g, const uint8_t* __restrict__ dirty, uint32_t t)
{
    if (t >= g.n_tiles) return kQNone;
    uint32_t q = t;
    if (first_in_chunk(g, t)) q |= kQFirst;
    if (!MASKED || dirty[chunk_of(g, t)] != 0) q |= kQPresent;
    return q;
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
    __shared__ uint32_t s_ent[16];     // ENT: codeword | length << 16 by slot (one bank each: no conflicts)
    __shared__ uint32_t s_len[16];     // ENT: length by slot
    if (ENT && threadIdx.x < 11u) {
        s_ent[threadIdx.x] = (threadIdx.x == 10u ? 0xFFFFu : ent_word(threadIdx.x, 0u)) | (ent_length(threadIdx.x) << 16);
        s_len[threadIdx.x] = ent_length(threadIdx.x);
    }
    Smem S = setup_smem(smem, tab);
    grid_dep_wait();                   // from here on the control block and the length table are ready
    grid_dep_launch();
    if (LEAVES && (ld_volatile_u32(&ws.ctrl->err) & 8u)) return;      // the leaf table was rejected
    if (threadIdx.x == 0) s_scanner = atomicCAS(&ws.ctrl->scan_lock, 0u, 1u) == 0u;
    __syncthreads();
    if (s_scanner) {
        uint32_t* win = reinterpret_cast<uint32_t*>(S.take(2048));      // 512 entries
        if (threadIdx.x < 32 && win) scan_tile_lengths(ws.lbk, g.n_tiles, threadIdx.x, ws.ctrl, win);
        return;
    }
    const uint32_t team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads;
    const uint32_t warp = tt / 32, lane = tt % 32;
    unsigned char* stage = nullptr;
    for (int i = 0; i < TEAMS; i++) {          // every thread carves the same blocks in the same order
        unsigned char* p = S.take(kTile);
        if ((uint32_t)i == team) stage = p;
    }
    EncTeamCtl* tc = reinterpret_cast<EncTeamCtl*>(S.take(TEAMS * sizeof(EncTeamCtl)));
    if (!S.ok) { if (threadIdx.x == 0) atomicOr(&ws.ctrl->err, 4u); return; }
    tc += team;

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
    auto publish_len = [&](uint32_t t, uint32_t len) { st_relaxed_u32(ws.lbk + t, kFlagA | (len / kUnit)); };
    // where tile t lives: the flat cache, or (leaf mode) the table that k_leaf_map filled
    auto tile_src = [&](uint32_t t) -> const unsigned char* {
        return LEAVES ? ws.tptr[t] : cache + (uint64_t)t * kTile;
    };
    auto start_copy = [&](uint32_t q, const unsigned char* src) {   // thread 0 of the team, after the barrier that frees the stage
        if (is_hot(q)) bulk_load(stage, src, kTile, &tc->mbar, pol_once);
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
    if (leader) {
        for (int i = 0; i < 8; i++) tc->wsum[i] = 0;
        mbar_init(&tc->mbar, 1);
        const uint32_t q0 = describe_tile<MASKED>(g, dirty, next_ticket(ws.ctrl));
        const uint32_t q1 = is_tile(q0) ? describe_tile<MASKED>(g, dirty, next_ticket(ws.ctrl)) : kQNone;
        claiming = is_tile(q1);
        tc->next[0] = q0;
        tc->next[1] = q1;
        tc->excl[0] = 0ull;
        tc->excl[1] = 0ull;
        if (LEAVES) {
            tc->nptr[0] = is_tile(q0) ? tile_src(q0 & kQTile) : nullptr;
            tc->nptr[1] = is_tile(q1) ? tile_src(q1 & kQTile) : nullptr;
            if (claiming) { qA = describe_tile<MASKED>(g, dirty, next_ticket(ws.ctrl)); claiming = is_tile(qA); }
        }
    }
    team_bar(team);
    qY = tc->next[0];
    if (leader) start_copy(qY, LEAVES ? tc->nptr[0] : tile_src(qY & kQTile));

    uint32_t trouble = 0;              // sticky: 1 the image does not fit, 2 a copy never arrived
    while (((qX & qV & qW & qY) & kQTile) != kQNone) {
        const bool hotY = is_hot(qY);
        if (hotY) {
            if (!mbar_wait(&tc->mbar, phase)) trouble |= 2u;
            phase ^= 1u;
#pragma unroll
            for (int i = 0; i < 16; i++) d[i] = my_words[i * 32];
        }
        team_bar(team);                   // stage free; what the leader left at the end of the last step is visible
        const uint32_t qN = tc->next[par ^ 1u];
        const unsigned long long exclX = tc->excl[par ^ 1u];
        // The team's single-lane chores are spread over its warps, because the team waits for
        // whichever warp has the most to do.  Warp 2 starts the copy of the next tile (it has the
        // whole step to arrive).  Two round trips to L2 are started now and used at the end of the
        // step: the ticket of the tile to measure two steps on (warp 0, the leader) and the offset
        // of the tile to pack in the next step (warp 3).  Warp 1 notes what is left about X.
        uint32_t pv = 0, tk = 0xFFFFFFFFu;
        const unsigned char* pA = nullptr;
        if (tt == 64u) start_copy(qN, LEAVES ? tc->nptr[par ^ 1u] : tile_src(qN & kQTile));
        if (tt == 96u && is_tile(qV)) pv = ld_relaxed_u32(ws.lbk + (qV & kQTile));
        if (leader) {
            if (claiming) tk = next_ticket(ws.ctrl);
            if (LEAVES && is_tile(qA)) pA = tile_src(qA & kQTile);
        }

        // ---- Y: digest, exponent ranges, length out, words parked
        const uint32_t slY = (sl + 3u) & 7u;
        const uint32_t tYn = qY & kQTile;
        if (hotY) {
#ifdef WM_AB_NOCRC
            const uint32_t v = d[3];
#else
            const uint32_t v = tile_digest_part(S, d, (qY & kQFirst) != 0, warp, lane);
#endif
            // From here on the words are kept rotated left by one bit: each half then reads
            // [E | mantissa | a sign bit], E in its high byte (the two sign bits of a word
            // land in each other's half; the packing step puts them right).
#pragma unroll
            for (int i = 0; i < 16; i++) d[i] = __funnelshift_l(d[i], d[i], 1);
            uint32_t gw[4];               // per group: base | width << 8
            uint32_t ent_w = 0;           // entropy option: anchor | halfwords << 8 of this warp's share
            if (ENT) {
                // the share's anchor (rounded mean of its 1024 exponents: bytes 1 and 3 of a rotated
                // word) and the halfwords its 32 strands need
                uint32_t acc = 0;
#pragma unroll
                for (int i = 0; i < 16; i++) acc += (d[i] >> 8) & 0x00FF00FFu;
                const uint32_t anchor = (__reduce_add_sync(0xFFFFFFFFu, (acc & 0xFFFFu) + (acc >> 16)) + 512u) >> 10;
                uint32_t bits = 0;
#pragma unroll
                for (int i = 0; i < 16; i++)
                    bits += s_len[ent_slot(__byte_perm(d[i], 0u, 0x4441), anchor)] + s_len[ent_slot(d[i] >> 24, anchor)];
                const uint32_t count = __reduce_add_sync(0xFFFFFFFFu, (bits + 15u) >> 4);
                ent_w = anchor | (count << 8);
            }
            {
#ifdef WM_AB_NOMINMAX
            gw[0] = gw[1] = gw[2] = gw[3] = 100u | (4u << 8);
#else
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
#endif
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
            // one lane leaves the warp's results; the warp that arrives last turns the 32 widths
            // into offsets and publishes the tile's length
            uint32_t last = 0;
            if (lane == 0) {
                tc->wdig[slY][warp] = v;
                *reinterpret_cast<uint4*>(&tc->wtab[slY][4 * warp]) = make_uint4(gw[0], gw[1], gw[2], gw[3]);
                if (ENT) tc->etab[slY][warp] = ent_w;
                __threadfence_block();
                last = (atomicAdd(&tc->wsum[slY], 1u) == 7u) ? 1u : 0u;
            }
            if (__shfl_sync(0xFFFFFFFFu, last, 0)) {
                __threadfence_block();
                // (kept short: this warp is the one the team's length waits for; the groups'
                // places inside the tile are worked out by each warp when it packs)
                const uint32_t wt = *reinterpret_cast<volatile uint32_t*>(&tc->wtab[slY][lane]);
                const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, (wt >> 8) & 15u);
                // entropy option: the ENT form is taken when it is shorter than the planes and than raw
                uint32_t halfwords = 0;
                if (ENT) halfwords = __reduce_add_sync(0xFFFFFFFFu, lane < 8u ? *reinterpret_cast<volatile uint32_t*>(&tc->etab[slY][lane]) >> 8 : 0u);
                const uint32_t plane_len = total <= 253u ? 8256u + 32u * total : kTile;
                const bool ent_tile = ENT && ent_tile_bytes(halfwords) < plane_len;
                // unused memory (every warp's first entry carries the mark): no payload
                // (one value throughout: every warp's first entry carries the mark and they are all alike;
                // a tile of zeros has no payload, any other value 32 bytes)
                const uint32_t wt0 = __shfl_sync(0xFFFFFFFFu, wt, 0);
                const bool const_tile = ZEROS && __all_sync(0xFFFFFFFFu, (lane & 3u) != 0u || ((wt & kWarpConst) != 0u && wt == wt0));
                const bool zero_tile = const_tile && (wt0 & kWarpAllZero) != 0u;
                if (lane == 0) {
                    tc->ssum[slY] = zero_tile ? kSumZeroTile : const_tile ? kSumConstTile : ent_tile ? kSumEnt | halfwords : total;
                    tc->wsum[slY] = 0;
                    publish_len(tYn, zero_tile ? 0u : const_tile ? 32u : ent_tile ? ent_tile_bytes(halfwords) : plane_len);
                }
            }
#ifndef WM_AB_NOTMEM
            tmem_store16(tmem_warp + 16u * (step & 3u), d);
#endif
        } else if (is_tile(qY)) {
            // rare: a tile of an absent chunk (length 0) or the ragged last tile (stored raw)
            const bool present = qY >= kQPresent;
            if (tt == 0) publish_len(tYn, present ? tile_left(g, tYn) : 0u);
            if (present) {
                load_tile_words_guarded(tile_src(tYn), tile_left(g, tYn), (qY & kQFirst) != 0, warp, lane, d);
                const uint32_t v = tile_digest_part(S, d, false, warp, lane);
                if (lane == 0) tc->wdig[slY][warp] = v;
            }
        }

        // ---- X: its words back from tensor memory, packed straight into the wire image
        const uint32_t tXn = qX & kQTile;
        if (is_hot(qX)) {
#ifndef WM_AB_NOTMEM
            tmem_load16(tmem_warp + 16u * ((step + 1u) & 3u), d);
#endif
            const uint32_t Smark = tc->ssum[sl];
            const bool ent_form = ENT && (Smark & kSumEnt) != 0u;
            const uint32_t Ssum = ent_form ? Smark & 0xFFFFu : Smark;       // halfwords, or the sum of the widths
            const bool packs = !ent_form && Ssum <= 253u;
            // (a tile of all-zero bytes, marked in ssum, is its table entry and nothing else)
            const uint32_t enc_len = ent_form ? ent_tile_bytes(Ssum)
                                         : packs ? 8256u + 32u * Ssum : (ZEROS && Ssum == kSumZeroTile) ? 0u
                                         : (ZEROS && Ssum == kSumConstTile) ? 32u : kTile;
            unsigned char* const dst = payload + exclX;
            if (exclX + enc_len > room) {
                trouble |= 1u;
            } else if (ent_form) {
                // header: anchors, stream lengths, 40 zero bytes; zero fill behind the last stream
                if (warp == 5) {
                    if (lane < 8u) {
                        const uint32_t wt = tc->etab[sl][lane];
                        stg_u8(dst + lane, wt & 0xFFu);
                        stg_u16(dst + 8u + 2u * lane, wt >> 8);
                    } else if (lane < 18u) {
                        st_stream_u32(dst + 24u + 4u * (lane - 8u), 0u);
                    }
                    if (2u * lane < enc_len - 8256u - 2u * Ssum) stg_u16(dst + 8256u + 2u * Ssum + 2u * lane, 0u);
                }
                unsigned char* const sm_dst = dst + sm_off;
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint32_t sa = __byte_perm(d[4 * j], d[4 * j + 1], 0x6420), sb = __byte_perm(d[4 * j + 2], d[4 * j + 3], 0x6420);
                    const uint32_t ya = __byte_perm(sa, sa, 0x2301), yb = __byte_perm(sb, sb, 0x2301);
                    stg_v2(sm_dst + 256 * j, (sa & 0xFEFEFEFEu) | (ya & 0x01010101u), (sb & 0xFEFEFEFEu) | (yb & 0x01010101u));
                }
                // this share's stream: it starts behind the streams of the warps before it
                const uint32_t before = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? tc->etab[sl][lane] >> 8 : 0u);
                const uint32_t anchor = tc->etab[sl][warp] & 0xFFu;
                unsigned char* const hw_dst = dst + 8256u + 2u * before;
                const uint32_t lt_mask = (1u << lane) - 1u;
                // acc: the strand's bits from the start of the halfword it took last (number `pend` of
                // the stream) on; n of them are valid.  Step 0: every strand takes one halfword.
                uint32_t acc = 0, n = 0, pend = lane, pos = 32;
#pragma unroll
                for (int i = 0; i < 32; i++) {
                    const uint32_t E = (i & 1) ? d[i >> 1] >> 24 : __byte_perm(d[i >> 1], 0u, 0x4441);
                    const uint32_t cw = s_ent[ent_slot(E, anchor)];
                    // (the table's escape entry is 0xFFFF: the AND lets the exponent through there only)
                    acc |= (cw & ((E << 8) | 0xFFu)) << n;
                    n += cw >> 16;
                    if (i == 0) continue;
                    const bool more = n > 16u;             // the codeword runs past what the strand has taken
                    const uint32_t takers = __ballot_sync(0xFFFFFFFFu, more);
                    if (more) {
                        stg_u16(hw_dst + 2u * pend, acc & 0xFFFFu);
                        acc >>= 16;
                        n -= 16u;
                        pend = pos + __popc(takers & lt_mask);
                    }
                    pos += __popc(takers);
                }
                stg_u16(hw_dst + 2u * pend, acc & 0xFFFFu);
            } else if (packs) {
#ifndef WM_AB_NOPACK
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
#else
                if (d[5] == 0x12345678u) stg_u8(dst + lane, d[1]);
#endif
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
                const unsigned char* src = tile_src(tXn);
                unsigned char* dst = payload + exclX;
                for (uint32_t i = tt; i < enc_len; i += kTeamThreads) dst[i] = src[i];
            }
        }

        // What is left to note about X is done by two other warps' first lanes (the leader's
        // warp is the one the team waits for): the digest by warp 1; the table entry, where its
        // chunk starts and the total by warp 4.
        if (tt == 32u && qX >= kQPresent && is_tile(qX)) ws.dig[tXn] = xor8(tc->wdig[sl]);
        if (tt == 128u && is_tile(qX)) {
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
            if (tXn + 1 == g.n_tiles) ws.ctrl->payload_total = exclX + enc_len;
        }
        if (leader) {
            uint32_t qn2 = kQNone;
            if (claiming) { qn2 = describe_tile<MASKED>(g, dirty, tk); claiming = is_tile(qn2); }
            if (LEAVES) {              // hand over the tile whose address arrived during this step
                tc->next[par] = qA;
                tc->nptr[par] = pA;
                qA = qn2;
            } else {
                tc->next[par] = qn2;
            }
        }
        if (tt == 96u) {
#ifdef WM_DEBUG_COUNTERS
            atomicAdd(&ws.ctrl->pad[(pv >> 30) == 2u ? 3 : 2], 1u);
#endif
            unsigned long long e = 0;
            if (is_tile(qV))
                e = (pv >> 30) == 2u ? (unsigned long long)(pv & kValMask) * kUnit : wait_prefix(ws.lbk, qV & kQTile, ws.ctrl);
            tc->excl[par] = e;
        }
        qX = qV; qV = qW; qW = qY; qY = qN;
        sl = (sl + 1u) & 7u;
        par ^= 1u;
        step++;
    }
    if (trouble && lane == 0) {
        atomicOr(&ws.ctrl->err, trouble);
        if (trouble & 2u) raise_poison(ws.ctrl);
    }
    // every warp is done with its tensor memory: hand it back before the block exits
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
        const unsigned long long po = *reinterpret_cast<const unsigned long long*>(dir + 16ull * c);
        const unsigned long long nx = (c + 1 < g.n_chunks)
                                          ? *reinterpret_cast<const unsigned long long*>(dir + 16ull * (c + 1)) : total;
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

// ---- metadata CRC and structure checks ----
// CRC32C of the metadata region wire[0, meta_end) with the meta_crc field read as zero.  The
// region is right-aligned in a whole number of virtual 16 KiB slices (leading zeros), one team
// per slice, four teams per block; the last block to finish folds the slice digests.  These
// kernels see a few hundred kilobytes: they use the small tables.

// The header against the call's arguments (decode step 1).
__device__ __forceinline__ bool header_matches(const unsigned char* wire, uint64_t wire_len, const Geo& g, uint32_t expect_ent)
{
    if (wire_len < 64) return false;
    const uint32_t* h = reinterpret_cast<const uint32_t*>(wire);
    const unsigned long long nb = h[2] | ((unsigned long long)h[3] << 32);
    const unsigned long long pb = h[8] | ((unsigned long long)h[9] << 32);
    const unsigned long long wl = h[10] | ((unsigned long long)h[11] << 32);
    return !(h[0] != 0x31564D57u || (h[1] & 0xFFFFu) != 1u || (h[1] >> 16) > 7u || ((h[1] >> 18) & 1u) != expect_ent || nb != g.nbytes ||
             h[4] != g.chunk_bytes || h[5] != kTile || h[6] != g.n_chunks || wl != wire_len ||
             wire_len < g.meta_end || pb != wire_len - g.meta_end);
}

// One team: its warps' parts of the digest of metadata slice s go to wdig[0..7].
__device__ __forceinline__ void meta_slice_parts(const unsigned char* wire, const Geo& g, uint32_t s, const uint32_t* sG,
                                                 const Tables* __restrict__ tab, uint32_t* wdig, uint32_t warp, uint32_t lane)
{
    const uint64_t pad = (uint64_t)g.n_meta_slices * kTile - g.meta_end;    // multiple of 4
    uint32_t w[kWordsPerLane];
#pragma unroll
    for (int i = 0; i < 16; i++) {
        const uint64_t vb = (uint64_t)s * kTile + (warp * 16 + i) * 128 + lane * 4;
        uint32_t v = 0;
        if (vb >= pad) {
            const uint64_t rb = vb - pad;
            v = *reinterpret_cast<const uint32_t*>(wire + rb);
            if (rb == 52) v = 0;                      // the meta_crc field reads as zero
            if (rb == 0) v ^= 0xFFFFFFFFu;            // the CRC's all-ones start value
        }
        w[i] = v;
    }
    const uint32_t v = tile_digest_part_small(sG, tab, w, warp, lane);
    if (lane == 0) wdig[warp] = v;
}

// Whole block: fold the slice digests (fetched 1024 at a time, one round trip to L2 per batch,
// folded by one thread out of shared memory).  The CRC is valid in thread 0.
__device__ uint32_t fold_meta_digests(const Geo& g, const Ws& ws, const uint32_t* sHT, uint32_t* s_dig)
{
    uint32_t st = 0;
    for (uint32_t b0 = 0; b0 < g.n_meta_slices; b0 += 1024) {
        const uint32_t nb = min(1024u, g.n_meta_slices - b0);
        __syncthreads();
        if (threadIdx.x < nb) s_dig[threadIdx.x] = ld_volatile_u32(&ws.mdig[b0 + threadIdx.x]);
        __syncthreads();
        if (threadIdx.x == 0)
            for (uint32_t i = 0; i < nb; i++) st = advance_tile(sHT, st) ^ s_dig[i];
    }
    return ~st;
}

// Encode: the metadata CRC goes into the header, the result record is written.  This kernel
// starts while k_encode_finish still runs, so copying the large tables costs nothing here and
// the digest itself is the fast one.
__global__ void __launch_bounds__(1024, 1)
k_meta_crc(unsigned char* wire, Geo g, Ws ws, const Tables* __restrict__ tab, wm_result* result)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ bool s_last;
    Smem S = setup_smem(smem, tab);
    const uint32_t team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads;
    const uint32_t warp = tt / 32, lane = tt % 32;
    uint32_t* s_wdig = reinterpret_cast<uint32_t*>(S.take(4 * 8 * 4));
    uint32_t* sHT = reinterpret_cast<uint32_t*>(S.take(4096));
    uint32_t* s_dig = reinterpret_cast<uint32_t*>(S.take(4096));
    if (!S.ok) { if (threadIdx.x == 0) atomicOr(&ws.ctrl->err, 4u); grid_dep_wait(); return; }
    s_wdig += 8 * team;
    sHT[threadIdx.x] = (&tab->HT[0][0])[threadIdx.x];
    grid_dep_wait();
    const uint64_t pad = (uint64_t)g.n_meta_slices * kTile - g.meta_end;    // multiple of 4
    const uint32_t s = blockIdx.x * 4 + team;
    if (s < g.n_meta_slices) {
        uint32_t w[kWordsPerLane];
#pragma unroll
        for (int i = 0; i < 16; i++) {
            const uint64_t vb = (uint64_t)s * kTile + (warp * 16 + i) * 128 + lane * 4;
            uint32_t v = 0;
            if (vb >= pad) {
                const uint64_t rb = vb - pad;
                v = *reinterpret_cast<const uint32_t*>(wire + rb);
                if (rb == 52) v = 0;                      // the meta_crc field reads as zero
                if (rb == 0) v ^= 0xFFFFFFFFu;            // the CRC's all-ones start value
            }
            w[i] = v;
        }
        const uint32_t v = tile_digest_part(S, w, false, warp, lane);
        if (lane == 0) s_wdig[warp] = v;
    }
    __syncthreads();
    if (tt == 0 && s < g.n_meta_slices) ws.mdig[s] = xor8(s_wdig);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&ws.ctrl->done_b, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const uint32_t crc = fold_meta_digests(g, ws, sHT, s_dig);
    if (threadIdx.x != 0) return;
    reinterpret_cast<uint32_t*>(wire)[13] = crc;
    wm_result r;
    memset(&r, 0, sizeof r);
    const uint32_t err = ld_volatile_u32(&ws.ctrl->err);
    r.status = (err & 8u) ? WM_ERR_ARG : (err & 4u) ? WM_ERR_CUDA : (err & 2u) ? WM_ERR_TIMEOUT : (err & 1u) ? WM_ERR_CAPACITY : WM_OK;
    r.n_present = ws.ctrl->hdr_n_present;
    r.payload_bytes = ws.ctrl->payload_total;
    r.wire_len = g.meta_end + ws.ctrl->payload_total;
    r.cache_crc = ws.ctrl->hdr_cache_crc;
    *result = r;
}

// ------------------------------------------------------------------ wm_decode_verify

__global__ void k_decode_init(Ws ws)
{
    grid_dep_launch();
    if (blockIdx.x == 0 && threadIdx.x < sizeof(Ctrl) / 4) {
        uint32_t v = 0;
        const uint32_t i = threadIdx.x;
        if (i == offsetof(Ctrl, bad3_first) / 4 || i == offsetof(Ctrl, bad4_first) / 4 ||
            i == offsetof(Ctrl, bad5_first) / 4 || i == offsetof(Ctrl, bad6_first) / 4 ||
            i == offsetof(Ctrl, bad4_key) / 4 || i == offsetof(Ctrl, bad4_key) / 4 + 1)
            v = 0xFFFFFFFFu;
        reinterpret_cast<uint32_t*>(ws.ctrl)[i] = v;
    }
}

__device__ __forceinline__ void fill_result(wm_result* result, const Ctrl* ctrl, uint64_t wire_len, int status,
                                            uint32_t first, uint32_t count)
{
    wm_result r;
    memset(&r, 0, sizeof r);
    r.status = status;
    r.first_bad_chunk = first;
    r.n_bad_chunks = count;
    r.n_present = ctrl->hdr_n_present;
    r.payload_bytes = ctrl->payload_total;
    r.wire_len = wire_len;
    r.cache_crc = ctrl->hdr_cache_crc;
    *result = r;
}

// Decode steps 1-3 in one kernel.  The first blocks digest the metadata slices (four teams
// each), the others check the structure chunk by chunk (one warp per chunk: tile entries
// against the chunk's length and enc_len; also each tile's offset inside its chunk's payload).
// Neither part follows anything it reads: every index comes from the call's geometry, so the
// structure pass is safe on damaged metadata and can run beside the CRC.  The last block to
// finish decides in the specified order: metadata CRC first (WM_ERR_META_CRC), then the
// structure (WM_ERR_STRUCT: per-chunk findings, payload offsets as the running sum of enc_len,
// totals against the header).  A header that does not match the call stops every block at
// once (WM_ERR_FORMAT).  A failure sets the gate that keeps the later kernels out.
__global__ void __launch_bounds__(1024)
k_decode_check(const unsigned char* __restrict__ wire, uint64_t wire_len, Geo g, Ws ws,
               const Tables* __restrict__ tab, wm_result* result, uint32_t meta_blocks, uint32_t expect_ent)
{
    __shared__ uint32_t sG[1024];
    __shared__ uint32_t sHT[1024];
    __shared__ uint32_t s_dig[1024];
    __shared__ uint32_t s_wdig[4][8];
    __shared__ unsigned long long s_warp[32];
    __shared__ unsigned long long s_carry;
    __shared__ uint32_t s_first, s_count;
    __shared__ bool s_last;
    __shared__ int s_format_bad;
    const uint32_t lane = threadIdx.x % 32, wblk = threadIdx.x / 32;
    sHT[threadIdx.x] = (&tab->HT[0][0])[threadIdx.x];
    load_small_chain_tables(sG, tab);
    grid_dep_wait();
    grid_dep_launch();
    if (ld_volatile_u32(&ws.ctrl->gate)) return;        // leaf mode: the destination table was rejected
    if (threadIdx.x == 0) s_format_bad = header_matches(wire, wire_len, g, expect_ent) ? 0 : 1;
    __syncthreads();
    if (s_format_bad) {
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            ws.ctrl->gate = (uint32_t)WM_ERR_FORMAT;
            wm_result r;
            memset(&r, 0, sizeof r);
            r.status = WM_ERR_FORMAT;
            *result = r;
        }
        return;
    }
    const unsigned char* dir = wire + 64;
    const bool zero_ok = ((reinterpret_cast<const uint32_t*>(wire)[1] >> 17) & 1u) != 0u;   // the image declares the option
    if (blockIdx.x < meta_blocks) {
        const uint32_t team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads;
        const uint32_t s = blockIdx.x * 4 + team;
        if (s < g.n_meta_slices) meta_slice_parts(wire, g, s, sG, tab, s_wdig[team], tt / 32, lane);
        __syncthreads();
        if (tt == 0 && s < g.n_meta_slices) ws.mdig[s] = xor8(s_wdig[team]);
    } else {
        const uint16_t* tab16 = reinterpret_cast<const uint16_t*>(wire + 64 + 16ull * g.n_chunks);
        const uint32_t c = (blockIdx.x - meta_blocks) * 32u + wblk;
        if (c < g.n_chunks) {
            const uint64_t clen = chunk_len_dev(g, c);
            const uint32_t t0 = c * g.tiles_per_chunk;
            const uint32_t ntc = (uint32_t)((clen + kTile - 1) / kTile);
            const uint32_t elen = *reinterpret_cast<const uint32_t*>(dir + 16ull * c + 8);
            unsigned long long carry = 0;
            bool ok = true, any = false, all = true;
            for (uint32_t i0 = 0; i0 < ntc; i0 += 32) {
                const uint32_t i = i0 + lane;
                uint32_t len = 0;
                bool l_ok = true, l_any = false, l_all = true, l_packs = false;
                if (i < ntc) {
                    const uint32_t e = tab16[t0 + i];
                    const uint64_t tl = clen - (uint64_t)i * kTile;
                    if (e == 0) l_all = false;
                    else {
                        l_any = true;
                        if (tl < kTile) { if (e != 0xFFFFu) l_ok = false; len = (uint32_t)tl; }
                        else if (e == 1u && zero_ok) len = 0;       // a tile of zeros: no payload
                        else if (e == 2u && zero_ok) len = 32;      // a tile of one value: the value
                        else if (e >= 258u && e <= 512u) { len = 32u * e; l_packs = e < 512u; }
                        else if (expect_ent && e >= (0x8000u | 259u) && e <= (0x8000u | 511u)) len = 32u * (e & 0x7FFFu);   // ENT tile
                        else l_ok = false;
                    }
                }
                uint32_t incl = len;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                    if (lane >= (uint32_t)d) incl += o;
                }
                if (i < ntc) ws.rel[t0 + i] = (uint32_t)(carry + incl - len);
                carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
                if (expect_ent && __any_sync(0xFFFFFFFFu, l_packs) && lane == 0) atomicOr(&ws.ctrl->has_pack, 1u);
                ok = ok && __all_sync(0xFFFFFFFFu, l_ok);
                any = any || __any_sync(0xFFFFFFFFu, l_any);
                all = all && __all_sync(0xFFFFFFFFu, l_all);
            }
            if (any && !all) ok = false;
            if (carry != elen) ok = false;
            if (lane == 0) {
                ws.cflag[c] = (any ? CF_PRESENT : 0u) | (ok ? 0u : CF_BAD3);
                if (!ok) { atomicMin(&ws.ctrl->bad3_first, c); atomicAdd(&ws.ctrl->bad3_count, 1u); }
                if (any) atomicAdd(&ws.ctrl->n_present, 1u);
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        s_carry = 0; s_first = 0xFFFFFFFFu; s_count = 0;
        __threadfence();
        s_last = atomicAdd(&ws.ctrl->done_b, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // ---- the last block: metadata CRC first
    const uint32_t crc = fold_meta_digests(g, ws, sHT, s_dig);
    if (threadIdx.x == 0) {
        const uint32_t* h = reinterpret_cast<const uint32_t*>(wire);
        ws.ctrl->hdr_n_present = h[7];
        ws.ctrl->hdr_cache_crc = h[12];
        ws.ctrl->payload_total = h[8] | ((unsigned long long)h[9] << 32);
        s_format_bad = 0;
        if (crc != h[13]) {
            s_format_bad = 1;
            ws.ctrl->gate = (uint32_t)WM_ERR_META_CRC;
            wm_result r;
            memset(&r, 0, sizeof r);
            r.status = WM_ERR_META_CRC;
            r.n_present = h[7];
            r.payload_bytes = ws.ctrl->payload_total;
            r.wire_len = wire_len;
            r.cache_crc = h[12];
            *result = r;
        }
    }
    __syncthreads();
    if (s_format_bad) return;

    // ---- then the structure across chunks
    for (uint32_t base = 0; base < g.n_chunks; base += 1024) {
        const uint32_t cc = base + threadIdx.x;
        unsigned long long len = 0, po = 0;
        if (cc < g.n_chunks) {
            po = *reinterpret_cast<const unsigned long long*>(dir + 16ull * cc);
            len = *reinterpret_cast<const uint32_t*>(dir + 16ull * cc + 8);
        }
        unsigned long long incl = len;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= (uint32_t)d) incl += o;
        }
        if (lane == 31) s_warp[wblk] = incl;
        __syncthreads();
        unsigned long long before = s_carry;
        for (uint32_t w2 = 0; w2 < wblk; w2++) before += s_warp[w2];
        if (cc < g.n_chunks && po != before + incl - len) {
            // a chunk already counted by the per-chunk pass must not be counted twice
            const uint32_t fl = ld_volatile_u32(&ws.cflag[cc]);
            if (!(fl & CF_BAD3)) {
                ws.cflag[cc] = fl | CF_BAD3;
                atomicMin(&s_first, cc);
                atomicAdd(&s_count, 1u);
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long tot = 0;
            for (int w2 = 0; w2 < 32; w2++) tot += s_warp[w2];
            s_carry += tot;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        uint32_t first = min(s_first, ld_volatile_u32(&ws.ctrl->bad3_first));
        uint32_t count = s_count + ld_volatile_u32(&ws.ctrl->bad3_count);
        if (count == 0 && (s_carry != ws.ctrl->payload_total ||
                           ld_volatile_u32(&ws.ctrl->n_present) != ws.ctrl->hdr_n_present)) {
            first = 0; count = 1;
        }
        if (count) {
            ws.ctrl->gate = (uint32_t)WM_ERR_STRUCT;
            fill_result(result, ws.ctrl, wire_len, WM_ERR_STRUCT, first, count);
        }
    }
}

struct DecSlot {                 // what the team's first thread prepares for a tile ahead of its turn
    uint32_t t;                  // tile (>= n_tiles: none left)
    uint32_t entry;              // tile table entry | (first tile of its chunk) << 16
    unsigned long long src;      // offset of the encoded tile inside the payload
};
struct DecTeamCtl {
    uint32_t wdig[2][8];
    DecSlot slot[4];             // ring: slot i & 3 belongs to the team's i-th tile
    unsigned long long mbar;     // completion of the bulk copy into the team's stage
    unsigned long long pad;
};
static_assert(sizeof(DecTeamCtl) % 16 == 0, "team control block keeps 16-byte alignment");

// The plane words of one group as stored (aligned per-lane units, see pack_group_planes):
// a = the 4-bit plane's word or the low half of an 8-bit plane; b = the 2-bit plane's 16 bits
// in the low half and the 1-bit plane's byte in bits 16-23, or the high half of an 8-bit plane.
struct PlaneWords { uint32_t a, b; };

// rec: shared-window address of the group's planes; l4 / l2 / l1: 4, 2, 1 times the lane number
__device__ __forceinline__ PlaneWords read_group_planes(uint32_t rec, uint32_t wd, uint32_t l4, uint32_t l2, uint32_t l1)
{
    PlaneWords pw;
    pw.a = 0; pw.b = 0;
    if (wd == 8u) {
        const uint2 v = lds_now_v2<0>(rec + 2u * l4);
        pw.a = v.x; pw.b = v.y;
        return pw;
    }
    if (wd & 4u) { pw.a = lds_now<0>(rec + l4); rec += 128u; }
    if (wd & 2u) { pw.b = lds_now_u16(rec + l2); rec += 64u; }
    if (wd & 1u) { pw.b |= lds_now_u8(rec + l1) << 16; }
    return pw;
}

// Inverse of pack_group_planes: the lane's eight exponent bytes (two words, coded order).
template <int W>
__device__ __forceinline__ void unpack_group_planes(const PlaneWords& pw, uint32_t base, uint32_t& ea, uint32_t& eb)
{
    uint32_t da = 0, db = 0;
    if (W == 8) { da = pw.a; db = pw.b; }
    else {
        int sh = 0;
        if (W & 4) {
            const uint32_t t = __byte_perm(pw.a, 0, 0x1100), u = __byte_perm(pw.a, 0, 0x3322);
            da = (t & 0x000F000Fu) | ((t >> 4) & 0x0F000F00u);
            db = (u & 0x000F000Fu) | ((u >> 4) & 0x0F000F00u);
            sh = 4;
        }
        if (W & 2) {        // byte -> four 2-bit fields, one per byte
            uint32_t xa = pw.b & 0xFFu, xb = (pw.b >> 8) & 0xFFu;
            xa = (xa * 0x1001u) & 0x000F000Fu; xa = (xa * 0x41u) & 0x03030303u;
            xb = (xb * 0x1001u) & 0x000F000Fu; xb = (xb * 0x41u) & 0x03030303u;
            da |= xa << sh; db |= xb << sh;
            sh += 2;
        }
        if (W & 1) {        // nibble -> four bits, one per byte
            const uint32_t xa = (((pw.b >> 16) & 0xFu) * 0x00204081u) & 0x01010101u;
            const uint32_t xb = (((pw.b >> 20) & 0xFu) * 0x00204081u) & 0x01010101u;
            da |= xa << sh; db |= xb << sh;
        }
    }
    const uint32_t b4 = base * 0x01010101u;
    if (base + ((1u << W) - 1u) <= 255u) {        // no byte can wrap: plain add
        ea = da + b4; eb = db + b4;
    } else {                                      // per byte (base + d) & 0xFF
        ea = ((da & 0x7F7F7F7Fu) + (b4 & 0x7F7F7F7Fu)) ^ ((da ^ b4) & 0x80808080u);
        eb = ((db & 0x7F7F7F7Fu) + (b4 & 0x7F7F7F7Fu)) ^ ((db ^ b4) & 0x80808080u);
    }
}

// Unpack + checksum of the decoded bytes.  Tiles are claimed by ticket.  The team owns one
// 16 KiB stage in shared memory; the encoded tile arrives there by one bulk copy (TMA) that is
// started a tile ahead, each lane takes what it needs (descriptors, its 8 sign-mantissa bytes
// and its plane words per group: at most 16 words) into registers, and the stage is handed to
// the next copy while the team unpacks, stores and checksums.  One team barrier per tile.
// Tiles are prepared ahead of their turn, one dependent step per tile so that nobody sits
// waiting for an answer from L2: claim a ticket (three tiles ahead, warp 3), look up that
// tile's table entry and offsets (two ahead, warp 0), start its copy (one ahead, warp 2); warp 1
// folds and stores the previous tile's digest.  (Spread over warps because the team runs at
// the pace of its slowest one.)  LEAVES: the decoded tiles go to a table of tensors.
// MODE 0: unpack, store, checksum (the normal call).  Strict calls run the kernel twice: MODE 1
// unpacks and checksums without storing anything; MODE 2, after the verdict, unpacks and stores.
// ENT 1 / 2: the image was written with the entropy option and holds ENT tiles only (1) or ENT
// and PACK tiles (2; the check kernel noted which).  A call launches both, and the one that does
// not apply returns at once: the kernel with a single kind of coded tile is the faster one.  A
// warp reads its share's stream of halfwords in phase 1 (the need test, the ballot and the fetch
// of every step) and leaves the exponent bytes where the plane words would be.
template <int TEAMS, bool LEAVES, int MODE, int ENT = 0>
__global__ void __launch_bounds__(TEAMS * 256, 1)
k_decode(const unsigned char* __restrict__ wire, Geo g, unsigned char* __restrict__ dst, Ws ws,
         const Tables* __restrict__ tab)
{
    extern __shared__ __align__(16) unsigned char smem[];
    // ENT: what the low byte of a strand's bits says about the codeword there: its length (16: the
    // escape) and u as a byte.  Two byte tables: the index needs no scaling and a look-up gives a
    // clean value.
    __shared__ unsigned char s_plen[ENT ? 256 : 4], s_pu[ENT ? 256 : 4];
    if (ENT != 0 && threadIdx.x < 256u) {
        const uint32_t s = ent_ones(threadIdx.x);
        s_plen[threadIdx.x] = (unsigned char)ent_parse_length(s);
        s_pu[threadIdx.x] = (unsigned char)(s == 8u ? 0u : ent_parse_value(threadIdx.x, s, 0u));
    }
    Smem S = setup_smem(smem, tab);
    grid_dep_wait();
    grid_dep_launch();
    if (ld_volatile_u32(&ws.ctrl->gate)) return;
    if (ENT != 0 && (ENT == 1) == (ld_volatile_u32(&ws.ctrl->has_pack) != 0u)) return;      // the other kernel's image
    const uint32_t team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads;
    const uint32_t warp = tt / 32, lane = tt % 32;
    unsigned char* stage = nullptr;
    for (int i = 0; i < TEAMS; i++) {          // every thread carves the same blocks in the same order
        unsigned char* p = S.take(kTile);
        if ((uint32_t)i == team) stage = p;
    }
    DecTeamCtl* tc = reinterpret_cast<DecTeamCtl*>(S.take(TEAMS * sizeof(DecTeamCtl)));
    if (!S.ok) { if (threadIdx.x == 0) atomicOr(&ws.ctrl->err, 4u); return; }
    tc += team;
    const unsigned char* const dir = wire + 64;
    const uint16_t* const tab16 = reinterpret_cast<const uint16_t*>(wire + 64 + 16ull * g.n_chunks);
    const unsigned char* const payload = wire + g.meta_end;
    const bool leader = (tt == 0);
    constexpr uint32_t kNone = 0xFFFFFFFFu;
    const uint32_t stage_s = (uint32_t)__cvta_generic_to_shared(stage);
    const uint32_t sm_s = stage_s + 64u + 1024u * warp + 8u * lane;     // this lane's sign-mantissa bytes, group 4 warp

    // a tile's entry word and payload offset (blocking: prologue only)
    auto lookup = [&](uint32_t t, DecSlot* sl) {
        sl->t = t;
        sl->entry = 0; sl->src = 0;
        if (t < g.n_tiles) {
            const uint32_t e = tab16[t];
            sl->entry = e | (first_in_chunk(g, t) ? 0x10000u : 0u);
            if (e) sl->src = *reinterpret_cast<const unsigned long long*>(dir + 16ull * chunk_of(g, t)) + ws.rel[t];
        }
    };
    // staged tiles: full RAW and PACK tiles (everything except absent tiles and the ragged tail)
    // (images with the entropy option hold ENT tiles too: entry 0x8000 | length / 32)
    auto is_ent_entry = [](uint32_t e) { return ENT != 0 && e > 0x8000u && e != 0xFFFFu; };
    auto is_pack_entry = [](uint32_t e) { return ENT != 1 && e >= 258u && e < 512u; };
    auto is_staged = [&](uint32_t e) { return e == 512u || is_pack_entry(e) || is_ent_entry(e); };
    auto start_copy = [&](const DecSlot& sl) {   // leader only
        const uint32_t e = sl.entry & 0xFFFFu;
        if (sl.t < g.n_tiles && is_staged(e)) bulk_load(stage, payload + sl.src, 32u * (e & 0x7FFFu), &tc->mbar, 0);
    };

    if (leader) {
        mbar_init(&tc->mbar, 1);
        lookup(atomicAdd(&ws.ctrl->ticket, 1u), &tc->slot[0]);
        lookup(atomicAdd(&ws.ctrl->ticket, 1u), &tc->slot[1]);
        tc->slot[2].t = atomicAdd(&ws.ctrl->ticket, 1u);      // its look-ups happen in the first step
        start_copy(tc->slot[0]);
    }
    team_bar(team);
    uint32_t phase = 0;
    uint32_t trouble = 0;              // sticky: a copy never arrived
    uint32_t t_done = kNone;           // tile whose digest parts wait in wdig[(it - 1) & 1]
    for (uint32_t it = 0;; it++) {
        const uint32_t t = tc->slot[it & 3u].t;
        if (t >= g.n_tiles) {
            team_bar(team);
            if (tt == 32u && t_done != kNone) ws.dig[t_done] = xor8(tc->wdig[(it & 1u) ^ 1u]);
            break;
        }
        const uint32_t ew = tc->slot[it & 3u].entry;
        const uint32_t e = ew & 0xFFFFu;
        // leaf mode: where this tile goes (asked for now, needed when the stores begin)
        unsigned char* const o_leaf = LEAVES ? ws.tptr[t] : nullptr;
        const uint32_t p = it & 1u;
        const bool is_ent = is_ent_entry(e);
        const bool is_pack = is_ent || is_pack_entry(e);            // a coded tile (in either form)
        bool decoded = true;
        uint32_t w[kWordsPerLane];
        uint32_t desc = 0;
        uint2 sm[4];
        PlaneWords pw[4];

        // ---- phase 1: everything this lane needs from the stage goes into registers
        if (is_staged(e)) {
            if (!mbar_wait(&tc->mbar, phase)) trouble = 1u;
            phase ^= 1u;
            if (!is_pack) {
                read_staged_words(stage, warp, lane, w);
            } else if (is_ent) {
                // ENT tile.  Header: the eight stream lengths against the entry (structure); then this
                // warp reads its share's stream the way the format interleaves it: at step i every
                // strand whose codeword i is not complete in the bits it holds takes the stream's next
                // halfword, strands in ascending order.  The stream must be used up exactly and the
                // bits left in every strand must be zero (descriptor error otherwise).
                const uint32_t cnt = lane < 8u ? lds_now_u16(stage_s + 8u + 2u * lane) : 0u;
                const bool cnt_bad = lane < 8u && (cnt < 128u || cnt > 1024u);
                const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, cnt);
                const uint32_t before = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? cnt : 0u);
                const uint32_t mine = __shfl_sync(0xFFFFFFFFu, cnt, warp);
                int verdict = (__any_sync(0xFFFFFFFFu, cnt_bad) || ent_tile_bytes(total) != 32u * (e & 0x7FFFu)) ? 2 : 0;
                if (!verdict) {
                    const uint32_t anchor = lds_now_u8(stage_s + warp);
                    const uint32_t st = stage_s + 8256u + 2u * before;
                    const uint32_t lt_mask = (1u << lane) - 1u;
                    uint32_t buf = 0, avail = 0, pos = 0, ew[8];
                    const uint32_t last = mine - 1u;           // (mine >= 128)
#pragma unroll
                    for (int j = 0; j < 8; j++) ew[j] = 0u;
#pragma unroll
                    for (int i = 0; i < 32; i++) {
                        const bool more = s_plen[buf & 0xFFu] > avail;
                        const uint32_t takers = __ballot_sync(0xFFFFFFFFu, more);
                        if (more) {
                            // (an index past the stream's end is only clamped here: the stream then
                            // fails the count check below, because every index is below the final pos)
                            const uint32_t idx = min(pos + __popc(takers & lt_mask), last);
                            buf |= lds_now_u16(st + 2u * idx) << avail;
                            avail += 16u;
                        }
                        pos += __popc(takers);
                        const uint32_t low = buf & 0xFFu;
                        const uint32_t len = s_plen[low];
                        const uint32_t E = len == 16u ? buf >> 8 : anchor + s_pu[low];      // (its low byte)
                        ew[i >> 2] = __byte_perm(ew[i >> 2], E, (i & 3) == 0 ? 0x3214 : (i & 3) == 1 ? 0x3240 : (i & 3) == 2 ? 0x3410 : 0x4210);
                        buf >>= len;
                        avail -= len;
                    }
                    if (__any_sync(0xFFFFFFFFu, buf != 0u) || pos != mine) verdict = 1;
#pragma unroll
                    for (int j = 0; j < 4; j++) {
                        sm[j] = j == 0 ? lds_now_v2<0>(sm_s) : j == 1 ? lds_now_v2<256>(sm_s) : j == 2 ? lds_now_v2<512>(sm_s) : lds_now_v2<768>(sm_s);
                        pw[j].a = ew[2 * j];
                        pw[j].b = ew[2 * j + 1];
                    }
                }
                if (verdict) {               // (a stream that does not fit is this warp's finding alone)
                    decoded = false;
                    if (lane == 0) {
                        atomicMin(&ws.ctrl->bad4_key, (unsigned long long)t * 2ull + (verdict == 2 ? 1ull : 0ull));
                        atomicOr(&ws.cflag[chunk_of(g, t)], CF_BAD4);
                    }
                }
            } else if (ENT != 1) {
#ifdef WM_AB_D_NOP1
                desc = 100u | (4u << 8);
                for (int j = 0; j < 4; j++) { sm[j] = make_uint2(lane, it); pw[j].a = t; pw[j].b = e; }
#else
                desc = lds_now_u16(stage_s + 2u * lane);
                const uint32_t wv = (desc >> 8) & 15u;
                const uint32_t base_l = desc & 0xFFu, chk = desc >> 12;
                const bool bad = wv > 8u || chk != (((base_l & 15u) ^ (base_l >> 4) ^ wv ^ 5u) & 15u);
                const bool anybad = __any_sync(0xFFFFFFFFu, bad);
                // sum of all 32 widths, and of the widths of the groups before this warp's four
                const uint32_t Ssum = __reduce_add_sync(0xFFFFFFFFu, wv);
                const uint32_t before = __reduce_add_sync(0xFFFFFFFFu, lane < 4u * warp ? wv : 0u);
                const int verdict = anybad ? 1 : (258u + Ssum != e ? 2 : 0);
                if (verdict) {               // every warp reaches the same verdict
                    decoded = false;
                    if (leader) {
                        atomicMin(&ws.ctrl->bad4_key, (unsigned long long)t * 2ull + (verdict == 2 ? 1ull : 0ull));
                        atomicOr(&ws.cflag[chunk_of(g, t)], CF_BAD4);
                    }
                } else {
                    // lanes 0..3 end up with the descriptors of the warp's four groups, each with its
                    // group's offset in the plane area in the high half
                    const uint32_t own = __shfl_sync(0xFFFFFFFFu, desc, 4 * warp + (lane & 3u)) & 0xFFFFu;
                    const uint32_t wo = (own >> 8) & 15u;
                    uint32_t off = before;                          // running offset over the four groups
                    const uint32_t w0 = __shfl_sync(0xFFFFFFFFu, wo, 0), w1 = __shfl_sync(0xFFFFFFFFu, wo, 1),
                                   w2 = __shfl_sync(0xFFFFFFFFu, wo, 2);
                    if ((lane & 3u) >= 1u) off += w0;
                    if ((lane & 3u) >= 2u) off += w1;
                    if ((lane & 3u) == 3u) off += w2;
                    desc = own | (off << 16);
#pragma unroll
                    for (int j = 0; j < 4; j++) {
                        const uint32_t dg = __shfl_sync(0xFFFFFFFFu, desc, j);
                        sm[j] = j == 0 ? lds_now_v2<0>(sm_s) : j == 1 ? lds_now_v2<256>(sm_s) : j == 2 ? lds_now_v2<512>(sm_s) : lds_now_v2<768>(sm_s);
                        pw[j] = read_group_planes(stage_s + 8256u + 32u * (dg >> 16), (dg >> 8) & 15u, 4u * lane, 2u * lane, lane);
                    }
                }
#endif
            }
        } else if (e == 1u || e == 2u) {
            // a tile of zeros (nothing was shipped) or of one value (the first two bytes of its 32):
            // from here on it goes the way of a raw tile
            uint32_t v = 0;
            if (e == 2u) v = __ldg(reinterpret_cast<const unsigned short*>(payload + tc->slot[it & 3u].src)) * 0x10001u;
#pragma unroll
            for (int i = 0; i < 16; i++) w[i] = v;
        }
        team_bar(team);                      // stage free; the slots the leader filled last step visible;
                                             // the previous tile's digest parts complete
        // The leader: next tile's copy; the previous tile's digest; look-ups for the tile two
        // ahead and the ticket of the tile three ahead (answers taken at the end of the step).
        uint32_t l_e = 0, l_rel = 0, l_tk = kNone;
        unsigned long long l_po = 0;
        // (spread over three warps: the team waits for whichever warp has the most to do)
        if (tt == 64u) start_copy(tc->slot[(it + 1u) & 3u]);
        if (tt == 32u && t_done != kNone) ws.dig[t_done] = xor8(tc->wdig[p ^ 1u]);
        uint32_t t_look = kNone;           // warps 0 and 3: the tile claimed a step ago (two tiles ahead)
        if (leader) {                      // its table entry and offsets
            t_look = tc->slot[(it + 2u) & 3u].t;
            if (t_look < g.n_tiles) {
                l_e = tab16[t_look];
                l_rel = __ldcg(ws.rel + t_look);
                l_po = *reinterpret_cast<const unsigned long long*>(dir + 16ull * chunk_of(g, t_look));
            }
        }
        if (tt == 96u) {                   // the ticket of the tile three ahead
            t_look = tc->slot[(it + 2u) & 3u].t;
            if (t_look < g.n_tiles) l_tk = atomicAdd(&ws.ctrl->ticket, 1u);
        }

        // ---- phase 2: unpack, store, checksum
        bool have_digest = false;
        if (e != 0) {
            unsigned char* o = LEAVES ? o_leaf : dst + (uint64_t)t * kTile;
            bool fold = (ew >> 16) != 0;
            if (e == 0xFFFFu) {
                const unsigned char* src = payload + tc->slot[it & 3u].src;
                const uint32_t len = g.tail_len;
                if (MODE != 1) for (uint32_t i = tt; i < len; i += kTeamThreads) o[i] = src[i];
                if (MODE != 2) load_tile_words_guarded(src, len, fold, warp, lane, w);
                fold = false;
            } else if (is_pack && decoded) {
#ifdef WM_AB_D_NOUNPACK
#pragma unroll
                for (int j = 0; j < 4; j++) { w[4 * j] = sm[j].x; w[4 * j + 1] = sm[j].y; w[4 * j + 2] = pw[j].a; w[4 * j + 3] = pw[j].b; }
#else
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint32_t dg = __shfl_sync(0xFFFFFFFFu, desc, j);
                    const uint32_t base = dg & 0xFFu, wd = (dg >> 8) & 15u;
                    uint32_t ea = base * 0x01010101u, eb = ea;
                    if (ENT == 1 || (ENT == 2 && is_ent)) { ea = pw[j].a; eb = pw[j].b; }     // the exponent bytes are already there
                    else if (wd == 4u) unpack_group_planes<4>(pw[j], base, ea, eb);       // by far the most frequent width
                    else switch (wd) {     // uniform across the warp
                        case 1: unpack_group_planes<1>(pw[j], base, ea, eb); break;
                        case 2: unpack_group_planes<2>(pw[j], base, ea, eb); break;
                        case 3: unpack_group_planes<3>(pw[j], base, ea, eb); break;
                        case 5: unpack_group_planes<5>(pw[j], base, ea, eb); break;
                        case 6: unpack_group_planes<6>(pw[j], base, ea, eb); break;
                        case 7: unpack_group_planes<7>(pw[j], base, ea, eb); break;
                        case 8: unpack_group_planes<8>(pw[j], base, ea, eb); break;
                        default: break;
                    }
                    // A word rotated left by one bit reads [E | m << 1 | sign of the other half] in
                    // each half: swap bit 0 inside the byte pairs of the sign-mantissa words, put
                    // the exponent bytes beside them, rotate back.
                    const uint32_t xa = __byte_perm(sm[j].x, sm[j].x, 0x2301), xb = __byte_perm(sm[j].y, sm[j].y, 0x2301);
                    const uint32_t sa = (sm[j].x & 0xFEFEFEFEu) | (xa & 0x01010101u), sb = (sm[j].y & 0xFEFEFEFEu) | (xb & 0x01010101u);
                    const uint32_t r0 = __byte_perm(sa, ea, 0x5140), r1 = __byte_perm(sa, ea, 0x7362);
                    const uint32_t r2 = __byte_perm(sb, eb, 0x5140), r3 = __byte_perm(sb, eb, 0x7362);
                    w[4 * j] = __funnelshift_r(r0, r0, 1);
                    w[4 * j + 1] = __funnelshift_r(r1, r1, 1);
                    w[4 * j + 2] = __funnelshift_r(r2, r2, 1);
                    w[4 * j + 3] = __funnelshift_r(r3, r3, 1);
                }
#endif
            }
            if (decoded) {
#ifndef WM_AB_D_NOSTORE
                if (MODE != 1 && e != 0xFFFFu) {
                    unsigned char* q = o + warp * 2048u + lane * 4u;
#pragma unroll
                    for (int i = 0; i < 16; i++) st_stream_u32(q + i * 128, w[i]);
                }
#else
                if (w[7] == 0x12345678u && e != 0xFFFFu) st_stream_u32(o + lane * 4u, w[2] ^ w[9] ^ w[12] ^ w[15] ^ w[0] ^ w[5]);
#endif
                if (MODE != 2) {
#ifdef WM_AB_D_NOCRC
                    const uint32_t v = w[3] ^ w[6] ^ w[8] ^ w[13] ^ w[1] ^ w[4] ^ w[10] ^ w[11] ^ w[14];
#else
                    const uint32_t v = tile_digest_part(S, w, fold, warp, lane);
#endif
                    if (lane == 0) tc->wdig[p][warp] = v;
                    have_digest = true;
                }
            }
        }
        t_done = have_digest ? t : kNone;
        if (leader && t_look < g.n_tiles) {
            DecSlot* s2 = &tc->slot[(it + 2u) & 3u];
            s2->entry = l_e | (first_in_chunk(g, t_look) ? 0x10000u : 0u);
            s2->src = l_po + l_rel;
        }
        if (tt == 96u) tc->slot[(it + 3u) & 3u].t = l_tk;      // (none once the tickets have run out)
    }
    if (trouble && lane == 0) atomicOr(&ws.ctrl->err, 2u);
}

// Steps 5..8: chunk CRCs of the decoded bytes against the directory, stale check, cache CRC;
// the last block to finish decides the status and, on success only, updates dst_crc_inout.
__global__ void __launch_bounds__(1024)
k_decode_finish(const unsigned char* __restrict__ wire, uint64_t wire_len, Geo g,
                const unsigned char* __restrict__ dst, uint32_t* __restrict__ dst_crc, Ws ws,
                const Tables* __restrict__ tab, wm_result* result, const __grid_constant__ ChunkPowers cp, uint32_t strict)
{
    __shared__ uint32_t sHT[1024];
    __shared__ uint32_t sT0[256];
    __shared__ FinishStage stage;
    __shared__ uint32_t s_acc;
    __shared__ bool s_last;
    __shared__ int s_status;
    load_ht_t0(sHT, sT0, tab);
    grid_dep_wait();
    if (ld_volatile_u32(&ws.ctrl->gate)) return;
    const uint32_t c0 = blockIdx.x * g.finish_cb;
    stage_chunk_digests(g, stage, ws.dig, c0);
    const unsigned char* dir = wire + 64;
    const uint32_t c = c0 + threadIdx.x;
    const bool step4_failed = ld_volatile_u32(reinterpret_cast<const uint32_t*>(&ws.ctrl->bad4_key)) != 0xFFFFFFFFu ||
                              ld_volatile_u32(reinterpret_cast<const uint32_t*>(&ws.ctrl->bad4_key) + 1) != 0xFFFFFFFFu;
    uint32_t term = 0;
    if (threadIdx.x < g.finish_cb && c < g.n_chunks) {
        const uint32_t fl = ws.cflag[c];
        const uint32_t want = *reinterpret_cast<const uint32_t*>(dir + 16ull * c + 12);
        if (step4_failed) {
            if (fl & CF_BAD4) { atomicMin(&ws.ctrl->bad4_first, c); atomicAdd(&ws.ctrl->bad4_count, 1u); }
        } else if (fl & CF_PRESENT) {
            // (a chunk shorter than four bytes is checksummed byte by byte: from dst, or, in a strict
            // call, where nothing has been stored yet, from its raw copy in the wire image)
            const unsigned char* tiny = chunk_first_byte(g, ws, dst, c);
            if (strict && chunk_len_dev(g, c) < 4)
                tiny = wire + g.meta_end + *reinterpret_cast<const unsigned long long*>(dir + 16ull * c);
            const uint32_t got = chunk_crc_staged(g, sHT, sT0, stage, ws.dig, tiny, c, threadIdx.x);
            if (got != want) { atomicMin(&ws.ctrl->bad5_first, c); atomicAdd(&ws.ctrl->bad5_count, 1u); }
        } else {
            if (dst_crc[c] != want) { atomicMin(&ws.ctrl->bad6_first, c); atomicAdd(&ws.ctrl->bad6_count, 1u); }
        }
        term = cache_crc_term(g, cp, want, c);
    }
    accumulate_cache_crc(ws.ctrl, term, &s_acc);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&ws.ctrl->done_a, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (threadIdx.x == 0) {
        const uint32_t cache_crc = ld_volatile_u32(&ws.ctrl->cache_acc);
        int status = WM_OK;
        uint32_t first = 0, count = 0;
        const unsigned long long key = *reinterpret_cast<volatile unsigned long long*>(&ws.ctrl->bad4_key);
        const uint32_t err = ld_volatile_u32(&ws.ctrl->err);
        if (err) {                     // the kernels themselves failed: nothing can be said about the image
            status = (err & 4u) ? WM_ERR_CUDA : WM_ERR_TIMEOUT;
        } else if (key != ~0ull) {
            status = (key & 1ull) ? WM_ERR_STRUCT : WM_ERR_DESC;
            first = ld_volatile_u32(&ws.ctrl->bad4_first); count = ld_volatile_u32(&ws.ctrl->bad4_count);
        } else if (ld_volatile_u32(&ws.ctrl->bad5_count)) {
            status = WM_ERR_CHUNK_CRC;
            first = ld_volatile_u32(&ws.ctrl->bad5_first); count = ld_volatile_u32(&ws.ctrl->bad5_count);
        } else if (ld_volatile_u32(&ws.ctrl->bad6_count)) {
            status = WM_ERR_STALE;
            first = ld_volatile_u32(&ws.ctrl->bad6_first); count = ld_volatile_u32(&ws.ctrl->bad6_count);
        } else if (cache_crc != ws.ctrl->hdr_cache_crc) {
            status = WM_ERR_CACHE_CRC;
        }
        fill_result(result, ws.ctrl, wire_len, status, first, count);
        s_status = status;
        if (strict) {                  // the storing pass follows: it starts from ticket 0 and stays out after a failure
            ws.ctrl->ticket = 0;
            if (status != WM_OK) ws.ctrl->gate = (uint32_t)status;
        }
    }
    __syncthreads();
    if (s_status == WM_OK) {
        for (uint32_t i = threadIdx.x; i < g.n_chunks; i += blockDim.x)
            if (ws.cflag[i] & CF_PRESENT) dst_crc[i] = *reinterpret_cast<const uint32_t*>(dir + 16ull * i + 12);
    }
}

// ------------------------------------------------------------------ host side

#ifndef WM_TEAMS
#define WM_TEAMS 4
#endif
constexpr int kTeams = WM_TEAMS;            // encode: teams per block (plus the scanner warp)
#ifndef WM_TEAMS_PLAIN
#define WM_TEAMS_PLAIN 4
#endif
constexpr int kTeamsPlain = WM_TEAMS_PLAIN;  // checksum / decode: teams per block

struct DeviceState {
    Tables* tables = nullptr;
    Tables* tables_zlib = nullptr;   // built on the first wm_checksum_poly call that asks for it
    int sm_count = 0;
    bool ready = false;
    cudaEvent_t ev[4][2] = {};   // optional timing of the four main kernels
};
static bool g_timing = false;
static bool g_zero_tiles = false;   // wm_zero_tiles_enable
static bool g_entropy = false;      // wm_entropy_enable

struct MainKernelTimer {        // records events around a main kernel when timing is enabled
    const DeviceState* ds; int kind; cudaStream_t s;
    MainKernelTimer(const DeviceState* d, int k, cudaStream_t st) : ds(d), kind(k), s(st)
    {
        if (g_timing) cudaEventRecord(ds->ev[kind][0], s);
    }
    ~MainKernelTimer()
    {
        if (g_timing) cudaEventRecord(ds->ev[kind][1], s);
    }
};
static DeviceState g_dev[64];
static std::mutex g_mutex;
static thread_local uint32_t g_launches = 0;

static const DeviceState* device_state()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& s = g_dev[dev];
    if (s.ready) return &s;
    static Tables host;
    build_tables(host);
    if (cudaMalloc(&s.tables, sizeof(Tables)) != cudaSuccess) return nullptr;
    if (cudaMemcpy(s.tables, &host, sizeof(Tables), cudaMemcpyHostToDevice) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    const int big = kDynSmem;
    {
        const void* enc[] = {(const void*)k_encode<kTeams, false, false, false>, (const void*)k_encode<kTeams, true, false, false>,
                             (const void*)k_encode<kTeams, false, true, false>,  (const void*)k_encode<kTeams, true, true, false>,
                             (const void*)k_encode<kTeams, false, false, true>,  (const void*)k_encode<kTeams, true, false, true>,
                             (const void*)k_encode<kTeams, false, true, true>,   (const void*)k_encode<kTeams, true, true, true>,
                             (const void*)k_encode<kTeams, false, false, false, true>, (const void*)k_encode<kTeams, true, false, false, true>,
                             (const void*)k_encode<kTeams, false, true, false, true>,  (const void*)k_encode<kTeams, true, true, false, true>,
                             (const void*)k_encode<kTeams, false, false, true, true>,  (const void*)k_encode<kTeams, true, false, true, true>,
                             (const void*)k_encode<kTeams, false, true, true, true>,   (const void*)k_encode<kTeams, true, true, true, true>};
        for (const void* f : enc)
            if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    }
    {
        const void* dec[] = {(const void*)k_decode<kTeamsPlain, false, 0>, (const void*)k_decode<kTeamsPlain, true, 0>,
                             (const void*)k_decode<kTeamsPlain, false, 1>, (const void*)k_decode<kTeamsPlain, true, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 2>, (const void*)k_decode<kTeamsPlain, true, 2>,
                             (const void*)k_decode<kTeamsPlain, false, 0, 1>, (const void*)k_decode<kTeamsPlain, true, 0, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 1, 1>, (const void*)k_decode<kTeamsPlain, true, 1, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 2, 1>, (const void*)k_decode<kTeamsPlain, true, 2, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 0, 2>, (const void*)k_decode<kTeamsPlain, true, 0, 2>,
                             (const void*)k_decode<kTeamsPlain, false, 1, 2>, (const void*)k_decode<kTeamsPlain, true, 1, 2>,
                             (const void*)k_decode<kTeamsPlain, false, 2, 2>, (const void*)k_decode<kTeamsPlain, true, 2, 2>};
        for (const void* f : dec)
            if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    }
    if (cudaFuncSetAttribute(k_tile_digests<kTeamsPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    if (cudaFuncSetAttribute(k_meta_crc, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    for (int k = 0; k < 4; k++)
        for (int j = 0; j < 2; j++)
            if (cudaEventCreate(&s.ev[k][j]) != cudaSuccess) return nullptr;
    s.ready = true;
    return &s;
}

// Launch a kernel that may start before the kernel enqueued just before it on the stream has
// finished (it waits inside, see grid_dep_wait).
template <typename... Params, typename... Args>
static void launch_after(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static wm_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? WM_OK : WM_ERR_CUDA;
}

}  // namespace wm

using namespace wm;

extern "C" {

uint64_t wm_num_chunks(uint64_t nbytes, uint32_t chunk_bytes)
{
    return chunk_bytes ? (nbytes + chunk_bytes - 1) / chunk_bytes : 0;
}

uint64_t wm_num_tiles(uint64_t nbytes) { return (nbytes + kTile - 1) / kTile; }

uint64_t wm_meta_bytes(uint64_t nbytes, uint32_t chunk_bytes)
{
    return (64ull + 16ull * wm_num_chunks(nbytes, chunk_bytes) + 2ull * wm_num_tiles(nbytes) + 31ull) & ~31ull;
}

uint64_t wm_wire_bound(uint64_t nbytes, uint32_t chunk_bytes) { return wm_meta_bytes(nbytes, chunk_bytes) + nbytes; }

uint64_t wm_workspace_bytes(uint64_t nbytes, uint32_t chunk_bytes)
{
    Geo g;
    if (!make_geo(nbytes, chunk_bytes, g)) return 0;
    return ws_layout(g).total;
}

uint32_t wm_last_launch_count(void) { return g_launches; }

void wm_timing_enable(int on) { g_timing = on != 0; }

void wm_zero_tiles_enable(int on) { g_zero_tiles = on != 0; }
void wm_entropy_enable(int on) { g_entropy = on != 0; }

int wm_timing_read_ms(int kind, float* ms)
{
    const DeviceState* ds = device_state();
    if (!ds || kind < 0 || kind > 3 || !ms) return WM_ERR_ARG;
    if (cudaEventSynchronize(ds->ev[kind][1]) != cudaSuccess) return WM_ERR_CUDA;
    return cudaEventElapsedTime(ms, ds->ev[kind][0], ds->ev[kind][1]) == cudaSuccess ? WM_OK : WM_ERR_CUDA;
}

wm_status wm_checksum(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, uint32_t* crc_out,
                      void* workspace, uint64_t workspace_bytes, void* stream)
{
    Geo g;
    if (!cache || !crc_out || !workspace || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (!aligned16(cache) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    const uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    {
        MainKernelTimer timer(ds, 0, s);
        k_tile_digests<kTeamsPlain><<<grid, kTeamsPlain * 256, kDynSmem, s>>>(c, g, ws, ds->tables);
    }
    launch_after(k_checksum_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, ws, ds->tables, crc_out);
    g_launches = 2;
    return launch_status();
}

// The checksum call with the polynomial as an argument.  The tile kernel and the finish kernel
// are the ones wm_checksum runs: the polynomial lives in the tables and in the geometry's powers.
static const Tables* zlib_tables()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& s = g_dev[dev];
    if (s.tables_zlib) return s.tables_zlib;
    static Tables host;
    build_tables(host, kPolyZlib);
    Tables* p = nullptr;
    if (cudaMalloc(&p, sizeof(Tables)) != cudaSuccess) return nullptr;
    if (cudaMemcpy(p, &host, sizeof(Tables), cudaMemcpyHostToDevice) != cudaSuccess) { cudaFree(p); return nullptr; }
    s.tables_zlib = p;
    return p;
}

wm_status wm_checksum_poly(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, int polynomial, uint32_t* crc_out,
                           void* workspace, uint64_t workspace_bytes, void* stream)
{
    if (polynomial == WM_POLY_CRC32C) return wm_checksum(cache, nbytes, chunk_bytes, crc_out, workspace, workspace_bytes, stream);
    if (polynomial != WM_POLY_ZLIB) return WM_ERR_ARG;
    Geo g;
    if (!cache || !crc_out || !workspace || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (!aligned16(cache) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    const Tables* tab = zlib_tables();
    if (!tab) return WM_ERR_CUDA;
    g.poly = kPolyZlib;
    g.k_tail = x_pow_bytes(g.tail_len, kPolyZlib);
    g.k_chunk = x_pow_bytes(g.chunk_bytes, kPolyZlib);
    g.k_last_chunk = x_pow_bytes(g.last_chunk_len, kPolyZlib);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    const uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    {
        MainKernelTimer timer(ds, 0, s);
        k_tile_digests<kTeamsPlain><<<grid, kTeamsPlain * 256, kDynSmem, s>>>(c, g, ws, tab);
    }
    launch_after(k_checksum_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, ws, tab, crc_out);
    g_launches = 2;
    return launch_status();
}

// ---- wm_checksum_noalloc: the checksum call for callers that must not allocate -------------
//
// Scratch and tables live in the library image itself: two file-scope __device__ arrays that
// every GPU loading the library carries until the process exits.  In host code their names
// are host-side stand-ins, not device addresses, so the addresses are asked for once per
// device with cudaGetSymbolAddress (with that device current) and only those go to kernels.
static __device__ __align__(256) unsigned char g_na_scratch[WM_NOALLOC_SCRATCH_BYTES];
static __device__ __align__(256) unsigned char g_na_tables[sizeof(wm::Tables)];

namespace wm {
struct NoAllocState {
    unsigned char* scratch = nullptr;
    Tables* tables = nullptr;
    int sm_count = 0;
    bool ready = false;
};
static NoAllocState g_na[64];

static const NoAllocState* noalloc_state()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    NoAllocState& s = g_na[dev];
    if (s.ready) return &s;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_na_scratch) != cudaSuccess || !p) return nullptr;
    s.scratch = static_cast<unsigned char*>(p);
    p = nullptr;
    if (cudaGetSymbolAddress(&p, g_na_tables) != cudaSuccess || !p) return nullptr;
    s.tables = static_cast<Tables*>(p);
    static Tables host;                          // static storage: no heap, no device allocation
    build_tables(host);
    if (cudaMemcpy(s.tables, &host, sizeof(Tables), cudaMemcpyHostToDevice) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    if (cudaFuncSetAttribute(k_tile_digests<kTeamsPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem)
        != cudaSuccess)
        return nullptr;
    s.ready = true;
    return &s;
}
}  // namespace wm

wm_status wm_checksum_noalloc(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, uint32_t* crc_out, void* stream)
{
    Geo g;
    if (!cache || !crc_out || !make_geo(nbytes, chunk_bytes, g) || !aligned16(cache)) return WM_ERR_ARG;
    if (nbytes > WM_NOALLOC_MAX_BYTES) return WM_ERR_ARG;          // the built-in scratch holds no more
    const NoAllocState* ns = noalloc_state();
    if (!ns) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // scratch: a control block, then one 32-bit digest per tile
    static_assert(WM_NOALLOC_SCRATCH_BYTES >= sizeof(Ctrl) + 4ull * (WM_NOALLOC_MAX_BYTES / WM_TILE_BYTES + 1),
                  "built-in scratch covers the stated maximum");
    Ws ws;
    memset(&ws, 0, sizeof ws);
    ws.ctrl = reinterpret_cast<Ctrl*>(ns->scratch);
    ws.dig = reinterpret_cast<uint32_t*>(ns->scratch + sizeof(Ctrl));
    // the array keeps the last call's contents; only the control block has to start at zero
    if (cudaMemsetAsync(ns->scratch, 0, sizeof(Ctrl), s) != cudaSuccess) return WM_ERR_CUDA;
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    const uint32_t grid = need < (uint32_t)ns->sm_count ? need : (uint32_t)ns->sm_count;
    k_tile_digests<kTeamsPlain><<<grid, kTeamsPlain * 256, kDynSmem, s>>>(c, g, ws, ns->tables);
    launch_after(k_checksum_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, ws, ns->tables, crc_out);
    g_launches = 2;
    return launch_status();
}

wm_status wm_dirty_diff(const void* cache, const void* prev, uint64_t nbytes, uint32_t chunk_bytes,
                        uint8_t* dirty_out, uint32_t* dirty_idx_out, uint32_t* n_dirty_out,
                        void* workspace, uint64_t workspace_bytes, void* stream)
{
    Geo g;
    if (!cache || !prev || !dirty_out || !n_dirty_out || !workspace || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (!aligned16(cache) || !aligned16(prev) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    k_diff_init<<<1, 32, 0, s>>>(ws);
    const uint32_t want = (uint32_t)ds->sm_count * 4;
    const uint32_t grid = g.n_chunks < want ? g.n_chunks : want;
    {
        MainKernelTimer timer(ds, 1, s);
        launch_after(k_diff, grid, 256, 0, s, static_cast<const unsigned char*>(cache), static_cast<const unsigned char*>(prev), g, ws, dirty_out);
    }
    launch_after(k_diff_compact, 1, 1024, 0, s, g, dirty_out, dirty_idx_out, n_dirty_out);
    g_launches = 3;
    return launch_status();
}

// Both forms of the encode call: a flat cache (leaves == nullptr) or a table of leaves.
// The options the plain calls use: the process-wide switches.
static uint32_t default_options()
{
    return (g_zero_tiles ? WM_OPT_ZERO_TILES : 0u) | (g_entropy ? WM_OPT_ENTROPY : 0u);
}

static wm_status encode_any(const void* cache, const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes,
                            const uint8_t* dirty, uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace,
                            uint64_t workspace_bytes, wm_result* result, void* stream, uint32_t options)
{
    Geo g;
    if (options & ~(WM_OPT_ZERO_TILES | WM_OPT_ENTROPY)) return WM_ERR_ARG;
    const bool opt_ent = (options & WM_OPT_ENTROPY) != 0, opt_zero = (options & WM_OPT_ZERO_TILES) != 0;
    if (!crc_inout || !wire || !workspace || !result || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (leaves ? (n_leaves == 0 || n_leaves > kMaxLeaves) : (!cache || !aligned16(cache))) return WM_ERR_ARG;
    if (!aligned16(wire) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total || wire_cap < g.meta_end)
        return WM_ERR_ARG;
    if (nbytes > kMaxCodecBytes) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    unsigned char* w = static_cast<unsigned char*>(wire);
    const uint32_t init_blocks = (g.n_tiles + 1023) / 1024 < 1024 ? (g.n_tiles + 1023) / 1024 : 1024;
    k_encode_init<<<init_blocks ? init_blocks : 1, 1024, 0, s>>>(g, ws, w);
    if (leaves) {
        const uint32_t map_blocks = (g.n_tiles + 4095) / 4096 < 64 ? (g.n_tiles + 4095) / 4096 : 64;
        launch_after(k_leaf_map, map_blocks ? map_blocks : 1, 1024, 0, s, leaves, n_leaves, g, ws, result, 0);
    }
    // one block per SM: one of them scans, the others encode
    const uint32_t need = (g.n_tiles + kTeams - 1) / kTeams + 1;
    const uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    {
        MainKernelTimer timer(ds, 2, s);
        const int variant = (dirty ? 1 : 0) | (leaves ? 2 : 0) | (opt_zero ? 4 : 0) | (opt_ent ? 8 : 0);
        auto go = [&](auto kernel) { launch_after(kernel, grid, kTeams * 256, kDynSmem, s, c, g, dirty, w, wire_cap, ws, ds->tables); };
        switch (variant) {
            case 0: go(k_encode<kTeams, false, false, false>); break;
            case 1: go(k_encode<kTeams, true, false, false>); break;
            case 2: go(k_encode<kTeams, false, true, false>); break;
            case 3: go(k_encode<kTeams, true, true, false>); break;
            case 4: go(k_encode<kTeams, false, false, true>); break;
            case 5: go(k_encode<kTeams, true, false, true>); break;
            case 6: go(k_encode<kTeams, false, true, true>); break;
            case 7: go(k_encode<kTeams, true, true, true>); break;
            case 8: go(k_encode<kTeams, false, false, false, true>); break;
            case 9: go(k_encode<kTeams, true, false, false, true>); break;
            case 10: go(k_encode<kTeams, false, true, false, true>); break;
            case 11: go(k_encode<kTeams, true, true, false, true>); break;
            case 12: go(k_encode<kTeams, false, false, true, true>); break;
            case 13: go(k_encode<kTeams, true, false, true, true>); break;
            case 14: go(k_encode<kTeams, false, true, true, true>); break;
            default: go(k_encode<kTeams, true, true, true, true>); break;
        }
    }
    launch_after(k_encode_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, dirty, crc_inout, w, ws, ds->tables,
                 chunk_powers(g), (opt_ent ? 4u : 0u) | (opt_zero ? 2u : 0u));
    launch_after(k_meta_crc, (g.n_meta_slices + 3) / 4, 1024, kDynSmem, s, w, g, ws, ds->tables, result);
    g_launches = leaves ? 5 : 4;
    return launch_status();
}

wm_status wm_encode(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
                    uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace, uint64_t workspace_bytes,
                    wm_result* result, void* stream)
{
    if (!cache) return WM_ERR_ARG;
    return encode_any(cache, nullptr, 0, nbytes, chunk_bytes, dirty, crc_inout, wire, wire_cap, workspace, workspace_bytes, result, stream,
                      default_options());
}

wm_status wm_encode_leaves(const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
                           uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace, uint64_t workspace_bytes,
                           wm_result* result, void* stream)
{
    if (!leaves) return WM_ERR_ARG;
    return encode_any(nullptr, leaves, n_leaves, nbytes, chunk_bytes, dirty, crc_inout, wire, wire_cap, workspace, workspace_bytes, result, stream,
                      default_options());
}

// Both forms of the decode call: a flat shadow buffer (leaves == nullptr) or a table of leaves.
// strict: nothing is stored until every check has passed (two passes over the wire image).
static wm_status decode_any(const void* wire, uint64_t wire_len, void* dst, const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes,
                            uint32_t chunk_bytes, uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes,
                            wm_result* result, void* stream, uint32_t options)
{
    Geo g;
    if (options & ~(WM_OPT_ZERO_TILES | WM_OPT_ENTROPY | WM_OPT_STRICT)) return WM_ERR_ARG;
    const bool strict = (options & WM_OPT_STRICT) != 0;
    if (!wire || !dst_crc_inout || !workspace || !result || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (leaves ? (n_leaves == 0 || n_leaves > kMaxLeaves) : (!dst || !aligned16(dst))) return WM_ERR_ARG;
    if (!aligned16(wire) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    if (nbytes > kMaxCodecBytes) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* w = static_cast<const unsigned char*>(wire);
    unsigned char* d = static_cast<unsigned char*>(dst);
    k_decode_init<<<1, 64, 0, s>>>(ws);
    if (leaves) {
        const uint32_t map_blocks = (g.n_tiles + 4095) / 4096 < 64 ? (g.n_tiles + 4095) / 4096 : 64;
        launch_after(k_leaf_map, map_blocks ? map_blocks : 1, 1024, 0, s, leaves, n_leaves, g, ws, result, 1);
    }
    // a wire shorter than the metadata is rejected by the header check before anything else is read
    const uint32_t meta_blocks = (g.n_meta_slices + 3) / 4;
    const bool ent = (options & WM_OPT_ENTROPY) != 0;      // the option says which kind of image the call expects
    launch_after(k_decode_check, meta_blocks + (g.n_chunks + 31) / 32, 1024, 0, s, w, wire_len, g, ws, ds->tables, result, meta_blocks,
                 ent ? 1u : 0u);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    const uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    auto pass = [&](auto flat_kernel, auto leaf_kernel) {
        if (leaves) launch_after(leaf_kernel, grid, kTeamsPlain * 256, kDynSmem, s, w, g, d, ws, ds->tables);
        else launch_after(flat_kernel, grid, kTeamsPlain * 256, kDynSmem, s, w, g, d, ws, ds->tables);
    };
    {
        MainKernelTimer timer(ds, 3, s);
        if (ent) {       // one of the two applies (ENT tiles only, or ENT and PACK tiles); the other returns at once
            if (strict) { pass(k_decode<kTeamsPlain, false, 1, 1>, k_decode<kTeamsPlain, true, 1, 1>); pass(k_decode<kTeamsPlain, false, 1, 2>, k_decode<kTeamsPlain, true, 1, 2>); }
            else { pass(k_decode<kTeamsPlain, false, 0, 1>, k_decode<kTeamsPlain, true, 0, 1>); pass(k_decode<kTeamsPlain, false, 0, 2>, k_decode<kTeamsPlain, true, 0, 2>); }
        } else {
            if (strict) pass(k_decode<kTeamsPlain, false, 1>, k_decode<kTeamsPlain, true, 1>);
            else pass(k_decode<kTeamsPlain, false, 0>, k_decode<kTeamsPlain, true, 0>);
        }
    }
    launch_after(k_decode_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, w, wire_len, g, d, dst_crc_inout, ws, ds->tables,
                 result, chunk_powers(g), strict ? 1u : 0u);
    if (strict) {
        if (ent) { pass(k_decode<kTeamsPlain, false, 2, 1>, k_decode<kTeamsPlain, true, 2, 1>); pass(k_decode<kTeamsPlain, false, 2, 2>, k_decode<kTeamsPlain, true, 2, 2>); }
        else pass(k_decode<kTeamsPlain, false, 2>, k_decode<kTeamsPlain, true, 2>);
    }
    g_launches = (leaves ? 5 : 4) + (strict ? 1 : 0) + (ent ? (strict ? 2 : 1) : 0);
    return launch_status();
}

wm_status wm_decode_verify(const void* wire, uint64_t wire_len, void* dst, uint64_t nbytes, uint32_t chunk_bytes,
                           uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes, wm_result* result,
                           void* stream)
{
    if (!dst) return WM_ERR_ARG;
    return decode_any(wire, wire_len, dst, nullptr, 0, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result, stream,
                      default_options());
}

wm_status wm_decode_verify_strict(const void* wire, uint64_t wire_len, void* dst, uint64_t nbytes, uint32_t chunk_bytes,
                                  uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes, wm_result* result,
                                  void* stream)
{
    if (!dst) return WM_ERR_ARG;
    return decode_any(wire, wire_len, dst, nullptr, 0, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result, stream,
                      default_options() | WM_OPT_STRICT);
}

wm_status wm_decode_verify_leaves(const void* wire, uint64_t wire_len, const wm_leaf* dst_leaves, uint32_t n_leaves, uint64_t nbytes,
                                  uint32_t chunk_bytes, uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes,
                                  wm_result* result, void* stream)
{
    if (!dst_leaves) return WM_ERR_ARG;
    return decode_any(wire, wire_len, nullptr, dst_leaves, n_leaves, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result,
                      stream, default_options());
}

// The calls with their options as an argument (nothing process-wide is read): a cache as one
// buffer (leaves == NULL) or as a table of leaves (cache / dst == NULL).
wm_status wm_encode_opt(const void* cache, const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes,
                        const uint8_t* dirty, uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace,
                        uint64_t workspace_bytes, uint32_t options, wm_result* result, void* stream)
{
    if ((cache != nullptr) == (leaves != nullptr)) return WM_ERR_ARG;
    return encode_any(cache, leaves, n_leaves, nbytes, chunk_bytes, dirty, crc_inout, wire, wire_cap, workspace, workspace_bytes, result, stream,
                      options);
}

wm_status wm_decode_verify_opt(const void* wire, uint64_t wire_len, void* dst, const wm_leaf* dst_leaves, uint32_t n_leaves,
                               uint64_t nbytes, uint32_t chunk_bytes, uint32_t* dst_crc_inout, void* workspace,
                               uint64_t workspace_bytes, uint32_t options, wm_result* result, void* stream)
{
    if ((dst != nullptr) == (dst_leaves != nullptr)) return WM_ERR_ARG;
    return decode_any(wire, wire_len, dst, dst_leaves, n_leaves, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result, stream,
                      options);
}

}  // extern "C"
