// Device-side building blocks shared by the kernels: shared-memory table layout, the
// word-strided CRC chain, GF(2) products, team barriers and small load/store helpers.
//
// Work unit: a "team" of 8 warps (256 threads) owns one 16 KiB tile at a time.  The tile is
// seen as 128 rows of 128 bytes; warp w owns rows 16w .. 16w+15 and lane l owns the 32-bit
// word l of each of those rows.  A lane therefore walks 16 words that are exactly 128 bytes
// apart, which makes its CRC contribution a Horner chain with ONE fixed multiplier
// (x^1024, table G); the lane's place inside the row and the warp's place inside the tile
// are folded in once per tile with two small nibble tables (NK, NW).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "wm_tables.h"

namespace wm {

constexpr uint32_t kTile = 16384;
constexpr uint32_t kTeamThreads = 256;
constexpr uint32_t kWordsPerLane = 16;

// Shared-memory image of the tables.  G and NK are stored once per lane ("replicated") so
// that lane l only ever touches bank l: data-dependent lookups are conflict free.
constexpr uint32_t kSmemG = 4 * 256 * 32 * 4;      // 131072
constexpr uint32_t kSmemNK = 8 * 16 * 32 * 4;      // 16384
constexpr uint32_t kSmemNW = 8 * 8 * 16 * 4;       // 4096
constexpr uint32_t kSmemTables = kSmemG + kSmemNK + kSmemNW;

struct SmemTables {
    const uint32_t* G;    // [(k*256 + b)*32 + lane]
    const uint32_t* NK;   // [(n*16 + v)*32 + lane]
    const uint32_t* NW;   // [(w*8 + n)*16 + v]
};

__device__ __forceinline__ SmemTables load_tables(unsigned char* smem, const Tables* __restrict__ tab)
{
    uint32_t* G = reinterpret_cast<uint32_t*>(smem);
    uint32_t* NK = reinterpret_cast<uint32_t*>(smem + kSmemG);
    uint32_t* NW = reinterpret_cast<uint32_t*>(smem + kSmemG + kSmemNK);
    const uint32_t* gG = &tab->G[0][0];
    const uint32_t* gNK = &tab->NK[0][0][0];
    const uint32_t* gNW = &tab->NW[0][0][0];
    for (uint32_t i = threadIdx.x; i < 4 * 256 * 32; i += blockDim.x) G[i] = gG[i >> 5];
    for (uint32_t i = threadIdx.x; i < 8 * 16 * 32; i += blockDim.x) NK[i] = gNK[(i & 31) * 128 + (i >> 5)];
    for (uint32_t i = threadIdx.x; i < 8 * 8 * 16; i += blockDim.x) NW[i] = gNW[i];
    __syncthreads();
    SmemTables t;
    t.G = G; t.NK = NK; t.NW = NW;
    return t;
}

__device__ __forceinline__ void team_bar(uint32_t team)
{
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(kTeamThreads) : "memory");
}

// One chain step: (state ^ word) advanced over 128 bytes.  Gl = G + lane.
__device__ __forceinline__ uint32_t chain_step(const uint32_t* Gl, uint32_t x)
{
    const char* p = reinterpret_cast<const char*>(Gl);
    uint32_t a = *reinterpret_cast<const uint32_t*>(p + ((x << 7) & 0x7F80u));
    uint32_t b = *reinterpret_cast<const uint32_t*>(p + 32768 + ((x >> 1) & 0x7F80u));
    uint32_t c = *reinterpret_cast<const uint32_t*>(p + 65536 + ((x >> 9) & 0x7F80u));
    uint32_t d = *reinterpret_cast<const uint32_t*>(p + 98304 + ((x >> 17) & 0x7F80u));
    return a ^ b ^ c ^ d;
}

// Lane finish: x advanced over 128 - 4*lane bytes.  NKl = NK + lane.
__device__ __forceinline__ uint32_t lane_finish(const uint32_t* NKl, uint32_t x)
{
    const char* p = reinterpret_cast<const char*>(NKl);
    uint32_t r = 0;
#pragma unroll
    for (int n = 0; n < 8; n++)
        r ^= *reinterpret_cast<const uint32_t*>(p + n * 2048 + (((x >> (4 * n)) & 15u) << 7));
    return r;
}

// CRC state (zero start) of a warp's 2048-byte block from the 16 words each lane holds.
__device__ __forceinline__ uint32_t warp_block_digest(const SmemTables& T, const uint32_t (&w)[kWordsPerLane],
                                                      uint32_t lane)
{
    const uint32_t* Gl = T.G + lane;
    uint32_t s = 0;
#pragma unroll
    for (int i = 0; i < 15; i++) s = chain_step(Gl, s ^ w[i]);
    uint32_t r = lane_finish(T.NK + lane, s ^ w[15]);
    return __reduce_xor_sync(0xFFFFFFFFu, r);
}

// Place a warp's block digest inside the tile: advance over 2048*(7 - warp) bytes.  Returns the
// warp's contribution to the tile digest in every lane.
__device__ __forceinline__ uint32_t warp_place(const SmemTables& T, uint32_t digest, uint32_t warp, uint32_t lane)
{
    uint32_t v = 0;
    if (lane < 8) v = T.NW[(warp * 8 + lane) * 16 + ((digest >> (4 * lane)) & 15u)];
    return __reduce_xor_sync(0xFFFFFFFFu, v);
}

// Generic product of two residues (bitwise; used a handful of times per call).
__device__ __forceinline__ uint32_t mulmod_dev(uint32_t a, uint32_t b)
{
    uint32_t r = 0;
#pragma unroll 8
    for (int i = 0; i < 32; i++) {
        r ^= b & (0u - (a >> 31));
        a <<= 1;
        b = (b >> 1) ^ (kPolyReflected & (0u - (b & 1u)));
    }
    return r;
}

// Advance a state over one tile (16384 bytes) with byte tables HT[4][256] (shared or global).
__device__ __forceinline__ uint32_t advance_tile(const uint32_t* HT, uint32_t s)
{
    return HT[s & 0xFF] ^ HT[256 + ((s >> 8) & 0xFF)] ^ HT[512 + ((s >> 16) & 0xFF)] ^ HT[768 + (s >> 24)];
}

__device__ __forceinline__ uint32_t ld_stream_u32(const void* p)
{
    uint32_t v;
    asm volatile("ld.global.cs.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream_u32(void* p, uint32_t v)
{
    asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint64_t ld_volatile_u64(const uint64_t* p)
{
    uint64_t v;
    asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_volatile_u64(uint64_t* p, uint64_t v)
{
    asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint32_t min_u16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("min.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Full tile, fast path: lane's word of row 16*warp + i.
__device__ __forceinline__ void load_tile_words(const unsigned char* tile, uint32_t warp, uint32_t lane,
                                                uint32_t (&w)[kWordsPerLane])
{
    const unsigned char* p = tile + warp * 2048u + lane * 4u;
#pragma unroll
    for (int i = 0; i < 16; i++) w[i] = ld_stream_u32(p + i * 128);
}

// Any tile of `len` (1..16384) real bytes, right-aligned in a virtual tile whose leading
// 16384 - len bytes are zero (leading zeros do not change a zero-start CRC state).  When
// `first_in_chunk`, the chunk's first four bytes are complemented (the all-ones CRC init).
// `skip_lo..skip_lo+3` (real byte offsets, or a negative value) are read as zero.
__device__ __forceinline__ void load_tile_words_guarded(const unsigned char* tile, uint32_t len, bool first_in_chunk,
                                                        int64_t skip_lo, uint32_t warp, uint32_t lane,
                                                        uint32_t (&w)[kWordsPerLane])
{
    const int64_t pad = (int64_t)kTile - (int64_t)len;
#pragma unroll
    for (int i = 0; i < 16; i++) {
        int64_t vb = (int64_t)(warp * 16 + i) * 128 + lane * 4;
        uint32_t word = 0;
#pragma unroll
        for (int j = 0; j < 4; j++) {
            int64_t rb = vb + j - pad;
            if (rb >= 0) {
                uint32_t b = tile[rb];
                if (rb >= skip_lo && rb < skip_lo + 4) b = 0;
                if (first_in_chunk && rb < 4) b ^= 0xFFu;
                word |= b << (8 * j);
            }
        }
        w[i] = word;
    }
}

// CRC32C of a short run computed byte by byte (chunks shorter than four bytes).
__device__ __forceinline__ uint32_t crc_bytewise(const uint32_t* T0, const unsigned char* p, uint32_t n)
{
    uint32_t crc = 0xFFFFFFFFu;
    for (uint32_t i = 0; i < n; i++) crc = T0[(crc ^ p[i]) & 0xFF] ^ (crc >> 8);
    return ~crc;
}

}  // namespace wm
