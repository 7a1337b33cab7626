// Leaf mode: the table of tensors turned into one descriptor per tile (k_leaf_map), and the
// byte-exact readers / writers for the few tiles that do not sit inside one leaf.
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

// ------------------------------------------------------------------ leaf tables

// The logical cache is the concatenation of `n` leaves (tensors) of any positive sizes; the
// 16 KiB tile grid is laid over that concatenation, so a tile may begin anywhere inside a leaf
// and may run across leaf boundaries (a scalar flag between two tensors, say).  k_leaf_map
// writes, per leaf, the logical offset at which it starts (ws.lstart, n + 1 entries) and, per
// tile, a 64-bit descriptor (ws.tptr):
//   bit 63 clear: the address of the tile's first byte.  All 16384 bytes sit in one leaf, and so
//       does the 16-byte aligned block around them, so the tile can be moved by a bulk copy from
//       the address rounded down to 16 (the main kernels shift the words by the remainder).
//   bit 63 set:   a "walked" tile; the low 32 bits are the leaf that holds its first byte.  The
//       tile crosses a leaf boundary, or is the ragged last tile, or ends within 16 bytes of the
//       end of a leaf whose size is not a multiple of 16 (the aligned block would reach past
//       the leaf).  Such tiles are read and written byte by byte through the leaf table; there
//       are at most two per leaf.
// Rules (a table that breaks one raises error bit 8; in decode mode it also closes the gate and
// writes the result record; nothing is read or written through a rejected table): 1..4096
// leaves, every pointer 16-byte aligned, every size positive and at most nbytes (so the sum
// cannot wrap), the sizes add up to nbytes.
constexpr unsigned long long kTileWalked = 1ull << 63;

__global__ void __launch_bounds__(1024)
k_leaf_map(const wm_leaf* __restrict__ leaves, uint32_t n, Geo g, Ws ws, wm_result* result, int decode)
{
    __shared__ unsigned long long s_start[kMaxLeaves + 1];      // logical offset of each leaf; [n] = nbytes
    __shared__ unsigned long long s_wsum[32];
    __shared__ uint32_t s_bad;
    const uint32_t lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    grid_dep_wait();
    grid_dep_launch();
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    // thread i owns leaves 4i .. 4i+3
    unsigned long long len[4], mine = 0;
    uint32_t bad = 0;
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const uint32_t i = 4 * threadIdx.x + k;
        len[k] = 0;
        if (i < n) {
            const unsigned long long nb = leaves[i].nbytes;
            const unsigned long long p = reinterpret_cast<unsigned long long>(leaves[i].ptr);
            if (nb == 0 || nb > g.nbytes || p == 0 || (p & 15ull) != 0) bad = 1;
            len[k] = nb <= g.nbytes ? nb : 0;          // (a refused size must not wrap the sum)
            mine += len[k];
        }
    }
    unsigned long long incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= (uint32_t)d) incl += o;
    }
    if (lane == 31) s_wsum[warp] = incl;
    if (bad) s_bad = 1;
    __syncthreads();
    unsigned long long run = incl - mine;
    for (uint32_t w2 = 0; w2 < warp; w2++) run += s_wsum[w2];
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const uint32_t i = 4 * threadIdx.x + k;
        if (i < n) s_start[i] = run;
        run += len[k];
    }
    if (threadIdx.x == 1023 && run != g.nbytes) s_bad = 1;      // the last thread's running sum is the total
    __syncthreads();
    if (threadIdx.x == 0) s_start[n] = g.nbytes;
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
    if (blockIdx.x == 0)
        for (uint32_t i = threadIdx.x; i <= n; i += blockDim.x) ws.lstart[i] = s_start[i];
    for (uint32_t t = blockIdx.x * blockDim.x + threadIdx.x; t < g.n_tiles; t += gridDim.x * blockDim.x) {
        const unsigned long long L0 = (unsigned long long)t * kTile;
        uint32_t lo = 0, hi = n;                       // the leaf with start[lo] <= L0 < start[lo + 1]
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) / 2;
            if (s_start[mid] <= L0) lo = mid; else hi = mid;
        }
        const unsigned long long in_leaf = L0 - s_start[lo];            // the tile's first byte inside its leaf
        const unsigned long long leaf_len = s_start[lo + 1] - s_start[lo];
        const unsigned long long addr = reinterpret_cast<unsigned long long>(leaves[lo].ptr) + in_leaf;
        const unsigned long long r = addr & 15ull;
        // whole, inside this leaf, and so is the aligned block that a shifted copy reads
        const bool direct = L0 + kTile <= g.nbytes && in_leaf + kTile + (r ? 16ull - r : 0ull) <= leaf_len;
        ws.tptr[t] = direct ? addr : (kTileWalked | lo);
    }
}

// ---- walked tiles: byte-exact access through the leaf table (rare, kept out of line) ----

struct LeafView {
    const wm_leaf* leaves;                 // [n] the caller's table
    const unsigned long long* lstart;      // [n + 1] logical offsets (k_leaf_map)
    uint32_t n;
};

// The address of logical byte L, walking forward from leaf k (k is moved along; L < nbytes).
__device__ __forceinline__ unsigned char* leaf_byte_addr(const LeafView& lv, uint32_t& k, unsigned long long L)
{
    while (k + 1 < lv.n && L >= lv.lstart[k + 1]) k++;
    return const_cast<unsigned char*>(static_cast<const unsigned char*>(lv.leaves[k].ptr)) + (L - lv.lstart[k]);
}

// A walked tile of `len` (1..16384) real bytes gathered into the team's stage in shared memory,
// byte for byte (thread tt of the team's 256 takes bytes 64 tt .. 64 tt + 63); bytes beyond `len`
// are set to zero.  `k0`: the leaf of the tile's first byte, `L0`: the tile's logical offset.  The
// caller puts a team barrier behind it.
__device__ __noinline__ void walked_tile_to_stage(LeafView lv, uint32_t k0, unsigned long long L0, uint32_t len,
                                                  unsigned char* stage, uint32_t tt)
{
    uint32_t k = k0;
    for (uint32_t w = 0; w < 16u; w++) {
        const uint32_t at = 64u * tt + 4u * w;
        uint32_t word = 0;
        for (uint32_t j = 0; j < 4u; j++)
            if (at + j < len) word |= (uint32_t)*leaf_byte_addr(lv, k, L0 + at + j) << (8u * j);
        reinterpret_cast<uint32_t*>(stage)[at / 4u] = word;
    }
}

// The reverse: a decoded tile standing in the team's stage scattered to where the leaf table says
// (thread tt takes bytes 64 tt .. 64 tt + 63; bytes beyond `len` are not part of the cache).
__device__ __noinline__ void stage_to_walked_tile(LeafView lv, uint32_t k0, unsigned long long L0, uint32_t len,
                                                  const unsigned char* stage, uint32_t tt)
{
    uint32_t k = k0;
    for (uint32_t w = 0; w < 16u; w++) {
        const uint32_t at = 64u * tt + 4u * w;
        const uint32_t word = reinterpret_cast<const uint32_t*>(stage)[at / 4u];
        for (uint32_t j = 0; j < 4u; j++)
            if (at + j < len) *leaf_byte_addr(lv, k, L0 + at + j) = (unsigned char)(word >> (8u * j));
    }
}

// The cache's last chunk when it is shorter than four bytes (its CRC is taken byte by byte).
__device__ __noinline__ uint32_t tiny_chunk_crc_leaves(const uint32_t* T0, LeafView lv, unsigned long long L0, uint32_t len)
{
    // (every leaf holds at least one byte, so the last `len` bytes sit in the last `len` leaves)
    uint32_t crc = 0xFFFFFFFFu, k = lv.n > len ? lv.n - len : 0u;
    for (uint32_t i = 0; i < len; i++) crc = T0[(crc ^ *leaf_byte_addr(lv, k, L0 + i)) & 0xFF] ^ (crc >> 8);
    return ~crc;
}

}  // namespace wm
