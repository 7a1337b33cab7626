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
// tile, the address the main kernels use for it (ws.tptr):
//   - a tile whose 16384 bytes sit in one leaf, together with the 16-byte aligned block around
//     them: the address of its first byte inside the leaf.  It moves by a bulk copy from the
//     address rounded down to 16; the main kernels shift the words by the remainder.
//   - any other tile (it crosses a leaf boundary, or is the ragged last tile, or ends within 16
//     bytes of the end of a leaf whose size is no multiple of 16: the aligned block would reach
//     past the leaf) is a "walked" tile: it gets a 16 KiB slot in the workspace's side buffer and
//     its address is the slot's.  k_leaf_gather fills the slots from the leaves before the encode
//     kernel runs, k_leaf_scatter empties them into the leaves after the decode kernel has run,
//     both run by run, byte by byte, so the main kernels see ordinary aligned tiles and carry no
//     code for the exception.  There are at most two walked tiles per leaf; ws.wlist keeps their
//     numbers, ctrl->n_walked their count.
// Rules (a table that breaks one raises error bit 8; in decode mode it also closes the gate and
// writes the result record; nothing is read or written through a rejected table): 1..4096
// leaves, every pointer 16-byte aligned, every size positive and at most nbytes (so the sum
// cannot wrap), the sizes add up to nbytes, at most kMaxWalked walked tiles.

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
    auto refuse = [&]() {
        atomicOr(&ws.ctrl->err, 8u);
        if (decode) {
            ws.ctrl->gate = (uint32_t)WM_ERR_ARG;
            wm_result r;
            memset(&r, 0, sizeof r);
            r.status = WM_ERR_ARG;
            *result = r;
        }
    };
    if (s_bad) {
        if (blockIdx.x == 0 && threadIdx.x == 0) refuse();
        return;
    }
    if (blockIdx.x == 0)
        for (uint32_t i = threadIdx.x; i <= n; i += blockDim.x) ws.lstart[i] = s_start[i];
    const uint32_t n_slots = g.n_tiles < kMaxWalked ? g.n_tiles : kMaxWalked;
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
        if (direct) {
            ws.tptr[t] = addr;
        } else {
            const uint32_t slot = atomicAdd(&ws.ctrl->n_walked, 1u);
            if (slot < n_slots) {
                ws.wlist[slot] = t;
                ws.tptr[t] = reinterpret_cast<unsigned long long>(ws.side + (size_t)slot * kTile);
            } else {
                ws.tptr[t] = 0ull;
                if (slot == n_slots) refuse();         // too many tiles cut by leaf boundaries for the side buffer
            }
        }
    }
}

// The runs of consecutive bytes a walked tile is made of (one per leaf it touches), handed to
// `f(leaf_bytes, tile_offset, run_length)`; every thread of the block goes through the same runs.
template <typename F>
__device__ __forceinline__ void for_each_run(const wm_leaf* __restrict__ leaves, const unsigned long long* __restrict__ lstart,
                                             uint32_t n, const Geo& g, uint32_t t, F f)
{
    const unsigned long long L0 = (unsigned long long)t * kTile;
    const uint32_t len = (uint32_t)min((unsigned long long)kTile, g.nbytes - L0);
    uint32_t lo = 0, hi = n;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) / 2;
        if (lstart[mid] <= L0) lo = mid; else hi = mid;
    }
    uint32_t done = 0;
    for (uint32_t k = lo; done < len && k < n; k++) {
        const unsigned long long at = L0 + done;                       // first byte of the run (lstart[k] <= at < lstart[k + 1])
        const uint32_t run = (uint32_t)min((unsigned long long)(len - done), lstart[k + 1] - at);
        f(const_cast<unsigned char*>(static_cast<const unsigned char*>(leaves[k].ptr)) + (at - lstart[k]), done, run);
        done += run;
    }
}

// Encode: every walked tile copied from the leaves into its slot (one block per tile at a time).
__global__ void __launch_bounds__(256)
k_leaf_gather(const wm_leaf* __restrict__ leaves, uint32_t n, Geo g, Ws ws)
{
    grid_dep_wait();
    grid_dep_launch();
    if (ld_volatile_u32(&ws.ctrl->err) & 8u) return;
    const uint32_t n_walked = ld_volatile_u32(&ws.ctrl->n_walked);
    for (uint32_t s = blockIdx.x; s < n_walked; s += gridDim.x) {
        unsigned char* slot = ws.side + (size_t)s * kTile;
        for_each_run(leaves, ws.lstart, n, g, ws.wlist[s], [&](const unsigned char* src, uint32_t off, uint32_t run) {
#pragma unroll 16
            for (uint32_t i = threadIdx.x; i < run; i += blockDim.x) slot[off + i] = src[i];
        });
    }
}

// Decode: every walked tile copied from its slot into the leaves.  Runs behind the decode kernel
// that stores; stays out when the gate is closed (nothing was decoded, the slots hold nothing).
__global__ void __launch_bounds__(256)
k_leaf_scatter(const wm_leaf* __restrict__ leaves, uint32_t n, Geo g, Ws ws)
{
    grid_dep_wait();
    grid_dep_launch();
    if (ld_volatile_u32(&ws.ctrl->gate)) return;
    const uint32_t n_walked = ld_volatile_u32(&ws.ctrl->n_walked);
    for (uint32_t s = blockIdx.x; s < n_walked; s += gridDim.x) {
        const uint32_t t = ws.wlist[s];
        if (!(ld_volatile_u32(&ws.cflag[chunk_of(g, t)]) & CF_PRESENT)) continue;     // a tile of an absent chunk was not decoded
        const unsigned char* slot = ws.side + (size_t)s * kTile;
        for_each_run(leaves, ws.lstart, n, g, t, [&](unsigned char* dst, uint32_t off, uint32_t run) {
#pragma unroll 16
            for (uint32_t i = threadIdx.x; i < run; i += blockDim.x) dst[i] = slot[off + i];
        });
    }
}

}  // namespace wm
