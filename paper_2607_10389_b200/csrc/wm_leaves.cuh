// Leaf mode: the table of tensors turned into one pointer per tile (k_leaf_map).
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

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

}  // namespace wm
