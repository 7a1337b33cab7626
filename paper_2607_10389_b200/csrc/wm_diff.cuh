// wm_dirty_diff: exact compare of two snapshots, chunk mask, count and index list.
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

// ------------------------------------------------------------------ wm_dirty_diff

__global__ void k_diff_init(Ws ws)
{
    grid_dep_launch();
    if (threadIdx.x == 0 && blockIdx.x == 0) { ws.ctrl->ticket = 0; ws.ctrl->n_present = 0; ws.ctrl->err = 0; }
}

// One block per chunk at a time (ticketed); the chunk is scanned in 16 KiB half-steps, two of
// them in flight, and dropped at the first one that shows a difference.
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
        // two half-steps in flight: the loads of the next one are issued before this one is judged,
        // so the block-wide vote never finds the memory pipe empty
        uint4 a[2][4], b[2][4];
        auto fetch = [&](uint64_t o, int slot) {
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const uint64_t p = o + ((uint64_t)k * 256 + threadIdx.x) * 16;
                if (p < vec_len) {
                    a[slot][k] = __ldcs(reinterpret_cast<const uint4*>(cache + base + p));
                    b[slot][k] = __ldcs(reinterpret_cast<const uint4*>(prev + base + p));
                } else {
                    a[slot][k] = make_uint4(0, 0, 0, 0); b[slot][k] = a[slot][k];
                }
            }
        };
        auto differs = [&](int slot) {
            uint32_t d = 0;
#pragma unroll
            for (int k = 0; k < 4; k++)
                d |= (a[slot][k].x ^ b[slot][k].x) | (a[slot][k].y ^ b[slot][k].y) | (a[slot][k].z ^ b[slot][k].z) | (a[slot][k].w ^ b[slot][k].w);
            return d != 0;
        };
        constexpr uint32_t kHalf = kStep / 2;
        if (vec_len) fetch(0, 0);
        for (uint64_t o = 0; o < vec_len; o += 2 * kHalf) {
            if (o + kHalf < vec_len) fetch(o + kHalf, 1);
            any = __syncthreads_or(differs(0));
            if (any || o + kHalf >= vec_len) break;
            if (o + 2 * kHalf < vec_len) fetch(o + 2 * kHalf, 0);
            any = __syncthreads_or(differs(1));
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

}  // namespace wm
