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

// Ascending index list of dirty chunks and their count: one block, every thread a run of
// consecutive chunks, one prefix over the threads' counts.
__global__ void __launch_bounds__(1024)
k_diff_compact(Geo g, const uint8_t* __restrict__ dirty, uint32_t* __restrict__ idx_out, uint32_t* __restrict__ n_out)
{
    __shared__ uint32_t s_part[33];
    grid_dep_wait();
    const uint32_t per = (g.n_chunks + 1023u) / 1024u;
    const uint32_t c0 = min(threadIdx.x * per, g.n_chunks), c1 = min(c0 + per, g.n_chunks);
    uint32_t mine = 0;
    for (uint32_t c = c0; c < c1; c++) mine += dirty[c] != 0 ? 1u : 0u;
    uint32_t total;
    uint32_t at = block_prefix(mine, s_part, total);
    if (idx_out)
        for (uint32_t c = c0; c < c1; c++)
            if (dirty[c] != 0) idx_out[at++] = c;
    if (threadIdx.x == 0) *n_out = total;
}

}  // namespace wm
