// wm_checksum_xxh64: the 64-bit xxHash of every chunk, as a checksum option beside the CRC.
// Part of the one translation unit wm_kernels.cu (included there, in this order).
//
// XXH64 takes its input in 32-byte stripes into four accumulators; lane k of a stripe feeds
// accumulator k through  acc = rotl(acc + in * P2, 31) * P1,  a serial chain over the whole chunk
// (digests of pieces cannot be combined, unlike a CRC).  So a chunk offers four threads of work
// and the parallelism is across chunks: thread 4c + k owns accumulator k of chunk c, a warp
// holds eight chunks, and one warp load fetches eight full 32-byte sectors.  What bounds the
// kernel with large chunks is the latency of that chain, so the loads run two batches of 32
// stripes ahead of it, in registers, and the product in * P2 is taken as a value arrives (off
// the chain: only the add, the rotate and the multiplication by P1 depend on the accumulator).
// With many small chunks (64 KiB) there are enough chains and the kernel runs at the memory rate.
#pragma once

namespace wm {

constexpr unsigned long long kXP1 = 0x9E3779B185EBCA87ull, kXP2 = 0xC2B2AE3D27D4EB4Full, kXP3 = 0x165667B19E3779F9ull,
                             kXP4 = 0x85EBCA77C2B2AE63ull, kXP5 = 0x27D4EB2F165667C5ull;

__device__ __forceinline__ unsigned long long x_rotl(unsigned long long v, int r) { return (v << r) | (v >> (64 - r)); }
__device__ __forceinline__ unsigned long long x_round(unsigned long long acc, unsigned long long in)
{
    return x_rotl(acc + in * kXP2, 31) * kXP1;
}
__device__ __forceinline__ unsigned long long x_merge(unsigned long long h, unsigned long long v)
{
    return (h ^ x_round(0ull, v)) * kXP1 + kXP4;
}

constexpr int kXBatch = 32;       // stripes per batch of loads

__global__ void __launch_bounds__(32)
k_xxh64(const unsigned char* __restrict__ cache, uint64_t nbytes, uint32_t chunk_bytes, uint32_t n_chunks,
        unsigned long long seed, unsigned long long* __restrict__ out)
{
    const uint32_t gt = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t c = gt >> 2, k = gt & 3u;
    const bool live = c < n_chunks;                     // (a quad is live or dead as a whole)
    const unsigned char* base = cache;
    uint64_t len = 0;
    if (live) {
        base = cache + (uint64_t)c * chunk_bytes;
        const uint64_t left = nbytes - (uint64_t)c * chunk_bytes;
        len = left < chunk_bytes ? left : chunk_bytes;
    }
    const uint64_t stripes = len / 32u;
    unsigned long long v = k == 0u ? seed + kXP1 + kXP2 : k == 1u ? seed + kXP2 : k == 2u ? seed : seed - kXP1;
    // (the cache is 16-byte aligned and chunks are multiples of 16 KiB: aligned 8-byte loads)
    const unsigned long long* p = reinterpret_cast<const unsigned long long*>(base) + k;
    unsigned long long a[kXBatch], b[kXBatch];
    uint64_t s = 0;
    if (stripes >= (uint64_t)kXBatch) {
#pragma unroll
        for (int i = 0; i < kXBatch; i++) a[i] = __ldcs(p + 4u * i) * kXP2;
        // two batches per turn: while one is folded into the accumulator the other is on its way
        while (s + 2u * kXBatch <= stripes) {
#pragma unroll
            for (int i = 0; i < kXBatch; i++) b[i] = __ldcs(p + 4u * (s + kXBatch + i)) * kXP2;
#pragma unroll
            for (int i = 0; i < kXBatch; i++) v = x_rotl(v + a[i], 31) * kXP1;
            s += kXBatch;
            if (s + 2u * kXBatch <= stripes) {
#pragma unroll
                for (int i = 0; i < kXBatch; i++) a[i] = __ldcs(p + 4u * (s + kXBatch + i)) * kXP2;
#pragma unroll
                for (int i = 0; i < kXBatch; i++) v = x_rotl(v + b[i], 31) * kXP1;
                s += kXBatch;
            } else {
#pragma unroll
                for (int i = 0; i < kXBatch; i++) a[i] = b[i];
            }
        }
        // a[] holds the batch that starts at s
#pragma unroll
        for (int i = 0; i < kXBatch; i++) v = x_rotl(v + a[i], 31) * kXP1;
        s += kXBatch;
    }
    for (; s < stripes; s++) v = x_round(v, __ldcs(p + 4u * s));

    // the quad's four accumulators to its first thread; merge, tail, avalanche
    const uint32_t q0 = threadIdx.x & ~3u;
    const unsigned long long v1 = __shfl_sync(0xFFFFFFFFu, v, q0), v2 = __shfl_sync(0xFFFFFFFFu, v, q0 + 1u),
                             v3 = __shfl_sync(0xFFFFFFFFu, v, q0 + 2u), v4 = __shfl_sync(0xFFFFFFFFu, v, q0 + 3u);
    if (!live || k != 0u) return;
    unsigned long long h;
    if (len >= 32u) {
        h = x_rotl(v1, 1) + x_rotl(v2, 7) + x_rotl(v3, 12) + x_rotl(v4, 18);
        h = x_merge(h, v1); h = x_merge(h, v2); h = x_merge(h, v3); h = x_merge(h, v4);
    } else {
        h = seed + kXP5;
    }
    h += len;
    const unsigned char* t = base + stripes * 32u;
    uint64_t left = len - stripes * 32u;
    while (left >= 8u) {
        h = x_rotl(h ^ x_round(0ull, *reinterpret_cast<const unsigned long long*>(t)), 27) * kXP1 + kXP4;
        t += 8; left -= 8u;
    }
    if (left >= 4u) {
        h = x_rotl(h ^ ((unsigned long long)*reinterpret_cast<const uint32_t*>(t) * kXP1), 23) * kXP2 + kXP3;
        t += 4; left -= 4u;
    }
    while (left) { h = x_rotl(h ^ ((unsigned long long)*t * kXP5), 11) * kXP1; t++; left--; }
    h ^= h >> 33; h *= kXP2; h ^= h >> 29; h *= kXP3; h ^= h >> 32;
    out[c] = h;
}

}  // namespace wm
