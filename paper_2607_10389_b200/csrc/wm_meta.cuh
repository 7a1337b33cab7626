// Metadata CRC of a wire image (encode side) and the header match / slice digests both sides share.
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

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

}  // namespace wm
