// wm_decode_verify: the gate (k_decode_check), the unpack + checksum kernel with its variants
// (leaves, strict passes, entropy option) and the verdict (k_decode_finish).
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

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
// each), the others check the structure chunk by chunk (tile entries against the chunk's length
// and enc_len; also each tile's offset inside its chunk's payload): one warp per chunk, or, when
// a chunk has 16 tiles or fewer, as many whole chunks as fit the warp's 32 lanes side by side.
// Neither part follows anything it reads: every index comes from the call's geometry, so the
// structure pass is safe on damaged metadata and can run beside the CRC.  The last block to
// finish decides in the specified order: metadata CRC first (WM_ERR_META_CRC), then the
// structure (WM_ERR_STRUCT: per-chunk findings, payload offsets as the running sum of enc_len,
// totals against the header).  The offsets are the running sum exactly when the first is 0 and
// every other one is its predecessor's plus that one's enc_len, which the structure pass checks
// chunk by chunk as it goes; only when that fails somewhere does the last block walk the whole
// directory to find which chunks differ from the running sum (the specified count).  A header that does not match the call stops every block at
// once (WM_ERR_FORMAT).  A failure sets the gate that keeps the later kernels out.
__host__ __device__ __forceinline__ uint32_t check_chunks_per_warp(uint32_t tiles_per_chunk)
{
    return tiles_per_chunk <= 16u ? 32u / tiles_per_chunk : 1u;
}

__global__ void __launch_bounds__(1024)
k_decode_check(const unsigned char* __restrict__ wire, uint64_t wire_len, Geo g, Ws ws,
               const Tables* __restrict__ tab, wm_result* result, uint32_t meta_blocks, uint32_t expect_ent)
{
    __shared__ uint32_t sG[1024];
    __shared__ uint32_t sHT[1024];
    __shared__ uint32_t s_dig[1024];
    __shared__ uint32_t s_wdig[4][8];
    __shared__ unsigned long long s_part[33];
    __shared__ uint32_t s_first, s_count;
    __shared__ bool s_last;
    __shared__ int s_format_bad;
    const uint32_t lane = threadIdx.x % 32, wblk = threadIdx.x / 32;
    if (blockIdx.x < meta_blocks) load_small_chain_tables(sG, tab);       // (the structure blocks need no tables)
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
        // one tile entry: its payload length and what it says about its chunk
        struct Entry { uint32_t len; bool ok, any, all, packs; };
        auto read_entry = [&](uint32_t t, uint64_t left) {      // left: bytes of the chunk from this tile on
            Entry r = {0u, true, false, true, false};
            const uint32_t e = tab16[t];
            if (e == 0) r.all = false;
            else {
                r.any = true;
                if (left < kTile) { if (e != 0xFFFFu) r.ok = false; r.len = (uint32_t)left; }
                else if (e == 1u && zero_ok) r.len = 0;       // a tile of zeros: no payload
                else if (e == 2u && zero_ok) r.len = 32;      // a tile of one value: the value
                else if (e >= 258u && e <= 512u) { r.len = 32u * e; r.packs = e < 512u; }
                else if (expect_ent && e >= (0x8000u | 259u) && e <= (0x8000u | 511u)) r.len = 32u * (e & 0x7FFFu);   // ENT tile
                else r.ok = false;
            }
            return r;
        };
        // chunk cc's offset against its predecessor's (one lane per chunk)
        auto offset_follows = [&](uint32_t cc) {
            const unsigned long long po = *reinterpret_cast<const unsigned long long*>(dir + 16ull * cc);
            if (cc == 0) return po == 0ull;
            const uint4 pr = *reinterpret_cast<const uint4*>(dir + 16ull * (cc - 1u));
            return po == (pr.x | ((unsigned long long)pr.y << 32)) + pr.z;
        };
        const uint32_t tpc = g.tiles_per_chunk, cpw = check_chunks_per_warp(tpc);
        const uint32_t cw = ((blockIdx.x - meta_blocks) * 32u + wblk) * cpw;        // the warp's first chunk
        bool present = false, bad = false;            // the verdict on chunk c, held by the lane that reports it
        uint32_t c = cw;
        if (cpw == 1u) {
            if (c < g.n_chunks) {
                const uint64_t clen = chunk_len_dev(g, c);
                const uint32_t t0 = c * tpc;
                const uint32_t ntc = (uint32_t)((clen + kTile - 1) / kTile);
                const uint32_t elen = *reinterpret_cast<const uint32_t*>(dir + 16ull * c + 8);
                unsigned long long carry = 0;
                bool ok = true, any = false, all = true;
                for (uint32_t i0 = 0; i0 < ntc; i0 += 32) {
                    const uint32_t i = i0 + lane;
                    Entry en = {0u, true, false, true, false};
                    if (i < ntc) en = read_entry(t0 + i, clen - (uint64_t)i * kTile);
                    uint32_t incl = en.len;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                        if (lane >= (uint32_t)d) incl += o;
                    }
                    if (i < ntc) ws.rel[t0 + i] = (uint32_t)(carry + incl - en.len);
                    carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
                    if (expect_ent && __any_sync(0xFFFFFFFFu, en.packs) && lane == 0) atomicOr(&ws.ctrl->has_pack, 1u);
                    ok = ok && __all_sync(0xFFFFFFFFu, en.ok);
                    any = any || __any_sync(0xFFFFFFFFu, en.any);
                    all = all && __all_sync(0xFFFFFFFFu, en.all);
                }
                if (any && !all) ok = false;
                if (carry != elen) ok = false;
                present = any && lane == 0;
                bad = !ok && lane == 0;
                if (lane == 0) {
                    ws.cflag[c] = (any ? CF_PRESENT : 0u) | (ok ? 0u : CF_BAD3);
                    if (!offset_follows(c)) ws.ctrl->off_bad = 1u;
                }
            }
        } else {
            // lanes [k * tpc, (k + 1) * tpc) hold chunk cw + k; the lanes behind the last whole chunk idle
            const uint32_t seg = lane / tpc, li = lane - seg * tpc;
            c = cw + seg;
            const bool active = seg < cpw && c < g.n_chunks;
            const uint64_t clen = active ? chunk_len_dev(g, c) : 0ull;
            const uint32_t ntc = (uint32_t)((clen + kTile - 1) / kTile);
            const bool in = active && li < ntc;
            Entry en = {0u, true, false, true, false};
            if (in) en = read_entry(c * tpc + li, clen - (uint64_t)li * kTile);
            uint32_t incl = en.len;
#pragma unroll
            for (int d = 1; d < 16; d <<= 1) {           // (a lane adds from inside its own chunk only)
                const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (li >= (uint32_t)d) incl += o;
            }
            if (in) ws.rel[c * tpc + li] = incl - en.len;
            const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, min(seg * tpc + tpc - 1u, 31u));      // (lanes behind the chunk's last tile add 0)
            const uint32_t segmask = active ? ((1u << tpc) - 1u) << (seg * tpc) : 0u;
            const bool ok_all = (__ballot_sync(0xFFFFFFFFu, en.ok) & segmask) == segmask;
            const bool any = (__ballot_sync(0xFFFFFFFFu, en.any) & segmask) != 0u;
            const bool all = (__ballot_sync(0xFFFFFFFFu, in && !en.all) & segmask) == 0u;
            if (expect_ent && __any_sync(0xFFFFFFFFu, en.packs) && lane == 0) atomicOr(&ws.ctrl->has_pack, 1u);
            if (active && li == 0) {
                const uint32_t elen = *reinterpret_cast<const uint32_t*>(dir + 16ull * c + 8);
                const bool ok = ok_all && !(any && !all) && tot == elen;
                present = any;
                bad = !ok;
                ws.cflag[c] = (any ? CF_PRESENT : 0u) | (ok ? 0u : CF_BAD3);
                if (!offset_follows(c)) ws.ctrl->off_bad = 1u;
            }
        }
        // (the present chunks, in any order: k_decode claims their tiles only; one count per warp)
        const uint32_t pres = __ballot_sync(0xFFFFFFFFu, present);
        uint32_t slot0 = 0;
        if (lane == 0 && pres) slot0 = atomicAdd(&ws.ctrl->n_present, (uint32_t)__popc(pres));
        slot0 = __shfl_sync(0xFFFFFFFFu, slot0, 0);
        if (present) ws.plist[slot0 + __popc(pres & ((1u << lane) - 1u))] = c;
        if (bad) { atomicMin(&ws.ctrl->bad3_first, c); atomicAdd(&ws.ctrl->bad3_count, 1u); }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        s_first = 0xFFFFFFFFu; s_count = 0;
        __threadfence();
        s_last = atomicAdd(&ws.ctrl->done_b, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // ---- the last block: metadata CRC first
    sHT[threadIdx.x] = (&tab->HT[0][0])[threadIdx.x];
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

    // ---- then the structure across chunks.  Every offset followed from its predecessor: the
    // offsets are the running sum, and the payload's length is the last chunk's end.  Otherwise
    // the chunks whose payload_off is not the sum of the lengths before it are found and counted:
    // every warp takes a run of consecutive chunks, 32 at a time (consecutive lanes read
    // consecutive directory entries); one prefix over the warps' sums gives each run its start.
    unsigned long long payload_sum;
    if (!ld_volatile_u32(&ws.ctrl->off_bad)) {       // (block-uniform)
        const uint4 en = *reinterpret_cast<const uint4*>(dir + 16ull * (g.n_chunks - 1u));
        payload_sum = (en.x | ((unsigned long long)en.y << 32)) + en.z;
    } else {
        const uint32_t per_w = (g.n_chunks + 31u) / 32u;
        const uint32_t w0 = min(wblk * per_w, g.n_chunks), w1 = min(w0 + per_w, g.n_chunks);
        unsigned long long mine = 0;
        for (uint32_t cc = w0 + lane; cc < w1; cc += 32u) mine += *reinterpret_cast<const uint32_t*>(dir + 16ull * cc + 8);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, d);      // the warp's sum, in every lane
        unsigned long long run = block_prefix(lane == 0 ? mine : 0ull, s_part, payload_sum);  // lane 0: where the warp's run starts
        run = __shfl_sync(0xFFFFFFFFu, run, 0);
        for (uint32_t base = w0; base < w1; base += 128u) {
            uint4 en[4];                   // (four rounds' entries asked for at once: one round trip to L2, not four)
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const uint32_t cc = base + 32u * k + lane;
                en[k] = cc < w1 ? *reinterpret_cast<const uint4*>(dir + 16ull * cc) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const uint32_t cc = base + 32u * k + lane;
                const unsigned long long po = en[k].x | ((unsigned long long)en[k].y << 32), len = en[k].z;
                unsigned long long incl = len;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                    if (lane >= (uint32_t)d) incl += o;
                }
                if (cc < w1 && po != run + incl - len) {
                    // a chunk already counted by the per-chunk pass must not be counted twice
                    const uint32_t fl = ld_volatile_u32(&ws.cflag[cc]);
                    if (!(fl & CF_BAD3)) {
                        ws.cflag[cc] = fl | CF_BAD3;
                        atomicMin(&s_first, cc);
                        atomicAdd(&s_count, 1u);
                    }
                }
                run += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t first = min(s_first, ld_volatile_u32(&ws.ctrl->bad3_first));
        uint32_t count = s_count + ld_volatile_u32(&ws.ctrl->bad3_count);
        if (count == 0 && (payload_sum != ws.ctrl->payload_total ||
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
    // what the leader asks for about the tile two ahead arrives here (the 16 bytes around its table
    // entry, around its offset inside its chunk, and its chunk's directory entry): answers that are
    // a step under way and would otherwise hold registers of every thread for that long
    uint4 in_tab, in_rel, in_dir;
    uint4 in_ptr;                // leaf mode: the 16 bytes around the tile's address in the leaves
    unsigned long long dstp[4];  // leaf mode, same ring as slot[]: where the tile goes
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
// warp reads its share's stream in phase 1, every lane its own strand, and leaves the exponent
// bytes where the plane words would be.
template <int TEAMS, bool LEAVES, int MODE, int ENT = 0>
__global__ void __launch_bounds__(TEAMS * 256, 1)
k_decode(const unsigned char* __restrict__ wire, Geo g, unsigned char* __restrict__ dst, Ws ws,
         const Tables* __restrict__ tab)
{
    extern __shared__ __align__(16) unsigned char smem[];
    // ENT: what the low byte of a strand's bits says about the codeword there: its length (16: the
    // escape) and u as a byte.  Two byte tables: the index needs no scaling and a look-up gives a
    // clean value.
    // (256-byte aligned: the window's low byte OR'ed into the table's address is the look-up's address)
    __shared__ __align__(256) unsigned char s_ptab[ENT ? 512 : 4];       // [0..255] length (16: the escape), [256..511] u
    if (ENT != 0 && threadIdx.x < 256u) {
        const uint32_t s = ent_ones(threadIdx.x);
        s_ptab[threadIdx.x] = (unsigned char)ent_parse_length(s);
        s_ptab[256u + threadIdx.x] = (unsigned char)(s == 8u ? 0u : ent_parse_value(threadIdx.x, s, 0u));
    }
    const uint32_t ptab_s = (uint32_t)__cvta_generic_to_shared(s_ptab);
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
    // The team's control block by its 32-bit shared-window address.  What every thread does with it
    // in the loop (its tile's slot, the copy's barrier, a warp's digest part) goes through that
    // address; the single-thread chores make themselves a pointer from it where they stand.  A
    // 64-bit pointer kept for the whole loop was the one value the kernel spilled, and it came
    // back from L2 (the L1 is small beside 225 KiB of shared memory) in every warp, every tile.
    const uint32_t tc_s = (uint32_t)__cvta_generic_to_shared(tc);
    auto TC = [&]() {
        uint32_t a = tc_s;
        asm volatile("" : "+r"(a));
        return static_cast<DecTeamCtl*>(__cvta_shared_to_generic((size_t)a));
    };
    // The image's parts.  Each is needed by one thread of a team once per tile, so they are worked
    // out from the kernel's arguments where they are used rather than kept in registers of every
    // thread for the whole loop (`fresh` keeps the compiler from hoisting the sums back out: the
    // kernel has no register to spare, and a value it spills costs every warp a trip to L2 per tile).
    auto fresh = [](const unsigned char* p) { asm volatile("" : "+l"(p)); return p; };
    auto dir_of = [&]() { return fresh(wire) + 64; };
    auto tab16_of = [&]() { return reinterpret_cast<const uint16_t*>(fresh(wire) + 64 + 16ull * g.n_chunks); };
    auto payload_of = [&]() { return fresh(wire) + g.meta_end; };
    const bool leader = (tt == 0);
    constexpr uint32_t kNone = 0xFFFFFFFFu;
    // The tile behind a ticket.  Without a mask tickets are tile numbers (one past the last tile:
    // none left).  An image made with a dirty mask (header flags bit 0) holds the tiles of its
    // present chunks only; k_decode_check listed those chunks (ws.plist, in any order: nothing here
    // depends on the order of tiles), and ticket k is tile k mod tiles_per_chunk of the
    // (k / tiles_per_chunk)-th listed chunk, so a sparse image costs nothing for what it leaves
    // out.  Only the cache's last chunk can have fewer tiles: a ticket that falls behind its end
    // has no tile, and the claimer draws the next one at once.
    const bool masked = ((reinterpret_cast<const uint32_t*>(wire)[1] >> 16) & 1u) != 0u;
    const uint32_t n_tickets = masked ? ld_volatile_u32(&ws.ctrl->n_present) * g.tiles_per_chunk : 0u;
    auto claim = [&]() -> uint32_t {
        uint32_t k = atomicAdd(&ws.ctrl->ticket, 1u);
        if (!masked) return k;
        while (k < n_tickets) {
            const uint32_t j = chunk_of(g, k);
            const uint32_t t = ws.plist[j] * g.tiles_per_chunk + (k - j * g.tiles_per_chunk);
            if (t < g.n_tiles) return t;
            k = atomicAdd(&ws.ctrl->ticket, 1u);
        }
        return kNone;
    };
    const uint32_t stage_s = (uint32_t)__cvta_generic_to_shared(stage);
    const uint32_t sm_s = stage_s + 64u + 1024u * warp + 8u * lane;     // this lane's sign-mantissa bytes, group 4 warp

    // a tile's entry word and payload offset (blocking: prologue only)
    auto lookup = [&](uint32_t t, DecSlot* sl) {
        if (LEAVES && t < g.n_tiles) tc->dstp[sl - tc->slot] = ws.tptr[t];
        sl->t = t;
        sl->entry = 0; sl->src = 0;
        if (t < g.n_tiles) {
            const uint32_t e = tab16_of()[t];
            sl->entry = e | (first_in_chunk(g, t) ? 0x10000u : 0u);
            if (e) sl->src = *reinterpret_cast<const unsigned long long*>(dir_of() + 16ull * chunk_of(g, t)) + ws.rel[t];
        }
    };
    // staged tiles: full RAW and PACK tiles (everything except absent tiles and the ragged tail)
    // (images with the entropy option hold ENT tiles too: entry 0x8000 | length / 32)
    auto is_ent_entry = [](uint32_t e) { return ENT != 0 && e > 0x8000u && e != 0xFFFFu; };
    auto is_pack_entry = [](uint32_t e) { return ENT != 1 && e >= 258u && e < 512u; };
    auto is_staged = [&](uint32_t e) { return e == 512u || is_pack_entry(e) || is_ent_entry(e); };
    auto start_copy = [&](const DecSlot& sl) {   // leader only
        const uint32_t e = sl.entry & 0xFFFFu;
        if (sl.t < g.n_tiles && is_staged(e) && !(g.inject & kInjectNoCopy)) bulk_load_at(stage_s, payload_of() + sl.src, 32u * (e & 0x7FFFu), tc_s + (uint32_t)offsetof(DecTeamCtl, mbar), 0);
    };

    if (leader) {
        mbar_init(&tc->mbar, 1);
        lookup(claim(), &tc->slot[0]);
        lookup(claim(), &tc->slot[1]);
        tc->slot[2].t = claim();      // its look-ups happen in the first step
        start_copy(tc->slot[0]);
    }
    team_bar(team);
    uint32_t phase = 0;
    uint32_t t_done = kNone;           // tile whose digest parts wait in wdig[(it - 1) & 1]
    for (uint32_t it = 0;; it++) {
        const uint32_t t = lds_now<offsetof(DecTeamCtl, slot)>(tc_s + 16u * (it & 3u));
        if (t >= g.n_tiles) {
            team_bar(team);
            if (tt == 32u && t_done != kNone) ws.dig[t_done] = xor8(TC()->wdig[(it & 1u) ^ 1u]);
            break;
        }
        const uint32_t ew = lds_now<offsetof(DecTeamCtl, slot) + 4>(tc_s + 16u * (it & 3u));
        const uint32_t e = ew & 0xFFFFu;
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
            wait_for_copy_at<ENT == 0>(tc_s + (uint32_t)offsetof(DecTeamCtl, mbar), phase, g.wait_ns, ws.ctrl, (g.inject & kInjectNoCopy) != 0u);
            phase ^= 1u;
            if (!is_pack) {
                read_staged_words_at(stage_s, warp, lane, w);
            } else if (is_ent) {
                // ENT tile.  Header: the eight word counts against the entry (structure).  Then lane l
                // reads strand l of this warp's share: the strands lie one behind the other in the
                // share's stream and their lengths are written down, so a prefix sum over the lanes
                // gives every lane the bit where its strand starts, and from there it reads its 32
                // codewords through a 64-bit window that is refilled a word at a time before every
                // second codeword.  No lane waits for another.
                const uint32_t cnt = lane < 8u ? lds_now_u16(stage_s + 8u + 2u * lane) : 0u;
                const bool cnt_bad = lane < 8u && (cnt < 64u || cnt > 319u);
                const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, cnt);
                const uint32_t before = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? cnt : 0u);
                const uint32_t mine = __shfl_sync(0xFFFFFFFFu, cnt, warp);
                int verdict = (__any_sync(0xFFFFFFFFu, cnt_bad) || ent_tile_bytes(total) != 32u * (e & 0x7FFFu)) ? 2 : 0;
                const uint32_t nb = 64u + lds_now_u8(stage_s + 8256u + 32u * warp + lane);      // this strand's bits
                uint32_t incl = nb;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                    if (lane >= (uint32_t)d) incl += o;
                }
                const uint32_t share_bits = __shfl_sync(0xFFFFFFFFu, incl, 31);
                if (!verdict && ((share_bits + 31u) >> 5) != mine) verdict = 1;
                if (!verdict) {
                    const uint32_t anchor = lds_now_u8(stage_s + warp);
                    const uint32_t st = stage_s + 8512u + 4u * before;
                    const uint32_t start = incl - nb, wi = start >> 5, sh = start & 31u;
                    // (a strand that runs past its length only fails the check below: no word beyond
                    // the share's last two is ever read)
                    // The window: lo holds the next 32 bits of the strand, hi what follows, `avail` of the
                    // 64 are real.  (PTX shifts clamp at 32, which is what the edge cases need.)
                    uint32_t lo = lds_now<0>(st + 4u * wi), hi = lds_now<4>(st + 4u * wi);
                    lo = __funnelshift_r(lo, hi, sh);
                    hi >>= sh;
                    uint32_t avail = 64u - sh, next = wi + 2u, ew[8];
#pragma unroll
                    for (int j = 0; j < 8; j++) ew[j] = 0u;
#pragma unroll
                    for (int i = 0; i < 32; i++) {
                        if ((i & 1) == 0 && avail <= 32u) {      // (two codewords take 32 bits at most)
                            const uint32_t w = lds_now<0>(st + 4u * min(next, mine + 1u));
                            lo |= shl_clamp(w, avail);
                            hi = shr_clamp(w, 32u - avail);
                            avail += 32u;
                            next++;
                        }
                        const uint32_t at = (lo & 0xFFu) | ptab_s;
                        const uint32_t len = lds_tab_u8(at);
                        const uint32_t E = len == 16u ? lo >> 8 : anchor + lds_tab_u8(at + 256u);      // (its low byte)
                        ew[i >> 2] = __byte_perm(ew[i >> 2], E, (i & 3) == 0 ? 0x3214 : (i & 3) == 1 ? 0x3240 : (i & 3) == 2 ? 0x3410 : 0x4210);
                        lo = __funnelshift_r(lo, hi, len);
                        hi >>= len;
                        avail -= len;
                    }
                    // the 32 codewords took exactly the strand's length; behind the last strand the
                    // stream's last word is zero
                    const uint32_t used = 32u * (next - wi) - sh - avail;
                    const uint32_t fill = 32u * mine - share_bits;
                    const bool fill_bad = lane == 31u && (lo & ((1u << fill) - 1u)) != 0u;
                    if (__any_sync(0xFFFFFFFFu, used != nb || fill_bad)) verdict = 1;
                    // the anchor must be what the encoder writes: the rounded mean of the share's exponents
                    // (otherwise the anchor of a share that holds escapes only could change unnoticed)
                    uint32_t esum = 0;
#pragma unroll
                    for (int j = 0; j < 8; j++) esum = __dp4a(ew[j], 0x01010101u, esum);
                    if (((__reduce_add_sync(0xFFFFFFFFu, esum) + 512u) >> 10) != anchor) verdict = 1;
                    // the bytes that carry nothing are zero: the header's spare 40, the fill behind the last stream
                    if (warp == 0u) {
                        const uint32_t spare = (lane >= 6u && lane < 16u) ? lds_now<0>(stage_s + 4u * lane) : 0u;
                        const uint32_t fill_at = 8512u + 4u * total + 4u * lane;
                        const uint32_t end_fill = fill_at < 32u * (e & 0x7FFFu) ? lds_now<0>(stage_s + fill_at) : 0u;
                        if (__any_sync(0xFFFFFFFFu, (spare | end_fill) != 0u)) verdict = 1;
                    }
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
                desc = lds_now_u16(stage_s + 2u * lane);
                // Whether the descriptors are sound (step 4) is one warp's business, the one without
                // a single-lane chore: its verdict goes to the control block and decides the call's
                // status.  The other warps do not wait for it; they only have to stay inside the
                // stage whatever they find, so a width the format does not have reads as 8 and an
                // offset stops where a sound tile's last group can start.  What they unpack from an
                // unsound tile is garbage in a destination that a failed call leaves unspecified.
                if (warp == 7u) {
                    const uint32_t wr = (desc >> 8) & 15u, base_l = desc & 0xFFu, chk = desc >> 12;
                    const bool bad = wr > 8u || chk != (((base_l & 15u) ^ (base_l >> 4) ^ wr ^ 5u) & 15u);
                    const bool anybad = __any_sync(0xFFFFFFFFu, bad);
                    const uint32_t Ssum = __reduce_add_sync(0xFFFFFFFFu, wr);
                    const int verdict = anybad ? 1 : (258u + Ssum != e ? 2 : 0);
                    if (verdict && lane == 0) {
                        atomicMin(&ws.ctrl->bad4_key, (unsigned long long)t * 2ull + (verdict == 2 ? 1ull : 0ull));
                        atomicOr(&ws.cflag[chunk_of(g, t)], CF_BAD4);
                    }
                }
                // widths of the groups before this warp's four
                const uint32_t wv = min((desc >> 8) & 15u, 8u);
                const uint32_t before = __reduce_add_sync(0xFFFFFFFFu, lane < 4u * warp ? wv : 0u);
                {
                    // lanes 0..3 end up with the descriptors of the warp's four groups, each with its
                    // group's offset in the plane area in the high half
                    const uint32_t own = __shfl_sync(0xFFFFFFFFu, desc, 4 * warp + (lane & 3u)) & 0xFFFFu;
                    const uint32_t wo = min((own >> 8) & 15u, 8u);
                    uint32_t off = before;                          // running offset over the four groups
                    const uint32_t w0 = __shfl_sync(0xFFFFFFFFu, wo, 0), w1 = __shfl_sync(0xFFFFFFFFu, wo, 1),
                                   w2 = __shfl_sync(0xFFFFFFFFu, wo, 2);
                    if ((lane & 3u) >= 1u) off += w0;
                    if ((lane & 3u) >= 2u) off += w1;
                    if ((lane & 3u) == 3u) off += w2;
                    off = min(off, 245u);                           // (8256 + 32 * 245 + 256 bytes of planes end inside the stage)
                    desc = (own & 0xF0FFu) | (wo << 8) | (off << 16);
#pragma unroll
                    for (int j = 0; j < 4; j++) {
                        const uint32_t dg = __shfl_sync(0xFFFFFFFFu, desc, j);
                        sm[j] = j == 0 ? lds_now_v2<0>(sm_s) : j == 1 ? lds_now_v2<256>(sm_s) : j == 2 ? lds_now_v2<512>(sm_s) : lds_now_v2<768>(sm_s);
                        pw[j] = read_group_planes(stage_s + 8256u + 32u * (dg >> 16), (dg >> 8) & 15u, 4u * lane, 2u * lane, lane);
                    }
                }
            }
        } else if (e == 1u || e == 2u) {
            // a tile of zeros (nothing was shipped) or of one value (the first two bytes of its 32):
            // from here on it goes the way of a raw tile
            uint32_t v = 0;
            if (e == 2u) {
                // (the value's 32 bytes: the value itself, and 30 bytes that must be zero)
                const uint32_t* cp = reinterpret_cast<const uint32_t*>(payload_of() + TC()->slot[it & 3u].src);
                const uint32_t x = lane < 8u ? __ldg(cp + lane) : 0u;
                v = (__shfl_sync(0xFFFFFFFFu, x, 0) & 0xFFFFu) * 0x10001u;
                if (__any_sync(0xFFFFFFFFu, (lane == 0u ? x >> 16 : x) != 0u)) {       // every warp reaches the same verdict
                    decoded = false;
                    if (leader) {
                        atomicMin(&ws.ctrl->bad4_key, (unsigned long long)t * 2ull);
                        atomicOr(&ws.cflag[chunk_of(g, t)], CF_BAD4);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 16; i++) w[i] = v;
        }
        team_bar(team);                      // stage free; the slots the leader filled last step visible;
                                             // the previous tile's digest parts complete
        // The leader: next tile's copy; the previous tile's digest; look-ups for the tile two
        // ahead and the ticket of the tile three ahead (answers taken at the end of the step).
        uint32_t l_tk = kNone;
        // (spread over three warps: the team waits for whichever warp has the most to do)
        if (tt == 64u) start_copy(TC()->slot[(it + 1u) & 3u]);
        if (tt == 32u && t_done != kNone) ws.dig[t_done] = xor8(TC()->wdig[p ^ 1u]);
        uint32_t t_look = kNone;           // warps 0 and 3: the tile claimed a step ago (two tiles ahead)
        if (leader) {                      // its table entry and offsets
            t_look = TC()->slot[(it + 2u) & 3u].t;
            if (t_look < g.n_tiles) {
                cp_async16(&TC()->in_tab, tab16_of() + (t_look & ~7u));
                cp_async16(&TC()->in_rel, ws.rel + (t_look & ~3u));
                cp_async16(&TC()->in_dir, dir_of() + 16ull * chunk_of(g, t_look));
                if (LEAVES) cp_async16(&TC()->in_ptr, ws.tptr + (t_look & ~1u));
            }
        }
        if (tt == 96u) {                   // the ticket of the tile three ahead
            t_look = TC()->slot[(it + 2u) & 3u].t;
            if (t_look < g.n_tiles) l_tk = claim();
        }

        // ---- phase 2: unpack, store, checksum
        bool have_digest = false;
        if (e != 0) {
            unsigned long long o_leaf = 0ull;
            if (LEAVES) {
                const uint2 v = lds_now_v2<offsetof(DecTeamCtl, dstp)>(tc_s + 8u * (it & 3u));
                o_leaf = v.x | ((unsigned long long)v.y << 32);
            }
            unsigned char* o = LEAVES ? reinterpret_cast<unsigned char*>(o_leaf) : dst + (uint64_t)t * kTile;
            bool fold = (ew >> 16) != 0;
            if (e == 0xFFFFu) {
                const unsigned char* src = payload_of() + TC()->slot[it & 3u].src;
                const uint32_t len = g.tail_len;
                // (leaf mode: the ragged tile has a slot of its own in the side buffer)
                if (MODE != 1) for (uint32_t i = tt; i < len; i += kTeamThreads) o[i] = src[i];
                if (MODE != 2) load_tile_words_guarded(src, len, fold, warp, lane, w);
                fold = false;
            }
            // where the decoded words go: word i of this lane to byte 128 i of its warp's 2 KiB.  In leaf
            // mode a tile may start off a four-byte boundary inside its leaf; it then takes halfword
            // or byte stores instead of the plain 32-bit one.
            unsigned char* const q = o + warp * 2048u + lane * 4u;
            const uint32_t how = !LEAVES ? 0u : (uint32_t)(o_leaf & 3ull) == 0u ? 0u : (o_leaf & 1ull) ? 2u : 1u;
            // (the rest of the step once per way of storing, so that the choice is made once per tile)
            auto rest_of_step = [&](auto how_c) {
            constexpr uint32_t HOW = decltype(how_c)::value;
            auto put = [&](int i, uint32_t v) {
                if (HOW == 0u) st_stream_u32(q + i * 128, v);
                else if (HOW == 1u) { stg_u16(q + i * 128, v); stg_u16(q + i * 128 + 2, v >> 16); }
                else { stg_u8(q + i * 128, v); stg_u16(q + i * 128 + 1, v >> 8); stg_u8(q + i * 128 + 3, v >> 24); }
            };
            if (is_pack && decoded) {
                // A coded tile goes group by group: four words are rebuilt, stored, and fed to the
                // checksum chain (which walks the lane's sixteen words in order anyway) before the next
                // group is touched, so only four decoded words are alive at a time and the chain's
                // table look-ups overlap the next group's arithmetic.
                const uint32_t fold_mask = (fold && warp == 0u && lane == 0u) ? 0xFFFFFFFFu : 0u;
                uint32_t st = 0, last = 0;
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
                    const uint32_t w0 = __funnelshift_r(r0, r0, 1), w1 = __funnelshift_r(r1, r1, 1);
                    const uint32_t w2 = __funnelshift_r(r2, r2, 1), w3 = __funnelshift_r(r3, r3, 1);
                    if (MODE != 1) { put(4 * j, w0); put(4 * j + 1, w1); put(4 * j + 2, w2); put(4 * j + 3, w3); }
                    if (MODE != 2) {
                        st = chain_step(S, st ^ w0 ^ (j == 0 ? fold_mask : 0u));
                        st = chain_step(S, st ^ w1);
                        st = chain_step(S, st ^ w2);
                        if (j < 3) st = chain_step(S, st ^ w3); else last = st ^ w3;
                    }
                }
                if (MODE != 2) {
                    const uint32_t v = warp_place(S, __reduce_xor_sync(0xFFFFFFFFu, lane_finish(S, last)), warp, lane);
                    if (lane == 0) sts_now(tc_s + (uint32_t)offsetof(DecTeamCtl, wdig) + 32u * p + 4u * warp, v);
                    have_digest = true;
                }
            } else if (decoded) {
                // raw, zero and constant tiles and the ragged tail: the sixteen words are there already
                if (MODE != 1 && e != 0xFFFFu) {
#pragma unroll
                    for (int i = 0; i < 16; i++) put(i, w[i]);
                }
                if (MODE != 2) {
                    const uint32_t v = tile_digest_part(S, w, fold, warp, lane);
                    if (lane == 0) sts_now(tc_s + (uint32_t)offsetof(DecTeamCtl, wdig) + 32u * p + 4u * warp, v);
                    have_digest = true;
                }
            }
            };
            if (!LEAVES || how == 0u) rest_of_step(std::integral_constant<uint32_t, 0u>());
            else if (how == 1u) rest_of_step(std::integral_constant<uint32_t, 1u>());
            else rest_of_step(std::integral_constant<uint32_t, 2u>());
        }
        t_done = have_digest ? t : kNone;
        if (leader && t_look < g.n_tiles) {
            cp_async_wait_all();
            DecSlot* s2 = &TC()->slot[(it + 2u) & 3u];
            const uint32_t l_e = reinterpret_cast<const volatile unsigned short*>(&TC()->in_tab)[t_look & 7u];
            const uint32_t l_rel = reinterpret_cast<const volatile uint32_t*>(&TC()->in_rel)[t_look & 3u];
            const unsigned long long l_po = *reinterpret_cast<const volatile unsigned long long*>(&TC()->in_dir);
            s2->entry = l_e | (first_in_chunk(g, t_look) ? 0x10000u : 0u);
            s2->src = l_po + l_rel;
            if (LEAVES) TC()->dstp[(it + 2u) & 3u] = reinterpret_cast<const volatile unsigned long long*>(&TC()->in_ptr)[t_look & 1u];
        }
        if (tt == 96u) TC()->slot[(it + 3u) & 3u].t = l_tk;      // (none once the tickets have run out)
    }
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
        // (both loads of a chunk are issued before either is looked at, eight chunks at a time:
        // a cache of many small chunks would otherwise pay two round trips to L2 per chunk, in a row)
        for (uint32_t base = threadIdx.x; base < g.n_chunks; base += 8u * blockDim.x) {
            uint32_t fl[8], want[8];
#pragma unroll
            for (int k = 0; k < 8; k++) {
                const uint32_t i = base + k * blockDim.x;
                fl[k] = 0;
                if (i < g.n_chunks) {
                    fl[k] = ws.cflag[i];
                    want[k] = *reinterpret_cast<const uint32_t*>(dir + 16ull * i + 12);
                }
            }
#pragma unroll
            for (int k = 0; k < 8; k++)
                if (fl[k] & CF_PRESENT) dst_crc[base + k * blockDim.x] = want[k];
        }
    }
}

}  // namespace wm
