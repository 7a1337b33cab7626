// Device-side building blocks shared by the kernels: shared-memory table layout, the
// word-strided CRC chain, GF(2) products, team barriers and small load/store helpers.
//
// Work unit: a "team" of 8 warps (256 threads) owns one 16 KiB tile at a time.  The tile is
// seen as 128 rows of 128 bytes; warp w owns rows 16w .. 16w+15 and lane l owns the 32-bit
// word l of each of those rows.  A lane therefore walks 16 words that are exactly 128 bytes
// apart, which makes its CRC contribution a Horner chain with ONE fixed multiplier
// (x^1024, table G); the lane's place inside the row and the warp's place inside the tile
// are folded in once per tile with two small nibble tables (NK, NW).
//
// Table lookups are the inner loop (one per byte), so their address arithmetic is reduced to
// a single byte permute: the tables sit at a 64 KiB-aligned shared address, entry b of a
// table starts at b*256 and holds one copy per lane (lane l only ever touches bank l: no
// bank conflicts on data-dependent indices), so address = base | b << 8 | lane*4 is
// PRMT(value, base | lane*4).  The second table of a pair lives 128 bytes further and is
// reached through the load's immediate offset.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "wm_tables.h"

namespace wm {

constexpr uint32_t kTile = 16384;
constexpr uint32_t kTeamThreads = 256;
constexpr uint32_t kWordsPerLane = 16;
// Dynamic shared memory every table-using kernel asks for: the 144 KiB image plus 81 KiB
// that the 64 KiB alignment splits into a part below and a part above the image (with the
// window starting at 1 KiB: 63 KiB below, 18 KiB above; a stage of the leaf-mode kernels is
// 16 bytes longer than a tile, and one of the four has to fit above).  227 KiB is the per-block
// maximum for static and dynamic shared memory together; the kernels' static part is below 1 KiB.
constexpr uint32_t kDynSmem = kImgBytes + 0x10000 + 0x4400;

struct Smem {
    uint32_t L01, L23, LNK;      // shared-window address of A01 / A23 / NK, or'ed with lane*4
    const uint32_t* NW;          // warp-position nibble tables [8][8][16]
    unsigned char* lo; uint32_t lo_bytes;    // free space below the image
    unsigned char* hi; uint32_t hi_bytes;    // free space above the image
    bool ok;

    // carve `bytes` (multiple of 16) from the free space; nullptr when it does not fit
    __device__ unsigned char* take(uint32_t bytes)
    {
        unsigned char* p = nullptr;
        if (lo_bytes >= bytes) { p = lo; lo += bytes; lo_bytes -= bytes; }
        else if (hi_bytes >= bytes) { p = hi; hi += bytes; hi_bytes -= bytes; }
        else ok = false;
        return p;
    }
};

// Copy the table image into shared memory (whole block; ends with __syncthreads).
__device__ __forceinline__ Smem setup_smem(unsigned char* smem, const Tables* __restrict__ tab)
{
    Smem s;
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t tab0 = (base + 0xFFFFu) & ~0xFFFFu;
    unsigned char* img = smem + (tab0 - base);
    s.ok = true;
    s.lo = smem; s.lo_bytes = tab0 - base;
    s.hi = img + kImgBytes; s.hi_bytes = kDynSmem - kImgBytes - (tab0 - base);
    const uint4* src = reinterpret_cast<const uint4*>(tab->image);
    uint4* dst = reinterpret_cast<uint4*>(img);
    for (uint32_t i = threadIdx.x; i < kImgBytes / 16; i += blockDim.x) dst[i] = src[i];
    uint32_t* nw = reinterpret_cast<uint32_t*>(s.take(8 * 8 * 16 * 4));
    if (nw) {
        const uint32_t* gNW = &tab->NW[0][0][0];
        for (uint32_t i = threadIdx.x; i < 8 * 8 * 16; i += blockDim.x) nw[i] = gNW[i];
    }
    s.NW = nw;
    const uint32_t lane4 = (threadIdx.x & 31u) * 4u;
    s.L01 = (tab0 + kImgA01) | lane4;
    s.L23 = (tab0 + kImgA23) | lane4;
    s.LNK = (tab0 + kImgNK) | lane4;
    __syncthreads();
    return s;
}

template <int OFF>
__device__ __forceinline__ uint32_t lds_off(uint32_t addr)
{
    uint32_t v;
    asm("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(OFF));
    return v;
}

// Loads of data that other threads or the copy engine write (stages, team control blocks),
// addressed by 32-bit shared-window addresses so that the address arithmetic stays in 32 bits.
// volatile: they keep their place relative to the barriers and mbarrier waits around them.
template <int OFF>
__device__ __forceinline__ uint32_t lds_now(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(OFF));
    return v;
}
template <int OFF>
__device__ __forceinline__ uint2 lds_now_v2(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(v.x), "=r"(v.y) : "r"(addr), "n"(OFF));
    return v;
}
__device__ __forceinline__ uint32_t lds_now_u16(uint32_t addr)
{
    uint32_t v;
    asm volatile("{\n\t.reg .u16 t;\n\tld.shared.u16 t, [%1];\n\tcvt.u32.u16 %0, t;\n\t}" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_now_u8(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// Look-ups in tables that do not change once they are set up (no volatile: the compiler may place them)
__device__ __forceinline__ uint32_t lds_tab_u8(uint32_t addr)
{
    uint32_t v;
    asm("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_tab_u16(uint32_t addr)
{
    uint32_t v;
    asm("{\n\t.reg .u16 t;\n\tld.shared.u16 t, [%1];\n\tcvt.u32.u16 %0, t;\n\t}" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_now(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// Programmatic dependent launch.  Every call enqueues a short chain of kernels; each kernel but
// the first is launched with permission to start before its predecessor has finished.  It then
// sets up what does not depend on the predecessor (tables into shared memory, allocations) and
// waits here; the wait returns once the predecessor has completed and its writes are visible.
// Every block of such a kernel must pass the wait before it exits or reads anything the chain
// produced.  A kernel tells the scheduler that its successor may be brought in with
// grid_dep_launch (the successor's blocks take SM resources as they become free).
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void team_bar(uint32_t team)
{
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(kTeamThreads) : "memory");
}

// One chain step: (state ^ word) advanced over 128 bytes.
__device__ __forceinline__ uint32_t chain_step(const Smem& S, uint32_t x)
{
    const uint32_t a = lds_off<0>(__byte_perm(x, S.L01, 0x7604));
    const uint32_t b = lds_off<128>(__byte_perm(x, S.L01, 0x7614));
    const uint32_t c = lds_off<0>(__byte_perm(x, S.L23, 0x7624));
    const uint32_t d = lds_off<128>(__byte_perm(x, S.L23, 0x7634));
    return a ^ b ^ c ^ d;
}

// Lane finish: x advanced over 128 - 4*lane bytes (eight nibble lookups).
__device__ __forceinline__ uint32_t lane_finish(const Smem& S, uint32_t x)
{
    const uint32_t xe = x & 0x0F0F0F0Fu, xo = (x >> 4) & 0x0F0F0F0Fu;
    uint32_t r = lds_off<0x0000>(__byte_perm(xe, S.LNK, 0x7604)) ^ lds_off<0x0080>(__byte_perm(xo, S.LNK, 0x7604));
    r ^= lds_off<0x1000>(__byte_perm(xe, S.LNK, 0x7614)) ^ lds_off<0x1080>(__byte_perm(xo, S.LNK, 0x7614));
    r ^= lds_off<0x2000>(__byte_perm(xe, S.LNK, 0x7624)) ^ lds_off<0x2080>(__byte_perm(xo, S.LNK, 0x7624));
    r ^= lds_off<0x3000>(__byte_perm(xe, S.LNK, 0x7634)) ^ lds_off<0x3080>(__byte_perm(xo, S.LNK, 0x7634));
    return r;
}

// CRC state (zero start) of a warp's 2048-byte block from the 16 words each lane holds.
__device__ __forceinline__ uint32_t warp_block_digest(const Smem& S, const uint32_t (&w)[kWordsPerLane])
{
    uint32_t s = 0;
#pragma unroll
    for (int i = 0; i < 15; i++) s = chain_step(S, s ^ w[i]);
    return __reduce_xor_sync(0xFFFFFFFFu, lane_finish(S, s ^ w[15]));
}

// Place a warp's block digest inside the tile: advance over 2048*(7 - warp) bytes.  Returns the
// warp's contribution to the tile digest in every lane.
__device__ __forceinline__ uint32_t warp_place(const Smem& S, uint32_t digest, uint32_t warp, uint32_t lane)
{
    uint32_t v = 0;
    if (lane < 8) v = S.NW[(warp * 8 + lane) * 16 + ((digest >> (4 * lane)) & 15u)];
    return __reduce_xor_sync(0xFFFFFFFFu, v);
}

// ---- the same digest with small tables, for kernels that see a few hundred kilobytes ----
// Copying the 144 KiB lane-replicated image costs more than such a kernel's whole work.  Here
// the chain uses one copy of the four byte tables (4 KiB in shared memory, taken from lane 0's
// column of the image; lookups may collide on a bank) and the two once-per-tile steps read the
// nibble tables straight from global memory.  Same result as warp_block_digest + warp_place.
__device__ __forceinline__ void load_small_chain_tables(uint32_t* sG, const Tables* __restrict__ tab)
{
    for (uint32_t i = threadIdx.x; i < 1024; i += blockDim.x) {
        const uint32_t k = i >> 8, b = i & 255u;
        sG[i] = tab->image[((k < 2 ? kImgA01 : kImgA23) + b * 256u + (k & 1u) * 128u) / 4u];
    }
    __syncthreads();
}
__device__ __forceinline__ uint32_t tile_digest_part_small(const uint32_t* sG, const Tables* __restrict__ tab,
                                                           const uint32_t (&w)[kWordsPerLane], uint32_t warp, uint32_t lane)
{
    uint32_t s = 0;
#pragma unroll
    for (int i = 0; i < 15; i++) {
        const uint32_t x = s ^ w[i];
        s = sG[x & 0xFFu] ^ sG[256u + ((x >> 8) & 0xFFu)] ^ sG[512u + ((x >> 16) & 0xFFu)] ^ sG[768u + (x >> 24)];
    }
    const uint32_t x = s ^ w[15];
    uint32_t r = 0;
#pragma unroll
    for (uint32_t n = 0; n < 8; n++)
        r ^= __ldg(&tab->image[(kImgNK + (n / 2u) * 0x1000u + ((x >> (4u * n)) & 15u) * 256u + (n & 1u) * 128u) / 4u + lane]);
    const uint32_t digest = __reduce_xor_sync(0xFFFFFFFFu, r);
    uint32_t v = 0;
    if (lane < 8) v = __ldg(&tab->NW[warp][lane][(digest >> (4 * lane)) & 15u]);
    return __reduce_xor_sync(0xFFFFFFFFu, v);
}

// Generic product of two residues (bitwise; used a handful of times per call).
__device__ __forceinline__ uint32_t mulmod_dev(uint32_t a, uint32_t b, uint32_t poly = kPolyReflected)
{
    uint32_t r = 0;
#pragma unroll 8
    for (int i = 0; i < 32; i++) {
        r ^= b & (0u - (a >> 31));
        a <<= 1;
        b = (b >> 1) ^ (poly & (0u - (b & 1u)));
    }
    return r;
}

// Advance a state over one tile (16384 bytes) with byte tables HT[4][256] (shared or global).
__device__ __forceinline__ uint32_t advance_tile(const uint32_t* HT, uint32_t s)
{
    return HT[s & 0xFF] ^ HT[256 + ((s >> 8) & 0xFF)] ^ HT[512 + ((s >> 16) & 0xFF)] ^ HT[768 + (s >> 24)];
}

__device__ __forceinline__ void st_stream_u32(void* p, uint32_t v)
{
    asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Shifts whose amount may be 32 (the result is then 0, as the hardware's shifts define it; in C
// a shift by the operand's width is undefined).
__device__ __forceinline__ uint32_t shl_clamp(uint32_t v, uint32_t n)
{
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(n));
    return r;
}
__device__ __forceinline__ uint32_t shr_clamp(uint32_t v, uint32_t n)
{
    uint32_t r;
    asm("shr.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(n));
    return r;
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

// ---- bulk (TMA) copies of whole tiles into shared memory, tracked by an mbarrier ----
// Loads that land in registers long before they are used tie up the warp's few scoreboards:
// every later shared-memory or global access that shares one waits for them, so "prefetching
// into registers" serialises instead of overlapping.  A bulk copy is issued by one thread,
// holds no registers while in flight, and its completion is observed on an mbarrier.
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// One 16-byte aligned copy of `bytes` (multiple of 16) from global to shared memory; the
// mbarrier's pending byte count is raised first.  `policy`: an L2 cache policy or 0.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, unsigned long long* bar,
                                          uint64_t policy)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
    if (policy)
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                     ::"r"(d), "l"(gsrc), "r"(bytes), "r"(b), "l"(policy) : "memory");
    else
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(d), "l"(gsrc), "r"(bytes), "r"(b) : "memory");
}

// The same with both shared-memory places given by their 32-bit shared-window addresses.
__device__ __forceinline__ void bulk_load_at(uint32_t d, const void* gsrc, uint32_t bytes, uint32_t b, uint64_t policy)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
    if (policy)
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                     ::"r"(d), "l"(gsrc), "r"(bytes), "r"(b), "l"(policy) : "memory");
    else
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(d), "l"(gsrc), "r"(bytes), "r"(b) : "memory");
}

// The low 32 bits of the GPU's wall clock in nanoseconds (they wrap every 4.29 s).  Every
// device-side wait is bounded by TIME against the call's budget (Geo::wait_ns, two seconds unless
// the caller set another, never more than four), not by a number of polls: a block that shares
// the GPU with other work can be descheduled for a long time, and a poll count says nothing about
// how long that was.  Differences of two readings are taken modulo 2^32, which is exact for
// spans below the wrap.
__device__ __forceinline__ uint32_t now_ns()
{
    uint32_t t;
    asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t));
    return t;
}

// Wait for the phase with the given parity to complete, for at most `budget_ns`.  Returns false
// when the time ran out.  try_wait suspends the thread in hardware until the phase completes or
// the time hint runs out, so a waiting warp does not burn issue slots that the other teams on
// the SM need.  (The waiting loop itself, wait_for_copy, follows the control block's definition.)
__device__ __forceinline__ uint32_t mbar_try(uint32_t bar_s, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar_s), "r"(parity), "r"(200000u) : "memory");
    return done;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// ---- tensor memory as a parking place for tiles in flight ----
// Each SM has 256 KB of tensor memory (128 lanes x 512 columns of 32 bits) next to its shared
// memory.  Nothing here multiplies matrices, so it is free, and it takes exactly the shape of
// what a team has to park: thread i of a warp owns lane 32 * (warp % 4) + i, and one
// instruction moves 16 consecutive columns between that lane and 16 registers.  A tile that has
// been measured waits there for its place in the wire image instead of being fetched again.
// The block allocates all 512 columns once (it is alone on its SM) and must free them before
// it exits.  All of these are warp-wide (.sync.aligned): every lane of the warp executes them.
__device__ __forceinline__ void tmem_alloc_all(uint32_t* smem_result)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_result);
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(a) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free_all(uint32_t taddr)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 registers -> 16 columns of this thread's lane, and back.  A store is waited for when the
// next one is issued (a step later) and once more before the memory is handed back: its data is
// fetched three steps on, with three such waits in between, so nobody stands still for it.
__device__ __forceinline__ void tmem_wait_stores() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_store16(uint32_t taddr, const uint32_t (&w)[16])
{
    tmem_wait_stores();
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 ::"r"(taddr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]),
                   "r"(w[8]), "r"(w[9]), "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15]) : "memory");
}
__device__ __forceinline__ void tmem_load16(uint32_t taddr, uint32_t (&w)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]),
                   "=r"(w[8]), "=r"(w[9]), "=r"(w[10]), "=r"(w[11]), "=r"(w[12]), "=r"(w[13]), "=r"(w[14]), "=r"(w[15])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 16 bytes from global to shared memory without a register in between (both 16-byte aligned;
// past L1).  A thread that has issued some waits for its own with cp_async_wait_all.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// A staged tile's words for this lane: word `lane` of rows 16*warp .. 16*warp+15 (conflict free).
__device__ __forceinline__ void read_staged_words(const unsigned char* stage, uint32_t warp, uint32_t lane,
                                                  uint32_t (&w)[16])
{
    const uint32_t* p = reinterpret_cast<const uint32_t*>(stage) + warp * 512u + lane;
#pragma unroll
    for (int i = 0; i < 16; i++) w[i] = p[i * 32];
}

// (the stage given by its 32-bit shared-window address)
__device__ __forceinline__ void read_staged_words_at(uint32_t stage_s, uint32_t warp, uint32_t lane, uint32_t (&w)[16])
{
    const uint32_t p = stage_s + 4u * (warp * 512u + lane);
    w[0] = lds_now<0>(p);     w[1] = lds_now<128>(p);   w[2] = lds_now<256>(p);   w[3] = lds_now<384>(p);
    w[4] = lds_now<512>(p);   w[5] = lds_now<640>(p);   w[6] = lds_now<768>(p);   w[7] = lds_now<896>(p);
    w[8] = lds_now<1024>(p);  w[9] = lds_now<1152>(p);  w[10] = lds_now<1280>(p); w[11] = lds_now<1408>(p);
    w[12] = lds_now<1536>(p); w[13] = lds_now<1664>(p); w[14] = lds_now<1792>(p); w[15] = lds_now<1920>(p);
}

// One 32-bit word of a tile of `len` (1..16384) real bytes that is right-aligned in a virtual
// tile whose leading 16384 - len bytes are zero (leading zeros do not change a zero-start CRC
// state).  `vb` is the word's byte offset inside the virtual tile.  When `first_in_chunk`, the
// chunk's first four bytes are complemented (the all-ones CRC init).  Rare path (one tile per
// call at most), kept out of line.
__device__ __noinline__ uint32_t guarded_word(const unsigned char* tile, uint32_t len, bool first_in_chunk, uint32_t vb)
{
    const int64_t pad = (int64_t)kTile - (int64_t)len;
    uint32_t word = 0;
    for (int j = 0; j < 4; j++) {
        const int64_t rb = (int64_t)vb + j - pad;
        if (rb >= 0) {
            uint32_t b = tile[rb];
            if (first_in_chunk && rb < 4) b ^= 0xFFu;
            word |= b << (8 * j);
        }
    }
    return word;
}

__device__ __forceinline__ void load_tile_words_guarded(const unsigned char* tile, uint32_t len, bool first_in_chunk,
                                                        uint32_t warp, uint32_t lane, uint32_t (&w)[kWordsPerLane])
{
#pragma unroll
    for (int i = 0; i < 16; i++) w[i] = guarded_word(tile, len, first_in_chunk, (warp * 16 + i) * 128 + lane * 4);
}

// CRC32C of a short run computed byte by byte (chunks shorter than four bytes).
__device__ __forceinline__ uint32_t crc_bytewise(const uint32_t* T0, const unsigned char* p, uint32_t n)
{
    uint32_t crc = 0xFFFFFFFFu;
    for (uint32_t i = 0; i < n; i++) crc = T0[(crc ^ p[i]) & 0xFF] ^ (crc >> 8);
    return ~crc;
}

// Exclusive prefix of `v` over the threads of a 1024-thread block, in thread order, and the
// block's total.  s_part: 33 values of shared memory.  Block-wide (two barriers); one use per
// kernel, or a barrier between uses.  The kernels that scan a per-chunk array give every thread
// a run of consecutive chunks, so one such prefix does for any number of chunks.
template <typename T>
__device__ __forceinline__ T block_prefix(T v, T* s_part, T& total)
{
    const uint32_t lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    T incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= (uint32_t)d) incl += o;
    }
    if (lane == 31) s_part[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const T p = s_part[lane];
        T pi = p;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const T o = __shfl_up_sync(0xFFFFFFFFu, pi, d);
            if (lane >= (uint32_t)d) pi += o;
        }
        s_part[lane] = pi - p;
        if (lane == 31) s_part[32] = pi;
    }
    __syncthreads();
    total = s_part[32];
    return s_part[warp] + incl - v;
}

}  // namespace wm
