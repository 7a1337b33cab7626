// CUDA kernels (sm_100a) and C ABI of the session mover's data path.
//
// Kernel map (every call enqueues a short chain on the caller's stream, no host sync):
//   wm_checksum      : k_tile_digests -> k_checksum_finish
//   wm_dirty_diff    : k_diff_init -> k_diff -> k_diff_compact
//   wm_encode        : k_encode_init -> k_encode (single pass; teams publish tile lengths, one
//                      scanner warp turns them into payload offsets) -> k_encode_finish (directory, cache CRC, header)
//                      -> k_meta_crc (metadata CRC, result)
//   wm_decode_verify : k_decode_init -> k_decode_check (header, metadata CRC, structure: the gate)
//                      -> k_decode (unpack + CRC of decoded bytes) -> k_decode_finish
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>
#include <type_traits>

#include <cuda_runtime.h>

#include "../../include/wm.h"
#include "wm_device.cuh"

// The kernels, one file per call (a single translation unit: the host side below launches them).
#include "wm_layout.cuh"
#include "wm_checksum.cuh"
#include "wm_diff.cuh"
#include "wm_leaves.cuh"
#include "wm_encode.cuh"
#include "wm_meta.cuh"
#include "wm_decode.cuh"
#include "wm_xxh64.cuh"

// Scratch and tables of wm_checksum_noalloc live in the library image itself: two file-scope
// __device__ arrays that every GPU loading the library carries until the process exits.  In host
// code their names are host-side stand-ins, not device addresses, so the addresses are asked for
// with cudaGetSymbolAddress (with the device in question current) and only those go to kernels.
static __device__ __align__(256) unsigned char g_na_scratch[WM_NOALLOC_SCRATCH_BYTES];
static __device__ __align__(256) unsigned char g_na_tables[sizeof(wm::Tables)];

namespace wm {

// ------------------------------------------------------------------ host side

constexpr int kTeams = 4;        // encode: teams per block (plus the scanner warp)
constexpr int kTeamsPlain = 4;   // checksum / decode: teams per block

struct DeviceState {
    Tables* tables = nullptr;
    Tables* tables_zlib = nullptr;   // built on the first wm_checksum_poly call that asks for it
    int sm_count = 0;
    bool ready = false;
    cudaEvent_t ev[4][2] = {};   // optional timing of the four main kernels
};
// Process-wide switches: read by calls on any thread, so they are atomics (a call sees the value at
// the moment it is issued; calls that must not depend on them take their options as an argument).
static std::atomic<bool> g_timing{false};
static std::atomic<bool> g_zero_tiles{false};   // wm_zero_tiles_enable
static std::atomic<bool> g_entropy{false};      // wm_entropy_enable

struct MainKernelTimer {        // records events around a main kernel when timing is enabled
    const DeviceState* ds; int kind; cudaStream_t s; bool on;
    MainKernelTimer(const DeviceState* d, int k, cudaStream_t st) : ds(d), kind(k), s(st)
    {
        on = g_timing.load(std::memory_order_relaxed);
        if (on) cudaEventRecord(ds->ev[kind][0], s);
    }
    ~MainKernelTimer()
    {
        if (on) cudaEventRecord(ds->ev[kind][1], s);
    }
};
static DeviceState g_dev[64];
static std::mutex g_mutex;
static thread_local uint32_t g_launches = 0;

static const DeviceState* device_state()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& s = g_dev[dev];
    if (s.ready) return &s;
    static Tables host;
    build_tables(host);
    if (cudaMalloc(&s.tables, sizeof(Tables)) != cudaSuccess) return nullptr;
    if (cudaMemcpy(s.tables, &host, sizeof(Tables), cudaMemcpyHostToDevice) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    const int big = kDynSmem;
    {
        const void* enc[] = {(const void*)k_encode<kTeams, false, false, false>, (const void*)k_encode<kTeams, true, false, false>,
                             (const void*)k_encode<kTeams, false, true, false>,  (const void*)k_encode<kTeams, true, true, false>,
                             (const void*)k_encode<kTeams, false, false, true>,  (const void*)k_encode<kTeams, true, false, true>,
                             (const void*)k_encode<kTeams, false, true, true>,   (const void*)k_encode<kTeams, true, true, true>,
                             (const void*)k_encode<kTeams, false, false, false, true>, (const void*)k_encode<kTeams, true, false, false, true>,
                             (const void*)k_encode<kTeams, false, true, false, true>,  (const void*)k_encode<kTeams, true, true, false, true>,
                             (const void*)k_encode<kTeams, false, false, true, true>,  (const void*)k_encode<kTeams, true, false, true, true>,
                             (const void*)k_encode<kTeams, false, true, true, true>,   (const void*)k_encode<kTeams, true, true, true, true>};
        for (const void* f : enc)
            if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    }
    {
        const void* dec[] = {(const void*)k_decode<kTeamsPlain, false, 0>, (const void*)k_decode<kTeamsPlain, true, 0>,
                             (const void*)k_decode<kTeamsPlain, false, 1>, (const void*)k_decode<kTeamsPlain, true, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 2>, (const void*)k_decode<kTeamsPlain, true, 2>,
                             (const void*)k_decode<kTeamsPlain, false, 0, 1>, (const void*)k_decode<kTeamsPlain, true, 0, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 1, 1>, (const void*)k_decode<kTeamsPlain, true, 1, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 2, 1>, (const void*)k_decode<kTeamsPlain, true, 2, 1>,
                             (const void*)k_decode<kTeamsPlain, false, 0, 2>, (const void*)k_decode<kTeamsPlain, true, 0, 2>,
                             (const void*)k_decode<kTeamsPlain, false, 1, 2>, (const void*)k_decode<kTeamsPlain, true, 1, 2>,
                             (const void*)k_decode<kTeamsPlain, false, 2, 2>, (const void*)k_decode<kTeamsPlain, true, 2, 2>};
        for (const void* f : dec)
            if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    }
    if (cudaFuncSetAttribute(k_tile_digests<kTeamsPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    if (cudaFuncSetAttribute(k_meta_crc, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess) return nullptr;
    for (int k = 0; k < 4; k++)
        for (int j = 0; j < 2; j++)
            if (cudaEventCreate(&s.ev[k][j]) != cudaSuccess) return nullptr;
    s.ready = true;
    return &s;
}

// Launch a kernel that may start before the kernel enqueued just before it on the stream has
// finished (it waits inside, see grid_dep_wait).
template <typename... Params, typename... Args>
static void launch_after(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static wm_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? WM_OK : WM_ERR_CUDA;
}

}  // namespace wm

using namespace wm;

extern "C" {

uint64_t wm_num_chunks(uint64_t nbytes, uint32_t chunk_bytes)
{
    return chunk_bytes ? (nbytes + chunk_bytes - 1) / chunk_bytes : 0;
}

uint64_t wm_num_tiles(uint64_t nbytes) { return (nbytes + kTile - 1) / kTile; }

uint64_t wm_meta_bytes(uint64_t nbytes, uint32_t chunk_bytes)
{
    return (64ull + 16ull * wm_num_chunks(nbytes, chunk_bytes) + 2ull * wm_num_tiles(nbytes) + 31ull) & ~31ull;
}

uint64_t wm_wire_bound(uint64_t nbytes, uint32_t chunk_bytes) { return wm_meta_bytes(nbytes, chunk_bytes) + nbytes; }

uint64_t wm_workspace_bytes(uint64_t nbytes, uint32_t chunk_bytes)
{
    Geo g;
    if (!make_geo(nbytes, chunk_bytes, g)) return 0;
    return ws_layout(g).total;
}

uint32_t wm_last_launch_count(void) { return g_launches; }

void wm_timing_enable(int on) { g_timing = on != 0; }

void wm_zero_tiles_enable(int on) { g_zero_tiles = on != 0; }
void wm_entropy_enable(int on) { g_entropy = on != 0; }

void wm_wait_budget_ms(uint32_t ms) { g_wait_ns = (ms == 0u ? 1u : ms > 4000u ? 4000u : ms) * 1000000u; }
void wm_inject_stall(int on) { g_inject = on ? (kInjectNoScanner | kInjectNoCopy) : 0u; }

wm_status wm_workspace_status(const void* workspace, void* stream)
{
    const Ctrl* ctrl = static_cast<const Ctrl*>(workspace);
    if (!ctrl) {                       // the built-in scratch of wm_checksum_noalloc on the current device
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_na_scratch) != cudaSuccess || !p) return WM_ERR_CUDA;
        ctrl = static_cast<const Ctrl*>(p);
    }
    uint32_t err = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&err, &ctrl->err, sizeof err, cudaMemcpyDeviceToHost, s) != cudaSuccess) return WM_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return WM_ERR_CUDA;
    return (err & 8u) ? WM_ERR_ARG : (err & 4u) ? WM_ERR_CUDA : (err & 2u) ? WM_ERR_TIMEOUT : (err & 1u) ? WM_ERR_CAPACITY : WM_OK;
}

int wm_timing_read_ms(int kind, float* ms)
{
    const DeviceState* ds = device_state();
    if (!ds || kind < 0 || kind > 3 || !ms) return WM_ERR_ARG;
    if (cudaEventSynchronize(ds->ev[kind][1]) != cudaSuccess) return WM_ERR_CUDA;
    return cudaEventElapsedTime(ms, ds->ev[kind][0], ds->ev[kind][1]) == cudaSuccess ? WM_OK : WM_ERR_CUDA;
}

wm_status wm_checksum(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, uint32_t* crc_out,
                      void* workspace, uint64_t workspace_bytes, void* stream)
{
    Geo g;
    if (!cache || !crc_out || !workspace || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (!aligned16(cache) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    const uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    // the control block starts at zero: the error word in it is this call's outcome (wm_workspace_status)
    if (cudaMemsetAsync(ws.ctrl, 0, sizeof(Ctrl), s) != cudaSuccess) return WM_ERR_CUDA;
    {
        MainKernelTimer timer(ds, 0, s);
        k_tile_digests<kTeamsPlain><<<grid, kTeamsPlain * 256, kDynSmem, s>>>(c, g, ws, ds->tables);
    }
    launch_after(k_checksum_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, ws, ds->tables, crc_out);
    g_launches = 2;
    return launch_status();
}

// The checksum call with the polynomial as an argument.  The tile kernel and the finish kernel
// are the ones wm_checksum runs: the polynomial lives in the tables and in the geometry's powers.
static const Tables* zlib_tables()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& s = g_dev[dev];
    if (s.tables_zlib) return s.tables_zlib;
    static Tables host;
    build_tables(host, kPolyZlib);
    Tables* p = nullptr;
    if (cudaMalloc(&p, sizeof(Tables)) != cudaSuccess) return nullptr;
    if (cudaMemcpy(p, &host, sizeof(Tables), cudaMemcpyHostToDevice) != cudaSuccess) { cudaFree(p); return nullptr; }
    s.tables_zlib = p;
    return p;
}

wm_status wm_checksum_poly(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, int polynomial, uint32_t* crc_out,
                           void* workspace, uint64_t workspace_bytes, void* stream)
{
    if (polynomial == WM_POLY_CRC32C) return wm_checksum(cache, nbytes, chunk_bytes, crc_out, workspace, workspace_bytes, stream);
    if (polynomial != WM_POLY_ZLIB) return WM_ERR_ARG;
    Geo g;
    if (!cache || !crc_out || !workspace || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (!aligned16(cache) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    const Tables* tab = zlib_tables();
    if (!tab) return WM_ERR_CUDA;
    g.poly = kPolyZlib;
    g.k_tail = x_pow_bytes(g.tail_len, kPolyZlib);
    g.k_chunk = x_pow_bytes(g.chunk_bytes, kPolyZlib);
    g.k_last_chunk = x_pow_bytes(g.last_chunk_len, kPolyZlib);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    const uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    // the control block starts at zero: the error word in it is this call's outcome (wm_workspace_status)
    if (cudaMemsetAsync(ws.ctrl, 0, sizeof(Ctrl), s) != cudaSuccess) return WM_ERR_CUDA;
    {
        MainKernelTimer timer(ds, 0, s);
        k_tile_digests<kTeamsPlain><<<grid, kTeamsPlain * 256, kDynSmem, s>>>(c, g, ws, tab);
    }
    launch_after(k_checksum_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, ws, tab, crc_out);
    g_launches = 2;
    return launch_status();
}

// XXH64 of every chunk: one kernel, no workspace, no tables.
wm_status wm_checksum_xxh64(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, uint64_t seed, uint64_t* hash_out,
                            void* stream)
{
    Geo g;
    if (!cache || !hash_out || !make_geo(nbytes, chunk_bytes, g) || !aligned16(cache)) return WM_ERR_ARG;
    if (!device_state()) return WM_ERR_CUDA;
    const uint32_t threads = 4u * g.n_chunks;
    k_xxh64<<<(threads + 31u) / 32u, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const unsigned char*>(cache), nbytes, chunk_bytes, g.n_chunks, seed,
        reinterpret_cast<unsigned long long*>(hash_out));
    g_launches = 1;
    return launch_status();
}

// ---- wm_checksum_noalloc: the checksum call for callers that must not allocate -------------
// (scratch and tables: the two file-scope __device__ arrays declared at the top of this file)

namespace wm {
struct NoAllocState {
    unsigned char* scratch = nullptr;
    Tables* tables = nullptr;
    int sm_count = 0;
    bool ready = false;
};
static NoAllocState g_na[64];

static const NoAllocState* noalloc_state()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    NoAllocState& s = g_na[dev];
    if (s.ready) return &s;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_na_scratch) != cudaSuccess || !p) return nullptr;
    s.scratch = static_cast<unsigned char*>(p);
    p = nullptr;
    if (cudaGetSymbolAddress(&p, g_na_tables) != cudaSuccess || !p) return nullptr;
    s.tables = static_cast<Tables*>(p);
    static Tables host;                          // static storage: no heap, no device allocation
    build_tables(host);
    if (cudaMemcpy(s.tables, &host, sizeof(Tables), cudaMemcpyHostToDevice) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    if (cudaFuncSetAttribute(k_tile_digests<kTeamsPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem)
        != cudaSuccess)
        return nullptr;
    s.ready = true;
    return &s;
}
}  // namespace wm

wm_status wm_checksum_noalloc(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, uint32_t* crc_out, void* stream)
{
    Geo g;
    if (!cache || !crc_out || !make_geo(nbytes, chunk_bytes, g) || !aligned16(cache)) return WM_ERR_ARG;
    if (nbytes > WM_NOALLOC_MAX_BYTES) return WM_ERR_ARG;          // the built-in scratch holds no more
    const NoAllocState* ns = noalloc_state();
    if (!ns) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // scratch: a control block, then one 32-bit digest per tile
    static_assert(WM_NOALLOC_SCRATCH_BYTES >= sizeof(Ctrl) + 4ull * (WM_NOALLOC_MAX_BYTES / WM_TILE_BYTES + 1),
                  "built-in scratch covers the stated maximum");
    Ws ws;
    memset(&ws, 0, sizeof ws);
    ws.ctrl = reinterpret_cast<Ctrl*>(ns->scratch);
    ws.dig = reinterpret_cast<uint32_t*>(ns->scratch + sizeof(Ctrl));
    // the array keeps the last call's contents; only the control block has to start at zero
    if (cudaMemsetAsync(ns->scratch, 0, sizeof(Ctrl), s) != cudaSuccess) return WM_ERR_CUDA;
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    const uint32_t grid = need < (uint32_t)ns->sm_count ? need : (uint32_t)ns->sm_count;
    k_tile_digests<kTeamsPlain><<<grid, kTeamsPlain * 256, kDynSmem, s>>>(c, g, ws, ns->tables);
    launch_after(k_checksum_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, ws, ns->tables, crc_out);
    g_launches = 2;
    return launch_status();
}

wm_status wm_dirty_diff(const void* cache, const void* prev, uint64_t nbytes, uint32_t chunk_bytes,
                        uint8_t* dirty_out, uint32_t* dirty_idx_out, uint32_t* n_dirty_out,
                        void* workspace, uint64_t workspace_bytes, void* stream)
{
    Geo g;
    if (!cache || !prev || !dirty_out || !n_dirty_out || !workspace || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (!aligned16(cache) || !aligned16(prev) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    k_diff_init<<<1, 32, 0, s>>>(ws);
    const uint32_t want = (uint32_t)ds->sm_count * 4;
    const uint32_t grid = g.n_chunks < want ? g.n_chunks : want;
    {
        MainKernelTimer timer(ds, 1, s);
        launch_after(k_diff, grid, 256, 0, s, static_cast<const unsigned char*>(cache), static_cast<const unsigned char*>(prev), g, ws, dirty_out);
    }
    launch_after(k_diff_compact, 1, 1024, 0, s, g, dirty_out, dirty_idx_out, n_dirty_out);
    g_launches = 3;
    return launch_status();
}

// Both forms of the encode call: a flat cache (leaves == nullptr) or a table of leaves.
// The options the plain calls use: the process-wide switches.
static uint32_t default_options()
{
    return (g_zero_tiles ? WM_OPT_ZERO_TILES : 0u) | (g_entropy ? WM_OPT_ENTROPY : 0u);
}

static wm_status encode_any(const void* cache, const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes,
                            const uint8_t* dirty, uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace,
                            uint64_t workspace_bytes, wm_result* result, void* stream, uint32_t options)
{
    Geo g;
    if (options & ~(WM_OPT_ZERO_TILES | WM_OPT_ENTROPY | WM_OPT_BLOCKS_MASK)) return WM_ERR_ARG;
    const uint32_t block_cap = (options & WM_OPT_BLOCKS_MASK) >> 8;       // 0: every SM
    if (block_cap == 1u) return WM_ERR_ARG;                               // one block scans, at least one encodes
    const bool opt_ent = (options & WM_OPT_ENTROPY) != 0, opt_zero = (options & WM_OPT_ZERO_TILES) != 0;
    if (!crc_inout || !wire || !workspace || !result || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (leaves ? (n_leaves == 0 || n_leaves > kMaxLeaves) : (!cache || !aligned16(cache))) return WM_ERR_ARG;
    if (!aligned16(wire) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total || wire_cap < g.meta_end)
        return WM_ERR_ARG;
    if (nbytes > kMaxCodecBytes) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* c = static_cast<const unsigned char*>(cache);
    unsigned char* w = static_cast<unsigned char*>(wire);
    const uint32_t init_blocks = (g.n_tiles + 1023) / 1024 < 1024 ? (g.n_tiles + 1023) / 1024 : 1024;
    k_encode_init<<<init_blocks ? init_blocks : 1, 1024, 0, s>>>(g, ws, w, dirty);
    if (leaves) {
        const uint32_t map_blocks = (g.n_tiles + 4095) / 4096 < 64 ? (g.n_tiles + 4095) / 4096 : 64;
        launch_after(k_leaf_map, map_blocks ? map_blocks : 1, 1024, 0, s, leaves, n_leaves, g, ws, result, 0);
        launch_after(k_leaf_gather, 1024, 256, 0, s, leaves, n_leaves, g, ws);
    }
    // one block per SM: one of them scans, the others encode
    // (tiles are claimed by ticket, so any number of blocks gives the same image; a caller that
    // shares the GPU with other work caps it)
    const uint32_t need = (g.n_tiles + kTeams - 1) / kTeams + 1;
    uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    if (block_cap && grid > block_cap) grid = block_cap;
    {
        MainKernelTimer timer(ds, 2, s);
        const int variant = (dirty ? 1 : 0) | (leaves ? 2 : 0) | (opt_zero ? 4 : 0) | (opt_ent ? 8 : 0);
        auto go = [&](auto kernel) { launch_after(kernel, grid, kTeams * 256, kDynSmem, s, c, g, dirty, w, wire_cap, ws, ds->tables); };
        switch (variant) {
            case 0: go(k_encode<kTeams, false, false, false>); break;
            case 1: go(k_encode<kTeams, true, false, false>); break;
            case 2: go(k_encode<kTeams, false, true, false>); break;
            case 3: go(k_encode<kTeams, true, true, false>); break;
            case 4: go(k_encode<kTeams, false, false, true>); break;
            case 5: go(k_encode<kTeams, true, false, true>); break;
            case 6: go(k_encode<kTeams, false, true, true>); break;
            case 7: go(k_encode<kTeams, true, true, true>); break;
            case 8: go(k_encode<kTeams, false, false, false, true>); break;
            case 9: go(k_encode<kTeams, true, false, false, true>); break;
            case 10: go(k_encode<kTeams, false, true, false, true>); break;
            case 11: go(k_encode<kTeams, true, true, false, true>); break;
            case 12: go(k_encode<kTeams, false, false, true, true>); break;
            case 13: go(k_encode<kTeams, true, false, true, true>); break;
            case 14: go(k_encode<kTeams, false, true, true, true>); break;
            default: go(k_encode<kTeams, true, true, true, true>); break;
        }
    }
    launch_after(k_encode_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, c, g, dirty, crc_inout, w, ws, ds->tables,
                 chunk_powers(g), (opt_ent ? 4u : 0u) | (opt_zero ? 2u : 0u));
    launch_after(k_meta_crc, (g.n_meta_slices + 3) / 4, 1024, kDynSmem, s, w, g, ws, ds->tables, result);
    g_launches = leaves ? 6 : 4;
    return launch_status();
}

wm_status wm_encode(const void* cache, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
                    uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace, uint64_t workspace_bytes,
                    wm_result* result, void* stream)
{
    if (!cache) return WM_ERR_ARG;
    return encode_any(cache, nullptr, 0, nbytes, chunk_bytes, dirty, crc_inout, wire, wire_cap, workspace, workspace_bytes, result, stream,
                      default_options());
}

wm_status wm_encode_leaves(const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes, const uint8_t* dirty,
                           uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace, uint64_t workspace_bytes,
                           wm_result* result, void* stream)
{
    if (!leaves) return WM_ERR_ARG;
    return encode_any(nullptr, leaves, n_leaves, nbytes, chunk_bytes, dirty, crc_inout, wire, wire_cap, workspace, workspace_bytes, result, stream,
                      default_options());
}

// Both forms of the decode call: a flat shadow buffer (leaves == nullptr) or a table of leaves.
// strict: nothing is stored until every check has passed (two passes over the wire image).
static wm_status decode_any(const void* wire, uint64_t wire_len, void* dst, const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes,
                            uint32_t chunk_bytes, uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes,
                            wm_result* result, void* stream, uint32_t options)
{
    Geo g;
    if (options & ~(WM_OPT_ZERO_TILES | WM_OPT_ENTROPY | WM_OPT_STRICT | WM_OPT_BLOCKS_MASK)) return WM_ERR_ARG;
    const uint32_t block_cap = (options & WM_OPT_BLOCKS_MASK) >> 8;       // 0: every SM
    const bool strict = (options & WM_OPT_STRICT) != 0;
    if (!wire || !dst_crc_inout || !workspace || !result || !make_geo(nbytes, chunk_bytes, g)) return WM_ERR_ARG;
    if (leaves ? (n_leaves == 0 || n_leaves > kMaxLeaves) : (!dst || !aligned16(dst))) return WM_ERR_ARG;
    if (!aligned16(wire) || !aligned16(workspace) || workspace_bytes < ws_layout(g).total) return WM_ERR_ARG;
    if (nbytes > kMaxCodecBytes) return WM_ERR_ARG;
    const DeviceState* ds = device_state();
    if (!ds) return WM_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Ws ws = ws_carve(workspace, g);
    const unsigned char* w = static_cast<const unsigned char*>(wire);
    unsigned char* d = static_cast<unsigned char*>(dst);
    k_decode_init<<<1, 64, 0, s>>>(ws);
    if (leaves) {
        const uint32_t map_blocks = (g.n_tiles + 4095) / 4096 < 64 ? (g.n_tiles + 4095) / 4096 : 64;
        launch_after(k_leaf_map, map_blocks ? map_blocks : 1, 1024, 0, s, leaves, n_leaves, g, ws, result, 1);
    }
    // a wire shorter than the metadata is rejected by the header check before anything else is read
    const uint32_t meta_blocks = (g.n_meta_slices + 3) / 4;
    const uint32_t chunks_per_block = 32u * check_chunks_per_warp(g.tiles_per_chunk);
    const bool ent = (options & WM_OPT_ENTROPY) != 0;      // the option says which kind of image the call expects
    launch_after(k_decode_check, meta_blocks + (g.n_chunks + chunks_per_block - 1) / chunks_per_block, 1024, 0, s, w, wire_len, g, ws, ds->tables, result, meta_blocks,
                 ent ? 1u : 0u);
    const uint32_t need = (g.n_tiles + kTeamsPlain - 1) / kTeamsPlain;
    uint32_t grid = need < (uint32_t)ds->sm_count ? need : (uint32_t)ds->sm_count;
    if (block_cap && grid > block_cap) grid = block_cap;
    auto pass = [&](auto flat_kernel, auto leaf_kernel) {
        if (leaves) launch_after(leaf_kernel, grid, kTeamsPlain * 256, kDynSmem, s, w, g, d, ws, ds->tables);
        else launch_after(flat_kernel, grid, kTeamsPlain * 256, kDynSmem, s, w, g, d, ws, ds->tables);
    };
    {
        MainKernelTimer timer(ds, 3, s);
        if (ent) {       // one of the two applies (ENT tiles only, or ENT and PACK tiles); the other returns at once
            if (strict) { pass(k_decode<kTeamsPlain, false, 1, 1>, k_decode<kTeamsPlain, true, 1, 1>); pass(k_decode<kTeamsPlain, false, 1, 2>, k_decode<kTeamsPlain, true, 1, 2>); }
            else { pass(k_decode<kTeamsPlain, false, 0, 1>, k_decode<kTeamsPlain, true, 0, 1>); pass(k_decode<kTeamsPlain, false, 0, 2>, k_decode<kTeamsPlain, true, 0, 2>); }
        } else {
            if (strict) pass(k_decode<kTeamsPlain, false, 1>, k_decode<kTeamsPlain, true, 1>);
            else pass(k_decode<kTeamsPlain, false, 0>, k_decode<kTeamsPlain, true, 0>);
        }
    }
    // leaf mode: the tiles that crossed leaf boundaries were decoded into the side buffer; they
    // go to their leaves behind the kernel that stores
    if (leaves && !strict) launch_after(k_leaf_scatter, 1024, 256, 0, s, leaves, n_leaves, g, ws);
    launch_after(k_decode_finish, (g.n_chunks + g.finish_cb - 1) / g.finish_cb, 1024, 0, s, w, wire_len, g, d, dst_crc_inout, ws, ds->tables,
                 result, chunk_powers(g), strict ? 1u : 0u);
    if (strict) {
        if (ent) { pass(k_decode<kTeamsPlain, false, 2, 1>, k_decode<kTeamsPlain, true, 2, 1>); pass(k_decode<kTeamsPlain, false, 2, 2>, k_decode<kTeamsPlain, true, 2, 2>); }
        else pass(k_decode<kTeamsPlain, false, 2>, k_decode<kTeamsPlain, true, 2>);
        if (leaves) launch_after(k_leaf_scatter, 1024, 256, 0, s, leaves, n_leaves, g, ws);
    }
    g_launches = (leaves ? 6 : 4) + (strict ? 1 : 0) + (ent ? (strict ? 2 : 1) : 0);
    return launch_status();
}

wm_status wm_decode_verify(const void* wire, uint64_t wire_len, void* dst, uint64_t nbytes, uint32_t chunk_bytes,
                           uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes, wm_result* result,
                           void* stream)
{
    if (!dst) return WM_ERR_ARG;
    return decode_any(wire, wire_len, dst, nullptr, 0, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result, stream,
                      default_options());
}

wm_status wm_decode_verify_strict(const void* wire, uint64_t wire_len, void* dst, uint64_t nbytes, uint32_t chunk_bytes,
                                  uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes, wm_result* result,
                                  void* stream)
{
    if (!dst) return WM_ERR_ARG;
    return decode_any(wire, wire_len, dst, nullptr, 0, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result, stream,
                      default_options() | WM_OPT_STRICT);
}

wm_status wm_decode_verify_leaves(const void* wire, uint64_t wire_len, const wm_leaf* dst_leaves, uint32_t n_leaves, uint64_t nbytes,
                                  uint32_t chunk_bytes, uint32_t* dst_crc_inout, void* workspace, uint64_t workspace_bytes,
                                  wm_result* result, void* stream)
{
    if (!dst_leaves) return WM_ERR_ARG;
    return decode_any(wire, wire_len, nullptr, dst_leaves, n_leaves, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result,
                      stream, default_options());
}

// The calls with their options as an argument (nothing process-wide is read): a cache as one
// buffer (leaves == NULL) or as a table of leaves (cache / dst == NULL).
wm_status wm_encode_opt(const void* cache, const wm_leaf* leaves, uint32_t n_leaves, uint64_t nbytes, uint32_t chunk_bytes,
                        const uint8_t* dirty, uint32_t* crc_inout, void* wire, uint64_t wire_cap, void* workspace,
                        uint64_t workspace_bytes, uint32_t options, wm_result* result, void* stream)
{
    if ((cache != nullptr) == (leaves != nullptr)) return WM_ERR_ARG;
    return encode_any(cache, leaves, n_leaves, nbytes, chunk_bytes, dirty, crc_inout, wire, wire_cap, workspace, workspace_bytes, result, stream,
                      options);
}

wm_status wm_decode_verify_opt(const void* wire, uint64_t wire_len, void* dst, const wm_leaf* dst_leaves, uint32_t n_leaves,
                               uint64_t nbytes, uint32_t chunk_bytes, uint32_t* dst_crc_inout, void* workspace,
                               uint64_t workspace_bytes, uint32_t options, wm_result* result, void* stream)
{
    if ((dst != nullptr) == (dst_leaves != nullptr)) return WM_ERR_ARG;
    return decode_any(wire, wire_len, dst, dst_leaves, n_leaves, nbytes, chunk_bytes, dst_crc_inout, workspace, workspace_bytes, result, stream,
                      options);
}

}  // extern "C"
