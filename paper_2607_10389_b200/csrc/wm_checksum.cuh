// wm_checksum: per-tile digests (k_tile_digests) and their fold into chunk CRCs (k_checksum_finish).
// Part of the one translation unit wm_kernels.cu (included there, in this order).
#pragma once

namespace wm {

// ------------------------------------------------------------------ wm_checksum

// Tile digests of the whole cache: static striding over tiles.  Each team owns one 16 KiB stage
// that bulk copies (TMA) fill; the team takes its 16 words per lane out of the stage, hands
// the stage to the copy of its next tile and digests from registers meanwhile.
struct DigTeamCtl {
    uint32_t wdig[2][8];
    unsigned long long mbar;
    unsigned long long pad;
};
static_assert(sizeof(DigTeamCtl) % 16 == 0, "team control block keeps 16-byte alignment");

template <int TEAMS>
__global__ void __launch_bounds__(TEAMS * 256, 1)
k_tile_digests(const unsigned char* __restrict__ cache, Geo g, Ws ws, const Tables* __restrict__ tab)
{
    grid_dep_launch();
    extern __shared__ __align__(16) unsigned char smem[];
    Smem S = setup_smem(smem, tab);
    const uint32_t team = threadIdx.x / kTeamThreads, tt = threadIdx.x % kTeamThreads;
    const uint32_t warp = tt / 32, lane = tt % 32;
    unsigned char* stage = nullptr;
    for (int i = 0; i < TEAMS; i++) {          // every thread carves the same blocks in the same order
        unsigned char* p = S.take(kTile);
        if ((uint32_t)i == team) stage = p;
    }
    DigTeamCtl* tc = reinterpret_cast<DigTeamCtl*>(S.take(TEAMS * sizeof(DigTeamCtl)));
    if (!S.ok) { if (threadIdx.x == 0) atomicOr(&ws.ctrl->err, 4u); return; }
    tc += team;
    const uint64_t stride = (uint64_t)gridDim.x * TEAMS;
    const uint64_t pol = l2_policy_evict_first();
    auto full = [&](uint64_t tile) { return tile < g.n_tiles && g.nbytes - tile * kTile >= kTile; };
    auto start_copy = [&](uint64_t tile) {     // one thread of the team
        if (full(tile) && !(g.inject & kInjectNoCopy)) bulk_load(stage, cache + tile * kTile, kTile, &tc->mbar, pol);
    };

    uint64_t t = (uint64_t)blockIdx.x * TEAMS + team;
    if (tt == 64u) { mbar_init(&tc->mbar, 1); start_copy(t); }
    team_bar(team);
    uint32_t phase = 0, par = 0;
    uint64_t t_done = ~0ull;                     // tile whose digest parts wait in wdig[par ^ 1]
    // One team barrier per tile.  The single-lane chores sit on different warps (the team waits
    // for whichever warp has the most to do): warp 2 starts the next copy, warp 1 folds and
    // stores the previous tile's digest once the barrier has made its parts complete.
    for (; t < g.n_tiles; t += stride) {
        const bool first = first_in_chunk(g, (uint32_t)t);
        uint32_t d[kWordsPerLane];
        bool fold = first;
        if (full(t)) {
            wait_for_copy<false>(&tc->mbar, phase, g.wait_ns, ws.ctrl, (g.inject & kInjectNoCopy) != 0u);
            phase ^= 1u;
            read_staged_words(stage, warp, lane, d);
        } else {
            load_tile_words_guarded(cache + t * kTile, (uint32_t)(g.nbytes - t * kTile), first, warp, lane, d);
            fold = false;
        }
        team_bar(team);                          // stage free; the previous tile's digest parts complete
        if (tt == 64u) start_copy(t + stride);
        if (tt == 32u && t_done != ~0ull) ws.dig[t_done] = xor8(tc->wdig[par ^ 1u]);
        const uint32_t v = tile_digest_part(S, d, fold, warp, lane);
        if (lane == 0) tc->wdig[par][warp] = v;
        t_done = t;
        par ^= 1u;
    }
    team_bar(team);
    if (tt == 32u && t_done != ~0ull) ws.dig[t_done] = xor8(tc->wdig[par ^ 1u]);
}

__global__ void __launch_bounds__(1024)
k_checksum_finish(const unsigned char* __restrict__ cache, Geo g, Ws ws, const Tables* __restrict__ tab,
                  uint32_t* __restrict__ crc_out)
{
    __shared__ uint32_t sHT[1024];
    __shared__ uint32_t sT0[256];
    __shared__ FinishStage stage;
    load_ht_t0(sHT, sT0, tab);
    grid_dep_wait();
    const uint32_t c0 = blockIdx.x * g.finish_cb;
    stage_chunk_digests(g, stage, ws.dig, c0);
    const uint32_t c = c0 + threadIdx.x;
    // Fail closed: when the digest kernel reported trouble (a wait that ran out, no room for its
    // stages) some digests are not those of the cache.  The vector is then zero-filled and the
    // control block keeps the reason for wm_workspace_status.
    const bool failed = ld_volatile_u32(&ws.ctrl->err) != 0u;
    if (threadIdx.x < g.finish_cb && c < g.n_chunks)
        crc_out[c] = failed ? 0u : chunk_crc_staged(g, sHT, sT0, stage, ws.dig, cache + (uint64_t)c * g.chunk_bytes, c, threadIdx.x);
}

}  // namespace wm
