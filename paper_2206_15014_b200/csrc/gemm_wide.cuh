// Wide CTA-pair kernel for 2:4 int8 weights with a long reduction (weights streamed through the stage ring).
//
// A pair tile is 512 output channels x BN tokens: each CTA of the pair owns 256 channels, as two blocks of
// 128 TMEM lanes with one accumulator each (columns [0, BN) and [BN, 2 BN)), and stages half of the X tile.
// Against the 256 x 192 tile of nm_gemm_pair_kernel every staged byte of X feeds twice as many MACs: per
// MAC the kernel moves 0.64x the bytes through L2 and through each SM's shared memory, issues half as many
// TMA loads and barrier operations, and one pipeline stage (128 reduction elements: 16 KB of weights + BN/2
// x 128 B of X) carries 448 tensor-core clocks of work at BN = 224 instead of 384 for a 40 KB stage.
//
// What changes with two accumulators of BN columns each in the 512 TMEM columns:
//   * The 2:4 index metadata can no longer stay resident for the whole reduction.  Four metadata warps (one
//     per TMEM lane quarter, both CTAs) copy the 16 bytes per weight row and block that a stage needs from
//     the canonical metadata in global memory into a ring of TMEM slots (8 columns per stage, same slot
//     index as the shared-memory stage) with tcgen05.st; the stage's "full" barrier also counts them.
//   * The accumulators are single-buffered.  The MMA thread runs block 1 SKEW stages behind block 0, so that
//     block 0's accumulator is handed to its four epilogue warps SKEW stages before block 1's and the next
//     tile's block-0 MMAs can start while block 1's accumulator is still being read.
//   * The MMA thread's instruction stream is kept short: descriptors are advanced with one add from values
//     formed once, ring positions are carried instead of divided out (a single thread's dependent
//     instructions cost several clocks each; 4 MMAs + commit took ~430 clocks in the 256 x 192 kernel).
#pragma once

namespace nm {

constexpr int kWideEpiWarps = 8;     // four per accumulator, one per TMEM lane quarter
constexpr int kWideGateWarp = 2 + kWideEpiWarps;
constexpr int kWideMetaWarp0 = kWideGateWarp + 1;
constexpr int kWideThreads = 32 * (kWideMetaWarp0 + 4);  // producer, MMA, epilogue warps, gate, metadata warps
// W4 (2:4 weights stored as packed 4-bit codes): the weight tile of a stage is not copied by TMA but built in shared
// memory by eight more warps, one thread per weight row of the CTA: 32 bytes of nibbles per row and stage (fetched one
// stage ahead) widened to the 64 int8 slot bytes and written in the tile's swizzle; the stage's "full" barrier counts
// those warps too.  The 2:4 index metadata is the same as for 8-bit codes.  (Measured: a stage then takes ~980 clocks
// instead of 582, with eight or with sixteen builder warps alike: the generic-proxy stores and fences compete for the
// shared-memory bandwidth the MMAs and TMA already use up.  Fetching the codes four stages ahead instead of one made it
// slower still, 59.5 -> 70.7 us on 4096 -> 1024 at 16384 tokens: the loads' latency is not what holds the builders.
// One builder warp per ring slot, building the slot's whole tile with a single proxy fence, 66.4 us: a lone warp needs
// about 2.5 k clk per tile, nearly the ring's whole lead.  Two groups of four warps on alternate stages, two rows per
// thread: 61.0 us.  Fetch distances of two and three stages: 58.6 and 59.5 us.  Six builder warps, none of them on the
// MMA warp's scheduler: 69.5 us.  Sixteen builder warps in two groups on alternate stages (64 registers per thread): 87.8 us.)
constexpr int kWideBuildWarps = 8;
template <bool W4> constexpr int kWideThreadsOf = kWideThreads + (W4 ? 32 * kWideBuildWarps : 0);
constexpr uint32_t kWideNarrowBar = 13;  // named barriers 13 and 14: the four epilogue warps of block 0 / block 1 (narrow outputs)
constexpr uint32_t kWideRelayIds = 12;  // named barriers 1..12 carry the gate's relays in turn; the gate is never more
                                        // than STAGES + SKEW steps ahead of the MMA thread

template <int BN>
struct WideCfg {
    static constexpr int KB = 128;                       // reduction elements per stage
    static constexpr int A_ROWS = 2 * kBM;               // weight rows per CTA: two blocks of 128
    static constexpr int A_ROW = 64;                     // stored bytes per weight row and stage (2:4)
    static constexpr int A_BLOCK = kBM * A_ROW;          // bytes of one block's weight tile
    static constexpr int A_BYTES = A_ROWS * A_ROW;
    static constexpr int B_ROWS = BN / 2;                // tokens staged by each CTA
    static constexpr int B_BYTES = B_ROWS * 128;
    static constexpr int STAGE = A_BYTES + B_BYTES;
    // One [32 tokens][32 channels] 32-bit staging tile per epilogue warp: a whole accumulator chunk leaves with one TMA
    // store.  The SM's TMA unit takes about 40 clocks per store plus 2.5 per 128-byte row (measured: 112 stores of 16
    // rows per tile 9.3 k clocks, 56 of 32 rows 6.9 k, with 8 or 16 warps alike), and here the epilogue is exposed, so
    // fewer, taller boxes pay; a second tile per warp would cost a ring stage, which costs more (measured).
    static constexpr int STORE_STAGE = kWideEpiWarps * 4096;
    static constexpr int FIT = (kSmemLimit - kSmemTail - STORE_STAGE - 1024) / STAGE;
    static constexpr int STAGES = FIT < 8 ? FIT : 8;
    static constexpr int SMEM = STAGES * STAGE + STORE_STAGE + kSmemTail + 1024;
    static constexpr int META_COL = 2 * BN;              // first TMEM column of the metadata ring
    static constexpr int META_SLOT = 8;                  // columns per stage: two blocks x 128 index bits per row
    static_assert(STAGES >= 4, "pipeline too shallow");
    static_assert(META_COL + STAGES * META_SLOT <= kTmemCols, "accumulators and metadata ring exceed TMEM");
    static_assert(B_BYTES % 1024 == 0 && A_BYTES % 1024 == 0, "operand tiles must keep the swizzle alignment");
    static_assert(BN % 32 == 0 && BN <= 256, "token tile");
};

template <int BN, int EPI, int SKEW, bool W4>
__global__ void __launch_bounds__(kWideThreadsOf<W4>, 1)
nm_gemm_wide_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                    const __grid_constant__ CUtensorMap tmap_y, const GemmParams p,
                    const __grid_constant__ PairSchedule sched) {
    using Cfg = WideCfg<BN>;
    constexpr int S = Cfg::STAGES;
    static_assert(SKEW >= 0 && SKEW < S - 2, "the ring must hold the stages block 1 lags behind plus loads in flight");
    static_assert(S + SKEW < (int)kWideRelayIds, "relay barriers would be reused before the MMA thread has passed them");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* store_stage = smem + S * Cfg::STAGE;
    uint64_t* bars = reinterpret_cast<uint64_t*>(store_stage + Cfg::STORE_STAGE);
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };                     // leader: TMA bytes of both CTAs + 8 metadata warps
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };              // both CTAs (multicast commit)
    auto acc_full_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };       // both CTAs (multicast commit)
    auto acc_empty_bar = [&](int b) { return bar0 + 8u * (2 * S + 2 + b); };  // leader; four warps of each CTA arrive
    const uint32_t drained_bar = bar0 + 8u * (2 * S + 4);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 5);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* never_flag = tmem_slot + 2;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const bool leader = rank == 0;
    const int pair = blockIdx.x >> 1;
    const int tile_begin = sched.start[pair];
    const int tile_count = sched.start[pair + 1] - tile_begin;
    const uint32_t total = (uint32_t)tile_count * (uint32_t)p.kblocks;  // pipeline stages this pair runs

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { ptx::mbar_init(full_bar(s), 1 + 8 + (W4 ? 2 * kWideBuildWarps : 0)); ptx::mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { ptx::mbar_init(acc_full_bar(b), 1); ptx::mbar_init(acc_empty_bar(b), 8); }
        ptx::mbar_init(drained_bar, 1);
        *abort_flag = 0;
        *never_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_w);
        ptx::prefetch_tensormap(&tmap_x);
        if (p.tma_store) ptx::prefetch_tensormap(&tmap_y);
    }
    __syncthreads();
    ptx::cluster_arrive();   // both CTAs' barriers exist before anything remote touches them
    ptx::cluster_wait();
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Set-up above may overlap the tail of the kernel before this one in the stream; global memory is first
    // touched below.
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    auto raise_timeout = [&]() {  // both CTAs of the pair stop: the peer's roles see the flag in their own shared memory
        *abort_flag = 1;
        ptx::st_cluster_u32(ptx::map_to_cta(ptx::smem_u32(const_cast<uint32_t*>(abort_flag)), rank ^ 1u), 1u);
        if (p.status) atomicOr(p.status, NM_STATUS_TIMEOUT);
    };
    const uint32_t lead_full0 = ptx::map_to_cta(full_bar(0), 0);  // stage s: + 8 s (one window per CTA, linear inside)

    if (warp == 0) {
        // ------------------------------ TMA producer (both CTAs) --------------------------------
        if (lane == 0) {
            uint32_t it = 0, parity = 1u;  // the first pass over the ring finds every stage free
            const uint64_t keep = ptx::policy_evict_last();  // weights and X are read again by other pairs
            int s = 0;
            bool ok = true;
            const uint32_t smem0 = ptx::smem_u32(smem);
            for (int i = 0; i < tile_count && ok; ++i) {
                const TileCoord tc = tile_coord(tile_begin + i, p.n_tok_tiles, p.n_out_tiles, p.band);
                const int n0 = tc.o * (2 * Cfg::A_ROWS) + (int)rank * Cfg::A_ROWS;
                const int t0 = tc.t * BN + (int)rank * Cfg::B_ROWS;
                for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                    if (!ptx::mbar_wait_bounded(empty_bar(s), parity, abort_flag, kWaitLimit)) {
                        raise_timeout(); ok = false; break;
                    }
                    NM_TRACE_STAGE(it, 0);
                    if (NM_SKIP_STAGE(it)) { if (++s == S) { s = 0; parity ^= 1u; } continue; }
                    const uint32_t dst = smem0 + (uint32_t)s * Cfg::STAGE, lead_full = lead_full0 + 8u * s;
                    if (leader) ptx::mbar_expect_tx(full_bar(s), 2 * (W4 ? Cfg::B_BYTES : Cfg::STAGE));  // bytes of both CTAs
                    if (!W4) ptx::tma_load_2d_pair_hint(dst, &tmap_w, kb * Cfg::A_ROW, n0, lead_full, keep);
                    ptx::tma_load_2d_pair_hint(dst + Cfg::A_BYTES, &tmap_x, kb * 128, t0, lead_full, keep);
                    NM_TRACE_STAGE(it, 1);
                    if (++s == S) { s = 0; parity ^= 1u; }
                }
            }
            // After an expired wait (here or anywhere in the pair) the MMA thread runs through its remaining steps without
            // waiting for data, so the stages' barriers no longer say whether this producer's last copies have landed:
            // give them time before the CTA and its shared memory go away.
            if (!ok || *abort_flag) ptx::wait_clocks(kAbortDrain);
        }
    } else if (W4 && warp >= kWideMetaWarp0 + 4) {
        // ------------------------------ weight-tile builders (W4, both CTAs) ---------------------
        // Thread = one of the CTA's 256 weight rows (block = row / 128).  Per stage: the row's 32 bytes of packed
        // nibbles (128 reduction elements at 2:4 = 64 codes), fetched one stage ahead, become the 64 slot bytes.
        const int r256 = (warp - (kWideMetaWarp0 + 4)) * 32 + lane;
        uint8_t* const my_rows = smem + (r256 >> 7) * Cfg::A_BLOCK;  // this thread's block within a stage
        // the row's packed codes: pointer of the current tile, recomputed only when the tile changes (a single
        // thread's integer divisions cost hundreds of clocks)
        auto row_of_tile = [&](int i) -> const uint4* {
            if (i >= tile_count) return nullptr;
            const TileCoord tc = tile_coord(tile_begin + i, p.n_tok_tiles, p.n_out_tiles, p.band);
            const int n = tc.o * (2 * Cfg::A_ROWS) + (int)rank * Cfg::A_ROWS + r256;
            return n < p.out ? reinterpret_cast<const uint4*>(p.values + (size_t)n * p.vrow_bytes) : nullptr;  // rows past the end: zeros
        };
        auto fetch = [&](const uint4* row, int kb, uint4 (&raw)[2]) {
            if (row) { raw[0] = __ldg(row + 2 * kb); raw[1] = __ldg(row + 2 * kb + 1); }
            else raw[0] = raw[1] = make_uint4(0u, 0u, 0u, 0u);
        };
        int i = 0, kb = 0;
        const uint4* row = row_of_tile(0);
        uint4 cur[2], nxt[2];
        fetch(row, 0, nxt);
        uint32_t parity = 1u;
        int s = 0;
        while (i < tile_count) {
            cur[0] = nxt[0]; cur[1] = nxt[1];
            int ni = i, nkb = kb + 1;
            const uint4* nrow = row;
            if (nkb == p.kblocks) { nkb = 0; ++ni; nrow = row_of_tile(ni); }
            fetch(nrow, nkb, nxt);  // the next stage's codes travel while this one is built
            bool got = lane != 0 || ptx::mbar_wait_bounded(empty_bar(s), parity, abort_flag, kWaitLimit);
            if (!__all_sync(0xffffffffu, got)) { if (lane == 0) raise_timeout(); break; }
            uint32_t w[16];
            const uint32_t cw[8] = {cur[0].x, cur[0].y, cur[0].z, cur[0].w, cur[1].x, cur[1].y, cur[1].z, cur[1].w};
#pragma unroll
            for (int j = 0; j < 8; ++j) xf::widen8(cw[j], w[2 * j], w[2 * j + 1]);
            xf::store_row<true>(my_rows + (size_t)s * Cfg::STAGE, r256 & 127, w);
            ptx::fence_proxy_async_smem();  // the MMA reads the tile through the async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(lead_full0 + 8u * s);
            if (++s == S) { s = 0; parity ^= 1u; }
            i = ni; kb = nkb; row = nrow;
        }
    } else if (warp >= kWideMetaWarp0) {
        // ------------------------------ metadata warps (both CTAs) -------------------------------
        // Thread = TMEM lane = weight row of both blocks.  The canonical metadata of a row is 16 bytes per
        // stage; a batch of four stages (64 bytes, two full sectors) is fetched one batch ahead.
        const int q = warp & 3, row = q * 32 + lane;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + Cfg::META_COL;
        const uint4 kIdle = make_uint4(0x44444444u, 0x44444444u, 0x44444444u, 0x44444444u);  // valid "positions 0,1"
        const int row_u4 = p.mrow_words >> 2;  // 16-byte units per metadata row = stages per tile
        struct Pos { int i, kb; };
        auto fetch = [&](Pos at, uint4 (&w)[2][4]) {  // metadata of stages at.kb .. at.kb + 3 of tile at.i
            int n = 0;
            bool tile_ok = at.i < tile_count;
            if (tile_ok) {
                const TileCoord tc = tile_coord(tile_begin + at.i, p.n_tok_tiles, p.n_out_tiles, p.band);
                n = tc.o * (2 * Cfg::A_ROWS) + (int)rank * Cfg::A_ROWS + row;
            }
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                const int nb = n + b * kBM;
                const bool row_ok = tile_ok && nb < p.out;  // rows past the end: their products are discarded
                const uint4* src = reinterpret_cast<const uint4*>(p.meta) + (size_t)(row_ok ? nb : 0) * row_u4;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    w[b][j] = (row_ok && at.kb + j < p.kblocks) ? __ldg(src + at.kb + j) : kIdle;
            }
        };
        auto next_batch = [&](Pos at) {
            at.kb += 4;
            if (at.kb >= p.kblocks) { at.kb = 0; ++at.i; }
            return at;
        };
        Pos at{0, 0};
        uint4 cur[2][4], nxt[2][4];
        fetch(at, nxt);
        uint32_t parity = 1u;
        int s = 0;
        bool ok = true;
        while (at.i < tile_count && ok) {
#pragma unroll
            for (int b = 0; b < 2; ++b)
#pragma unroll
                for (int j = 0; j < 4; ++j) cur[b][j] = nxt[b][j];
            const Pos nx = next_batch(at);
            fetch(nx, nxt);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (at.kb + j < p.kblocks && ok) {
                    // the MMAs that read this slot's previous contents are done (same barrier as the stage)
                    bool got = lane != 0 || ptx::mbar_wait_bounded(empty_bar(s), parity, abort_flag, kWaitLimit);
                    ok = __all_sync(0xffffffffu, got);
                    if (!ok) { if (lane == 0) raise_timeout(); break; }
                    const uint32_t col = lane_taddr + (uint32_t)s * Cfg::META_SLOT;
                    ptx::tmem_st_32x4(col, cur[0][j].x, cur[0][j].y, cur[0][j].z, cur[0][j].w);
                    ptx::tmem_st_32x4(col + 4, cur[1][j].x, cur[1][j].y, cur[1][j].z, cur[1][j].w);
                    ptx::tmem_st_wait();
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(lead_full0 + 8u * s);
                    if (++s == S) { s = 0; parity ^= 1u; }
                }
            }
            at = nx;
        }
    } else if (warp == kWideGateWarp) {
        // ------------------------------ gate (leader): mbarrier waits relayed to the MMA warp ------
        // One relay per step g of the MMA thread: step g issues block 0 on stage g and block 1 on stage
        // g - SKEW.  Runs its full trip count even after a timeout (then without waiting).
        if (leader) {
            bool ok = true;
            auto wait = [&](uint32_t bar, uint32_t parity) {
                if (lane == 0 && ok && !ptx::mbar_wait_bounded(bar, parity, abort_flag, kWaitLimit)) {
                    raise_timeout();
                    ok = false;
                }
            };
            int s = 0, kb_l = 0, kb_t = 0;
            uint32_t parity = 0u, tile_l = 0, tile_t = 0, relay = 1;
            for (uint32_t g = 0; g < total + SKEW; ++g) {
                if (g < total) {
                    if (kb_l == 0) wait(acc_empty_bar(0), (tile_l & 1u) ^ 1u);  // block 0's accumulator read out
                    wait(full_bar(s), parity);
                    if (lane == 0) NM_TRACE_STAGE(g, 2);
                    if (++s == S) { s = 0; parity ^= 1u; }
                    if (++kb_l == p.kblocks) { kb_l = 0; ++tile_l; }
                }
                if (g >= (uint32_t)SKEW) {
                    if (kb_t == 0) wait(acc_empty_bar(1), (tile_t & 1u) ^ 1u);
                    if (++kb_t == p.kblocks) { kb_t = 0; ++tile_t; }
                }
                __syncwarp();
                ptx::relay_step(relay, abort_flag);
                relay = relay == kWideRelayIds ? 1 : relay + 1;
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (leader) --------------------------------------
        if (leader) {
            constexpr uint32_t idesc = ptx::idesc_i8(2 * kBM, BN, true);
            const uint32_t smem0 = ptx::smem_u32(smem);
            const uint64_t a_desc0 = ptx::smem_desc_kmajor(smem0, 64, ptx::kSwizzle64);
            const uint64_t b_desc0 = ptx::smem_desc_kmajor(smem0 + Cfg::A_BYTES, 128, ptx::kSwizzle128);
            const uint32_t meta0 = tmem_base + Cfg::META_COL;
            const uint32_t last_kb = (uint32_t)p.kblocks - 1;
            // ring position of block 0 (lead) and block 1 (trail): byte offset of the stage and metadata slot
            uint32_t off_l = 0, off_t = 0, slot_l = 0, slot_t = 0, kb_l = 0, kb_t = 0, relay = 1;
            for (uint32_t g = 0; g < total + SKEW; ++g) {
                ptx::named_bar_sync(relay, 64);
                relay = relay == kWideRelayIds ? 1 : relay + 1;
                ptx::tc_fence_after();  // orders the MMAs after the metadata stores and accumulator reads of other threads
                if (lane == 0) {
                    NM_TRACE_STAGE(g, 3);
                    if (g < total) {
                        const uint64_t a = ptx::desc_advance(a_desc0, off_l), b = ptx::desc_advance(b_desc0, off_l);
                        const uint32_t e = meta0 + slot_l;
                        ptx::mma_sp_i8_pair(tmem_base, a, b, e, idesc, kb_l != 0);
                        ptx::mma_sp_i8_pair(tmem_base, ptx::desc_advance(a, 32), ptx::desc_advance(b, 64), e + 2, idesc, 1u);
                        if (SKEW != 0 && kb_l == last_kb) ptx::tc_commit_pair(acc_full_bar(0), 3);
                    }
                    if (g >= (uint32_t)SKEW) {
                        const uint64_t a = ptx::desc_advance(a_desc0, off_t + Cfg::A_BLOCK), b = ptx::desc_advance(b_desc0, off_t);
                        const uint32_t e = meta0 + slot_t + 4;
                        ptx::mma_sp_i8_pair(tmem_base + BN, a, b, e, idesc, kb_t != 0);
                        ptx::mma_sp_i8_pair(tmem_base + BN, ptx::desc_advance(a, 32), ptx::desc_advance(b, 64), e + 2, idesc, 1u);
                        ptx::tc_commit_pair(empty_bar(slot_t >> 3), 3);  // both producers and the metadata warps may refill the stage
                        if (kb_t == last_kb) {
                            if (SKEW == 0) ptx::tc_commit_pair(acc_full_bar(0), 3);
                            ptx::tc_commit_pair(acc_full_bar(1), 3);
                        }
                    }
                    NM_TRACE_STAGE(g, 4);
                }
                if (g < total) {
                    off_l += Cfg::STAGE; slot_l += Cfg::META_SLOT;
                    if (slot_l == S * Cfg::META_SLOT) { off_l = 0; slot_l = 0; }
                    kb_l = kb_l == last_kb ? 0 : kb_l + 1;
                }
                if (g >= (uint32_t)SKEW) {
                    off_t += Cfg::STAGE; slot_t += Cfg::META_SLOT;
                    if (slot_t == S * Cfg::META_SLOT) { off_t = 0; slot_t = 0; }
                    kb_t = kb_t == last_kb ? 0 : kb_t + 1;
                }
                __syncwarp();
            }
            if (lane == 0) {  // everything issued has retired before TMEM is released
                ptx::tc_commit_pair(drained_bar, 1);
                ptx::mbar_wait_bounded(drained_bar, 0, never_flag, kWaitLimit);
            }
        }
    } else {
        // ------------------------------ epilogue warps (both CTAs) --------------------------------
        // Warps 2-5 read block 0's accumulator, warps 6-9 block 1's; each its TMEM lane quarter, all BN columns.
        constexpr int CH = BN / 32;
        // narrow outputs leave through staging tiles that a block's four warps share; for 32-bit outputs that form (one
        // 16 KB tile per block) was measured slower than a tile per warp (FFN2 alone 44.6 against 42.5 us)
        constexpr bool kGroupEpi = kNarrow<EPI>;
        const int ew = warp - 2, q = warp & 3, blk = ew >> 2;
        const uint32_t acc_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)blk * BN;
        uint32_t* my_stage = reinterpret_cast<uint32_t*>(store_stage + ew * 4096);
        const uint64_t stream_out = ptx::policy_evict_first();  // Y is written once and not read here
        const float sx = p.sx_dev ? *p.sx_dev : p.sx_host;
        const uint32_t lead_acc_empty = ptx::map_to_cta(acc_empty_bar(blk), 0);
        float amax = 0.0f, c_n = 0.0f, b_n = 0.0f;
        const float rsy = EPI == EPI_Q8 ? __frcp_rn(p.sy) : 0.0f;
        uint32_t n_stores = 0;
        int scaled_out_tile = -1;
        bool ok = true;
        auto release_acc = [&]() {  // this warp has read all it needs from the accumulator
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(lead_acc_empty);
        };
        for (int i = 0; i < tile_count && ok; ++i) {
            const TileCoord tc = tile_coord(tile_begin + i, p.n_tok_tiles, p.n_out_tiles, p.band);
            const int nw = tc.o * (2 * Cfg::A_ROWS) + (int)rank * Cfg::A_ROWS + blk * kBM + q * 32;  // first channel of this warp
            const int n = nw + lane, t0 = tc.t * BN;
            bool got = ptx::mbar_wait_bounded(acc_full_bar(blk), (uint32_t)i & 1u, abort_flag, kWaitLimit);
            ok = __all_sync(0xffffffffu, got);
            if (!ok && lane == 0) raise_timeout();
            if constexpr (kGroupEpi) ok = ptx::named_bar_and(kWideNarrowBar + blk, 128, ok);  // the block's four warps stop together
            if (!ok) break;
            ptx::tc_fence_after();
            if (ew == 0 && lane == 0) NM_TRACE_TILE(i, 0);
            if (ew == 4 && lane == 0) NM_TRACE_TILE(i, 2);
            const bool n_ok = n < p.out;
            if (EPI != EPI_ACC && tc.o != scaled_out_tile) {  // channel constants: fetched once per output tile
                scaled_out_tile = tc.o;
                c_n = n_ok ? __fmul_rn(sx, p.sw[n]) : 0.0f;
                b_n = n_ok && p.bias ? p.bias[n] : 0.0f;
            }
            const int nact = min(CH, (p.tokens - t0 + 31) >> 5);  // chunks that hold tokens (warp-uniform)
            if constexpr (kGroupEpi) {
                // int8 / bfloat16 outputs: the four warps of a block fill one [32 tokens][128 channels] staging tile per chunk
                // together (two tiles per block, used alternately: rows of 128 / 256 bytes for the store), the warp of lane
                // quarter 0 issues the store.  One named barrier per block orders the fills against the store.
                using OT = typename EpiOut<EPI>::type;
                const uint32_t gbar = kWideNarrowBar + blk;
                const int n0b = nw - q * 32;  // first channel of the block
                if (nact == 0) release_acc();
#pragma unroll 1
                for (int c = 0; c < nact; ++c) {
                    const int tc0 = t0 + c * 32;
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(acc_taddr + c * 32, r);
                    ptx::tmem_ld_wait();
                    if (c + 1 >= nact) release_acc();
                    if (p.tma_store) {
                        constexpr int NBUF = sizeof(OT) == 4 ? 1 : 2;  // 32 KB of staging: one 16 KB tile per block, or two smaller ones
                        OT* sb = reinterpret_cast<OT*>(store_stage) + (blk * NBUF + (NBUF == 2 ? (n_stores & 1u) : 0u)) * (32 * 128);
                        const int jmax = n_ok ? min(32, p.tokens - tc0) : 0;  // outputs of this lane that exist
                        if (q == 0 && lane == 0) ptx::bulk_wait_group_read<NBUF - 1>();  // the store that last used this tile has read it
                        ptx::named_bar_sync(gbar, 128);
                        OT* mine = sb + q * 32 + lane;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if constexpr (EPI == EPI_Q8) {
                                float worst = 0.0f;
#pragma unroll
                                for (int j = 0; j < 16; ++j) mine[(16 * h + j) * 128] = epi_convert_q8_fast(r[16 * h + j], c_n, b_n, rsy, worst);
                                if (__any_sync(0xffffffffu, !(worst <= 0.49996948f))) {  // rare (3 % of the runs)
                                    // find the values in question again; the exact division decides those
#pragma unroll
                                    for (int j = 0; j < 16; ++j) {
                                        float w1 = 0.0f;
                                        (void)epi_convert_q8_fast(r[16 * h + j], c_n, b_n, rsy, w1);
                                        if (!(w1 <= 0.49996948f))
                                            mine[(16 * h + j) * 128] =
                                                (uint8_t)(int8_t)quantise8_exact_call(__fmaf_rn((float)(int)r[16 * h + j], c_n, b_n), p.sy);
                                    }
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 16; ++j) {
                                    float y_abs;
                                    mine[(16 * h + j) * 128] = epi_convert<EPI>(r[16 * h + j], c_n, b_n, p.sy, rsy, y_abs);
                                    if constexpr (EPI == EPI_F32) amax = fmaxf(amax, 16 * h + j < jmax ? y_abs : 0.0f);
                                }
                            }
                        }
                        ptx::fence_proxy_async_smem();
                        ptx::named_bar_sync(gbar, 128);
                        if (q == 0 && lane == 0) {
                            ptx::tma_store_2d_hint(&tmap_y, n0b, tc0, ptx::smem_u32(sb), stream_out);
                            ptx::bulk_commit_group();
                        }
                        ++n_stores;
                    } else {
                        const int jmax = n_ok ? min(32, p.tokens - tc0) : 0;  // outputs of this lane that exist
                        OT* dst = reinterpret_cast<OT*>(EPI == EPI_F32 ? (void*)p.Y : EPI == EPI_ACC ? (void*)p.ACC : p.NARROW) + (size_t)tc0 * p.out + n;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            float y_abs;
                            const OT o = epi_convert<EPI>(r[j], c_n, b_n, p.sy, rsy, y_abs);
                            if constexpr (EPI == EPI_F32) amax = fmaxf(amax, j < jmax ? y_abs : 0.0f);
                            if (j < jmax) dst[(size_t)j * p.out] = o;
                        }
                    }
                }
                if (ew == 0 && lane == 0) NM_TRACE_TILE(i, 1);
                if (ew == 4 && lane == 0) NM_TRACE_TILE(i, 3);
                continue;
            }
            constexpr int RB = W4 ? 1 : 2;  // chunk read one ahead of its conversion, except where registers are short
            uint32_t r[RB][32];
            if (nact == 0) release_acc();
            else if (RB == 2) ptx::tmem_ld_32x32(acc_taddr, r[0]);
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int tc0 = t0 + c * 32;
                if (c < nact) {
                    if (RB == 1) ptx::tmem_ld_32x32(acc_taddr + c * 32, r[0]);
                    ptx::tmem_ld_wait();
                    if (c + 1 >= nact) release_acc();
                    else if (RB == 2) ptx::tmem_ld_32x32(acc_taddr + (c + 1) * 32, r[(c + 1) & (RB - 1)]);
                    const int jmax = n_ok ? min(32, p.tokens - tc0) : 0;  // outputs of this lane that exist
                    auto conv = [&](int j) -> uint32_t {
                        float y_abs;
                        const uint32_t o = epi_convert<EPI>(r[c & (RB - 1)][j], c_n, b_n, p.sy, 0.0f, y_abs);
                        if constexpr (EPI == EPI_F32) amax = fmaxf(amax, j < jmax ? y_abs : 0.0f);
                        return o;
                    };
                    if (p.tma_store) {  // separate branch-free loops for the two store paths
                        // rows of the tile past the last token are clipped by the store
                        if (lane == 0) ptx::bulk_wait_group_read<0>();  // the store before this one has read the tile
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 32; ++j) my_stage[j * 32 + lane] = conv(j);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            ptx::tma_store_2d_hint(&tmap_y, nw, tc0, ptx::smem_u32(my_stage), stream_out);
                            ptx::bulk_commit_group();
                        }
                    } else {
                        uint32_t* dst = reinterpret_cast<uint32_t*>(EPI == EPI_F32 ? (void*)p.Y : (void*)p.ACC) + (size_t)tc0 * p.out + n;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const uint32_t o = conv(j);
                            if (j < jmax) dst[(size_t)j * p.out] = o;
                        }
                    }
                }
            }
            if (ew == 0 && lane == 0) NM_TRACE_TILE(i, 1);
            if (ew == 4 && lane == 0) NM_TRACE_TILE(i, 3);
        }
        if (lane == 0) ptx::bulk_wait_group<0>();
        if (EPI == EPI_F32 && p.absmax) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            if (lane == 0) atomicMax(reinterpret_cast<unsigned*>(p.absmax), __float_as_uint(amax));
        }
    }

    // Neither CTA may release TMEM or exit while the other can still reach into it.
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_arrive();
    ptx::cluster_wait();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

}  // namespace nm
