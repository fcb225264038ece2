// Integer N:M linear layer on tcgen05 tensor cores with the dequantisation epilogue fused in.
//
// The sparse operand of tcgen05.mma.sp is A, so the kernel computes D = Wq * X^T: a tile is
// 128 output channels (TMEM lanes) x BN tokens (TMEM columns).  In TMEM one lane therefore holds
// one output channel, whose scale and bias are per-thread constants in the epilogue.
//
// One persistent CTA per SM walks a contiguous range of tiles ordered output-tile-major, so the
// weight tile (and its metadata) changes at most a few times per CTA.
//   warp 0      TMA producer: X tile and W tile of every 128-wide k-block into a ring of stages
//   warp 1      allocates TMEM; one lane issues tcgen05.mma[.sp] and commits to mbarriers.  It never
//               polls an mbarrier itself: a wait in the issuing thread leaves the tensor pipe idle for
//               its whole latency, so readiness reaches it through hardware named barriers
//   warps 2-9   copy the index metadata of the current 128 output channels into TMEM
//               (tcgen05.st, once per output tile, whole K), then run the epilogue of tile i
//               (tcgen05.ld -> fma -> shared staging -> TMA store) while the MMAs of tile i+1 fill
//               the other accumulator; two warps share a TMEM lane quarter and alternate chunks
//   warp 10     gate: waits on the "stage full" / "accumulator free" / "metadata ready" mbarriers and
//               relays each k-block to warp 1 with bar.arrive
//   warps 11-   (only for weights that are not stored in the tensor core's form: 4-bit codes, 1:4, 2:8,
//               1:8, 4:8) groups of four warps build the weight tile of every k-block in shared
//               memory from the packed codes and metadata (xform.cuh), the groups taking k-blocks
//               round-robin; the producer then loads X only
// Every mbarrier wait is bounded; on expiry the CTA raises NM_STATUS_TIMEOUT, drains and exits.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "xform.cuh"
#include "tmap.cuh"
#include "tileplan.cuh"
#include <cuda.h>
#include <cuda_runtime.h>
#include <mutex>
#include <algorithm>
#include <cstdlib>
#include <cstring>

namespace nm {

constexpr int kBM = 128;            // output channels per tile (MMA M)
constexpr int kKB = 128;            // reduction elements per pipeline stage
constexpr int kEpiWarps = 8;        // epilogue warps when the weights come straight from TMA (two per TMEM lane quarter)
constexpr int kEpiWarpsXf = 8;      // with the weight-building warps present
constexpr int kBuildGroups = 3;     // groups of four weight-building warps; group g takes k-blocks g, g + groups, ...
constexpr int kGemmThreads = 32 * (3 + kEpiWarps);        // producer, MMA, epilogue warps, gate
constexpr int kXformThreads = 32 * (3 + kEpiWarpsXf + 4 * kBuildGroups); // ... plus the warps that build the weight tiles
constexpr int kTmemCols = 512;
constexpr int kSmemLimit = 232448;  // 227 KB of dynamic shared memory per CTA
constexpr int kSmemTail = 2048;     // barriers, TMEM slot, abort flag, slot tables
constexpr int kStoreStage = 8 * 4096;  // per epilogue warp two [16 tokens][32 channels] fp32 staging tiles, used alternately
constexpr int kMaxStages = 7;       // the relay cycles through 8 named barriers
#ifndef NM_WAIT_LIMIT
#define NM_WAIT_LIMIT (1ll << 31)
#endif
constexpr long long kAbortDrain = 1ll << 17;  // SM clocks a producer of a CTA pair waits after an expired wait so that its copies in flight land
constexpr long long kWaitLimit = NM_WAIT_LIMIT;  // SM clocks per device-side wait (about a second; test builds shorten it)

// What the epilogue writes: y = fma(acc, sx * sw[o], b[o]) as fp32; the raw int32 accumulators; y re-quantised
// to 8 bits with a scale fixed ahead of time (Eq. 5, b = 8); y rounded to bfloat16.
enum { EPI_F32 = 0, EPI_ACC = 1, EPI_Q8 = 2, EPI_BF16 = 3 };
template <int EPI> struct EpiOut { using type = uint32_t; };          // fp32 / int32 move as 32-bit patterns
template <> struct EpiOut<EPI_Q8> { using type = uint8_t; };
template <> struct EpiOut<EPI_BF16> { using type = uint16_t; };
// Narrow outputs leave through [16 tokens][128 channels] tiles that the four warps of a TMEM-lane-quarter
// group fill together (rows of 128 / 256 bytes instead of 32 / 64): named barriers kNarrowFree + half and
// kNarrowFull + half order the fills against the one warp that issues the TMA store, kNarrowAgree + half
// makes the group take a timed-out wait together so that nobody is left alone on a barrier.
// EPI_Q8 without a branch per value: the code from the reciprocal rsy = RN(1 / sy), exact unless the product sits
// within 2^-15 of a rounding tie (6 values in 100000), where only the IEEE division decides.  `worst` keeps the largest
// distance of a product from its rounded integer over a run of values; beyond 0.49996948 the caller fills the run again
// with the exact quantiser.  The clamp to [-128.49, 127.49] before the add of 1.5 * 2^23 (whose own rounding rounds to
// the nearest-even integer) leaves nothing to clamp afterwards, and the low byte of the sum's bit pattern
// 0x4B400000 + code is the code.
__device__ __forceinline__ uint8_t epi_convert_q8_fast(uint32_t acc, float c_n, float b_n, float rsy, float& worst) {
    constexpr float kMagic = 12582912.0f;
    const float y = __fmaf_rn((float)(int)acc, c_n, b_n);
    const float qc = fminf(fmaxf(__fmul_rn(y, rsy), -128.49f), 127.49f);
    const float t = __fadd_rn(qc, kMagic);
    worst = fmaxf(worst, fabsf(__fsub_rn(qc, __fsub_rn(t, kMagic))));
    return (uint8_t)__float_as_uint(t);
}

// The exact quantiser as a call: the repair of near-ties runs for a few values in 10^5, its code stays out of the loops.
__device__ __noinline__ int quantise8_exact_call(float y, float sy) { return quantise8_exact(y, sy); }

template <int EPI> constexpr bool kNarrow = EPI == EPI_Q8 || EPI == EPI_BF16;
constexpr uint32_t kNarrowFree = 9, kNarrowFull = 11, kNarrowAgree = 13;

// One output element from an accumulator: fp32 value y, then the narrowing the epilogue kind asks for.
template <int EPI>
__device__ __forceinline__ typename EpiOut<EPI>::type epi_convert(uint32_t acc, float c_n, float b_n, float sy, float rsy, float& y_abs) {
    if constexpr (EPI == EPI_ACC) {
        y_abs = 0.0f;
        return acc;
    } else {
        const float y = __fmaf_rn((float)(int)acc, c_n, b_n);
        y_abs = fabsf(y);
        if constexpr (EPI == EPI_F32) {
            return __float_as_uint(y);
        } else if constexpr (EPI == EPI_Q8) {
            // the IEEE quotient y / sy rounded half to even and clamped to [-128, 127]
            (void)rsy;
            return (uint8_t)(int8_t)quantise8_exact(y, sy);
        } else {
            uint16_t h;
            asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(y));
            return h;
        }
    }
}
// Where the weight operand comes from: TMA (already in tensor-core form), built per k-block into the
// stage ring, or built once per output tile into a resident region (reduction length <= kResidentKB k-blocks).
enum { W_TMA = 0, W_BUILD = 1, W_RESIDENT = 2 };
constexpr int kResidentKB = 8;

struct GemmParams {
    int tokens, out, in;
    int n_tok_tiles, n_tiles, kblocks;
    int n_out_tiles, band;  // pair kernel: tiles are ordered band by band (see tile_coord)
    const uint32_t* meta;  // canonical metadata [out, mrow_words] (sparse modes)
    int mrow_words;
    const uint8_t* values; // packed codes (transform modes)
    int vrow_bytes, mrow_bytes, pat;
    int tma_store;         // 1: epilogue writes through shared memory + TMA; 0: direct stores
    const float* sw;
    const float* bias;
    const float* sx_dev;
    float sx_host;
    float* Y;
    int32_t* ACC;
    void* NARROW;          // int8 (EPI_Q8) or bfloat16 (EPI_BF16) output [tokens, out]
    float sy;              // static output scale of EPI_Q8
    float* absmax;
    uint32_t* status;
    unsigned long long* trace;  // NM_TRACE builds: time stamps of CTA 0 (see nm_debug_set_trace); NULL otherwise
    int skip_stage;             // NM_TEST_HOOKS builds: CTA 0's producer leaves this pipeline stage unissued (-1: none)
};

// Time stamps for profiling, compiled in with -DNM_TRACE only (a second library, never the product's):
// CTA 0 writes clock64() into row `it` (one row of 8 words per pipeline stage, kTraceStages rows) or, for
// per-tile events, into row kTraceStages + tile.  The kernels' work is unchanged.
constexpr int kTraceStages = 512, kTraceTiles = 64;
// Test hook, compiled in with -DNM_TEST_HOOKS only (the library the timeout test loads, never the product's): CTA 0's
// producer skips pipeline stage `skip_stage` -- nothing is armed, nothing is copied, no address is touched -- so that
// the stage's "full" barrier never completes and the bounded waits downstream run out.
#ifdef NM_TEST_HOOKS
#define NM_SKIP_STAGE(it) (p.skip_stage >= 0 && blockIdx.x == 0 && (it) == (uint32_t)p.skip_stage)
#else
#define NM_SKIP_STAGE(it) false
#endif

#ifdef NM_TRACE
#define NM_TRACE_STAGE(it, col) do { if (p.trace && blockIdx.x == 0 && (it) < (uint32_t)kTraceStages) p.trace[8 * (size_t)(it) + (col)] = clock64(); } while (0)
#define NM_TRACE_TILE(i, col) do { if (p.trace && blockIdx.x == 0 && (i) < kTraceTiles) p.trace[8 * (size_t)(kTraceStages + (i)) + (col)] = clock64(); } while (0)
// Phases of the first epilogue warp's work on a tile, summed per tile into columns 3..7 of the tile's row: waiting for the
// accumulator chunk, waiting for the staging tile to be free, converting and filling it, the proxy fence, issuing the store.
#define NM_TRACE_EPI_DECL long long tr_t = clock64(), tr_acc[5] = {0, 0, 0, 0, 0}
#define NM_TRACE_EPI_MARK() do { tr_t = clock64(); } while (0)
#define NM_TRACE_EPI_ADD(k) do { const long long tr_now = clock64(); tr_acc[k] += tr_now - tr_t; tr_t = tr_now; } while (0)
#define NM_TRACE_EPI_FLUSH(i) do { if (p.trace && blockIdx.x == 0 && (i) < kTraceTiles) { for (int k = 0; k < 5; ++k) { p.trace[8 * (size_t)(kTraceStages + (i)) + 3 + k] = tr_acc[k]; tr_acc[k] = 0; } } } while (0)
#else
#define NM_TRACE_STAGE(it, col) do { } while (0)
#define NM_TRACE_TILE(i, col) do { } while (0)
#define NM_TRACE_EPI_DECL do { } while (0)
#define NM_TRACE_EPI_MARK() do { } while (0)
#define NM_TRACE_EPI_ADD(k) do { } while (0)
#define NM_TRACE_EPI_FLUSH(i) do { } while (0)
#endif

template <bool SPARSE, int BN, bool RESIDENT = false>
struct GemmCfg {
    static constexpr int A_ROW = SPARSE ? 64 : 128;   // bytes of one weight row per stage
    static constexpr int A_BYTES = kBM * A_ROW;
    static constexpr int B_BYTES = BN * 128;
    static constexpr int A_RES = RESIDENT ? kResidentKB * A_BYTES : 0;  // whole-K weight tile kept across token tiles
    static constexpr int B_OFF = RESIDENT ? 0 : A_BYTES;                // X tile within a stage
    static constexpr int STAGE = B_OFF + B_BYTES;
    static constexpr int FIT = (kSmemLimit - kSmemTail - kStoreStage - 1024 - A_RES) / STAGE;
    static constexpr int STAGES = FIT < kMaxStages ? FIT : kMaxStages;
    static constexpr int SMEM = STAGES * STAGE + A_RES + kStoreStage + kSmemTail + 1024;
    static constexpr int META_COL = 2 * BN;           // first TMEM column of the metadata
    static constexpr int META_COLS = kTmemCols - 2 * BN;
    static_assert(STAGES >= 3, "pipeline too shallow");
    static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "token tile");
};

template <bool SPARSE, int BN, int EPI, int WSRC>
__global__ void __launch_bounds__(WSRC != W_TMA ? kXformThreads : kGemmThreads, 1)
nm_gemm_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
               const __grid_constant__ CUtensorMap tmap_y, const GemmParams p) {
    constexpr bool XF = WSRC != W_TMA, RES = WSRC == W_RESIDENT;
    using Cfg = GemmCfg<SPARSE, BN, RES>;
    constexpr int S = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* a_res = smem + S * Cfg::STAGE;  // resident weight tile: kResidentKB k-blocks of A_BYTES
    uint8_t* store_stage = a_res + Cfg::A_RES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(store_stage + kStoreStage);
    // bars[0..S) full, [S..2S) empty, then acc_full[2], acc_empty[2], meta_ready, drained, a_full, a_free
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
    auto acc_full_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };
    auto acc_empty_bar = [&](int b) { return bar0 + 8u * (2 * S + 2 + b); };
    const uint32_t meta_bar = bar0 + 8u * (2 * S + 4);
    const uint32_t drained_bar = bar0 + 8u * (2 * S + 5);
    const uint32_t a_full_bar = bar0 + 8u * (2 * S + 6);  // resident weight tile built (all builder warps)
    const uint32_t a_free_bar = bar0 + 8u * (2 * S + 7);  // ... and no longer read by any MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 8);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* never_flag = tmem_slot + 2;  // stays 0: for the drain waits after an abort
    uint32_t* lut = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(bars) + 512);

    constexpr int EW = XF ? kEpiWarpsXf : kEpiWarps, kGateWarp = 2 + EW;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per = p.n_tiles / gridDim.x, rem = p.n_tiles % gridDim.x;
    const int tile_begin = blockIdx.x * per + min((int)blockIdx.x, rem);
    const int tile_count = per + ((int)blockIdx.x < rem ? 1 : 0);

    if (threadIdx.x == 0) {
        // a stage is full when its TMA bytes have landed and, in transform mode, the four warps building it are done
        for (int s = 0; s < S; ++s) { ptx::mbar_init(full_bar(s), WSRC == W_BUILD ? 5 : 1); ptx::mbar_init(empty_bar(s), 1); }
        ptx::mbar_init(a_full_bar, 4 * kBuildGroups);
        ptx::mbar_init(a_free_bar, 1);
        for (int b = 0; b < 2; ++b) { ptx::mbar_init(acc_full_bar(b), 1); ptx::mbar_init(acc_empty_bar(b), XF ? kEpiWarpsXf : kEpiWarps); }
        ptx::mbar_init(meta_bar, 4);
        ptx::mbar_init(drained_bar, 1);
        *abort_flag = 0;
        *never_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_w);
        ptx::prefetch_tensormap(&tmap_x);
        if (p.tma_store) ptx::prefetch_tensormap(&tmap_y);
    }
    if (XF) xf::build_lut(lut, threadIdx.x, blockDim.x);
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Set-up above overlaps the tail of the kernel before this one in the stream (when launched as its
    // programmatic dependent); nothing in global memory is read or written before this point.
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    auto raise_timeout = [&]() {
        *abort_flag = 1;
        if (p.status) atomicOr(p.status, NM_STATUS_TIMEOUT);
    };

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int i = 0; i < tile_count && ok; ++i) {
                const int tile = tile_begin + i;
                const int n0 = (tile / p.n_tok_tiles) * kBM, t0 = (tile % p.n_tok_tiles) * BN;
                for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                    const int s = it % S;
                    if (!ptx::mbar_wait_bounded(empty_bar(s), ((it / S) & 1u) ^ 1u, abort_flag, kWaitLimit)) {
                        raise_timeout(); ok = false; break;
                    }
                    if (NM_SKIP_STAGE(it)) continue;
                    const uint32_t a_dst = ptx::smem_u32(smem + s * Cfg::STAGE);
                    ptx::mbar_expect_tx(full_bar(s), XF ? Cfg::B_BYTES : Cfg::STAGE);
                    if (!XF) ptx::tma_load_2d(a_dst, &tmap_w, kb * Cfg::A_ROW, n0, full_bar(s));
                    ptx::tma_load_2d(a_dst + Cfg::B_OFF, &tmap_x, kb * 128, t0, full_bar(s));
                }
            }
            if (!ok) {
                // let copies already in flight land before the CTA goes away
                const uint32_t first = it > (uint32_t)S ? it - S : 0;
                for (uint32_t j = first; j < it; ++j)
                    ptx::mbar_wait_bounded(full_bar(j % S), (j / S) & 1u, never_flag, kWaitLimit >> 4);
            }
        }
    } else if (XF && warp >= kGateWarp + 1) {
        // ------------------------------ weight-tile builders (transform modes) ------------------
        // One thread builds one row of a k-block.  The work of one k-block is a long dependent chain
        // (unpack, table lookups, byte permutes, stores, fence), so several groups of four warps
        // take the k-blocks round-robin: group g builds pipeline steps g, g + G, g + 2G, ...
        constexpr int G = kBuildGroups;
        static_assert(RES || S > G, "every group needs a stage of its own in flight");
        const int bw = warp - (kGateWarp + 1), grp = bw >> 2;
        const int tr = (bw & 3) * 32 + lane;  // row of the 128-row weight tile
        const int cb = xf::code_bytes(p.pat), mb = xf::meta_bytes(p.pat);
        const uint8_t* meta8 = reinterpret_cast<const uint8_t*>(p.meta);
        if constexpr (RES) {
            // Short reductions: the whole-K weight tile of an output tile is built once and stays in
            // shared memory for all token tiles of that output tile; the ring then carries X only.
            int prev_out_tile = -1;
            uint32_t free_parity = 1u;  // nothing reads the region before the first build
            for (int i = 0; i < tile_count; ++i) {
                const int out_tile = (tile_begin + i) / p.n_tok_tiles;
                if (out_tile == prev_out_tile) continue;
                prev_out_tile = out_tile;
                const int n = out_tile * kBM + tr;
                const bool row_ok = n < p.out;
                const uint8_t* v = p.values + (size_t)(row_ok ? n : 0) * p.vrow_bytes;
                const uint8_t* m = meta8 + (size_t)(row_ok ? n : 0) * p.mrow_bytes;
                xf::Raw cur = xf::load_raw(p.pat, v + (size_t)grp * cb, m + (size_t)grp * mb, row_ok && grp < p.kblocks);
                // the MMAs of the previous output tile have finished reading the region
                bool got = lane != 0 || ptx::mbar_wait_bounded(a_free_bar, free_parity, abort_flag, kWaitLimit);
                free_parity ^= 1u;
                if (!__all_sync(0xffffffffu, got)) { if (lane == 0) raise_timeout(); break; }
                for (int kb = grp; kb < p.kblocks; kb += G) {
                    const int nkb = kb + G;
                    xf::Raw nxt = xf::load_raw(p.pat, v + (size_t)nkb * cb, m + (size_t)nkb * mb, row_ok && nkb < p.kblocks);
                    uint32_t w[SPARSE ? 16 : 32];
                    xf::build_row<SPARSE>(p.pat, cur, lut, w);
                    xf::store_row<SPARSE>(a_res + kb * Cfg::A_BYTES, tr, w);
                    cur = nxt;
                }
                ptx::fence_proxy_async_smem();  // the MMA reads the tile through the async proxy
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(a_full_bar);
            }
        } else {
        // position of a pipeline step: tile index i within this CTA's range, k-block kb; row pointers follow i
        struct Pos { int i, kb; const uint8_t* v; const uint8_t* m; bool ok; };
        auto locate = [&](Pos& q) {  // row pointers and validity for tile q.i
            q.ok = q.i < tile_count;
            const int n = q.ok ? ((tile_begin + q.i) / p.n_tok_tiles) * kBM + tr : 0;
            q.ok = q.ok && n < p.out;
            q.v = p.values + (size_t)n * p.vrow_bytes;
            q.m = meta8 + (size_t)n * p.mrow_bytes;
        };
        auto advance = [&](Pos& q) {  // G pipeline steps further
            q.kb += G;
            if (q.kb >= p.kblocks) {
                do { q.kb -= p.kblocks; ++q.i; } while (q.kb >= p.kblocks);
                locate(q);
            }
        };
        Pos at{0, 0, nullptr, nullptr, false};
        at.kb = grp;
        while (at.kb >= p.kblocks) { at.kb -= p.kblocks; ++at.i; }
        locate(at);
        int s = grp % S;
        uint32_t parity = 1u;  // of the empty barrier: the first pass over the ring finds every stage free
        xf::Raw cur = xf::load_raw(p.pat, at.v + (size_t)at.kb * cb, at.m + (size_t)at.kb * mb, at.ok);
        while (at.i < tile_count) {
            // fetch this group's next k-block before working on the current one
            Pos nx = at;
            advance(nx);
            xf::Raw nxt = xf::load_raw(p.pat, nx.v + (size_t)nx.kb * cb, nx.m + (size_t)nx.kb * mb, nx.ok);
            bool got = lane != 0 || ptx::mbar_wait_bounded(empty_bar(s), parity, abort_flag, kWaitLimit);
            if (!__all_sync(0xffffffffu, got)) { if (lane == 0) raise_timeout(); break; }
            uint32_t w[SPARSE ? 16 : 32];
            xf::build_row<SPARSE>(p.pat, cur, lut, w);
            xf::store_row<SPARSE>(smem + s * Cfg::STAGE, tr, w);
            ptx::fence_proxy_async_smem();  // the MMA reads the tile through the async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(full_bar(s));
            cur = nxt;
            at = nx;
            s += G;
            if (s >= S) { s -= S; parity ^= 1u; }
        }
        }
    } else if (warp == kGateWarp) {
        // ------------------------------ gate: mbarrier waits relayed to the MMA warp ------------
        // Runs its full trip count even after a timeout (then without waiting), so that the MMA
        // warp, which blocks on the named barriers, always gets its arrivals.
        uint32_t it = 0, meta_phase = 0, a_phase = 0;
        int prev_out_tile = -1;
        bool ok = true;
        auto wait = [&](uint32_t bar, uint32_t parity) {
            if (lane == 0 && ok && !ptx::mbar_wait_bounded(bar, parity, abort_flag, kWaitLimit)) {
                raise_timeout();
                ok = false;
            }
        };
        for (int i = 0; i < tile_count; ++i) {
            const int tile = tile_begin + i, out_tile = tile / p.n_tok_tiles, buf = i & 1;
            if (out_tile != prev_out_tile) {
                if (SPARSE) { wait(meta_bar, meta_phase); meta_phase ^= 1u; }
                if (RES) { wait(a_full_bar, a_phase); a_phase ^= 1u; }
                prev_out_tile = out_tile;
            }
            wait(acc_empty_bar(buf), ((i >> 1) & 1u) ^ 1u);
            for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                wait(full_bar(it % S), (it / S) & 1u);
                __syncwarp();
                ptx::relay_step(1 + (it & 7u), abort_flag);
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ---------------------------------------------
        constexpr uint32_t idesc = ptx::idesc_i8(kBM, BN, SPARSE);
        uint32_t it = 0;
        for (int i = 0; i < tile_count; ++i) {
            const int buf = i & 1;
            const uint32_t d_tmem = tmem_base + buf * BN;
            const bool last_of_out_tile = RES && (tile_begin + i + 1) / p.n_tok_tiles != (tile_begin + i) / p.n_tok_tiles;
            for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                const int s = it % S;
                ptx::named_bar_sync(1 + (it & 7u), 64);  // stage s holds k-block kb (and, for kb = 0, the
                                                         // accumulator is free and the metadata in place)
                // The tcgen05 fence orders the MMAs after other threads' TMEM accesses (accumulator read
                // back, metadata stores): needed once per tile.  Executed every stage it drains the MMA
                // pipe (measured ~585 clk per stage); the staged operands are ordered by the mbarrier.
                if (kb == 0) ptx::tc_fence_after();
                if (lane == 0) {
                    const uint32_t st_addr = ptx::smem_u32(smem + s * Cfg::STAGE), b_addr = st_addr + Cfg::B_OFF;
                    const uint32_t a_addr = RES ? ptx::smem_u32(a_res + kb * Cfg::A_BYTES) : st_addr;
                    if constexpr (SPARSE) {
#pragma unroll
                        for (int j = 0; j < 2; ++j)  // 64 logical k each: 32 stored bytes of A, 64 of B
                            ptx::mma_sp_i8(d_tmem, ptx::smem_desc_kmajor(a_addr + 32 * j, 64, ptx::kSwizzle64),
                                           ptx::smem_desc_kmajor(b_addr + 64 * j, 128, ptx::kSwizzle128),
                                           tmem_base + Cfg::META_COL + kb * 4 + 2 * j, idesc, (kb | j) != 0);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j)  // 32 k each
                            ptx::mma_i8(d_tmem, ptx::smem_desc_kmajor(a_addr + 32 * j, 128, ptx::kSwizzle128),
                                        ptx::smem_desc_kmajor(b_addr + 32 * j, 128, ptx::kSwizzle128), idesc, (kb | j) != 0);
                    }
                    ptx::tc_commit(empty_bar(s));  // stage reusable once these MMAs have read it
                    if (kb == p.kblocks - 1) {
                        ptx::tc_commit(acc_full_bar(buf));
                        if (RES && last_of_out_tile) ptx::tc_commit(a_free_bar);  // the builders may overwrite the weight tile
                    }
                }
                __syncwarp();
            }
        }
        if (lane == 0) {  // everything issued has retired before TMEM is released
            ptx::tc_commit(drained_bar);
            ptx::mbar_wait_bounded(drained_bar, 0, never_flag, kWaitLimit);
        }
    } else {
        // ------------------------------ metadata + epilogue warps ------------------------------
        // Warp w may touch TMEM lanes 32 * (w % 4) ... + 31.  With eight warps two share a lane quarter
        // and take alternate 32-column chunks of the accumulator.
        constexpr int EWH = EW / 4;               // warps per lane quarter
        constexpr int CH = BN / 32;               // chunks per accumulator
        constexpr int CI = (CH + EWH - 1) / EWH;  // chunks per warp
        const int ew = warp - 2, q = warp & 3, half = ew >> 2, row = q * 32 + lane;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        float* my_stage = reinterpret_cast<float*>(store_stage + ew * 4096);
        const float sx = p.sx_dev ? *p.sx_dev : p.sx_host;
        float amax = 0.0f, c_n = 0.0f, b_n = 0.0f;
        const float rsy = EPI == EPI_Q8 ? __frcp_rn(p.sy) : 0.0f;
        int scaled_out_tile = -1;
        uint32_t n_stores = 0;
        bool ok = true;

        auto load_meta = [&](int out_tile) {
            const int n = out_tile * kBM + row;
            const uint4* src = reinterpret_cast<const uint4*>(p.meta + (size_t)n * p.mrow_words);
            for (int c = 0; c < p.mrow_words; c += 4) {
                // rows past the end get a valid "positions 0,1" pattern; their products are discarded
                uint4 w = make_uint4(0x44444444u, 0x44444444u, 0x44444444u, 0x44444444u);
                if (n < p.out) {
                    if constexpr (XF) w = xf::hw_meta(p.pat, reinterpret_cast<const uint8_t*>(p.meta) + (size_t)n * p.mrow_bytes + (size_t)(c >> 2) * xf::meta_bytes(p.pat), lut);
                    else w = __ldg(src + (c >> 2));
                }
                ptx::tmem_st_32x4(lane_taddr + Cfg::META_COL + c, w.x, w.y, w.z, w.w);
            }
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(meta_bar);
        };
        auto release_acc = [&](int buf) {  // this warp has read all it needs from the accumulator
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty_bar(buf));
        };

        for (int i = 0; i < tile_count && ok; ++i) {
            const int tile = tile_begin + i, out_tile = tile / p.n_tok_tiles, buf = i & 1;
            const int n0 = out_tile * kBM, n = n0 + row, t0 = (tile % p.n_tok_tiles) * BN;
            if (SPARSE && i == 0 && half == 0) load_meta(out_tile);
            bool got = ptx::mbar_wait_bounded(acc_full_bar(buf), (i >> 1) & 1u, abort_flag, kWaitLimit);
            ok = __all_sync(0xffffffffu, got);
            if (!ok && lane == 0) raise_timeout();
            if constexpr (kNarrow<EPI>) ok = ptx::named_bar_and(kNarrowAgree + half, 128, ok);  // the group stops together
            if (!ok) break;
            ptx::tc_fence_after();
            if (SPARSE && half == 0 && i + 1 < tile_count) {
                const int next_out_tile = (tile + 1) / p.n_tok_tiles;
                if (next_out_tile != out_tile) load_meta(next_out_tile);  // MMAs of this output tile are done
            }
            const bool n_ok = n < p.out;
            if (EPI != EPI_ACC && out_tile != scaled_out_tile) {  // channel constants: fetched once per output tile
                scaled_out_tile = out_tile;
                c_n = n_ok ? __fmul_rn(sx, p.sw[n]) : 0.0f;
                b_n = n_ok && p.bias ? p.bias[n] : 0.0f;
            }
            const int nact = min(CH, (p.tokens - t0 + 31) >> 5);  // chunks that hold tokens (warp-uniform)
            // Accumulator chunks are read one ahead of their conversion (two register buffers); the
            // transform kernels, short of registers with their extra warps, read each chunk when it is due.
            // narrow outputs: the conversion code of one chunk is long; the chunk loop stays a loop (one copy of that code
            // instead of CI, which no longer fit the instruction cache) and every chunk is read when it is due
            constexpr int RB = (XF || kNarrow<EPI>) ? 1 : 2;
            uint32_t r[RB][32];
            if (half >= nact) release_acc(buf);
            else if (RB == 2) ptx::tmem_ld_32x32(lane_taddr + buf * BN + half * 32, r[0]);
#pragma unroll (kNarrow<EPI> ? 1 : CI)
            for (int ci = 0; ci < CI; ++ci) {
                const int c = half + ci * EWH, tc0 = t0 + c * 32;
                if (c < nact) {
                    if (RB == 1) ptx::tmem_ld_32x32(lane_taddr + buf * BN + c * 32, r[0]);
                    ptx::tmem_ld_wait();
                    if (c + EWH >= nact) release_acc(buf);
                    else if (RB == 2) ptx::tmem_ld_32x32(lane_taddr + buf * BN + (c + EWH) * 32, r[(ci + 1) & (RB - 1)]);
                    // conversion of accumulator column j of this chunk; jmax = outputs of this lane that exist
                    const int jmax = n_ok ? min(32, p.tokens - tc0) : 0;
                    using OT = typename EpiOut<EPI>::type;
                    auto conv = [&](int j) -> OT {
                        float y_abs;
                        const OT o = epi_convert<EPI>(r[ci & (RB - 1)][j], c_n, b_n, p.sy, rsy, y_abs);
                        if constexpr (EPI == EPI_F32) amax = fmaxf(amax, j < jmax ? y_abs : 0.0f);
                        return o;
                    };
                    // The two store paths are separate loops: a branch inside the unrolled loop costs a
                    // pipeline refill per column (measured ~30 clk each), far more than its arithmetic.
                    if (p.tma_store) {
                        // two stores of 16 tokens each, through alternating staging tiles: while one is
                        // being read by its TMA store the other is filled
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (tc0 + 16 * h >= p.tokens) continue;  // warp-uniform (and the same in all warps of a group)
                            if constexpr (kNarrow<EPI>) {
                                OT* sb = reinterpret_cast<OT*>(store_stage) + (half * 2 + (n_stores & 1u)) * (16 * 128);
                                if (q == 0 && lane == 0) ptx::bulk_wait_group_read<1>();  // the store before the last has read this tile
                                ptx::named_bar_sync(kNarrowFree + half, 128);
                                if constexpr (EPI == EPI_Q8) {
                                    float worst = 0.0f;
#pragma unroll
                                    for (int j = 0; j < 16; ++j)
                                        sb[j * 128 + q * 32 + lane] = epi_convert_q8_fast(r[ci & (RB - 1)][16 * h + j], c_n, b_n, rsy, worst);
                                    if (__any_sync(0xffffffffu, !(worst <= 0.49996948f))) {  // rare (3 % of the runs)
                                        // find the values in question again; the exact division decides those
#pragma unroll
                                        for (int j = 0; j < 16; ++j) {
                                            float w1 = 0.0f;
                                            (void)epi_convert_q8_fast(r[ci & (RB - 1)][16 * h + j], c_n, b_n, rsy, w1);
                                            if (!(w1 <= 0.49996948f))
                                                sb[j * 128 + q * 32 + lane] = (uint8_t)(int8_t)quantise8_exact_call(
                                                    __fmaf_rn((float)(int)r[ci & (RB - 1)][16 * h + j], c_n, b_n), p.sy);
                                        }
                                    }
                                } else {
#pragma unroll
                                    for (int j = 0; j < 16; ++j) sb[j * 128 + q * 32 + lane] = conv(16 * h + j);
                                }
                                ptx::fence_proxy_async_smem();
                                ptx::named_bar_sync(kNarrowFull + half, 128);
                                if (q == 0 && lane == 0) {
                                    ptx::tma_store_2d(&tmap_y, n0, tc0 + 16 * h, ptx::smem_u32(sb));
                                    ptx::bulk_commit_group();
                                }
                                ++n_stores;
                            } else {
                                OT* sb = reinterpret_cast<OT*>(my_stage + (n_stores & 1u) * 512);
                                if (lane == 0) ptx::bulk_wait_group_read<1>();  // the store before the last has read this tile
                                __syncwarp();
#pragma unroll
                                for (int j = 0; j < 16; ++j) sb[j * 32 + lane] = conv(16 * h + j);
                                ptx::fence_proxy_async_smem();
                                __syncwarp();
                                if (lane == 0) {
                                    ptx::tma_store_2d(&tmap_y, n0 + q * 32, tc0 + 16 * h, ptx::smem_u32(sb));
                                    ptx::bulk_commit_group();
                                }
                                ++n_stores;
                            }
                        }
                    } else {  // output rows not 16-byte aligned: lane = channel, j = token
                        OT* dst = reinterpret_cast<OT*>(EPI == EPI_F32 ? (void*)p.Y : EPI == EPI_ACC ? (void*)p.ACC : p.NARROW) + (size_t)tc0 * p.out + n;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const OT o = conv(j);
                            if (j < jmax) dst[(size_t)j * p.out] = o;
                        }
                    }
                }
            }
        }
        if (lane == 0) ptx::bulk_wait_group<0>();
        if (EPI == EPI_F32 && p.absmax) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            if (lane == 0) atomicMax(reinterpret_cast<unsigned*>(p.absmax), __float_as_uint(amax));
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------------
// CTA-pair variant (cluster of two, tcgen05 cta_group::2) for weights already in tensor-core form.
// A pair tile is 256 output channels x BN tokens.  Each CTA stages its own 128 weight rows and HALF of
// the X tile (BN/2 tokens); one MMA issued by the leader CTA (cluster rank 0) spans both CTAs: every
// CTA's tensor core accumulates its 128 rows over all BN tokens, taking the other half of X from the
// peer's shared memory.  Per MAC this moves 0.63x the bytes of the one-CTA kernel through L2 and
// through each SM's shared-memory port, and the sparse MMA is no longer shared-memory bound.
// Protocol differences: both producers' TMA bytes are counted on the LEADER's "full" barrier; the
// leader's commits are multicast to the "empty" / "accumulator full" barriers of both CTAs; the
// peer's epilogue and metadata warps arrive remotely on the leader's barriers; the pair synchronises
// as a cluster before the first remote operation and before TMEM is released.
// ---------------------------------------------------------------------------------------------
constexpr int kPairThreads = 32 * (3 + kEpiWarps);
constexpr int kPairBuildWarps = 8;  // two groups of four (one thread per weight row of the CTA) taking alternate 128-wide k-blocks
template <bool BUILD> constexpr int kPairThreadsOf = kPairThreads + (BUILD ? 32 * kPairBuildWarps : 0);
// Narrow outputs from resident weights: the epilogue sets the pace there and is a chain of waits (accumulator read, staging
// tile, fence, store issue) that eight warps do not overlap; sixteen epilogue warps in four groups take 16-token units.
// The second eight sit behind the gate warp, where the builder warps of the BUILD form are.
template <int EPI, bool RES, bool BUILD> constexpr int kPairEpiWarps = (kNarrow<EPI> && RES && !BUILD) ? 16 : kEpiWarps;
template <int EPI, bool RES, bool BUILD> constexpr int kPairThreadsFor = kPairThreadsOf<BUILD> + 32 * (kPairEpiWarps<EPI, RES, BUILD> - kEpiWarps);
constexpr uint32_t kNarrowGroup = 9;  // named barriers 9-12: one per group of four epilogue warps in that form
constexpr int kPairMaxStages = 7;   // the relay cycles through 8 named barriers (ids 1-8; 9-14 serve the narrow-output epilogue)

constexpr int kPairResStages = 4;   // stages of weights a CTA can keep resident (1024 reduction elements at 2:4)

template <bool SPARSE, int BN, bool RES = false>
struct PairCfg {
    // A stage holds 128 stored bytes of every weight row (256 reduction elements when 2:4 compressed,
    // 128 when dense) and the matching 128-byte-wide slices of X: one TMA operation each, four MMAs.
    static constexpr int KB = SPARSE ? 256 : 128;
    static constexpr int A_ROW = 128;
    static constexpr int A_BYTES = kBM * A_ROW;
    static constexpr int B_ROWS = BN / 2;            // tokens staged by each CTA
    static constexpr int B_SUB = B_ROWS * 128;       // one 128-byte-wide slice of the X half tile
    static constexpr int B_BYTES = B_SUB * (KB / 128);
    // RES: the whole-K weight rows of the CTA stay in shared memory across the token tiles of an
    // output tile; the ring then carries X only and holds more of it.
    static constexpr int A_RES = RES ? kPairResStages * A_BYTES : 0;
    static constexpr int B_OFF = RES ? 0 : A_BYTES;
    static constexpr int STAGE = B_OFF + B_BYTES;
    // Epilogue staging: two [16 tokens][32 channels] fp32 tiles per warp where the epilogue sets the pace
    // (short reductions, RES); one where the main loop does and a fifth stage in the ring is worth more.
    static constexpr int STORE_BUFS = RES ? 2 : 1;
    static constexpr int STORE_STAGE = kEpiWarps * STORE_BUFS * 2048;
    static constexpr int FIT = (kSmemLimit - kSmemTail - STORE_STAGE - 1024 - A_RES) / STAGE;
    static constexpr int STAGES = FIT < kPairMaxStages ? FIT : kPairMaxStages;
    static constexpr int SMEM = STAGES * STAGE + A_RES + STORE_STAGE + kSmemTail + 1024;
    static_assert(STAGES >= 3, "pipeline too shallow");
    static constexpr int META_COL = 2 * BN;
    static constexpr int META_COLS = kTmemCols - 2 * BN;
    static_assert(B_SUB % 1024 == 0, "X half tile must keep the swizzle alignment");
    static_assert(BN % 32 == 0 && BN <= 256, "token tile");
};

// BUILD (with RES, sparse target): the weights are not stored in the tensor core's form (packed 4-bit codes, 1:4, 2:8,
// 1:8).  Instead of a TMA copy, eight builder warps rebuild the CTA's 128 weight rows for the whole reduction in the resident
// region once per output tile (xform.cuh: widening, placement into 2-of-4 slots), and the metadata warps derive the
// hardware metadata from the canonical one; everything else is the resident-weight kernel.
template <bool SPARSE, int BN, int EPI, bool RES, bool BUILD = false>
__global__ void __launch_bounds__(kPairThreadsFor<EPI, RES, BUILD>, 1)
nm_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                    const __grid_constant__ CUtensorMap tmap_y, const GemmParams p,
                    const __grid_constant__ PairSchedule sched) {
    using Cfg = PairCfg<SPARSE, BN, RES>;
    constexpr int S = Cfg::STAGES;
    constexpr int EW = kPairEpiWarps<EPI, RES, BUILD>, kGateWarp = 2 + kEpiWarps;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* a_res = smem + S * Cfg::STAGE;  // resident weight rows: kPairResStages stages of A_BYTES
    uint8_t* store_stage = a_res + Cfg::A_RES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(store_stage + Cfg::STORE_STAGE);
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };              // used in the leader
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };       // both CTAs (multicast commit)
    auto acc_full_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };   // both CTAs (multicast commit)
    auto acc_empty_bar = [&](int b) { return bar0 + 8u * (2 * S + 2 + b); };  // leader; arrivals from both
    const uint32_t meta_bar = bar0 + 8u * (2 * S + 4);                 // leader; arrivals from both
    const uint32_t drained_bar = bar0 + 8u * (2 * S + 5);
    const uint32_t a_full_bar = bar0 + 8u * (2 * S + 6);               // leader: resident weights of both CTAs landed
    const uint32_t a_free_bar = bar0 + 8u * (2 * S + 7);               // both CTAs (multicast commit): no MMA reads them any more
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 8);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* never_flag = tmem_slot + 2;
    uint32_t* lut = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(bars) + 512);  // BUILD: slot tables (xform.cuh)
    static_assert(!BUILD || (RES && SPARSE), "weights are rebuilt only in the resident-weight, sparse-target form");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const bool leader = rank == 0;
    const int pair = blockIdx.x >> 1;
    const int tile_begin = sched.start[pair];
    const int tile_count = sched.start[pair + 1] - tile_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { ptx::mbar_init(acc_full_bar(b), 1); ptx::mbar_init(acc_empty_bar(b), 2 * EW); }
        ptx::mbar_init(meta_bar, 8);
        ptx::mbar_init(drained_bar, 1);
        ptx::mbar_init(a_full_bar, BUILD ? 2 * kPairBuildWarps : 1);  // the builder warps of both CTAs, or the TMA bytes
        ptx::mbar_init(a_free_bar, 1);
        *abort_flag = 0;
        *never_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_w);
        ptx::prefetch_tensormap(&tmap_x);
        if (p.tma_store) ptx::prefetch_tensormap(&tmap_y);
    }
    if (BUILD) xf::build_lut(lut, threadIdx.x, blockDim.x);
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
    // Set-up above overlaps the tail of the kernel before this one in the stream (when launched as its
    // programmatic dependent); nothing in global memory is read or written before this point.
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    auto raise_timeout = [&]() {  // both CTAs of the pair stop: the peer's roles see the flag in their own shared memory
        *abort_flag = 1;
        ptx::st_cluster_u32(ptx::map_to_cta(ptx::smem_u32(const_cast<uint32_t*>(abort_flag)), rank ^ 1u), 1u);
        if (p.status) atomicOr(p.status, NM_STATUS_TIMEOUT);
    };

    if (warp == 0) {
        // ------------------------------ TMA producer (both CTAs) --------------------------------
        if (lane == 0) {
            uint32_t it = 0, free_parity = 1u;  // nothing reads the resident region before the first load
            int prev_out_tile = -1;
            bool ok = true;
            const uint64_t keep = ptx::policy_evict_last();  // X is read again for every output tile
            for (int i = 0; i < tile_count && ok; ++i) {
                const int tile = tile_begin + i;
                const TileCoord tc = tile_coord(tile, p.n_tok_tiles, p.n_out_tiles, p.band);
                const int n0 = tc.o * (2 * kBM) + (int)rank * kBM;
                const int t0 = tc.t * BN + (int)rank * Cfg::B_ROWS;
                if (RES && !BUILD && tc.o != prev_out_tile) {
                    // new output tile: once the MMAs of the previous one are done, fetch this CTA's weight rows for the whole reduction
                    prev_out_tile = tc.o;
                    if (!ptx::mbar_wait_bounded(a_free_bar, free_parity, abort_flag, kWaitLimit)) {
                        raise_timeout(); ok = false; break;
                    }
                    free_parity ^= 1u;
                    const uint32_t lead_a_full = ptx::map_to_cta(a_full_bar, 0);
                    if (leader) ptx::mbar_expect_tx(a_full_bar, 2 * p.kblocks * Cfg::A_BYTES);  // bytes of both CTAs
                    for (int kb = 0; kb < p.kblocks; ++kb)
                        ptx::tma_load_2d_pair(ptx::smem_u32(a_res + kb * Cfg::A_BYTES), &tmap_w, kb * Cfg::A_ROW, n0, lead_a_full);
                }
                for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                    const int s = it % S;
                    if (!ptx::mbar_wait_bounded(empty_bar(s), ((it / S) & 1u) ^ 1u, abort_flag, kWaitLimit)) {
                        raise_timeout(); ok = false; break;
                    }
                    NM_TRACE_STAGE(it, 0);
                    if (NM_SKIP_STAGE(it)) continue;
                    const uint32_t a_dst = ptx::smem_u32(smem + s * Cfg::STAGE);
                    const uint32_t lead_full = ptx::map_to_cta(full_bar(s), 0);
                    if (leader) ptx::mbar_expect_tx(full_bar(s), 2 * Cfg::STAGE);  // bytes of both CTAs
                    if (!RES) ptx::tma_load_2d_pair(a_dst, &tmap_w, kb * Cfg::A_ROW, n0, lead_full);
                    // X is mapped as [k-slice][token][128 bytes]: both slices of the stage in one operation
                    ptx::tma_load_3d_pair_hint(a_dst + Cfg::B_OFF, &tmap_x, 0, t0, kb * (Cfg::KB / 128), lead_full, keep);
                    NM_TRACE_STAGE(it, 1);
                }
            }
            // After an expired wait (here or anywhere in the pair) the MMA thread runs through its remaining steps without
            // waiting for data, so the stages' barriers no longer say whether this producer's last copies have landed:
            // give them time before the CTA and its shared memory go away.
            if (!ok || *abort_flag) ptx::wait_clocks(kAbortDrain);
        }
    } else if (BUILD && warp > kGateWarp) {
        // ------------------------------ weight builders (both CTAs) ------------------------------
        // One thread = one of the CTA's 128 weight rows; group g builds the 128-wide k-blocks g, g + 2, ... of the row
        // into the resident region (two k-blocks per 128-byte row of a stage), once per output tile.
        const int bw = warp - (kGateWarp + 1), grp = bw >> 2, tr = (bw & 3) * 32 + lane;
        const int cb = xf::code_bytes(p.pat), mb = xf::meta_bytes(p.pat);
        const uint8_t* meta8 = reinterpret_cast<const uint8_t*>(p.meta);
        const int kb_real = p.in >> 7, kb_all = 2 * p.kblocks;  // k-blocks of the reduction / of the stages (a last half stage gets zeros)
        const uint32_t lead_a_full = ptx::map_to_cta(a_full_bar, 0);
        int prev_out_tile = -1;
        uint32_t free_parity = 1u;  // nothing reads the region before the first build
        for (int i = 0; i < tile_count; ++i) {
            const int out_tile = tile_coord(tile_begin + i, p.n_tok_tiles, p.n_out_tiles, p.band).o;
            if (out_tile == prev_out_tile) continue;
            prev_out_tile = out_tile;
            const int n = out_tile * (2 * kBM) + (int)rank * kBM + tr;
            const bool row_ok = n < p.out;
            const uint8_t* v = p.values + (size_t)(row_ok ? n : 0) * p.vrow_bytes;
            const uint8_t* m = meta8 + (size_t)(row_ok ? n : 0) * p.mrow_bytes;
            xf::Raw cur = xf::load_raw(p.pat, v + (size_t)grp * cb, m + (size_t)grp * mb, row_ok && grp < kb_real);
            // the MMAs of the previous output tile have finished reading the region
            bool got = lane != 0 || ptx::mbar_wait_bounded(a_free_bar, free_parity, abort_flag, kWaitLimit);
            free_parity ^= 1u;
            if (!__all_sync(0xffffffffu, got)) { if (lane == 0) raise_timeout(); break; }
            for (int kb = grp; kb < kb_all; kb += 2) {
                const int nkb = kb + 2;
                xf::Raw nxt = xf::load_raw(p.pat, v + (size_t)nkb * cb, m + (size_t)nkb * mb, row_ok && nkb < kb_real);
                uint32_t w[16];
                xf::build_row<true>(p.pat, cur, lut, w);
                xf::store_half_row128(a_res + (kb >> 1) * Cfg::A_BYTES, tr, kb & 1, w);
                cur = nxt;
            }
            ptx::fence_proxy_async_smem();  // the MMA reads the tile through the async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(lead_a_full);
        }
    } else if (warp == kGateWarp) {
        // ------------------------------ gate (leader): mbarrier waits relayed to the MMA warp ------
        if (leader) {
            uint32_t it = 0, meta_phase = 0, a_phase = 0;
            int prev_out_tile = -1;
            bool ok = true;
            auto wait = [&](uint32_t bar, uint32_t parity) {
                if (lane == 0 && ok && !ptx::mbar_wait_bounded(bar, parity, abort_flag, kWaitLimit)) {
                    raise_timeout();
                    ok = false;
                }
            };
            for (int i = 0; i < tile_count; ++i) {
                const int tile = tile_begin + i, out_tile = tile_coord(tile, p.n_tok_tiles, p.n_out_tiles, p.band).o, buf = i & 1;
                if (out_tile != prev_out_tile) {
                    if (SPARSE) { wait(meta_bar, meta_phase); meta_phase ^= 1u; }
                    if (RES) { wait(a_full_bar, a_phase); a_phase ^= 1u; }
                    prev_out_tile = out_tile;
                }
                wait(acc_empty_bar(buf), ((i >> 1) & 1u) ^ 1u);
                for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                    wait(full_bar(it % S), (it / S) & 1u);
                    if (lane == 0) NM_TRACE_STAGE(it, 2);
                    __syncwarp();
                    ptx::relay_step(1 + (it & 7u), abort_flag);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (leader) --------------------------------------
        if (leader) {
            constexpr uint32_t idesc = ptx::idesc_i8(2 * kBM, BN, SPARSE);
            uint32_t it = 0;
            for (int i = 0; i < tile_count; ++i) {
                const int buf = i & 1;
                const uint32_t d_tmem = tmem_base + buf * BN;
                const bool last_of_out_tile = RES && (tile_begin + i + 1 >= p.n_tiles ||
                    tile_coord(tile_begin + i + 1, p.n_tok_tiles, p.n_out_tiles, p.band).o != tile_coord(tile_begin + i, p.n_tok_tiles, p.n_out_tiles, p.band).o);
                for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                    const int s = it % S;
                    ptx::named_bar_sync(1 + (it & 7u), 64);
                    if (kb == 0) ptx::tc_fence_after();  // once per tile (see the one-CTA kernel)
                    if (lane == 0) {
                        NM_TRACE_STAGE(it, 3);
                        const uint32_t st_addr = ptx::smem_u32(smem + s * Cfg::STAGE), b_addr = st_addr + Cfg::B_OFF;
                        const uint32_t a_addr = RES ? ptx::smem_u32(a_res + kb * Cfg::A_BYTES) : st_addr;
                        if constexpr (SPARSE) {
#pragma unroll
                            for (int j = 0; j < 4; ++j)  // 64 reduction elements each: 32 stored bytes of A, 64 of X
                                ptx::mma_sp_i8_pair(d_tmem, ptx::smem_desc_kmajor(a_addr + 32 * j, 128, ptx::kSwizzle128),
                                                    ptx::smem_desc_kmajor(b_addr + (j >> 1) * Cfg::B_SUB + 64 * (j & 1), 128, ptx::kSwizzle128),
                                                    tmem_base + Cfg::META_COL + kb * 8 + 2 * j, idesc, (kb | j) != 0);
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                ptx::mma_i8_pair(d_tmem, ptx::smem_desc_kmajor(a_addr + 32 * j, 128, ptx::kSwizzle128),
                                                 ptx::smem_desc_kmajor(b_addr + 32 * j, 128, ptx::kSwizzle128), idesc, (kb | j) != 0);
                        }
                        ptx::tc_commit_pair(empty_bar(s), 3);   // both producers may refill the stage
                        if (kb == p.kblocks - 1) {
                            ptx::tc_commit_pair(acc_full_bar(buf), 3);
                            if (last_of_out_tile) ptx::tc_commit_pair(a_free_bar, 3);  // both producers may replace the weights
                        }
                        NM_TRACE_STAGE(it, 4);
                    }
                    __syncwarp();
                }
            }
            if (lane == 0) {
                ptx::tc_commit_pair(drained_bar, 1);
                ptx::mbar_wait_bounded(drained_bar, 0, never_flag, kWaitLimit);
            }
        }
    } else {
        // ------------------------------ metadata + epilogue warps (both CTAs) ----------------------
        constexpr int EWH = EW / 4, CH = BN / 32, CI = (CH + EWH - 1) / EWH;
        const int ew = warp - 2 - (warp > kGateWarp ? 1 : 0), q = warp & 3, half = ew >> 2, row = q * 32 + lane;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        constexpr int NB = Cfg::STORE_BUFS;
        float* my_stage = reinterpret_cast<float*>(store_stage + ew * (NB * 2048));
        const float sx = p.sx_dev ? *p.sx_dev : p.sx_host;
        const uint32_t lead_meta = ptx::map_to_cta(meta_bar, 0);
        float amax = 0.0f, c_n = 0.0f, b_n = 0.0f;
        const float rsy = EPI == EPI_Q8 ? __frcp_rn(p.sy) : 0.0f;
        int scaled_out_tile = -1;
        uint32_t n_stores = 0;
        bool ok = true;

        auto load_meta = [&](int out_tile) {
            const int n = out_tile * (2 * kBM) + (int)rank * kBM + row;
            const uint4* src = reinterpret_cast<const uint4*>(p.meta + (size_t)n * p.mrow_words);
            // A stage spans KB reduction elements; when the reduction ends inside the last stage (in % KB != 0)
            // its remaining MMAs multiply zero-filled weights, but their index fields must still be valid 2:4
            // patterns: the columns past the row's metadata get "positions 0,1", as rows past `out` do.
            for (int c = 0; c < p.kblocks * (Cfg::KB / 32); c += 4) {
                uint4 w = make_uint4(0x44444444u, 0x44444444u, 0x44444444u, 0x44444444u);
                if (n < p.out && c < p.mrow_words) {
                    if constexpr (BUILD) w = xf::hw_meta(p.pat, reinterpret_cast<const uint8_t*>(p.meta) + (size_t)n * p.mrow_bytes + (size_t)(c >> 2) * xf::meta_bytes(p.pat), lut);
                    else w = __ldg(src + (c >> 2));
                }
                ptx::tmem_st_32x4(lane_taddr + Cfg::META_COL + c, w.x, w.y, w.z, w.w);
            }
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(lead_meta);
        };
        auto release_acc = [&](int buf) {
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(acc_empty_bar(buf), 0));
        };
        const uint64_t stream_out = ptx::policy_evict_first();  // Y is written once and not read here

        NM_TRACE_EPI_DECL;
        for (int i = 0; i < tile_count && ok; ++i) {
            const TileCoord tc = tile_coord(tile_begin + i, p.n_tok_tiles, p.n_out_tiles, p.band);
            const int out_tile = tc.o, tok_tile = tc.t, buf = i & 1;
            const int n0 = out_tile * (2 * kBM) + (int)rank * kBM, n = n0 + row, t0 = tok_tile * BN;
            if (SPARSE && i == 0 && half == 0) load_meta(out_tile);
            bool got = ptx::mbar_wait_bounded(acc_full_bar(buf), (i >> 1) & 1u, abort_flag, kWaitLimit);
            ok = __all_sync(0xffffffffu, got);
            if (!ok && lane == 0) raise_timeout();
            if constexpr (kNarrow<EPI>) ok = ptx::named_bar_and(EW == 16 ? kNarrowGroup + half : kNarrowAgree + half, 128, ok);  // the group stops together
            if (!ok) break;
            ptx::tc_fence_after();
            if (ew == 0 && lane == 0) NM_TRACE_TILE(i, 0);
            NM_TRACE_EPI_MARK();
            // the next tile starts a new output tile: its metadata can go in now, the MMAs of this one are done
            if (SPARSE && half == 0 && i + 1 < tile_count) {
                const int next_out_tile = tile_coord(tile_begin + i + 1, p.n_tok_tiles, p.n_out_tiles, p.band).o;
                if (next_out_tile != out_tile) load_meta(next_out_tile);
            }
            const bool n_ok = n < p.out;
            if (EPI != EPI_ACC && out_tile != scaled_out_tile) {  // channel constants: fetched once per output tile
                scaled_out_tile = out_tile;
                c_n = n_ok ? __fmul_rn(sx, p.sw[n]) : 0.0f;
                b_n = n_ok && p.bias ? p.bias[n] : 0.0f;
            }
            if constexpr (EW == 16) {
                // Four groups of four warps (one per TMEM lane quarter); group g takes the 16-token units g, g + 4, ... of the
                // tile: reads 16 accumulator columns, fills its quarter of the group's [16 tokens][128 channels] staging tile
                // (two per group, used alternately), and the group's warp of lane quarter 0 issues the store.
                using OT = typename EpiOut<EPI>::type;
                constexpr int UNITS = BN / 16;
                const int nunits = min(UNITS, (p.tokens - t0 + 15) >> 4);  // units that hold tokens (the same for the whole group)
                const uint32_t gbar = kNarrowGroup + half;
                bool released = false;
#pragma unroll 1
                for (int u = half; u < nunits; u += 4) {
                    const int tc0 = t0 + 16 * u;
                    uint32_t r[16];
                    ptx::tmem_ld_32x16(lane_taddr + buf * BN + 16 * u, r);
                    ptx::tmem_ld_wait();
                    NM_TRACE_EPI_ADD(0);
                    if (u + 4 >= nunits) { release_acc(buf); released = true; }
                    if (p.tma_store) {
                        OT* sb = reinterpret_cast<OT*>(store_stage) + (half * 2 + (n_stores & 1u)) * (16 * 128);
                        if (q == 0 && lane == 0) ptx::bulk_wait_group_read<1>();  // the store before the last has read this tile
                        ptx::named_bar_sync(gbar, 128);
                        NM_TRACE_EPI_ADD(1);
                        if constexpr (EPI == EPI_Q8) {
                            float worst = 0.0f;
#pragma unroll
                            for (int j = 0; j < 16; ++j) sb[j * 128 + q * 32 + lane] = epi_convert_q8_fast(r[j], c_n, b_n, rsy, worst);
                            if (__any_sync(0xffffffffu, !(worst <= 0.49996948f))) {  // rare (3 % of the runs)
                                // find the values in question again; the exact division decides those
#pragma unroll
                                for (int j = 0; j < 16; ++j) {
                                    float w1 = 0.0f;
                                    (void)epi_convert_q8_fast(r[j], c_n, b_n, rsy, w1);
                                    if (!(w1 <= 0.49996948f))
                                        sb[j * 128 + q * 32 + lane] =
                                            (uint8_t)(int8_t)quantise8_exact_call(__fmaf_rn((float)(int)r[j], c_n, b_n), p.sy);
                                }
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                float y_abs;
                                sb[j * 128 + q * 32 + lane] = epi_convert<EPI>(r[j], c_n, b_n, p.sy, rsy, y_abs);
                            }
                        }
                        NM_TRACE_EPI_ADD(2);
                        ptx::fence_proxy_async_smem();
                        ptx::named_bar_sync(gbar, 128);
                        NM_TRACE_EPI_ADD(3);
                        if (q == 0 && lane == 0) {
                            ptx::tma_store_2d_hint(&tmap_y, n0, tc0, ptx::smem_u32(sb), stream_out);
                            ptx::bulk_commit_group();
                        }
                        NM_TRACE_EPI_ADD(4);
                        ++n_stores;
                    } else {
                        const int jmax = n_ok ? min(16, p.tokens - tc0) : 0;  // outputs of this lane that exist
                        OT* dst = reinterpret_cast<OT*>(p.NARROW) + (size_t)tc0 * p.out + n;
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            float y_abs;
                            const OT o = epi_convert<EPI>(r[j], c_n, b_n, p.sy, rsy, y_abs);
                            if (j < jmax) dst[(size_t)j * p.out] = o;
                        }
                    }
                }
                if (!released) release_acc(buf);
                if (ew == 0 && lane == 0) { NM_TRACE_TILE(i, 1); NM_TRACE_EPI_FLUSH(i); }
                continue;
            }
            const int nact = min(CH, (p.tokens - t0 + 31) >> 5);
            // chunks are read one ahead of their conversion; with the builder warps present registers are short and
            // every chunk is read when it is due
            constexpr int RB = (BUILD || kNarrow<EPI>) ? 1 : 2;  // narrow outputs: see the one-CTA kernel
            uint32_t r[RB][32];
            if (half >= nact) release_acc(buf);
            else if (RB == 2) ptx::tmem_ld_32x32(lane_taddr + buf * BN + half * 32, r[0]);
#pragma unroll (kNarrow<EPI> ? 1 : CI)
            for (int ci = 0; ci < CI; ++ci) {
                const int c = half + ci * EWH, tc0 = t0 + c * 32;
                if (c < nact) {
                    if (RB == 1) ptx::tmem_ld_32x32(lane_taddr + buf * BN + c * 32, r[0]);
                    ptx::tmem_ld_wait();
                    NM_TRACE_EPI_ADD(0);
                    if (c + EWH >= nact) release_acc(buf);
                    else if (RB == 2) ptx::tmem_ld_32x32(lane_taddr + buf * BN + (c + EWH) * 32, r[(ci + 1) & (RB - 1)]);
                    const int jmax = n_ok ? min(32, p.tokens - tc0) : 0;  // outputs of this lane that exist
                    using OT = typename EpiOut<EPI>::type;
                    auto conv = [&](int j) -> OT {
                        float y_abs;
                        const OT o = epi_convert<EPI>(r[ci & (RB - 1)][j], c_n, b_n, p.sy, rsy, y_abs);
                        if constexpr (EPI == EPI_F32) amax = fmaxf(amax, j < jmax ? y_abs : 0.0f);
                        return o;
                    };
                    if (p.tma_store) {  // separate branch-free loops for the two store paths
#pragma unroll
                        for (int h = 0; h < 2; ++h) {  // 16 tokens per store, alternating staging tiles
                            if (tc0 + 16 * h >= p.tokens) continue;  // warp-uniform (and the same in all warps of a group)
                            if constexpr (kNarrow<EPI>) {  // one [16 tokens][128 channels] tile per four warps
                                OT* sb = reinterpret_cast<OT*>(store_stage) + (half * 2 + (n_stores & 1u)) * (16 * 128);
                                if (q == 0 && lane == 0) ptx::bulk_wait_group_read<1>();  // the store before the last has read this tile
                                ptx::named_bar_sync(kNarrowFree + half, 128);
                                NM_TRACE_EPI_ADD(1);
                                if constexpr (EPI == EPI_Q8) {
                                    float worst = 0.0f;
#pragma unroll
                                    for (int j = 0; j < 16; ++j)
                                        sb[j * 128 + q * 32 + lane] = epi_convert_q8_fast(r[ci & (RB - 1)][16 * h + j], c_n, b_n, rsy, worst);
                                    if (__any_sync(0xffffffffu, !(worst <= 0.49996948f))) {  // rare (3 % of the runs)
                                        // find the values in question again; the exact division decides those
#pragma unroll
                                        for (int j = 0; j < 16; ++j) {
                                            float w1 = 0.0f;
                                            (void)epi_convert_q8_fast(r[ci & (RB - 1)][16 * h + j], c_n, b_n, rsy, w1);
                                            if (!(w1 <= 0.49996948f))
                                                sb[j * 128 + q * 32 + lane] = (uint8_t)(int8_t)quantise8_exact_call(
                                                    __fmaf_rn((float)(int)r[ci & (RB - 1)][16 * h + j], c_n, b_n), p.sy);
                                        }
                                    }
                                } else {
#pragma unroll
                                    for (int j = 0; j < 16; ++j) sb[j * 128 + q * 32 + lane] = conv(16 * h + j);
                                }
                                NM_TRACE_EPI_ADD(2);
                                ptx::fence_proxy_async_smem();
                                ptx::named_bar_sync(kNarrowFull + half, 128);
                                NM_TRACE_EPI_ADD(3);
                                if (q == 0 && lane == 0) {
                                    ptx::tma_store_2d(&tmap_y, n0, tc0 + 16 * h, ptx::smem_u32(sb));
                                    ptx::bulk_commit_group();
                                }
                                NM_TRACE_EPI_ADD(4);
                                ++n_stores;
                            } else {
                                OT* sb = reinterpret_cast<OT*>(my_stage + (NB == 2 ? (n_stores & 1u) * 512 : 0));
                                if (lane == 0) ptx::bulk_wait_group_read<NB - 1>();  // the store that last used this tile has read it
                                __syncwarp();
                                NM_TRACE_EPI_ADD(1);
#pragma unroll
                                for (int j = 0; j < 16; ++j) sb[j * 32 + lane] = conv(16 * h + j);
                                NM_TRACE_EPI_ADD(2);
                                ptx::fence_proxy_async_smem();
                                __syncwarp();
                                NM_TRACE_EPI_ADD(3);
                                if (lane == 0) {
                                    ptx::tma_store_2d_hint(&tmap_y, n0 + q * 32, tc0 + 16 * h, ptx::smem_u32(sb), stream_out);
                                    ptx::bulk_commit_group();
                                }
                                NM_TRACE_EPI_ADD(4);
                                ++n_stores;
                            }
                        }
                    } else {
                        OT* dst = reinterpret_cast<OT*>(EPI == EPI_F32 ? (void*)p.Y : EPI == EPI_ACC ? (void*)p.ACC : p.NARROW) + (size_t)tc0 * p.out + n;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const OT o = conv(j);
                            if (j < jmax) dst[(size_t)j * p.out] = o;
                        }
                    }
                }
            }
            if (ew == 0 && lane == 0) { NM_TRACE_TILE(i, 1); NM_TRACE_EPI_FLUSH(i); }
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

#include "gemm_wide.cuh"

namespace nm {

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
// Kernel-choice overrides for measurements and tests (nm_debug_set_option); all zero = the library's own choice.
struct DebugOptions {
    int no_pdl;       // launch without the programmatic-dependent-launch attribute
    int no_pair;      // one-CTA kernels only
    int no_resident;  // always stream the weights through the stage ring
    int no_wide;      // never the 512-channel pair kernel
    int wide_any;     // the 512-channel pair kernel whenever the shape allows it, however few tiles there are
    int wide_bn;      // token-tile width of that kernel: 224 or 192 (0 = automatic)
    int band;         // band size of the streamed pair kernel's tile order (0 = automatic)
    int skip_stage;   // NM_TEST_HOOKS builds: 1 + the pipeline stage CTA 0's producer leaves out (0 = none)
};
static DebugOptions g_opt = {0, 0, 0, 0, 0, 0, 0, 0};

// Trace buffer of NM_TRACE builds (device, kTraceStages + kTraceTiles rows of 8 u64), handed to every GEMM launch.
static unsigned long long* g_trace_buffer = nullptr;

// cudaFuncSetAttribute(max dynamic shared memory) once per kernel and device instead of on every launch.
static cudaError_t allow_dynamic_smem(const void* fn, int bytes) {
    struct Done { const void* fn; int dev; };
    static Done done[64];
    static int n_done = 0;
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_done; ++i)
        if (done[i].fn == fn && done[i].dev == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && n_done < 64) done[n_done++] = Done{fn, dev};
    return e;
}

struct LinearArgs {
    const int8_t* X; int tokens; const nm_packed_t* W;
    float sx; const float* sx_dev; const float* sw; const float* bias;
    float* Y; int32_t* ACC; float* absmax; uint32_t* status; cudaStream_t stream;
    void* NARROW = nullptr; float sy = 1.0f;
};

// Tensor map of the output for the epilogue's TMA stores ([16 tokens][32 channels] boxes).  The epilogue stores
// through TMA when the output can be described by a tensor map (16-byte aligned base and row pitch);
// otherwise *tma_store is cleared, the threads store directly and the map describes X as a stand-in.
template <int EPI>
static int make_store_map(CUtensorMap* ty, const LinearArgs& a, bool* tma_store, uint32_t box_rows = 16, uint32_t box_cols = 0) {
    const nm_packed_t& W = *a.W;
    constexpr uint32_t es = (uint32_t)sizeof(typename EpiOut<EPI>::type);
    void* ybase = EPI == EPI_F32 ? (void*)a.Y : EPI == EPI_ACC ? (void*)a.ACC : a.NARROW;
    *tma_store = aligned(ybase, 16) && ((size_t)W.out * es) % 16 == 0;
    const CUtensorMapDataType dt = EPI == EPI_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : EPI == EPI_ACC ? CU_TENSOR_MAP_DATA_TYPE_INT32
                                 : EPI == EPI_Q8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    if (!*tma_store)
        return make_map(ty, a.X, (uint64_t)a.tokens, (uint64_t)W.in / 4, 16, 32, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_DATA_TYPE_INT32, 4);
    return make_map(ty, ybase, (uint64_t)a.tokens, (uint64_t)W.out, box_rows, box_cols ? box_cols : (kNarrow<EPI> ? 128 : 32), CU_TENSOR_MAP_SWIZZLE_NONE, dt, es);
}

template <bool SPARSE, int BN, int EPI, int WSRC>
static int launch_gemm(const LinearArgs& a) {
    constexpr bool XF = WSRC != W_TMA;
    using Cfg = GemmCfg<SPARSE, BN, WSRC == W_RESIDENT>;
    const nm_packed_t& W = *a.W;
    CUtensorMap tw, tx, ty;
    // transform modes build the weight tile in shared memory and never use this map: describe X instead
    int rc = XF ? make_map(&tw, a.X, (uint64_t)a.tokens, (uint64_t)W.in, BN, 128, CU_TENSOR_MAP_SWIZZLE_128B)
                : make_map(&tw, W.values, (uint64_t)W.out, (uint64_t)(SPARSE ? W.in / 2 : W.in), kBM, Cfg::A_ROW,
                           SPARSE ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != NM_OK) return rc;
    rc = make_map(&tx, a.X, (uint64_t)a.tokens, (uint64_t)W.in, BN, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != NM_OK) return rc;
    bool tma_store = false;
    rc = make_store_map<EPI>(&ty, a, &tma_store);
    if (rc != NM_OK) return rc;
    GemmParams p{};
    p.tma_store = tma_store ? 1 : 0;
    p.tokens = a.tokens; p.out = W.out; p.in = W.in;
    p.n_tok_tiles = (a.tokens + BN - 1) / BN;
    p.n_tiles = p.n_tok_tiles * ((W.out + kBM - 1) / kBM);
    p.kblocks = W.in / kKB;
    p.meta = (const uint32_t*)W.meta; p.mrow_words = W.in / 32;  // hardware metadata words per row (4 per k-block)
    p.values = (const uint8_t*)W.values;
    p.vrow_bytes = (int)values_row_bytes(W.in, W.n, W.m, W.bits);
    p.mrow_bytes = (int)meta_row_words(W.in, W.n, W.m) * 4;
    p.pat = xf::pattern_of(W.n, W.m, W.bits);
    p.sw = a.sw; p.bias = a.bias; p.sx_dev = a.sx_dev; p.sx_host = a.sx;
    p.Y = a.Y; p.ACC = a.ACC; p.NARROW = a.NARROW; p.sy = a.sy; p.absmax = a.absmax; p.status = a.status; p.trace = g_trace_buffer; p.skip_stage = g_opt.skip_stage - 1;
    auto fn = nm_gemm_kernel<SPARSE, BN, EPI, WSRC>;
    NM_CUDA_TRY(allow_dynamic_smem((const void*)fn, Cfg::SMEM));
    const int grid = p.n_tiles < sm_count() ? p.n_tiles : sm_count();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(XF ? kXformThreads : kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM;
    cfg.stream = a.stream;
    // as for the pair kernel: set-up may overlap the previous kernel's tail, global memory waits for it
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = g_opt.no_pdl ? 0 : 1;
    NM_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, tw, tx, ty, p));
    return NM_OK;
}

// The plan costs a pass over all tiles on the host; layers are launched again and again with the same shape, so
// the last few plans are kept.
static int cached_pair_plan(int n_tok_tiles, int n_out_tiles, int pairs, bool resident, int band_request, PairSchedule& out) {
    struct Entry { int key[5]; int band; PairSchedule sched; bool used; };
    static Entry cache[8];
    static unsigned next = 0;
    static std::mutex mu;
    const int key[5] = {n_tok_tiles, n_out_tiles, pairs, resident ? 1 : 0, band_request};
    std::lock_guard<std::mutex> lock(mu);
    for (Entry& e : cache)
        if (e.used && std::equal(key, key + 5, e.key)) { out = e.sched; return e.band; }
    Entry& e = cache[next++ % 8];
    std::copy(key, key + 5, e.key);
    e.band = plan_pair_tiles(n_tok_tiles, n_out_tiles, pairs, resident, band_request, e.sched.start);
    e.used = true;
    out = e.sched;
    return e.band;
}

template <bool SPARSE, int BN, int EPI, bool RES, bool BUILD = false>
static int launch_gemm_pair(const LinearArgs& a) {
    using Cfg = PairCfg<SPARSE, BN, RES>;
    const nm_packed_t& W = *a.W;
    CUtensorMap tw, tx, ty;
    // rebuilt weights are read by the builder warps, not by TMA: the weight map then describes X as a stand-in
    int rc = BUILD ? make_map(&tw, a.X, (uint64_t)a.tokens, (uint64_t)W.in, kBM, 128, CU_TENSOR_MAP_SWIZZLE_128B)
                   : make_map(&tw, W.values, (uint64_t)W.out, (uint64_t)(SPARSE ? W.in / 2 : W.in), kBM, Cfg::A_ROW,
                              CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != NM_OK) return rc;
    rc = make_map_x3(&tx, a.X, (uint64_t)a.tokens, (uint64_t)W.in, Cfg::B_ROWS, Cfg::KB / 128);
    if (rc != NM_OK) return rc;
    bool tma_store = false;
    rc = make_store_map<EPI>(&ty, a, &tma_store);
    if (rc != NM_OK) return rc;
    GemmParams p{};
    p.tma_store = tma_store ? 1 : 0;
    p.tokens = a.tokens; p.out = W.out; p.in = W.in;
    p.n_tok_tiles = (a.tokens + BN - 1) / BN;
    p.n_out_tiles = (W.out + 2 * kBM - 1) / (2 * kBM);
    p.n_tiles = p.n_tok_tiles * p.n_out_tiles;
    p.kblocks = (W.in + Cfg::KB - 1) / Cfg::KB;
    p.meta = (const uint32_t*)W.meta; p.mrow_words = W.in / 32;
    p.values = (const uint8_t*)W.values;
    p.vrow_bytes = (int)values_row_bytes(W.in, W.n, W.m, W.bits);
    p.mrow_bytes = (int)meta_row_words(W.in, W.n, W.m) * 4;
    p.pat = xf::pattern_of(W.n, W.m, W.bits);
    p.sw = a.sw; p.bias = a.bias; p.sx_dev = a.sx_dev; p.sx_host = a.sx;
    p.Y = a.Y; p.ACC = a.ACC; p.NARROW = a.NARROW; p.sy = a.sy; p.absmax = a.absmax; p.status = a.status; p.trace = g_trace_buffer; p.skip_stage = g_opt.skip_stage - 1;
    auto fn = nm_gemm_pair_kernel<SPARSE, BN, EPI, RES, BUILD>;
    NM_CUDA_TRY(allow_dynamic_smem((const void*)fn, Cfg::SMEM));
    int pairs = p.n_tiles < sm_count() / 2 ? p.n_tiles : sm_count() / 2;
    if (pairs > kMaxPairs) pairs = kMaxPairs;
    // Contiguous tile ranges of about equal cost: a tile costs 1, entering a new output tile inside a range
    // costs `crossing` tiles (weights resident: ~1, the reload waits for the MMAs to drain; streamed: metadata only).
    // Streamed weights: a change of output tile only costs the metadata, so the tiles are banded by about
    // one pair's share and neighbouring pairs share X tiles in L2.  Resident weights: long runs.
    PairSchedule sched;
    p.band = cached_pair_plan(p.n_tok_tiles, p.n_out_tiles, pairs, RES, g_opt.band, sched);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(kPairThreadsFor<EPI, RES, BUILD>, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    // the kernel's set-up may start while the previous kernel of the stream drains; it waits for that kernel
    // (griddepcontrol.wait) before its first access to global memory
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = g_opt.no_pdl ? 1 : 2;
    NM_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, tw, tx, ty, p, sched));
    return NM_OK;
}

// Wide pair kernel (512 channels x BN tokens per pair): 2:4 int8 weights streamed, fp32 / int32 outputs.
template <int BN, int EPI, bool W4 = false>
static int launch_gemm_wide(const LinearArgs& a) {
    using Cfg = WideCfg<BN>;
    constexpr int SKEW = 0;
    const nm_packed_t& W = *a.W;
    CUtensorMap tw, tx, ty;
    // packed 4-bit codes are read by the builder warps, not by TMA: the weight map then describes X as a stand-in
    int rc = W4 ? make_map(&tw, a.X, (uint64_t)a.tokens, (uint64_t)W.in, Cfg::B_ROWS, 128, CU_TENSOR_MAP_SWIZZLE_128B)
                : make_map(&tw, W.values, (uint64_t)W.out, (uint64_t)W.in / 2, Cfg::A_ROWS, Cfg::A_ROW, CU_TENSOR_MAP_SWIZZLE_64B);
    if (rc != NM_OK) return rc;
    rc = make_map(&tx, a.X, (uint64_t)a.tokens, (uint64_t)W.in, Cfg::B_ROWS, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != NM_OK) return rc;
    bool tma_store = false;
    rc = make_store_map<EPI>(&ty, a, &tma_store, 32);
    if (rc != NM_OK) return rc;
    GemmParams p{};
    p.tma_store = tma_store ? 1 : 0;
    p.tokens = a.tokens; p.out = W.out; p.in = W.in;
    p.n_tok_tiles = (a.tokens + BN - 1) / BN;
    p.n_out_tiles = (W.out + 2 * Cfg::A_ROWS - 1) / (2 * Cfg::A_ROWS);
    p.n_tiles = p.n_tok_tiles * p.n_out_tiles;
    p.kblocks = W.in / Cfg::KB;
    p.meta = (const uint32_t*)W.meta; p.mrow_words = W.in / 32;
    p.values = (const uint8_t*)W.values; p.vrow_bytes = (int)values_row_bytes(W.in, W.n, W.m, W.bits);
    p.sw = a.sw; p.bias = a.bias; p.sx_dev = a.sx_dev; p.sx_host = a.sx;
    p.Y = a.Y; p.ACC = a.ACC; p.NARROW = a.NARROW; p.sy = a.sy; p.absmax = a.absmax; p.status = a.status; p.trace = g_trace_buffer; p.skip_stage = g_opt.skip_stage - 1;
    auto fn = nm_gemm_wide_kernel<BN, EPI, SKEW, W4>;
    NM_CUDA_TRY(allow_dynamic_smem((const void*)fn, Cfg::SMEM));
    int pairs = p.n_tiles < sm_count() / 2 ? p.n_tiles : sm_count() / 2;
    if (pairs > kMaxPairs) pairs = kMaxPairs;
    PairSchedule sched;
    p.band = cached_pair_plan(p.n_tok_tiles, p.n_out_tiles, pairs, false, 0, sched);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(kWideThreadsOf<W4>, 1, 1);
    cfg.dynamicSmemBytes = Cfg::SMEM;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = g_opt.no_pdl ? 1 : 2;
    NM_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, tw, tx, ty, p, sched));
    return NM_OK;
}

// Token-tile width of the wide kernel: the one whose slowest pair has the least to do (tiles per pair, rounded
// up, times the tile width); 0 = the wide kernel does not apply (short reductions keep their weights resident in
// the 256-channel kernel; a matrix of at most 256 channels would leave one of the two blocks idle; narrow outputs
// and small problems stay on the other kernels).
template <int EPI>
static int wide_bn(const LinearArgs& a) {
    if (g_opt.no_wide || g_opt.no_pair) return 0;
    const nm_packed_t& W = *a.W;
    if (W.in <= kPairResStages * PairCfg<true, 192>::KB || W.out <= 2 * kBM) return 0;
    const long long pairs = sm_count() / 2, out_tiles = (W.out + 4 * kBM - 1) / (4 * kBM);
    int best = 0;
    long long best_cost = 0;
    for (int bn : {224, 192}) {
        if (g_opt.wide_bn && bn != g_opt.wide_bn) continue;
        const long long tiles = out_tiles * ((a.tokens + bn - 1) / bn);
        if (2 * tiles < pairs && !g_opt.wide_any) continue;  // measured: with half the pairs busy it still beats the 256-channel kernel
        const long long cost = ((tiles + pairs - 1) / pairs) * bn;
        if (!best || cost < best_cost) { best = bn; best_cost = cost; }
    }
    return best;
}

// The pair kernel pays off when there is enough work for every SM pair; small problems stay on one CTA.
template <bool SPARSE, int EPI>
static bool use_pair(const LinearArgs& a) {
    if (g_opt.no_pair) return false;
    const long long tiles = (long long)((a.W->out + 2 * kBM - 1) / (2 * kBM)) * ((a.tokens + 191) / 192);
    const bool fits = !SPARSE || a.W->in / 32 <= PairCfg<SPARSE, 192>::META_COLS;
    return fits && tiles >= sm_count() / 2;
}

// Pair kernel with the weights streamed through the ring, or (2:4, reduction up to 1024) kept resident.
template <bool SPARSE, int EPI>
static int pick_pair(const LinearArgs& a) {
    if constexpr (SPARSE) {
        if (a.W->in <= kPairResStages * PairCfg<true, 192>::KB && !g_opt.no_resident)
            return launch_gemm_pair<true, 192, EPI, true>(a);
    }
    return launch_gemm_pair<SPARSE, 192, EPI, false>(a);
}

template <bool SPARSE, int EPI, bool XF>
static int pick_bn(const LinearArgs& a) {
    const int out_tiles = (a.W->out + kBM - 1) / kBM, sms = sm_count();
    if constexpr (!XF) {
        const bool fits192 = !SPARSE || a.W->in / 32 <= GemmCfg<SPARSE, 192>::META_COLS;
        if (fits192 && (long long)out_tiles * ((a.tokens + 191) / 192) >= sms) return launch_gemm<SPARSE, 192, EPI, W_TMA>(a);
        if ((long long)out_tiles * ((a.tokens + 127) / 128) >= sms) return launch_gemm<SPARSE, 128, EPI, W_TMA>(a);
        return launch_gemm<SPARSE, 64, EPI, W_TMA>(a);
    } else {
        // Sparse-target formats with a short reduction and work for every SM pair: the CTA-pair kernel with the weights
        // rebuilt once per output tile into its resident region (32-bit outputs).
        if constexpr (SPARSE && (EPI == EPI_F32 || EPI == EPI_ACC)) {
            const long long pair_tiles = (long long)((a.W->out + 2 * kBM - 1) / (2 * kBM)) * ((a.tokens + 191) / 192);
            if (a.W->in <= kPairResStages * PairCfg<true, 192>::KB && pair_tiles >= sms / 2 && !g_opt.no_pair && !g_opt.no_resident)
                return launch_gemm_pair<true, 192, EPI, true, true>(a);
        }
        // Short reductions with many token tiles per output tile: build each weight tile once and keep it.
        constexpr int BNR = SPARSE ? 192 : 128;
        if (a.W->in / kKB <= kResidentKB && (long long)out_tiles * ((a.tokens + BNR - 1) / BNR) >= sms && !g_opt.no_resident)
            return launch_gemm<SPARSE, BNR, EPI, W_RESIDENT>(a);
        if constexpr (SPARSE) {  // wider token tiles: each built weight tile serves more columns
            if (a.W->in / 32 <= GemmCfg<SPARSE, 192>::META_COLS && (long long)out_tiles * ((a.tokens + 191) / 192) >= sms)
                return launch_gemm<SPARSE, 192, EPI, W_BUILD>(a);
        }
        if ((long long)out_tiles * ((a.tokens + 127) / 128) >= sms) return launch_gemm<SPARSE, 128, EPI, W_BUILD>(a);
        return launch_gemm<SPARSE, 64, EPI, W_BUILD>(a);
    }
}

static int check_linear(int tokens, int out, int in, int n, int m, int bits) {
    int rc = check_pattern(out, in, n, m, bits);
    if (rc != NM_OK) return rc;
    if (tokens < 0) return NM_ERR_SHAPE;
    if (in % kKB) return NM_ERR_SHAPE;          // reduction length: whole 128-wide k-blocks
    if (in > 8192) return NM_ERR_UNSUPPORTED;   // metadata of one output tile must fit in TMEM
    return NM_OK;
}

template <int EPI>
static int run_linear_epi(const LinearArgs& a, bool xform, bool sparse) {
    if (sparse && (!xform || xf::pattern_of(a.W->n, a.W->m, a.W->bits) == xf::P24_4)) {  // 2:4 with 8-bit or packed 4-bit codes
        const int bn = wide_bn<EPI>(a);
        if (bn == 224) return xform ? launch_gemm_wide<224, EPI, true>(a) : launch_gemm_wide<224, EPI>(a);
        if (bn == 192) return xform ? launch_gemm_wide<192, EPI, true>(a) : launch_gemm_wide<192, EPI>(a);
    }
    if (xform) return sparse ? pick_bn<true, EPI, true>(a) : pick_bn<false, EPI, true>(a);
    if (sparse) return use_pair<true, EPI>(a) ? pick_pair<true, EPI>(a) : pick_bn<true, EPI, false>(a);
    return use_pair<false, EPI>(a) ? pick_pair<false, EPI>(a) : pick_bn<false, EPI, false>(a);
}

static int run_linear(const LinearArgs& a, int epi) {
    if (!a.W) return NM_ERR_NULL;
    const nm_packed_t& W = *a.W;
    int rc = check_linear(a.tokens, W.out, W.in, W.n, W.m, W.bits);
    if (rc != NM_OK) return rc;
    const int pat = xf::pattern_of(W.n, W.m, W.bits);
    const bool xform = pat != xf::PNONE;
    const bool sparse = xform ? xf::sparse_target(pat) : W.n != W.m;  // tensor-core form of the weights
    if (!a.X || !W.values || (W.n != W.m && !W.meta)) return NM_ERR_NULL;
    if (epi != EPI_ACC && !a.sw) return NM_ERR_NULL;
    if (epi == EPI_F32 && !a.Y) return NM_ERR_NULL;
    if (epi == EPI_ACC && !a.ACC) return NM_ERR_NULL;
    if ((epi == EPI_Q8 || epi == EPI_BF16) && !a.NARROW) return NM_ERR_NULL;
    if (epi == EPI_Q8 && !(a.sy >= 1.17549435e-38f && a.sy <= 3.402823466e38f)) return NM_ERR_SHAPE;  // positive, normal, finite
    if (!aligned(a.X, 16) || !aligned(W.values, 16) || (W.meta && !aligned(W.meta, 16))) return NM_ERR_ALIGN;
    if ((a.Y && !aligned(a.Y, 4)) || (a.ACC && !aligned(a.ACC, 4))) return NM_ERR_ALIGN;
    if (epi == EPI_BF16 && !aligned(a.NARROW, 2)) return NM_ERR_ALIGN;
    if (a.tokens == 0 || W.out == 0) return NM_OK;
    switch (epi) {
        case EPI_F32: return run_linear_epi<EPI_F32>(a, xform, sparse);
        case EPI_ACC: return run_linear_epi<EPI_ACC>(a, xform, sparse);
        case EPI_Q8: return run_linear_epi<EPI_Q8>(a, xform, sparse);
        default: return run_linear_epi<EPI_BF16>(a, xform, sparse);
    }
}

}  // namespace nm

extern "C" {

int nm_pair_tile_plan(int n_tok_tiles, int n_out_tiles, int pairs, int resident, int band_request, int* start,
                      int* tile_out, int* tile_tok) {
    if (!start) return NM_ERR_NULL;
    if (n_tok_tiles < 1 || n_out_tiles < 1 || pairs < 1 || pairs > nm::kMaxPairs ||
        (long long)n_tok_tiles * n_out_tiles > 0x7fffffffll || pairs > n_tok_tiles * n_out_tiles)
        return NM_ERR_SHAPE;
    const int band = nm::plan_pair_tiles(n_tok_tiles, n_out_tiles, pairs, resident != 0, band_request, start);
    for (int t = 0; t < n_tok_tiles * n_out_tiles; ++t) {
        const nm::TileCoord c = nm::tile_coord(t, n_tok_tiles, n_out_tiles, band);
        if (tile_out) tile_out[t] = c.o;
        if (tile_tok) tile_tok[t] = c.t;
    }
    return band;
}

int nm_debug_set_option(const char* name, int value) {
    if (!name) return NM_ERR_NULL;
    struct { const char* name; int* slot; } table[] = {
        {"no_pdl", &nm::g_opt.no_pdl}, {"no_pair", &nm::g_opt.no_pair}, {"no_resident", &nm::g_opt.no_resident},
        {"no_wide", &nm::g_opt.no_wide}, {"wide_any", &nm::g_opt.wide_any}, {"wide_bn", &nm::g_opt.wide_bn},
        {"band", &nm::g_opt.band}, {"pack_form", &nm::g_pack_form}};
    for (auto& e : table)
        if (!strcmp(name, e.name)) { *e.slot = value; return NM_OK; }
#ifdef NM_TEST_HOOKS
    if (!strcmp(name, "skip_stage")) { nm::g_opt.skip_stage = value; return NM_OK; }
    if (!strcmp(name, "skip_pack_copy")) return nm::pack_set_skip_unit(value - 1);
#endif
    return NM_ERR_UNSUPPORTED;
}

int nm_debug_set_trace(unsigned long long* buffer) {
#ifdef NM_TRACE
    nm::g_trace_buffer = buffer;
    return NM_OK;
#else
    (void)buffer;
    return NM_ERR_UNSUPPORTED;
#endif
}

int nm_int_linear_check(int tokens, int out, int in, int n, int m, int bits) {
    return nm::check_linear(tokens, out, in, n, m, bits);
}

size_t nm_int_linear_workspace_bytes(int, int, int, int, int, int) { return 0; }

int nm_int_linear(const int8_t* X, int tokens, const nm_packed_t* W, float sx, const float* sw,
                  const float* bias, float* Y, void*, size_t, uint32_t* status, void* stream) {
    nm::LinearArgs a{X, tokens, W, sx, nullptr, sw, bias, Y, nullptr, nullptr, status, (cudaStream_t)stream};
    return nm::run_linear(a, nm::EPI_F32);
}

int nm_int_linear_dsx(const int8_t* X, int tokens, const nm_packed_t* W, const float* sx_dev,
                      const float* sw, const float* bias, float* Y, float* absmax_out, void*, size_t,
                      uint32_t* status, void* stream) {
    if (!sx_dev) return NM_ERR_NULL;
    nm::LinearArgs a{X, tokens, W, 0.0f, sx_dev, sw, bias, Y, nullptr, absmax_out, status, (cudaStream_t)stream};
    return nm::run_linear(a, nm::EPI_F32);
}

int nm_int_linear_q8(const int8_t* X, int tokens, const nm_packed_t* W, float sx, const float* sw,
                     const float* bias, float sy, int8_t* Yq, void*, size_t, uint32_t* status, void* stream) {
    nm::LinearArgs a{X, tokens, W, sx, nullptr, sw, bias, nullptr, nullptr, nullptr, status, (cudaStream_t)stream};
    a.NARROW = Yq; a.sy = sy;
    return nm::run_linear(a, nm::EPI_Q8);
}

int nm_int_linear_bf16(const int8_t* X, int tokens, const nm_packed_t* W, float sx, const float* sw,
                       const float* bias, uint16_t* Ybf16, void*, size_t, uint32_t* status, void* stream) {
    nm::LinearArgs a{X, tokens, W, sx, nullptr, sw, bias, nullptr, nullptr, nullptr, status, (cudaStream_t)stream};
    a.NARROW = Ybf16;
    return nm::run_linear(a, nm::EPI_BF16);
}

int nm_int_linear_acc(const int8_t* X, int tokens, const nm_packed_t* W, int32_t* ACC, void*, size_t,
                      uint32_t* status, void* stream) {
    nm::LinearArgs a{X, tokens, W, 1.0f, nullptr, nullptr, nullptr, nullptr, ACC, nullptr, status, (cudaStream_t)stream};
    return nm::run_linear(a, nm::EPI_ACC);
}

}  // extern "C"
