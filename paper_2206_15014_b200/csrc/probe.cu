// Traffic probe: replays the tile walk of the CTA-pair GEMM kernels with their TMA boxes and no arithmetic.
//
// Every CTA of a pair loads, per pipeline stage, the weight rows it would feed to the tensor core (a box of
// `a_rows` rows x `a_row_bytes`) and its half of the X tile (`b_rows` tokens x `b_slices` 128-byte-wide slices,
// through the 3-D view of X), in the same order and with the same ring of stages as the GEMM; a consumer thread
// takes each stage as soon as it has landed, optionally holds it for `delay` clocks (the time the MMAs of a
// stage would need) and hands it back; eight store warps write the CTA's share of the output tile as
// [16 tokens][32 channels] fp32 boxes from shared memory, as the GEMM's epilogue does.  What it measures is the
// ceiling the memory system sets for a given tile shape: bytes per clock per SM and TB/s over the chip when
// nothing but the copies runs.  All waits are bounded; all addresses come from tensor maps of the caller's
// buffers (out-of-range parts of a box are clipped by the hardware).
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"
#include "tileplan.cuh"

namespace nm {

struct ProbeParams {
    int a_rows, a_row_bytes, b_rows, b_slices;
    int stages, kblocks, n_tok_tiles, n_out_tiles, band, repeat, delay, loads, stores, producers, poll;
    int store_cols, store_rows;  // shape of the store boxes (channels x tokens; `stores` carries the channel count)
    unsigned long long* trace;   // [kProbeTrace][8] of CTA 0, clock64 per stage: producer before / after its wait, after arming the
                                 // barrier, after the W load, after the X load; consumer when the stage had landed, was handed back
    unsigned long long* clocks;  // [grid][4]: clock64 at start and end, globaltimer at start and end
    uint32_t* status;
};

constexpr int kProbeStoreWarps = 8;
constexpr int kProbeThreads = 32 * (3 + kProbeStoreWarps);  // producer, consumer, store warps, second producer
// one store box per store warp: [16 tokens][32 channels] fp32 (2 KB) as in the GEMMs, or the 8 KB boxes of the wider shapes
__host__ __device__ inline int probe_staging(int store_cols, int store_rows) { return kProbeStoreWarps * store_cols * store_rows * 4; }
constexpr int kProbeTail = 1024;
constexpr int kProbeSmemLimit = 232448;
constexpr int kProbeMaxStages = 16;
constexpr int kProbeTrace = 512;
constexpr long long kProbeWaitLimit = 1ll << 28;

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__global__ void __launch_bounds__(kProbeThreads, 1)
tma_probe_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                 const __grid_constant__ CUtensorMap tmap_y, const ProbeParams p,
                 const __grid_constant__ PairSchedule sched) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int S = p.stages;
    const uint32_t a_bytes = (uint32_t)p.a_rows * p.a_row_bytes, b_bytes = (uint32_t)p.b_rows * 128u * p.b_slices;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    uint8_t* staging = smem + (size_t)S * stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(staging + probe_staging(p.store_cols, p.store_rows));
    const uint32_t bar0 = ptx::smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
    auto tile_done_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };
    auto store_done_bar = [&](int b) { return bar0 + 8u * (2 * S + 2 + b); };
    volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(bars + 2 * S + 4);
    volatile uint32_t* never_flag = abort_flag + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)ptx::cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int tile_begin = sched.start[pair], tile_count = sched.start[pair + 1] - tile_begin;
    const int total = tile_count * p.repeat;  // tiles this pair walks, the range repeated

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { ptx::mbar_init(full_bar(s), p.producers); ptx::mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { ptx::mbar_init(tile_done_bar(b), 1); ptx::mbar_init(store_done_bar(b), kProbeStoreWarps); }
        *abort_flag = 0;
        *never_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_w);
        ptx::prefetch_tensormap(&tmap_x);
        ptx::prefetch_tensormap(&tmap_y);
    }
    __syncthreads();
    unsigned long long c0 = 0, g0 = 0;
    if (threadIdx.x == 0) { c0 = clock64(); g0 = global_ns(); }

    auto raise_timeout = [&]() {
        *abort_flag = 1;
        if (p.status) atomicOr(p.status, NM_STATUS_TIMEOUT);
    };

    if (warp == 0 || warp == 2 + kProbeStoreWarps) {
        // ------------------------------ producer(s): the GEMM's loads --------------------------
        // One thread issues both boxes of a stage, or (producers == 2) warp 0 the weight boxes and the last
        // warp the X boxes, each arming the stage's barrier with its own bytes.
        const int which = warp == 0 ? (p.producers == 2 ? 1 : 3) : (p.producers == 2 ? 2 : 0);
        const int mine = which & p.loads;
        if (lane == 0 && which != 0) {
            uint32_t it = 0, parity = 1u;  // of the "empty" barriers: the first pass over the ring finds every stage free
            int s = 0;                     // ring position, advanced without a division: one thread's instructions run
            bool ok = true;                // one dependent step every few clocks, a modulo alone costs ~150 clocks
            const uint32_t tx = ((mine & 1) ? a_bytes : 0u) + ((mine & 2) ? b_bytes : 0u);
            const uint32_t smem0 = ptx::smem_u32(smem);
            for (int i = 0; i < total && ok; ++i) {
                const TileCoord tc = tile_coord(tile_begin + i % tile_count, p.n_tok_tiles, p.n_out_tiles, p.band);
                const int n0 = (tc.o * 2 + rank) * p.a_rows, t0 = (tc.t * 2 + rank) * p.b_rows;
                for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                    const bool tr = p.trace && blockIdx.x == 0 && warp == 0 && it < kProbeTrace;
                    unsigned long long* row = p.trace + 8 * (size_t)(tr ? it : 0);
                    if (tr) row[0] = clock64();
                    if (!ptx::mbar_wait_bounded(empty_bar(s), parity, abort_flag, kProbeWaitLimit)) {
                        raise_timeout(); ok = false; break;
                    }
                    if (tr) row[1] = clock64();
                    const uint32_t dst = smem0 + (uint32_t)s * stage_bytes;
                    if (tx) ptx::mbar_expect_tx(full_bar(s), tx); else ptx::mbar_arrive(full_bar(s));
                    if (tr) row[2] = clock64();
                    if (mine & 1) ptx::tma_load_2d(dst, &tmap_w, kb * p.a_row_bytes, n0, full_bar(s));
                    if (tr) row[3] = clock64();
                    if (mine & 2) ptx::tma_load_3d(dst + a_bytes, &tmap_x, 0, t0, kb * p.b_slices, full_bar(s));
                    if (tr) row[4] = clock64();
                    if (++s == S) { s = 0; parity ^= 1u; }
                }
            }
            if (!ok) {  // let copies already in flight land before the CTA goes away
                const uint32_t first = it > (uint32_t)S ? it - S : 0;
                for (uint32_t j = first; j < it; ++j)
                    ptx::mbar_wait_bounded(full_bar(j % S), (j / S) & 1u, never_flag, kProbeWaitLimit >> 4);
            }
        }
    } else if (warp == 1) {
        // ------------------------------ consumer: takes and returns every stage ----------------
        if (lane == 0) {
            uint32_t it = 0, parity = 0u;
            int s = 0;
            bool ok = true;
            for (int i = 0; i < total && ok; ++i) {
                const int buf = i & 1;
                if (p.poll != 2 && !ptx::mbar_wait_bounded(store_done_bar(buf), ((i >> 1) & 1u) ^ 1u, abort_flag, kProbeWaitLimit)) {
                    raise_timeout(); break;
                }
                for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
                    if (!ptx::mbar_wait_bounded(full_bar(s), parity, abort_flag, kProbeWaitLimit)) {
                        raise_timeout(); ok = false; break;
                    }
                    const long long t = clock64();
                    if (p.delay > 0) {
                        while (clock64() - t < p.delay) { }
                    }
                    ptx::mbar_arrive(empty_bar(s));
                    if (p.trace && blockIdx.x == 0 && it < kProbeTrace) { p.trace[8 * it + 5] = t; p.trace[8 * it + 6] = clock64(); }
                    if (++s == S) { s = 0; parity ^= 1u; }
                }
                if (ok) ptx::mbar_arrive(tile_done_bar(buf));
            }
        }
    } else {
        // ------------------------------ store warps: the epilogue's TMA stores -------------------
        const int sw = warp - 2;
        float* my_stage = reinterpret_cast<float*>(staging + sw * (p.store_cols * p.store_rows * 4));
        const int boxes_c = p.a_rows / p.store_cols, boxes_t = (2 * p.b_rows) / p.store_rows, boxes = boxes_c * boxes_t;
        const int box_words = p.store_cols * p.store_rows;
        for (int i = 0; i < total; ++i) {
            const int buf = i & 1;
            if (p.poll == 2) break;  // producer and consumer alone
            bool got = true;
            if (p.poll == 0) {
                got = ptx::mbar_wait_bounded(tile_done_bar(buf), (i >> 1) & 1u, abort_flag, kProbeWaitLimit);
            } else if (lane == 0) {  // one lane polls and sleeps between polls
                const long long t0 = clock64();
                while (!ptx::mbar_try_wait(tile_done_bar(buf), (i >> 1) & 1u)) {
                    __nanosleep(256);
                    if (*abort_flag || clock64() - t0 > kProbeWaitLimit) { got = false; break; }
                }
            }
            if (!__all_sync(0xffffffffu, got)) { if (lane == 0) raise_timeout(); break; }
            if (p.stores) {
                const TileCoord tc = tile_coord(tile_begin + i % tile_count, p.n_tok_tiles, p.n_out_tiles, p.band);
                const int n0 = (tc.o * 2 + rank) * p.a_rows, t0 = tc.t * 2 * p.b_rows;
                for (int b = sw; b < boxes; b += kProbeStoreWarps) {
                    const int bc = b % boxes_c, bt = b / boxes_c;
                    float* sb = my_stage;
                    if (lane == 0) ptx::bulk_wait_group_read<0>();  // the store before this one has read the tile
                    __syncwarp();
                    const float v = (float)(i + b);
                    for (int j = lane; j < box_words; j += 32) sb[j] = v;
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_2d(&tmap_y, n0 + bc * p.store_cols, t0 + bt * p.store_rows, ptx::smem_u32(sb));
                        ptx::bulk_commit_group();
                    }
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(store_done_bar(buf));
        }
        if (lane == 0) ptx::bulk_wait_group<0>();
    }
    __syncthreads();
    if (threadIdx.x == 0 && p.clocks) {
        p.clocks[4 * blockIdx.x + 0] = c0;
        p.clocks[4 * blockIdx.x + 1] = clock64();
        p.clocks[4 * blockIdx.x + 2] = g0;
        p.clocks[4 * blockIdx.x + 3] = global_ns();
    }
}

}  // namespace nm

extern "C" int nm_probe_tma_stream(const void* W, int w_rows, int w_row_bytes, const void* X, int tokens, int k_bytes,
                                   float* Y, int a_rows, int a_row_bytes, int b_rows, int b_slices, int stages,
                                   int band, int repeat, int delay_clocks, int loads, int stores, int producers, int poll,
                                   unsigned long long* clocks, unsigned long long* trace, uint32_t* status, void* stream) {
    using namespace nm;
    if (!W || !X || !Y) return NM_ERR_NULL;
    if (!aligned(W, 16) || !aligned(X, 16) || !aligned(Y, 16)) return NM_ERR_ALIGN;
    if (a_rows < 32 || a_rows > 256 || a_rows % 32 || (a_row_bytes != 64 && a_row_bytes != 128)) return NM_ERR_SHAPE;
    if (b_rows < 8 || b_rows > 256 || b_rows % 8 || b_slices < 1 || b_slices > 4) return NM_ERR_SHAPE;
    if (w_rows < 1 || tokens < 1 || w_row_bytes < a_row_bytes || w_row_bytes % a_row_bytes || k_bytes % (128 * b_slices)) return NM_ERR_SHAPE;
    if (w_row_bytes / a_row_bytes != k_bytes / (128 * b_slices)) return NM_ERR_SHAPE;  // both operands cover the same k-blocks
    if ((w_rows * 4) % 16) return NM_ERR_ALIGN;
    if (poll < 0 || poll > 2 || (poll == 2 && stores) || producers < 1 || producers > 2 || stages < 2 || stages > kProbeMaxStages || repeat < 1 || delay_clocks < 0 || delay_clocks > (1 << 20)) return NM_ERR_SHAPE;
    const int stage_bytes = a_rows * a_row_bytes + b_rows * 128 * b_slices;
    if (stage_bytes % 1024) return NM_ERR_SHAPE;
    CUtensorMap tw, tx, ty;
    int rc = make_map(&tw, W, (uint64_t)w_rows, (uint64_t)w_row_bytes, (uint32_t)a_rows, (uint32_t)a_row_bytes,
                      a_row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B);
    if (rc != NM_OK) return rc;
    rc = make_map_x3(&tx, X, (uint64_t)tokens, (uint64_t)k_bytes, (uint32_t)b_rows, (uint32_t)b_slices);
    if (rc != NM_OK) return rc;
    // `stores`: 0 = none, 1 = the GEMMs' [16 tokens][32 channels] boxes, else the channels per box (32, 64 or 128; boxes
    // of 8 KB: 64, 32 or 16 tokens high)
    const int store_cols = stores <= 1 ? 32 : stores, store_rows = stores <= 1 ? 16 : 8192 / (4 * store_cols);
    if (store_cols != 32 && store_cols != 64 && store_cols != 128) return NM_ERR_SHAPE;
    if (a_rows % store_cols || (2 * b_rows) % store_rows) return NM_ERR_SHAPE;
    const int smem = stages * stage_bytes + probe_staging(store_cols, store_rows) + kProbeTail + 1024;
    if (smem > kProbeSmemLimit) return NM_ERR_UNSUPPORTED;
    rc = make_map(&ty, Y, (uint64_t)tokens, (uint64_t)w_rows, (uint32_t)store_rows, (uint32_t)store_cols, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4);
    if (rc != NM_OK) return rc;
    ProbeParams p{};
    p.a_rows = a_rows; p.a_row_bytes = a_row_bytes; p.b_rows = b_rows; p.b_slices = b_slices;
    p.stages = stages; p.kblocks = w_row_bytes / a_row_bytes;
    p.n_tok_tiles = (tokens + 2 * b_rows - 1) / (2 * b_rows);
    p.n_out_tiles = (w_rows + 2 * a_rows - 1) / (2 * a_rows);
    p.repeat = repeat; p.delay = delay_clocks; p.loads = loads & 3; p.stores = stores ? 1 : 0; p.producers = producers; p.poll = poll; p.store_cols = store_cols; p.store_rows = store_rows;
    p.clocks = clocks; p.trace = trace; p.status = status;
    const long long n_tiles = (long long)p.n_tok_tiles * p.n_out_tiles;
    const int sms = sm_count();
    int pairs = sms / 2 < kMaxPairs ? sms / 2 : kMaxPairs;
    if (n_tiles < pairs) pairs = (int)n_tiles;
    PairSchedule sched;
    p.band = plan_pair_tiles(p.n_tok_tiles, p.n_out_tiles, pairs, false, band, sched.start);
    NM_CUDA_TRY(cudaFuncSetAttribute((const void*)tma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(kProbeThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;  // the two CTAs of a pair sit on neighbouring SMs, as in the GEMM
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    NM_CUDA_TRY(cudaLaunchKernelEx(&cfg, tma_probe_kernel, tw, tx, ty, p, sched));
    return 2 * pairs;  // CTAs launched = entries of `clocks` written (4 words each)
}
