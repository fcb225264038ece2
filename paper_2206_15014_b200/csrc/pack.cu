// N:M magnitude projection + per-channel symmetric quantisation + packing (one HBM pass).
//
// Work decomposition: a warp owns a chunk of 1024 consecutive weights of one row; a row is
// covered by 1, 2, 4 ... 32 warps of the same block.  Loads are coalesced 16-byte accesses
// (lane l, step j -> float4 number j*32+l of the chunk); the sum V = W + U goes through a
// swizzled shared-memory tile so that afterwards every lane holds 32 CONSECUTIVE values (8 groups
// of 4 or 4 groups of 8).  From there everything is lane-local: the lane's share of the packed
// values and of the metadata is a whole number of bytes, written with one vector store each.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include <cuda_runtime.h>
#include <vector>
#include <mutex>
#include <algorithm>
#include <cstdlib>

namespace nm {

struct PackJobDev {
    const float* W;
    const float* U;
    uint8_t* values;
    uint32_t* meta;
    float* scales;
    int out, in;
    int wpr_log2;         // log2(warps per row)
    unsigned unit_begin;  // first block of this job inside the launch
    unsigned vrow_bytes;  // bytes of one row of values
    unsigned mrow_words;  // words of one row of metadata
};

// Dense outputs of one job of a batched ADMM step (parallel to the PackJobDev table).
struct DenseOutDev {
    float* Z;
    float* U_next;
};

// Job tables of up to kInlineJobs entries travel as a kernel parameter: no table in device memory, no
// host-to-device copy in front of the launch.  A single matrix is a table of one.
static constexpr int kInlineJobs = 8;
struct PackJobInline {
    PackJobDev j[kInlineJobs];
};

static constexpr int kPackMinWarps = 4;
#ifndef NM_WAIT_LIMIT
#define NM_WAIT_LIMIT (1ll << 31)
#endif
static constexpr long long kPackWaitLimit = NM_WAIT_LIMIT;  // SM clocks a warp waits for its staged chunk (about a second)

// Test hook, compiled in with -DNM_TEST_HOOKS only (the library the timeout test loads, never the product's): in the
// staged form, warp 0 of block 0 leaves the copies of its unit number `d_pack_skip_unit` (counted per block) unissued --
// nothing is armed, nothing is copied, no address is touched -- so that the wait for that chunk runs out.
#ifdef NM_TEST_HOOKS
__device__ int d_pack_skip_unit = -1;
int pack_set_skip_unit(int unit) {
    NM_CUDA_TRY(cudaMemcpyToSymbol(d_pack_skip_unit, &unit, sizeof(unit)));
    return NM_OK;
}
#define NM_PACK_SKIP(iter) (blockIdx.x == 0 && w == 0 && (iter) == d_pack_skip_unit)
#else
#define NM_PACK_SKIP(iter) false
#endif
// group_mode of pack_kernel: scale per row from the row itself; only fold the row maxima per group into
// `scales`; take the scales found in `scales`.
enum { kGroupNone = 0, kGroupMaxPass = 1, kGroupScalesGiven = 2 };

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

// Bit mask of the positions kept in one group: position i is kept iff fewer than N others beat it,
// where j beats i when |v_j| > |v_i|, or |v_j| == |v_i| and j < i.
// n = 1, and 2 of 8: the kept values and their positions straight from one or two passes of
// "largest magnitude, first one on equality" (strict >), positions ascending.
template <int N, int M>
__device__ __forceinline__ void select_passes(const float* v, float* sel, unsigned* selp) {
    float best = fabsf(v[0]), bv = v[0];
    unsigned bi = 0;
#pragma unroll
    for (int j = 1; j < M; ++j) {
        const float aj = fabsf(v[j]);
        const bool gt = aj > best;
        best = gt ? aj : best;
        bv = gt ? v[j] : bv;
        bi = gt ? (unsigned)j : bi;
    }
    if constexpr (N == 1) {
        sel[0] = bv; selp[0] = bi;
    } else {
        float best2 = -1.0f, bv2 = 0.0f;  // magnitudes are >= 0
        unsigned bj = 0;
#pragma unroll
        for (int j = 0; j < M; ++j) {
            const float aj = fabsf(v[j]);
            const bool gt = (aj > best2) && ((unsigned)j != bi);
            best2 = gt ? aj : best2;
            bv2 = gt ? v[j] : bv2;
            bj = gt ? (unsigned)j : bj;
        }
        const bool sw = bj < bi;
        sel[0] = sw ? bv2 : bv; selp[0] = sw ? bj : bi;
        sel[1] = sw ? bv : bv2; selp[1] = sw ? bi : bj;
    }
}

// Two of four by a tournament on the pairs (0,1) and (2,3).  With "larger magnitude first, lower index first
// among equals" the two kept positions are 0 and 1 when the smaller of the first pair is >= the larger of the
// second, 2 and 3 when the smaller of the second pair is > the larger of the first, and otherwise the larger of
// each pair (the first one of a pair on equality).  Kept values and positions come out in ascending position.
__device__ __forceinline__ void select_2_of_4(const float* v, float* sel, unsigned* selp) {
    const float a0 = fabsf(v[0]), a1 = fabsf(v[1]), a2 = fabsf(v[2]), a3 = fabsf(v[3]);
    const bool i01 = a1 > a0, i23 = a3 > a2;
    const float hi01 = fmaxf(a0, a1), lo01 = fminf(a0, a1), hi23 = fmaxf(a2, a3), lo23 = fminf(a2, a3);
    const bool both01 = lo01 >= hi23, both23 = lo23 > hi01;
    const float w01 = i01 ? v[1] : v[0], w23 = i23 ? v[3] : v[2];
    sel[0] = both01 ? v[0] : (both23 ? v[2] : w01);
    sel[1] = both01 ? v[1] : (both23 ? v[3] : w23);
    selp[0] = both01 ? 0u : (both23 ? 2u : (i01 ? 1u : 0u));
    selp[1] = both01 ? 1u : (both23 ? 3u : (i23 ? 3u : 2u));
}

template <int N, int M>
__device__ __forceinline__ unsigned keep_mask(const float* a) {
    if constexpr (N == 1 || (N == 2 && M == 8)) {  // (the pack kernel's 2:4 has its own tournament, select_2_of_4)
        // One or two passes of "largest magnitude, first one on equality" (a strict > keeps the lower
        // index): the same support as the rank rule, with 7 + 7 compares instead of 28 for m = 8.
        float best = a[0];
        unsigned bi = 0;
#pragma unroll
        for (int j = 1; j < M; ++j) {
            const bool gt = a[j] > best;
            best = gt ? a[j] : best;
            bi = gt ? (unsigned)j : bi;
        }
        unsigned mask = 1u << bi;
        if constexpr (N == 2) {
            float best2 = -1.0f;  // magnitudes are >= 0
            unsigned bj = 0;
#pragma unroll
            for (int j = 0; j < M; ++j) {
                const bool gt = (a[j] > best2) && ((unsigned)j != bi);
                best2 = gt ? a[j] : best2;
                bj = gt ? (unsigned)j : bj;
            }
            mask |= 1u << bj;
        }
        return mask;
    }
    if constexpr (N == 4 && M == 8) {
        // Four of eight: the fourth largest magnitude T from a selection network (both halves sorted with five
        // compare-exchanges each, then the four maxima of a bitonic half-cleaner hold the four largest and their
        // minimum is T), the support as a >= T.  Equal magnitudes at the threshold make that more than four
        // positions; only then does the rank network below decide (lower index first).
        auto cx = [](float& hi, float& lo) { const float h = fmaxf(hi, lo), l = fminf(hi, lo); hi = h; lo = l; };
        float x0 = a[0], x1 = a[1], x2 = a[2], x3 = a[3], y0 = a[4], y1 = a[5], y2 = a[6], y3 = a[7];
        cx(x0, x1); cx(x2, x3); cx(x0, x2); cx(x1, x3); cx(x1, x2);   // x0 >= x1 >= x2 >= x3
        cx(y0, y1); cx(y2, y3); cx(y0, y2); cx(y1, y3); cx(y1, y2);   // y0 >= y1 >= y2 >= y3
        const float T = fminf(fminf(fmaxf(x0, y3), fmaxf(x1, y2)), fminf(fmaxf(x2, y1), fmaxf(x3, y0)));
        unsigned mask = 0;
#pragma unroll
        for (int i = 0; i < M; ++i) mask |= (a[i] >= T ? 1u : 0u) << i;
        if (__popc(mask) == N) return mask;
    }
    int rank[M];
#pragma unroll
    for (int i = 0; i < M; ++i) rank[i] = 0;
#pragma unroll
    for (int i = 0; i < M; ++i)
#pragma unroll
        for (int j = i + 1; j < M; ++j) {
            bool ge = a[i] >= a[j];  // i (the lower index) beats j on >=, j beats i otherwise
            rank[j] += ge ? 1 : 0;
            rank[i] += ge ? 0 : 1;
        }
    unsigned mask = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) mask |= (rank[i] < N ? 1u : 0u) << i;
    return mask;
}

template <int NBYTES>
__device__ __forceinline__ void store_bytes_vec(uint8_t* dst, const unsigned* w) {
    if constexpr (NBYTES == 2) *reinterpret_cast<uint16_t*>(dst) = (uint16_t)w[0];
    else if constexpr (NBYTES == 4) *reinterpret_cast<uint32_t*>(dst) = w[0];
    else if constexpr (NBYTES == 8) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
    else if constexpr (NBYTES == 16) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    else {
        static_assert(NBYTES == 32, "unexpected lane share");
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
}

template <int MAXBYTES>
__device__ __forceinline__ void store_bytes_slow(uint8_t* dst, const unsigned* w, int nbytes) {
#pragma unroll
    for (int i = 0; i < MAXBYTES; ++i)
        if (i < nbytes) dst[i] = (uint8_t)(w[i >> 2] >> ((i & 3) * 8));
}

// N == M: dense (quantise only, no metadata), processed in groups of 4.
// DENSE_OUT: the ADMM step / STE forward form.  Besides (or instead of: values, meta and scales may then be
// null) the packed outputs the kernel writes Z = s * code as dense fp32, zero where pruned, and, when
// U_next is not null, the dual update U_next = (W + U) - Z.  Both go back through the shared-memory
// tile so that the stores are as coalesced as the loads.
//
// A "unit" is what one block does at a time: `warps >> wpr_log2` rows of one job, one 1024-value chunk per warp.
// PIPE (blocks of four warps): the grid is persistent, block b takes the units b, b + gridDim.x, ...; every warp
// fetches the chunk of its NEXT unit (W and U, 4 KB each) with two bulk copies into the other half of a
// double buffer in shared memory while it works on the current one, so that loading and arithmetic overlap
// inside a warp and not only between blocks that happen to be out of step.  Without PIPE one block = one unit
// and the chunk is loaded with 16-byte global loads.

// Where a warp stands inside a unit of a job.
struct UnitPos {
    long long row;
    int chunk, row_in_block, elems;  // elems: values of the chunk that lie inside the row (0 when the row does not exist)
    bool row_ok;
};

__device__ __forceinline__ UnitPos unit_pos(const PackJobDev& job, unsigned unit, int w, int warps) {
    UnitPos u;
    const int wpr = 1 << job.wpr_log2;
    u.row_in_block = w >> job.wpr_log2;
    u.chunk = w & (wpr - 1);
    u.row = (long long)(unit - job.unit_begin) * (warps >> job.wpr_log2) + u.row_in_block;
    u.row_ok = u.row < job.out;
    u.elems = u.row_ok ? max(0, min(1024, job.in - u.chunk * 1024)) : 0;
    return u;
}

// The job whose units contain `unit` (tables ascend in unit_begin) and its number in the table.
__device__ __forceinline__ PackJobDev find_job(const PackJobDev* __restrict__ jobs, int njobs, const PackJobInline& inl,
                                               unsigned unit, int& index) {
    PackJobDev job;
    if (jobs) {
        int lo = 0, hi = njobs - 1;  // last job whose unit_begin <= unit
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (jobs[mid].unit_begin <= unit) lo = mid; else hi = mid - 1;
        }
        job = jobs[lo];
        index = lo;
    } else {
        // table in the kernel's parameters (a single matrix is a table of one)
        int lo = 0;
#pragma unroll
        for (int i = 1; i < kInlineJobs; ++i)
            if (i < njobs && inl.j[i].unit_begin <= unit) lo = i;
        job = inl.j[0];
#pragma unroll
        for (int i = 1; i < kInlineJobs; ++i)
            if (lo == i) job = inl.j[i];
        index = lo;
    }
    return job;
}

// Units of a job in a launch whose blocks have `warps` warps.
__device__ __forceinline__ unsigned units_of(const PackJobDev& job, int warps) {
    const int rpb = warps >> job.wpr_log2;
    return (unsigned)((job.out + rpb - 1) / rpb);
}

// Everything after the load: `mytile` holds the warp's chunk of V = W + U in the swizzled layout, `amax` and
// `poison` are the lane's running |max| and non-finite detector.  `red` is this unit's slot array for the row
// maximum across the warps of a row.  Every warp of the block calls it (block-wide barrier when a row spans warps).
template <int N, int M, int BITS, bool DENSE_OUT>
__device__ __forceinline__ void pack_finish(const PackJobDev& job, const UnitPos& up, int lane, int w, float4* mytile,
                                            float* red, const uint16_t* pos48, float amax, float poison, uint32_t* status,
                                            float* __restrict__ Zout, float* __restrict__ Unext, int group_mode, int group_rows) {
    constexpr bool kDense = (N == M);
    constexpr int G = 32 / M;                          // groups per lane
    constexpr int F = (M == 4) ? 2 : 4;                // metadata field width
    constexpr int VBITS = G * N * BITS;                // value bits per lane (16 .. 256)
    constexpr int VWORDS = (VBITS + 31) / 32;
    constexpr int MBITS = kDense ? 0 : G * N * F;      // metadata bits per lane (0, 16, 32, 64)
    constexpr int MWORDS = kDense ? 1 : (MBITS + 31) / 32;
    const int wpr = 1 << job.wpr_log2;
    const int row_in_block = up.row_in_block, chunk = up.chunk;
    const long long row = up.row;
    const bool row_ok = up.row_ok;
    const int in4 = job.in >> 2;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const bool bad = __any_sync(0xffffffffu, poison != poison) || !(amax <= 3.402823466e+38f);
    if (bad && lane == 0 && status) atomicOr(status, NM_STATUS_NONFINITE);
    if (wpr > 1) {
        if (lane == 0) red[w] = amax;
        __syncthreads();
        for (int c = 0; c < wpr; ++c) amax = fmaxf(amax, red[row_in_block * wpr + c]);
    } else {
        __syncwarp();
    }

    // ---- group-wise scales, first pass: fold this row's maximum into the first entry of its group -----
    if (group_mode == kGroupMaxPass) {
        if (row_ok && chunk == 0 && lane == 0) {
            const int G = (group_rows <= 0 || group_rows > job.out) ? job.out : group_rows;
            atomicMax(reinterpret_cast<unsigned*>(job.scales) + (size_t)(row / G) * G, __float_as_uint(amax));
        }
        return;
    }

    // ---- ADMM-Max scale ---------------------------------------------------------------------
    constexpr float qmax = (float)((1 << (BITS - 1)) - 1);
    // group-wise quantisation hands the scale in (one per row, equal within a group of rows)
    const float s = group_mode == kGroupScalesGiven ? job.scales[row_ok ? row : 0]
                                                    : ((amax == 0.0f) ? 1.0f : __fdiv_rn(amax, qmax));
    if (row_ok && chunk == 0 && lane == 0 && (!DENSE_OUT || job.scales)) job.scales[row] = s;
    const float rs = __frcp_rn(s);  // correctly rounded reciprocal, once per row
    const bool fast_ok = (s >= 1.17549435e-38f) && (s <= 4.25e37f);  // rs is a normal number

    // ---- this lane's 32 consecutive values ----------------------------------------------------
    float v[32];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) {
        float4 t = mytile[lane * 8 + (jj ^ (lane & 7))];
        v[jj * 4 + 0] = t.x; v[jj * 4 + 1] = t.y; v[jj * 4 + 2] = t.z; v[jj * 4 + 3] = t.w;
    }
    const int lane_first = chunk * 1024 + lane * 32;             // first column of this lane
    const int nvals = max(0, min(32, job.in - lane_first));      // columns inside the row
    if (!DENSE_OUT && (!row_ok || nvals == 0)) return;
    float z[DENSE_OUT ? 32 : 1];  // dequantised projection of this lane's values (DENSE_OUT)
    if constexpr (DENSE_OUT) {
#pragma unroll
        for (int i = 0; i < 32; ++i) z[i] = 0.0f;
    }

    unsigned vw[VWORDS], mw[MWORDS];
#pragma unroll
    for (int i = 0; i < VWORDS; ++i) vw[i] = 0;
#pragma unroll
    for (int i = 0; i < MWORDS; ++i) mw[i] = 0;

#pragma unroll
    for (int g = 0; g < G; ++g) {
        if (g * M < nvals) {
            if constexpr (kDense) {
#pragma unroll
                for (int p = 0; p < M; ++p) {
                    const int pos = (g * M + p) * BITS;
                    const int code = quantise_shared_scale<BITS>(v[g * M + p], s, rs, fast_ok);
                    vw[pos >> 5] |= ((unsigned)code & ((1u << BITS) - 1u)) << (pos & 31);
                    if constexpr (DENSE_OUT) z[g * M + p] = __fmul_rn(s, (float)code);
                }
            } else {
                float sel[N];
                unsigned selp[N];
#pragma unroll
                for (int c = 0; c < N; ++c) { sel[c] = 0.0f; selp[c] = 0; }
                constexpr bool kPasses = (N == 1) || (N == 2 && M == 8) || (N == 2 && M == 4);
                unsigned mask = 0;
                if constexpr (N == 2 && M == 4) {
                    select_2_of_4(v + g * M, sel, selp);
                } else if constexpr (kPasses) {
                    select_passes<N, M>(v + g * M, sel, selp);
                } else {
                    float a[M];
#pragma unroll
                    for (int p = 0; p < M; ++p) a[p] = fabsf(v[g * M + p]);
                    mask = keep_mask<N, M>(a);
                }
                // compaction: slot c receives the c-th kept position (ascending)
                if constexpr (kPasses) {
                } else if constexpr (N == 4 && M == 8) {
                    const unsigned pos4 = pos48[mask];
                    const float* tile_f = reinterpret_cast<const float*>(mytile);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        selp[c] = (pos4 >> (4 * c)) & 7u;
                        const unsigned e = (unsigned)(g * 8) + selp[c];  // element of this lane, in the tile's swizzle
                        sel[c] = tile_f[(lane * 8 + ((e >> 2) ^ (lane & 7))) * 4 + (e & 3u)];
                    }
                } else {
#pragma unroll
                for (int p = 0; p < M; ++p) {
                    const bool kept = (mask >> p) & 1u;
                    const int before = __popc(mask & ((1u << p) - 1u));
#pragma unroll
                    for (int c = 0; c < N; ++c) {
                        // position p can only land in slot c if c <= p and enough positions remain
                        if (c <= p && (M - p) >= (N - c)) {
                            const bool hit = kept && before == c;
                            sel[c] = hit ? v[g * M + p] : sel[c];
                            selp[c] = hit ? (unsigned)p : selp[c];
                        }
                    }
                }
                }
#pragma unroll
                for (int c = 0; c < N; ++c) {
                    const int vpos = (g * N + c) * BITS, mpos = (g * N + c) * F;
                    const int code = quantise_shared_scale<BITS>(sel[c], s, rs, fast_ok);
                    vw[vpos >> 5] |= ((unsigned)code & ((1u << BITS) - 1u)) << (vpos & 31);
                    mw[mpos >> 5] |= selp[c] << (mpos & 31);
                    if constexpr (DENSE_OUT) {
                        const float zc = __fmul_rn(s, (float)code);
#pragma unroll
                        for (int p = 0; p < M; ++p) z[g * M + p] = (selp[c] == (unsigned)p) ? zc : z[g * M + p];
                    }
                }
            }
        }
    }

    // ---- dense outputs (ADMM step): back through the tile, then coalesced 16-byte stores --------
    if constexpr (DENSE_OUT) {
        auto write_back = [&](const float* x, float* dst_base) {
#pragma unroll
            for (int jj = 0; jj < 8; ++jj)
                mytile[lane * 8 + (jj ^ (lane & 7))] = make_float4(x[jj * 4], x[jj * 4 + 1], x[jj * 4 + 2], x[jj * 4 + 3]);
            __syncwarp();
            float4* D4 = reinterpret_cast<float4*>(dst_base) + (row_ok ? row * in4 : 0);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int fl = j * 32 + lane, owner = fl >> 3, jj = fl & 7, f = chunk * 256 + fl;
                const float4 t = mytile[owner * 8 + (jj ^ (owner & 7))];
                if (row_ok && f < in4) __stcs(D4 + f, t);
            }
            __syncwarp();
        };
        write_back(z, Zout);
        if (Unext) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __fsub_rn(v[i], z[i]);  // (W + U) - Z
            write_back(v, Unext);
        }
        if (!row_ok || nvals == 0) return;
    }

    // ---- stores -----------------------------------------------------------------------------
    const int lane_global = chunk * 32 + lane;
    const bool full = (nvals == 32);
    if (!DENSE_OUT || job.values) {
        constexpr int LB = VBITS / 8;
        uint8_t* dst = job.values + (size_t)row * job.vrow_bytes + (size_t)lane_global * LB;
        if (full && (reinterpret_cast<uintptr_t>(dst) % (LB < 16 ? LB : 16)) == 0) store_bytes_vec<LB>(dst, vw);
        else store_bytes_slow<LB>(dst, vw, nvals / M * N * BITS / 8);
    }
    if constexpr (!kDense) {
        if (DENSE_OUT && !job.meta) return;
        constexpr int MB = MBITS / 8;
        const unsigned lane_off = (unsigned)lane_global * MB;
        const unsigned row_bytes = job.mrow_words * 4u;
        uint8_t* dst = reinterpret_cast<uint8_t*>(job.meta + (size_t)row * job.mrow_words) + lane_off;
        const bool last = (lane_first + 32 >= job.in);  // lane holding the end of the row
        if (full && !last && (reinterpret_cast<uintptr_t>(dst) % MB) == 0) {  // aligned vector store
            store_bytes_vec<MB>(dst, mw);
        } else {
            // the last lane also writes the zero padding up to the row's word boundary
            const unsigned wpad[3] = {mw[0], MWORDS > 1 ? mw[MWORDS - 1] : 0u, 0u};
            store_bytes_slow<MB + 4>(dst, wpad, last ? (int)min(row_bytes - lane_off, (unsigned)(MB + 4)) : MB);
        }
    }
}

// Loads the warp's chunk with coalesced 16-byte global loads, leaves V = W + U in `mytile` (swizzled).
__device__ __forceinline__ void load_chunk_global(const PackJobDev& job, const UnitPos& up, int lane, float4* mytile,
                                                  float& amax, float& poison) {
    const int in4 = job.in >> 2;
    const float4* W4 = reinterpret_cast<const float4*>(job.W) + (up.row_ok ? up.row * in4 : 0);
    const float4* U4 = job.U ? reinterpret_cast<const float4*>(job.U) + (up.row_ok ? up.row * in4 : 0) : nullptr;
    float4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        int f = up.chunk * 256 + j * 32 + lane;
        v[j] = (up.row_ok && f < in4) ? ld_stream(W4 + f) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (U4) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int f = up.chunk * 256 + j * 32 + lane;
            if (up.row_ok && f < in4) {
                float4 u = ld_stream(U4 + f);
                v[j].x = __fadd_rn(v[j].x, u.x); v[j].y = __fadd_rn(v[j].y, u.y);
                v[j].z = __fadd_rn(v[j].z, u.z); v[j].w = __fadd_rn(v[j].w, u.w);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v[j].x), fabsf(v[j].y)), fmaxf(fabsf(v[j].z), fabsf(v[j].w))));
        poison = __fmaf_rn(v[j].x, 0.0f, poison); poison = __fmaf_rn(v[j].y, 0.0f, poison);
        poison = __fmaf_rn(v[j].z, 0.0f, poison); poison = __fmaf_rn(v[j].w, 0.0f, poison);
        int fl = j * 32 + lane, owner = fl >> 3, jj = fl & 7;
        mytile[owner * 8 + (jj ^ (owner & 7))] = v[j];
    }
}

// The same from the chunk that the bulk copies left in shared memory (`wbuf`, `ubuf`: 256 float4 each, in
// memory order); V = W + U replaces W in place, swizzled inside each 128-byte row.
__device__ __forceinline__ void load_chunk_staged(const PackJobDev& job, const UnitPos& up, int lane, float4* wbuf,
                                                  const float4* ubuf, float& amax, float& poison) {
    const int n4 = up.elems >> 2;  // float4 of the chunk that the copy brought
    float4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int fl = j * 32 + lane;
        v[j] = fl < n4 ? wbuf[fl] : make_float4(0.f, 0.f, 0.f, 0.f);
        if (job.U && fl < n4) {
            const float4 u = ubuf[fl];
            v[j].x = __fadd_rn(v[j].x, u.x); v[j].y = __fadd_rn(v[j].y, u.y);
            v[j].z = __fadd_rn(v[j].z, u.z); v[j].w = __fadd_rn(v[j].w, u.w);
        }
    }
    __syncwarp();  // every lane has read its part before the rows are rewritten in place
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v[j].x), fabsf(v[j].y)), fmaxf(fabsf(v[j].z), fabsf(v[j].w))));
        poison = __fmaf_rn(v[j].x, 0.0f, poison); poison = __fmaf_rn(v[j].y, 0.0f, poison);
        poison = __fmaf_rn(v[j].z, 0.0f, poison); poison = __fmaf_rn(v[j].w, 0.0f, poison);
        int fl = j * 32 + lane, owner = fl >> 3, jj = fl & 7;
        wbuf[owner * 8 + (jj ^ (owner & 7))] = v[j];
    }
}

// Forms of the kernel.  kDirect: one block = one unit, 16-byte global loads.  kStaged2: persistent, two chunk
// buffers per warp (16 KB), the next unit's copies are issued before the current unit is touched; for the forms that
// keep using the tile to the end of the unit (4:8, dense outputs).
// kAhead: persistent, 16-byte global loads as in kDirect, but every warp first asks for its NEXT unit's chunk to be
// brought into L2 (a bulk prefetch: no registers, no shared memory), so that DRAM streams from the first cycle on and
// the loads of all units but the first are L2 hits.
enum { kDirect = 0, kStaged2 = 1, kAhead = 2 };
__host__ __device__ constexpr int pack_blocks_per_sm(int pipe) { return pipe == kStaged2 ? 3 : 8; }

template <int N, int M, int BITS, int MAXT, bool DENSE_OUT = false, int PIPE = kDirect>
__global__ void __launch_bounds__(MAXT, PIPE != kDirect ? pack_blocks_per_sm(PIPE) : (MAXT == 128 ? (DENSE_OUT ? 4 : 8) : 1))
pack_kernel(const PackJobDev* __restrict__ jobs, int njobs, const __grid_constant__ PackJobInline inl, uint32_t* status,
            float* __restrict__ Zout, float* __restrict__ Unext, const DenseOutDev* __restrict__ dense_jobs,
            int group_mode, int group_rows, unsigned nunits) {
    static_assert(PIPE == kDirect || MAXT == 128, "the staged forms are built for blocks of four warps");
    // staged: [warps][2 buffers][W, U][256] float4; else [warps][256] float4.  Then [2][warps] floats for the row
    // maximum, 256 u16 (4:8 positions), and for the staged forms [warps][2] mbarriers and the abort flag.
    extern __shared__ float4 tile[];
    const int warps = blockDim.x >> 5;
    float* red = reinterpret_cast<float*>(tile + warps * (PIPE == kStaged2 ? 1024 : 256));
    // a kernel launched as this one's programmatic dependent may begin its set-up on SMs this grid has left
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // four of eight: table from the 8-bit keep mask to its four positions (4-bit fields, ascending), which is
    // also the group's metadata; the kept values are then fetched from the warp's tile by position
    uint16_t* pos48 = reinterpret_cast<uint16_t*>(red + 2 * warps);
    if constexpr (N == 4 && M == 8) {
        for (unsigned mk = threadIdx.x; mk < 256; mk += blockDim.x) {
            unsigned r = 0, c = 0;
#pragma unroll
            for (unsigned p8 = 0; p8 < 8; ++p8)
                if ((mk >> p8) & 1u) { r |= p8 << (4 * (c & 3u)); ++c; }
            pos48[mk] = (uint16_t)r;
        }
        __syncthreads();
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;

    if constexpr (PIPE == kAhead) {
        float4* mytile = tile + w * 256;
        auto ask = [&](const PackJobDev& j, const UnitPos& up) {
            if (up.elems == 0 || lane != 0) return;
            const size_t first = (size_t)up.row * j.in + (size_t)up.chunk * 1024;
            ptx::bulk_prefetch_l2(j.W + first, (uint32_t)up.elems * 4u);
            if (j.U) ptx::bulk_prefetch_l2(j.U + first, (uint32_t)up.elems * 4u);
        };
        int index = 0;
        unsigned unit = blockIdx.x;
        PackJobDev job{};
        if (unit < nunits) job = find_job(jobs, njobs, inl, unit, index);
        for (int it = 0; unit < nunits; ++it, unit += gridDim.x) {
            const UnitPos up = unit_pos(job, unit, w, warps);
            const unsigned next = unit + gridDim.x;
            PackJobDev njob = job;
            int nindex = index;
            if (next < nunits) {
                if (next - job.unit_begin >= units_of(job, warps)) njob = find_job(jobs, njobs, inl, next, nindex);
                ask(njob, unit_pos(njob, next, w, warps));
            }
            if constexpr (DENSE_OUT) {
                if (jobs) { Zout = dense_jobs[index].Z; Unext = dense_jobs[index].U_next; }
            }
            float amax = 0.0f, poison = 0.0f;
            load_chunk_global(job, up, lane, mytile, amax, poison);
            pack_finish<N, M, BITS, DENSE_OUT>(job, up, lane, w, mytile, red + (it & 1) * warps, pos48, amax, poison,
                                              status, Zout, Unext, group_mode, group_rows);
            __syncwarp();  // the tile is rewritten by the next unit
            job = njob; index = nindex;
        }
    } else if constexpr (PIPE == kDirect) {
        int index = 0;
        const PackJobDev job = find_job(jobs, njobs, inl, blockIdx.x, index);
        if constexpr (DENSE_OUT) {
            if (jobs) { Zout = dense_jobs[index].Z; Unext = dense_jobs[index].U_next; }
        }
        const UnitPos up = unit_pos(job, blockIdx.x, w, warps);
        float4* mytile = tile + w * 256;
        float amax = 0.0f, poison = 0.0f;
        load_chunk_global(job, up, lane, mytile, amax, poison);
        pack_finish<N, M, BITS, DENSE_OUT>(job, up, lane, w, mytile, red, pos48, amax, poison, status, Zout, Unext,
                                          group_mode, group_rows);
    } else {
        uint64_t* bars = reinterpret_cast<uint64_t*>(pos48 + 256);       // [warps][2]
        volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 2 * warps);
        float4* mybuf = tile + w * 1024;                                  // [buffer][W, U][256]
        const uint32_t bar0 = ptx::smem_u32(bars + 2 * w);
        if (lane == 0) {
            ptx::mbar_init(bar0, 1);
            ptx::mbar_init(bar0 + 8, 1);
            if (threadIdx.x == 0) *abort_flag = 0;
            ptx::fence_mbar_init();
        }
        __syncthreads();
        // every lane calls it; lane 0 issues one bulk copy per operand, completion counted in bytes on the buffer's barrier
        auto issue = [&](const PackJobDev& j, const UnitPos& up, int buf, int iter) {
            if (up.elems == 0) return;      // the same for the whole warp; the unit then waits for nothing
            if (NM_PACK_SKIP(iter)) return;
            ptx::fence_proxy_async_smem();  // this lane's generic accesses to the buffer before the copy's writes
            __syncwarp();                   // the buffer's last reader is done
            if (lane == 0) {
                const uint32_t bytes = (uint32_t)up.elems * 4u, bar = bar0 + 8u * buf;
                const size_t first = (size_t)up.row * j.in + (size_t)up.chunk * 1024;
                ptx::mbar_expect_tx(bar, j.U ? 2 * bytes : bytes);
                ptx::bulk_load(ptx::smem_u32(mybuf + buf * 512), j.W + first, bytes, bar);
                if (j.U) ptx::bulk_load(ptx::smem_u32(mybuf + buf * 512 + 256), j.U + first, bytes, bar);
            }
        };
        int index = 0;
        unsigned unit = blockIdx.x;
        PackJobDev job{};
        UnitPos up{};
        if (unit < nunits) {
            job = find_job(jobs, njobs, inl, unit, index);
            up = unit_pos(job, unit, w, warps);
            issue(job, up, 0, 0);
        }
        uint32_t phase = 0;  // bit b: parity of buffer b's next completion
        for (int it = 0; unit < nunits; ++it, unit += gridDim.x) {
            const int buf = it & 1;
            // the next unit's chunk goes into the other buffer while this one is worked on
            const unsigned next = unit + gridDim.x;
            PackJobDev njob = job;
            int nindex = index;
            UnitPos nup{};
            if (next < nunits) {
                if (next - job.unit_begin >= units_of(job, warps)) njob = find_job(jobs, njobs, inl, next, nindex);
                nup = unit_pos(njob, next, w, warps);
                issue(njob, nup, buf ^ 1, it + 1);
            }
            if constexpr (DENSE_OUT) {
                if (jobs) { Zout = dense_jobs[index].Z; Unext = dense_jobs[index].U_next; }
            }
            if (up.elems != 0) {
                if (!ptx::mbar_wait_bounded(bar0 + 8u * buf, (phase >> buf) & 1u, abort_flag, kPackWaitLimit)) {
                    // recorded; the unit is then worked on with whatever the buffer holds (in bounds, results void)
                    *abort_flag = 1u;
                    if (status) atomicOr(status, NM_STATUS_TIMEOUT);
                }
                phase ^= 1u << buf;
            }
            float4* mytile = mybuf + buf * 512;
            float amax = 0.0f, poison = 0.0f;
            load_chunk_staged(job, up, lane, mytile, mytile + 256, amax, poison);
            pack_finish<N, M, BITS, DENSE_OUT>(job, up, lane, w, mytile, red + (it & 1) * warps, pos48, amax, poison,
                                              status, Zout, Unext, group_mode, group_rows);
            job = njob; index = nindex; up = nup;
        }
        // after an expired wait a copy may still be on its way into this block's shared memory
        if (*abort_flag) ptx::wait_clocks(1 << 17);
    }
}

// ---------------------------------------------------------------------------------------------
// Group-wise scales: rows r with the same r / group_rows share one ADMM-Max scale.  A first pass folds
// max |W + U| of every row into the first entry of its group in `scales` (non-negative floats order like
// their bit patterns, so an unsigned atomicMax does it); a second turns each group's maximum into the
// scale and writes it to all rows of the group (one thread per group: reads before it writes).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) group_absmax_kernel(const float* __restrict__ W, const float* __restrict__ U,
                                                           int out, int in, int group_rows, float* scales) {
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= out) return;
    const int in4 = in >> 2;
    const float4* W4 = reinterpret_cast<const float4*>(W) + (size_t)row * in4;
    const float4* U4 = U ? reinterpret_cast<const float4*>(U) + (size_t)row * in4 : nullptr;
    float a = 0.0f;
    for (int f = lane; f < in4; f += 32) {
        float4 v = __ldg(W4 + f);  // read again by the projection pass: keep it cached
        if (U4) {
            const float4 u = __ldg(U4 + f);
            v.x = __fadd_rn(v.x, u.x); v.y = __fadd_rn(v.y, u.y); v.z = __fadd_rn(v.z, u.z); v.w = __fadd_rn(v.w, u.w);
        }
        a = fmaxf(a, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    if (lane == 0) atomicMax(reinterpret_cast<unsigned*>(scales) + (size_t)(row / group_rows) * group_rows, __float_as_uint(a));
}

__global__ void __launch_bounds__(128) group_scale_kernel(int out, int group_rows, int bits, float* scales) {
    const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long first = g * group_rows;
    if (first >= out) return;
    const float a = scales[first];
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const float s = (a == 0.0f) ? 1.0f : __fdiv_rn(a, qmax);
    const long long last = min((long long)out, first + group_rows);
    for (long long r = first; r < last; ++r) scales[r] = s;
}

// Batched form over a job table: block j serves job j.  phase 0 clears the scales (the maxima are folded
// in by the pack kernel's kGroupMaxPass), phase 1 turns each group's maximum into the scale of its rows.
__global__ void __launch_bounds__(256) group_prepare_kernel(const PackJobDev* __restrict__ jobs, int group_rows,
                                                            int bits, int phase) {
    const PackJobDev job = jobs[blockIdx.x];
    if (phase == 0) {
        for (int r = threadIdx.x; r < job.out; r += blockDim.x) job.scales[r] = 0.0f;
        return;
    }
    const int G = (group_rows <= 0 || group_rows > job.out) ? job.out : group_rows;
    const float qmax = (float)((1 << (bits - 1)) - 1);
    for (long long first = (long long)threadIdx.x * G; first < job.out; first += (long long)blockDim.x * G) {
        const float a = job.scales[first];
        const float s = (a == 0.0f) ? 1.0f : __fdiv_rn(a, qmax);
        const long long last = min((long long)job.out, first + G);
        for (long long r = first; r < last; ++r) job.scales[r] = s;
    }
}

static int launch_group_scales(const float* W, const float* U, int out, int in, int bits, int group_rows,
                               float* scales, cudaStream_t stream) {
    const int G = group_rows <= 0 ? out : (group_rows > out ? out : group_rows);
    NM_CUDA_TRY(cudaMemsetAsync(scales, 0, (size_t)out * sizeof(float), stream));
    group_absmax_kernel<<<(out + 3) / 4, 128, 0, stream>>>(W, U, out, in, G, scales);
    NM_CUDA_TRY(cudaGetLastError());
    const int ngroups = (out + G - 1) / G;
    group_scale_kernel<<<(ngroups + 127) / 128, 128, 0, stream>>>(out, G, bits, scales);
    NM_CUDA_TRY(cudaGetLastError());
    return NM_OK;
}

// ---------------------------------------------------------------------------------------------
// ADMM-Dist scale (Sec. 3.3.1, "Minimize Quantization Distance"): per output channel the scale that
// minimises the squared distance between the N:M-projected channel and its quantised form, searched
// over the candidates s_j = fl32(s_max * (64 - j) / 64), j = 0 .. ncand-1 (s_max = the ADMM-Max scale;
// lowest j on equal distance).  The kernel writes the winning scale to `scales`; the projection /
// packing kernel then runs with the scales handed in.
//
// Same decomposition as pack_kernel: a warp owns 1024 consecutive weights, a lane 32 consecutive ones,
// of which it keeps G*N in registers (as fp32 for the quantiser, as fp64 for the distance).  Per
// candidate and kept value: the code from the reciprocal product (true division when the quotient is
// within 2^-15 of a rounding tie or the scale is outside the range where the reciprocal is accurate),
// converted to a double, then d = v - s*code and E += d*d as two fp64 FMAs (the
// product s*code is exact in double).  E is summed per lane, over the lanes by a butterfly, over the
// warps of a row through shared memory: a fixed order, so the result is deterministic.  The work is
// bound by instruction issue (about 15 instructions per candidate and kept value), not by HBM.
// ---------------------------------------------------------------------------------------------
template <int N, int M>
__device__ __forceinline__ void kept_values(const float* v, float* sel) {
    if constexpr (N == M) {
#pragma unroll
        for (int p = 0; p < M; ++p) sel[p] = v[p];
    } else if constexpr ((N == 1) || (N == 2 && M == 8)) {
        unsigned selp[N];
        select_passes<N, M>(v, sel, selp);
    } else {
        float a[M];
#pragma unroll
        for (int p = 0; p < M; ++p) a[p] = fabsf(v[p]);
        const unsigned mask = keep_mask<N, M>(a);
        if constexpr (N == 2 && M == 4) {
            const bool b0 = mask & 1u, b1 = mask & 2u, b2 = mask & 4u, b3 = mask & 8u;
            sel[0] = b0 ? v[0] : (b1 ? v[1] : v[2]);
            sel[1] = b3 ? v[3] : (b2 ? v[2] : v[1]);
        } else {
#pragma unroll
            for (int c = 0; c < N; ++c) sel[c] = 0.0f;
#pragma unroll
            for (int p = 0; p < M; ++p) {
                const bool kept = (mask >> p) & 1u;
                const int before = __popc(mask & ((1u << p) - 1u));
#pragma unroll
                for (int c = 0; c < N; ++c)
                    if (c <= p && (M - p) >= (N - c)) sel[c] = (kept && before == c) ? v[p] : sel[c];
            }
        }
    }
}

template <int N, int M, int BITS, int MAXT>
__global__ void __launch_bounds__(MAXT, MAXT == 128 ? (32 / M * N > 16 ? 4 : 5) : 1) dist_scale_kernel(const PackJobDev* __restrict__ jobs, int njobs,
                                                                              PackJobDev single, uint32_t* status, int ncand,
                                                                              int32_t* __restrict__ cand_out) {
    constexpr int G = 32 / M;
    constexpr int KN = G * N;  // kept values per lane
    extern __shared__ float4 tile[];  // [warps][256] float4, [warps][32] doubles, [warps] floats
    const int warps = blockDim.x >> 5;
    double* red_e = reinterpret_cast<double*>(tile + warps * 256);
    float* red = reinterpret_cast<float*>(red_e + warps * 32);

    PackJobDev job;
    if (jobs) {
        int lo = 0, hi = njobs - 1;  // last job whose unit_begin <= blockIdx.x
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (jobs[mid].unit_begin <= blockIdx.x) lo = mid; else hi = mid - 1;
        }
        job = jobs[lo];
    } else {
        job = single;
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int wpr = 1 << job.wpr_log2;
    const int row_in_block = w >> job.wpr_log2, chunk = w & (wpr - 1);
    const int rows_per_block = warps >> job.wpr_log2;
    const long long row = (long long)(blockIdx.x - job.unit_begin) * rows_per_block + row_in_block;
    const bool row_ok = row < job.out;
    const int in4 = job.in >> 2;

    // ---- V = W + U (coalesced; kept in cache for the projection pass that follows), |max|, transpose ----
    float4* mytile = tile + w * 256;
    float amax = 0.0f, poison = 0.0f;
    {
        const float4* W4 = reinterpret_cast<const float4*>(job.W) + (row_ok ? row * in4 : 0);
        const float4* U4 = job.U ? reinterpret_cast<const float4*>(job.U) + (row_ok ? row * in4 : 0) : nullptr;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int f = chunk * 256 + j * 32 + lane;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row_ok && f < in4) {
                t = __ldg(W4 + f);
                if (U4) {
                    const float4 u = __ldg(U4 + f);
                    t.x = __fadd_rn(t.x, u.x); t.y = __fadd_rn(t.y, u.y);
                    t.z = __fadd_rn(t.z, u.z); t.w = __fadd_rn(t.w, u.w);
                }
            }
            amax = fmaxf(amax, fmaxf(fmaxf(fabsf(t.x), fabsf(t.y)), fmaxf(fabsf(t.z), fabsf(t.w))));
            poison = __fmaf_rn(t.x, 0.0f, poison); poison = __fmaf_rn(t.y, 0.0f, poison);
            poison = __fmaf_rn(t.z, 0.0f, poison); poison = __fmaf_rn(t.w, 0.0f, poison);
            const int fl = j * 32 + lane, owner = fl >> 3, jj = fl & 7;
            mytile[owner * 8 + (jj ^ (owner & 7))] = t;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const bool bad = __any_sync(0xffffffffu, poison != poison) || !(amax <= 3.402823466e+38f);
    if (bad && lane == 0 && status) atomicOr(status, NM_STATUS_NONFINITE);
    if (wpr > 1) {
        if (lane == 0) red[w] = amax;
        __syncthreads();
        for (int c = 0; c < wpr; ++c) amax = fmaxf(amax, red[row_in_block * wpr + c]);
    } else {
        __syncwarp();
    }

    // ---- this lane's kept values (columns beyond the row were loaded as zeros: they add nothing) --------
    float x[KN];
    double xd[KN];
    {
        float v[32];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const float4 t = mytile[lane * 8 + (jj ^ (lane & 7))];
            v[jj * 4 + 0] = t.x; v[jj * 4 + 1] = t.y; v[jj * 4 + 2] = t.z; v[jj * 4 + 3] = t.w;
        }
#pragma unroll
        for (int g = 0; g < G; ++g) kept_values<N, M>(v + g * M, x + g * N);
#pragma unroll
        for (int i = 0; i < KN; ++i) xd[i] = (double)x[i];
    }

    constexpr float qmax = (float)((1 << (BITS - 1)) - 1);
    constexpr float kLo = -(float)(1 << (BITS - 1)) - 0.49f, kHi = qmax + 0.49f;
    constexpr float kMagic = 12582912.0f;             // 1.5 * 2^23 = 0x4B400000
    const float smax = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, qmax);
    double mine = __longlong_as_double(0x7ff0000000000000ll);  // lane j ends up with candidate j's distance
    for (int j = 0; j < ncand; ++j) {
        const float sj = __fmul_rn(smax, (float)(64 - j) * 0.015625f);
        const float rj = __frcp_rn(sj);
        const double nsd = -(double)sj;
        // outside [2^-126, 2^125] the reciprocal is subnormal, infinite or the product loses bits
        const bool fast_ok = (sj >= 1.17549435e-38f) && (sj <= 4.25e37f);
        // fast pass: code from the reciprocal product; the rounded quotient (an integer-valued float) goes to
        // the fp64 pipe through one conversion
        bool near_tie = !fast_ok;
        double e0 = 0.0, e1 = 0.0;
#pragma unroll
        for (int i = 0; i < KN; ++i) {
            const float qc = fminf(fmaxf(__fmul_rn(x[i], rj), kLo), kHi);
            const float r = __fsub_rn(__fadd_rn(qc, kMagic), kMagic);  // nearest-even integer of qc
            near_tie |= !(fabsf(__fsub_rn(qc, r)) <= 0.49996948f);
            const double d = fma(nsd, (double)r, xd[i]);
            if (i & 1) e1 = fma(d, d, e1); else e0 = fma(d, d, e0);
        }
        if (near_tie) {  // some quotient of this lane sits next to a rounding tie: the whole candidate again, exactly
            e0 = 0.0; e1 = 0.0;
#pragma unroll
            for (int i = 0; i < KN; ++i) {
                const float qc = fminf(fmaxf(__fdiv_rn(x[i], sj), kLo), kHi);
                const float r = __fsub_rn(__fadd_rn(qc, kMagic), kMagic);
                const double d = fma(nsd, (double)r, xd[i]);
                if (i & 1) e1 = fma(d, d, e1); else e0 = fma(d, d, e0);
            }
        }
        double e = e0 + e1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
        if (lane == j) mine = e;
    }
    if (wpr > 1) {
        red_e[w * 32 + lane] = mine;
        __syncthreads();
        mine = 0.0;
        for (int c = 0; c < wpr; ++c) mine += red_e[(row_in_block * wpr + c) * 32 + lane];
    }
    int bj = lane;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double oe = __shfl_xor_sync(0xffffffffu, mine, o);
        const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
        const bool take = (oe < mine) || (oe == mine && oj < bj);
        mine = take ? oe : mine;
        bj = take ? oj : bj;
    }
    if (bj >= ncand) bj = 0;  // only when every distance is NaN or infinite (non-finite input, flagged above)
    if (row_ok && chunk == 0 && lane == 0) {
        job.scales[row] = __fmul_rn(smax, (float)(64 - bj) * 0.015625f);
        if (cand_out) cand_out[row] = bj;
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
using PackFnPtr = void (*)(const PackJobDev*, int, const PackJobInline, uint32_t*, float*, float*, const DenseOutDev*, int, int, unsigned);
struct PackFn { PackFnPtr fn; int form; };  // kernel and its form (kDirect, kStaged2, kAhead)

// nm_debug_set_option("pack_form"): 0 = automatic, 1 = kDirect, 2 = kStaged2, 3 = kAhead for blocks of four warps.
int g_pack_form = 0;


template <int N, int M, bool DENSE_OUT, int FORM>
static PackFn pick_form(int bits) {
    return bits == 8 ? PackFn{(PackFnPtr)pack_kernel<N, M, 8, 128, DENSE_OUT, FORM>, FORM}
                     : PackFn{(PackFnPtr)pack_kernel<N, M, 4, 128, DENSE_OUT, FORM>, FORM};
}

template <int N, int M, bool DENSE_OUT>
static PackFn pick_bits(int bits, int warps, unsigned blocks) {
    if (warps <= kPackMinWarps) {
        // Blocks of four warps.  Measured choices (GB/s on the 24-layer sweep, one unit per block / staged / ahead:
        // 1:4 6231 / 5916 / 6011, 2:4 5520 / 5276 / 5746, 2:8 5643 / 5175 / 5282, 4:8 5090 / 4435 / 5046; one 2:4 layer
        // alone 26.8 / 24.7 / 25.1 us; 72 matrices in four formats, four launches: 130 / 197 / 156 us; dense outputs on
        // the sweep 0.83 / 0.95 / 0.60 of the copy rate):
        //  - dense outputs: staged;
        //  - 2:4: staged for launches of a few rounds per resident block (blocks that start together otherwise alternate
        //    between loading and arithmetic), ahead for very long ones, one unit per block between;
        //  - every other pattern: one unit per block.
        const unsigned staged_blocks = (unsigned)(sm_count() * pack_blocks_per_sm(kStaged2));
        const unsigned ahead_blocks = (unsigned)(sm_count() * pack_blocks_per_sm(kAhead));
        int form = kDirect;
        if (DENSE_OUT) form = kStaged2;
        else if (N == 2 && M == 4) form = blocks <= 8u * staged_blocks ? kStaged2 : (blocks >= 32u * ahead_blocks ? kAhead : kDirect);
        if (g_pack_form >= 1 && g_pack_form <= 3) form = g_pack_form == 1 ? kDirect : g_pack_form == 2 ? kStaged2 : kAhead;
        if (form == kDirect) return pick_form<N, M, DENSE_OUT, kDirect>(bits);
        if (form == kStaged2) return pick_form<N, M, DENSE_OUT, kStaged2>(bits);
        return pick_form<N, M, DENSE_OUT, kAhead>(bits);
    }
    if constexpr (DENSE_OUT) {  // the dense outputs need ~128 registers: blocks of at most 512 threads get them
        if (warps <= 16)
            return bits == 8 ? PackFn{(PackFnPtr)pack_kernel<N, M, 8, 512, true>, kDirect} : PackFn{(PackFnPtr)pack_kernel<N, M, 4, 512, true>, kDirect};
    }
    return bits == 8 ? PackFn{(PackFnPtr)pack_kernel<N, M, 8, 1024, DENSE_OUT>, kDirect} : PackFn{(PackFnPtr)pack_kernel<N, M, 4, 1024, DENSE_OUT>, kDirect};
}

template <bool DENSE_OUT = false>
static PackFn pick_kernel(int n, int m, int bits, int warps, unsigned blocks) {
    if (n == m) return pick_bits<4, 4, DENSE_OUT>(bits, warps, blocks);
    if (m == 4) return n == 1 ? pick_bits<1, 4, DENSE_OUT>(bits, warps, blocks) : pick_bits<2, 4, DENSE_OUT>(bits, warps, blocks);
    if (n == 1) return pick_bits<1, 8, DENSE_OUT>(bits, warps, blocks);
    if (n == 2) return pick_bits<2, 8, DENSE_OUT>(bits, warps, blocks);
    return pick_bits<4, 8, DENSE_OUT>(bits, warps, blocks);
}

static int validate_job(const nm_pack_job_t& j) {
    int rc = check_pattern(j.out, j.in, j.n, j.m, j.bits);
    if (rc != NM_OK) return rc;
    if (!j.W || !j.values || !j.scales) return NM_ERR_NULL;
    if (j.n != j.m && !j.meta) return NM_ERR_NULL;
    if (j.in % 4) return NM_ERR_SHAPE;
    if (j.n == j.m && j.in % 4) return NM_ERR_SHAPE;
    if (j.in > 32768) return NM_ERR_UNSUPPORTED;
    if (!aligned(j.W, 16) || (j.U && !aligned(j.U, 16)) || !aligned(j.values, 16) ||
        (j.meta && !aligned(j.meta, 4)) || !aligned(j.scales, 4))
        return NM_ERR_ALIGN;
    return NM_OK;
}

static int wpr_log2_of(int in) {
    int chunks = (in + 1023) / 1024, l = 0;
    while ((1 << l) < chunks) ++l;
    return l;
}

static PackJobDev to_dev(const nm_pack_job_t& j) {
    PackJobDev d;
    d.W = j.W; d.U = j.U; d.values = (uint8_t*)j.values; d.meta = (uint32_t*)j.meta; d.scales = j.scales;
    d.out = j.out; d.in = j.in; d.wpr_log2 = wpr_log2_of(j.in); d.unit_begin = 0;
    d.vrow_bytes = (unsigned)values_row_bytes(j.in, j.n, j.m, j.bits);
    d.mrow_words = (unsigned)meta_row_words(j.in, j.n, j.m);
    return d;
}

// jobs_dev != nullptr: table of njobs entries in device memory; else the first njobs (>= 1) entries of `inl`.
static int launch_table(PackFn k, const PackJobDev* jobs_dev, int njobs, const PackJobInline& inl, unsigned blocks,
                        int warps, uint32_t* status, cudaStream_t stream, float* Z, float* U_next,
                        const DenseOutDev* dense_jobs, int group_mode, int group_rows) {
    // chunk tile(s), two sets of row-maximum slots, the 4:8 position table; staged form: also two barriers per warp
    // and the abort flag, and a grid that stays resident
    const bool staged = k.form == kStaged2, persistent = k.form != kDirect;
    size_t smem = (size_t)warps * ((staged ? 1024 : 256) * sizeof(float4) + 2 * sizeof(float)) + 512 +
                  (staged ? (size_t)warps * 16 + 16 : 0);
    const PackFnPtr fn = k.fn;
    if (smem > 48 * 1024) {  // the attribute is set once per kernel and device
        struct Done { const void* fn; int dev; };
        static std::mutex mu;
        static std::vector<Done> done;
        int dev = 0;
        NM_CUDA_TRY(cudaGetDevice(&dev));
        std::lock_guard<std::mutex> lock(mu);
        bool found = false;
        for (const Done& d : done) found = found || (d.fn == (const void*)fn && d.dev == dev);
        if (!found) {
            NM_CUDA_TRY(cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            done.push_back(Done{(const void*)fn, dev});
        }
    }
    const unsigned grid = persistent ? std::min(blocks, (unsigned)(sm_count() * pack_blocks_per_sm(k.form))) : blocks;
    fn<<<grid, warps * 32, smem, stream>>>(jobs_dev, njobs, inl, status, Z, U_next, dense_jobs, group_mode, group_rows, blocks);
    NM_CUDA_TRY(cudaGetLastError());
    return NM_OK;
}

static int launch(PackFn fn, const PackJobDev* jobs_dev, int njobs, const PackJobDev& single,
                  unsigned blocks, int warps, uint32_t* status, cudaStream_t stream,
                  float* Z = nullptr, float* U_next = nullptr, const DenseOutDev* dense_jobs = nullptr,
                  int group_mode = kGroupNone, int group_rows = 0) {
    PackJobInline inl{};
    inl.j[0] = single;
    return launch_table(fn, jobs_dev, njobs, inl, blocks, warps, status, stream, Z, U_next, dense_jobs, group_mode, group_rows);
}

using DistFn = void (*)(const PackJobDev*, int, PackJobDev, uint32_t*, int, int32_t*);

template <int N, int M>
static DistFn pick_dist_bits(int bits, int warps) {
    if (warps <= kPackMinWarps)
        return bits == 8 ? (DistFn)dist_scale_kernel<N, M, 8, 128> : (DistFn)dist_scale_kernel<N, M, 4, 128>;
    if (warps <= 16)  // the kept values as fp32 and fp64 need up to ~128 registers
        return bits == 8 ? (DistFn)dist_scale_kernel<N, M, 8, 512> : (DistFn)dist_scale_kernel<N, M, 4, 512>;
    return bits == 8 ? (DistFn)dist_scale_kernel<N, M, 8, 1024> : (DistFn)dist_scale_kernel<N, M, 4, 1024>;
}

static DistFn pick_dist(int n, int m, int bits, int warps) {
    if (n == m) return pick_dist_bits<4, 4>(bits, warps);
    if (m == 4) return n == 1 ? pick_dist_bits<1, 4>(bits, warps) : pick_dist_bits<2, 4>(bits, warps);
    if (n == 1) return pick_dist_bits<1, 8>(bits, warps);
    if (n == 2) return pick_dist_bits<2, 8>(bits, warps);
    return pick_dist_bits<4, 8>(bits, warps);
}

static int launch_dist(DistFn fn, const PackJobDev* jobs_dev, int njobs, const PackJobDev& single, unsigned blocks,
                       int warps, uint32_t* status, cudaStream_t stream, int ncand, int32_t* cand) {
    size_t smem = (size_t)warps * (256 * sizeof(float4) + 32 * sizeof(double) + sizeof(float));
    if (smem > 48 * 1024)
        NM_CUDA_TRY(cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    fn<<<blocks, warps * 32, smem, stream>>>(jobs_dev, njobs, single, status, ncand, cand);
    NM_CUDA_TRY(cudaGetLastError());
    return NM_OK;
}

// One matrix: the ADMM-Dist scales into job.scales (and the winning candidate numbers into `cand`).
static int launch_dist_single(const nm_pack_job_t& j, int ncand, int32_t* cand, uint32_t* status, cudaStream_t stream) {
    PackJobDev d = to_dev(j);
    const int warps = std::max(kPackMinWarps, 1 << d.wpr_log2);
    const int rows_per_block = warps >> d.wpr_log2;
    const unsigned blocks = (unsigned)((j.out + rows_per_block - 1) / rows_per_block);
    return launch_dist(pick_dist(j.n, j.m, j.bits, warps), nullptr, 0, d, blocks, warps, status, stream, ncand, cand);
}

// Shared by the batched entry points: groups the jobs that can share one launch (same pattern, code width
// and block size), writes the device job table(s) into `ws` and launches one kernel per group.
template <bool DENSE_OUT>
static int launch_batched(const nm_pack_job_t* jobs, const DenseOutDev* dense, int njobs, void* ws,
                          uint32_t* status, cudaStream_t s, bool grouped = false, int group_rows = 0,
                          int dist_ncand = 0) {
    // Group jobs that can share one launch: same (n == m ? dense : n, m), bits and block size.
    struct Key { int n, m, bits, warps; };
    std::vector<Key> keys;
    std::vector<std::vector<int>> groups;
    for (int i = 0; i < njobs; ++i) {
        const nm_pack_job_t& j = jobs[i];
        if (j.out == 0 || j.in == 0) continue;
        Key k{j.n == j.m ? 4 : j.n, j.n == j.m ? 4 : j.m, j.bits,
              std::max(nm::kPackMinWarps, 1 << nm::wpr_log2_of(j.in))};
        size_t g = 0;
        for (; g < keys.size(); ++g)
            if (keys[g].n == k.n && keys[g].m == k.m && keys[g].bits == k.bits && keys[g].warps == k.warps) break;
        if (g == keys.size()) { keys.push_back(k); groups.emplace_back(); }
        groups[g].push_back(i);
    }
    std::vector<nm::PackJobDev> table;
    std::vector<DenseOutDev> dense_table;  // same order as `table`
    table.reserve(njobs);
    std::vector<unsigned> group_blocks(keys.size());
    std::vector<size_t> group_first(keys.size());
    for (size_t g = 0; g < keys.size(); ++g) {
        unsigned blocks = 0;
        group_first[g] = table.size();
        for (int i : groups[g]) {
            nm::PackJobDev d = nm::to_dev(jobs[i]);
            int rows_per_block = keys[g].warps >> d.wpr_log2;
            d.unit_begin = blocks;
            unsigned long long nb = ((unsigned long long)d.out + rows_per_block - 1) / rows_per_block;
            if (blocks + nb > 0x7fffffffull) return NM_ERR_UNSUPPORTED;
            blocks += (unsigned)nb;
            table.push_back(d);
            if (DENSE_OUT) dense_table.push_back(dense[i]);
        }
        group_blocks[g] = blocks;
    }
    // Small plain batches: every group's table fits in the kernel's parameters, nothing is copied to `ws`.
    if (!DENSE_OUT && !grouped && dist_ncand == 0) {
        bool fits = true;
        for (size_t g = 0; g < keys.size(); ++g) fits = fits && groups[g].size() <= (size_t)kInlineJobs;
        if (fits) {
            for (size_t g = 0; g < keys.size(); ++g) {
                PackJobInline inl{};
                for (size_t i = 0; i < groups[g].size(); ++i) inl.j[i] = table[group_first[g] + i];
                int rc = nm::launch_table(nm::pick_kernel<DENSE_OUT>(keys[g].n, keys[g].m, keys[g].bits, keys[g].warps, group_blocks[g]), nullptr,
                                          (int)groups[g].size(), inl, group_blocks[g], keys[g].warps, status, s, nullptr,
                                          nullptr, nullptr, kGroupNone, 0);
                if (rc != NM_OK) return rc;
            }
            return NM_OK;
        }
    }
    // The job table goes to `ws` with an asynchronous copy from this function's own (pageable) vector.  Launched
    // eagerly the source is staged before the call returns, so `table` may go away.  Under stream capture the
    // copy node would keep the host pointer and every replay of the graph would read freed memory (and the
    // kernels would follow whatever pointers they find there): such a call is refused before anything is enqueued.
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    NM_CUDA_TRY(cudaStreamIsCapturing(s, &capture));
    if (capture != cudaStreamCaptureStatusNone) return NM_ERR_UNSUPPORTED;
    NM_CUDA_TRY(cudaMemcpyAsync(ws, table.data(), table.size() * sizeof(nm::PackJobDev),
                                cudaMemcpyHostToDevice, s));
    // the dense-output table follows the job table (njobs entries were reserved for each)
    DenseOutDev* dense_dev = reinterpret_cast<DenseOutDev*>(reinterpret_cast<PackJobDev*>(ws) + njobs);
    if (DENSE_OUT)
        NM_CUDA_TRY(cudaMemcpyAsync(dense_dev, dense_table.data(), dense_table.size() * sizeof(DenseOutDev),
                                    cudaMemcpyHostToDevice, s));
    if (grouped) {
        // group-wise scales: clear, fold the row maxima per group (a first pass of the same kernel), finish
        for (size_t g = 0; g < keys.size(); ++g) {
            const nm::PackJobDev* dev = reinterpret_cast<const nm::PackJobDev*>(ws) + group_first[g];
            group_prepare_kernel<<<(unsigned)groups[g].size(), 256, 0, s>>>(dev, group_rows, keys[g].bits, 0);
            NM_CUDA_TRY(cudaGetLastError());
            int rc = nm::launch(nm::pick_kernel<DENSE_OUT>(keys[g].n, keys[g].m, keys[g].bits, keys[g].warps, group_blocks[g]), dev,
                                (int)groups[g].size(), nm::PackJobDev{}, group_blocks[g], keys[g].warps, status, s,
                                nullptr, nullptr, DENSE_OUT ? dense_dev + group_first[g] : nullptr, kGroupMaxPass, group_rows);
            if (rc != NM_OK) return rc;
            group_prepare_kernel<<<(unsigned)groups[g].size(), 256, 0, s>>>(dev, group_rows, keys[g].bits, 1);
            NM_CUDA_TRY(cudaGetLastError());
        }
    }
    if (dist_ncand > 0) {
        // ADMM-Dist: the scale search writes every job's scales, the projection below takes them
        for (size_t g = 0; g < keys.size(); ++g) {
            const nm::PackJobDev* dev = reinterpret_cast<const nm::PackJobDev*>(ws) + group_first[g];
            int rc = nm::launch_dist(nm::pick_dist(keys[g].n, keys[g].m, keys[g].bits, keys[g].warps), dev,
                                     (int)groups[g].size(), nm::PackJobDev{}, group_blocks[g], keys[g].warps, status, s,
                                     dist_ncand, nullptr);
            if (rc != NM_OK) return rc;
        }
    }
    for (size_t g = 0; g < keys.size(); ++g) {
        const nm::PackJobDev* dev = reinterpret_cast<const nm::PackJobDev*>(ws) + group_first[g];
        int rc = nm::launch(nm::pick_kernel<DENSE_OUT>(keys[g].n, keys[g].m, keys[g].bits, keys[g].warps, group_blocks[g]), dev,
                            (int)groups[g].size(), nm::PackJobDev{}, group_blocks[g], keys[g].warps,
                            status, s, nullptr, nullptr, DENSE_OUT ? dense_dev + group_first[g] : nullptr,
                            (grouped || dist_ncand > 0) ? kGroupScalesGiven : kGroupNone, group_rows);
        if (rc != NM_OK) return rc;
    }
    return NM_OK;
}

static int validate_admm(const float* W, const float* U, int out, int in, int n, int m, int bits, const float* Z,
                         const float* U_next, const void* values, const void* meta, const float* scales) {
    int rc = check_pattern(out, in, n, m, bits);
    if (rc != NM_OK) return rc;
    if (!W || !Z) return NM_ERR_NULL;
    if (in % 4) return NM_ERR_SHAPE;
    if (in > 32768) return NM_ERR_UNSUPPORTED;
    if (!aligned(W, 16) || (U && !aligned(U, 16)) || !aligned(Z, 16) || (U_next && !aligned(U_next, 16)) ||
        (values && !aligned(values, 16)) || (meta && !aligned(meta, 4)) || (scales && !aligned(scales, 4)))
        return NM_ERR_ALIGN;
    return NM_OK;
}

}  // namespace nm

extern "C" {

int nm_project_pack(const float* W, const float* U, int out, int in, int n, int m, int bits,
                    void* values, void* meta, float* scales, uint32_t* status, void* stream) {
    nm_pack_job_t j{W, U, out, in, n, m, bits, values, meta, scales};
    int rc = nm::validate_job(j);
    if (rc != NM_OK) return rc;
    if (out == 0 || in == 0) return NM_OK;
    nm::PackJobDev d = nm::to_dev(j);
    int warps = std::max(nm::kPackMinWarps, 1 << d.wpr_log2);
    int rows_per_block = warps >> d.wpr_log2;
    unsigned blocks = (unsigned)((out + rows_per_block - 1) / rows_per_block);
    return nm::launch(nm::pick_kernel(n, m, bits, warps, blocks), nullptr, 0, d, blocks, warps, status, (cudaStream_t)stream);
}

int nm_admm_project(const float* W, const float* U, int out, int in, int n, int m, int bits, float* Z,
                    float* U_next, void* values, void* meta, float* scales, uint32_t* status, void* stream) {
    int rc = nm::validate_admm(W, U, out, in, n, m, bits, Z, U_next, values, meta, scales);
    if (rc != NM_OK) return rc;
    if (out == 0 || in == 0) return NM_OK;
    nm_pack_job_t j{W, U, out, in, n, m, bits, values, meta, scales};
    nm::PackJobDev d = nm::to_dev(j);
    int warps = std::max(nm::kPackMinWarps, 1 << d.wpr_log2);
    int rows_per_block = warps >> d.wpr_log2;
    unsigned blocks = (unsigned)((out + rows_per_block - 1) / rows_per_block);
    return nm::launch(nm::pick_kernel<true>(n, m, bits, warps, blocks), nullptr, 0, d, blocks, warps, status,
                      (cudaStream_t)stream, Z, U_next);
}

int nm_project_pack_grouped(const float* W, const float* U, int out, int in, int n, int m, int bits,
                            int group_rows, void* values, void* meta, float* scales, uint32_t* status,
                            void* stream) {
    nm_pack_job_t j{W, U, out, in, n, m, bits, values, meta, scales};
    int rc = nm::validate_job(j);
    if (rc != NM_OK) return rc;
    if (out == 0 || in == 0) return NM_OK;
    rc = nm::launch_group_scales(W, U, out, in, bits, group_rows, scales, (cudaStream_t)stream);
    if (rc != NM_OK) return rc;
    nm::PackJobDev d = nm::to_dev(j);
    int warps = std::max(nm::kPackMinWarps, 1 << d.wpr_log2);
    int rows_per_block = warps >> d.wpr_log2;
    unsigned blocks = (unsigned)((out + rows_per_block - 1) / rows_per_block);
    return nm::launch(nm::pick_kernel(n, m, bits, warps, blocks), nullptr, 0, d, blocks, warps, status, (cudaStream_t)stream,
                      nullptr, nullptr, nullptr, nm::kGroupScalesGiven, group_rows);
}

int nm_admm_project_grouped(const float* W, const float* U, int out, int in, int n, int m, int bits,
                            int group_rows, float* Z, float* U_next, void* values, void* meta, float* scales,
                            uint32_t* status, void* stream) {
    int rc = nm::validate_admm(W, U, out, in, n, m, bits, Z, U_next, values, meta, scales);
    if (rc != NM_OK) return rc;
    if (!scales) return NM_ERR_NULL;  // also the scratch of the group maxima
    if (out == 0 || in == 0) return NM_OK;
    rc = nm::launch_group_scales(W, U, out, in, bits, group_rows, scales, (cudaStream_t)stream);
    if (rc != NM_OK) return rc;
    nm_pack_job_t j{W, U, out, in, n, m, bits, values, meta, scales};
    nm::PackJobDev d = nm::to_dev(j);
    int warps = std::max(nm::kPackMinWarps, 1 << d.wpr_log2);
    int rows_per_block = warps >> d.wpr_log2;
    unsigned blocks = (unsigned)((out + rows_per_block - 1) / rows_per_block);
    return nm::launch(nm::pick_kernel<true>(n, m, bits, warps, blocks), nullptr, 0, d, blocks, warps, status,
                      (cudaStream_t)stream, Z, U_next, nullptr, nm::kGroupScalesGiven, group_rows);
}

int nm_dist_scales(const float* W, const float* U, int out, int in, int n, int m, int bits, int ncand,
                   float* scales, int32_t* cand, uint32_t* status, void* stream) {
    int rc = nm::check_pattern(out, in, n, m, bits);
    if (rc != NM_OK) return rc;
    if (ncand < 1 || ncand > NM_DIST_MAX_CANDIDATES) return NM_ERR_SHAPE;
    if (!W || !scales) return NM_ERR_NULL;
    if (in % 4) return NM_ERR_SHAPE;
    if (in > 32768) return NM_ERR_UNSUPPORTED;
    if (!nm::aligned(W, 16) || (U && !nm::aligned(U, 16)) || !nm::aligned(scales, 4) || (cand && !nm::aligned(cand, 4)))
        return NM_ERR_ALIGN;
    if (out == 0 || in == 0) return NM_OK;
    nm_pack_job_t j{W, U, out, in, n, m, bits, nullptr, nullptr, scales};
    return nm::launch_dist_single(j, ncand, cand, status, (cudaStream_t)stream);
}

int nm_project_pack_dist(const float* W, const float* U, int out, int in, int n, int m, int bits, int ncand,
                         void* values, void* meta, float* scales, uint32_t* status, void* stream) {
    nm_pack_job_t j{W, U, out, in, n, m, bits, values, meta, scales};
    int rc = nm::validate_job(j);
    if (rc != NM_OK) return rc;
    if (ncand < 1 || ncand > NM_DIST_MAX_CANDIDATES) return NM_ERR_SHAPE;
    if (out == 0 || in == 0) return NM_OK;
    rc = nm::launch_dist_single(j, ncand, nullptr, status, (cudaStream_t)stream);
    if (rc != NM_OK) return rc;
    nm::PackJobDev d = nm::to_dev(j);
    int warps = std::max(nm::kPackMinWarps, 1 << d.wpr_log2);
    int rows_per_block = warps >> d.wpr_log2;
    unsigned blocks = (unsigned)((out + rows_per_block - 1) / rows_per_block);
    return nm::launch(nm::pick_kernel(n, m, bits, warps, blocks), nullptr, 0, d, blocks, warps, status, (cudaStream_t)stream,
                      nullptr, nullptr, nullptr, nm::kGroupScalesGiven, 0);
}

int nm_admm_project_dist(const float* W, const float* U, int out, int in, int n, int m, int bits, int ncand,
                         float* Z, float* U_next, void* values, void* meta, float* scales, uint32_t* status,
                         void* stream) {
    int rc = nm::validate_admm(W, U, out, in, n, m, bits, Z, U_next, values, meta, scales);
    if (rc != NM_OK) return rc;
    if (!scales) return NM_ERR_NULL;  // the search hands its result to the projection through it
    if (ncand < 1 || ncand > NM_DIST_MAX_CANDIDATES) return NM_ERR_SHAPE;
    if (out == 0 || in == 0) return NM_OK;
    nm_pack_job_t j{W, U, out, in, n, m, bits, values, meta, scales};
    rc = nm::launch_dist_single(j, ncand, nullptr, status, (cudaStream_t)stream);
    if (rc != NM_OK) return rc;
    nm::PackJobDev d = nm::to_dev(j);
    int warps = std::max(nm::kPackMinWarps, 1 << d.wpr_log2);
    int rows_per_block = warps >> d.wpr_log2;
    unsigned blocks = (unsigned)((out + rows_per_block - 1) / rows_per_block);
    return nm::launch(nm::pick_kernel<true>(n, m, bits, warps, blocks), nullptr, 0, d, blocks, warps, status,
                      (cudaStream_t)stream, Z, U_next, nullptr, nm::kGroupScalesGiven, 0);
}

int nm_project_pack_dist_batched(const nm_pack_job_t* jobs, int njobs, int ncand, void* ws, size_t ws_bytes,
                                 uint32_t* status, void* stream) {
    if (njobs < 0) return NM_ERR_SHAPE;
    if (ncand < 1 || ncand > NM_DIST_MAX_CANDIDATES) return NM_ERR_SHAPE;
    if (njobs == 0) return NM_OK;
    if (!jobs) return NM_ERR_NULL;
    if (!ws || ws_bytes < nm_pack_workspace_bytes(njobs)) return NM_ERR_WORKSPACE;
    if (!nm::aligned(ws, 16)) return NM_ERR_ALIGN;
    for (int i = 0; i < njobs; ++i) {
        int rc = nm::validate_job(jobs[i]);
        if (rc != NM_OK) return rc;
    }
    return nm::launch_batched<false>(jobs, nullptr, njobs, ws, status, (cudaStream_t)stream, false, 0, ncand);
}

size_t nm_pack_workspace_bytes(int njobs) {
    return njobs <= 0 ? 0 : (size_t)njobs * sizeof(nm::PackJobDev);
}

int nm_project_pack_batched(const nm_pack_job_t* jobs, int njobs, void* ws, size_t ws_bytes,
                            uint32_t* status, void* stream) {
    if (njobs < 0) return NM_ERR_SHAPE;
    if (njobs == 0) return NM_OK;
    if (!jobs) return NM_ERR_NULL;
    if (!ws || ws_bytes < nm_pack_workspace_bytes(njobs)) return NM_ERR_WORKSPACE;
    if (!nm::aligned(ws, 16)) return NM_ERR_ALIGN;
    for (int i = 0; i < njobs; ++i) {
        int rc = nm::validate_job(jobs[i]);
        if (rc != NM_OK) return rc;
    }
    return nm::launch_batched<false>(jobs, nullptr, njobs, ws, status, (cudaStream_t)stream);
}

int nm_admm_project_grouped_batched(const nm_admm_job_t* jobs, int njobs, int group_rows, void* ws,
                                    size_t ws_bytes, uint32_t* status, void* stream) {
    if (njobs < 0) return NM_ERR_SHAPE;
    if (njobs == 0) return NM_OK;
    if (!jobs) return NM_ERR_NULL;
    if (!ws || ws_bytes < nm_admm_workspace_bytes(njobs)) return NM_ERR_WORKSPACE;
    if (!nm::aligned(ws, 16)) return NM_ERR_ALIGN;
    std::vector<nm_pack_job_t> pj(njobs);
    std::vector<nm::DenseOutDev> dj(njobs);
    for (int i = 0; i < njobs; ++i) {
        const nm_admm_job_t& a = jobs[i];
        int rc = nm::validate_admm(a.W, a.U, a.out, a.in, a.n, a.m, a.bits, a.Z, a.U_next, a.values, a.meta, a.scales);
        if (rc != NM_OK) return rc;
        if (!a.scales) return NM_ERR_NULL;  // also the scratch of the group maxima
        pj[i] = nm_pack_job_t{a.W, a.U, a.out, a.in, a.n, a.m, a.bits, a.values, a.meta, a.scales};
        dj[i] = nm::DenseOutDev{a.Z, a.U_next};
    }
    return nm::launch_batched<true>(pj.data(), dj.data(), njobs, ws, status, (cudaStream_t)stream, true, group_rows);
}

int nm_project_pack_grouped_batched(const nm_pack_job_t* jobs, int njobs, int group_rows, void* ws,
                                    size_t ws_bytes, uint32_t* status, void* stream) {
    if (njobs < 0) return NM_ERR_SHAPE;
    if (njobs == 0) return NM_OK;
    if (!jobs) return NM_ERR_NULL;
    if (!ws || ws_bytes < nm_pack_workspace_bytes(njobs)) return NM_ERR_WORKSPACE;
    if (!nm::aligned(ws, 16)) return NM_ERR_ALIGN;
    for (int i = 0; i < njobs; ++i) {
        int rc = nm::validate_job(jobs[i]);
        if (rc != NM_OK) return rc;
    }
    return nm::launch_batched<false>(jobs, nullptr, njobs, ws, status, (cudaStream_t)stream, true, group_rows);
}

int nm_admm_project_dist_batched(const nm_admm_job_t* jobs, int njobs, int ncand, void* ws, size_t ws_bytes,
                                 uint32_t* status, void* stream) {
    if (njobs < 0) return NM_ERR_SHAPE;
    if (ncand < 1 || ncand > NM_DIST_MAX_CANDIDATES) return NM_ERR_SHAPE;
    if (njobs == 0) return NM_OK;
    if (!jobs) return NM_ERR_NULL;
    if (!ws || ws_bytes < nm_admm_workspace_bytes(njobs)) return NM_ERR_WORKSPACE;
    if (!nm::aligned(ws, 16)) return NM_ERR_ALIGN;
    std::vector<nm_pack_job_t> pj(njobs);
    std::vector<nm::DenseOutDev> dj(njobs);
    for (int i = 0; i < njobs; ++i) {
        const nm_admm_job_t& a = jobs[i];
        int rc = nm::validate_admm(a.W, a.U, a.out, a.in, a.n, a.m, a.bits, a.Z, a.U_next, a.values, a.meta, a.scales);
        if (rc != NM_OK) return rc;
        if (!a.scales) return NM_ERR_NULL;  // the search hands its result to the projection through it
        pj[i] = nm_pack_job_t{a.W, a.U, a.out, a.in, a.n, a.m, a.bits, a.values, a.meta, a.scales};
        dj[i] = nm::DenseOutDev{a.Z, a.U_next};
    }
    return nm::launch_batched<true>(pj.data(), dj.data(), njobs, ws, status, (cudaStream_t)stream, false, 0, ncand);
}

size_t nm_admm_workspace_bytes(int njobs) {
    return njobs <= 0 ? 0 : (size_t)njobs * (sizeof(nm::PackJobDev) + sizeof(nm::DenseOutDev));
}

int nm_admm_project_batched(const nm_admm_job_t* jobs, int njobs, void* ws, size_t ws_bytes,
                            uint32_t* status, void* stream) {
    if (njobs < 0) return NM_ERR_SHAPE;
    if (njobs == 0) return NM_OK;
    if (!jobs) return NM_ERR_NULL;
    if (!ws || ws_bytes < nm_admm_workspace_bytes(njobs)) return NM_ERR_WORKSPACE;
    if (!nm::aligned(ws, 16)) return NM_ERR_ALIGN;
    std::vector<nm_pack_job_t> pj(njobs);
    std::vector<nm::DenseOutDev> dj(njobs);
    for (int i = 0; i < njobs; ++i) {
        const nm_admm_job_t& a = jobs[i];
        int rc = nm::validate_admm(a.W, a.U, a.out, a.in, a.n, a.m, a.bits, a.Z, a.U_next, a.values, a.meta, a.scales);
        if (rc != NM_OK) return rc;
        pj[i] = nm_pack_job_t{a.W, a.U, a.out, a.in, a.n, a.m, a.bits, a.values, a.meta, a.scales};
        dj[i] = nm::DenseOutDev{a.Z, a.U_next};
    }
    return nm::launch_batched<true>(pj.data(), dj.data(), njobs, ws, status, (cudaStream_t)stream);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Batched projection without any caller-provided or library-allocated scratch.
// The job table lives in a fixed device array that is part of the loaded library image.
// ---------------------------------------------------------------------------------------------
namespace nm {

constexpr int kNoAllocMaxJobs = 1024;  // 1024 jobs x 64 bytes = 64 KB held on every GPU that loads the library
static __device__ __align__(256) unsigned char g_noalloc_job_table[kNoAllocMaxJobs * sizeof(PackJobDev)];

// In host code `g_noalloc_job_table` is only a handle; its device address has to be asked for,
// once per device, with that device current.
static int noalloc_table_address(void** out) {
    static void* cached[64] = {nullptr};
    static std::mutex mu;
    int dev = 0;
    NM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return record_text_error("device ordinal beyond 63");
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void* p = nullptr;
        NM_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_job_table));
        cached[dev] = p;
    }
    *out = cached[dev];
    return NM_OK;
}

}  // namespace nm

extern "C" int nm_project_pack_batched_noalloc(const nm_pack_job_t* jobs, int njobs, uint32_t* status,
                                               void* stream) {
    if (njobs < 0) return NM_ERR_SHAPE;
    if (njobs > nm::kNoAllocMaxJobs) return NM_ERR_UNSUPPORTED;  // beyond NM_NOALLOC_MAX_JOBS
    if (njobs == 0) return NM_OK;
    void* table = nullptr;
    int rc = nm::noalloc_table_address(&table);
    if (rc != NM_OK) return rc;
    return nm_project_pack_batched(jobs, njobs, table, sizeof(nm::g_noalloc_job_table), status, stream);
}
