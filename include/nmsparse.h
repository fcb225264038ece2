/*
 * nmsparse.h -- C ABI of the B200 (sm_100a) N:M-sparse low-bit integer linear layer and of the
 * projection / quantise / pack step that produces its weights.
 *
 * The operations are those of "Compressing Pre-trained Transformers via Low-Bit NxM Sparsity"
 * (arxiv 2206.15014).  Patterns are written kept:group -- "2:4" keeps n = 2 of every m = 4
 * consecutive weights (the paper writes the same pattern "4:2").
 *
 * General rules for every entry point
 *   - Pointers are DEVICE pointers unless the comment says "host".  The caller owns every buffer;
 *     the library allocates nothing and keeps no pointer after a call returns.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     return without synchronising, unless stated.
 *   - Return value: NM_OK or a negative NM_ERR_* code detected on the host; nothing is enqueued
 *     when an error is returned.  Conditions only the device can see (non-finite weights, a bounded
 *     wait that expired) are OR-ed as NM_STATUS_* bits into the optional `status` device word,
 *     which the caller zeroes beforehand and reads with nm_poll_status().
 *   - No exceptions, no exit(), no output to stdout/stderr.
 *
 * Layouts
 *   W, U     fp32 [out, in] row-major (nn.Linear layout).  Groups of m run along `in`, the reduction
 *            dimension.  `in` must be a multiple of m and of 4; rows must start 16-byte aligned.
 *   values   kept integer codes in ascending position inside each group, row-major
 *            [out, in*n/m].  bits = 8: one int8 per code.  bits = 4: two's-complement nibbles, even
 *            element in bits 3:0 and odd element in bits 7:4 of a byte.
 *   meta     position-in-group of each kept code: 2-bit fields for m = 4, 4-bit fields for m = 8,
 *            least-significant field first in element order, in little-endian u32 words; every row
 *            is padded with zero bits to a whole number of words.  n == m (dense) has no metadata.
 *   scales   fp32 [out], one symmetric scale per output channel.
 *   X        int8 [tokens, in] row-major;  Y fp32 [tokens, out] row-major.
 */
#ifndef NMSPARSE_H_
#define NMSPARSE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NM_OK 0
#define NM_ERR_NULL (-1)        /* a required pointer is NULL */
#define NM_ERR_SHAPE (-2)       /* n < 1, n > m, in % m != 0, negative size, row not a whole number of bytes */
#define NM_ERR_UNSUPPORTED (-3) /* m not in {4, 8} (unless n == m), bits not in {4, 8}, size beyond a stated limit */
#define NM_ERR_ALIGN (-4)       /* pointer or row pitch not aligned as the call requires */
#define NM_ERR_WORKSPACE (-5)   /* workspace missing or smaller than nm_*_workspace_bytes() */
#define NM_ERR_CUDA (-6)        /* a CUDA runtime / driver call failed (see nm_last_cuda_error) */
#define NM_ERR_NONFINITE (-7)   /* reported by nm_poll_status: NaN or Inf met in W + U */
#define NM_ERR_TIMEOUT (-8)     /* reported by nm_poll_status: a bounded device-side wait expired */

#define NM_STATUS_NONFINITE 1u /* bit in the device status word */
#define NM_STATUS_TIMEOUT 2u   /* bit in the device status word */

/* A packed weight matrix: host struct holding device pointers (see "Layouts"). */
typedef struct nm_packed_t {
    int32_t out, in; /* output channels, input features (reduction length) */
    int32_t n, m;    /* kept : group; n == m means dense */
    int32_t bits;    /* 8 or 4 */
    const void *values;
    const void *meta; /* NULL iff n == m */
} nm_packed_t;

/* One matrix of a batched projection (host struct, device pointers). */
typedef struct nm_pack_job_t {
    const float *W;
    const float *U; /* NULL: project W alone */
    int32_t out, in, n, m, bits;
    void *values;
    void *meta; /* NULL iff n == m */
    float *scales;
} nm_pack_job_t;

/*
 * Sizes in bytes of `values` and `meta` for an [out, in] matrix (host only, touches no device).
 * Storage accounting of Table 1 / Table 4: value bits plus index bits per kept weight.
 */
int nm_packed_sizes(int out, int in, int n, int m, int bits, size_t *values_bytes,
                    size_t *meta_bytes);

/*
 * N:M magnitude projection + per-output-channel symmetric quantisation + packing of one matrix.
 *   V = W + U                          argument of the ADMM Z-update, Eq. 3 (U may be NULL)
 *   support = the n largest |v| of every group of m, equal magnitudes -> lower index kept
 *                                      (Euclidean projection onto the N:M constraint, Sec. 3.2)
 *   s[r] = max_k |V[r,k]| / (2^(bits-1) - 1),  s[r] = 1 for an all-zero row
 *                                      (ADMM-Max scale, Sec. 3.3.1)
 *   q = clamp(rne(v / s[r]), -2^(bits-1), 2^(bits-1) - 1)      (Eq. 5, offset 0)
 * The same arithmetic is the forward fake-quantisation of STE-QAT (Sec. 3.3.2): s * q.
 * Accepted: (n, m) in {1:4, 2:4, 1:8, 2:8, 4:8} or n == m; bits in {4, 8}; in <= 32768.
 * W, U, values 16-byte aligned, meta and scales 4-byte aligned.
 * Sets NM_STATUS_NONFINITE in *status (nullable) when W + U holds NaN/Inf; outputs of such rows are
 * unspecified.  One pass over W and U; outputs are written once.  Rows of at most 4096 values reach the
 * kernel through bulk copies whose arrival a warp awaits for about a second at most: NM_STATUS_TIMEOUT in
 * *status when such a wait expired (the outputs are then void); the same holds for every entry point below
 * that projects.
 */
int nm_project_pack(const float *W, const float *U, int out, int in, int n, int m, int bits,
                    void *values, void *meta, float *scales, uint32_t *status, void *stream);

/*
 * One ADMM projection step with dense outputs (Eq. 3 for the joint constraint: the sparsity and the
 * quantisation projection solved in sequence, Sec. 3.3.1), also the forward pass of the STE
 * fake-quantiser (Sec. 3.3.2) when U and U_next are NULL:
 *   V = W + U (U NULL = 0);  s[r] = ADMM-Max scale of row r of V;
 *   Z[r,k]      = s[r] * code[r,k] where (r,k) is kept, 0 where it is pruned   (Eq. 5 then Eq. 4)
 *   U_next[r,k] = V[r,k] - Z[r,k]                  (scaled-form dual update U + W - Z; NULL = not wanted)
 * with exactly the support, scales and codes nm_project_pack produces.  Z, U_next: device fp32
 * [out, in] row-major, 16-byte aligned, caller-owned; U_next may alias U, Z may not alias W or U.
 * values / meta / scales: the packed outputs of nm_project_pack, each may be NULL when not wanted.
 * One pass over HBM: W and U read once, every output written once.  Shapes, errors and the
 * NM_STATUS_NONFINITE bit as for nm_project_pack.
 */
int nm_admm_project(const float *W, const float *U, int out, int in, int n, int m, int bits, float *Z,
                    float *U_next, void *values, void *meta, float *scales, uint32_t *status,
                    void *stream);

/*
 * Group-wise quantisation (Sec. 3.3: several neurons of a weight matrix may share one scale, whole
 * neurons always do; the paper's experiments use 32 per scale): output channels r with the same
 * r / group_rows share the ADMM-Max scale max |W + U| over those rows / (2^(bits-1) - 1); group_rows
 * <= 0 means one scale for the whole matrix; the last group may be short.  scales[r] (required: it
 * is also the scratch of the group maxima) receives the scale of row r's group, so that it can be
 * handed to nm_int_linear unchanged.  Otherwise as nm_project_pack / nm_admm_project.  Two passes
 * over W and U (the maxima, then the projection); for matrices that fit in L2 the second pass is
 * served from there.
 */
int nm_project_pack_grouped(const float *W, const float *U, int out, int in, int n, int m, int bits,
                            int group_rows, void *values, void *meta, float *scales,
                            uint32_t *status, void *stream);
int nm_admm_project_grouped(const float *W, const float *U, int out, int in, int n, int m, int bits,
                            int group_rows, float *Z, float *U_next, void *values, void *meta,
                            float *scales, uint32_t *status, void *stream);
/* nm_project_pack_grouped for many matrices (jobs, ws as for nm_project_pack_batched; one group_rows for all):
 * per group of jobs that share (n, m, bits) and block size one launch folds the row maxima, one
 * finishes the scales and one projects and packs. */
int nm_project_pack_grouped_batched(const nm_pack_job_t *jobs, int njobs, int group_rows, void *ws,
                                    size_t ws_bytes, uint32_t *status, void *stream);

/*
 * The same for many matrices with one launch per group of jobs that share (n, m, bits) and block
 * size.  `jobs`: host array of host structs holding device pointers, with the meaning of
 * nm_admm_project's arguments; `ws`: device scratch of at least nm_admm_workspace_bytes(njobs)
 * bytes, 16-byte aligned, caller-owned, reusable once the stream has passed the call.
 */
typedef struct nm_admm_job_t {
    const float *W;
    const float *U; /* NULL: project W alone */
    int32_t out, in, n, m, bits;
    float *Z;
    float *U_next; /* NULL: not wanted; may be U */
    void *values;  /* packed outputs: each NULL when not wanted */
    void *meta;
    float *scales;
} nm_admm_job_t;
size_t nm_admm_workspace_bytes(int njobs);
int nm_admm_project_batched(const nm_admm_job_t *jobs, int njobs, void *ws, size_t ws_bytes,
                            uint32_t *status, void *stream);
/* nm_admm_project_dist for many matrices (one ncand for all; scales required in every job). */
int nm_admm_project_dist_batched(const nm_admm_job_t *jobs, int njobs, int ncand, void *ws,
                                 size_t ws_bytes, uint32_t *status, void *stream);
/* nm_admm_project_grouped for many matrices (one group_rows for all; scales required in every job). */
int nm_admm_project_grouped_batched(const nm_admm_job_t *jobs, int njobs, int group_rows, void *ws,
                                    size_t ws_bytes, uint32_t *status, void *stream);

/*
 * ADMM-Dist scale (Sec. 3.3.1, "Minimize Quantization Distance"): per output channel the scale that
 * minimises the squared Euclidean distance between the channel and its quantised form.  With N:M
 * sparsity the sparsity projection comes first (Sec. 3.3.1, last paragraph), so the distance runs
 * over the kept entries of V = W + U.  The paper states the objective and no procedure; this
 * library sweeps `ncand` candidates (1 .. NM_DIST_MAX_CANDIDATES)
 *     s_j = fl32(s_max * (64 - j) / 64),  j = 0 .. ncand-1,  s_max = the ADMM-Max scale of the row,
 * evaluates E_j = sum over kept k of (v_k - s_j * code_jk)^2 in double (code_jk = Eq. 5 at scale
 * s_j), and takes the smallest E_j, the lowest j among equal ones.  ncand = 1 is ADMM-Max.
 *   nm_dist_scales        scales[out] <- the chosen scale; cand[out] (device int32, nullable) <- j.
 *   nm_project_pack_dist  the search, then nm_project_pack with that scale (codes beyond the
 *                         shrunken range clamp to -2^(bits-1) / 2^(bits-1)-1 as Eq. 5 says).
 *   nm_admm_project_dist  the search, then nm_admm_project with that scale; `scales` is required.
 *   nm_project_pack_dist_batched  many matrices (jobs, ws as for nm_project_pack_batched): per
 *                         group of jobs that share (n, m, bits) and block size one launch searches
 *                         and one projects and packs.
 * Two passes over W and U (the second is served from L2 for matrices that fit there).  The search
 * is bound by arithmetic, not by memory.  Pointers, shapes, errors and the NM_STATUS_NONFINITE bit
 * as for nm_project_pack; ncand out of range returns NM_ERR_SHAPE.  Which of two candidates whose
 * distances agree to the last few bits of a double wins depends on the order of the summation.
 */
#define NM_DIST_MAX_CANDIDATES 32
int nm_dist_scales(const float *W, const float *U, int out, int in, int n, int m, int bits, int ncand,
                   float *scales, int32_t *cand, uint32_t *status, void *stream);
int nm_project_pack_dist(const float *W, const float *U, int out, int in, int n, int m, int bits,
                         int ncand, void *values, void *meta, float *scales, uint32_t *status,
                         void *stream);
int nm_admm_project_dist(const float *W, const float *U, int out, int in, int n, int m, int bits,
                         int ncand, float *Z, float *U_next, void *values, void *meta, float *scales,
                         uint32_t *status, void *stream);

/*
 * nm_project_pack for a list of matrices with as few launches as their (n, m, bits) allow (one when
 * all jobs share them).  `jobs` is a host array; `ws` is device scratch of at least
 * nm_pack_workspace_bytes(njobs) bytes, 16-byte aligned, which must stay untouched until the
 * enqueued work has finished.  The host array may be reused as soon as the call returns.
 * (Batches in which no more than eight jobs share one (n, m, bits) and block size pass their job table
 * in the kernel's parameters and leave `ws` untouched; it must be provided all the same.)
 * Stream capture: a call that needs the job table in `ws` (more than eight jobs per kernel variant, and every
 * *_batched call of the dense-output, group-wise and ADMM-Dist forms) uploads it from host memory the
 * library owns only until the call returns, so it must not be captured into a CUDA graph: on a capturing
 * stream such a call returns NM_ERR_UNSUPPORTED and enqueues nothing.  The same holds for
 * nm_project_pack_batched_noalloc.
 */
int nm_project_pack_batched(const nm_pack_job_t *jobs, int njobs, void *ws, size_t ws_bytes,
                            uint32_t *status, void *stream);
size_t nm_pack_workspace_bytes(int njobs);
int nm_project_pack_dist_batched(const nm_pack_job_t *jobs, int njobs, int ncand, void *ws,
                                 size_t ws_bytes, uint32_t *status, void *stream);

/*
 * nm_project_pack_batched for callers that cannot provide scratch memory.  (The paper has no
 * counterpart: this entry point exists for deployment reasons only.)
 *
 * Some hosts of this library must not allocate device memory once they are running: inference
 * servers that hand the whole GPU to a memory pool at start-up, real-time loops in which a
 * cudaMalloc (which may synchronise the device and take an unbounded time) is forbidden, and
 * plug-ins that run inside another framework's stream callbacks where allocation is not allowed.
 * For them the job table that nm_project_pack_batched keeps in `ws` lives instead in a fixed
 * device array inside the library image: NM_NOALLOC_MAX_JOBS entries of 64 bytes = 64 KB, present
 * on every GPU that loads the library until the process exits.  This call performs no cudaMalloc,
 * cudaFree or other allocating call; inputs and outputs are still the caller's buffers.
 *
 *   - njobs > NM_NOALLOC_MAX_JOBS returns NM_ERR_UNSUPPORTED and enqueues nothing.
 *   - The first call on each device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one table and each call overwrites the entries it uses
 *     (nothing in it needs clearing).  Two calls whose work overlaps on the GPU -- different
 *     streams, or different host threads on different streams -- race on it: serialise them
 *     (same stream, or an event between them).
 * Results are identical to nm_project_pack_batched on the same jobs.
 */
#define NM_NOALLOC_MAX_JOBS 1024
int nm_project_pack_batched_noalloc(const nm_pack_job_t *jobs, int njobs, uint32_t *status,
                                    void *stream);

/*
 * Integer N:M linear layer (Sec. 5.3: 8-bit activations, weights of <= 8 bits widened to 8 bits for
 * the multipliers, N:M skipping the pruned half of the products) with the dequantisation of Eq. 4
 * fused in:
 *   acc[t,o] = sum_k X[t,k] * Wq[o,k]              exact, int32
 *   Y[t,o]   = fma((float)acc[t,o], sx * sw[o], bias[o])      fp32; bias NULL = 0
 * W is a host struct; sw = per-channel scales from nm_project_pack; sx = activation scale.
 * 2:4, 1:4, 2:8 and 1:8 weights run on the sparse tensor-core path, 4:8 and dense weights on the
 * dense path after decompression in shared memory.  Shape and alignment requirements are those
 * nm_int_linear_check() tests; X, values and meta 16-byte aligned (NM_ERR_ALIGN otherwise; buffers that
 * nm_project_pack filled meet this when they start on a 16-byte boundary); Y, sw, bias 4-byte aligned.
 * `ws`/`ws_bytes`: device scratch of nm_int_linear_workspace_bytes() (may be 0 -> ws may be NULL).
 */
int nm_int_linear(const int8_t *X, int tokens, const nm_packed_t *W, float sx, const float *sw,
                  const float *bias, float *Y, void *ws, size_t ws_bytes, uint32_t *status,
                  void *stream);

/*
 * The same with the activation scale read from device memory (*sx_dev), so that a chain of layers
 * needs no host round trip, and with an optional running maximum: when absmax_out is not NULL the
 * kernel folds max|Y| into *absmax_out (a float the caller zeroes first; updated atomically).
 */
int nm_int_linear_dsx(const int8_t *X, int tokens, const nm_packed_t *W, const float *sx_dev,
                      const float *sw, const float *bias, float *Y, float *absmax_out, void *ws,
                      size_t ws_bytes, uint32_t *status, void *stream);

/*
 * Narrow outputs of the same layer, for encoders that keep their activations at 8 bits between
 * layers (Sec. 4.5, Sec. 5.3) or hand them on in bfloat16: y = fma((float)acc, sx * sw[o], bias[o])
 * is formed as in nm_int_linear and leaves the kernel as
 *   nm_int_linear_q8:   Yq[t,o] = clamp(rne(y / sy), -128, 127)   (Eq. 5 with b = 8 and the scale sy
 *                       fixed ahead of time; IEEE fp32 division, round half to even), int8
 *                       [tokens, out] row-major, directly usable as the next layer's X with sx = sy;
 *                       sy must be a positive, normal, finite float (NM_ERR_SHAPE otherwise);
 *   nm_int_linear_bf16: Y[t,o] = y rounded to bfloat16 (nearest, ties to even), bit patterns as
 *                       uint16 [tokens, out] row-major; 2-byte aligned.
 * All other arguments, errors and ownership as for nm_int_linear.  The output goes through the
 * TMA-store epilogue when its base and row pitch are multiples of 16 bytes (out % 16 == 0 for
 * int8, out % 8 == 0 for bfloat16), else through plain stores.
 */
int nm_int_linear_q8(const int8_t *X, int tokens, const nm_packed_t *W, float sx, const float *sw,
                     const float *bias, float sy, int8_t *Yq, void *ws, size_t ws_bytes,
                     uint32_t *status, void *stream);
int nm_int_linear_bf16(const int8_t *X, int tokens, const nm_packed_t *W, float sx, const float *sw,
                       const float *bias, uint16_t *Ybf16, void *ws, size_t ws_bytes,
                       uint32_t *status, void *stream);

/* The raw int32 accumulators acc[t,o] (row-major [tokens, out]) of the same product, no epilogue. */
int nm_int_linear_acc(const int8_t *X, int tokens, const nm_packed_t *W, int32_t *ACC, void *ws,
                      size_t ws_bytes, uint32_t *status, void *stream);

size_t nm_int_linear_workspace_bytes(int tokens, int out, int in, int n, int m, int bits);

/*
 * Host-only: how the CTA-pair kernel of nm_int_linear walks an [n_out_tiles x n_tok_tiles] grid of tiles
 * with `pairs` CTA pairs (for inspection and tests; it launches nothing).  The tiles are numbered band
 * by band of token tiles, output-tile-major inside a band; pair p works on tiles start[p] ..
 * start[p + 1] - 1 of that numbering, ranges of about equal cost.  resident != 0: weights kept in shared
 * memory (one long run per output tile); else bands of about one pair's share, or of band_request > 0
 * token tiles.  start: [pairs + 1]; tile_out / tile_tok (nullable): [n_out_tiles * n_tok_tiles], the
 * output tile and token tile of every tile number.  Returns the band size (>= 1) or a negative error
 * (pairs must not exceed the number of tiles nor 128).
 */
int nm_pair_tile_plan(int n_tok_tiles, int n_out_tiles, int pairs, int resident, int band_request,
                      int *start, int *tile_out, int *tile_tok);

/*
 * Measurement aid (the paper has no counterpart): the memory traffic of the CTA-pair kernel of nm_int_linear
 * without its arithmetic.  Every CTA pair walks the tiles nm_pair_tile_plan gives it (streamed form); per
 * pipeline stage each CTA loads a box of `a_rows` x `a_row_bytes` (64 or 128) from W, a row-major byte matrix
 * [w_rows, w_row_bytes], and `b_rows` tokens x `b_slices` 128-byte-wide slices from X, int8 [tokens, k_bytes],
 * into a ring of `stages` shared-memory stages; a consumer hands every stage back once it has landed and
 * `delay_clocks` SM clocks have passed; when `stores` != 0 eight warps write the CTA's share of the output
 * tile to Y (fp32 [tokens, w_rows], overwritten with arbitrary values): stores == 1 as [16 tokens][32 channels]
 * boxes, stores == 32 / 64 / 128 as 8 KB boxes that many channels wide.
 * A pair's tile is 2 * a_rows output channels x 2 * b_rows tokens; w_row_bytes / a_row_bytes must equal
 * k_bytes / (128 * b_slices) (the stages per tile).  `loads`: bit 0 = W boxes, bit 1 = X boxes; `producers`: 1 = one thread
 * issues both boxes of a stage, 2 = one thread per operand.  `poll`: how the store warps wait for a tile: 0 = all
 * lanes poll the barrier, 1 = one lane polls and sleeps between polls, 2 (only with stores == 0) = they leave at
 * once, producer and consumer run alone.  `band`: as
 * band_request of nm_pair_tile_plan.  `repeat`: times every pair walks its range.  `clocks` (nullable): u64
 * [CTAs][4] = clock64 at start, at end, global timer (ns) at start, at end of every CTA.  `trace`
 * (nullable): u64 [512][8], for the first 512 stages of CTA 0 the clock64 of the producer before and after its wait for the
 * stage, after arming the barrier, after issuing the W load, after issuing the X load, and of the consumer when the
 * stage had landed and when it was handed back (last word unused).  W, X, Y: device,
 * 16-byte aligned, caller-owned; w_rows % 4 == 0.  Returns the number of CTAs launched (> 0) or a negative
 * NM_ERR_* code.  Waits are bounded: NM_STATUS_TIMEOUT in *status (nullable) when one expired.
 */
int nm_probe_tma_stream(const void *W, int w_rows, int w_row_bytes, const void *X, int tokens, int k_bytes,
                        float *Y, int a_rows, int a_row_bytes, int b_rows, int b_slices, int stages, int band,
                        int repeat, int delay_clocks, int loads, int stores, int producers, int poll, unsigned long long *clocks,
                        unsigned long long *trace, uint32_t *status, void *stream);

/*
 * Measurement and test aid (the paper has no counterpart): overrides the kernel nm_int_linear and its variants
 * (and, with "pack_form", the projection entry points) pick, process-wide, for every later call (not thread-safe against calls in flight on other host threads).
 * All options are 0 by default = the library's own choice.  Names: "no_pdl" (launch without the programmatic-
 * dependent-launch attribute), "no_pair" (one-CTA kernels only), "no_resident" (always stream the weights),
 * "no_wide" (never the 512-channel pair kernel), "wide_any" (the 512-channel pair kernel whenever the shape
 * allows it, however few tiles there are), "wide_bn" (its token-tile width, 224 or 192), "band" (band size of the streamed pair kernel's tile order),
 * "pack_form" (form of the projection kernel in blocks of four warps: 1 = one unit per block, 2 = persistent with
 * chunks staged in shared memory by bulk copies, 3 = persistent with the next chunk asked for ahead into L2).
 * Results never depend on them.  Returns NM_ERR_UNSUPPORTED for an unknown name.  A library built with
 * -DNM_TEST_HOOKS (build.py --variant shortwait: device-side waits limited to about a millisecond) also takes
 * "skip_stage" = 1 + the pipeline stage that CTA 0's producer leaves unissued (0 = none): the bounded waits then
 * run out, the kernel drains and returns, and nm_poll_status reports NM_ERR_TIMEOUT.  The same build takes
 * "skip_pack_copy" = 1 + the unit (counted per block) whose bulk copies warp 0 of block 0 of the staged projection
 * kernel leaves unissued, with the same outcome for the projection entry points.
 */
int nm_debug_set_option(const char *name /* host */, int value);

/*
 * Profiling aid (the paper has no counterpart).  Only a library built with -DNM_TRACE accepts it (build.py
 * --variant trace -> libnmsparse_trace.so); the product library returns NM_ERR_UNSUPPORTED and its kernels carry
 * no time stamps.  `buffer`: device, u64 [512 + 64][8], zeroed by the caller, or NULL to switch tracing off.  Every
 * later CTA-pair GEMM launch has its CTA 0 write clock64() values: row `it` (pipeline stage `it` < 512 of that CTA):
 * [0] producer got the free stage, [1] issued its loads, [2] gate saw the stage full, [3] MMA thread was handed
 * the stage, [4] had issued the stage's MMAs and commits; row 512 + i (tile i < 64 of that CTA): [0] an epilogue
 * warp saw the accumulator full, [1] had finished the tile.
 */
int nm_debug_set_trace(unsigned long long *buffer);

/* Host-only validation of a linear-layer problem: NM_OK or the error nm_int_linear would return. */
int nm_int_linear_check(int tokens, int out, int in, int n, int m, int bits);

/*
 * Dynamic per-tensor symmetric 8-bit activation quantiser (Eq. 5 with bits = 8; the activations
 * of the integer layers are 8 bit, Sec. 5.3):
 *   nm_absmax:        *absmax = max(*absmax, max_i |Y[i]|)   (caller zeroes *absmax first)
 *   nm_quantize_act:  sx = *absmax / 127 (1 if *absmax == 0);  Xq[i] = clamp(rne(Y[i] / sx), -128, 127)
 *                     *sx_out (nullable) receives sx.
 * Y and Xq must be 16-byte aligned.  sx_out must not be the same word as absmax (other blocks still read the
 * maximum while the scale is written): NM_ERR_SHAPE.
 */
int nm_absmax(const float *Y, size_t count, float *absmax, void *stream);
int nm_quantize_act(const float *Y, size_t count, const float *absmax, int8_t *Xq, float *sx_out,
                    void *stream);

/*
 * Synchronises `stream`, reads the device status word and returns NM_OK, NM_ERR_NONFINITE,
 * NM_ERR_TIMEOUT or NM_ERR_CUDA.  `status` may be NULL (then only the stream is checked).
 */
int nm_poll_status(const uint32_t *status, void *stream);

/* Text for an NM_* code (static storage). */
const char *nm_strerror(int code);

/* Text of the last CUDA error this thread met inside the library (static storage, "" if none). */
const char *nm_last_cuda_error(void);

/*
 * Cost model behind the paper's size and FLOP columns (Table 1, Table 4; Sec. 4: a compression
 * scheme is scored without running it).  Host-only arithmetic.
 *   nm_bits_per_param: stored bits per dense parameter of an n:m sparse b-bit matrix = n/m * (bits +
 *     index_bits); dense (n == m): bits.  index_bits < 0 selects this library's metadata field (2 for
 *     m = 4, 4 for m = 8); the paper's tables use 2 at m = 4; 0 gives the headline ratios that ignore
 *     metadata.  Returns -1 for an invalid pattern.
 *   nm_encoder_cost: one encoder whose six linear components (Q, K, V, attention output, FFN1, FFN2,
 *     in this order; relative sizes 1, 1, 1, 1, 4, 4) each have their own (n, m, bits):
 *     *compression = 1 - stored bits / (32 bits per parameter), *mac_reduction = fraction of the dense
 *     multiply-accumulates saved (one half for every component that runs on the 2-of-4 sparse path:
 *     1:4, 2:4, 1:8, 2:8; nothing for dense and 4:8).  Either output may be NULL.
 */
typedef struct {
    int32_t n, m, bits;
} nm_component_cfg_t;
double nm_bits_per_param(int n, int m, int bits, int index_bits);
int nm_encoder_cost(const nm_component_cfg_t *cfg /* [6], host */, int index_bits, double *compression,
                    double *mac_reduction);

/* Library version, major * 100 + minor. */
int nm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* NMSPARSE_H_ */
