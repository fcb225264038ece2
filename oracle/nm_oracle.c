/*
 * nm_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, scalar CPU statement of what the N:M low-bit path computes,
 * written from the paper (arxiv 2206.15014) so that the CUDA library can be
 * checked against it.  It shares no code, header, table or helper with the
 * CUDA path and is only ever called from tests, from the smoke check and from
 * the benchmark's CPU-baseline leg.
 *
 * Conventions (kept:group, i.e. "2:4" keeps n=2 of every m=4):
 *   W, U        fp32 [out, in] row-major (nn.Linear layout); groups of m run
 *               along `in`, the reduction dimension.
 *   values      kept integer codes, ascending position inside each group,
 *               row-major [out, in*n/m]; 8-bit: one byte each; 4-bit: two's
 *               complement nibbles, even element in bits 3:0, odd in bits 7:4.
 *   meta        position-in-group of each kept element; 2-bit fields for m=4,
 *               4-bit fields for m=8, LSB first in element order, packed into
 *               little-endian u32 words, each row padded to whole words.
 *               n == m has no metadata.
 *   scales      fp32 [out], one per output channel.
 *
 * Parity status of the pieces:
 *   projection (Eq. 3, Sec. 3.2), ADMM-Max scale (Sec. 3.3.1), quantiser
 *   (Eq. 5), dequantisation (Eq. 4), integer linear layer (Sec. 5.3): pinned by
 *   the CPU tests (brute-force Euclidean projection, idempotence, scale
 *   invariance under pruning, textbook absmax quantisation, int64 numpy matmul,
 *   double-precision epilogue, the paper's Table 1 / Table 4 size accounting).
 *   The byte-level packing of values and metadata is this library's own
 *   convention (the paper specifies none): parity unpinned beyond the
 *   pack -> unpack round trip and the 2-index-bits-per-kept-value accounting.
 *   One ADMM step with dense outputs (joint projection Z as fp32, dual update
 *   U + W - Z; the paper prints the projection, Eq. 3, the dual update is the
 *   standard scaled form): pinned as the composition of the pieces above, against
 *   the packed path, numpy's own fp32 subtraction, the constraint on Z, the
 *   half-step bound on the dual and the fixed point Z(Z) = Z.
 *   Narrow forms of the layer's output -- Eq. 5 with a scale fixed ahead of
 *   time (8-bit activations handed to the next layer, Sec. 4.5) and binary32 ->
 *   bfloat16 rounding: pinned by closed forms (exact multiples, ties), exact
 *   rational arithmetic, error bounds and an independent conversion routine.
 *   ADMM-Dist scale (Sec. 3.3.1, "Minimize Quantization Distance"; the paper
 *   names the objective and gives no search procedure, so the candidate sweep
 *   is this library's reading): pinned by its one-candidate case (= ADMM-Max),
 *   by exact rational arithmetic over every candidate on small rows, by the
 *   distance recomputed from the packed output with the pinned unpack and
 *   projection routines, and by invariance under powers of two.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_SHAPE -1
#define ORACLE_ERR_NONFINITE -2
#define ORACLE_ERR_OVERFLOW -3

static int g_threads = 1;

/* Number of OpenMP threads used by the row loops (1 = serial). */
void oracle_set_threads(int t) { g_threads = t < 1 ? 1 : t; }
int oracle_get_threads(void) { return g_threads; }
int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

static int field_bits(int m) { return m == 4 ? 2 : 4; }

static int shape_ok(int out, int in, int n, int m, int bits)
{
    if (out < 0 || in < 0 || n < 1 || m < 1 || n > m) return 0;
    if (bits != 4 && bits != 8) return 0;
    if (n != m && m != 4 && m != 8) return 0;
    if (in % m) return 0;
    if (((long long)(in / m) * n * bits) % 8) return 0;
    return 1;
}

/* Bytes of one packed row of values / words of one row of metadata. */
static size_t values_row_bytes(int in, int n, int m, int bits)
{
    return (size_t)(in / m) * n * bits / 8;
}
static size_t meta_row_words(int in, int n, int m)
{
    if (n == m) return 0;
    size_t row_bits = (size_t)(in / m) * n * field_bits(m);
    return (row_bits + 31) / 32;
}

int oracle_packed_sizes(int out, int in, int n, int m, int bits, size_t *values_bytes,
                        size_t *meta_bytes)
{
    if (!shape_ok(out, in, n, m, bits)) return ORACLE_ERR_SHAPE;
    *values_bytes = (size_t)out * values_row_bytes(in, n, m, bits);
    *meta_bytes = (size_t)out * meta_row_words(in, n, m) * 4;
    return ORACLE_OK;
}

/*
 * Support of the Euclidean projection of one group onto "at most n non-zeros
 * out of m" (Eq. 2-3; Sec. 3.2: keep the largest entries of each contiguous
 * group).  The largest are the largest in magnitude -- that is what minimises
 * the Frobenius distance.  Equal magnitudes: the lower index is kept.  A stable
 * insertion sort by descending |v| gives exactly that order.  keep[] receives
 * the n chosen positions in ascending order.
 */
static void group_support(const float *v, int n, int m, int *keep)
{
    int idx[64];
    for (int i = 0; i < m; ++i) idx[i] = i;
    for (int i = 1; i < m; ++i) {
        int cur = idx[i];
        float a = fabsf(v[cur]);
        int j = i - 1;
        while (j >= 0 && fabsf(v[idx[j]]) < a) { /* strict: equal keys keep their order */
            idx[j + 1] = idx[j];
            --j;
        }
        idx[j + 1] = cur;
    }
    /* first n of the sorted order, then ascending by position */
    for (int i = 0; i < n; ++i) keep[i] = idx[i];
    for (int i = 1; i < n; ++i) {
        int cur = keep[i], j = i - 1;
        while (j >= 0 && keep[j] > cur) {
            keep[j + 1] = keep[j];
            --j;
        }
        keep[j + 1] = cur;
    }
}

/*
 * ADMM-Max scale of one output channel (Sec. 3.3.1, "Minimize Error on the
 * Largest Parameter"): the largest magnitude of W+U divided by the largest
 * integer code 2^(b-1)-1.  An all-zero channel gets scale 1.
 */
static float row_scale(const float *v, int in, int bits)
{
    float a = 0.0f;
    for (int k = 0; k < in; ++k) {
        float t = fabsf(v[k]);
        if (t > a) a = t;
    }
    float qmax = (float)((1 << (bits - 1)) - 1);
    return a == 0.0f ? 1.0f : a / qmax;
}

/* Eq. 5 with offset 0: clamp(round(x / s), -2^(b-1), 2^(b-1)-1), round = half to even. */
static int quantise(float x, float s, int bits)
{
    int hi = (1 << (bits - 1)) - 1, lo = -(1 << (bits - 1));
    float r = nearbyintf(x / s); /* default rounding mode: to nearest, ties to even */
    if (r > (float)hi) return hi;
    if (r < (float)lo) return lo;
    return (int)r;
}

static int row_finite(const float *v, int in)
{
    for (int k = 0; k < in; ++k)
        if (!isfinite(v[k])) return 0;
    return 1;
}

/*
 * Joint projection of Sec. 3.3.1 (last paragraph): sparsity constraint, then
 * quantisation constraint, scale from ADMM-Max.  V = W + U is the Z-update's
 * argument (Eq. 3); U may be NULL.
 */
static int project_pack_impl(const float *W, const float *U, int out, int in, int n, int m, int bits,
                             const float *given_scales, uint8_t *values, uint32_t *meta, float *scales)
{
    if (!shape_ok(out, in, n, m, bits)) return ORACLE_ERR_SHAPE;
    const size_t vrb = values_row_bytes(in, n, m, bits);
    const size_t mrw = meta_row_words(in, n, m);
    const int fb = field_bits(m);
    int status = ORACLE_OK;
#pragma omp parallel for schedule(static) num_threads(g_threads)
    for (int r = 0; r < out; ++r) {
        float *v = (float *)malloc(sizeof(float) * (size_t)(in > 0 ? in : 1));
        for (int k = 0; k < in; ++k) {
            float w = W[(size_t)r * in + k];
            v[k] = U ? w + U[(size_t)r * in + k] : w;
        }
        if (!row_finite(v, in)) {
#pragma omp atomic write
            status = ORACLE_ERR_NONFINITE;
        }
        float s = given_scales ? given_scales[r] : row_scale(v, in, bits);
        scales[r] = s;
        uint8_t *vrow = values + (size_t)r * vrb;
        uint32_t *mrow = meta ? meta + (size_t)r * mrw : NULL;
        memset(vrow, 0, vrb);
        if (mrow) memset(mrow, 0, mrw * 4);
        size_t e = 0; /* index of the kept element inside the row */
        for (int g = 0; g < in / m; ++g) {
            int keep[64];
            group_support(v + (size_t)g * m, n, m, keep);
            for (int i = 0; i < n; ++i, ++e) {
                int q = quantise(v[(size_t)g * m + keep[i]], s, bits);
                if (bits == 8) {
                    vrow[e] = (uint8_t)(int8_t)q;
                } else {
                    uint8_t nib = (uint8_t)(q & 0xF);
                    vrow[e / 2] |= (e & 1) ? (uint8_t)(nib << 4) : nib;
                }
                if (mrow) {
                    size_t bit = e * (size_t)fb;
                    mrow[bit / 32] |= (uint32_t)keep[i] << (bit % 32);
                }
            }
        }
        free(v);
    }
    return status;
}

int oracle_project_pack(const float *W, const float *U, int out, int in, int n, int m, int bits,
                        uint8_t *values, uint32_t *meta, float *scales)
{
    return project_pack_impl(W, U, out, in, n, m, bits, NULL, values, meta, scales);
}

/*
 * Group-wise quantisation (Sec. 3.3, "subsets of neurons within a single weight
 * matrix are quantized using different scales"; whole neurons always share a
 * scale): rows r with the same r / group_rows share one ADMM-Max scale, the
 * largest magnitude of W + U over those rows divided by the largest integer
 * (group_rows <= 0: one scale for the whole matrix; the last group may be
 * short).  scales[r] receives the scale of row r's group.  Everything else is
 * oracle_project_pack.
 */
int oracle_project_pack_grouped(const float *W, const float *U, int out, int in, int n, int m,
                                int bits, int group_rows, uint8_t *values, uint32_t *meta,
                                float *scales)
{
    if (!shape_ok(out, in, n, m, bits)) return ORACLE_ERR_SHAPE;
    const int G = group_rows <= 0 ? (out > 0 ? out : 1) : group_rows;
    const float qmax = (float)((1 << (bits - 1)) - 1);
    float *gs = (float *)malloc(sizeof(float) * (size_t)(out > 0 ? out : 1));
    for (int g0 = 0; g0 < out; g0 += G) {
        float a = 0.0f;
        for (int r = g0; r < out && r < g0 + G; ++r)
            for (int k = 0; k < in; ++k) {
                float w = W[(size_t)r * in + k];
                float t = fabsf(U ? w + U[(size_t)r * in + k] : w);
                if (t > a) a = t;
            }
        float sg = a == 0.0f ? 1.0f : a / qmax;
        for (int r = g0; r < out && r < g0 + G; ++r) gs[r] = sg;
    }
    int rc = project_pack_impl(W, U, out, in, n, m, bits, gs, values, meta, scales);
    free(gs);
    return rc;
}

/*
 * ADMM-Dist (Sec. 3.3.1, "Minimize Quantization Distance"): the scale of an
 * output channel is the one that minimises the squared Euclidean distance
 * between the channel and its quantised form.  With the sparsity constraint the
 * sparsity projection comes first (Sec. 3.3.1, last paragraph), so the distance
 * is taken over the kept entries: pruned entries are zero on both sides.
 *
 * The paper gives no procedure for the minimisation.  Reading taken here: a
 * sweep over `ncand` candidate scales (1 <= ncand <= 32)
 *     s_j = fl32(s_max * c_j),  c_j = (64 - j) / 64,  j = 0 .. ncand-1,
 * where s_max is the ADMM-Max scale of the channel (so j = 0 is ADMM-Max and the
 * candidates shrink the representable range down to about half of it).  For
 * every candidate
 *     E_j = sum over kept k of (v_k - s_j * q_jk)^2,  q_jk = Eq. 5 at scale s_j,
 * evaluated in double from the fp32 v_k and s_j (the product s_j * q is exact in
 * double), summed in index order.  The smallest E_j wins, the lowest j on
 * equality.  An all-zero channel has s_max = 1 and E_j = 0 for all j: j = 0.
 *
 * E (nullable) receives E_j as [out][ncand]; S (nullable) the candidate scales
 * [out][ncand]; scales (nullable) the chosen scale; cand (nullable) the chosen j.
 */
int oracle_dist_search(const float *W, const float *U, int out, int in, int n, int m, int bits,
                       int ncand, double *E, float *S, float *scales, int32_t *cand)
{
    if (!shape_ok(out, in, n, m, bits)) return ORACLE_ERR_SHAPE;
    if (ncand < 1 || ncand > 32) return ORACLE_ERR_SHAPE;
    int status = ORACLE_OK;
#pragma omp parallel for schedule(static) num_threads(g_threads)
    for (int r = 0; r < out; ++r) {
        float *v = (float *)malloc(sizeof(float) * (size_t)(in > 0 ? in : 1));
        int *kept = (int *)malloc(sizeof(int) * (size_t)(in > 0 ? in : 1));
        for (int k = 0; k < in; ++k) {
            float w = W[(size_t)r * in + k];
            v[k] = U ? w + U[(size_t)r * in + k] : w;
        }
        if (!row_finite(v, in)) {
#pragma omp atomic write
            status = ORACLE_ERR_NONFINITE;
        }
        size_t nk = 0;
        for (int g = 0; g < in / m; ++g) {
            int keep[64];
            group_support(v + (size_t)g * m, n, m, keep);
            for (int i = 0; i < n; ++i) kept[nk++] = g * m + keep[i];
        }
        const float smax = row_scale(v, in, bits);
        int best = 0;
        double best_e = 0.0;
        float best_s = smax;
        for (int j = 0; j < ncand; ++j) {
            const float cj = (float)(64 - j) / 64.0f; /* exact */
            const float sj = smax * cj;
            double e = 0.0;
            for (size_t i = 0; i < nk; ++i) {
                const float x = v[kept[i]];
                const int q = quantise(x, sj, bits);
                const double d = (double)x - (double)sj * (double)q;
                e += d * d;
            }
            if (E) E[(size_t)r * ncand + j] = e;
            if (S) S[(size_t)r * ncand + j] = sj;
            if (j == 0 || e < best_e) { best = j; best_e = e; best_s = sj; }
        }
        if (scales) scales[r] = best_s;
        if (cand) cand[r] = best;
        free(kept);
        free(v);
    }
    return status;
}

/* The joint projection with scales handed in (one per output channel). */
int oracle_project_pack_scaled(const float *W, const float *U, int out, int in, int n, int m,
                               int bits, const float *given_scales, uint8_t *values,
                               uint32_t *meta, float *scales)
{
    return project_pack_impl(W, U, out, in, n, m, bits, given_scales, values, meta, scales);
}

/* Joint projection with the ADMM-Dist scale: sparsify, search the scale, quantise, pack. */
int oracle_project_pack_dist(const float *W, const float *U, int out, int in, int n, int m,
                             int bits, int ncand, uint8_t *values, uint32_t *meta, float *scales)
{
    float *gs = (float *)malloc(sizeof(float) * (size_t)(out > 0 ? out : 1));
    int rc = oracle_dist_search(W, U, out, in, n, m, bits, ncand, NULL, NULL, gs, NULL);
    if (rc == ORACLE_OK || rc == ORACLE_ERR_NONFINITE) {
        int rc2 = project_pack_impl(W, U, out, in, n, m, bits, gs, values, meta, scales);
        if (rc == ORACLE_OK) rc = rc2;
    }
    free(gs);
    return rc;
}

/* Inverse of the packing: dense integer codes [out, in], zero where pruned. */
int oracle_unpack(const uint8_t *values, const uint32_t *meta, int out, int in, int n, int m,
                  int bits, int8_t *Wq)
{
    if (!shape_ok(out, in, n, m, bits)) return ORACLE_ERR_SHAPE;
    const size_t vrb = values_row_bytes(in, n, m, bits);
    const size_t mrw = meta_row_words(in, n, m);
    const int fb = field_bits(m);
    for (int r = 0; r < out; ++r) {
        const uint8_t *vrow = values + (size_t)r * vrb;
        const uint32_t *mrow = meta ? meta + (size_t)r * mrw : NULL;
        int8_t *drow = Wq + (size_t)r * in;
        memset(drow, 0, (size_t)in);
        size_t e = 0;
        for (int g = 0; g < in / m; ++g) {
            for (int i = 0; i < n; ++i, ++e) {
                int q;
                if (bits == 8) {
                    q = (int8_t)vrow[e];
                } else {
                    int nib = (vrow[e / 2] >> ((e & 1) ? 4 : 0)) & 0xF;
                    q = nib >= 8 ? nib - 16 : nib;
                }
                int pos = i;
                if (n != m) {
                    size_t bit = e * (size_t)fb;
                    pos = (int)((mrow[bit / 32] >> (bit % 32)) & ((1u << fb) - 1u));
                }
                drow[(size_t)g * m + pos] = (int8_t)q;
            }
        }
    }
    return ORACLE_OK;
}

/* Sparsity projection alone (Eq. 3): Z = Pi_S(W + U) as dense fp32. */
int oracle_project_dense(const float *W, const float *U, int out, int in, int n, int m, float *Z)
{
    if (n < 1 || n > m || m > 64 || in % m) return ORACLE_ERR_SHAPE;
    for (int r = 0; r < out; ++r)
        for (int g = 0; g < in / m; ++g) {
            float v[64];
            int keep[64];
            size_t base = (size_t)r * in + (size_t)g * m;
            for (int i = 0; i < m; ++i) {
                v[i] = U ? W[base + i] + U[base + i] : W[base + i];
                Z[base + i] = 0.0f;
            }
            group_support(v, n, m, keep);
            for (int i = 0; i < n; ++i) Z[base + keep[i]] = v[keep[i]];
        }
    return ORACLE_OK;
}

/* Per-channel ADMM-Max scales of an fp32 matrix (Sec. 3.3.1). */
int oracle_row_scales(const float *V, int out, int in, int bits, float *scales)
{
    for (int r = 0; r < out; ++r) scales[r] = row_scale(V + (size_t)r * in, in, bits);
    return ORACLE_OK;
}

/*
 * STE forward pass (Sec. 3.3.2): the weight the forward pass sees is the
 * dequantised quantised one, x_d = s * x_q (Eq. 4 with o = 0), here applied to
 * an fp32 matrix Z elementwise with the given per-row scales.
 */
int oracle_fake_quant(const float *Z, int out, int in, int bits, const float *scales, float *Zq)
{
    for (int r = 0; r < out; ++r)
        for (int k = 0; k < in; ++k) {
            size_t i = (size_t)r * in + k;
            Zq[i] = scales[r] * (float)quantise(Z[i], scales[r], bits);
        }
    return ORACLE_OK;
}

/*
 * One ADMM projection step for the joint constraint (Eq. 3 with the sparsity and
 * quantisation projections solved in sequence, Sec. 3.3.1 last paragraph), dense
 * outputs:
 *   V = W + U;  s_r = ADMM-Max scale of row r of V;
 *   Z = s_r * clamp(round(Pi_S(V) / s_r))     (Eq. 5 then Eq. 4, zero where pruned)
 *   U_next = V - Z                             (scaled-form dual update U + W - Z)
 * With U == NULL and U_next == NULL this is the forward pass of the STE
 * fake-quantiser on a weight that is also N:M-projected (Sec. 3.3.2).
 * scales (nullable) receives s_r.
 */
static int admm_step_impl(const float *W, const float *U, int out, int in, int n, int m, int bits,
                          const float *given_scales, float *Z, float *U_next, float *scales)
{
    if (n < 1 || n > m || m > 64 || in % m || bits < 2 || bits > 8) return ORACLE_ERR_SHAPE;
    float *v = (float *)malloc((size_t)in * sizeof(float));
    if (!v) return ORACLE_ERR_SHAPE;
    int status = ORACLE_OK;
    for (int r = 0; r < out; ++r) {
        size_t base = (size_t)r * in;
        for (int k = 0; k < in; ++k) v[k] = U ? W[base + k] + U[base + k] : W[base + k];
        if (!row_finite(v, in)) { status = ORACLE_ERR_NONFINITE; break; }
        float s = given_scales ? given_scales[r] : row_scale(v, in, bits);
        if (scales) scales[r] = s;
        for (int g = 0; g < in / m; ++g) {
            int keep[64];
            for (int i = 0; i < m; ++i) Z[base + (size_t)g * m + i] = 0.0f;
            group_support(v + (size_t)g * m, n, m, keep);
            for (int i = 0; i < n; ++i) {
                size_t k = (size_t)g * m + keep[i];
                Z[base + k] = s * (float)quantise(v[k], s, bits);
            }
        }
        if (U_next)
            for (int k = 0; k < in; ++k) U_next[base + k] = v[k] - Z[base + k];
    }
    free(v);
    return status;
}

int oracle_admm_step(const float *W, const float *U, int out, int in, int n, int m, int bits,
                     float *Z, float *U_next, float *scales)
{
    return admm_step_impl(W, U, out, in, n, m, bits, NULL, Z, U_next, scales);
}

/* The same step with the ADMM-Dist scale (oracle_dist_search) in place of ADMM-Max. */
int oracle_admm_step_dist(const float *W, const float *U, int out, int in, int n, int m, int bits,
                          int ncand, float *Z, float *U_next, float *scales)
{
    if (!shape_ok(out, in, n, m, bits)) return ORACLE_ERR_SHAPE;
    float *gs = (float *)malloc(sizeof(float) * (size_t)(out > 0 ? out : 1));
    int rc = oracle_dist_search(W, U, out, in, n, m, bits, ncand, NULL, NULL, gs, NULL);
    if (rc == ORACLE_OK) rc = admm_step_impl(W, U, out, in, n, m, bits, gs, Z, U_next, scales);
    free(gs);
    return rc;
}

/*
 * Integer linear layer (Sec. 5.3): 8-bit activations times weights widened to
 * 8 bits, exact integer accumulation, then dequantisation (Eq. 4):
 *   acc[t,o] = sum_k X[t,k] * Wq[o,k]          (int64, every k, zeros included)
 *   y[t,o]   = fma((float)acc, sx * sw[o], bias[o])
 * ACC (nullable) receives the accumulators as int32.
 */
int oracle_int_linear(const int8_t *X, int tokens, const int8_t *Wq, int out, int in, float sx,
                      const float *sw, const float *bias, int32_t *ACC, float *Y)
{
    int status = ORACLE_OK;
#pragma omp parallel for schedule(static) num_threads(g_threads)
    for (int t = 0; t < tokens; ++t) {
        const int8_t *x = X + (size_t)t * in;
        for (int o = 0; o < out; ++o) {
            const int8_t *w = Wq + (size_t)o * in;
            int64_t acc = 0;
            for (int k = 0; k < in; ++k) acc += (int64_t)x[k] * (int64_t)w[k];
            if (acc > INT32_MAX || acc < INT32_MIN) {
#pragma omp atomic write
                status = ORACLE_ERR_OVERFLOW;
            }
            if (ACC) ACC[(size_t)t * out + o] = (int32_t)acc;
            if (Y) {
                float c = sx * sw[o];
                float b = bias ? bias[o] : 0.0f;
                Y[(size_t)t * out + o] = fmaf((float)(int32_t)acc, c, b);
            }
        }
    }
    return status;
}

/*
 * The same accumulators, summed over the kept positions only, walking the
 * packed form: "only computing half the operations" (Sec. 5.3) must not change
 * the result.
 */
int oracle_int_linear_kept(const int8_t *X, int tokens, const uint8_t *values, const uint32_t *meta,
                           int out, int in, int n, int m, int bits, int32_t *ACC)
{
    if (!shape_ok(out, in, n, m, bits)) return ORACLE_ERR_SHAPE;
    const size_t vrb = values_row_bytes(in, n, m, bits);
    const size_t mrw = meta_row_words(in, n, m);
    const int fb = field_bits(m);
    for (int t = 0; t < tokens; ++t)
        for (int o = 0; o < out; ++o) {
            const uint8_t *vrow = values + (size_t)o * vrb;
            const uint32_t *mrow = meta ? meta + (size_t)o * mrw : NULL;
            int64_t acc = 0;
            size_t e = 0;
            for (int g = 0; g < in / m; ++g)
                for (int i = 0; i < n; ++i, ++e) {
                    int q;
                    if (bits == 8) {
                        q = (int8_t)vrow[e];
                    } else {
                        int nib = (vrow[e / 2] >> ((e & 1) ? 4 : 0)) & 0xF;
                        q = nib >= 8 ? nib - 16 : nib;
                    }
                    int pos = i;
                    if (n != m) {
                        size_t bit = e * (size_t)fb;
                        pos = (int)((mrow[bit / 32] >> (bit % 32)) & ((1u << fb) - 1u));
                    }
                    acc += (int64_t)X[(size_t)t * in + (size_t)g * m + pos] * q;
                }
            ACC[(size_t)t * out + o] = (int32_t)acc;
        }
    return ORACLE_OK;
}

/*
 * Dynamic per-tensor symmetric 8-bit activation quantiser: Eq. 5 with b = 8 and
 * the scale chosen as for ADMM-Max over the whole tensor (max|y| / 127).
 */
int oracle_quantize_act(const float *Y, size_t count, int8_t *Xq, float *sx)
{
    float a = 0.0f;
    for (size_t i = 0; i < count; ++i) {
        float t = fabsf(Y[i]);
        if (t > a) a = t;
    }
    float s = a == 0.0f ? 1.0f : a / 127.0f;
    *sx = s;
    for (size_t i = 0; i < count; ++i) Xq[i] = (int8_t)quantise(Y[i], s, 8);
    return ORACLE_OK;
}

/*
 * Static-scale 8-bit re-quantiser: Eq. 5 with b = 8 and a scale sy fixed ahead of
 * time instead of taken from the tensor.  It is the form in which an integer
 * encoder hands the output of one linear layer to the next as 8-bit activations
 * (Sec. 4.5: all activations kept at 8 bits).
 */
int oracle_requantize_static(const float *Y, size_t count, float sy, int8_t *Yq)
{
    if (!(sy > 0.0f) || !isfinite(sy)) return ORACLE_ERR_SHAPE;
    for (size_t i = 0; i < count; ++i) {
        if (!isfinite(Y[i])) return ORACLE_ERR_NONFINITE;
        Yq[i] = (int8_t)quantise(Y[i], sy, 8);
    }
    return ORACLE_OK;
}

/*
 * binary32 -> bfloat16 (the upper 16 bits of the binary32 pattern), rounded to
 * nearest with ties to even, for finite inputs: the discarded 16 bits decide.
 */
int oracle_to_bf16(const float *Y, size_t count, uint16_t *out)
{
    for (size_t i = 0; i < count; ++i) {
        if (!isfinite(Y[i])) return ORACLE_ERR_NONFINITE;
        uint32_t u;
        memcpy(&u, &Y[i], sizeof u);
        uint32_t upper = u >> 16, lower = u & 0xFFFFu;
        if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1u;
        out[i] = (uint16_t)upper;
    }
    return ORACLE_OK;
}

/*
 * Storage accounting behind the paper's size columns (Table 1, Table 4): bits
 * per dense parameter of an n:m sparse b-bit matrix = value bits of the kept
 * entries plus index bits per kept entry.  index_bits < 0 selects this
 * library's field width (2 for m=4, 4 for m=8); the paper's tables correspond
 * to index_bits = 2 at m = 4.
 */
double oracle_bits_per_param(int n, int m, int bits, int index_bits)
{
    if (n == m) return (double)bits;
    int ib = index_bits < 0 ? field_bits(m) : index_bits;
    return ((double)n / (double)m) * (double)(bits + ib);
}
