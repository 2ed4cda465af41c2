/*
 * RS-DGC reference oracle (plain C, one thread, no blocking, no fusion).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, literal statement of what the
 * gradient-compression path computes, written from the paper's equations.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline leg.
 * It shares no code, header, table or helper with the CUDA library and must never
 * be reached from the product path.
 *
 * Every function cites the passage of the paper (arxiv 2312.17530) it follows.
 * Notation: a layer is a row-major rows x cols matrix (Sec. III-C, "two-dimensional
 * plane"), partitioned into nh x nw neighborhoods ("p x p patch", Eq. 7, read as a
 * non-overlapping partition because Eq. 11 counts numel/(p*p) of them).  Tiles on
 * the right/bottom edge are clipped; statistics divide by the true element count.
 * Tile index k = tile_row * ceil(cols/nw) + tile_col.
 *
 * Floating point: every "f32" quantity is produced by single IEEE-754 binary32
 * operations in the order written here (build with -ffp-contract=off so that no
 * multiply-add is fused); every "ref" quantity is evaluated in binary64.
 *
 * Pins (see tests/): hand-derived closed forms on a 6x6 worked example, constant /
 * single-spike tiles, homogeneity, the 1x1-tile special case against a library
 * top-k, brute-force subset enumeration, conservation sent + residual == input,
 * and a full-sort definition of the ratio rule.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <float.h>

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* Number of neighborhoods K_l of a layer (Algorithm 1, inner loop bound; Eq. 11's
 * numel/(p*p) generalised to clipped edge tiles). */
int64_t rsdgc_oracle_tile_count(int64_t rows, int64_t cols, int32_t nh, int32_t nw)
{
    return ceil_div(rows, nh) * ceil_div(cols, nw);
}

/* bfloat16 -> binary32: the 16 stored bits are the upper half of the binary32. */
static float bf16_to_f32(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* Local gradient accumulation v = v_prev + g (Eq. 12, second line), one binary32
 * add per element.  r is the carried accumulator ("residual"). */
void rsdgc_oracle_accumulate_f32(const float *g, const float *r, float *v, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) v[i] = g[i] + r[i];
}

/* Same with the incoming gradient stored as bfloat16: it is widened exactly, then
 * added in binary32 (the accumulator, the indicator and the payload stay binary32). */
void rsdgc_oracle_accumulate_bf16(const uint16_t *g, const float *r, float *v, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) v[i] = bf16_to_f32(g[i]) + r[i];
}

/* Momentum correction ahead of the accumulation (Eq. 12, first and second line):
 * u = m * u_prev + g, v = v_prev + u; product, sum, sum, each rounded to binary32.
 * u is updated in place; it is not masked where neighborhoods are sent (Eq. 12 has no
 * such step). */
void rsdgc_oracle_accumulate_momentum_f32(const float *g, float *u, const float *r, float *v, float m, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) {
        float mu = m * u[i];
        u[i] = mu + g[i];
        v[i] = r[i] + u[i];
    }
}

/* Same with the incoming gradient stored as bfloat16 (widened exactly first). */
void rsdgc_oracle_accumulate_momentum_bf16(const uint16_t *g, float *u, const float *r, float *v, float m,
                                           int64_t n)
{
    for (int64_t i = 0; i < n; ++i) {
        float mu = m * u[i];
        u[i] = mu + bf16_to_f32(g[i]);
        v[i] = r[i] + u[i];
    }
}

/*
 * Neighborhood Statistical Indicator of every tile (Eq. 8-10):
 *   mean_p = (1/n) sum |v_i|                           (Eq. 9)
 *   std_p  = sqrt( (1/n) sum (v_i - (1/n) sum v_j)^2 ) (Eq. 10, population std)
 *   NSI    = alpha * mean_p + (1 - alpha) * std_p      (Eq. 8)
 * nsi_ref: binary64 from the binary32 inputs.
 * nsi_f32: binary32, elements visited row-major inside the tile, plain running
 *          sums, mean first and squared deviations in a second sweep; the factor
 *          1/p^2 of Eq. 9-10 is formed once (1/n rounded to binary32) and each of
 *          the three sums is multiplied by it, as the equations are written.
 * A non-finite nsi_f32 is replaced by +infinity (so it ranks first, deterministically)
 * and counted in the return value.
 */
int64_t rsdgc_oracle_nsi(const float *v, int64_t rows, int64_t cols, int32_t nh, int32_t nw,
                         float alpha, double *nsi_ref, float *nsi_f32)
{
    const int64_t TR = ceil_div(rows, nh), TC = ceil_div(cols, nw);
    int64_t nonfinite = 0;
    for (int64_t tr = 0; tr < TR; ++tr) {
        for (int64_t tc = 0; tc < TC; ++tc) {
            const int64_t i0 = tr * nh, i1 = (i0 + nh < rows) ? i0 + nh : rows;
            const int64_t j0 = tc * nw, j1 = (j0 + nw < cols) ? j0 + nw : cols;
            const int64_t cnt = (i1 - i0) * (j1 - j0);
            const int64_t k = tr * TC + tc;

            /* binary64 reference */
            double da = 0.0, dm = 0.0;
            for (int64_t i = i0; i < i1; ++i)
                for (int64_t j = j0; j < j1; ++j) {
                    double x = (double)v[i * cols + j];
                    da += fabs(x);
                    dm += x;
                }
            da /= (double)cnt;
            dm /= (double)cnt;
            double dq = 0.0;
            for (int64_t i = i0; i < i1; ++i)
                for (int64_t j = j0; j < j1; ++j) {
                    double d = (double)v[i * cols + j] - dm;
                    dq += d * d;
                }
            if (nsi_ref)
                nsi_ref[k] = (double)alpha * da + (1.0 - (double)alpha) * sqrt(dq / (double)cnt);

            /* binary32, fixed order */
            float sa = 0.0f, sv = 0.0f;
            for (int64_t i = i0; i < i1; ++i)
                for (int64_t j = j0; j < j1; ++j) {
                    float x = v[i * cols + j];
                    sa = sa + fabsf(x);
                    sv = sv + x;
                }
            const float inv_n = 1.0f / (float)cnt;
            const float a = sa * inv_n;
            const float m = sv * inv_n;
            float sq = 0.0f;
            for (int64_t i = i0; i < i1; ++i)
                for (int64_t j = j0; j < j1; ++j) {
                    float d = v[i * cols + j] - m;
                    float dd = d * d;
                    sq = sq + dd;
                }
            const float s = sqrtf(sq * inv_n);
            const float t1 = alpha * a;
            const float t2 = (1.0f - alpha) * s;
            float nsi = t1 + t2;
            if (!(nsi <= FLT_MAX)) { /* NaN or infinity */
                nsi = INFINITY;
                ++nonfinite;
            }
            if (nsi_f32) nsi_f32[k] = nsi;
        }
    }
    return nonfinite;
}

/* Number of neighborhoods to keep, k = ceil(K * ratio) (Eq. 11), limited to
 * [0, K]; with clamp_min1 a layer always transmits at least one neighborhood. */
int64_t rsdgc_oracle_keep_count(int64_t K, float ratio, int32_t clamp_min1)
{
    double x = ceil((double)K * (double)ratio);
    int64_t k = (x > 0.0) ? ((x >= (double)K) ? K : (int64_t)x) : 0;
    if (clamp_min1 && k < 1) k = 1;
    if (k > K) k = K;
    return k;
}

static const float *g_sort_key_f32;
static int cmp_desc_key_then_index_i32(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    float ka = g_sort_key_f32[a], kb = g_sort_key_f32[b];
    if (ka > kb) return -1;
    if (ka < kb) return 1;
    return (a > b) - (a < b);
}
static int cmp_i32(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/* Ranking of the indicator inside one layer and choice of the top k (Algorithm 1,
 * "Conduct a ranking of NSI" / "preserving the gradients in neighborhood with the
 * top-ranked NSI").  Full sort, indicator descending, equal values by lower index.
 * sel receives the k chosen tile indices in ascending order.  Returns the
 * indicator of the last tile taken (0 when k == 0). */
float rsdgc_oracle_select(const float *nsi_f32, int64_t K, int64_t k, int32_t *sel)
{
    if (k <= 0) return 0.0f;
    int32_t *order = (int32_t *)malloc((size_t)K * sizeof(int32_t));
    for (int64_t i = 0; i < K; ++i) order[i] = (int32_t)i;
    g_sort_key_f32 = nsi_f32;
    qsort(order, (size_t)K, sizeof(int32_t), cmp_desc_key_then_index_i32);
    float thr = nsi_f32[order[k - 1]];
    memcpy(sel, order, (size_t)k * sizeof(int32_t));
    qsort(sel, (size_t)k, sizeof(int32_t), cmp_i32);
    free(order);
    return thr;
}

/* Payload and accumulator update for one layer (Sec. III-C: "preserve all gradient
 * values in the neighborhood ... and transmit the corresponding neighborhood
 * index"; Eq. 12: what is not sent stays in v).  For each chosen tile, ascending:
 * idx gets the tile index, val gets its nh*nw values row-major (clipped tiles are
 * padded with +0), and the tile's entries of v are overwritten with +0. */
void rsdgc_oracle_pack(float *v, int64_t rows, int64_t cols, int32_t nh, int32_t nw,
                       const int32_t *sel, int64_t k, int32_t *idx, float *val)
{
    const int64_t TC = ceil_div(cols, nw);
    const int64_t slot = (int64_t)nh * nw;
    for (int64_t s = 0; s < k; ++s) {
        const int64_t t = sel[s], tr = t / TC, tc = t % TC;
        idx[s] = (int32_t)t;
        for (int32_t a = 0; a < nh; ++a)
            for (int32_t b = 0; b < nw; ++b) {
                const int64_t i = tr * nh + a, j = tc * nw + b;
                float x = 0.0f;
                if (i < rows && j < cols) {
                    x = v[i * cols + j];
                    v[i * cols + j] = 0.0f;
                }
                val[s * slot + a * nw + b] = x;
            }
    }
}

/* binary32 -> bfloat16 (1 sign, 8 exponent, 7 fraction bits: the upper half of a binary32
 * word), round to nearest, ties to even; overflow goes to infinity as IEEE rounding does.
 * NaN stays a quiet NaN with its sign. */
uint16_t rsdgc_oracle_f32_to_bf16(float x)
{
    uint32_t b;
    memcpy(&b, &x, sizeof b);
    if ((b & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((b >> 16) | 0x0040u);
    const uint32_t lower = b & 0xFFFFu, upper = b >> 16;
    uint32_t q = upper;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) q = upper + 1u; /* carries into the exponent as it must */
    return (uint16_t)q;
}

float rsdgc_oracle_bf16_to_f32(uint16_t h)
{
    const uint32_t b = (uint32_t)h << 16;
    float x;
    memcpy(&x, &b, sizeof x);
    return x;
}

/* The same payload with 16-bit values (an option of this implementation, not of the paper):
 * q = bfloat16(v) is what is sent, and the accumulator keeps v - q, the part of v that was
 * not sent (Eq. 12: what is not transmitted stays in v); the subtraction is exact in
 * binary32.  Clipped tiles are padded with +0. */
void rsdgc_oracle_pack_bf16(float *v, int64_t rows, int64_t cols, int32_t nh, int32_t nw,
                            const int32_t *sel, int64_t k, int32_t *idx, uint16_t *val)
{
    const int64_t TC = ceil_div(cols, nw);
    const int64_t slot = (int64_t)nh * nw;
    for (int64_t s = 0; s < k; ++s) {
        const int64_t t = sel[s], tr = t / TC, tc = t % TC;
        idx[s] = (int32_t)t;
        for (int32_t a = 0; a < nh; ++a)
            for (int32_t b = 0; b < nw; ++b) {
                const int64_t i = tr * nh + a, j = tc * nw + b;
                uint16_t q = 0;
                if (i < rows && j < cols) {
                    const float x = v[i * cols + j];
                    q = rsdgc_oracle_f32_to_bf16(x);
                    v[i * cols + j] = x - rsdgc_oracle_bf16_to_f32(q);
                }
                val[s * slot + a * nw + b] = q;
            }
    }
}

/* Aggregation of one worker's payload into the dense gradient of one layer
 * (Eq. 12, third line: sum over workers of sparse(v); Eq. 2, Sync):
 * dense[i] = dense[i] + scale * sent[i], product then sum, each rounded to binary32.
 * The caller applies workers in the order 0, 1, ... */
void rsdgc_oracle_decompress(float *dense, int64_t rows, int64_t cols, int32_t nh, int32_t nw,
                             const int32_t *idx, const float *val, int64_t k, float scale)
{
    const int64_t TC = ceil_div(cols, nw);
    const int64_t slot = (int64_t)nh * nw;
    for (int64_t s = 0; s < k; ++s) {
        const int64_t t = idx[s], tr = t / TC, tc = t % TC;
        for (int32_t a = 0; a < nh; ++a)
            for (int32_t b = 0; b < nw; ++b) {
                const int64_t i = tr * nh + a, j = tc * nw + b;
                if (i < rows && j < cols) {
                    float p = scale * val[s * slot + a * nw + b];
                    dense[i * cols + j] = dense[i * cols + j] + p;
                }
            }
    }
}

static const float *g_sort_absw;
static int cmp_desc_abs_then_index_i64(const void *pa, const void *pb)
{
    int64_t a = *(const int64_t *)pa, b = *(const int64_t *)pb;
    float ka = g_sort_absw[a], kb = g_sort_absw[b];
    if (ka > kb) return -1;
    if (ka < kb) return 1;
    return (a > b) - (a < b);
}

/* Layer-wise dynamic compression ratio (Eq. 3-5, Algorithm 1 first half):
 * importance mu = |w| (Eq. 3); one ranking across all layers; the n_keep =
 * ceil(rho * G) highest-ranked weights survive (Eq. 4; equal magnitudes by lower
 * flat index); ratio_l = survivors_l / G_l (Eq. 5).  w holds the layers back to
 * back, sizes[l] = G_l.  survivors (optional) receives the per-layer counts.
 * Returns n_keep. */
int64_t rsdgc_oracle_update_ratios(const float *w, const int64_t *sizes, int32_t L, float rho,
                                   float *ratios, int64_t *survivors)
{
    int64_t G = 0;
    for (int32_t l = 0; l < L; ++l) G += sizes[l];
    double x = ceil((double)rho * (double)G);
    int64_t n_keep = (x > 0.0) ? ((x >= (double)G) ? G : (int64_t)x) : 0;

    float *mu = (float *)malloc((size_t)(G > 0 ? G : 1) * sizeof(float));
    int64_t *order = (int64_t *)malloc((size_t)(G > 0 ? G : 1) * sizeof(int64_t));
    for (int64_t i = 0; i < G; ++i) {
        mu[i] = fabsf(w[i]);
        order[i] = i;
    }
    g_sort_absw = mu;
    qsort(order, (size_t)G, sizeof(int64_t), cmp_desc_abs_then_index_i64);

    int64_t *cnt = (int64_t *)calloc((size_t)L, sizeof(int64_t));
    int64_t *start = (int64_t *)malloc((size_t)(L + 1) * sizeof(int64_t));
    start[0] = 0;
    for (int32_t l = 0; l < L; ++l) start[l + 1] = start[l] + sizes[l];
    for (int64_t r = 0; r < n_keep; ++r) {
        int64_t i = order[r];
        int32_t lo = 0, hi = L; /* layer with start[lo] <= i < start[lo+1] */
        while (hi - lo > 1) {
            int32_t mid = (lo + hi) / 2;
            if (start[mid] <= i) lo = mid; else hi = mid;
        }
        cnt[lo] += 1;
    }
    for (int32_t l = 0; l < L; ++l) {
        ratios[l] = (sizes[l] > 0) ? (float)((double)cnt[l] / (double)sizes[l]) : 0.0f;
        if (survivors) survivors[l] = cnt[l];
    }
    free(mu); free(order); free(cnt); free(start);
    return n_keep;
}
