/*
 * qgbdt_oracle.c -- plain, slow, single-threaded CPU statement of quantized GBDT training.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the correctness authority that the CUDA
 * library is compared with.  It shares no source, header, table or helper with the
 * CUDA path, and nothing in the product path may call it.  Build with
 *     gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
 * so that every floating-point operation below is one individually rounded IEEE
 * operation (no fused contraction except where fmaf() is written out).
 *
 * What follows the paper, and where:
 *   qo_quantize        Eq. 5 (interval lengths), Eq. 6 (scaling), Eq. 8 (SR / RN)
 *   qo_histogram       Algorithm 1 with the integer gradients of Sec. 4.1
 *   qo_histogram_fp    Algorithm 1 as printed, with the original floating-point gradients
 *   qo_find_split      Eq. 7 (gain from integer sums), exhaustive scan of Sec. 3
 *   qo_partition       the index sets I_s of Sec. 3 (stable filter)
 *   qo_refit           Eq. 3 with the original gradients (Sec. 4.2, leaf-value refitting)
 *   qo_leaf_value_quantized   the leaf value from the quantized sums (Sec. 4.2, first formula)
 *   qo_gradients       Eq. 1 for the logistic and the squared loss (Sec. 5)
 *   qo_train_tree      Sec. 3 greedy leaf-wise growth + Fig. 1 workflow
 *
 * Conventions the paper leaves open (random source, rounding arithmetic, validity
 * rules, tie-breaks, the deterministic sigmoid, fixed-point refit sums) are fixed
 * here, each where it is used, with the reason beside it.
 *
 * Pins: every function here is pinned by the CPU tests (brute force, closed forms,
 * invariants, the paper's worked examples) except the exact output values of the
 * counter hash qo_sr_uniforms, which are a convention of this build: that function
 * is pinned only statistically (uniformity, independence, unbiased rounding).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define QO_OK 0
#define QO_ERR_ARG (-1)
#define QO_ERR_VALUE (-6) /* non-finite gradient, negative hessian, or |g| >= 256 */

typedef struct {
    int32_t bits;             /* B in 2..8 */
    int32_t objective;        /* 0 logistic, 1 squared loss (constant hessian 1) */
    int32_t num_leaves;
    int32_t num_trees;
    int32_t min_data_in_leaf;
    double learning_rate;
    double lambda_l2;
    double min_sum_hessian;
    double min_gain;
    uint64_t seed;
    int32_t hess_levels_mode; /* 0: 2^B-2 hessian intervals (Eq. 5); 1: 2^B-1 */
    int32_t rounding;         /* 0 stochastic rounding, 1 round to nearest */
} qo_params;

typedef struct {
    int32_t feature, bin;
    double gain;
    int64_t gl, hl, gr, hr;
    int64_t nl_est, nr_est;
    int32_t valid;
} qo_split;

/* ------------------------------------------------------------------ levels */

/* Eq. 5: 2^(B-1)-1 positive gradient levels; 2^B-2 hessian intervals. */
int qo_levels_g(int bits) { return (1 << (bits - 1)) - 1; }
int qo_levels_h(int bits, int hess_levels_mode) {
    return hess_levels_mode == 0 ? (1 << bits) - 2 : (1 << bits) - 1;
}

/* ------------------------------------------------------- counter-based hash */

static uint32_t qo_mix(uint32_t x) {
    x ^= x >> 16;
    x *= 0x9E3779B9u;
    x ^= x >> 15;
    x *= 0xBB67AE85u;
    x ^= x >> 16;
    return x;
}

/* Two 24-bit uniforms for (seed, tree, row): the random source of Eq. 8's SR. */
void qo_sr_uniforms(uint64_t seed, uint32_t tree, uint32_t row, uint32_t *u_g, uint32_t *u_h) {
    uint32_t seed_lo = (uint32_t)(seed & 0xFFFFFFFFu);
    uint32_t seed_hi = (uint32_t)(seed >> 32);
    uint32_t key = qo_mix(qo_mix(qo_mix(seed_lo ^ 0x6A09E667u) + seed_hi) ^ tree);
    uint32_t r = qo_mix(key ^ row);
    *u_g = qo_mix(r) >> 8;
    *u_h = qo_mix(r + 0x6A09E667u) >> 8;
}

/* The same for rows row0 .. row0+n-1 (convenience for statistical tests). */
void qo_sr_uniforms_range(uint64_t seed, uint32_t tree, uint32_t row0, int64_t n, uint32_t *u_g,
                          uint32_t *u_h) {
    for (int64_t i = 0; i < n; ++i) qo_sr_uniforms(seed, tree, row0 + (uint32_t)i, u_g + i, u_h + i);
}

/* ----------------------------------------------------------------- rounding */

/* Eq. 8.  x already scaled to integer units and clamped to [lo, hi].
 * SR: floor(x) + [u < floor(frac * 2^24)], u a 24-bit uniform, so P(up) = frac
 * to within 2^-24.  RN: floor(x) + [frac >= 1/2] (ties go up). */
static int qo_round(float x, int rounding, uint32_t u) {
    float f = floorf(x);
    float frac = x - f; /* exact */
    if (rounding == 1) return (int)f + (frac >= 0.5f ? 1 : 0);
    uint32_t t = (uint32_t)(frac * 16777216.0f); /* exact scaling, truncation */
    return (int)f + (u < t ? 1 : 0);
}

/* Eq. 5 + Eq. 6 + Eq. 8 over all n training rows of one boosting iteration.
 * h == NULL means a constant hessian: it is not quantized (Sec. 4.1), every
 * row carries the integer 1 and the hessian scale is 1.
 * Outputs: gq[n] in [-k_g, k_g], hq[n] in [0, k_h], gmax = max|g|, hmax = max h. */
int qo_quantize(const float *g, const float *h, int64_t n, int bits, int hess_levels_mode,
                int rounding, uint64_t seed, uint32_t tree, int8_t *gq, uint8_t *hq,
                float *gmax_out, float *hmax_out) {
    if (!g || !gq || !hq || n < 0 || bits < 2 || bits > 8) return QO_ERR_ARG;
    int kg = qo_levels_g(bits), kh = qo_levels_h(bits, hess_levels_mode);
    float gmax = 0.0f, hmax = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        if (!isfinite(g[i]) || fabsf(g[i]) >= 256.0f) return QO_ERR_VALUE;
        if (fabsf(g[i]) > gmax) gmax = fabsf(g[i]);
        if (h) {
            if (!isfinite(h[i]) || h[i] < 0.0f || h[i] >= 256.0f) return QO_ERR_VALUE;
            if (h[i] > hmax) hmax = h[i];
        }
    }
    if (!h) hmax = 1.0f;
    float inv_g = gmax > 0.0f ? (float)kg / gmax : 0.0f; /* 1 / delta_g */
    float inv_h = hmax > 0.0f ? (float)kh / hmax : 0.0f; /* 1 / delta_h */
    for (int64_t i = 0; i < n; ++i) {
        uint32_t ug, uh;
        qo_sr_uniforms(seed, tree, (uint32_t)i, &ug, &uh);
        float x = g[i] * inv_g;
        if (x > (float)kg) x = (float)kg;
        if (x < -(float)kg) x = -(float)kg;
        gq[i] = (int8_t)qo_round(x, rounding, ug);
        if (h) {
            float y = h[i] * inv_h;
            if (y > (float)kh) y = (float)kh;
            if (y < 0.0f) y = 0.0f;
            hq[i] = (uint8_t)qo_round(y, rounding, uh);
        } else {
            hq[i] = 1;
        }
    }
    *gmax_out = gmax;
    *hmax_out = hmax;
    return QO_OK;
}

/* ---------------------------------------------------------------- histogram */

/* Algorithm 1 with integer gradients.  data is the bin matrix data[N][J] (row-major,
 * one byte per entry); idx lists I_s (NULL: rows 0..n_s-1).  hist_g / hist_h are
 * [J][n_bins] and are overwritten. */
int qo_histogram(const uint8_t *data, int64_t n_rows, int32_t n_features, int32_t n_bins,
                 const int8_t *gq, const uint8_t *hq, const uint32_t *idx, int64_t n_s,
                 int64_t *hist_g, int64_t *hist_h) {
    if (!data || !gq || !hq || !hist_g || !hist_h) return QO_ERR_ARG;
    memset(hist_g, 0, sizeof(int64_t) * (size_t)n_features * (size_t)n_bins);
    memset(hist_h, 0, sizeof(int64_t) * (size_t)n_features * (size_t)n_bins);
    for (int64_t p = 0; p < n_s; ++p) {
        int64_t i = idx ? (int64_t)idx[p] : p;
        if (i >= n_rows) return QO_ERR_ARG;
        for (int32_t j = 0; j < n_features; ++j) {
            int32_t bin = data[i * n_features + j];
            if (bin >= n_bins) return QO_ERR_ARG;
            hist_g[(int64_t)j * n_bins + bin] += gq[i];
            hist_h[(int64_t)j * n_bins + bin] += hq[i];
        }
    }
    return QO_OK;
}

/* Algorithm 1 as the paper prints it, before quantization: the original gradients g_i, h_i
 * (h == NULL: a constant hessian 1) summed per (feature, bin), here in double precision.  This
 * is what a floating-point histogram (the unquantized baseline of Sec. 7.2) has to approximate. */
int qo_histogram_fp(const uint8_t *data, int64_t n_rows, int32_t n_features, int32_t n_bins,
                    const float *g, const float *h, const uint32_t *idx, int64_t n_s,
                    double *hist_g, double *hist_h) {
    if (!data || !g || !hist_g || !hist_h) return QO_ERR_ARG;
    for (int64_t k = 0; k < (int64_t)n_features * n_bins; ++k) { hist_g[k] = 0.0; hist_h[k] = 0.0; }
    for (int64_t p = 0; p < n_s; ++p) {
        int64_t i = idx ? (int64_t)idx[p] : p;
        if (i >= n_rows) return QO_ERR_ARG;
        for (int32_t j = 0; j < n_features; ++j) {
            int32_t bin = data[i * n_features + j];
            if (bin >= n_bins) return QO_ERR_ARG;
            hist_g[(int64_t)j * n_bins + bin] += (double)g[i];
            hist_h[(int64_t)j * n_bins + bin] += h ? (double)h[i] : 1.0;
        }
    }
    return QO_OK;
}

/* --------------------------------------------------------------- split gain */

/* One term of Eq. 7: (G~ delta_g)^2 / (H~ delta_h [+ lambda]). */
static double qo_term(int64_t G, int64_t H, double dg, double dh, double lambda_l2) {
    double gd = (double)G * dg;
    double hd = (double)H * dh + lambda_l2;
    return (gd * gd) / hd;
}

/* Eq. 7 for one candidate: 1/2 (term(L) + term(R) - term(P)). */
double qo_gain(int64_t gl, int64_t hl, int64_t gr, int64_t hr, double dg, double dh,
               double lambda_l2) {
    double tl = qo_term(gl, hl, dg, dh, lambda_l2);
    double tr = qo_term(gr, hr, dg, dh, lambda_l2);
    double tp = qo_term(gl + gr, hl + hr, dg, dh, lambda_l2);
    return 0.5 * ((tl + tr) - tp);
}

/* Exhaustive scan over (feature, threshold bin): rows with bin <= t go left.
 * G, H, n_s are the leaf's integer totals and row count; gmax/hmax the iteration's
 * maxima (delta_g = gmax/k_g, delta_h = hmax/k_h; constant hessian: delta_h = 1).
 * Row counts per side are estimated from hessian sums (exact when the hessian is
 * constant), since the histogram carries no count field. */
int qo_find_split(const int64_t *hist_g, const int64_t *hist_h, int32_t n_features,
                  int32_t n_bins, int64_t G, int64_t H, int64_t n_s, float gmax, float hmax,
                  int const_hessian, const qo_params *prm, qo_split *out) {
    if (!hist_g || !hist_h || !prm || !out) return QO_ERR_ARG;
    int kg = qo_levels_g(prm->bits), kh = qo_levels_h(prm->bits, prm->hess_levels_mode);
    double dg = (double)gmax / (double)kg;
    double dh = const_hessian ? 1.0 : (double)hmax / (double)kh;
    memset(out, 0, sizeof(*out));
    out->feature = -1;
    out->bin = -1;
    for (int32_t f = 0; f < n_features; ++f) {
        int64_t gl = 0, hl = 0;
        for (int32_t t = 0; t + 1 < n_bins; ++t) {
            gl += hist_g[(int64_t)f * n_bins + t];
            hl += hist_h[(int64_t)f * n_bins + t];
            int64_t gr = G - gl, hr = H - hl;
            if (hl <= 0 || hr <= 0) continue;
            int64_t nl;
            if (const_hessian) nl = hl;
            else nl = (int64_t)(((uint64_t)hl * (uint64_t)n_s + (uint64_t)(H / 2)) / (uint64_t)H);
            int64_t nr = n_s - nl;
            if (nl < prm->min_data_in_leaf || nr < prm->min_data_in_leaf) continue;
            if ((double)hl * dh < prm->min_sum_hessian || (double)hr * dh < prm->min_sum_hessian)
                continue;
            double gain = qo_gain(gl, hl, gr, hr, dg, dh, prm->lambda_l2);
            if (!(gain > prm->min_gain)) continue;
            if (!out->valid || gain > out->gain) { /* strict: lowest (f, t) wins ties */
                out->valid = 1;
                out->feature = f;
                out->bin = t;
                out->gain = gain;
                out->gl = gl; out->hl = hl; out->gr = gr; out->hr = hr;
                out->nl_est = nl; out->nr_est = nr;
            }
        }
    }
    return QO_OK;
}

/* ---------------------------------------------------------------- partition */

/* Stable split of I_s: rows with data[i][feature] <= bin first (order kept), then
 * the rest (order kept).  Returns the number of rows that went left. */
int64_t qo_partition(const uint8_t *data, int32_t n_features, const uint32_t *idx, int64_t n_s,
                     int32_t feature, int32_t bin, uint32_t *out_idx) {
    int64_t nl = 0;
    for (int64_t p = 0; p < n_s; ++p)
        if (data[(int64_t)idx[p] * n_features + feature] <= bin) out_idx[nl++] = idx[p];
    int64_t w = nl;
    for (int64_t p = 0; p < n_s; ++p)
        if (data[(int64_t)idx[p] * n_features + feature] > bin) out_idx[w++] = idx[p];
    return nl;
}

/* -------------------------------------------------------------------- refit */

/* Eq. 3 with the ORIGINAL gradients of the rows in one leaf.  Sums are taken in
 * 2^-30 fixed point (each term rounded once, the int64 sum is then exact and
 * order-independent), w = -sum g / (sum h + lambda); the leaf output is
 * (float)(learning_rate * w); a non-positive denominator gives 0. */
int qo_refit(const float *g, const float *h, const uint32_t *idx, int64_t n_s, double lambda_l2,
             double learning_rate, double *w_out, float *value_out) {
    int64_t sg = 0, sh = 0;
    for (int64_t p = 0; p < n_s; ++p) {
        uint32_t i = idx[p];
        sg += llrint((double)g[i] * 1073741824.0);
        sh += h ? llrint((double)h[i] * 1073741824.0) : (int64_t)1073741824;
    }
    double den = (double)sh + lambda_l2 * 1073741824.0;
    double w = den > 0.0 ? -(double)sg / den : 0.0;
    *w_out = w;
    *value_out = (float)(learning_rate * w);
    return QO_OK;
}

/* Sec. 4.2, the leaf value without refitting: w~ = -(G~ delta_g) / (H~ delta_h), from the
 * integer sums of the leaf and the interval lengths of Eq. 5 (constant hessian: delta_h = 1).
 * lambda_l2 joins the denominator as in Eq. 7's terms; a non-positive denominator gives 0.
 * The leaf output is (float)(learning_rate * w~). */
int qo_leaf_value_quantized(int64_t G, int64_t H, float gmax, float hmax, int bits,
                            int hess_levels_mode, int const_hessian, double lambda_l2,
                            double learning_rate, double *w_out, float *value_out) {
    double dg = (double)gmax / (double)qo_levels_g(bits);
    double dh = const_hessian ? 1.0 : (double)hmax / (double)qo_levels_h(bits, hess_levels_mode);
    double gd = (double)G * dg;
    double hd = (double)H * dh + lambda_l2;
    double w = hd > 0.0 ? -gd / hd : 0.0;
    *w_out = w;
    *value_out = (float)(learning_rate * w);
    return QO_OK;
}

/* ---------------------------------------------------------------- gradients */

/* A sigmoid built only from exactly rounded primitives (rintf, fmaf, one divide)
 * so that any IEEE machine gives the same bits: e = exp(-|s|) by range reduction
 * with a split ln 2 and a degree-6 polynomial, then 1/(1+e) or e/(1+e). */
float qo_sigmoid(float s) {
    float a = fabsf(s);
    if (a > 40.0f) a = 40.0f;
    float x = -a;
    float n = rintf(x * 0x1.715476p+0f);
    float r = fmaf(n, -0x1.62e400p-1f, x);
    r = fmaf(n, -0x1.7f7d1cp-20f, r);
    float p = 0x1.6c16c2p-10f;          /* 1/720 */
    p = fmaf(p, r, 0x1.111112p-7f);     /* 1/120 */
    p = fmaf(p, r, 0x1.555556p-5f);     /* 1/24  */
    p = fmaf(p, r, 0x1.555556p-3f);     /* 1/6   */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    int32_t bits;
    memcpy(&bits, &p, 4);
    bits += ((int32_t)n) << 23;          /* times 2^n, n in [-58, 0]: stays normal */
    float e;
    memcpy(&e, &bits, 4);
    float d = 1.0f + e;
    return s >= 0.0f ? 1.0f / d : e / d;
}

/* Eq. 1.  objective 0: logistic loss with labels in {0,1}: g = p - y, h = p(1-p).
 * objective 1: squared loss 1/2 (s - y)^2: g = s - y, constant hessian (h untouched). */
int qo_gradients(int objective, const float *scores, const float *labels, int64_t n, float *g,
                 float *h) {
    for (int64_t i = 0; i < n; ++i) {
        if (objective == 0) {
            float p = qo_sigmoid(scores[i]);
            g[i] = p - labels[i];
            float q = 1.0f - p;
            h[i] = p * q;
        } else {
            g[i] = scores[i] - labels[i];
        }
    }
    return QO_OK;
}

/* ----------------------------------------------------------------- training */

/* One boosting iteration (Fig. 1): gradients -> quantize -> leaf-wise growth with
 * integer histograms -> refit -> score update.  Every child histogram is built
 * directly by Algorithm 1 (no subtraction shortcut).
 * Tree output: node arrays [num_leaves-1] (feature, threshold bin, left, right;
 * a child c < 0 is leaf ~c), node gain, leaf_value[num_leaves], leaf_count[num_leaves].
 * Splitting leaf l keeps l as the left child and makes leaf `n_leaves` the right one.
 * row_leaf[n] (optional) receives the leaf of every row.  Returns the leaf count
 * (>= 1) or a negative error.
 * leaf_values_from_quantized_sums != 0: the leaf values are w~ of Sec. 4.2 (no refit). */
int qo_train_tree_opt(const uint8_t *data, int64_t n, int32_t n_features, int32_t n_bins,
                      const float *labels, float *scores, const qo_params *prm, uint32_t tree,
                      int leaf_values_from_quantized_sums, int32_t *node_feature,
                      int32_t *node_bin, int32_t *node_left, int32_t *node_right,
                      double *node_gain, float *leaf_value, int64_t *leaf_count,
                      int32_t *row_leaf) {
    if (!data || !labels || !scores || !prm || n <= 0 || prm->num_leaves < 1) return QO_ERR_ARG;
    int L = prm->num_leaves;
    int const_h = prm->objective == 1;
    size_t hsz = (size_t)n_features * (size_t)n_bins;
    float *g = malloc(sizeof(float) * (size_t)n);
    float *h = const_h ? NULL : malloc(sizeof(float) * (size_t)n);
    int8_t *gq = malloc((size_t)n);
    uint8_t *hq = malloc((size_t)n);
    uint32_t *idx = malloc(sizeof(uint32_t) * (size_t)n);
    uint32_t *tmp = malloc(sizeof(uint32_t) * (size_t)n);
    int64_t *hg = malloc(sizeof(int64_t) * hsz), *hh = malloc(sizeof(int64_t) * hsz);
    int64_t *off = calloc((size_t)L, sizeof(int64_t)), *cnt = calloc((size_t)L, sizeof(int64_t));
    int64_t *tot_g = calloc((size_t)L, sizeof(int64_t)), *tot_h = calloc((size_t)L, sizeof(int64_t));
    int32_t *parent_node = malloc(sizeof(int32_t) * (size_t)L); /* node owning the leaf, and side */
    int32_t *parent_side = malloc(sizeof(int32_t) * (size_t)L);
    qo_split *best = calloc((size_t)L, sizeof(qo_split));
    int rc = QO_OK, n_leaves = 1;
    float gmax, hmax;

    qo_gradients(prm->objective, scores, labels, n, g, h);
    rc = qo_quantize(g, h, n, prm->bits, prm->hess_levels_mode, prm->rounding, prm->seed, tree, gq,
                     hq, &gmax, &hmax);
    if (rc != QO_OK) goto done;

    for (int64_t i = 0; i < n; ++i) { idx[i] = (uint32_t)i; tot_g[0] += gq[i]; tot_h[0] += hq[i]; }
    off[0] = 0; cnt[0] = n; parent_node[0] = -1; parent_side[0] = 0;
    qo_histogram(data, n, n_features, n_bins, gq, hq, idx, n, hg, hh);
    qo_find_split(hg, hh, n_features, n_bins, tot_g[0], tot_h[0], n, gmax, hmax, const_h, prm,
                  &best[0]);

    while (n_leaves < L) {
        int pick = -1;
        for (int l = 0; l < n_leaves; ++l)
            if (best[l].valid && (pick < 0 || best[l].gain > best[pick].gain)) pick = l;
        if (pick < 0) break;
        qo_split s = best[pick];
        int64_t nl = qo_partition(data, n_features, idx + off[pick], cnt[pick], s.feature, s.bin, tmp);
        memcpy(idx + off[pick], tmp, sizeof(uint32_t) * (size_t)cnt[pick]);
        int node = n_leaves - 1, right = n_leaves;
        node_feature[node] = s.feature;
        node_bin[node] = s.bin;
        node_left[node] = ~pick;
        node_right[node] = ~right;
        node_gain[node] = s.gain;
        if (parent_node[pick] >= 0) {
            if (parent_side[pick] == 0) node_left[parent_node[pick]] = node;
            else node_right[parent_node[pick]] = node;
        }
        parent_node[pick] = node; parent_side[pick] = 0;
        parent_node[right] = node; parent_side[right] = 1;
        off[right] = off[pick] + nl; cnt[right] = cnt[pick] - nl; cnt[pick] = nl;
        tot_g[pick] = s.gl; tot_h[pick] = s.hl; tot_g[right] = s.gr; tot_h[right] = s.hr;
        n_leaves++;
        int child[2] = {pick, right};
        for (int c = 0; c < 2; ++c) {
            int l = child[c];
            qo_histogram(data, n, n_features, n_bins, gq, hq, idx + off[l], cnt[l], hg, hh);
            qo_find_split(hg, hh, n_features, n_bins, tot_g[l], tot_h[l], cnt[l], gmax, hmax,
                          const_h, prm, &best[l]);
        }
    }

    for (int l = 0; l < n_leaves; ++l) {
        double w;
        if (leaf_values_from_quantized_sums) /* Sec. 4.2: w~ from the leaf's integer sums */
            qo_leaf_value_quantized(tot_g[l], tot_h[l], gmax, hmax, prm->bits, prm->hess_levels_mode,
                                    const_h, prm->lambda_l2, prm->learning_rate, &w, &leaf_value[l]);
        else
            qo_refit(g, h, idx + off[l], cnt[l], prm->lambda_l2, prm->learning_rate, &w, &leaf_value[l]);
        leaf_count[l] = cnt[l];
        for (int64_t p = 0; p < cnt[l]; ++p) {
            uint32_t i = idx[off[l] + p];
            scores[i] = scores[i] + leaf_value[l];
            if (row_leaf) row_leaf[i] = l;
        }
    }
    rc = n_leaves;
done:
    free(g); free(h); free(gq); free(hq); free(idx); free(tmp); free(hg); free(hh);
    free(off); free(cnt); free(tot_g); free(tot_h); free(parent_node); free(parent_side); free(best);
    return rc;
}

/* The same with the leaf values refitted from the original gradients (the default of Sec. 4.2). */
int qo_train_tree(const uint8_t *data, int64_t n, int32_t n_features, int32_t n_bins,
                  const float *labels, float *scores, const qo_params *prm, uint32_t tree,
                  int32_t *node_feature, int32_t *node_bin, int32_t *node_left,
                  int32_t *node_right, double *node_gain, float *leaf_value,
                  int64_t *leaf_count, int32_t *row_leaf) {
    return qo_train_tree_opt(data, n, n_features, n_bins, labels, scores, prm, tree, 0, node_feature,
                             node_bin, node_left, node_right, node_gain, leaf_value, leaf_count,
                             row_leaf);
}

/* Full training: num_trees iterations; tree k's arrays live at offset k*(L-1) (nodes)
 * and k*L (leaves).  tree_leaves[k] receives each tree's leaf count. */
int qo_train(const uint8_t *data, int64_t n, int32_t n_features, int32_t n_bins,
             const float *labels, float *scores, const qo_params *prm, int32_t *tree_leaves,
             int32_t *node_feature, int32_t *node_bin, int32_t *node_left, int32_t *node_right,
             double *node_gain, float *leaf_value, int64_t *leaf_count) {
    int L = prm->num_leaves;
    for (int k = 0; k < prm->num_trees; ++k) {
        size_t no = (size_t)k * (size_t)(L - 1), lo = (size_t)k * (size_t)L;
        int rc = qo_train_tree(data, n, n_features, n_bins, labels, scores, prm, (uint32_t)k,
                               node_feature + no, node_bin + no, node_left + no, node_right + no,
                               node_gain + no, leaf_value + lo, leaf_count + lo, NULL);
        if (rc < 0) return rc;
        tree_leaves[k] = rc;
    }
    return QO_OK;
}

/* Leaf reached by one row of bin codes in a tree given as node arrays. */
int qo_predict_leaf(const uint8_t *row, int32_t n_leaves, const int32_t *node_feature,
                    const int32_t *node_bin, const int32_t *node_left, const int32_t *node_right) {
    if (n_leaves <= 1) return 0;
    int node = 0;
    for (;;) {
        int next = row[node_feature[node]] <= node_bin[node] ? node_left[node] : node_right[node];
        if (next < 0) return ~next;
        node = next;
    }
}
