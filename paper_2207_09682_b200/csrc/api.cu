// C ABI of libqgbdt: context management, argument checks, and the host-side sequencing of
// the kernels.  No arithmetic of the method happens on the host except picking the leaf
// with the largest stored gain and bookkeeping of leaf ranges.
#include <cstdarg>
#include <cstring>
#include <new>

#include "qgbdt_internal.cuh"

int qg_fail(qgbdt_ctx *c, int code, const char *fmt, ...) {
    if (c) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->err, sizeof(c->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

int qg_phase_begin(qgbdt_ctx *c, int phase, cudaStream_t st) {
    if (!c->profile_hist) return QGBDT_OK;
    if (c->hist_events_used + 2 > c->hist_events.size()) {
        for (int i = 0; i < 2; ++i) {
            cudaEvent_t e;
            QG_CUDA(c, cudaEventCreate(&e));
            c->hist_events.push_back(e);
        }
        c->hist_event_phase.push_back(phase);
    }
    c->hist_event_phase[c->hist_events_used / 2] = phase;
    QG_CUDA(c, cudaEventRecord(c->hist_events[c->hist_events_used], st));
    c->hist_events_used += 2;
    return QGBDT_OK;
}

int qg_phase_end(qgbdt_ctx *c, cudaStream_t st) {
    if (!c->profile_hist || c->hist_events_used < 2) return QGBDT_OK;
    QG_CUDA(c, cudaEventRecord(c->hist_events[c->hist_events_used - 1], st));
    return QGBDT_OK;
}

int qg_allreduce(qgbdt_ctx *c, void *d_buf, int64_t count, int kind, cudaStream_t st) {
    if (!qg_sharded(c) || count <= 0) return QGBDT_OK;
    if (c->dist_reduce(c->dist_user, d_buf, count, kind, st) != 0)
        return qg_fail(c, QGBDT_ERR_CUDA, "the all-reduce callback failed (%lld words, kind %d)", (long long)count, kind);
    return QGBDT_OK;
}

static_assert(sizeof(qgbdt_params) == 72 && sizeof(qgbdt_split) == 72 && sizeof(qgbdt_bin) == 8,
              "ABI struct sizes are part of the interface");

namespace {

constexpr size_t PINNED_BYTES = 128 * 1024;
constexpr size_t PINNED_SCALARS = 64 * 1024;  // offset of the small-scalar area
constexpr int MAX_LEAVES = 4096;

template <typename T>
int dev_alloc(qgbdt_ctx *c, T **p, size_t count) {
    void *q = nullptr;
    cudaError_t e = cudaMalloc(&q, count * sizeof(T) > 0 ? count * sizeof(T) : 16);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return qg_fail(c, QGBDT_ERR_ALLOC, "cudaMalloc of %zu bytes failed: %s", count * sizeof(T), cudaGetErrorString(e));
    }
    *p = reinterpret_cast<T *>(q);
    return QGBDT_OK;
}

template <typename T>
void dev_free(T *&p) {
    if (p) cudaFree(p);
    p = nullptr;
}

void free_data(qgbdt_ctx *c) {
    qg_grow_graph_destroy(c);   // its launches point into the buffers freed below
    for (void *p : c->tile_allocs) cudaFree(p);
    c->tile_allocs.clear();
    c->tiles.clear();
    dev_free(c->d_tiles);
    dev_free(c->d_partial);
    dev_free(c->d_codes);
    dev_free(c->d_codes_nat);
    dev_free(c->d_idx);
    dev_free(c->d_idx_tmp);
    dev_free(c->d_part_counts);
    dev_free(c->d_part_bits);
    dev_free(c->d_feat_best);
    dev_free(c->d_g);
    dev_free(c->d_h);
    dev_free(c->d_hist_pool);
    dev_free(c->d_leaves);
    dev_free(c->d_recs);
    dev_free(c->d_rec_gain);
    dev_free(c->d_rec_child);
    dev_free(c->d_rec_pos);
    dev_free(c->d_rec_parent);
    dev_free(c->d_front);
    dev_free(c->d_grow_bits);
    dev_free(c->d_grow_partial);
    dev_free(c->d_grow_prep);
    dev_free(c->d_ent0);
    dev_free(c->d_ent1);
    dev_free(c->d_leaf_id);
    dev_free(c->d_cand);
    dev_free(c->d_feat_rec);
    dev_free(c->d_colmajor);
    c->col_stride = 0;
    dev_free(c->d_m_num_leaves);
    dev_free(c->d_m_feature);
    dev_free(c->d_m_bin);
    dev_free(c->d_m_left);
    dev_free(c->d_m_right);
    dev_free(c->d_m_gain);
    dev_free(c->d_m_leaf_value);
    dev_free(c->d_m_leaf_count);
    c->model_cap = 0;
    c->loaded = false;
    c->quantized = false;
}

int next_pow2(int v) {
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

// Feature tiles: full tiles of 128 features, then the remainder either padded to a power-of-two
// number of words (cheap padding, or a matrix narrower than one tile: one row = one aligned
// segment, which keeps row gathers sector-exact) or split into power-of-two pieces.
void plan_tiles(int F, std::vector<TileDesc> &out) {
    int f = 0;
    auto add = [&](int nf, int words) {
        TileDesc t;
        t.data = nullptr;
        t.f0 = f;
        t.nf = nf;
        int lw = 0;
        while ((1 << lw) < words) ++lw;
        t.logW = lw;
        t.words_used = (nf + 3) / 4;
        out.push_back(t);
        f += nf;
    };
    while (F - f >= 128) add(128, 32);
    while (F - f > 0) {
        const int rem = F - f;
        const int w = (rem + 3) / 4;
        const int P = next_pow2(w);
        if (F < 128 || (P - w) * 4 * 20 <= F) {
            add(rem, P);
        } else {
            int q = P / 2;  // largest power of two below w
            add(q * 4, q);
        }
    }
}

// Histogram plan.  Tiles of equal width form a group that is built by one launch (the full
// 128-feature tiles, then the remainder tiles); a group's tiles get equal shares of the SMs, and with
// more tiles than SMs every tile gets one CTA.  Fills parts / cta0 of the tiles; part p of a tile
// owns partial-histogram slot cta0 + p.
void plan_hist_ctas(int sm_count, std::vector<TileDesc> &tiles, int &n_ctas, int &max_parts) {
    const int T = (int)tiles.size();
    n_ctas = 0;
    max_parts = 1;
    for (int t0 = 0; t0 < T;) {
        int t1 = t0 + 1;
        while (t1 < T && tiles[t1].logW == tiles[t0].logW) ++t1;
        const int g = t1 - t0;
        for (int i = t0; i < t1; ++i) {
            int p = sm_count / g;   // equal shares: (parts, tiles of the group) is then a grid of at most one CTA per SM
            if (p < 1) p = 1;
            tiles[i].parts = p;
            tiles[i].cta0 = n_ctas;
            n_ctas += p;
            if (p > max_parts) max_parts = p;
        }
        t0 = t1;
    }
}

int check_loaded(qgbdt_ctx *c) {
    if (!c) return QGBDT_ERR_ARG;
    if (!c->loaded) return qg_fail(c, QGBDT_ERR_STATE, "no bin matrix loaded");
    return QGBDT_OK;
}

void reset_leaf_state(qgbdt_ctx *c) {
    c->n_leaves = 1;
    c->refit_leaves = 0;
    c->leaf_off.assign(c->prm.num_leaves, 0);
    c->leaf_n.assign(c->prm.num_leaves, 0);
    c->leaf_n[0] = c->N;
}

void rec_to_split(const SplitRec &r, int64_t G, int64_t H, int64_t n_rows, bool const_h, qgbdt_split *out) {
    memset(out, 0, sizeof(*out));
    out->feature = -1;
    out->bin = -1;
    if (!r.valid) return;
    out->valid = 1;
    out->feature = r.feature;
    out->bin = r.bin;
    out->gain = r.gain;
    out->gl = r.gl;
    out->hl = r.hl;
    out->gr = G - r.gl;
    out->hr = H - r.hl;
    // row estimate of the candidate (same integer formula as the scan kernel)
    out->nl_est = const_h ? r.hl
                          : (int64_t)(((unsigned long long)r.hl * (unsigned long long)n_rows + (unsigned long long)(H / 2)) /
                                      (unsigned long long)H);
    out->nr_est = n_rows - out->nl_est;
}

int load_common(qgbdt_ctx *c, const uint8_t *d_bins, int64_t n_rows, int32_t n_features, int32_t n_bins,
                int32_t layout, int64_t ld, cudaStream_t st) {
    free_data(c);
    c->N = n_rows;
    c->F = n_features;
    c->nb = n_bins;
    c->code_bytes = c->prm.bits <= 4 ? 1 : 2;   // packed gradient + hessian code of a row that the method has to move (Sec. 6.2)
    plan_tiles(n_features, c->tiles);
    plan_hist_ctas(c->sm_count, c->tiles, c->hist_grid, c->max_parts);
    int rc;
    for (TileDesc &t : c->tiles) {
        uint32_t *p = nullptr;
        if ((rc = dev_alloc(c, &p, (size_t)n_rows << t.logW)) != QGBDT_OK) return rc;
        c->tile_allocs.push_back(p);
        t.data = p;
    }
    if ((rc = dev_alloc(c, &c->d_tiles, c->tiles.size())) != QGBDT_OK) return rc;
    QG_CUDA(c, cudaMemcpyAsync(c->d_tiles, c->tiles.data(), sizeof(TileDesc) * c->tiles.size(),
                               cudaMemcpyHostToDevice, st));
    if (c->max_parts > 1 &&
        (rc = dev_alloc(c, &c->d_partial, (size_t)c->hist_grid * 4 * n_bins * 32)) != QGBDT_OK)
        return rc;
    if ((rc = dev_alloc(c, &c->d_codes, ((size_t)n_rows + 15) / 16 * 16 * 2 + 16)) != QGBDT_OK) return rc;
    if ((rc = dev_alloc(c, &c->d_codes_nat, (size_t)n_rows * 2 + 16)) != QGBDT_OK) return rc;
    if ((rc = dev_alloc(c, &c->d_idx, (size_t)n_rows)) != QGBDT_OK) return rc;
    if ((rc = dev_alloc(c, &c->d_idx_tmp, (size_t)n_rows)) != QGBDT_OK) return rc;
    // block counts of the step-wise partition (a block per 2048 rows), or the warp and block counts
    // of the partition launches of tree growth (nine words per block)
    c->grow_pb_total = c->sm_count * 8 + GROW_MAX_JOBS;
    {
        size_t need = (size_t)n_rows / 2048 + 8, grow = (size_t)c->grow_pb_total * 9 + 8;
        if ((rc = dev_alloc(c, &c->d_part_counts, need > grow ? need : grow)) != QGBDT_OK) return rc;
    }
    {
        std::vector<FeatRec> fr((size_t)n_features);
        int tile_no = -1;
        for (const TileDesc &t : c->tiles) {
            ++tile_no;
            for (int f = t.f0; f < t.f0 + t.nf; ++f) {
                const int fl = f - t.f0;
                fr[f].col = t.data + (fl >> 2);
                fr[f].logW = t.logW;
                fr[f].byte = fl & 3;
                fr[f].cta0 = t.cta0;
                fr[f].parts = t.parts;
                fr[f].fl = fl;
                fr[f].tile = tile_no;
                fr[f].col8 = nullptr;
            }
        }
        if ((rc = dev_alloc(c, &c->d_feat_rec, (size_t)n_features)) != QGBDT_OK) return rc;
        QG_CUDA(c, cudaMemcpy(c->d_feat_rec, fr.data(), sizeof(FeatRec) * fr.size(), cudaMemcpyHostToDevice));
    }
    if ((rc = dev_alloc(c, &c->d_part_bits, ((size_t)n_rows + 2048) / 32 + 64)) != QGBDT_OK) return rc;
    if ((rc = dev_alloc(c, &c->d_feat_best, (size_t)n_features)) != QGBDT_OK) return rc;
    QG_CUDA(c, cudaMemsetAsync(c->d_state, 0, sizeof(DevState), st));
    if ((rc = qg_relayout(c, d_bins, layout, ld, st)) != QGBDT_OK) return rc;
    if ((rc = qg_iota(c, st)) != QGBDT_OK) return rc;
    DevState *hs = reinterpret_cast<DevState *>(reinterpret_cast<char *>(c->h_pinned) + PINNED_SCALARS);
    QG_CUDA(c, cudaMemcpyAsync(hs, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    if (hs->bad_value) {
        free_data(c);
        return qg_fail(c, QGBDT_ERR_VALUE, "a bin code is >= n_bins (%d)", n_bins);
    }
    c->loaded = true;
    reset_leaf_state(c);
    return QGBDT_OK;
}

int check_load_args(qgbdt_ctx *c, const uint8_t *bins, int64_t n_rows, int32_t n_features, int32_t n_bins,
                    int32_t layout, int64_t ld) {
    if (!c) return QGBDT_ERR_ARG;
    if (!bins) return qg_fail(c, QGBDT_ERR_ARG, "bins is NULL");
    if (n_rows < 1 || n_rows >= (1ll << 31)) return qg_fail(c, QGBDT_ERR_ARG, "n_rows must be in [1, 2^31)");
    if (n_features < 1 || n_features > (1 << 20)) return qg_fail(c, QGBDT_ERR_ARG, "n_features out of range");
    if (n_bins < 2 || n_bins > 256) return qg_fail(c, QGBDT_ERR_ARG, "n_bins must be in [2, 256]");
    if (layout != 0 && layout != 1) return qg_fail(c, QGBDT_ERR_ARG, "layout must be 0 or 1");
    if (ld < (layout == 0 ? (int64_t)n_features : n_rows)) return qg_fail(c, QGBDT_ERR_ARG, "ld too small");
    const int64_t kg = qg_levels_g(c->prm.bits), kh = qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    if (n_rows * kg > 2147483647ll || n_rows * kh > 4294967295ll)
        return qg_fail(c, QGBDT_ERR_OVERFLOW, "n_rows * levels exceeds the 32+32-bit histogram word");
    return QGBDT_OK;
}

}  // namespace

extern "C" {

int qgbdt_create(qgbdt_ctx **out, const qgbdt_params *p) {
    if (!out || !p) return QGBDT_ERR_ARG;
    *out = nullptr;
    if (p->bits < 2 || p->bits > 8 || (p->objective != 0 && p->objective != 1) || p->num_leaves < 1 ||
        p->num_leaves > MAX_LEAVES || p->min_data_in_leaf < 0 || !(p->learning_rate == p->learning_rate) ||
        p->lambda_l2 < 0 || (p->hess_levels_mode != 0 && p->hess_levels_mode != 1) ||
        (p->rounding != 0 && p->rounding != 1))
        return QGBDT_ERR_ARG;
    qgbdt_ctx *c = new (std::nothrow) qgbdt_ctx();
    if (!c) return QGBDT_ERR_ALLOC;
    c->prm = *p;
    cudaDeviceProp prop;
    if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return QGBDT_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    c->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    c->coop_ok = prop.cooperativeLaunch != 0;
    const int L = p->num_leaves;
    bool ok = cudaMalloc(reinterpret_cast<void **>(&c->d_state), sizeof(DevState)) == cudaSuccess &&
              cudaMalloc(reinterpret_cast<void **>(&c->d_split_out), sizeof(SplitRec) * 4) == cudaSuccess &&
              cudaMalloc(reinterpret_cast<void **>(&c->d_leaf_sums), sizeof(long long) * 2 * L) == cudaSuccess &&
              cudaMalloc(reinterpret_cast<void **>(&c->d_leaf_table), sizeof(uint32_t) * 2 * L) == cudaSuccess &&
              cudaMalloc(reinterpret_cast<void **>(&c->d_leaf_value), sizeof(float) * L) == cudaSuccess &&
              cudaMalloc(reinterpret_cast<void **>(&c->d_leaf_w), sizeof(double) * L) == cudaSuccess &&
              cudaMallocHost(&c->h_pinned, PINNED_BYTES) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        qgbdt_destroy(c);
        return QGBDT_ERR_ALLOC;
    }
    *out = c;
    return QGBDT_OK;
}

int qgbdt_destroy(qgbdt_ctx *c) {
    if (!c) return QGBDT_ERR_ARG;
    free_data(c);
    dev_free(c->d_state);
    dev_free(c->d_gs);
    dev_free(c->d_split_out);
    dev_free(c->d_leaf_sums);
    dev_free(c->d_leaf_table);
    dev_free(c->d_leaf_value);
    dev_free(c->d_leaf_w);
    if (c->h_pinned) cudaFreeHost(c->h_pinned);
    for (cudaEvent_t e : c->hist_events) cudaEventDestroy(e);
    delete c;
    return QGBDT_OK;
}

const char *qgbdt_last_error(const qgbdt_ctx *c) { return c ? c->err : "null context"; }

int qgbdt_load_binned(qgbdt_ctx *c, const uint8_t *d_bins, int64_t n_rows, int32_t n_features, int32_t n_bins,
                      int32_t layout, int64_t ld, void *stream) {
    int rc = check_load_args(c, d_bins, n_rows, n_features, n_bins, layout, ld);
    if (rc != QGBDT_OK) return rc;
    return load_common(c, d_bins, n_rows, n_features, n_bins, layout, ld, (cudaStream_t)stream);
}

int qgbdt_load_binned_host(qgbdt_ctx *c, const uint8_t *h_bins, int64_t n_rows, int32_t n_features, int32_t n_bins,
                           int32_t layout, int64_t ld, void *stream) {
    int rc = check_load_args(c, h_bins, n_rows, n_features, n_bins, layout, ld);
    if (rc != QGBDT_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t bytes = (size_t)ld * (size_t)(layout == 0 ? n_rows : n_features);
    uint8_t *tmp = nullptr;
    if ((rc = dev_alloc(c, &tmp, bytes)) != QGBDT_OK) return rc;
    cudaError_t e = cudaMemcpyAsync(tmp, h_bins, bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) {
        cudaFree(tmp);
        return qg_fail(c, QGBDT_ERR_CUDA, "copy of the bin matrix failed: %s", cudaGetErrorString(e));
    }
    rc = load_common(c, tmp, n_rows, n_features, n_bins, layout, ld, st);
    cudaStreamSynchronize(st);
    cudaFree(tmp);
    return rc;
}

int qgbdt_compute_gradients(qgbdt_ctx *c, const float *d_scores, const float *d_labels, float *d_g, float *d_h,
                            void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!d_scores || !d_labels || !d_g || (c->prm.objective == 0 && !d_h))
        return qg_fail(c, QGBDT_ERR_ARG, "null pointer");
    return qg_gradients(c, d_scores, d_labels, d_g, d_h, false, false, (cudaStream_t)stream);
}

int qgbdt_quantize_gradients(qgbdt_ctx *c, const float *d_g, const float *d_h, uint32_t tree, int8_t *d_gq,
                             uint8_t *d_hq, double *g_scale, double *h_scale, int64_t *G_total, int64_t *H_total,
                             void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!d_g) return qg_fail(c, QGBDT_ERR_ARG, "d_g is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    c->quantized = false;
    c->const_hess = d_h == nullptr;
    if ((rc = qg_absmax(c, d_g, d_h, st)) != QGBDT_OK) return rc;
    // sharded rows: the maxima (and the bad-value flag) and the totals are those of all ranks
    if ((rc = qg_allreduce(c, &c->d_state->gmax_bits, 3, QGBDT_REDUCE_MAX_U32, st)) != QGBDT_OK) return rc;
    if ((rc = qg_quantize(c, d_g, d_h, tree, d_gq, d_hq, st)) != QGBDT_OK) return rc;
    if ((rc = qg_allreduce(c, &c->d_state->tot_g, 2, QGBDT_REDUCE_SUM_I64, st)) != QGBDT_OK) return rc;
    DevState *hs = reinterpret_cast<DevState *>(reinterpret_cast<char *>(c->h_pinned) + PINNED_SCALARS);
    QG_CUDA(c, cudaMemcpyAsync(hs, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    if (hs->bad_value)
        return qg_fail(c, QGBDT_ERR_VALUE, "gradient or hessian out of domain (non-finite, h < 0, or magnitude >= 256)");
    memcpy(&c->gmax, &hs->gmax_bits, 4);
    memcpy(&c->hmax, &hs->hmax_bits, 4);
    if (c->const_hess) c->hmax = 1.0f;
    c->quantized = true;
    const int kg = qg_levels_g(c->prm.bits), kh = qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    if (g_scale) *g_scale = (double)c->gmax / (double)kg;
    if (h_scale) *h_scale = c->const_hess ? 1.0 : (double)c->hmax / (double)kh;
    if (G_total) *G_total = hs->tot_g;
    if (H_total) *H_total = hs->tot_h;
    return QGBDT_OK;
}

int qgbdt_build_histograms(qgbdt_ctx *c, int32_t leaf, qgbdt_bin *d_hist, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!c->quantized) return qg_fail(c, QGBDT_ERR_STATE, "quantize gradients before building histograms");
    if (!d_hist) return qg_fail(c, QGBDT_ERR_ARG, "d_hist is NULL");
    if (leaf < 0 || leaf >= c->n_leaves) return qg_fail(c, QGBDT_ERR_ARG, "leaf %d does not exist", leaf);
    const bool root = c->n_leaves == 1 && c->idx_is_identity;
    return qg_hist(c, root ? nullptr : c->d_idx, c->leaf_off[leaf], c->leaf_n[leaf],
                   reinterpret_cast<unsigned long long *>(d_hist), (cudaStream_t)stream);
}

int qgbdt_build_histograms_rows(qgbdt_ctx *c, const uint32_t *d_rows, int64_t n, qgbdt_bin *d_hist, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!c->quantized) return qg_fail(c, QGBDT_ERR_STATE, "quantize gradients before building histograms");
    if (!d_hist || (n > 0 && !d_rows) || n < 0 || n >= (1ll << 32)) return qg_fail(c, QGBDT_ERR_ARG, "bad argument");
    // a list may repeat rows, so its length, not n_rows, bounds the sums of a bin
    const int64_t kg = qg_levels_g(c->prm.bits), kh = c->const_hess ? 1 : qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    if (n * kg > 2147483647ll || n * kh > 4294967295ll)
        return qg_fail(c, QGBDT_ERR_OVERFLOW, "a list of %lld rows could exceed the 32+32-bit histogram word", (long long)n);
    return qg_hist(c, d_rows, 0, n, reinterpret_cast<unsigned long long *>(d_hist), (cudaStream_t)stream);
}

int qgbdt_build_histograms_fp32(qgbdt_ctx *c, const float *d_g, const float *d_h, const uint32_t *d_rows, int64_t n,
                                float *d_hist, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!d_g || !d_hist || n < 0 || n >= (1ll << 32) || (!d_rows && n != c->N))
        return qg_fail(c, QGBDT_ERR_ARG, "bad argument (without a row list n must be n_rows)");
    return qg_hist_fp32(c, d_g, d_h, d_rows, n, d_hist, (cudaStream_t)stream);
}

int qgbdt_subtract_histograms(qgbdt_ctx *c, const qgbdt_bin *d_parent, const qgbdt_bin *d_small, qgbdt_bin *d_large,
                              void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!d_parent || !d_small || !d_large) return qg_fail(c, QGBDT_ERR_ARG, "null pointer");
    return qg_subtract(c, reinterpret_cast<const unsigned long long *>(d_parent),
                       reinterpret_cast<const unsigned long long *>(d_small),
                       reinterpret_cast<unsigned long long *>(d_large), (cudaStream_t)stream);
}

int qgbdt_find_best_split(qgbdt_ctx *c, const qgbdt_bin *d_hist, int64_t G, int64_t H, int64_t n_rows,
                          qgbdt_split *h_out, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!c->quantized) return qg_fail(c, QGBDT_ERR_STATE, "quantize gradients before searching splits");
    if (!d_hist || !h_out || n_rows < 0 || H < 0) return qg_fail(c, QGBDT_ERR_ARG, "bad argument");
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = qg_find_split(c, reinterpret_cast<const unsigned long long *>(d_hist), G, H, n_rows, c->d_split_out,
                            st)) != QGBDT_OK)
        return rc;
    SplitRec *hr = reinterpret_cast<SplitRec *>(reinterpret_cast<char *>(c->h_pinned) + PINNED_SCALARS + 256);
    QG_CUDA(c, cudaMemcpyAsync(hr, c->d_split_out, sizeof(SplitRec), cudaMemcpyDeviceToHost, st));
    DevState *hs = reinterpret_cast<DevState *>(reinterpret_cast<char *>(c->h_pinned) + PINNED_SCALARS);
    QG_CUDA(c, cudaMemcpyAsync(hs, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    // a histogram kernel that refused to run (earlier on this stream) left d_hist unwritten
    if (hs->kernel_error) return qg_fail(c, QGBDT_ERR_CUDA, "a histogram kernel refused its launch configuration");
    rec_to_split(*hr, G, H, n_rows, c->const_hess, h_out);
    return QGBDT_OK;
}

int qgbdt_split_leaf(qgbdt_ctx *c, int32_t leaf, int32_t feature, int32_t bin, int32_t *right_leaf, int64_t *n_left,
                     int64_t *n_right, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (leaf < 0 || leaf >= c->n_leaves) return qg_fail(c, QGBDT_ERR_ARG, "leaf %d does not exist", leaf);
    if (c->n_leaves >= c->prm.num_leaves) return qg_fail(c, QGBDT_ERR_STATE, "the tree already has num_leaves leaves");
    if (feature < 0 || feature >= c->F || bin < 0 || bin >= c->nb) return qg_fail(c, QGBDT_ERR_ARG, "bad (feature, bin)");
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t off = c->leaf_off[leaf], n = c->leaf_n[leaf];
    int64_t nl = 0;
    if (n > 0) {
        if ((rc = qg_partition(c, off, n, feature, bin, st)) != QGBDT_OK) return rc;
        DevState *hs = reinterpret_cast<DevState *>(reinterpret_cast<char *>(c->h_pinned) + PINNED_SCALARS);
        QG_CUDA(c, cudaMemcpyAsync(hs, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, st));
        QG_CUDA(c, cudaStreamSynchronize(st));
        if (hs->kernel_error) return qg_fail(c, QGBDT_ERR_CUDA, "a histogram kernel refused its launch configuration");
        nl = hs->part_nl;
    }
    const int r = c->n_leaves++;
    c->refit_leaves = 0;
    c->leaf_n[leaf] = nl;
    c->leaf_off[r] = off + nl;
    c->leaf_n[r] = n - nl;
    if (right_leaf) *right_leaf = r;
    if (n_left) *n_left = nl;
    if (n_right) *n_right = n - nl;
    return QGBDT_OK;
}

int qgbdt_get_leaf_rows(qgbdt_ctx *c, int32_t leaf, const uint32_t **d_rows, int64_t *n) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (leaf < 0 || leaf >= c->n_leaves || !d_rows || !n) return qg_fail(c, QGBDT_ERR_ARG, "bad argument");
    *d_rows = c->d_idx + c->leaf_off[leaf];
    *n = c->leaf_n[leaf];
    return QGBDT_OK;
}

int qgbdt_reset_leaves(qgbdt_ctx *c, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    reset_leaf_state(c);
    return qg_iota(c, (cudaStream_t)stream);
}

int qgbdt_refit_leaves(qgbdt_ctx *c, const float *d_g, const float *d_h, double *h_w, float *h_value, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!d_g) return qg_fail(c, QGBDT_ERR_ARG, "d_g is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = qg_refit(c, d_g, d_h, st)) != QGBDT_OK) return rc;
    const int L = c->n_leaves;
    char *base = reinterpret_cast<char *>(c->h_pinned) + PINNED_SCALARS + 1024;
    double *hw = reinterpret_cast<double *>(base);
    float *hv = reinterpret_cast<float *>(base + sizeof(double) * MAX_LEAVES);
    QG_CUDA(c, cudaMemcpyAsync(hw, c->d_leaf_w, sizeof(double) * L, cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaMemcpyAsync(hv, c->d_leaf_value, sizeof(float) * L, cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    if (h_w) memcpy(h_w, hw, sizeof(double) * L);
    if (h_value) memcpy(h_value, hv, sizeof(float) * L);
    c->refit_leaves = L;
    return QGBDT_OK;
}

int qgbdt_apply_leaf_values(qgbdt_ctx *c, float *d_scores, void *stream) {
    int rc = check_loaded(c);
    if (rc != QGBDT_OK) return rc;
    if (!d_scores) return qg_fail(c, QGBDT_ERR_ARG, "d_scores is NULL");
    if (c->refit_leaves != c->n_leaves) return qg_fail(c, QGBDT_ERR_STATE, "refit the current leaves first");
    return qg_apply_leaf_values(c, d_scores, (cudaStream_t)stream);
}

int qgbdt_set_distributed(qgbdt_ctx *c, int32_t rank, int32_t world, int64_t row_offset, int64_t total_rows,
                          qgbdt_allreduce_fn reduce, void *user) {
    if (!c) return QGBDT_ERR_ARG;
    if (world <= 1 || !reduce) {
        c->dist_rank = 0; c->dist_world = 1; c->row_offset = 0; c->total_rows = 0;
        c->dist_reduce = nullptr; c->dist_user = nullptr;
        return QGBDT_OK;
    }
    if (rank < 0 || rank >= world || row_offset < 0 || total_rows < 1 || total_rows >= (1ll << 32) ||
        (c->loaded && row_offset + c->N > total_rows))
        return qg_fail(c, QGBDT_ERR_ARG, "rank, row_offset or total_rows out of range");
    const int64_t kg = qg_levels_g(c->prm.bits), kh = qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    if (total_rows * kg > 2147483647ll || total_rows * kh > 4294967295ll)
        return qg_fail(c, QGBDT_ERR_OVERFLOW, "total_rows * levels exceeds the 32+32-bit histogram word");
    c->dist_rank = rank; c->dist_world = world; c->row_offset = row_offset; c->total_rows = total_rows;
    c->dist_reduce = reduce; c->dist_user = user;
    return QGBDT_OK;
}

int qgbdt_set_option(qgbdt_ctx *c, int32_t option, int64_t value) {
    if (!c) return QGBDT_ERR_ARG;
    switch (option) {
        case QGBDT_OPT_COLUMN_COPY:
            if (value != 0 && value != 1) return qg_fail(c, QGBDT_ERR_ARG, "QGBDT_OPT_COLUMN_COPY takes 0 or 1");
            c->want_column_copy = value != 0;
            return QGBDT_OK;
        case QGBDT_OPT_LEAF_VALUES:
            if (value != 0 && value != 1) return qg_fail(c, QGBDT_ERR_ARG, "QGBDT_OPT_LEAF_VALUES takes 0 or 1");
            c->leaf_values_quantized = value != 0;
            return QGBDT_OK;
        default:
            return qg_fail(c, QGBDT_ERR_ARG, "unknown option %d", option);
    }
}

int qgbdt_get_info(const qgbdt_ctx *c, int32_t what, int64_t *value) {
    if (!c || !value) return QGBDT_ERR_ARG;
    switch (what) {
        case QGBDT_INFO_COLUMN_COPY:
            *value = c->d_colmajor != nullptr ? 1 : 0;
            return QGBDT_OK;
        default:
            return QGBDT_ERR_ARG;
    }
}

int qgbdt_get_counters(const qgbdt_ctx *c, int64_t *kernel_launches, int64_t *hist_builds, int64_t *hist_row_features) {
    if (!c) return QGBDT_ERR_ARG;
    if (kernel_launches) *kernel_launches = c->n_launches;
    if (hist_builds) *hist_builds = c->n_hist_builds;
    if (hist_row_features) *hist_row_features = c->n_hist_row_features;
    return QGBDT_OK;
}

int qgbdt_profile_histograms(qgbdt_ctx *c, int32_t enable) {
    if (!c) return QGBDT_ERR_ARG;
    c->profile_hist = enable != 0;
    c->hist_events_used = 0;
    c->hist_prof_bytes = 0;
    c->hist_prof_launches = 0;
    return QGBDT_OK;
}

int qgbdt_get_timings(qgbdt_ctx *c, double *ms, int64_t *intervals) {
    if (!c || !ms) return QGBDT_ERR_ARG;
    for (int p = 0; p < QG_N_PHASES; ++p) {
        ms[p] = 0.0;
        if (intervals) intervals[p] = 0;
    }
    for (size_t i = 0; i + 1 < c->hist_events_used; i += 2) {
        QG_CUDA(c, cudaEventSynchronize(c->hist_events[i + 1]));
        float t = 0.f;
        QG_CUDA(c, cudaEventElapsedTime(&t, c->hist_events[i], c->hist_events[i + 1]));
        const int p = c->hist_event_phase[i / 2];
        if (p >= 0 && p < QG_N_PHASES) {
            ms[p] += t;
            if (intervals) intervals[p]++;
        }
    }
    return QGBDT_OK;
}

int qgbdt_get_histogram_profile(qgbdt_ctx *c, double *total_ms, int64_t *total_bytes, int64_t *builds) {
    if (!c) return QGBDT_ERR_ARG;
    double ms = 0.0;
    for (size_t i = 0; i + 1 < c->hist_events_used; i += 2) {
        const int p = c->hist_event_phase[i / 2];
        if (p != QG_PHASE_ROOT_HIST && p != QG_PHASE_CHILD_HIST) continue;
        QG_CUDA(c, cudaEventSynchronize(c->hist_events[i + 1]));
        float t = 0.f;
        QG_CUDA(c, cudaEventElapsedTime(&t, c->hist_events[i], c->hist_events[i + 1]));
        ms += t;
    }
    if (total_ms) *total_ms = ms;
    if (total_bytes) *total_bytes = c->hist_prof_bytes;
    if (builds) *builds = c->hist_prof_launches;
    c->hist_events_used = 0;
    c->hist_prof_bytes = 0;
    c->hist_prof_launches = 0;
    return QGBDT_OK;
}

}  // extern "C"
