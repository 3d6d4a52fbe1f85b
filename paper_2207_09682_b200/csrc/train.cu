// Fig. 1 workflow: the boosting loop with leaf-wise (best-first) tree growth (Sec. 3).
// Per iteration: gradients (Eq. 1) -> scales and stochastic rounding (Eq. 5, 6, 8) -> root
// histogram (Algorithm 1) -> repeat { take the leaf with the largest gain, partition its rows,
// build the smaller child's histogram, get the larger one by subtraction, find both children's
// best splits (Eq. 7) } -> refit leaf values from the original gradients (Eq. 3) -> add them to
// the scores.  The host only orders the kernels and compares stored gains.
#include <cstring>

#include "qgbdt_internal.cuh"

namespace {

// One boosting iteration, enqueued without waiting for any result.
int train_one_tree(qgbdt_ctx *c, const float *d_labels, float *d_scores, uint32_t tree, int slot, bool first,
                   cudaStream_t st) {
    const bool const_h = c->prm.objective == 1;
    int rc;
    c->const_hess = const_h;
    c->quantized = false;
    if ((rc = qg_phase_begin(c, QG_PHASE_GRADIENTS, st)) != QGBDT_OK) return rc;
    if ((rc = qg_gradients(c, d_scores, d_labels, c->d_g, const_h ? nullptr : c->d_h, true, first, st)) != QGBDT_OK)
        return rc;
    if ((rc = qg_phase_end(c, st)) != QGBDT_OK) return rc;
    // sharded rows (Sec. 7.3): Eq. 5's maxima run over all rows of all ranks (with them the flag for
    // gradients out of domain), and so do the totals of the quantized gradients
    if ((rc = qg_allreduce(c, &c->d_state->gmax_bits, 3, QGBDT_REDUCE_MAX_U32, st)) != QGBDT_OK) return rc;
    if ((rc = qg_phase_begin(c, QG_PHASE_QUANTIZE, st)) != QGBDT_OK) return rc;
    if ((rc = qg_quantize(c, c->d_g, const_h ? nullptr : c->d_h, tree, nullptr, nullptr, st)) != QGBDT_OK) return rc;
    if ((rc = qg_phase_end(c, st)) != QGBDT_OK) return rc;
    if ((rc = qg_allreduce(c, &c->d_state->tot_g, 2, QGBDT_REDUCE_SUM_I64, st)) != QGBDT_OK) return rc;
    c->quantized = true;
    if ((rc = qg_grow_tree(c, slot, st)) != QGBDT_OK) return rc;
    return qg_refit_grown(c, c->d_g, const_h ? nullptr : c->d_h, d_scores, slot, st);
}

template <typename T>
int alloc_dev(qgbdt_ctx *c, T **p, size_t count, const char *what) {
    void *q = nullptr;
    if (cudaMalloc(&q, (count ? count : 1) * sizeof(T)) != cudaSuccess) {
        cudaGetLastError();
        return qg_fail(c, QGBDT_ERR_ALLOC, "%s allocation of %zu bytes failed", what, count * sizeof(T));
    }
    *p = reinterpret_cast<T *>(q);
    return QGBDT_OK;
}

template <typename T>
void free_dev(T *&p) {
    if (p) cudaFree(p);
    p = nullptr;
}

int ensure_train_buffers(qgbdt_ctx *c, int num_trees, cudaStream_t st) {
    const int L = c->prm.num_leaves;
    int rc;
    if (!c->d_g && (rc = alloc_dev(c, &c->d_g, (size_t)c->N, "gradient buffer")) != QGBDT_OK) return rc;
    if (!c->d_h && c->prm.objective == 0 && (rc = alloc_dev(c, &c->d_h, (size_t)c->N, "hessian buffer")) != QGBDT_OK)
        return rc;
    // leaves split per pass: fewer with many thousands of features (the histogram pool has a slot of
    // F x bins words for every leaf that may be split ahead)
    if (c->grow_jobs <= 1 || !c->d_recs) {
        int k = 65536 / (c->F > 0 ? c->F : 1);
        c->grow_jobs = k < 2 ? 2 : (k > GROW_MAX_JOBS ? GROW_MAX_JOBS : k);
        // histogram CTAs per tile a pass may use: twice one leaf's share of the SMs, four times with several
        // tiles (a leaf's share is then small, and CTAs of unequal leaves fill the SMs better in more pieces:
        // 2 % per tree at 2000 features; six and eight times were slower again)
        c->grow_xcap = (c->tiles.size() > 1 ? 4 : 2) * qg_grow_parts_cap(c) + c->grow_jobs;
        int max_logw = 0;
        for (const TileDesc &t : c->tiles) max_logw = t.logW > max_logw ? t.logW : max_logw;
        // rows per histogram CTA of a pass, at least.  Rows of up to 32 bytes: every CTA of a leaf adds its
        // whole local histogram into the leaf's sums (one reduction per non-zero word), and those reductions
        // are still draining from L2 when the finishing kernel starts; 3072 rows was the best trade against
        // the parallelism of the build (1024: 3 % slower per tree on 1 M rows).  Wider rows: 1024 per 32 bytes.
        c->grow_rows_min = max_logw > 3 ? 1024 << (max_logw - 3) : 3072;
        c->grow_bits_stride = ((size_t)c->N + 31) / 32 + 64;
    }
    if (!c->d_hist_pool &&
        (rc = alloc_dev(c, &c->d_hist_pool, (size_t)qg_grow_max_slots(c) * c->F * c->nb, "histogram pool")) != QGBDT_OK)
        return rc;
    if (!c->d_leaves && (rc = alloc_dev(c, &c->d_leaves, (size_t)L, "leaf records")) != QGBDT_OK) return rc;
    if (!c->d_recs && (rc = alloc_dev(c, &c->d_recs, (size_t)qg_grow_max_recs(c), "growth records")) != QGBDT_OK) return rc;
    if (!c->d_rec_gain && (rc = alloc_dev(c, &c->d_rec_gain, (size_t)qg_grow_max_recs(c), "growth records")) != QGBDT_OK) return rc;
    if (!c->d_rec_child && (rc = alloc_dev(c, &c->d_rec_child, (size_t)qg_grow_max_recs(c), "growth records")) != QGBDT_OK) return rc;
    if (!c->d_rec_pos && (rc = alloc_dev(c, &c->d_rec_pos, (size_t)qg_grow_max_recs(c), "growth records")) != QGBDT_OK) return rc;
    if (!c->d_rec_parent && (rc = alloc_dev(c, &c->d_rec_parent, (size_t)qg_grow_max_recs(c), "growth records")) != QGBDT_OK) return rc;
    if (!c->d_front && (rc = alloc_dev(c, &c->d_front, (size_t)L, "leaf table")) != QGBDT_OK) return rc;
    if (!c->d_grow_bits &&
        (rc = alloc_dev(c, &c->d_grow_bits, c->grow_bits_stride * (size_t)c->grow_jobs, "partition bits")) != QGBDT_OK)
        return rc;
    if (!c->d_grow_partial &&
        (rc = alloc_dev(c, &c->d_grow_partial, (size_t)c->grow_xcap * c->tiles.size() * 4 * c->nb * 32,
                        "partial histograms of tree growth")) != QGBDT_OK)
        return rc;
    // the CTAs of a histogram build add into these sums and whoever reads them clears them: every call
    // starts from zero, whatever state an earlier call that ended in an error left
    bool shared_slots = false;
    for (const auto &t : c->tiles) shared_slots = shared_slots || t.logW < QG_SHARED_PARTIAL_LOGW;
    if (shared_slots)
        QG_CUDA(c, cudaMemsetAsync(c->d_grow_partial, 0,
                                   (size_t)c->grow_xcap * c->tiles.size() * 4 * c->nb * 32 * sizeof(unsigned long long), st));
    if (!c->d_grow_prep && (rc = alloc_dev(c, &c->d_grow_prep, (size_t)GROW_MAX_JOBS, "per-leaf constants")) != QGBDT_OK) return rc;
    if (!c->d_ent0 && (rc = alloc_dev(c, &c->d_ent0, (size_t)c->N, "row/code pairs")) != QGBDT_OK) return rc;
    if (!c->d_ent1 && (rc = alloc_dev(c, &c->d_ent1, (size_t)c->N, "row/code pairs")) != QGBDT_OK) return rc;
    if (!c->d_leaf_id && (rc = alloc_dev(c, &c->d_leaf_id, (size_t)c->N, "leaf numbers")) != QGBDT_OK) return rc;
    if (!c->d_cand && (rc = alloc_dev(c, &c->d_cand, (size_t)2 * c->F * c->grow_jobs, "candidate records")) != QGBDT_OK)
        return rc;
    if ((rc = qg_build_columns(c, st)) != QGBDT_OK) return rc;
    if (!c->d_gs) {
        if ((rc = alloc_dev(c, &c->d_gs, 1, "grow state")) != QGBDT_OK) return rc;
        QG_CUDA(c, cudaMemsetAsync(c->d_gs, 0, sizeof(GrowState), st));
    }
    if (num_trees > c->model_cap) {
        qg_grow_graph_destroy(c);   // the captured launches hold the old array addresses
        free_dev(c->d_m_num_leaves); free_dev(c->d_m_feature); free_dev(c->d_m_bin); free_dev(c->d_m_left);
        free_dev(c->d_m_right); free_dev(c->d_m_gain); free_dev(c->d_m_leaf_value); free_dev(c->d_m_leaf_count);
        c->model_cap = 0;
        const size_t nn = (size_t)num_trees * (L > 1 ? L - 1 : 1), nl = (size_t)num_trees * L;
        if ((rc = alloc_dev(c, &c->d_m_num_leaves, (size_t)num_trees, "model")) != QGBDT_OK ||
            (rc = alloc_dev(c, &c->d_m_feature, nn, "model")) != QGBDT_OK ||
            (rc = alloc_dev(c, &c->d_m_bin, nn, "model")) != QGBDT_OK ||
            (rc = alloc_dev(c, &c->d_m_left, nn, "model")) != QGBDT_OK ||
            (rc = alloc_dev(c, &c->d_m_right, nn, "model")) != QGBDT_OK ||
            (rc = alloc_dev(c, &c->d_m_gain, nn, "model")) != QGBDT_OK ||
            (rc = alloc_dev(c, &c->d_m_leaf_value, nl, "model")) != QGBDT_OK ||
            (rc = alloc_dev(c, &c->d_m_leaf_count, nl, "model")) != QGBDT_OK)
            return rc;
        c->model_cap = num_trees;
    }
    return QGBDT_OK;
}

bool model_ok(const qgbdt_model *m) {
    return m && m->num_leaves && m->feature && m->bin && m->left && m->right && m->gain && m->leaf_value &&
           m->leaf_count;
}

}  // namespace

extern "C" {

int qgbdt_train(qgbdt_ctx *c, const float *d_labels, float *d_scores, uint32_t first_tree, int32_t num_trees,
                qgbdt_model *model, void *stream) {
    if (!c) return QGBDT_ERR_ARG;
    if (!c->loaded) return qg_fail(c, QGBDT_ERR_STATE, "no bin matrix loaded");
    if (!d_labels || !d_scores || num_trees < 0 || !model_ok(model)) return qg_fail(c, QGBDT_ERR_ARG, "bad argument");
    if (num_trees == 0) return QGBDT_OK;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = ensure_train_buffers(c, num_trees, st);
    if (rc != QGBDT_OK) return rc;
    const int L = c->prm.num_leaves;
    char *scal = reinterpret_cast<char *>(c->h_pinned) + 64 * 1024;
    DevState *hs = reinterpret_cast<DevState *>(scal);
    GrowState *hg = reinterpret_cast<GrowState *>(scal + 256);
    GrowState before;
    QG_CUDA(c, cudaMemcpyAsync(hg, c->d_gs, sizeof(GrowState), cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    before = *hg;
    for (int k = 0; k < num_trees; ++k) {
        if ((rc = train_one_tree(c, d_labels, d_scores, first_tree + (uint32_t)k, k, k == 0, st)) != QGBDT_OK) return rc;
    }
    // the trees, the flags and the counters come back once, after the last tree
    const size_t nn = (size_t)num_trees * (L > 1 ? L - 1 : 1), nl = (size_t)num_trees * L;
    QG_CUDA(c, cudaMemcpyAsync(model->num_leaves, c->d_m_num_leaves, sizeof(int32_t) * num_trees, cudaMemcpyDeviceToHost, st));
    if (L > 1) {
        QG_CUDA(c, cudaMemcpyAsync(model->feature, c->d_m_feature, sizeof(int32_t) * nn, cudaMemcpyDeviceToHost, st));
        QG_CUDA(c, cudaMemcpyAsync(model->bin, c->d_m_bin, sizeof(int32_t) * nn, cudaMemcpyDeviceToHost, st));
        QG_CUDA(c, cudaMemcpyAsync(model->left, c->d_m_left, sizeof(int32_t) * nn, cudaMemcpyDeviceToHost, st));
        QG_CUDA(c, cudaMemcpyAsync(model->right, c->d_m_right, sizeof(int32_t) * nn, cudaMemcpyDeviceToHost, st));
        QG_CUDA(c, cudaMemcpyAsync(model->gain, c->d_m_gain, sizeof(double) * nn, cudaMemcpyDeviceToHost, st));
    }
    QG_CUDA(c, cudaMemcpyAsync(model->leaf_value, c->d_m_leaf_value, sizeof(float) * nl, cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaMemcpyAsync(model->leaf_count, c->d_m_leaf_count, sizeof(long long) * nl, cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaMemcpyAsync(hs, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaMemcpyAsync(hg, c->d_gs, sizeof(GrowState), cudaMemcpyDeviceToHost, st));
    // leave the step-wise interface in a defined state: one root leaf, rows ascending
    c->n_leaves = 1;
    c->refit_leaves = 0;
    c->leaf_off.assign(L, 0);
    c->leaf_n.assign(L, 0);
    c->leaf_n[0] = c->N;
    if ((rc = qg_iota(c, st)) != QGBDT_OK) return rc;
    QG_CUDA(c, cudaStreamSynchronize(st));
    if (!c->profile_hist) {
        // launches replayed from the growth graphs: per tree the first commit, then the passes
        int64_t passes = (int64_t)(hg->passes - before.passes) - num_trees;
        if (passes < 0) passes = 0;
        c->n_launches += num_trees + passes * c->grow_pass_launches;
    }
    c->n_passes += (int64_t)(hg->passes - before.passes);
    c->n_extra_builds += (int64_t)(hg->extra_builds - before.extra_builds);
    c->n_hist_builds += (int64_t)(hg->hist_builds - before.hist_builds);
    c->n_hist_row_features += (int64_t)(hg->hist_rows - before.hist_rows) * c->F;
    c->hist_prof_bytes += (int64_t)(hg->hist_rows - before.hist_rows) * (c->F + c->code_bytes + 4) +
                          (int64_t)(hg->hist_builds - before.hist_builds) * c->F * c->nb * 8;
    c->hist_prof_launches += (int64_t)(hg->hist_builds - before.hist_builds);
    memcpy(&c->gmax, &hs->gmax_bits, 4);
    memcpy(&c->hmax, &hs->hmax_bits, 4);
    if (c->prm.objective == 1) c->hmax = 1.0f;
    if (hs->kernel_error) return qg_fail(c, QGBDT_ERR_CUDA, "a histogram kernel refused its launch configuration");
    if (hs->bad_value)
        return qg_fail(c, QGBDT_ERR_VALUE, "gradient or hessian out of domain during trees %u .. %u", first_tree,
                       first_tree + (uint32_t)num_trees - 1);
    return QGBDT_OK;
}

int qgbdt_train_host(qgbdt_ctx *c, const float *h_labels, float *h_scores, uint32_t first_tree, int32_t num_trees,
                     qgbdt_model *model, void *stream) {
    if (!c) return QGBDT_ERR_ARG;
    if (!c->loaded) return qg_fail(c, QGBDT_ERR_STATE, "no bin matrix loaded");
    if (!h_labels || !h_scores) return qg_fail(c, QGBDT_ERR_ARG, "null pointer");
    cudaStream_t st = (cudaStream_t)stream;
    float *d_labels = nullptr, *d_scores = nullptr;
    const size_t bytes = sizeof(float) * (size_t)c->N;
    if (cudaMalloc(reinterpret_cast<void **>(&d_labels), bytes) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void **>(&d_scores), bytes) != cudaSuccess) {
        cudaGetLastError();
        if (d_labels) cudaFree(d_labels);
        return qg_fail(c, QGBDT_ERR_ALLOC, "label / score buffer allocation failed");
    }
    int rc = QGBDT_OK;
    if (cudaMemcpyAsync(d_labels, h_labels, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(d_scores, h_scores, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
        rc = qg_fail(c, QGBDT_ERR_CUDA, "copy to the device failed");
    if (rc == QGBDT_OK) rc = qgbdt_train(c, d_labels, d_scores, first_tree, num_trees, model, st);
    if (rc == QGBDT_OK && (cudaMemcpyAsync(h_scores, d_scores, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
                           cudaStreamSynchronize(st) != cudaSuccess))
        rc = qg_fail(c, QGBDT_ERR_CUDA, "copy to the host failed");
    cudaStreamSynchronize(st);
    cudaFree(d_labels);
    cudaFree(d_scores);
    return rc;
}

}  // extern "C"
