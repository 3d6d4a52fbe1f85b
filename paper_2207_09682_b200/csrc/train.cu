// Fig. 1 workflow: the boosting loop with leaf-wise (best-first) tree growth (Sec. 3).
// Per iteration: gradients (Eq. 1) -> scales and stochastic rounding (Eq. 5, 6, 8) -> root
// histogram (Algorithm 1) -> repeat { take the leaf with the largest gain, partition its rows,
// build the smaller child's histogram, get the larger one by subtraction, find both children's
// best splits (Eq. 7) } -> refit leaf values from the original gradients (Eq. 3) -> add them to
// the scores.  The host only orders the kernels and compares stored gains.
#include <cstring>

#include "qgbdt_internal.cuh"

namespace {

struct HostSplit {
    SplitRec rec;
    long long G, H;  // totals of the leaf the record belongs to
};

int train_one_tree(qgbdt_ctx *c, const float *d_labels, float *d_scores, uint32_t tree, int slot,
                   qgbdt_model *model, cudaStream_t st) {
    const int L = c->prm.num_leaves;
    const size_t hist_words = (size_t)c->F * c->nb;
    const bool const_h = c->prm.objective == 1;
    int rc;
    char *scal = reinterpret_cast<char *>(c->h_pinned) + 64 * 1024;
    DevState *hs = reinterpret_cast<DevState *>(scal);
    SplitRec *hrec = reinterpret_cast<SplitRec *>(scal + 256);

    c->const_hess = const_h;
    c->quantized = false;
    if ((rc = qg_gradients(c, d_scores, d_labels, c->d_g, const_h ? nullptr : c->d_h, true, st)) != QGBDT_OK) return rc;
    if ((rc = qg_quantize(c, c->d_g, const_h ? nullptr : c->d_h, tree, nullptr, nullptr, st)) != QGBDT_OK) return rc;
    c->n_leaves = 1;
    c->leaf_off.assign(L, 0);
    c->leaf_n.assign(L, 0);
    c->leaf_n[0] = c->N;
    if (!c->idx_is_identity && (rc = qg_iota(c, st)) != QGBDT_OK) return rc;
    QG_CUDA(c, cudaMemcpyAsync(hs, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    if (hs->bad_value) return qg_fail(c, QGBDT_ERR_VALUE, "gradient or hessian out of domain in tree %u", tree);
    memcpy(&c->gmax, &hs->gmax_bits, 4);
    memcpy(&c->hmax, &hs->hmax_bits, 4);
    if (const_h) c->hmax = 1.0f;
    c->quantized = true;

    std::vector<HostSplit> best(L);
    std::vector<int> hist_slot(L, 0), parent_node(L, -1), parent_side(L, 0);
    int next_slot = 1;
    auto hist_of = [&](int s) { return c->d_hist_pool + (size_t)s * hist_words; };

    best[0].G = hs->tot_g;
    best[0].H = hs->tot_h;
    if ((rc = qg_hist(c, nullptr, 0, c->N, hist_of(0), st)) != QGBDT_OK) return rc;
    if ((rc = qg_find_split(c, hist_of(0), best[0].G, best[0].H, c->N, c->d_split_out, st)) != QGBDT_OK) return rc;
    QG_CUDA(c, cudaMemcpyAsync(hrec, c->d_split_out, sizeof(SplitRec), cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    best[0].rec = hrec[0];

    int32_t *nf = model->feature + (size_t)slot * (L - 1), *nbn = model->bin + (size_t)slot * (L - 1);
    int32_t *nl_ = model->left + (size_t)slot * (L - 1), *nr_ = model->right + (size_t)slot * (L - 1);
    double *ng = model->gain + (size_t)slot * (L - 1);

    while (c->n_leaves < L) {
        int pick = -1;
        for (int l = 0; l < c->n_leaves; ++l)
            if (best[l].rec.valid && (pick < 0 || best[l].rec.gain > best[pick].rec.gain)) pick = l;
        if (pick < 0) break;
        const SplitRec s = best[pick].rec;
        const long long PG = best[pick].G, PH = best[pick].H;
        const int64_t off = c->leaf_off[pick], n = c->leaf_n[pick];
        if ((rc = qg_partition(c, off, n, s.feature, s.bin, st)) != QGBDT_OK) return rc;
        QG_CUDA(c, cudaMemcpyAsync(hs, c->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, st));
        QG_CUDA(c, cudaStreamSynchronize(st));
        if (hs->kernel_error) return qg_fail(c, QGBDT_ERR_CUDA, "a histogram kernel refused its launch configuration");
        const int64_t nl = hs->part_nl, nr = n - nl;
        const int node = c->n_leaves - 1, right = c->n_leaves;
        nf[node] = s.feature;
        nbn[node] = s.bin;
        nl_[node] = ~pick;
        nr_[node] = ~right;
        ng[node] = s.gain;
        if (parent_node[pick] >= 0) {
            if (parent_side[pick] == 0) nl_[parent_node[pick]] = node;
            else nr_[parent_node[pick]] = node;
        }
        parent_node[pick] = node; parent_side[pick] = 0;
        parent_node[right] = node; parent_side[right] = 1;
        c->leaf_n[pick] = nl;
        c->leaf_off[right] = off + nl;
        c->leaf_n[right] = nr;
        c->n_leaves++;
        best[pick].G = s.gl; best[pick].H = s.hl;
        best[right].G = PG - s.gl; best[right].H = PH - s.hl;

        // smaller child by Algorithm 1, larger child = parent - smaller (ties: left is "smaller")
        const int small = nl <= nr ? pick : right, large = nl <= nr ? right : pick;
        const int pslot = hist_slot[pick];
        hist_slot[small] = next_slot++;
        hist_slot[large] = pslot;
        if ((rc = qg_hist(c, c->d_idx, c->leaf_off[small], c->leaf_n[small], hist_of(hist_slot[small]), st)) != QGBDT_OK)
            return rc;
        if ((rc = qg_subtract(c, hist_of(pslot), hist_of(hist_slot[small]), hist_of(pslot), st)) != QGBDT_OK) return rc;
        if ((rc = qg_find_split(c, hist_of(hist_slot[pick]), best[pick].G, best[pick].H, nl, c->d_split_out, st)) != QGBDT_OK)
            return rc;
        if ((rc = qg_find_split(c, hist_of(hist_slot[right]), best[right].G, best[right].H, nr, c->d_split_out + 1, st)) !=
            QGBDT_OK)
            return rc;
        QG_CUDA(c, cudaMemcpyAsync(hrec, c->d_split_out, 2 * sizeof(SplitRec), cudaMemcpyDeviceToHost, st));
        QG_CUDA(c, cudaStreamSynchronize(st));
        best[pick].rec = hrec[0];
        best[right].rec = hrec[1];
    }

    if ((rc = qg_refit(c, c->d_g, const_h ? nullptr : c->d_h, st)) != QGBDT_OK) return rc;
    if ((rc = qg_apply_leaf_values(c, d_scores, st)) != QGBDT_OK) return rc;
    float *hv = reinterpret_cast<float *>(scal + 1024);
    QG_CUDA(c, cudaMemcpyAsync(hv, c->d_leaf_value, sizeof(float) * c->n_leaves, cudaMemcpyDeviceToHost, st));
    QG_CUDA(c, cudaStreamSynchronize(st));
    model->num_leaves[slot] = c->n_leaves;
    for (int l = 0; l < c->n_leaves; ++l) {
        model->leaf_value[(size_t)slot * L + l] = hv[l];
        model->leaf_count[(size_t)slot * L + l] = c->leaf_n[l];
    }
    return QGBDT_OK;
}

int ensure_train_buffers(qgbdt_ctx *c) {
    if (!c->d_g) {
        void *p = nullptr;
        if (cudaMalloc(&p, sizeof(float) * (size_t)c->N) != cudaSuccess) {
            cudaGetLastError();
            return qg_fail(c, QGBDT_ERR_ALLOC, "gradient buffer allocation failed");
        }
        c->d_g = reinterpret_cast<float *>(p);
    }
    if (!c->d_h && c->prm.objective == 0) {
        void *p = nullptr;
        if (cudaMalloc(&p, sizeof(float) * (size_t)c->N) != cudaSuccess) {
            cudaGetLastError();
            return qg_fail(c, QGBDT_ERR_ALLOC, "hessian buffer allocation failed");
        }
        c->d_h = reinterpret_cast<float *>(p);
    }
    if (!c->d_hist_pool) {
        void *p = nullptr;
        const size_t bytes = (size_t)c->prm.num_leaves * c->F * c->nb * sizeof(unsigned long long);
        if (cudaMalloc(&p, bytes) != cudaSuccess) {
            cudaGetLastError();
            return qg_fail(c, QGBDT_ERR_ALLOC, "histogram pool allocation of %zu bytes failed", bytes);
        }
        c->d_hist_pool = reinterpret_cast<unsigned long long *>(p);
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
    int rc = ensure_train_buffers(c);
    if (rc != QGBDT_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    for (int k = 0; k < num_trees; ++k)
        if ((rc = train_one_tree(c, d_labels, d_scores, first_tree + (uint32_t)k, k, model, st)) != QGBDT_OK) return rc;
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
