// Eq. 7: best split of a leaf from its integer histogram.  One warp scans one feature
// (prefix sums over bins by warp shuffles), gains in double precision with every operation
// individually rounded; a second kernel takes the best feature.  Ties: lowest feature,
// then lowest bin.
#include "split_scan.cuh"

namespace {

constexpr int SCAN_WARPS = 8;

__global__ void __launch_bounds__(SCAN_WARPS * 32) k_split_scan(const unsigned long long *__restrict__ hist, int F,
                                                                int nb, SplitParams p, const DevState *state,
                                                                SplitRec *__restrict__ feat_best) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int f = blockIdx.x * SCAN_WARPS + warp;
    if (f >= F) return;
    double dg, dh;
    qg_scales(state, p, dg, dh);
    const double tp = qg_gain_term(p.G, p.H, dg, dh, p.lambda);
    ScanState s;
    qg_scan_init(s);
    for (int base = 0; base < nb - 1; base += 32) {
        const int t = base + lane;
        const unsigned long long v = t < nb - 1 ? hist[(size_t)f * nb + t] : 0ull;
        qg_scan_step(s, v, t, nb, p, dg, dh, tp);
    }
    const SplitRec r = qg_scan_finish(s, f);
    if (lane == 0) feat_best[f] = r;
}

__global__ void __launch_bounds__(256) k_split_reduce(const SplitRec *__restrict__ feat_best, int F,
                                                      SplitRec *__restrict__ out) {
    __shared__ SplitRec sm[256];
    SplitRec b = qg_invalid_rec();
    for (int f = threadIdx.x; f < F; f += 256) {
        const SplitRec r = feat_best[f];
        if (qg_rec_better(r, b)) b = r;
    }
    sm[threadIdx.x] = b;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (threadIdx.x < s) {
            const SplitRec o = sm[threadIdx.x + s];
            SplitRec &m = sm[threadIdx.x];
            if (qg_rec_better(o, m)) m = o;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = sm[0];
}

}  // namespace

int qg_find_split(qgbdt_ctx *c, const unsigned long long *d_hist, long long G, long long H, long long n_rows,
                  SplitRec *d_out, cudaStream_t st) {
    SplitParams p;
    p.G = G; p.H = H; p.n_s = n_rows;
    p.kg = qg_levels_g(c->prm.bits);
    p.kh = qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    p.const_h = c->const_hess ? 1 : 0;
    p.min_data = c->prm.min_data_in_leaf;
    p.min_sum_h = c->prm.min_sum_hessian;
    p.min_gain = c->prm.min_gain;
    p.lambda = c->prm.lambda_l2;
    const unsigned grid = (unsigned)((c->F + SCAN_WARPS - 1) / SCAN_WARPS);
    k_split_scan<<<grid, SCAN_WARPS * 32, 0, st>>>(d_hist, c->F, c->nb, p, c->d_state, c->d_feat_best);
    QG_LAUNCH_CHECK(c);
    k_split_reduce<<<1, 256, 0, st>>>(c->d_feat_best, c->F, d_out);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}
