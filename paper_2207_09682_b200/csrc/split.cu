// Eq. 7: best split of a leaf from its integer histogram.  One warp scans one feature
// (prefix sums over bins by warp shuffles), gains in double precision with every operation
// individually rounded; a second kernel takes the best feature.  Ties: lowest feature,
// then lowest bin.
#include "qgbdt_internal.cuh"

namespace {

struct SplitParams {
    long long G, H, n_s;
    int kg, kh, const_h, min_data;
    double min_sum_h, min_gain, lambda;
};

__device__ inline double gain_term(long long G, long long H, double dg, double dh, double lambda) {
    const double gd = __dmul_rn((double)G, dg);
    const double hd = __dadd_rn(__dmul_rn((double)H, dh), lambda);
    return __ddiv_rn(__dmul_rn(gd, gd), hd);
}

// a strictly better than b?  (gain first; equal gains: the lower position wins)
__device__ inline bool better(bool av, double ag, int apos, bool bv, double bg, int bpos) {
    if (!av) return false;
    if (!bv) return true;
    if (ag > bg) return true;
    if (ag < bg) return false;
    return apos < bpos;
}

constexpr int SCAN_WARPS = 8;

__global__ void __launch_bounds__(SCAN_WARPS * 32) k_split_scan(const unsigned long long *__restrict__ hist, int F,
                                                                int nb, SplitParams p, const DevState *state,
                                                                SplitRec *__restrict__ feat_best) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int f = blockIdx.x * SCAN_WARPS + warp;
    if (f >= F) return;
    const double dg = __ddiv_rn((double)__uint_as_float(state->gmax_bits), (double)p.kg);
    const double dh = p.const_h ? 1.0 : __ddiv_rn((double)__uint_as_float(state->hmax_bits), (double)p.kh);
    const double tp = gain_term(p.G, p.H, dg, dh, p.lambda);

    long long carry_g = 0, carry_h = 0;
    bool bv = false;
    double bgain = 0.0;
    int bbin = -1;
    long long bgl = 0, bhl = 0;
    for (int base = 0; base < nb - 1; base += 32) {
        const int t = base + lane;
        long long g = 0, h = 0;
        if (t < nb - 1) {
            const unsigned long long v = hist[(size_t)f * nb + t];
            g = (long long)(int)(v >> 32);
            h = (long long)(unsigned int)(v & 0xFFFFFFFFull);
        }
        for (int o = 1; o < 32; o <<= 1) {
            const long long ug = __shfl_up_sync(0xffffffffu, g, o);
            const long long uh = __shfl_up_sync(0xffffffffu, h, o);
            if (lane >= o) { g += ug; h += uh; }
        }
        const long long gl = carry_g + g, hl = carry_h + h;
        carry_g += __shfl_sync(0xffffffffu, g, 31);
        carry_h += __shfl_sync(0xffffffffu, h, 31);
        if (t < nb - 1) {
            const long long gr = p.G - gl, hr = p.H - hl;
            if (hl > 0 && hr > 0) {
                long long nl;
                if (p.const_h) nl = hl;
                else nl = (long long)(((unsigned long long)hl * (unsigned long long)p.n_s +
                                       (unsigned long long)(p.H / 2)) / (unsigned long long)p.H);
                const long long nr = p.n_s - nl;
                if (nl >= p.min_data && nr >= p.min_data &&
                    !(__dmul_rn((double)hl, dh) < p.min_sum_h) && !(__dmul_rn((double)hr, dh) < p.min_sum_h)) {
                    const double tl = gain_term(gl, hl, dg, dh, p.lambda);
                    const double tr = gain_term(gr, hr, dg, dh, p.lambda);
                    const double gain = __dmul_rn(0.5, __dsub_rn(__dadd_rn(tl, tr), tp));
                    if (gain > p.min_gain && (!bv || gain > bgain)) {
                        bv = true; bgain = gain; bbin = t; bgl = gl; bhl = hl;
                    }
                }
            }
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const bool ov = __shfl_xor_sync(0xffffffffu, (int)bv, o) != 0;
        const double og = __shfl_xor_sync(0xffffffffu, bgain, o);
        const int ob = __shfl_xor_sync(0xffffffffu, bbin, o);
        const long long ogl = __shfl_xor_sync(0xffffffffu, bgl, o);
        const long long ohl = __shfl_xor_sync(0xffffffffu, bhl, o);
        if (better(ov, og, ob, bv, bgain, bbin)) { bv = ov; bgain = og; bbin = ob; bgl = ogl; bhl = ohl; }
    }
    if (lane == 0) {
        SplitRec r;
        r.gain = bgain; r.gl = bgl; r.hl = bhl; r.feature = f; r.bin = bbin; r.valid = bv ? 1 : 0; r.pad = 0;
        feat_best[f] = r;
    }
}

__global__ void __launch_bounds__(256) k_split_reduce(const SplitRec *__restrict__ feat_best, int F,
                                                      SplitRec *__restrict__ out) {
    __shared__ SplitRec sm[256];
    SplitRec b;
    b.valid = 0; b.gain = 0.0; b.feature = -1; b.bin = -1; b.gl = 0; b.hl = 0; b.pad = 0;
    for (int f = threadIdx.x; f < F; f += 256) {
        const SplitRec r = feat_best[f];
        if (better(r.valid != 0, r.gain, r.feature, b.valid != 0, b.gain, b.feature)) b = r;
    }
    sm[threadIdx.x] = b;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (threadIdx.x < s) {
            const SplitRec o = sm[threadIdx.x + s];
            SplitRec &m = sm[threadIdx.x];
            if (better(o.valid != 0, o.gain, o.feature, m.valid != 0, m.gain, m.feature)) m = o;
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
