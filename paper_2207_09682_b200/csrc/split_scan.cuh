// Eq. 7 evaluated by one warp over the bins of one feature: shared by the stand-alone split
// search and by the tree-growing kernels.  Gains are double precision with every operation
// individually rounded; ties go to the lowest bin (and, between features, the lowest feature).
#pragma once

#include "qgbdt_internal.cuh"

struct SplitParams {
    long long G, H, n_s;   // integer totals and row count of the leaf
    int kg, kh, const_h, min_data;
    double min_sum_h, min_gain, lambda;
};

__device__ inline double qg_gain_term(long long G, long long H, double dg, double dh, double lambda) {
    const double gd = __dmul_rn((double)G, dg);
    const double hd = __dadd_rn(__dmul_rn((double)H, dh), lambda);
    return __ddiv_rn(__dmul_rn(gd, gd), hd);
}

// a strictly better than b?  (gain first; equal gains: the lower position wins)
__device__ inline bool qg_better(bool av, double ag, int apos, bool bv, double bg, int bpos) {
    if (!av) return false;
    if (!bv) return true;
    if (ag > bg) return true;
    if (ag < bg) return false;
    return apos < bpos;
}

// Interval lengths of Eq. 5 from the maxima stored by the quantizer.
__device__ inline void qg_scales(const DevState *state, const SplitParams &p, double &dg, double &dh) {
    dg = __ddiv_rn((double)__uint_as_float(state->gmax_bits), (double)p.kg);
    dh = p.const_h ? 1.0 : __ddiv_rn((double)__uint_as_float(state->hmax_bits), (double)p.kh);
}

// Threshold candidate with left sums (gl, hl): admissible?  If so its gain (Eq. 7).
__device__ inline bool qg_eval_candidate(long long gl, long long hl, const SplitParams &p, double dg, double dh,
                                         double tp, double &gain) {
    const long long gr = p.G - gl, hr = p.H - hl;
    if (!(hl > 0 && hr > 0)) return false;
    long long nl;
    if (p.const_h) nl = hl;
    else nl = (long long)(((unsigned long long)hl * (unsigned long long)p.n_s + (unsigned long long)(p.H / 2)) /
                          (unsigned long long)p.H);
    const long long nr = p.n_s - nl;
    if (!(nl >= p.min_data && nr >= p.min_data)) return false;
    if (__dmul_rn((double)hl, dh) < p.min_sum_h || __dmul_rn((double)hr, dh) < p.min_sum_h) return false;
    const double tl = qg_gain_term(gl, hl, dg, dh, p.lambda);
    const double tr = qg_gain_term(gr, hr, dg, dh, p.lambda);
    gain = __dmul_rn(0.5, __dsub_rn(__dadd_rn(tl, tr), tp));
    return gain > p.min_gain;
}

// Running state of one feature's scan in one lane.
struct ScanState {
    long long carry_g, carry_h;   // sums of the bins before the current group of 32
    bool bv;
    double bgain;
    int bbin;
    long long bgl, bhl;
};

__device__ inline void qg_scan_init(ScanState &s) {
    s.carry_g = 0; s.carry_h = 0; s.bv = false; s.bgain = 0.0; s.bbin = -1; s.bgl = 0; s.bhl = 0;
}

// One group of 32 bins: lane holds the packed word of bin t = base + lane (0 beyond the last
// threshold nb - 2).  Evaluates threshold t for this lane and keeps the lane's best.
__device__ inline void qg_scan_step(ScanState &s, unsigned long long word, int t, int nb, const SplitParams &p,
                                    double dg, double dh, double tp) {
    const int lane = threadIdx.x & 31;
    long long g = 0, h = 0;
    if (t < nb - 1) {
        g = (long long)(int)(word >> 32);
        h = (long long)(unsigned int)(word & 0xFFFFFFFFull);
    }
    for (int o = 1; o < 32; o <<= 1) {
        const long long ug = __shfl_up_sync(0xffffffffu, g, o);
        const long long uh = __shfl_up_sync(0xffffffffu, h, o);
        if (lane >= o) { g += ug; h += uh; }
    }
    const long long gl = s.carry_g + g, hl = s.carry_h + h;
    s.carry_g += __shfl_sync(0xffffffffu, g, 31);
    s.carry_h += __shfl_sync(0xffffffffu, h, 31);
    if (t < nb - 1) {
        double gain;
        if (qg_eval_candidate(gl, hl, p, dg, dh, tp, gain) && (!s.bv || gain > s.bgain)) {
            s.bv = true; s.bgain = gain; s.bbin = t; s.bgl = gl; s.bhl = hl;
        }
    }
}

// Best of the 32 lanes (lowest bin on equal gain), as the record of feature f; valid in every lane.
__device__ inline SplitRec qg_scan_finish(ScanState s, int f) {
    for (int o = 16; o > 0; o >>= 1) {
        const bool ov = __shfl_xor_sync(0xffffffffu, (int)s.bv, o) != 0;
        const double og = __shfl_xor_sync(0xffffffffu, s.bgain, o);
        const int ob = __shfl_xor_sync(0xffffffffu, s.bbin, o);
        const long long ogl = __shfl_xor_sync(0xffffffffu, s.bgl, o);
        const long long ohl = __shfl_xor_sync(0xffffffffu, s.bhl, o);
        if (qg_better(ov, og, ob, s.bv, s.bgain, s.bbin)) { s.bv = ov; s.bgain = og; s.bbin = ob; s.bgl = ogl; s.bhl = ohl; }
    }
    SplitRec r;
    r.gain = s.bgain; r.gl = s.bgl; r.hl = s.bhl; r.feature = f; r.bin = s.bbin; r.valid = s.bv ? 1 : 0; r.pad = 0;
    return r;
}

__device__ inline SplitRec qg_invalid_rec() {
    SplitRec b;
    b.valid = 0; b.gain = 0.0; b.feature = -1; b.bin = -1; b.gl = 0; b.hl = 0; b.pad = 0;
    return b;
}

// Better of two per-feature records (lowest feature on equal gain).
__device__ inline bool qg_rec_better(const SplitRec &a, const SplitRec &b) {
    return qg_better(a.valid != 0, a.gain, a.feature, b.valid != 0, b.gain, b.feature);
}
