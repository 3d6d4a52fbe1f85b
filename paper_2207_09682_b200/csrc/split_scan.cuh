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

// Threshold candidate with left sums (gl, hl): everything of its admissibility that needs no gain.
// The row estimate of a side is floor((hl * n_s + H / 2) / H) (exact count with a constant hessian);
// it is only compared with min_data, so the comparisons are made on the products instead of
// dividing: floor(X / H) >= m  <=>  X >= m * H, and floor(X / H) <= k  <=>  X < (k + 1) * H.
__device__ inline bool qg_candidate_admissible(long long gl, long long hl, const SplitParams &p, double dh) {
    (void)gl;
    const long long hr = p.H - hl;
    if (!(hl > 0 && hr > 0)) return false;
    if (p.const_h) {
        if (!(hl >= p.min_data && p.n_s - hl >= p.min_data)) return false;
    } else {
        const unsigned long long H = (unsigned long long)p.H, X = (unsigned long long)hl * (unsigned long long)p.n_s + H / 2;
        const long long k = p.n_s - p.min_data;          // the left side may have at most this many rows
        if (X < (unsigned long long)p.min_data * H) return false;
        if (k < 0 || X >= (unsigned long long)(k + 1) * H) return false;
    }
    if (__dmul_rn((double)hl, dh) < p.min_sum_h || __dmul_rn((double)hr, dh) < p.min_sum_h) return false;
    return true;
}

// Eq. 7 for an admissible candidate, every operation individually rounded in double precision.
__device__ inline double qg_candidate_gain(long long gl, long long hl, const SplitParams &p, double dg, double dh, double tp) {
    const double tl = qg_gain_term(gl, hl, dg, dh, p.lambda);
    const double tr = qg_gain_term(p.G - gl, p.H - hl, dg, dh, p.lambda);
    return __dmul_rn(0.5, __dsub_rn(__dadd_rn(tl, tr), tp));
}

// Threshold candidate with left sums (gl, hl): admissible?  If so its gain (Eq. 7).
__device__ inline bool qg_eval_candidate(long long gl, long long hl, const SplitParams &p, double dg, double dh,
                                         double tp, double &gain) {
    if (!qg_candidate_admissible(gl, hl, p, dh)) return false;
    gain = qg_candidate_gain(gl, hl, p, dg, dh, tp);
    return gain > p.min_gain;
}

// Single-precision bounds [lo, hi] on the double-precision gain of an admissible candidate, about a
// sixth of the cost of the gain itself (no double-precision division).  Every term of Eq. 7 comes
// out with a relative error of at most 12 * 2^-24 (conversions, products, one division each), so the
// gain is off by less than 16 * 2^-24 * (term L + term R + term P); the bounds take four times
// that.  A search that keeps every candidate whose `hi` reaches the largest `lo` keeps every
// candidate that can have the largest gain.
struct GainScale {
    float dg, dh, lambda;
};
__device__ inline void qg_gain_bounds(long long gl, long long hl, const SplitParams &p, const GainScale &sc, float tp,
                                      float &lo, float &hi) {
    const float gdl = __fmul_rn((float)gl, sc.dg), gdr = __fmul_rn((float)(p.G - gl), sc.dg);
    const float hdl = __fadd_rn(__fmul_rn((float)hl, sc.dh), sc.lambda), hdr = __fadd_rn(__fmul_rn((float)(p.H - hl), sc.dh), sc.lambda);
    const float tl = __fdiv_rn(__fmul_rn(gdl, gdl), hdl), tr = __fdiv_rn(__fmul_rn(gdr, gdr), hdr);
    const float gain = __fmul_rn(0.5f, __fsub_rn(__fadd_rn(tl, tr), tp));
    const float err = __fmul_rn(3.814697265625e-6f, __fadd_rn(__fadd_rn(tl, tr), tp));   // 64 * 2^-24
    lo = __fsub_rn(gain, err);
    hi = __fadd_rn(gain, err);
    if (!(fabsf(gain) <= 3.0e38f) || !(err <= 3.0e38f)) {   // out of single-precision range: no information
        lo = -__int_as_float(0x7f800000);
        hi = __int_as_float(0x7f800000);
    }
}

// The same two tests for the tree-growing kernels, on 32-bit sums (a leaf's gradient and hessian sums
// fit 32 bits: checked when the rows are loaded) and with the per-leaf constants taken out.
__device__ inline Admit32 qg_admit32(const SplitParams &p, double dh) {
    Admit32 a;
    a.G = (int)p.G; a.H = (uint32_t)p.H; a.n_s = (uint32_t)p.n_s; a.half = a.H / 2;
    a.min_data = (uint32_t)p.min_data;
    a.const_h = p.const_h;
    const long long k = p.n_s - p.min_data;
    a.x_min = (unsigned long long)p.min_data * a.H;
    a.x_end = k < 0 ? 0ull : (unsigned long long)(k + 1) * a.H;
    // the single-precision product is off by less than 4 * 2^-24 relative; 2^-20 above the limit is safe
    a.q_sure = __fmul_ru(__double2float_ru(p.min_sum_h), 1.00000095367431640625f);
    a.min_sum_h = p.min_sum_h;
    a.dh = dh;
    return a;
}

// qg_candidate_admissible for left hessian sum hl, same decisions: the products with the interval
// length are compared in single precision where that is certain, in double precision otherwise.
__device__ inline bool qg_admissible32(uint32_t hl, const Admit32 &a, const GainScale &sc) {
    const uint32_t hr = a.H - hl;
    if (hl == 0 || hr == 0) return false;
    if (a.const_h) {
        if (!(hl >= a.min_data && a.n_s - hl >= a.min_data)) return false;
    } else {
        const unsigned long long X = (unsigned long long)hl * a.n_s + a.half;
        if (X < a.x_min || X >= a.x_end) return false;
    }
    if (!(__fmul_rn((float)hl, sc.dh) >= a.q_sure) || !(__fmul_rn((float)hr, sc.dh) >= a.q_sure)) {
        if (__dmul_rn((double)hl, a.dh) < a.min_sum_h || __dmul_rn((double)hr, a.dh) < a.min_sum_h) return false;
    }
    return true;
}

// qg_gain_bounds on 32-bit sums, with the fast division (2 units in the last place: every term of
// Eq. 7 still comes out within 16 * 2^-24 relative, of which the bounds take four times).
__device__ inline void qg_gain_bounds32(int gl, uint32_t hl, const Admit32 &a, const GainScale &sc, float tp,
                                        float &lo, float &hi) {
    const float gdl = __fmul_rn((float)gl, sc.dg), gdr = __fmul_rn((float)(a.G - gl), sc.dg);
    const float hdl = __fadd_rn(__fmul_rn((float)hl, sc.dh), sc.lambda), hdr = __fadd_rn(__fmul_rn((float)(a.H - hl), sc.dh), sc.lambda);
    const float tl = __fdividef(__fmul_rn(gdl, gdl), hdl), tr = __fdividef(__fmul_rn(gdr, gdr), hdr);
    const float gain = __fmul_rn(0.5f, __fsub_rn(__fadd_rn(tl, tr), tp));
    // 64 * 2^-24 of the terms, and room for results that left the normal range on the way
    const float err = __fadd_rn(__fmul_rn(3.814697265625e-6f, __fadd_rn(__fadd_rn(tl, tr), tp)), 1.0e-37f);
    lo = __fsub_rn(gain, err);
    hi = __fadd_rn(gain, err);
    // out of the range in which single precision (and its fast division) says anything: no information.
    // (A non-zero gradient sum times dg >= 1e-15 squares to a normal number.)
    if (!(fabsf(gain) <= 3.0e38f) || !(err <= 3.0e38f) || !(fmaxf(hdl, hdr) <= 1.0e30f) || !(fminf(hdl, hdr) >= 1.0e-30f) ||
        !(sc.dg >= 1.0e-15f)) {
        lo = -__int_as_float(0x7f800000);
        hi = __int_as_float(0x7f800000);
    }
}

// What the finishing kernel needs of a leaf being split that is the same for all its features (known
// once the rows of both sides are: after the partition of the pass).
__device__ inline JobPrep qg_job_prep(const GrowState *gs, int j, const DevState *state, const SplitParams &sp,
                                      uint32_t rows_min) {
    const GrowJob *job = gs->jobs + j;
    const uint32_t n = job->n, nl = job->nl, nr = n - nl;
    const uint32_t n_all = job->n_all, nl_all = (uint32_t)gs->nl_all[j], nr_all = n_all - nl_all;
    const long long gl = job->gl, hl = job->hl, gr = job->PG - gl, hr = job->PH - hl;
    JobPrep r;
    r.small_is_left = nl_all <= nr_all ? 1 : 0;
    SplitParams pS = sp, pL = sp;
    pS.G = r.small_is_left ? gl : gr; pS.H = r.small_is_left ? hl : hr; pS.n_s = r.small_is_left ? nl_all : nr_all;
    pL.G = r.small_is_left ? gr : gl; pL.H = r.small_is_left ? hr : hl; pL.n_s = r.small_is_left ? nr_all : nl_all;
    qg_scales(state, sp, r.dg, r.dh);
    r.tpS = qg_gain_term(pS.G, pS.H, r.dg, r.dh, sp.lambda);
    r.tpL = qg_gain_term(pL.G, pL.H, r.dg, r.dh, sp.lambda);
    r.aS = qg_admit32(pS, r.dh);
    r.aL = qg_admit32(pL, r.dh);
    r.P = qg_grow_parts((uint32_t)job->parts, r.small_is_left ? nl : nr, rows_min);
    return r;
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
