// Leaf-wise (best-first) growth of one tree (Sec. 3) in ONE persistent cooperative kernel: one CTA
// per SM, every decision taken on the device, grid-wide barriers between the phases of a split.
//
// Per split: (B) one predicate bit per row of the leaf being split and the number of left rows
// per warp range; barrier; (C) stable scatter of the (row, gradient code) pairs into the other
// pair buffer, left rows first; barrier; (D) Algorithm 1 on the smaller child's rows (partial
// histograms per CTA, or the finished histogram when one CTA does it all); barrier; (E) per
// feature: the smaller child's histogram from the partials, the larger child's as parent minus
// smaller, both children's best splits (Eq. 7); barrier; (F) every CTA reduces the per-feature
// candidates, updates its copy of the leaf gains and picks the leaf with the largest gain.
//
// The leaf gains (what the next pick needs) are replicated in every CTA's shared memory and
// updated identically, so no CTA waits for another one's decision; CTA 0 alone writes the tree
// and the leaf records to global memory.  Data that another CTA wrote during the kernel is read
// with L1-bypassing loads.
#include <cooperative_groups.h>

#include "hist_cta.cuh"
#include "split_scan.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int GROW_THREADS = 512;   // 128 registers per thread: the phases keep their state out of local memory
constexpr int GROW_WARPS = GROW_THREADS / 32;

struct GrowArgs {
    GrowState *gs;
    LeafRec *leaves;
    const DevState *state;
    const int32_t *feat_tile;
    uint2 *ent0, *ent1;              // the two (row, code) pair buffers
    uint32_t *bits, *counts;         // predicate bits of the leaf being split, left rows per warp range
    unsigned long long *pool;        // [L][F][nb]
    SplitRec *cand;                  // [F][2] best candidates of every feature for the two children
    int F, L, n_tiles;
    uint32_t N;
    SplitParams sp;                  // G, H, n_s are filled per leaf on the device
    HistArgs h;                      // tiles, codes, nb, partial, flush_rows, state for the histogram phase
    // tree output (device arrays of the current tree)
    int32_t *m_feature, *m_bin, *m_left, *m_right;
    double *m_gain;
};

__device__ inline SplitRec load_rec_cg(const SplitRec *p) {   // bypasses L1: written by another CTA of this kernel
    const long long *q = reinterpret_cast<const long long *>(p);
    long long v[5];
#pragma unroll
    for (int i = 0; i < 5; ++i) v[i] = __ldcg(q + i);
    SplitRec r;
    memcpy(&r, v, sizeof(r));
    return r;
}
static_assert(sizeof(SplitRec) == 40, "SplitRec is copied as five 64-bit words");
static_assert(sizeof(LeafRec) % 8 == 0, "LeafRec is copied as 64-bit words");

__device__ inline LeafRec load_leaf_cg(const LeafRec *p) {
    const long long *q = reinterpret_cast<const long long *>(p);
    long long v[sizeof(LeafRec) / 8];
#pragma unroll
    for (int i = 0; i < (int)(sizeof(LeafRec) / 8); ++i) v[i] = __ldcg(q + i);
    LeafRec r;
    memcpy(&r, v, sizeof(r));
    return r;
}

// Words of 32 rows [w0, w1) of grid-wide warp gw: every warp takes the same number of consecutive
// words (at least 4), so the warps with work are a prefix [0, active).
__device__ inline void warp_range(uint32_t nw, uint32_t gw, uint32_t n_count, uint32_t &w0, uint32_t &w1,
                                  uint32_t &active) {
    uint32_t per = (nw + n_count - 1) / n_count;
    if (per < 4) per = 4;
    active = (nw + per - 1) / per;
    w0 = gw * per < nw ? gw * per : nw;
    w1 = w0 + per < nw ? w0 + per : nw;
}

// The split being executed, identical in every CTA.
struct Cur {
    int pick, feature, bin, buf, slot, parent_node, parent_side;
    const uint32_t *col;   // word of the split feature in row 0 of its tile
    int logW, shift;       // words per row (log2) of that tile, bit position of the feature's byte
    uint32_t off, n;
    long long gl, hl, PG, PH;
    double gain;
};

// (B) predicate bits and left counts.  Four words of 32 rows at a time, so that the dependent
// loads (pair -> bin word) of the four are in flight together.
__device__ __forceinline__ void phase_flags(const GrowArgs &a, const Cur &cur, uint32_t gw, uint32_t n_count, int lane) {
    const uint32_t nw = (cur.n + 31) >> 5;
    uint32_t w0, w1, active;
    warp_range(nw, gw, n_count, w0, w1, active);
    if (gw >= active) return;
    const uint2 *src = cur.buf < 0 ? nullptr : (cur.buf ? a.ent1 : a.ent0);
    const uint32_t *col = cur.col;
    const int logW = cur.logW, shift = cur.shift;
    const uint32_t thr = (uint32_t)cur.bin, n = cur.n, off = cur.off;
    uint32_t lefts = 0;
    for (uint32_t w = w0; w < w1; w += 4) {
        uint32_t row[4], word[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = ((w + k) << 5) + lane;
            row[k] = (w + k < w1 && e < n) ? (src ? __ldcg(&src[off + e].x) : off + e) : 0xFFFFFFFFu;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) word[k] = row[k] != 0xFFFFFFFFu ? col[(size_t)row[k] << logW] : 0xFFFFFFFFu;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool left = row[k] != 0xFFFFFFFFu && ((word[k] >> shift) & 0xFFu) <= thr;
            const uint32_t b = __ballot_sync(0xffffffffu, left);
            if (w + k < w1) {
                if (lane == 0) a.bits[w + k] = b;
                lefts += __popc(b);
            }
        }
    }
    if (lane == 0) a.counts[gw] = lefts;
}

// Left rows before warp gw's range and in the whole leaf (sums of the warp counts).
__device__ __forceinline__ void count_lefts(const GrowArgs &a, const Cur &cur, uint32_t gw, uint32_t n_count, int lane,
                                   uint32_t &before, uint32_t &total) {
    const uint32_t nw = (cur.n + 31) >> 5;
    uint32_t w0, w1, active;
    warp_range(nw, gw, n_count, w0, w1, active);
    before = 0;
    total = 0;
    for (uint32_t j = lane; j < active; j += 32) {
        const uint32_t v = __ldcg(a.counts + j);
        total += v;
        if (j < gw) before += v;
    }
    for (int o = 16; o > 0; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
}

// (C) stable scatter of (row, code) pairs: left rows first, relative order kept.
__device__ __forceinline__ void phase_scatter(const GrowArgs &a, const Cur &cur, uint32_t gw, uint32_t n_count, int lane,
                                     uint32_t before, uint32_t total) {
    const uint32_t nw = (cur.n + 31) >> 5;
    uint32_t w0, w1, active;
    warp_range(nw, gw, n_count, w0, w1, active);
    if (gw >= active) return;
    const uint2 *src = cur.buf < 0 ? nullptr : (cur.buf ? a.ent1 : a.ent0);
    uint2 *dst = cur.buf == 0 ? a.ent1 : a.ent0;
    const uint32_t n = cur.n, off = cur.off;
    for (uint32_t w = w0; w < w1; w += 4) {
        uint32_t bw[4];
        uint2 ent[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = ((w + k) << 5) + lane;
            const bool ok = w + k < w1 && e < n;
            bw[k] = w + k < w1 ? __ldcg(a.bits + w + k) : 0u;
            if (ok) {
                if (src) {
                    ent[k] = __ldcg(src + off + e);
                } else {
                    ent[k].x = off + e;
                    ent[k].y = a.h.codes_nat[off + e];
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = ((w + k) << 5) + lane;
            if (w + k < w1 && e < n) {
                const uint32_t rank_l = __popc(bw[k] & ((1u << lane) - 1u));
                const bool left = (bw[k] >> lane) & 1u;
                const uint32_t dest = left ? before + rank_l : total + (((w + k) << 5) - before) + (lane - rank_l);
                dst[off + dest] = ent[k];
            }
            before += __popc(bw[k]);
        }
    }
}

__device__ inline void group_sync(int grp) { asm volatile("bar.sync %0, 256;" ::"r"(grp + 1) : "memory"); }

// What the per-feature finishing needs about the two children of the split being executed
// ("small" was built by Algorithm 1, "large" is parent - small); ROOT uses the small side only.
struct FinishCtx {
    SplitParams pS, pL;
    double dg, dh, tpS, tpL;
    uint32_t n_small;
    int new_slot, parent_slot;
};

// (E) for feature f, by one group of 256 threads: one thread per bin sums the partial histograms
// of the smaller child and takes the larger child's bin by subtraction; warps 0 and 1 of the
// group then scan the two children's bins.
template <bool ROOT>
__device__ __forceinline__ void finish_feature(const GrowArgs &a, const FinishCtx &fc, int f, int grp,
                                      unsigned long long *binS, unsigned long long *binL) {
    const int gt = threadIdx.x & 255, gwarp = gt >> 5, lane = gt & 31;
    const int nb = a.h.nb;
    const size_t hw = (size_t)a.F * nb;
    const TileDesc td = a.h.tiles[a.feat_tile[f]];
    const int fl = f - td.f0, W = 1 << td.logW;
    const uint32_t P = ROOT ? 1u : effective_parts((uint32_t)td.parts, fc.n_small);
    const size_t pstride = (size_t)4 * nb * 32;
    const unsigned long long *part = a.h.partial + (size_t)td.cta0 * pstride + (size_t)(fl & 3) * nb * W + (fl >> 2);
    unsigned long long *S = a.pool + (size_t)fc.new_slot * hw + (size_t)f * nb;
    unsigned long long *Pp = a.pool + (size_t)fc.parent_slot * hw + (size_t)f * nb;
    ScanState sc;
    qg_scan_init(sc);
    for (int base = 0; base < nb; base += 256) {
        const int b = base + gt;
        unsigned long long s = 0, l = 0;
        if (b < nb) {
            if (ROOT) {
                s = __ldcg(S + b);
            } else {
                if (P > 1) {
                    const unsigned long long *q = part + (size_t)b * W;
                    for (uint32_t i0 = 0; i0 < P; i0 += 16) {   // 16 independent loads in flight
                        unsigned long long x[16];
#pragma unroll
                        for (int k = 0; k < 16; ++k) x[k] = i0 + k < P ? __ldcg(q + (size_t)(i0 + k) * pstride) : 0ull;
#pragma unroll
                        for (int k = 0; k < 16; ++k) s += x[k];
                    }
                    S[b] = s;
                } else {
                    s = __ldcg(S + b);
                }
                l = __ldcg(Pp + b) - s;   // no field borrows: every child sum is at most the parent's
                Pp[b] = l;
            }
        }
        binS[gt] = s;
        binL[gt] = l;
        group_sync(grp);
        if (gwarp < (ROOT ? 1 : 2)) {
            const unsigned long long *bins = gwarp == 0 ? binS : binL;
            const SplitParams &pp = gwarp == 0 ? fc.pS : fc.pL;
            const double tp = gwarp == 0 ? fc.tpS : fc.tpL;
            for (int g = 0; g < 256 && base + g < nb; g += 32)
                qg_scan_step(sc, bins[g + lane], base + g + lane, nb, pp, fc.dg, fc.dh, tp);
        }
        group_sync(grp);
    }
    if (gwarp < 2) {
        const SplitRec r = (ROOT && gwarp == 1) ? qg_invalid_rec() : qg_scan_finish(sc, f);
        if (lane == 0) a.cand[2 * f + gwarp] = r;
    }
}

__device__ inline SplitRec warp_best(SplitRec r) {
    for (int o = 16; o > 0; o >>= 1) {
        SplitRec x;
        x.gain = __shfl_xor_sync(0xffffffffu, r.gain, o);
        x.gl = __shfl_xor_sync(0xffffffffu, r.gl, o);
        x.hl = __shfl_xor_sync(0xffffffffu, r.hl, o);
        x.feature = __shfl_xor_sync(0xffffffffu, r.feature, o);
        x.bin = __shfl_xor_sync(0xffffffffu, r.bin, o);
        x.valid = __shfl_xor_sync(0xffffffffu, r.valid, o);
        x.pad = 0;
        if (qg_rec_better(x, r)) r = x;
    }
    return r;
}

// (F) best candidates over all features for the two children (0 small, 1 large); the results are
// valid in every thread.  s_red: [2][32] scratch.
__device__ __forceinline__ void reduce_cand(const GrowArgs &a, SplitRec *s_red, SplitRec &outS, SplitRec &outL) {
    SplitRec bS = qg_invalid_rec(), bL = qg_invalid_rec();
    for (int f = threadIdx.x; f < a.F; f += GROW_THREADS) {
        const SplitRec x = load_rec_cg(a.cand + 2 * f), y = load_rec_cg(a.cand + 2 * f + 1);
        if (qg_rec_better(x, bS)) bS = x;
        if (qg_rec_better(y, bL)) bL = y;
    }
    bS = warp_best(bS);
    bL = warp_best(bL);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) { s_red[warp] = bS; s_red[32 + warp] = bL; }
    __syncthreads();
    outS = warp_best(lane < GROW_WARPS ? s_red[lane] : qg_invalid_rec());
    outL = warp_best(lane < GROW_WARPS ? s_red[32 + lane] : qg_invalid_rec());
}

// Leaf with the largest gain (lowest number on equal gain) among sh_gain[0 .. n), or -1.
__device__ __forceinline__ int pick_leaf(const double *sh_gain, int n, double *s_pg, int *s_pi) {
    const double NEG = -__longlong_as_double(0x7FF0000000000000LL);
    double bg = NEG;
    int bi = -1;
    for (int i = threadIdx.x; i < n; i += GROW_THREADS) {
        const double g = sh_gain[i];
        if (g > bg) { bg = g; bi = i; }   // ascending i: the first maximum stays
    }
    for (int o = 16; o > 0; o >>= 1) {
        const double og = __shfl_xor_sync(0xffffffffu, bg, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (oi >= 0 && (bi < 0 || og > bg || (og == bg && oi < bi))) { bg = og; bi = oi; }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) { s_pg[warp] = bg; s_pi[warp] = bi; }
    __syncthreads();
    bg = lane < GROW_WARPS ? s_pg[lane] : NEG;
    bi = lane < GROW_WARPS ? s_pi[lane] : -1;
    for (int o = 16; o > 0; o >>= 1) {
        const double og = __shfl_xor_sync(0xffffffffu, bg, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (oi >= 0 && (bi < 0 || og > bg || (og == bg && oi < bi))) { bg = og; bi = oi; }
    }
    return bi;
}

template <bool WIDE>
__device__ __forceinline__ void run_hist_unit(HistArgs &ha, const TileDesc &td, uint32_t part, uint32_t P, int *sh) {
    for (int pass = 0; pass < (WIDE ? 2 : 1); ++pass) {
        if (WIDE) {
            if (threadIdx.x == 0) ha.pass = pass;
            __syncthreads();
        }
        switch (td.logW) {
            case 5: hist_cta<GROW_THREADS, 5, WIDE, 2>(ha, td, part, P, sh); break;
            case 3: hist_cta<GROW_THREADS, 3, WIDE, 2>(ha, td, part, P, sh); break;
            default: hist_cta<GROW_THREADS, -1, WIDE, 2>(ha, td, part, P, sh); break;
        }
        __syncthreads();   // the local histogram is reused by the next pass / unit
    }
}

template <bool WIDE>
__global__ void __launch_bounds__(GROW_THREADS, 1) k_grow(const GrowArgs args) {
    extern __shared__ __align__(1024) int sh[];
    // arguments and per-split context live in shared memory: with 210 KB of it carved out there is
    // hardly any L1 left for per-thread local copies
    __shared__ GrowArgs s_args;
    __shared__ FinishCtx s_fc;
    __shared__ HistArgs s_ha;
    if (threadIdx.x == 0) s_args = args;
    __syncthreads();
    const GrowArgs &a = s_args;
    cg::grid_group grid = cg::this_grid();
    const uint32_t G = gridDim.x, cta = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const uint32_t n_count = G * GROW_WARPS, gw = (uint32_t)warp * G + cta;   // neighbouring ranges on different SMs
    const int grp = tid >> 8;
    const int nb = a.h.nb;
    const size_t hw = (size_t)a.F * nb;

    // the leaf gains live below the 64 KB-aligned local histogram (the same for every CTA)
    const uint32_t sbase = smem_u32(sh);
    const uint32_t h0 = (sbase + 65535u) & ~65535u;
    uint32_t dyn_size;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_size));
    if (h0 + 131072u > sbase + dyn_size || (uint32_t)a.L * 8u > h0 - sbase) {
        if (cta == 0 && tid == 0) atomicExch(&a.h.state->kernel_error, 1);
        return;   // every CTA takes this branch: no barrier is left waiting
    }
    double *sh_gain = reinterpret_cast<double *>(sh);
    __shared__ unsigned long long s_bins[GROW_THREADS / 256][2][256];
    __shared__ SplitRec s_red[64];
    __shared__ double s_pg[32];
    __shared__ int s_pi[32];
    __shared__ Cur s_cur;
    __shared__ LeafRec s_child[2];
    __shared__ int s_child_id[2];
    const double NEG = -__longlong_as_double(0x7FF0000000000000LL);
    for (int i = tid; i < a.L; i += GROW_THREADS) sh_gain[i] = NEG;

    // ---- root: scan its histogram (pool slot 0, built before this kernel)
    const long long G0 = a.state->tot_g, H0 = a.state->tot_h;
    FinishCtx &fc = s_fc;
    if (tid == 0) {
        fc.pS = a.sp; fc.pL = a.sp;
        fc.pS.G = G0; fc.pS.H = H0; fc.pS.n_s = a.N;
        qg_scales(a.state, fc.pS, fc.dg, fc.dh);
        fc.tpS = qg_gain_term(G0, H0, fc.dg, fc.dh, fc.pS.lambda);
        fc.tpL = 0.0;
        fc.n_small = a.N; fc.new_slot = 0; fc.parent_slot = 0;
        s_ha = a.h;
    }
    __syncthreads();
    for (int f = (int)cta * (GROW_THREADS / 256) + grp; f < a.F; f += (int)G * (GROW_THREADS / 256)) finish_feature<true>(a, fc, f, grp, s_bins[grp][0], s_bins[grp][1]);
    __syncthreads();
    grid.sync();
    {
        SplitRec b, unused;
        reduce_cand(a, s_red, b, unused);
        if (tid == 0) {
            LeafRec r;
            r.off = 0; r.n = a.N; r.buf = -1; r.slot = 0; r.G = G0; r.H = H0; r.best = b;
            r.parent_node = -1; r.parent_side = 0;
            s_child[0] = r;
            s_child_id[0] = 0;
            s_child_id[1] = -1;
            if (b.valid) sh_gain[0] = b.gain;
            if (cta == 0) a.leaves[0] = r;
        }
    }
    int n_leaves = 1;
    unsigned long long hist_rows = 0;
    __syncthreads();

    for (int split = 1; split < a.L; ++split) {
        // ---- (A) the leaf to split
        const int pick = pick_leaf(sh_gain, n_leaves, s_pg, s_pi);
        if (pick < 0) break;   // identical in every CTA
        if (tid == 0) {
            const LeafRec r = pick == s_child_id[0] ? s_child[0] : (pick == s_child_id[1] ? s_child[1] : load_leaf_cg(a.leaves + pick));
            Cur c;
            c.pick = pick; c.feature = r.best.feature; c.bin = r.best.bin; c.buf = r.buf; c.slot = r.slot;
            c.parent_node = r.parent_node; c.parent_side = r.parent_side;
            {
                const TileDesc td = a.h.tiles[a.feat_tile[r.best.feature]];
                const int fl = r.best.feature - td.f0;
                c.col = td.data + (fl >> 2);
                c.logW = td.logW;
                c.shift = 8 * (fl & 3);
            }
            c.off = r.off; c.n = r.n; c.gl = r.best.gl; c.hl = r.best.hl; c.PG = r.G; c.PH = r.H; c.gain = r.best.gain;
            s_cur = c;
        }
        __syncthreads();
        const Cur &cur = s_cur;

        // ---- (B) flags
        phase_flags(a, cur, gw, n_count, lane);
        grid.sync();
        // ---- (C) scatter
        uint32_t before, nl;
        count_lefts(a, cur, gw, n_count, lane, before, nl);
        phase_scatter(a, cur, gw, n_count, lane, before, nl);
        const uint32_t nr = cur.n - nl;
        const bool small_is_left = nl <= nr;
        const uint32_t n_small = small_is_left ? nl : nr;
        grid.sync();
        // ---- (D) histogram of the smaller child (ties: the left one) into pool slot n_leaves
        {
            HistArgs &ha = s_ha;
            if (tid == 0) {
                ha.ents = cur.buf == 0 ? a.ent1 : a.ent0;
                ha.rows = nullptr;
                ha.off = small_is_left ? cur.off : cur.off + nl;
                ha.n = n_small;
                ha.hist = a.pool + (size_t)n_leaves * hw;
            }
            __syncthreads();
            uint32_t ubase = 0;
            for (int t = 0; t < a.n_tiles; ++t) {
                const TileDesc td = a.h.tiles[t];
                const uint32_t P = effective_parts((uint32_t)td.parts, n_small);
                for (uint32_t p = (cta + G - ubase % G) % G; p < P; p += G) run_hist_unit<WIDE>(ha, td, p, P, sh);
                ubase += P;
            }
        }
        grid.sync();
        // ---- (E) per feature: merge, subtract, scan
        if (tid == 0) {
            const long long gl = cur.gl, hl = cur.hl, gr = cur.PG - gl, hr = cur.PH - hl;
            fc.pS.G = small_is_left ? gl : gr; fc.pS.H = small_is_left ? hl : hr; fc.pS.n_s = small_is_left ? nl : nr;
            fc.pL.G = small_is_left ? gr : gl; fc.pL.H = small_is_left ? hr : hl; fc.pL.n_s = small_is_left ? nr : nl;
            fc.tpS = qg_gain_term(fc.pS.G, fc.pS.H, fc.dg, fc.dh, fc.pS.lambda);
            fc.tpL = qg_gain_term(fc.pL.G, fc.pL.H, fc.dg, fc.dh, fc.pL.lambda);
            fc.n_small = n_small; fc.new_slot = n_leaves; fc.parent_slot = cur.slot;
        }
        __syncthreads();
        for (int f = (int)cta * (GROW_THREADS / 256) + grp; f < a.F; f += (int)G * (GROW_THREADS / 256))
            finish_feature<false>(a, fc, f, grp, s_bins[grp][0], s_bins[grp][1]);
        __syncthreads();
        grid.sync();
        // ---- (F) every CTA: the children's best splits, the new leaves, the gains
        SplitRec bS, bL;
        reduce_cand(a, s_red, bS, bL);
        if (tid == 0) {
            const int right = n_leaves, node = n_leaves - 1;
            const int dstbuf = cur.buf == 0 ? 1 : 0;
            LeafRec lf, rt;
            lf.off = cur.off; lf.n = nl; lf.buf = dstbuf; lf.G = cur.gl; lf.H = cur.hl;
            lf.parent_node = node; lf.parent_side = 0;
            rt.off = cur.off + nl; rt.n = nr; rt.buf = dstbuf; rt.G = cur.PG - cur.gl; rt.H = cur.PH - cur.hl;
            rt.parent_node = node; rt.parent_side = 1;
            lf.slot = small_is_left ? n_leaves : cur.slot;
            rt.slot = small_is_left ? cur.slot : n_leaves;
            lf.best = small_is_left ? bS : bL;
            rt.best = small_is_left ? bL : bS;
            s_child[0] = lf; s_child_id[0] = pick;
            s_child[1] = rt; s_child_id[1] = right;
            sh_gain[pick] = lf.best.valid ? lf.best.gain : NEG;
            sh_gain[right] = rt.best.valid ? rt.best.gain : NEG;
            if (cta == 0) {
                a.leaves[pick] = lf;
                a.leaves[right] = rt;
                a.m_feature[node] = cur.feature;
                a.m_bin[node] = cur.bin;
                a.m_left[node] = ~pick;
                a.m_right[node] = ~right;
                a.m_gain[node] = cur.gain;
                if (cur.parent_node >= 0) {
                    if (cur.parent_side == 0) a.m_left[cur.parent_node] = node;
                    else a.m_right[cur.parent_node] = node;
                }
            }
        }
        hist_rows += n_small;
        ++n_leaves;
        __syncthreads();
    }
    if (cta == 0 && tid == 0) {
        a.gs->n_leaves = n_leaves;
        a.gs->hist_rows += hist_rows;
        a.gs->hist_builds += (unsigned long long)(n_leaves - 1);
    }
}

}  // namespace

// Grows the tree of boosting iteration slot `tree_slot` of the current train call.  Gradients must
// have been quantized on the same stream (the state holds the totals and maxima).  Asynchronous.
int qg_grow_tree(qgbdt_ctx *c, int tree_slot, cudaStream_t st) {
    const int L = c->prm.num_leaves;
    int rc = qg_hist(c, nullptr, 0, c->N, c->d_hist_pool, st);   // root: all rows, contiguous, into slot 0
    if (rc != QGBDT_OK) return rc;

    GrowArgs a;
    a.gs = c->d_gs;
    a.leaves = c->d_leaves;
    a.state = c->d_state;
    a.feat_tile = c->d_feat_tile;
    a.ent0 = c->d_ent0;
    a.ent1 = c->d_ent1;
    a.bits = c->d_part_bits;
    a.counts = c->d_part_counts;
    a.pool = c->d_hist_pool;
    a.cand = c->d_cand;
    a.F = c->F;
    a.L = L;
    a.n_tiles = (int)c->tiles.size();
    a.N = (uint32_t)c->N;
    a.sp.G = a.sp.H = a.sp.n_s = 0;
    a.sp.kg = qg_levels_g(c->prm.bits);
    a.sp.kh = qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    a.sp.const_h = c->const_hess ? 1 : 0;
    a.sp.min_data = c->prm.min_data_in_leaf;
    a.sp.min_sum_h = c->prm.min_sum_hessian;
    a.sp.min_gain = c->prm.min_gain;
    a.sp.lambda = c->prm.lambda_l2;
    const int kh = c->const_hess ? 1 : a.sp.kh;
    a.h.tiles = c->d_tiles;
    a.h.codes = reinterpret_cast<const uint16_t *>(c->d_codes);
    a.h.codes_nat = reinterpret_cast<const uint16_t *>(c->d_codes_nat);
    a.h.tile0 = 0;
    a.h.rows = nullptr;
    a.h.ents = nullptr;
    a.h.off = 0;
    a.h.n = 0;
    a.h.nb = c->nb;
    a.h.hist = nullptr;
    a.h.partial = c->d_partial;
    const uint32_t by_h = 65535u / (uint32_t)kh, by_g = 32767u / (uint32_t)a.sp.kg;
    a.h.flush_rows = by_h < by_g ? by_h : by_g;
    a.h.pass = 0;
    a.h.state = c->d_state;
    const size_t no = (size_t)tree_slot * (L > 1 ? L - 1 : 1);
    a.m_feature = c->d_m_feature + no;
    a.m_bin = c->d_m_bin + no;
    a.m_left = c->d_m_left + no;
    a.m_right = c->d_m_right + no;
    a.m_gain = c->d_m_gain + no;

    const bool wide = c->prm.bits >= 6;
    const void *kern = wide ? reinterpret_cast<const void *>(k_grow<true>) : reinterpret_cast<const void *>(k_grow<false>);
    static bool configured[2] = {false, false};
    if (!configured[wide ? 1 : 0]) {
        QG_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_SMEM));
        int coop = 0, per_sm = 0;
        QG_CUDA(c, cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device));
        QG_CUDA(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, GROW_THREADS, HIST_SMEM));
        if (!coop || per_sm < 1)
            return qg_fail(c, QGBDT_ERR_CUDA, "the device cannot co-schedule one tree-growing CTA per SM");
        configured[wide ? 1 : 0] = true;
    }
    void *params[] = {&a};
    QG_CUDA(c, cudaLaunchCooperativeKernel(kern, dim3((unsigned)c->sm_count), dim3(GROW_THREADS), params, HIST_SMEM, st));
    c->n_launches++;
    return QGBDT_OK;
}
