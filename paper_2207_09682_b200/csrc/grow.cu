// Leaf-wise (best-first) growth of one tree (Sec. 3) with every decision taken on the device:
// the host enqueues a fixed sequence of kernels per split and never waits for a result.
//
// Per split: (1) k_grow_flags: one predicate bit per row of the leaf being split and the number
// of left rows per warp range; (2) k_grow_scatter: stable scatter of the (row, gradient code)
// pairs into the other pair buffer (left rows first); (3) the histogram kernel on the smaller child's rows
// (Algorithm 1); (4) k_grow_finish: per feature, the smaller child's histogram from the partial
// histograms, the larger child's as parent minus smaller, both children's best splits (Eq. 7);
// the last block to finish records the split in the tree, creates the leaf records and picks
// the leaf with the largest gain for the next split.
#include "split_scan.cuh"

namespace {

constexpr int PART_THREADS = 256;
constexpr int PART_WARPS = PART_THREADS / 32;
constexpr uint32_t MIN_ROWS_PER_CTA = 1024;   // same rule as the histogram kernel

__device__ __host__ inline uint32_t effective_parts(uint32_t parts, uint32_t n) {
    uint32_t want = (n + MIN_ROWS_PER_CTA - 1) / MIN_ROWS_PER_CTA;
    if (want < 1) want = 1;
    return want < parts ? want : parts;
}

struct GrowArgs {
    GrowState *gs;
    LeafRec *leaves;
    const DevState *state;
    const FeatRec *feat_rec;         // [F]
    double *leaf_gain;               // [L] gain of every leaf's best split, -inf when it has none
    uint32_t N;
    uint2 *ent0, *ent1;              // the two (row, gradient code) pair buffers
    const uint16_t *codes_nat;       // codes in row order (the root's identity list has no pairs yet)
    uint32_t *bits, *counts;         // predicate bits of the leaf being split, left rows per warp range
    int n_count;                     // warp ranges (= warps of the flag / scatter grids)
    unsigned long long *pool;        // [L][F][nb]
    const unsigned long long *partial;
    SplitRec *cand;                  // [F][2] best candidates of every feature for the two children
    int F, nb, L;
    SplitParams sp;                  // G, H, n_s are filled per leaf on the device
    // tree output (device arrays of the current tree)
    int32_t *m_feature, *m_bin, *m_left, *m_right;
    double *m_gain;
};

__global__ void k_grow_begin(GrowState *gs, LeafRec *leaves, const DevState *state, uint32_t N, int tree_slot) {
    gs->tree_slot = tree_slot;
    LeafRec r;
    r.off = 0; r.n = N; r.buf = -1; r.slot = 0;
    r.G = state->tot_g; r.H = state->tot_h;
    r.best = qg_invalid_rec();
    r.parent_node = -1; r.parent_side = 0;
    leaves[0] = r;
    gs->n_leaves = 1;
    // gradients out of domain (the flag is sticky over the trees of a train call): the split
    // kernels of this tree return at once, the call reports the error when it ends
    gs->done = state->bad_value ? 1 : 0;
    gs->finish_count = 0;
}

// Words of 32 rows [w0, w1) of warp gw: every warp takes the same number of consecutive words
// (at least 4), so the warps with work are a prefix [0, active) of the grid.
__device__ inline void warp_range(uint32_t nw, uint32_t gw, uint32_t n_count, uint32_t &w0, uint32_t &w1,
                                  uint32_t &active) {
    uint32_t per = (nw + n_count - 1) / n_count;
    if (per < 4) per = 4;
    active = (nw + per - 1) / per;
    w0 = gw * per < nw ? gw * per : nw;
    w1 = w0 + per < nw ? w0 + per : nw;
}

// Four words of 32 rows at a time, so that the dependent loads (pair -> bin word) of the four are
// in flight together.
__global__ void __launch_bounds__(PART_THREADS) k_grow_flags(GrowArgs a) {
    const GrowState *gs = a.gs;
    // every field at once (one round trip to memory), then the early exits
    const int done = gs->done, buf = gs->buf;
    const uint32_t n = gs->n, off = gs->off;
    const uint32_t *col = gs->col;
    const uint8_t *col8 = gs->col8;
    const int logW = gs->logW, shift = 8 * gs->byte;
    const uint32_t thr = (uint32_t)gs->bin;
    if (done) return;
    const int lane = threadIdx.x & 31;
    const uint32_t gw = blockIdx.x * PART_WARPS + (threadIdx.x >> 5);
    const uint32_t nw = (n + 31) >> 5;
    uint32_t w0, w1, active;
    warp_range(nw, gw, (uint32_t)a.n_count, w0, w1, active);
    if (blockIdx.x * PART_WARPS >= active) return;   // no warp of this block has work
    const uint2 *src = buf < 0 ? nullptr : (buf ? a.ent1 : a.ent0);
    uint32_t lefts = 0;
    for (uint32_t w = w0; w < w1; w += 4) {
        uint32_t row[4], word[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = ((w + k) << 5) + lane;
            row[k] = (w + k < w1 && e < n) ? (src ? src[off + e].x : off + e) : 0xFFFFFFFFu;
        }
        // the bin code of the split feature: one byte of the column-major copy (ascending rows share
        // DRAM granules), or, without that copy, a word of the tile (a granule per row)
        if (col8) {
#pragma unroll
            for (int k = 0; k < 4; ++k) word[k] = row[k] != 0xFFFFFFFFu ? (uint32_t)col8[row[k]] << shift : 0xFFFFFFFFu;
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) word[k] = row[k] != 0xFFFFFFFFu ? col[(size_t)row[k] << logW] : 0xFFFFFFFFu;
        }
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
    // left rows of every warp range and of every block's ranges (the scatter kernel adds up the
    // blocks before its own and the warps before it inside its block)
    __shared__ uint32_t block_lefts[PART_WARPS];
    if (lane == 0) {
        a.counts[gw] = lefts;
        block_lefts[threadIdx.x >> 5] = lefts;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
#pragma unroll
        for (int v = 0; v < PART_WARPS; ++v) t += block_lefts[v];
        a.counts[a.n_count + blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(PART_THREADS) k_grow_scatter(GrowArgs a) {
    GrowState *gs = a.gs;
    const int done = gs->done, buf = gs->buf;   // every field at once, then the early exits
    const uint32_t n = gs->n, off = gs->off;
    if (done) return;
    const int lane = threadIdx.x & 31;
    const uint32_t gw = blockIdx.x * PART_WARPS + (threadIdx.x >> 5);
    const uint32_t nw = (n + 31) >> 5;
    uint32_t w0, w1, active;
    warp_range(nw, gw, (uint32_t)a.n_count, w0, w1, active);
    if (gw >= active && gw != 0) return;
    // left rows before this warp's range, and in the whole leaf: the totals of the blocks, and
    // the warps of this block before this one
    uint32_t before = 0, total = 0;
    const uint32_t active_blocks = (active + PART_WARPS - 1) / PART_WARPS;
    const uint32_t *block_counts = a.counts + a.n_count;
    for (uint32_t j0 = 0; j0 < active_blocks; j0 += 256) {   // eight independent loads per lane in flight
        uint32_t v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t j = j0 + 32 * k + lane;
            v[k] = j < active_blocks ? block_counts[j] : 0u;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            total += v[k];
            if (j0 + 32 * k + lane < blockIdx.x) before += v[k];
        }
    }
    {
        const uint32_t j = blockIdx.x * PART_WARPS + lane;
        if (lane < PART_WARPS && j < gw) before += a.counts[j];
    }
    for (int o = 16; o > 0; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if (gw == 0 && lane == 0) gs->nl = total;
    const uint2 *src = buf < 0 ? nullptr : (buf ? a.ent1 : a.ent0);
    uint2 *dst = buf == 0 ? a.ent1 : a.ent0;
    for (uint32_t w = w0; w < w1; w += 4) {
        uint32_t bw[4];
        uint2 ent[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = ((w + k) << 5) + lane;
            bw[k] = w + k < w1 ? a.bits[w + k] : 0u;
            if (w + k < w1 && e < n) {
                if (src) {
                    ent[k] = src[off + e];
                } else {
                    ent[k].x = off + e;
                    ent[k].y = a.codes_nat[off + e];
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

__device__ inline SplitRec load_rec_cg(const SplitRec *p) {   // bypasses L1: written by another block of this kernel
    const long long *q = reinterpret_cast<const long long *>(p);
    long long v[5];
#pragma unroll
    for (int i = 0; i < 5; ++i) v[i] = __ldcg(q + i);
    SplitRec r;
    memcpy(&r, v, sizeof(r));
    return r;
}
static_assert(sizeof(SplitRec) == 40, "SplitRec is copied as five 64-bit words");

__device__ inline SplitRec shfl_xor_rec(const SplitRec &r, int o) {
    SplitRec x;
    x.gain = __shfl_xor_sync(0xffffffffu, r.gain, o);
    x.gl = __shfl_xor_sync(0xffffffffu, r.gl, o);
    x.hl = __shfl_xor_sync(0xffffffffu, r.hl, o);
    x.feature = __shfl_xor_sync(0xffffffffu, r.feature, o);
    x.bin = __shfl_xor_sync(0xffffffffu, r.bin, o);
    x.valid = __shfl_xor_sync(0xffffffffu, r.valid, o);
    x.pad = 0;
    return x;
}

// ROOT: scans the root histogram (pool slot 0).  Otherwise: completes the split recorded in the
// grow state.  One block per feature.
// BPT bins per thread: 1 (256 threads) or 2 (128 threads: with thousands of features twice as many
// blocks are resident, and the grid fits the SMs in one wave).
template <bool ROOT, int BPT>
__global__ void __launch_bounds__(256 / BPT) k_grow_finish(GrowArgs a) {
    constexpr int FIN_WARPS = 8 / BPT;
    GrowState *gs = a.gs;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int f = blockIdx.x;   // one block per feature
    // everything the block needs from the state, at once (one round trip to memory), then the early exit
    const int done = gs->done, n_leaves = gs->n_leaves, parent_slot = ROOT ? 0 : gs->parent_slot;
    const uint32_t gs_n = gs->n, gs_nl = gs->nl;
    const long long gs_gl = gs->gl, gs_hl = gs->hl, gs_PG = gs->PG, gs_PH = gs->PH;
    const long long tot_g = a.state->tot_g, tot_h = a.state->tot_h;
    const uint32_t gmax_bits = a.state->gmax_bits, hmax_bits = a.state->hmax_bits;
    const FeatRec fr = a.feat_rec[f];
    if (done) return;
    const size_t hw = (size_t)a.F * a.nb;

    // the two children: "small" was built by Algorithm 1, "large" is parent - small
    const uint32_t n = ROOT ? a.N : gs_n, nl = ROOT ? n : gs_nl, nr = n - nl;
    const bool small_is_left = nl <= nr;
    SplitParams pS = a.sp, pL = a.sp;
    if (ROOT) {
        pS.G = tot_g; pS.H = tot_h; pS.n_s = n;
    } else {
        const long long gl = gs_gl, hl = gs_hl, gr = gs_PG - gl, hr = gs_PH - hl;
        pS.G = small_is_left ? gl : gr; pS.H = small_is_left ? hl : hr; pS.n_s = small_is_left ? nl : nr;
        pL.G = small_is_left ? gr : gl; pL.H = small_is_left ? hr : hl; pL.n_s = small_is_left ? nr : nl;
    }
    // ---- phase A: one thread per bin: the smaller child's sum over the partial histograms, the
    //      larger child's bin by subtraction
    __shared__ SplitRec sm[2][FIN_WARPS];
    __shared__ bool is_last;
    // interval lengths of Eq. 5 from the maxima stored by the quantizer
    const double dg = __ddiv_rn((double)__uint_as_float(gmax_bits), (double)pS.kg);
    const double dh = pS.const_h ? 1.0 : __ddiv_rn((double)__uint_as_float(hmax_bits), (double)pS.kh);
    const double tpS = qg_gain_term(pS.G, pS.H, dg, dh, pS.lambda);
    const double tpL = ROOT ? 0.0 : qg_gain_term(pL.G, pL.H, dg, dh, pL.lambda);
    const int fl = fr.fl, W = 1 << fr.logW;
    const uint32_t P = ROOT ? 1u : effective_parts((uint32_t)fr.parts, (uint32_t)pS.n_s);
    const size_t pstride = (size_t)4 * a.nb * 32;
    const unsigned long long *part = a.partial + (size_t)fr.cta0 * pstride + (size_t)(fl & 3) * a.nb * W + (fl >> 2);
    unsigned long long *S = a.pool + (ROOT ? 0 : (size_t)n_leaves * hw) + (size_t)f * a.nb;
    unsigned long long *Pp = ROOT ? nullptr : a.pool + (size_t)parent_slot * hw + (size_t)f * a.nb;
    __shared__ long long wtot[4][FIN_WARPS];
    SplitRec rS = qg_invalid_rec(), rL = qg_invalid_rec();
    rS.feature = f;
    rL.feature = f;
    if (BPT == 1) {
        // n_bins <= 256: thread b owns bin b
        const int b = (int)threadIdx.x;
        unsigned long long s = 0, l = 0;
        if (b < a.nb) {
            if (ROOT) {
                s = S[b];
            } else {
                if (P > 1) {
                    const unsigned long long *q = part + (size_t)b * W;
                    for (uint32_t i0 = 0; i0 < P; i0 += 8) {   // 8 independent loads in flight
                        unsigned long long x[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) x[k] = i0 + k < P ? q[(size_t)(i0 + k) * pstride] : 0ull;
#pragma unroll
                        for (int k = 0; k < 8; ++k) s += x[k];
                    }
                    S[b] = s;
                } else {
                    s = S[b];
                }
                l = Pp[b] - s;   // no field borrows: every child sum is at most the parent's
                Pp[b] = l;
            }
        }
        // ---- phase B: prefix sums over the bins by all eight warps (warp scan, then the warp totals),
        //      every thread evaluates the threshold at its own bin for both children
        const bool in = b < a.nb - 1;   // thresholds 0 .. nb-2
        long long v[4];
        v[0] = in ? (long long)(int)(s >> 32) : 0;
        v[1] = in ? (long long)(unsigned int)(s & 0xFFFFFFFFull) : 0;
        v[2] = in ? (long long)(int)(l >> 32) : 0;
        v[3] = in ? (long long)(unsigned int)(l & 0xFFFFFFFFull) : 0;
#pragma unroll
        for (int c = 0; c < (ROOT ? 2 : 4); ++c) {
            for (int o = 1; o < 32; o <<= 1) {
                const long long u = __shfl_up_sync(0xffffffffu, v[c], o);
                if (lane >= o) v[c] += u;
            }
            if (lane == 31) wtot[c][warp] = v[c];
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < (ROOT ? 2 : 4); ++c)
            for (int w = 0; w < warp; ++w) v[c] += wtot[c][w];
        if (in) {
            double gain;
            if (qg_eval_candidate(v[0], v[1], pS, dg, dh, tpS, gain)) {
                rS.valid = 1; rS.gain = gain; rS.bin = b; rS.gl = v[0]; rS.hl = v[1];
            }
            if (!ROOT && qg_eval_candidate(v[2], v[3], pL, dg, dh, tpL, gain)) {
                rL.valid = 1; rL.gain = gain; rL.bin = b; rL.gl = v[2]; rL.hl = v[3];
            }
        }
    } else {
        // n_bins <= 256: thread t owns bins BPT t .. BPT t + BPT - 1
        unsigned long long sv[BPT], lv[BPT];
        {
            unsigned long long pv[BPT];
#pragma unroll
            for (int j = 0; j < BPT; ++j) {
                const int b = (int)threadIdx.x * BPT + j;
                sv[j] = 0; lv[j] = 0; pv[j] = 0;
                if (b < a.nb) {
                    if (!ROOT) pv[j] = Pp[b];
                    if (!ROOT && P > 1) {
                        const unsigned long long *q = part + (size_t)b * W;
                        for (uint32_t i0 = 0; i0 < P; i0 += 16) {   // 16 independent loads in flight
                            unsigned long long x[16];
#pragma unroll
                            for (int k = 0; k < 16; ++k) x[k] = i0 + k < P ? q[(size_t)(i0 + k) * pstride] : 0ull;
#pragma unroll
                            for (int k = 0; k < 16; ++k) sv[j] += x[k];
                        }
                    } else {
                        sv[j] = S[b];
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < BPT; ++j) {
                const int b = (int)threadIdx.x * BPT + j;
                if (!ROOT && b < a.nb) {
                    if (P > 1) S[b] = sv[j];
                    lv[j] = pv[j] - sv[j];   // no field borrows: every child sum is at most the parent's
                    Pp[b] = lv[j];
                }
            }
        }
        // ---- phase B: prefix sums over the bins by all warps (the thread's own bins, a warp scan of
        //      the threads' totals, then the warp totals); every thread evaluates the thresholds at its
        //      own bins for both children
        long long x[BPT][4], v[4] = {0, 0, 0, 0};   // per bin; v: inclusive sum up to the thread's last bin
#pragma unroll
        for (int j = 0; j < BPT; ++j) {
            const bool in = (int)threadIdx.x * BPT + j < a.nb - 1;   // thresholds 0 .. nb-2
            x[j][0] = in ? (long long)(int)(sv[j] >> 32) : 0;
            x[j][1] = in ? (long long)(unsigned int)(sv[j] & 0xFFFFFFFFull) : 0;
            x[j][2] = in ? (long long)(int)(lv[j] >> 32) : 0;
            x[j][3] = in ? (long long)(unsigned int)(lv[j] & 0xFFFFFFFFull) : 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) v[c] += x[j][c];
        }
#pragma unroll
        for (int c = 0; c < (ROOT ? 2 : 4); ++c) {
            for (int o = 1; o < 32; o <<= 1) {
                const long long u = __shfl_up_sync(0xffffffffu, v[c], o);
                if (lane >= o) v[c] += u;
            }
            if (lane == 31) wtot[c][warp] = v[c];
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < (ROOT ? 2 : 4); ++c)
            for (int w = 0; w < warp; ++w) v[c] += wtot[c][w];
        // thresholds from the thread's last bin down (the lower bin wins on equal gain)
#pragma unroll
        for (int j = BPT - 1; j >= 0; --j) {
            const int b = (int)threadIdx.x * BPT + j;
            if (b < a.nb - 1) {
                double gain;
                if (qg_eval_candidate(v[0], v[1], pS, dg, dh, tpS, gain) &&
                    qg_better(true, gain, b, rS.valid != 0, rS.gain, rS.bin)) {
                    rS.valid = 1; rS.gain = gain; rS.bin = b; rS.gl = v[0]; rS.hl = v[1];
                }
                if (!ROOT && qg_eval_candidate(v[2], v[3], pL, dg, dh, tpL, gain) &&
                    qg_better(true, gain, b, rL.valid != 0, rL.gain, rL.bin)) {
                    rL.valid = 1; rL.gain = gain; rL.bin = b; rL.gl = v[2]; rL.hl = v[3];
                }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) v[c] -= x[j][c];
        }
    }
    // best threshold of the feature: largest gain, lowest bin on equal gain
    for (int o = 16; o > 0; o >>= 1) {
        SplitRec x = rS, y = rL;
        x.gain = __shfl_xor_sync(0xffffffffu, rS.gain, o); y.gain = __shfl_xor_sync(0xffffffffu, rL.gain, o);
        x.gl = __shfl_xor_sync(0xffffffffu, rS.gl, o);     y.gl = __shfl_xor_sync(0xffffffffu, rL.gl, o);
        x.hl = __shfl_xor_sync(0xffffffffu, rS.hl, o);     y.hl = __shfl_xor_sync(0xffffffffu, rL.hl, o);
        x.bin = __shfl_xor_sync(0xffffffffu, rS.bin, o);   y.bin = __shfl_xor_sync(0xffffffffu, rL.bin, o);
        x.valid = __shfl_xor_sync(0xffffffffu, rS.valid, o); y.valid = __shfl_xor_sync(0xffffffffu, rL.valid, o);
        if (qg_better(x.valid != 0, x.gain, x.bin, rS.valid != 0, rS.gain, rS.bin)) rS = x;
        if (qg_better(y.valid != 0, y.gain, y.bin, rL.valid != 0, rL.gain, rL.bin)) rL = y;
    }
    if (lane == 0) { sm[0][warp] = rS; sm[1][warp] = rL; }
    __syncthreads();
    if (threadIdx.x < 2) {
        SplitRec r = sm[threadIdx.x][0];
        for (int w = 1; w < FIN_WARPS; ++w) {
            const SplitRec o = sm[threadIdx.x][w];
            if (qg_better(o.valid != 0, o.gain, o.bin, r.valid != 0, r.gain, r.bin)) r = o;
        }
        a.cand[2 * f + threadIdx.x] = r;
        __threadfence();
    }
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(&gs->finish_count, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // ---- the last block: best candidates over all features, the new leaves, the next pick.
    //      Every thread ends up with the same reduced values (warp shuffles, then the eight warp
    //      results from shared memory), so thread 0 needs no further round of barriers.
    const double NEG = -__longlong_as_double(0x7FF0000000000000LL);
    const int leaves_now = ROOT ? 1 : n_leaves + 1;
    // gains of the older leaves, fetched while the candidates are being reduced
    double my_gain[4];
#pragma unroll
    for (int k2 = 0; k2 < 4; ++k2) {
        const int i2 = (int)threadIdx.x + k2 * FIN_WARPS * 32;
        my_gain[k2] = i2 < leaves_now ? __ldcg(a.leaf_gain + i2) : NEG;
    }
    SplitRec bS = qg_invalid_rec(), bL = qg_invalid_rec();
    for (int i2 = threadIdx.x; i2 < (int)gridDim.x; i2 += FIN_WARPS * 32) {
        const SplitRec x = load_rec_cg(a.cand + 2 * i2), y = load_rec_cg(a.cand + 2 * i2 + 1);
        if (qg_rec_better(x, bS)) bS = x;
        if (qg_rec_better(y, bL)) bL = y;
    }
    for (int o = 16; o > 0; o >>= 1) {
        const SplitRec x = shfl_xor_rec(bS, o), y = shfl_xor_rec(bL, o);
        if (qg_rec_better(x, bS)) bS = x;
        if (qg_rec_better(y, bL)) bL = y;
    }
    if (lane == 0) { sm[0][warp] = bS; sm[1][warp] = bL; }
    __syncthreads();
    bS = sm[0][0];
    bL = sm[1][0];
    for (int w = 1; w < FIN_WARPS; ++w) {
        if (qg_rec_better(sm[0][w], bS)) bS = sm[0][w];
        if (qg_rec_better(sm[1][w], bL)) bL = sm[1][w];
    }
    // where the winning features live (needed if one of the new leaves is picked next)
    FeatRec fS = {}, fL = {};
    if (threadIdx.x == 0) {
        if (bS.valid) fS = a.feat_rec[bS.feature];
        if (!ROOT && bL.valid) fL = a.feat_rec[bL.feature];
    }
    // the leaves this split made (ROOT: only the root) and their gains
    const int id0 = ROOT ? 0 : gs->pick, id1 = ROOT ? -1 : n_leaves;
    const SplitRec best0 = ROOT ? bS : (small_is_left ? bS : bL);   // of leaf id0 (the left child)
    const SplitRec best1 = small_is_left ? bL : bS;                 // of leaf id1 (the right child)
    const double gain0 = best0.valid ? best0.gain : NEG, gain1 = best1.valid ? best1.gain : NEG;

    // the next leaf to split: largest gain, lowest leaf number on equal gain
    __shared__ double pg[FIN_WARPS];
    __shared__ int pi[FIN_WARPS];
    double bg = NEG;
    int bi = -1;
    if (leaves_now < a.L) {
#pragma unroll
        for (int k2 = 0; k2 < 4; ++k2) {
            const int i2 = (int)threadIdx.x + k2 * FIN_WARPS * 32;
            if (i2 < leaves_now) {
                double g = my_gain[k2];
                if (i2 == id0) g = gain0;
                if (i2 == id1) g = gain1;
                if (g > bg) { bg = g; bi = i2; }
            }
        }
        for (int i2 = (int)threadIdx.x + 4 * FIN_WARPS * 32; i2 < leaves_now; i2 += FIN_WARPS * 32) {   // more than 1024 leaves
            double g = __ldcg(a.leaf_gain + i2);
            if (i2 == id0) g = gain0;
            if (i2 == id1) g = gain1;
            if (g > bg) { bg = g; bi = i2; }
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const double og = __shfl_xor_sync(0xffffffffu, bg, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (oi >= 0 && (bi < 0 || og > bg || (og == bg && oi < bi))) { bg = og; bi = oi; }
    }
    if (lane == 0) { pg[warp] = bg; pi[warp] = bi; }
    __syncthreads();
    if (threadIdx.x != 0) return;
    bg = pg[0];
    bi = pi[0];
    for (int w = 1; w < FIN_WARPS; ++w) {
        const double og = pg[w];
        const int oi = pi[w];
        if (oi >= 0 && (bi < 0 || og > bg || (og == bg && oi < bi))) { bg = og; bi = oi; }
    }
    const int pick = bi;

    LeafRec lf, rt;   // ROOT: lf is the root
    if (ROOT) {
        lf.off = 0; lf.n = a.N; lf.buf = -1; lf.slot = 0; lf.G = pS.G; lf.H = pS.H; lf.best = bS;
        lf.parent_node = -1; lf.parent_side = 0;
        a.leaves[0] = lf;
        a.leaf_gain[0] = gain0;
        rt = lf;
        gs->n_leaves = 1;
    } else {
        const int right = n_leaves, node = n_leaves - 1;
        // node arrays of the tree being grown (the slot is device state: the launch arguments
        // are the same for every tree, so the launches can be replayed from a CUDA graph)
        const size_t no = (size_t)gs->tree_slot * (a.L > 1 ? a.L - 1 : 1);
        const int pn = gs->parent_node;
        a.m_feature[no + node] = gs->feature;
        a.m_bin[no + node] = gs->bin;
        a.m_left[no + node] = ~id0;
        a.m_right[no + node] = ~right;
        a.m_gain[no + node] = gs->gain;
        if (pn >= 0) {
            if (gs->parent_side == 0) a.m_left[no + pn] = node;
            else a.m_right[no + pn] = node;
        }
        const int dstbuf = gs->buf == 0 ? 1 : 0;
        lf.off = gs->off; lf.n = nl; lf.buf = dstbuf;
        lf.G = gs->gl; lf.H = gs->hl;
        lf.parent_node = node; lf.parent_side = 0;
        rt.off = gs->off + nl; rt.n = nr; rt.buf = dstbuf;
        rt.G = gs->PG - gs->gl; rt.H = gs->PH - gs->hl;
        rt.parent_node = node; rt.parent_side = 1;
        lf.slot = small_is_left ? n_leaves : gs->parent_slot;
        rt.slot = small_is_left ? gs->parent_slot : n_leaves;
        lf.best = best0;
        rt.best = best1;
        a.leaves[id0] = lf;
        a.leaves[right] = rt;
        a.leaf_gain[id0] = gain0;
        a.leaf_gain[right] = gain1;
        gs->n_leaves = n_leaves + 1;
        gs->hist_rows += small_is_left ? nl : nr;
        gs->hist_builds += 1;
    }
    gs->finish_count = 0;
    if (pick < 0) {
        gs->done = 1;
        return;
    }
    LeafRec lr;
    FeatRec pf;
    if (pick == id0) {
        lr = lf;
        pf = ROOT || small_is_left ? fS : fL;
    } else if (pick == id1) {
        lr = rt;
        pf = small_is_left ? fL : fS;
    } else {
        lr = a.leaves[pick];
        pf = a.feat_rec[lr.best.feature];
    }
    gs->pick = pick;
    gs->feature = lr.best.feature;
    gs->bin = lr.best.bin;
    gs->col = pf.col;
    gs->col8 = pf.col8;
    gs->logW = pf.logW;
    gs->byte = pf.byte;
    gs->off = lr.off;
    gs->n = lr.n;
    gs->buf = lr.buf;
    gs->gl = lr.best.gl;
    gs->hl = lr.best.hl;
    gs->PG = lr.G;
    gs->PH = lr.H;
    gs->gain = lr.best.gain;
    gs->parent_slot = lr.slot;
    gs->parent_node = lr.parent_node;
    gs->parent_side = lr.parent_side;
}

}  // namespace

namespace {

void fill_args(qgbdt_ctx *c, GrowArgs &a, int &part_blocks) {
    const int L = c->prm.num_leaves;
    a.gs = c->d_gs;
    a.leaves = c->d_leaves;
    a.state = c->d_state;
    a.feat_rec = c->d_feat_rec;
    a.leaf_gain = c->d_leaf_gain;
    a.N = (uint32_t)c->N;
    a.ent0 = c->d_ent0;
    a.ent1 = c->d_ent1;
    a.codes_nat = reinterpret_cast<const uint16_t *>(c->d_codes_nat);
    a.bits = c->d_part_bits;
    a.counts = c->d_part_counts;
    part_blocks = c->sm_count * 4;
    a.n_count = part_blocks * PART_WARPS;
    a.pool = c->d_hist_pool;
    a.partial = c->d_partial;
    a.cand = c->d_cand;
    a.F = c->F;
    a.nb = c->nb;
    a.L = L;
    a.sp.G = a.sp.H = a.sp.n_s = 0;
    a.sp.kg = qg_levels_g(c->prm.bits);
    a.sp.kh = qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    a.sp.const_h = c->const_hess ? 1 : 0;
    a.sp.min_data = c->prm.min_data_in_leaf;
    a.sp.min_sum_h = c->prm.min_sum_hessian;
    a.sp.min_gain = c->prm.min_gain;
    a.sp.lambda = c->prm.lambda_l2;
    a.m_feature = c->d_m_feature;
    a.m_bin = c->d_m_bin;
    a.m_left = c->d_m_left;
    a.m_right = c->d_m_right;
    a.m_gain = c->d_m_gain;
}

// The L - 1 splits of a tree: four kernels each, every size read from the grow state.
int enqueue_splits(qgbdt_ctx *c, const GrowArgs &a, int part_blocks, cudaStream_t st) {
    const unsigned fin_blocks = (unsigned)c->F;
    for (int split = 1; split < c->prm.num_leaves; ++split) {
        k_grow_flags<<<part_blocks, PART_THREADS, 0, st>>>(a);
        QG_LAUNCH_CHECK(c);
        k_grow_scatter<<<part_blocks, PART_THREADS, 0, st>>>(a);
        QG_LAUNCH_CHECK(c);
        const int rc = qg_hist_grow(c, st);
        if (rc != QGBDT_OK) return rc;
        if (c->F > c->sm_count * 8) k_grow_finish<false, 2><<<fin_blocks, 128, 0, st>>>(a);
        else k_grow_finish<false, 1><<<fin_blocks, 256, 0, st>>>(a);
        QG_LAUNCH_CHECK(c);
    }
    return QGBDT_OK;
}

}  // namespace

void qg_grow_graph_destroy(qgbdt_ctx *c) {
    if (c->grow_graph_exec) cudaGraphExecDestroy(reinterpret_cast<cudaGraphExec_t>(c->grow_graph_exec));
    c->grow_graph_exec = nullptr;
    c->grow_graph_launches = 0;
}

// The split loop of one tree as a CUDA graph (about a thousand launches whose arguments never
// change: what differs from tree to tree is device state).  Built once per context and objective;
// with the histogram event timers on, the launches go to the stream instead.
static int build_grow_graph(qgbdt_ctx *c, const GrowArgs &a, int part_blocks) {
    cudaStream_t cs = nullptr;
    QG_CUDA(c, cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking));
    const int64_t launches_before = c->n_launches;
    int rc = qg_hist_grow_configure(c);
    cudaGraph_t graph = nullptr;
    if (rc == QGBDT_OK) {
        cudaError_t e = cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal);
        if (e == cudaSuccess) {
            rc = enqueue_splits(c, a, part_blocks, cs);
            e = cudaStreamEndCapture(cs, &graph);
        }
        if (e != cudaSuccess || rc != QGBDT_OK || !graph) {
            cudaGetLastError();
            if (graph) cudaGraphDestroy(graph);
            cudaStreamDestroy(cs);
            c->n_launches = launches_before;
            return rc != QGBDT_OK ? rc : qg_fail(c, QGBDT_ERR_CUDA, "capturing the split loop failed: %s", cudaGetErrorString(e));
        }
        cudaGraphExec_t exec = nullptr;
        e = cudaGraphInstantiate(&exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) {
            cudaGetLastError();
            cudaStreamDestroy(cs);
            c->n_launches = launches_before;
            return qg_fail(c, QGBDT_ERR_CUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(e));
        }
        c->grow_graph_exec = exec;
        c->grow_graph_launches = c->n_launches - launches_before;
        c->grow_graph_const_hess = c->const_hess;
    }
    c->n_launches = launches_before;
    cudaStreamDestroy(cs);
    return rc;
}

// Grows the tree of boosting iteration slot `tree_slot` of the current train call.  Gradients must
// have been quantized on the same stream (the state holds the totals and maxima).  Asynchronous.
int qg_grow_tree(qgbdt_ctx *c, int tree_slot, cudaStream_t st) {
    GrowArgs a;
    int part_blocks;
    fill_args(c, a, part_blocks);
    k_grow_begin<<<1, 1, 0, st>>>(c->d_gs, c->d_leaves, c->d_state, (uint32_t)c->N, tree_slot);
    QG_LAUNCH_CHECK(c);
    int rc = qg_hist(c, nullptr, 0, c->N, c->d_hist_pool, st);   // root: all rows, contiguous
    if (rc != QGBDT_OK) return rc;
    k_grow_finish<true, 1><<<(unsigned)c->F, 256, 0, st>>>(a);
    QG_LAUNCH_CHECK(c);
    if (c->prm.num_leaves < 2) return QGBDT_OK;
    if (c->profile_hist) return enqueue_splits(c, a, part_blocks, st);   // event records around every build
    if (c->grow_graph_exec && c->grow_graph_const_hess != c->const_hess) qg_grow_graph_destroy(c);
    if (!c->grow_graph_exec && (rc = build_grow_graph(c, a, part_blocks)) != QGBDT_OK) return rc;
    QG_CUDA(c, cudaGraphLaunch(reinterpret_cast<cudaGraphExec_t>(c->grow_graph_exec), st));
    c->n_launches += c->grow_graph_launches;
    return QGBDT_OK;
}
