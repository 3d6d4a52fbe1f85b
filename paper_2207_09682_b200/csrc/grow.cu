// Leaf-wise (best-first) growth of one tree (Sec. 3) with every decision taken on the device.
//
// A tree grows in passes, several leaves per pass (the batch rule and the commit step that keeps
// the result equal to best-first growth are described with the structures in the internal header).
// Per pass, for all leaves of the batch at once:
//   (1) k_grow_flags    one predicate bit per row of a leaf being split, left rows per warp range;
//   (2) k_grow_scatter  stable scatter of the (row, gradient code) pairs into the other pair buffer
//                       (left rows first);
//   (3) the histogram kernel on the smaller child's rows (Algorithm 1);
//   (4) k_grow_finish   per feature: the smaller child's histogram from the partial histograms, the
//                       larger child's as parent minus smaller, both children's best splits (Eq. 7);
//                       the last block of a leaf writes the children's growth records;
//   (5) k_grow_commit   replays the best-first order over the leaves split so far (numbers the
//                       children, records the nodes), then picks the next batch and plans its launches.
// The passes of a tree are the body of a conditional (while) node of a CUDA graph: the commit kernel
// clears the node's condition when the tree is full or no leaf can be split, so the host enqueues one
// graph launch per tree and never waits for a result.
#include "split_scan.cuh"

namespace {

constexpr int PART_THREADS = 256;
constexpr int PART_WARPS = PART_THREADS / 32;
constexpr int COMMIT_THREADS = 1024;
struct GrowArgs {
    GrowState *gs;
    NodeRec *recs;
    double *rec_gain;                // per growth record: gain of its best split (-inf: none) ...
    int32_t *rec_child;              // ... first child record if it has been split, else -1 ...
    int32_t *rec_pos;                // ... (node << 1 | side) of its parent once it is numbered, else -1 ...
    int32_t *rec_parent;             // ... and the record it was split from (-1: the root)
    LeafRec *leaves;
    int32_t *front;                  // [L] growth record of every numbered leaf
    DevState *state;
    const FeatRec *feat_rec;         // [F]
    uint32_t N;                      // rows of this context
    uint32_t N_all;                  // rows over all ranks (= N unless the rows are sharded)
    int merged;                      // sharded rows: the smaller children's histograms were merged and summed over
                                     // the ranks before the finishing kernel, which then reads them as they are
    uint2 *ent0, *ent1;              // the two (row, gradient code) pair buffers
    const uint16_t *codes_nat;       // codes in row order (the root's identity list has no pairs yet)
    uint32_t *bits;                  // [jobs][bits_stride] predicate bits of the leaves being split
    size_t bits_stride;
    uint32_t *counts;                // [pb_total * PART_WARPS] left rows per warp range, then [pb_total] per block
    int pb_total;                    // blocks of a partition launch
    unsigned long long *pool;        // [slots][F][nb]
    unsigned long long *partial;       // per leaf of the batch and tile: sums of the smaller child's CTAs (zero between passes)
    JobPrep *prep;                   // [jobs] per-leaf constants (thousands of features: k_grow_prep writes them)
    SplitRec *cand;                  // [jobs][F][2] best candidates of every feature for the two children
    int F, nb, L;
    int K, slack;                    // leaves per pass; leaves that may be split ahead of their confirmation
    int xcap, parts_cap, n_tiles;    // histogram CTAs per tile of a launch, of one leaf; tiles
    uint32_t rows_min;               // rows per histogram CTA, at least (see qg_grow_parts)
    int max_recs, max_slots;         // growth records and histogram slots allocated
    SplitParams sp;                  // G, H, n_s are filled per leaf on the device
    // tree output (device arrays of the current train call)
    int32_t *m_feature, *m_bin, *m_left, *m_right;
    double *m_gain;
    cudaGraphConditionalHandle cond; // condition of the graph's while node
    int use_cond;
    int sep_reduce;                  // the best split over the features is taken by k_grow_reduce, not by the last
                                     // block of the finishing kernel                    // 0: launched on a stream, the host reads gs->done
};

__global__ void k_grow_begin(GrowState *gs, NodeRec *recs, double *rec_gain, int32_t *rec_child, int32_t *rec_pos,
                             LeafRec *leaves, int32_t *front, const DevState *state, uint32_t N, uint32_t N_all,
                             int tree_slot) {
    rec_gain[0] = -__longlong_as_double(0x7FF0000000000000LL);
    rec_child[0] = -1;
    rec_pos[0] = -1;
    gs->tree_slot = tree_slot;
    NodeRec r;
    r.off = 0; r.n = N; r.n_all = N_all; r.buf = -1; r.slot = 0;
    r.G = state->tot_g; r.H = state->tot_h;
    r.best = qg_invalid_rec();
    r.state = 0; r.child0 = -1; r.nl = 0;
    r.parent_node = -1; r.parent_side = 0;
    recs[0] = r;
    LeafRec l;
    l.off = 0; l.n = N; l.buf = -1; l.rec = 0; l.n_all = N_all; l.pad = 0;
    leaves[0] = l;
    front[0] = 0;
    gs->n_leaves = 1;
    gs->n_exec = 0;
    gs->n_recs = 1;
    gs->n_jobs = 0;
    // gradients out of domain (the flag is sticky over the trees of a train call): this tree stays
    // a single leaf, the call reports the error when it ends
    gs->done = state->bad_value ? 1 : 0;
    for (int j = 0; j < GROW_MAX_JOBS; ++j) { gs->jobs[j].finish_count = 0; gs->jobs[j].lb[0] = gs->jobs[j].lb[1] = 0; }
}

// Words of 32 rows [w0, w1) of warp gw: every warp takes the same number of consecutive words
// (at least 4), so the warps with work are a prefix [0, active) of the leaf's warps.
__device__ inline void warp_range(uint32_t nw, uint32_t gw, uint32_t n_count, uint32_t &w0, uint32_t &w1,
                                  uint32_t &active) {
    uint32_t per = (nw + n_count - 1) / n_count;
    if (per < 4) per = 4;
    active = (nw + per - 1) / per;
    w0 = gw * per < nw ? gw * per : nw;
    w1 = w0 + per < nw ? w0 + per : nw;
}

// The job whose block range [pb0, pb0 + pb) holds block b, or -1: lane i of the calling warp looks
// at job i.
__device__ inline int job_of_block(const GrowState *gs, int n_jobs, int b) {
    const int li = threadIdx.x & 31;
    const int p0 = gs->jobs[li].pb0, pn = gs->jobs[li].pb;
    const unsigned hit = __ballot_sync(0xffffffffu, li < n_jobs && b >= p0 && b < p0 + pn);
    return hit ? __ffs(hit) - 1 : -1;
}

// Four words of 32 rows at a time, so that the dependent loads (pair -> bin word) of the four are
// in flight together.
__global__ void __launch_bounds__(PART_THREADS) k_grow_flags(GrowArgs a) {
    const GrowState *gs = a.gs;
    const int done = gs->done, n_jobs = gs->n_jobs;
    const int j = job_of_block(gs, n_jobs, (int)blockIdx.x);
    if (done || j < 0) return;
    const GrowJob *job = gs->jobs + j;
    // every field at once (one round trip to memory)
    const int buf = job->buf, pb0 = job->pb0, pb = job->pb;
    const uint32_t n = job->n, off = job->off;
    const uint32_t *col = job->col;
    const uint8_t *col8 = job->col8;
    const int logW = job->logW, shift = 8 * job->byte;
    const uint32_t thr = (uint32_t)job->bin;
    const int lane = threadIdx.x & 31;
    const uint32_t lb = blockIdx.x - (uint32_t)pb0;                      // block inside the job
    const uint32_t gw = lb * PART_WARPS + (threadIdx.x >> 5);
    const uint32_t nw = (n + 31) >> 5;
    uint32_t w0, w1, active;
    warp_range(nw, gw, (uint32_t)pb * PART_WARPS, w0, w1, active);
    uint32_t *bits = a.bits + (size_t)j * a.bits_stride;
    uint32_t *wcounts = a.counts + (size_t)pb0 * PART_WARPS;
    uint32_t *bcounts = a.counts + (size_t)a.pb_total * PART_WARPS + pb0;
    if (lb * PART_WARPS >= active) return;                               // no warp of this block has work
    const uint2 *src = buf < 0 ? nullptr : (buf ? a.ent1 : a.ent0);
    uint32_t lefts = 0;
    uint32_t w = w0;
    // whole groups of eight words of 32 rows, all rows inside the leaf: no tests in the loop
    const uint32_t w_full = n >> 5;   // words below this one have 32 rows
    if (src && col8) {
        const uint2 *ps = src + off + lane;
        for (; w + 8 <= w1 && w + 8 <= w_full; w += 8) {
            uint32_t row[8], code[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) row[k] = ps[(size_t)(w + k) << 5].x;
#pragma unroll
            for (int k = 0; k < 8; ++k) code[k] = col8[row[k]];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t b = __ballot_sync(0xffffffffu, code[k] <= thr);
                if (lane == k) bits[w + k] = b;
                lefts += __popc(b);
            }
        }
    }
    for (; w < w1; w += 8) {
        uint32_t row[8], word[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t e = ((w + k) << 5) + lane;
            row[k] = (w + k < w1 && e < n) ? (src ? src[off + e].x : off + e) : 0xFFFFFFFFu;
        }
        // the bin code of the split feature: one byte of the column-major copy (ascending rows share
        // DRAM granules), or, without that copy, a word of the tile (a granule per row)
        if (col8) {
#pragma unroll
            for (int k = 0; k < 8; ++k) word[k] = row[k] != 0xFFFFFFFFu ? (uint32_t)col8[row[k]] << shift : 0xFFFFFFFFu;
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) word[k] = row[k] != 0xFFFFFFFFu ? col[(size_t)row[k] << logW] : 0xFFFFFFFFu;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const bool left = row[k] != 0xFFFFFFFFu && ((word[k] >> shift) & 0xFFu) <= thr;
            const uint32_t b = __ballot_sync(0xffffffffu, left);
            if (w + k < w1) {
                if (lane == 0) bits[w + k] = b;
                lefts += __popc(b);
            }
        }
    }
    // left rows of every warp range and of every block's ranges (the scatter kernel adds up the
    // blocks before its own and the warps before it inside its block)
    __shared__ uint32_t block_lefts[PART_WARPS];
    if (lane == 0) {
        wcounts[gw] = lefts;
        block_lefts[threadIdx.x >> 5] = lefts;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
#pragma unroll
        for (int v = 0; v < PART_WARPS; ++v) t += block_lefts[v];
        bcounts[lb] = t;
    }
}

__global__ void __launch_bounds__(PART_THREADS) k_grow_scatter(GrowArgs a) {
    GrowState *gs = a.gs;
    const int done = gs->done, n_jobs = gs->n_jobs;
    const int j = job_of_block(gs, n_jobs, (int)blockIdx.x);
    if (done || j < 0) return;
    GrowJob *job = gs->jobs + j;
    const int buf = job->buf, pb0 = job->pb0, pb = job->pb;   // every field at once
    const uint32_t n = job->n, off = job->off;
    const int lane = threadIdx.x & 31;
    const uint32_t lb = blockIdx.x - (uint32_t)pb0;
    const uint32_t gw = lb * PART_WARPS + (threadIdx.x >> 5);
    const uint32_t nw = (n + 31) >> 5;
    uint32_t w0, w1, active;
    warp_range(nw, gw, (uint32_t)pb * PART_WARPS, w0, w1, active);
    if (gw >= active && gw != 0) return;
    const uint32_t *bits = a.bits + (size_t)j * a.bits_stride;
    const uint32_t *wcounts = a.counts + (size_t)pb0 * PART_WARPS;
    const uint32_t *block_counts = a.counts + (size_t)a.pb_total * PART_WARPS + pb0;
    // left rows before this warp's range, and in the whole leaf: the totals of the blocks, and
    // the warps of this block before this one
    uint32_t before = 0, total = 0;
    const uint32_t active_blocks = (active + PART_WARPS - 1) / PART_WARPS;
    for (uint32_t j0 = 0; j0 < active_blocks; j0 += 256) {   // eight independent loads per lane in flight
        uint32_t v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t jj = j0 + 32 * k + lane;
            v[k] = jj < active_blocks ? block_counts[jj] : 0u;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            total += v[k];
            if (j0 + 32 * k + lane < lb) before += v[k];
        }
    }
    {
        const uint32_t jj = lb * PART_WARPS + lane;
        if (lane < PART_WARPS && jj < gw && jj < active) before += wcounts[jj];
    }
    for (int o = 16; o > 0; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if (gw == 0 && lane == 0) {
        job->nl = total;
        gs->nl_all[j] = (long long)total;   // sharded rows: summed over the ranks before the histograms
    }
    const uint2 *src = buf < 0 ? nullptr : (buf ? a.ent1 : a.ent0);
    uint2 *dst = buf == 0 ? a.ent1 : a.ent0;
    uint32_t w = w0;
    const uint32_t w_full = n >> 5;   // words below this one have 32 rows
    if (src) {
        // whole groups of four words, all rows inside the leaf: no tests in the loop
        const uint2 *ps = src + off + lane;
        uint2 *pd = dst + off;
        const uint32_t below = (1u << lane) - 1u;
        for (; w + 4 <= w1 && w + 4 <= w_full; w += 4) {
            uint32_t bw[4];
            uint2 ent[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                bw[k] = bits[w + k];
                ent[k] = ps[(size_t)(w + k) << 5];
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t rank_l = __popc(bw[k] & below);
                const bool left = (bw[k] >> lane) & 1u;
                // left rows keep their order at the front; right rows theirs behind all `total` left rows
                const uint32_t dest = left ? before + rank_l : total + (((w + k) << 5) - before) + (lane - rank_l);
                pd[dest] = ent[k];
                before += __popc(bw[k]);
            }
        }
    }
    for (; w < w1; w += 4) {
        uint32_t bw[4];
        uint2 ent[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = ((w + k) << 5) + lane;
            bw[k] = w + k < w1 ? bits[w + k] : 0u;
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

// Floats as unsigned integers of the same order (every such integer is at least 1: 0 can stand for "none").
__device__ __forceinline__ unsigned int float_order_bits(float f) {
    const unsigned int u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float order_bits_float(unsigned int k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Best threshold of a warp: every lane brings its best (gain, bin >= 0, packed left sums) or bin < 0;
// all lanes return the warp's best (largest gain, lowest bin on equal gain; bin < 0: none).
__device__ __forceinline__ void warp_best(double &gain, int &bin, unsigned long long &w) {
    if (!__any_sync(0xffffffffu, bin >= 0)) return;
    double g = gain;
    int b = bin;
    for (int o = 16; o > 0; o >>= 1) {
        const double og = __shfl_xor_sync(0xffffffffu, g, o);
        const int ob = __shfl_xor_sync(0xffffffffu, b, o);
        if (qg_better(ob >= 0, og, ob, b >= 0, g, b)) { g = og; b = ob; }
    }
    // the bins of the lanes are distinct: the lane that brought the winning bin owns the sums
    const unsigned int owner = __ballot_sync(0xffffffffu, bin == b);
    w = __shfl_sync(0xffffffffu, w, __ffs(owner) - 1);
    gain = g;
    bin = b;
}

// What a warp of the finishing kernel leaves for the block's first thread.
struct WarpBest {
    double gain;
    unsigned long long w;
    int bin, pad;
};

constexpr int FIN_THREADS = 128, FIN_WARPS = FIN_THREADS / 32, FIN_BLOCKS_PER_SM = 8;

// Last step for one leaf being split (ROOT: for the root), by one block once every feature's best
// thresholds are written: the best over all features (lowest feature on equal gain), then the growth
// records of the two children (ROOT: the root's best split).
struct TailIn {   // what the step needs of the job, read before the wait for the other blocks
    int parent_slot, small_slot, child0, rec, buf;
    uint32_t n, nl, off, n_all, nl_all;
    long long gl, hl, PG, PH;
};
__device__ __forceinline__ TailIn tail_in(const GrowState *gs, int j) {
    const GrowJob *job = gs->jobs + j;
    TailIn t;
    t.parent_slot = job->parent_slot; t.small_slot = job->small_slot; t.child0 = job->child0; t.rec = job->rec; t.buf = job->buf;
    t.n = job->n; t.nl = job->nl; t.off = job->off; t.n_all = job->n_all; t.nl_all = (uint32_t)gs->nl_all[j];
    t.gl = job->gl; t.hl = job->hl; t.PG = job->PG; t.PH = job->PH;
    return t;
}
template <bool ROOT>
__device__ __forceinline__ void finish_tail(const GrowArgs &a, const int j, const TailIn &t) {
    __threadfence();
    GrowState *gs = a.gs;
    GrowJob *job = gs->jobs + j;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const SplitRec *cand = a.cand + (size_t)j * a.F * 2;
    __shared__ SplitRec fin_rec[2][FIN_WARPS];
    SplitRec bS = qg_invalid_rec(), bL = qg_invalid_rec();
    for (int i2 = threadIdx.x; i2 < a.F; i2 += FIN_THREADS) {
        const SplitRec x = load_rec_cg(cand + 2 * i2), y = load_rec_cg(cand + 2 * i2 + 1);
        if (qg_rec_better(x, bS)) bS = x;
        if (qg_rec_better(y, bL)) bL = y;
    }
    for (int o = 16; o > 0; o >>= 1) {
        const SplitRec x = shfl_xor_rec(bS, o), y = shfl_xor_rec(bL, o);
        if (qg_rec_better(x, bS)) bS = x;
        if (qg_rec_better(y, bL)) bL = y;
    }
    if (lane == 0) { fin_rec[0][warp] = bS; fin_rec[1][warp] = bL; }
    __syncthreads();
    if (threadIdx.x != 0) return;
    bS = fin_rec[0][0];
    bL = fin_rec[1][0];
    for (int w = 1; w < FIN_WARPS; ++w) {
        if (qg_rec_better(fin_rec[0][w], bS)) bS = fin_rec[0][w];
        if (qg_rec_better(fin_rec[1][w], bL)) bL = fin_rec[1][w];
    }
    job->finish_count = 0;
    job->lb[0] = job->lb[1] = 0;
    const double NEG = -__longlong_as_double(0x7FF0000000000000LL);
    if (ROOT) {
        a.recs[0].best = bS;
        a.rec_gain[0] = bS.valid ? bS.gain : NEG;
        return;
    }
    const int parent_slot = t.parent_slot, small_slot = t.small_slot;
    const int child0 = t.child0, jrec = t.rec;
    const uint32_t nl = t.nl, nr = t.n - nl, off = t.off;
    const uint32_t nl_all = t.nl_all, nr_all = t.n_all - nl_all;
    const long long gl = t.gl, hl = t.hl;
    const bool small_is_left = nl_all <= nr_all;
    const int dstbuf = t.buf == 0 ? 1 : 0;
    NodeRec lf, rt;
    lf.off = off; lf.n = nl; lf.n_all = nl_all; lf.buf = dstbuf;
    lf.G = gl; lf.H = hl;
    rt.off = off + nl; rt.n = nr; rt.n_all = nr_all; rt.buf = dstbuf;
    rt.G = t.PG - gl; rt.H = t.PH - hl;
    lf.slot = small_is_left ? small_slot : parent_slot;
    rt.slot = small_is_left ? parent_slot : small_slot;
    lf.best = small_is_left ? bS : bL;
    rt.best = small_is_left ? bL : bS;
    lf.state = rt.state = 0;
    lf.child0 = rt.child0 = -1;
    lf.nl = rt.nl = 0;
    lf.parent_node = rt.parent_node = -1;
    lf.parent_side = 0; rt.parent_side = 1;
    a.recs[child0] = lf;
    a.recs[child0 + 1] = rt;
    a.recs[jrec].nl = nl;
    a.rec_gain[child0] = lf.best.valid ? lf.best.gain : NEG;
    a.rec_gain[child0 + 1] = rt.best.valid ? rt.best.gain : NEG;
    a.rec_child[child0] = a.rec_child[child0 + 1] = -1;
    a.rec_pos[child0] = a.rec_pos[child0 + 1] = -1;
    a.rec_parent[child0] = a.rec_parent[child0 + 1] = jrec;
}

// One feature of one leaf being split (ROOT: of the root): the work of a block of k_grow_finish.
// 128 threads, thread t owns bins 2 t and 2 t + 1 (n_bins <= 256).  A bin is one 64-bit word, the
// gradient sum in the upper half and the hessian sum in the lower; the sums of a whole leaf fit the
// halves (checked when the rows are loaded), so prefix sums are taken on the words themselves.
template <bool ROOT, bool SEP>
__device__ __forceinline__ void finish_one(const GrowArgs &a, const int f, const int j) {
    GrowState *gs = a.gs;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    GrowJob *job = gs->jobs + j;
    // everything the block needs from the state, at once (one round trip to memory)
    const int parts = job->parts, slot0 = job->slot0;
    const TailIn ti = tail_in(gs, j);
    const int parent_slot = ROOT ? 0 : ti.parent_slot, small_slot = ROOT ? 0 : ti.small_slot;
    constexpr bool sep_reduce = SEP;   // k_grow_reduce takes the last step
    const FeatRec fr = a.feat_rec[f];
    const size_t hw = (size_t)a.F * a.nb;

    // the two children: "small" was built by Algorithm 1, "large" is parent - small.  Which child is
    // "small" and every row count that enters the split search are the ones over all ranks.  What is
    // the same for every feature of the leaf comes from the histogram kernel of the pass (ROOT: is
    // worked out here).
    SplitParams pS = a.sp, pL = a.sp;
    double dg, dh, tpS, tpL = 0.0;
    Admit32 aS, aL;
    bool small_is_left = true;
    uint32_t P = 1u;
    if (ROOT) {
        pS.G = a.state->tot_g; pS.H = a.state->tot_h; pS.n_s = a.N_all;
        qg_scales(a.state, pS, dg, dh);   // interval lengths of Eq. 5 from the maxima stored by the quantizer
        tpS = qg_gain_term(pS.G, pS.H, dg, dh, pS.lambda);
        aS = qg_admit32(pS, dh);
        aL = aS;
    } else {
        // thousands of features: worked out once per leaf by k_grow_prep; else here, for every feature
        const JobPrep pr = SEP ? a.prep[j] : qg_job_prep(gs, j, a.state, a.sp, a.rows_min);
        dg = pr.dg; dh = pr.dh; tpS = pr.tpS; tpL = pr.tpL;
        aS = pr.aS; aL = pr.aL;
        small_is_left = pr.small_is_left != 0;
        P = a.merged ? 1u : pr.P;
        pS.G = aS.G; pS.H = aS.H; pS.n_s = aS.n_s;
        pL.G = aL.G; pL.H = aL.H; pL.n_s = aL.n_s;
    }
    __shared__ WarpBest sm[2][FIN_WARPS];
    __shared__ bool is_last;
    __shared__ unsigned long long wtot[2][FIN_WARPS];
    GainScale sc;
    sc.dg = (float)dg; sc.dh = (float)dh; sc.lambda = (float)pS.lambda;

    // ---- phase A: the smaller child's bins summed over the partial histograms, the larger child's
    //      by subtraction from the parent's
    const int fl = fr.fl, W = 1 << fr.logW;
    const size_t pstride = (size_t)4 * a.nb * 32;
    unsigned long long *part = a.partial + (size_t)(slot0 + fr.tile * parts) * pstride +
                               (size_t)(fl & 3) * a.nb * W + (fl >> 2);
    unsigned long long *S = a.pool + (size_t)small_slot * hw + (size_t)f * a.nb;
    unsigned long long *Pp = ROOT ? nullptr : a.pool + (size_t)parent_slot * hw + (size_t)f * a.nb;
    unsigned long long sv[2], lv[2];
    {
        unsigned long long pv[2];
#pragma unroll
        for (int jb = 0; jb < 2; ++jb) {
            const int b = (int)threadIdx.x * 2 + jb;
            sv[jb] = 0; lv[jb] = 0; pv[jb] = 0;
            if (b < a.nb) {
                if (!ROOT) pv[jb] = Pp[b];
                if (!ROOT && P > 1 && fr.logW < QG_SHARED_PARTIAL_LOGW) {
                    // the CTAs of the tile added their sums into its first partial slot: take them, leave zero
                    unsigned long long *q = part + (size_t)b * W;
                    sv[jb] = *q;
                    *q = 0ull;
                } else if (!ROOT && P > 1) {
                    const unsigned long long *q = part + (size_t)b * W;
                    for (uint32_t i0 = 0; i0 < P; i0 += 16) {   // 16 independent loads in flight
                        unsigned long long x[16];
#pragma unroll
                        for (int k = 0; k < 16; ++k) x[k] = i0 + k < P ? q[(size_t)(i0 + k) * pstride] : 0ull;
#pragma unroll
                        for (int k = 0; k < 16; ++k) sv[jb] += x[k];
                    }
                } else {
                    sv[jb] = S[b];
                }
            }
        }
#pragma unroll
        for (int jb = 0; jb < 2; ++jb) {
            const int b = (int)threadIdx.x * 2 + jb;
            if (!ROOT && b < a.nb) {
                if (P > 1) S[b] = sv[jb];
                lv[jb] = pv[jb] - sv[jb];   // no field borrows: every child sum is at most the parent's
                Pp[b] = lv[jb];
            }
        }
    }
    // ---- phase B: prefix sums over the bins (the thread's two bins, a warp scan of the threads'
    //      totals, then the totals of the warps before); thresholds are the bins 0 .. nb-2
    const int b0 = (int)threadIdx.x * 2;
    const bool in0 = b0 < a.nb - 1, in1 = b0 + 1 < a.nb - 1;
    const unsigned long long xS1 = in1 ? sv[1] : 0ull, xL1 = in1 ? lv[1] : 0ull;
    unsigned long long vS = (in0 ? sv[0] : 0ull) + xS1, vL = (in0 ? lv[0] : 0ull) + xL1;
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long uS = __shfl_up_sync(0xffffffffu, vS, o);
        if (lane >= o) vS += uS;
        if (!ROOT) {
            const unsigned long long uL = __shfl_up_sync(0xffffffffu, vL, o);
            if (lane >= o) vL += uL;
        }
    }
    if (lane == 31) { wtot[0][warp] = vS; wtot[1][warp] = vL; }
    __syncthreads();
    for (int w = 0; w < warp; ++w) { vS += wtot[0][w]; vL += wtot[1][w]; }
    // inclusive sums at the thread's bins: [1] at bin b0 + 1, [0] at bin b0
    const unsigned long long pS2[2] = {vS - xS1, vS}, pL2[2] = {vL - xL1, vL};

    // ---- phase C: cheap single-precision bounds on every admissible threshold's gain; the exact gain
    //      (two double-precision divisions) only where the upper bound reaches the largest lower bound
    //      the warp knows of: its own, and the largest any warp working on this leaf has published so
    //      far, whatever its feature.  A threshold whose upper bound lies below a lower bound has a
    //      strictly smaller gain than some admissible threshold of the leaf and cannot be its best
    //      (which warps came first changes the work, never the result).
    const float NEGF = -__int_as_float(0x7f800000);
    bool okS[2], okL[2];
    float hiS[2], hiL[2], mS = NEGF, mL = NEGF;
#pragma unroll
    for (int jb = 0; jb < 2; ++jb) {
        const bool in = jb == 0 ? in0 : in1;
        const int glS = (int)(pS2[jb] >> 32), glL = (int)(pL2[jb] >> 32);
        const uint32_t hlS = (uint32_t)pS2[jb], hlL = (uint32_t)pL2[jb];
        okS[jb] = in && qg_admissible32(hlS, aS, sc);
        okL[jb] = !ROOT && in && qg_admissible32(hlL, aL, sc);
        float lo;
        hiS[jb] = hiL[jb] = NEGF;
        if (okS[jb]) { qg_gain_bounds32(glS, hlS, aS, sc, (float)tpS, lo, hiS[jb]); mS = fmaxf(mS, lo); }
        if (okL[jb]) { qg_gain_bounds32(glL, hlL, aL, sc, (float)tpL, lo, hiL[jb]); mL = fmaxf(mL, lo); }
    }
    for (int o = 16; o > 0; o >>= 1) {
        mS = fmaxf(mS, __shfl_xor_sync(0xffffffffu, mS, o));
        if (!ROOT) mL = fmaxf(mL, __shfl_xor_sync(0xffffffffu, mL, o));
    }
    if (lane < (ROOT ? 1 : 2)) {
        const unsigned int mine = float_order_bits(lane == 0 ? mS : mL);
        unsigned int seen = *reinterpret_cast<volatile unsigned int *>(&job->lb[lane]);
        if (mine > seen) seen = max(atomicMax(&job->lb[lane], mine), mine);
        mS = order_bits_float(seen);   // lane 0: smaller child, lane 1: larger child
    }
    mL = __shfl_sync(0xffffffffu, mS, 1);
    mS = __shfl_sync(0xffffffffu, mS, 0);
    double gS = 0.0, gL = 0.0;
    int binS = -1, binL = -1;
    unsigned long long wS = 0, wL = 0;
    // thresholds from the thread's upper bin down (the lower bin wins on equal gain)
#pragma unroll
    for (int jb = 1; jb >= 0; --jb) {
        if (okS[jb] && hiS[jb] >= mS) {
            const double gain = qg_candidate_gain((long long)(int)(pS2[jb] >> 32), (long long)(uint32_t)pS2[jb], pS, dg, dh, tpS);
            if (gain > pS.min_gain && (binS < 0 || gain >= gS)) { gS = gain; binS = b0 + jb; wS = pS2[jb]; }
        }
        if (okL[jb] && hiL[jb] >= mL) {
            const double gain = qg_candidate_gain((long long)(int)(pL2[jb] >> 32), (long long)(uint32_t)pL2[jb], pL, dg, dh, tpL);
            if (gain > pL.min_gain && (binL < 0 || gain >= gL)) { gL = gain; binL = b0 + jb; wL = pL2[jb]; }
        }
    }
    // best threshold of the feature: largest gain, lowest bin on equal gain
    warp_best(gS, binS, wS);
    if (!ROOT) warp_best(gL, binL, wL);
    if (lane == 0) {
        sm[0][warp].gain = gS; sm[0][warp].bin = binS; sm[0][warp].w = wS;
        sm[1][warp].gain = gL; sm[1][warp].bin = binL; sm[1][warp].w = wL;
    }
    __syncthreads();
    SplitRec *cand = a.cand + (size_t)j * a.F * 2;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            WarpBest r = sm[c][0];
            for (int w = 1; w < FIN_WARPS; ++w) {
                const WarpBest o = sm[c][w];
                if (qg_better(o.bin >= 0, o.gain, o.bin, r.bin >= 0, r.gain, r.bin)) r = o;
            }
            SplitRec x = qg_invalid_rec();
            x.feature = f;
            if (r.bin >= 0) { x.valid = 1; x.gain = r.gain; x.bin = r.bin; x.gl = (long long)(int)(r.w >> 32); x.hl = (long long)(uint32_t)r.w; }
            cand[2 * f + c] = x;
        }
        if (!sep_reduce) {
            __threadfence();
            is_last = atomicAdd(&job->finish_count, 1u) == (unsigned int)a.F - 1u;
        }
    }
    if (sep_reduce) return;   // k_grow_reduce follows
    __syncthreads();
    if (is_last) finish_tail<ROOT>(a, j, ti);
}

// ROOT: scans the root histogram (pool slot 0), one block per feature.  Otherwise: completes the
// splits of the current pass: the (leaf, feature) pairs of the batch, leaf-major, are dealt round-robin
// to a grid sized to what the SMs hold at once, so that every block gets the same number of pairs to
// within one, whatever the batch size.
template <bool ROOT, bool SEP>
__global__ void __launch_bounds__(FIN_THREADS, FIN_BLOCKS_PER_SM) k_grow_finish(GrowArgs a) {
    if (a.gs->done) return;
    if (ROOT) {
        finish_one<ROOT, SEP>(a, (int)blockIdx.x, 0);
        return;
    }
    const int items = a.gs->n_jobs * a.F;
    for (int it = (int)blockIdx.x; it < items; it += (int)gridDim.x) {
        const int j = it / a.F;
        // the shared arrays of finish_one need no barrier in between: each is last read before a
        // barrier that every thread passes before the next leaf's first write to it
        finish_one<ROOT, SEP>(a, it - j * a.F, j);
    }
}

// With thousands of features: lane j works out what is the same for all features of leaf j, once, before
// the finishing kernel (one warp).
__global__ void __launch_bounds__(32) k_grow_prep(GrowArgs a) {
    if (a.gs->done || (int)threadIdx.x >= a.gs->n_jobs) return;
    a.prep[threadIdx.x] = qg_job_prep(a.gs, (int)threadIdx.x, a.state, a.sp, a.rows_min);
}

// With thousands of features the last step runs as a kernel of its own, one block per leaf of the
// batch: left to whichever block of the finishing kernel comes last, a block that has fallen behind
// takes that step for one leaf after the other and falls further behind each time.
__global__ void __launch_bounds__(FIN_THREADS) k_grow_reduce(GrowArgs a) {
    if (a.gs->done || (int)blockIdx.x >= a.gs->n_jobs) return;
    finish_tail<false>(a, (int)blockIdx.x, tail_in(a.gs, (int)blockIdx.x));
}

// Sharded rows only: sums the partial histograms of every smaller child of the pass into its pool
// slot, so that the slots can be added over the ranks before the finishing kernel.  Grid (F, Y) like
// the finishing kernel, one thread per bin.
__global__ void __launch_bounds__(256) k_grow_merge(GrowArgs a) {
    const GrowState *gs = a.gs;
    const int f = blockIdx.x;
    const int done = gs->done, n_jobs = gs->n_jobs;
    const FeatRec fr = a.feat_rec[f];
    if (done) return;
    for (int j = (int)blockIdx.y; j < n_jobs; j += (int)gridDim.y) {   // the leaves y, y + Y, ... of the batch
        const GrowJob *job = gs->jobs + j;
        const int small_slot = job->small_slot, parts = job->parts, slot0 = job->slot0;
        const uint32_t n = job->n, nl = job->nl, n_all = job->n_all, nl_all = (uint32_t)gs->nl_all[j];
        const bool small_is_left = nl_all <= n_all - nl_all;
        const uint32_t P = qg_grow_parts((uint32_t)parts, small_is_left ? nl : n - nl, a.rows_min);
        if (P <= 1) continue;   // a single CTA wrote the slot itself
        const int fl = fr.fl, W = 1 << fr.logW;
        const size_t pstride = (size_t)4 * a.nb * 32;
        unsigned long long *part = a.partial + (size_t)(slot0 + fr.tile * parts) * pstride +
                                   (size_t)(fl & 3) * a.nb * W + (fl >> 2);
        unsigned long long *S = a.pool + (size_t)small_slot * a.F * a.nb + (size_t)f * a.nb;
        for (int b = threadIdx.x; b < a.nb; b += 256) {
            unsigned long long *q = part + (size_t)b * W;
            unsigned long long v = 0;
            if (fr.logW < QG_SHARED_PARTIAL_LOGW) {   // one slot holds the sum: take it, leave zero
                v = *q;
                *q = 0ull;
            } else {
                for (uint32_t i0 = 0; i0 < P; i0 += 8) {
                    unsigned long long x[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) x[k] = i0 + k < P ? q[(size_t)(i0 + k) * pstride] : 0ull;
#pragma unroll
                    for (int k = 0; k < 8; ++k) v += x[k];
                }
            }
            S[b] = v;
        }
    }
}

// Shared memory of the commit kernel.  A region that first holds, per numbered leaf, its gain, its
// growth record and the list of splits confirmed in this launch, and later the compacted list of
// the records whose split is not confirmed (the gain that orders them, the record, and the records
// by rank); then, per growth record, its gain, its children (or -1) and its place in the tree.
// Records whose split may be open at once (at least the 1024 entries the sort pads to; a multiple of
// four so that the arrays behind one another stay 16-byte aligned).
__host__ __device__ inline int commit_max_cand(int L) {
    const int n = L + 2 * GROW_SLACK + 2 * GROW_MAX_JOBS + 8;
    return n < 1024 ? 1024 : (n + 3) & ~3;
}
__host__ __device__ inline size_t commit_region_bytes(int L) {
    const size_t a = (size_t)L * (sizeof(double) + 3 * sizeof(int));
    const size_t n = (size_t)commit_max_cand(L);
    const size_t b = n * (sizeof(double) + 2 * sizeof(int)) + 1024 * (sizeof(double) + sizeof(int));   // + the sort's second buffer
    return ((a > b ? a : b) + 15) / 16 * 16;
}
__host__ __device__ inline size_t commit_smem_bytes(int L, int max_recs) {
    return commit_region_bytes(L) + (size_t)max_recs * (sizeof(double) + 2 * sizeof(int)) + 16;
}

// Doubles as unsigned keys of the same order (-inf is the smallest key of a real gain; 0 is below all).
__device__ inline unsigned long long gain_key(double g) {
    const long long b = __double_as_longlong(g);
    return (unsigned long long)(b ^ ((b >> 63) | (long long)0x8000000000000000ULL));
}

// One block.  (1) Replays best-first growth over what has been split so far: takes the numbered
// leaf with the largest gain (lowest number on equal gain); if it has been split, numbers its
// children (the left child keeps the number, the right child gets the next one), records the node
// and goes on; stops at a leaf that has not been split yet, at a full tree, or when no leaf has an
// admissible split.  (2) Picks the next batch: that leaf, then the unsplit leaves of largest gain
// among all growth records.  (3) Fills the job table and shares out the blocks of the next launches.
__global__ void __launch_bounds__(COMMIT_THREADS) k_grow_commit(GrowArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    GrowState *gs = a.gs;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const double NEG = -__longlong_as_double(0x7FF0000000000000LL);
    if (gs->done) {
        if (tid == 0) {
            gs->n_jobs = 0;
            if (a.use_cond) cudaGraphSetConditional(a.cond, 0);
        }
        return;
    }
    const int L = a.L, R = a.max_recs;
    // the region, first use
    double *fg = reinterpret_cast<double *>(smem_raw);          // [L] gain of numbered leaf i
    int *sf = reinterpret_cast<int *>(fg + L);                  // [L] record of numbered leaf i
    int *cl_rec = sf + L;                                       // [L] confirmed in this launch: the record split ...
    int *cl_leaf = cl_rec + L;                                  // [L] ... and the number of the leaf it was
    // the region, second use
    const int max_cand = commit_max_cand(L);
    unsigned long long *cand_k = reinterpret_cast<unsigned long long *>(smem_raw);   // [max_cand] ordering keys of the open records
    int *cand_r = reinterpret_cast<int *>(cand_k + max_cand);   // [max_cand] the records
    // per record
    double *cg = reinterpret_cast<double *>(smem_raw + commit_region_bytes(L));   // [R]
    int *cs = reinterpret_cast<int *>(cg + R);                  // [R] first child record of a split record, else -1
    int *spn = cs + R;                                          // [R] (node << 1 | side) of a numbered record's parent, -1
    __shared__ int s_done, s_leaves, s_mand, s_commits, s_ncand;
    __shared__ unsigned long long s_rows;
    __shared__ int s_pick[GROW_MAX_JOBS];

    const int n_leaves0 = gs->n_leaves, n_recs = gs->n_recs, n_exec = gs->n_exec, tree_slot = gs->tree_slot;
    for (int r = tid; r < n_recs; r += COMMIT_THREADS) {
        cg[r] = a.rec_gain[r];
        cs[r] = a.rec_child[r];
        spn[r] = a.rec_pos[r];
    }
    for (int i = tid; i < n_leaves0; i += COMMIT_THREADS) sf[i] = a.front[i];
    if (tid == 0) { s_rows = 0; s_ncand = 0; }
    __syncthreads();
    for (int i = tid; i < n_leaves0; i += COMMIT_THREADS) fg[i] = cg[sf[i]];
    __syncthreads();

    // ---- (1) warp 0 replays the best-first order.  Lane l keeps the best of the leaves l, l + 32, ...
    //      and looks at them again only when one of them changes.  Up to 256 leaves the keys of a
    //      lane's leaves stay in its registers (the replay is one long chain of dependent steps: every
    //      shared-memory round trip taken out of it counts); beyond, in the shared array.
    if (warp == 0) {
        constexpr int RS = 8;
        const bool reg_keys = L <= 32 * RS;
        int n_leaves = n_leaves0, mand = -1, done = 0, commits = 0;
        unsigned long long lk = 0;   // key of the lane's best gain (0: the lane has no leaf)
        int li = 0x7FFFFFFF;
        unsigned long long kreg[RS];
#pragma unroll
        for (int q = 0; q < RS; ++q) {
            const int i = lane + 32 * q;
            kreg[q] = (reg_keys && i < n_leaves) ? gain_key(fg[i]) : 0ull;
        }
        auto rescan = [&]() {
            lk = 0;
            li = 0x7FFFFFFF;
            if (reg_keys) {
#pragma unroll
                for (int q = 0; q < RS; ++q)
                    if (kreg[q] > lk) { lk = kreg[q]; li = lane + 32 * q; }
            } else {
                for (int i = lane; i < n_leaves; i += 32) {
                    const unsigned long long k = gain_key(fg[i]);
                    if (k > lk) { lk = k; li = i; }
                }
            }
        };
        rescan();
        const unsigned long long neg_key = gain_key(NEG);
        for (;;) {
            if (n_leaves >= L) { done = 1; break; }
            const unsigned hi = (unsigned)(lk >> 32), lo = (unsigned)lk;
            const unsigned mh = __reduce_max_sync(0xffffffffu, hi);
            const unsigned ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
            const bool top = hi == mh && lo == ml;
            const int bi = (int)__reduce_min_sync(0xffffffffu, top ? (unsigned)li : 0x7FFFFFFFu);
            if ((((unsigned long long)mh << 32) | ml) <= neg_key || bi == 0x7FFFFFFF) { done = 1; break; }
            const int r = sf[bi], c0 = cs[r];
            if (c0 < 0) { mand = r; break; }
            const int node = n_leaves - 1, right = n_leaves;
            const double g0 = cg[c0], g1 = cg[c0 + 1];   // gains of the two new numbered leaves
            if (lane == 0) {   // shared memory only: the node arrays are written after the replay, in parallel
                spn[c0] = node << 1;
                spn[c0 + 1] = node << 1 | 1;
                sf[bi] = c0;
                sf[right] = c0 + 1;
                cl_rec[commits] = r;
                cl_leaf[commits] = bi;
            }
            if (reg_keys) {
                const unsigned long long k0 = gain_key(g0), k1 = gain_key(g1);
#pragma unroll
                for (int q = 0; q < RS; ++q) {
                    if (lane + 32 * q == bi) kreg[q] = k0;
                    if (lane + 32 * q == right) kreg[q] = k1;
                }
            } else if (lane < 2) {
                fg[lane == 0 ? bi : right] = lane == 0 ? g0 : g1;
            }
            __syncwarp();
            ++n_leaves;
            ++commits;
            if (lane == (bi & 31) || lane == (right & 31)) rescan();
        }
        if (lane == 0) { s_done = done; s_leaves = n_leaves; s_mand = mand; s_commits = commits; }
    }
    __syncthreads();
    const int n_leaves = s_leaves, commits = s_commits, done = s_done, mand = s_mand;

    // ---- the splits confirmed above, one thread each: node arrays and tree positions
    {
        const size_t no = (size_t)tree_slot * (L > 1 ? L - 1 : 1);
        unsigned long long rows = 0;
        for (int t = tid; t < commits; t += COMMIT_THREADS) {
            const int r = cl_rec[t], node = n_leaves0 - 1 + t, c0 = cs[r];
            // children of the node: a child that was confirmed in this launch too is a node (the place of
            // its own children names it), else the leaf number the replay gave it (left: the parent's,
            // right: the next free one at the time)
            const int gl = cs[c0], gr = cs[c0 + 1];
            a.m_left[no + node] = (gl >= 0 && spn[gl] >= 0) ? (spn[gl] >> 1) : ~cl_leaf[t];
            a.m_right[no + node] = (gr >= 0 && spn[gr] >= 0) ? (spn[gr] >> 1) : ~(n_leaves0 + t);
            // a parent from an earlier launch learns of its new child node here (one from this launch above)
            const int p = spn[r];
            if (p >= 0 && (p >> 1) < n_leaves0 - 1) {
                if ((p & 1) == 0) a.m_left[no + (p >> 1)] = node;
                else a.m_right[no + (p >> 1)] = node;
            }
            const NodeRec *q = a.recs + r;
            a.m_feature[no + node] = q->best.feature;
            a.m_bin[no + node] = q->best.bin;
            a.m_gain[no + node] = q->best.gain;
            a.rec_pos[c0] = node << 1;
            a.rec_pos[c0 + 1] = node << 1 | 1;
            const NodeRec *lc = a.recs + c0, *rc = lc + 1;
            rows += lc->n_all <= rc->n_all ? lc->n : rc->n;   // this context's rows of the child that was built
        }
        // leaf records: a leaf number may change hands more than once in a launch (a child that was
        // split ahead is confirmed right after its parent), so they are written from the replay's
        // final table, for the numbers whose record changed
        for (int i = tid; i < n_leaves; i += COMMIT_THREADS) {
            const int r = sf[i];
            if (i >= n_leaves0 || a.front[i] != r) {
                const NodeRec *q = a.recs + r;
                LeafRec x;
                x.off = q->off; x.n = q->n; x.buf = q->buf; x.rec = r; x.n_all = q->n_all; x.pad = 0;
                a.leaves[i] = x;
                a.front[i] = r;
            }
        }
        // one shared atomic per warp (64-bit shared atomics are compare-and-swap loops)
        for (int o = 16; o > 0; o >>= 1) rows += __shfl_xor_sync(0xffffffffu, rows, o);
        if (lane == 0 && rows) atomicAdd(&s_rows, rows);
    }
    __syncthreads();   // the region is free from here on
    if (tid == 0) {
        gs->n_leaves = n_leaves;
        gs->hist_rows += s_rows;
        gs->hist_builds += (unsigned long long)commits;
        gs->passes += 1;
    }
    if (done) {
        if (tid == 0) {
            gs->done = 1;
            gs->n_jobs = 0;
            gs->extra_builds += (unsigned long long)(n_exec - (n_leaves - 1));   // split ahead, not used by this tree
            if (a.use_cond) cudaGraphSetConditional(a.cond, 0);
        }
        return;
    }

    // ---- (2) the next batch.  Best-first growth takes a leaf when its gain is the largest among the
    //      leaves that exist, and a leaf exists once its parent has been taken; so, as far as the gains
    //      are known, the records whose split is not confirmed yet will be taken in the order of
    //      min(own gain, gains of the ancestors not taken yet), and only the first `budget` of them,
    //      the splits the tree still has room for.  The batch is the leaf needed next, then the unsplit
    //      records in that order, as long as few enough leaves are split ahead of their confirmation.
    const int ahead = n_exec - (n_leaves - 1);            // split, not confirmed
    const int budget = L - n_leaves;                      // splits the tree can still take
    int extra = a.K - 1;
    if (extra > a.slack - ahead) extra = a.slack - ahead;
    if (extra > (R - n_recs) / 2 - 1) extra = (R - n_recs) / 2 - 1;
    if (extra > a.max_slots - 2 - n_exec) extra = a.max_slots - 2 - n_exec;
    if (extra < 0) extra = 0;
    if ((R - n_recs) / 2 < 1 || a.max_slots - 1 - n_exec < 1) {
        // cannot happen within the bounds above (records and slots are sized for num_leaves - 1 splits
        // plus the slack): refuse rather than write out of bounds
        if (tid == 0) {
            atomicExch(&a.state->kernel_error, 1);
            gs->done = 1;
            gs->n_jobs = 0;
            if (a.use_cond) cudaGraphSetConditional(a.cond, 0);
        }
        return;
    }
    int *by_rank = cand_r + max_cand;                     // [max_cand] record at every rank if it may join the batch, else -1
    if (extra > 0) {
        for (int r0 = 0; r0 < n_recs; r0 += COMMIT_THREADS) {
            const int r = r0 + tid;
            bool open = false;       // a split that is not confirmed, with an admissible gain
            double e = NEG;
            if (r < n_recs) {
                const int c0 = cs[r];
                e = cg[r];
                open = e > NEG && !(c0 >= 0 && spn[c0] >= 0);
                if (open) {
                    int p = r;
                    while (p != 0 && spn[p] < 0) {       // not numbered: its parent has not been taken yet
                        p = a.rec_parent[p];
                        const double pg = cg[p];
                        e = pg < e ? pg : e;
                    }
                }
            }
            const unsigned m = __ballot_sync(0xffffffffu, open);
            int base = 0;
            if (lane == 0 && m) base = atomicAdd(&s_ncand, __popc(m));
            base = __shfl_sync(0xffffffffu, base, 0);
            if (open) {
                const int k = base + __popc(m & ((1u << lane) - 1u));
                if (k < max_cand) {
                    cand_k[k] = gain_key(e);
                    cand_r[k] = r;
                }
            }
        }
    }
    __syncthreads();
    int n_cand = s_ncand;
    if (n_cand > max_cand) n_cand = max_cand;   // cannot happen: the bound counts every record without a confirmed split
    // the open records in order: larger gain first, lower record on equal gain
    if (n_cand <= 448) {
        // few enough to count: the rank of a pair is the number of pairs that belong before it.  Every
        // thread reads all pairs from shared memory, four at a time (the list is padded to a multiple of
        // four with pairs that belong after every other): fewer dependent steps than a sorting network.
        const int n4 = (n_cand + 3) & ~3;
        if (tid >= n_cand && tid < n4) {
            cand_k[tid] = 0ull;
            cand_r[tid] = 0x7FFFFFFF;
        }
        __syncthreads();
        if (tid < n_cand) {
            const unsigned long long key = cand_k[tid];
            const int rec = cand_r[tid];
            const ulonglong2 *k2 = reinterpret_cast<const ulonglong2 *>(cand_k);
            const int4 *r4 = reinterpret_cast<const int4 *>(cand_r);
            int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
#pragma unroll 2
            for (int q = 0; q < (n4 >> 2); ++q) {
                const ulonglong2 ka = k2[2 * q], kb = k2[2 * q + 1];
                const int4 rr = r4[q];
                c0 += (ka.x > key || (ka.x == key && rr.x < rec)) ? 1 : 0;
                c1 += (ka.y > key || (ka.y == key && rr.y < rec)) ? 1 : 0;
                c2 += (kb.x > key || (kb.x == key && rr.z < rec)) ? 1 : 0;
                c3 += (kb.y > key || (kb.y == key && rr.w < rec)) ? 1 : 0;
            }
            const int rank = c0 + c1 + c2 + c3;
            by_rank[rank] = (rank < budget && cs[rec] == -1 && rec != mand) ? rec : -1;
        }
    } else if (n_cand <= 1024) {
        // bitonic sort of the (key, record) pairs, one per thread in registers, padded to a power of two
        // with entries that sort last.  Partners less than 32 apart exchange by shuffle; the others through
        // shared memory, in two buffers used in turn (one barrier per such step).
        int m = 32;
        while (m < n_cand) m <<= 1;
        unsigned long long key = tid < n_cand ? cand_k[tid] : 0ull;
        int rec = tid < n_cand ? cand_r[tid] : 0x7FFFFFFF;
        unsigned long long *sort_k = reinterpret_cast<unsigned long long *>(by_rank + max_cand);   // [1024]
        int *sort_r = reinterpret_cast<int *>(sort_k + 1024);                                       // [1024]
        __syncthreads();   // every thread holds its pair: the arrays become the first exchange buffer
        int pb = 0;
        for (int k = 2; k <= m; k <<= 1) {
            const bool first_low = (tid & k) == 0;   // this run of k entries ends up with the first entry lowest
            for (int jj = k >> 1; jj > 0; jj >>= 1) {
                unsigned long long ok;
                int orr;
                if (jj >= 32) {
                    unsigned long long *bk = pb ? sort_k : cand_k;
                    int *br = pb ? sort_r : cand_r;
                    bk[tid] = key;
                    br[tid] = rec;
                    __syncthreads();
                    ok = bk[tid ^ jj];
                    orr = br[tid ^ jj];
                    pb ^= 1;
                } else {
                    ok = __shfl_xor_sync(0xffffffffu, key, jj);
                    orr = __shfl_xor_sync(0xffffffffu, rec, jj);
                }
                const bool mine_first = key > ok || (key == ok && rec < orr);   // mine belongs before the partner's
                const bool lower = (tid & jj) == 0;
                if (mine_first != (lower == first_low)) { key = ok; rec = orr; }
            }
        }
        if (tid < n_cand) by_rank[tid] = (tid < budget && cs[rec] == -1 && rec != mand) ? rec : -1;
    } else {
        for (int i = tid; i < n_cand; i += COMMIT_THREADS) {
            const unsigned long long g = cand_k[i];
            const int r = cand_r[i];
            int rank = 0;
            for (int k = 0; k < n_cand; ++k) {
                const unsigned long long og = cand_k[k];
                rank += (og > g || (og == g && cand_r[k] < r)) ? 1 : 0;
            }
            by_rank[rank] = (rank < budget && cs[r] == -1 && r != mand) ? r : -1;
        }
    }
    if (tid == 0) s_pick[0] = mand;
    __syncthreads();
    if (warp != 0) return;
    // the first `extra` unsplit records in rank order
    int n_jobs = 1;
    for (int k0 = 0; k0 < n_cand && n_jobs < 1 + extra; k0 += 32) {
        const int k = k0 + lane;
        const int r = k < n_cand ? by_rank[k] : -1;
        const unsigned m = __ballot_sync(0xffffffffu, r >= 0);
        const int pos = n_jobs + __popc(m & ((1u << lane) - 1u));
        if (r >= 0 && pos < 1 + extra) s_pick[pos] = r;
        n_jobs += __popc(m);
    }
    if (n_jobs > 1 + extra) n_jobs = 1 + extra;
    __syncwarp();

    // ---- (3) the job table, by warp 0: lane j fills job j, then the lanes share out the blocks
    uint32_t n_j = 0;
    if (lane < n_jobs) {
        const int r = s_pick[lane];
        NodeRec *q = a.recs + r;
        const SplitRec best = q->best;
        const FeatRec pf = a.feat_rec[best.feature];
        GrowJob *job = gs->jobs + lane;
        n_j = q->n;
        job->rec = r;
        job->feature = best.feature;
        job->bin = best.bin;
        job->logW = pf.logW;
        job->byte = pf.byte;
        job->col = pf.col;
        job->col8 = pf.col8;
        job->off = q->off;
        job->n = n_j;
        job->n_all = q->n_all;
        job->buf = q->buf;
        job->nl = 0;
        job->gl = best.gl;
        job->hl = best.hl;
        job->PG = q->G;
        job->PH = q->H;
        job->parent_slot = q->slot;
        job->small_slot = 1 + n_exec + lane;
        job->child0 = n_recs + 2 * lane;
        job->finish_count = 0;
        job->lb[0] = job->lb[1] = 0;
        q->state = 1;
        q->child0 = n_recs + 2 * lane;
        a.rec_child[r] = n_recs + 2 * lane;
    }
    // blocks of the partition kernels: in proportion to the rows, at least one per leaf; histogram
    // CTAs per tile: one per rows_min rows of half the leaf (the smaller child has at most that many
    // rows), at most a leaf's share of the SMs; both scaled down when the batch wants more than a
    // launch has
    const uint32_t pb_cap = (uint32_t)(a.pb_total - a.K), xc = (uint32_t)(a.xcap - a.K);
    uint32_t wpb = 0, wpt = 0;
    if (lane < n_jobs) {
        wpb = (n_j + 2047u) / 2048u;
        wpb = wpb < 1u ? 1u : (wpb > pb_cap ? pb_cap : wpb);
        wpt = (n_j / 2u + a.rows_min - 1u) / a.rows_min;
        wpt = wpt < 1u ? 1u : (wpt > (uint32_t)a.parts_cap ? (uint32_t)a.parts_cap : wpt);
    }
    const uint32_t spb = __reduce_add_sync(0xffffffffu, wpb), spt = __reduce_add_sync(0xffffffffu, wpt);
    if (lane < n_jobs) {
        if (spb > pb_cap) { wpb = wpb * pb_cap / spb; if (wpb < 1u) wpb = 1u; }
        if (spt > xc) { wpt = wpt * xc / spt; if (wpt < 1u) wpt = 1u; }
    }
    uint32_t apb = wpb, apt = wpt;   // inclusive prefix sums over the lanes
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xffffffffu, apb, o), v = __shfl_up_sync(0xffffffffu, apt, o);
        if (lane >= o) { apb += u; apt += v; }
    }
    if (lane < n_jobs) {
        GrowJob *job = gs->jobs + lane;
        job->pb0 = (int)(apb - wpb);
        job->pb = (int)wpb;
        job->cta0 = (int)(apt - wpt);
        job->parts = (int)wpt;
        job->slot0 = (int)(apt - wpt) * a.n_tiles;
    }
    if (lane == 0) {
        gs->n_jobs = n_jobs;
        gs->n_exec = n_exec + n_jobs;
        gs->n_recs = n_recs + 2 * n_jobs;
    }
}

void fill_args(qgbdt_ctx *c, GrowArgs &a) {
    const int L = c->prm.num_leaves;
    a.gs = c->d_gs;
    a.recs = c->d_recs;
    a.rec_gain = c->d_rec_gain;
    a.rec_child = c->d_rec_child;
    a.rec_pos = c->d_rec_pos;
    a.rec_parent = c->d_rec_parent;
    a.leaves = c->d_leaves;
    a.front = c->d_front;
    a.state = c->d_state;
    a.feat_rec = c->d_feat_rec;
    a.N = (uint32_t)c->N;
    a.N_all = qg_sharded(c) ? (uint32_t)c->total_rows : (uint32_t)c->N;
    a.merged = qg_sharded(c) ? 1 : 0;
    a.ent0 = c->d_ent0;
    a.ent1 = c->d_ent1;
    a.codes_nat = reinterpret_cast<const uint16_t *>(c->d_codes_nat);
    a.bits = c->d_grow_bits;
    a.bits_stride = c->grow_bits_stride;
    a.counts = c->d_part_counts;
    a.pb_total = c->grow_pb_total;
    a.pool = c->d_hist_pool;
    a.partial = c->d_grow_partial;
    a.prep = c->d_grow_prep;
    a.cand = c->d_cand;
    a.F = c->F;
    a.nb = c->nb;
    a.L = L;
    a.K = c->grow_jobs;
    a.slack = qg_grow_slack(c);
    a.xcap = c->grow_xcap;
    a.rows_min = (uint32_t)c->grow_rows_min;
    a.n_tiles = (int)c->tiles.size();
    a.parts_cap = qg_grow_parts_cap(c);
    a.max_recs = qg_grow_max_recs(c);
    a.max_slots = qg_grow_max_slots(c);
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
    a.cond = 0;
    a.use_cond = 0;
    a.sep_reduce = c->F > 512;
}

int launch_commit(qgbdt_ctx *c, const GrowArgs &a, cudaStream_t st) {
    int rc = qg_phase_begin(c, QG_PHASE_COMMIT, st);
    if (rc != QGBDT_OK) return rc;
    k_grow_commit<<<1, COMMIT_THREADS, commit_smem_bytes(a.L, a.max_recs), st>>>(a);
    QG_LAUNCH_CHECK(c);
    return qg_phase_end(c, st);
}

// One pass: the kernels that split the leaves of the current batch, then the commit step.
// n_jobs, first_slot: only for sharded rows (the host follows the passes and knows them): leaves in
// the batch and the pool slot of the first one's smaller child.
int enqueue_pass(qgbdt_ctx *c, const GrowArgs &a, cudaStream_t st, int n_jobs = 0, int first_slot = 0) {
    int rc = qg_phase_begin(c, QG_PHASE_PARTITION, st);
    if (rc != QGBDT_OK) return rc;
    k_grow_flags<<<a.pb_total, PART_THREADS, 0, st>>>(a);
    QG_LAUNCH_CHECK(c);
    k_grow_scatter<<<a.pb_total, PART_THREADS, 0, st>>>(a);
    QG_LAUNCH_CHECK(c);
    if ((rc = qg_phase_end(c, st)) != QGBDT_OK) return rc;
    // sharded rows: left rows of every leaf of the batch over all ranks (which child is the smaller one)
    if (a.merged && (rc = qg_allreduce(c, c->d_gs->nl_all, n_jobs, QGBDT_REDUCE_SUM_I64, st)) != QGBDT_OK) return rc;
    if ((rc = qg_hist_grow(c, st)) != QGBDT_OK) return rc;
    int fin_y = (c->sm_count * 24 + c->F - 1) / c->F;   // blocks for about one and a half rounds of all SMs
    fin_y = fin_y < 1 ? 1 : (fin_y > a.K ? a.K : fin_y);
    const dim3 fin((unsigned)c->F, (unsigned)fin_y);
    if (a.merged) {
        // the smaller children's histograms: merged here, then summed over the ranks (their pool slots
        // are consecutive: 1 + splits before this pass + job)
        k_grow_merge<<<fin, 256, 0, st>>>(a);
        QG_LAUNCH_CHECK(c);
        const size_t hw = (size_t)c->F * c->nb;
        if ((rc = qg_allreduce(c, c->d_hist_pool + (size_t)first_slot * hw, (int64_t)n_jobs * (int64_t)hw,
                               QGBDT_REDUCE_SUM_I64, st)) != QGBDT_OK)
            return rc;
    }
    if ((rc = qg_phase_begin(c, QG_PHASE_FINISH, st)) != QGBDT_OK) return rc;
    {
        const int resident = c->sm_count * FIN_BLOCKS_PER_SM, all = c->F * a.K;
        const unsigned grid = (unsigned)(all < resident ? all : resident);
        if (a.sep_reduce) {
            k_grow_prep<<<1, 32, 0, st>>>(a);
            QG_LAUNCH_CHECK(c);
        }
        if (a.sep_reduce) k_grow_finish<false, true><<<grid, FIN_THREADS, 0, st>>>(a);
        else k_grow_finish<false, false><<<grid, FIN_THREADS, 0, st>>>(a);
    }
    QG_LAUNCH_CHECK(c);
    if (a.sep_reduce) {
        k_grow_reduce<<<(unsigned)a.K, FIN_THREADS, 0, st>>>(a);
        QG_LAUNCH_CHECK(c);
    }
    if ((rc = qg_phase_end(c, st)) != QGBDT_OK) return rc;
    return launch_commit(c, a, st);
}

}  // namespace

int qg_grow_parts_cap(const qgbdt_ctx *c) {
    const int t = (int)c->tiles.size();
    const int p = c->sm_count / (t > 0 ? t : 1);
    return p < 1 ? 1 : p;
}

int qg_grow_slack(const qgbdt_ctx *c) {
    const int s = 3 * c->grow_jobs;
    return s > GROW_SLACK ? GROW_SLACK : s;
}
int qg_grow_max_recs(const qgbdt_ctx *c) { return 1 + 2 * (c->prm.num_leaves - 1 + qg_grow_slack(c)) + 2 * c->grow_jobs; }
int qg_grow_max_slots(const qgbdt_ctx *c) { return c->prm.num_leaves + qg_grow_slack(c) + c->grow_jobs + 2; }

void qg_grow_graph_destroy(qgbdt_ctx *c) {
    if (c->grow_graph_exec) cudaGraphExecDestroy(reinterpret_cast<cudaGraphExec_t>(c->grow_graph_exec));
    c->grow_graph_exec = nullptr;
    c->grow_pass_launches = 0;
}

// The growth of one tree after its root as a CUDA graph: a commit kernel (which picks the first
// batch), then a while node whose body is one pass.  The launch arguments never change (what
// differs from pass to pass and from tree to tree is device state), so the graph is built once per
// context and objective.
static int build_grow_graph(qgbdt_ctx *c, GrowArgs a) {
    const int64_t launches_before = c->n_launches;
    int rc = qg_hist_grow_configure(c);
    if (rc != QGBDT_OK) return rc;
    cudaGraph_t graph = nullptr;
    cudaStream_t cs = nullptr;
    cudaGraphExec_t exec = nullptr;
    const char *what = "cudaGraphCreate";
    cudaError_t e = cudaGraphCreate(&graph, 0);
    if (e == cudaSuccess) {
        what = "cudaGraphConditionalHandleCreate";
        e = cudaGraphConditionalHandleCreate(&a.cond, graph, 1, cudaGraphCondAssignDefault);
    }
    a.use_cond = 1;
    cudaGraphNode_t first = nullptr, loop = nullptr;
    if (e == cudaSuccess) {
        what = "cudaGraphAddKernelNode";
        void *params[] = {&a};
        cudaKernelNodeParams kp = {};
        kp.func = reinterpret_cast<void *>(k_grow_commit);
        kp.gridDim = dim3(1);
        kp.blockDim = dim3(COMMIT_THREADS);
        kp.sharedMemBytes = (unsigned)commit_smem_bytes(a.L, a.max_recs);
        kp.kernelParams = params;
        e = cudaGraphAddKernelNode(&first, graph, nullptr, 0, &kp);
    }
    cudaGraph_t body = nullptr;
    if (e == cudaSuccess) {
        what = "cudaGraphAddNode (while)";
        cudaGraphNodeParams np = {};
        np.type = cudaGraphNodeTypeConditional;
        np.conditional.handle = a.cond;
        np.conditional.type = cudaGraphCondTypeWhile;
        np.conditional.size = 1;
        e = cudaGraphAddNode(&loop, graph, &first, 1, &np);
        if (e == cudaSuccess) body = np.conditional.phGraph_out[0];
    }
    if (e == cudaSuccess) {
        what = "cudaStreamCreateWithFlags";
        e = cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking);
    }
    if (e == cudaSuccess) {
        what = "capturing a pass";
        e = cudaStreamBeginCaptureToGraph(cs, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal);
        if (e == cudaSuccess) {
            rc = enqueue_pass(c, a, cs);
            cudaGraph_t out = nullptr;
            e = cudaStreamEndCapture(cs, &out);
        }
    }
    const int64_t pass_launches = c->n_launches - launches_before;
    c->n_launches = launches_before;
    if (e == cudaSuccess && rc == QGBDT_OK) {
        what = "cudaGraphInstantiate";
        e = cudaGraphInstantiate(&exec, graph, 0);
    }
    if (cs) cudaStreamDestroy(cs);
    if (graph) cudaGraphDestroy(graph);
    if (rc != QGBDT_OK) return rc;
    if (e != cudaSuccess) {
        cudaGetLastError();
        return qg_fail(c, QGBDT_ERR_CUDA, "building the growth graph failed at %s: %s", what, cudaGetErrorString(e));
    }
    c->grow_graph_exec = exec;
    c->grow_pass_launches = pass_launches;
    c->grow_graph_const_hess = c->const_hess;
    return QGBDT_OK;
}

// Grows the tree of boosting iteration slot `tree_slot` of the current train call.  Gradients must
// have been quantized on the same stream (the state holds the totals and maxima).  Asynchronous,
// unless the histogram event timers are on: then the passes go to the stream one by one and the
// host reads after each whether the tree is finished.
int qg_grow_tree(qgbdt_ctx *c, int tree_slot, cudaStream_t st) {
    GrowArgs a;
    fill_args(c, a);
    const size_t smem = commit_smem_bytes(a.L, a.max_recs);
    if (smem > 48 * 1024) {
        if (smem > (size_t)c->max_smem_optin) return qg_fail(c, QGBDT_ERR_ARG, "num_leaves too large for the commit step");
        QG_CUDA(c, cudaFuncSetAttribute(k_grow_commit, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    k_grow_begin<<<1, 1, 0, st>>>(c->d_gs, c->d_recs, c->d_rec_gain, c->d_rec_child, c->d_rec_pos, c->d_leaves, c->d_front,
                                  c->d_state, (uint32_t)c->N, a.N_all, tree_slot);
    QG_LAUNCH_CHECK(c);
    int rc = qg_hist(c, nullptr, 0, c->N, c->d_hist_pool, st);   // root: all rows, contiguous
    if (rc != QGBDT_OK) return rc;
    if ((rc = qg_allreduce(c, c->d_hist_pool, (int64_t)c->F * c->nb, QGBDT_REDUCE_SUM_I64, st)) != QGBDT_OK) return rc;
    if ((rc = qg_phase_begin(c, QG_PHASE_FINISH, st)) != QGBDT_OK) return rc;
    k_grow_finish<true, false><<<(unsigned)c->F, FIN_THREADS, 0, st>>>(a);
    QG_LAUNCH_CHECK(c);
    if ((rc = qg_phase_end(c, st)) != QGBDT_OK) return rc;
    if (c->prm.num_leaves < 2) return QGBDT_OK;
    if (c->profile_hist || a.merged) {
        // event records around every phase, or exchanges between the ranks inside a pass: the passes
        // go to the stream one by one and the host reads after each what the commit step decided
        if ((rc = launch_commit(c, a, st)) != QGBDT_OK) return rc;
        int *h_gs = reinterpret_cast<int *>(reinterpret_cast<char *>(c->h_pinned) + 64 * 1024 + 8192);
        for (int pass = 0; pass < c->prm.num_leaves; ++pass) {
            // n_jobs, done, n_leaves, n_exec: the first four words of the grow state
            QG_CUDA(c, cudaMemcpyAsync(h_gs, c->d_gs, 4 * sizeof(int), cudaMemcpyDeviceToHost, st));
            QG_CUDA(c, cudaStreamSynchronize(st));
            if (h_gs[1]) break;
            if ((rc = enqueue_pass(c, a, st, h_gs[0], 1 + h_gs[3] - h_gs[0])) != QGBDT_OK) return rc;
        }
        return QGBDT_OK;
    }
    if (c->grow_graph_exec && c->grow_graph_const_hess != c->const_hess) qg_grow_graph_destroy(c);
    if (!c->grow_graph_exec && (rc = build_grow_graph(c, a)) != QGBDT_OK) return rc;
    QG_CUDA(c, cudaGraphLaunch(reinterpret_cast<cudaGraphExec_t>(c->grow_graph_exec), st));
    return QGBDT_OK;
}
