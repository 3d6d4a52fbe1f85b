// Internal declarations shared by the CUDA sources of libqgbdt (never installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <cstddef>
#include <cstdio>
#include <vector>

#include "qgbdt.h"

// ---------------------------------------------------------------------------
// Data layout in device memory
//
// Bin matrix: split by features into tiles of at most 128 features.  A tile stores
// its features row-major, W = 2^logW 32-bit words per row (W in 1..32), four
// consecutive features per word (feature 4a+k of the tile in byte k of word a).
// Features beyond the tile's real width are stored as code 0 and never reported.
// A warp that reads 32 consecutive words therefore reads R = 32/W whole rows; lane
// l holds word a = l % W of row slot b = l / W.
//
// Packed gradient codes (Sec. 6.2 packs g and h of a sample the same way as the
// bins): two bytes per row, signed gradient in the high byte, hessian in the low
// byte.  Inside every block of 16 rows the codes are stored 4 x 4 transposed (the
// code of row 16 b + 4 j + s sits at position 16 b + 4 s + j), so that a lane of the
// histogram kernel reads the codes of its four rows with one 8-byte load.
//
// Histogram plan: tiles of equal width are built by one launch and share the SMs equally;
// a tile owns `parts` partial-histogram slots starting at `cta0`; the grid is (part, tile).  A build of n rows uses the first
// min(parts, ceil(n / 1024)) parts of every tile.
//
// Row lists: one uint32 array of N entries; leaf l owns [leaf_off[l], +leaf_n[l]).
// ---------------------------------------------------------------------------

struct TileDesc {
    const uint32_t *data;  // [N][W] words
    int32_t f0;            // first feature of the tile
    int32_t nf;            // real features in the tile (<= 4 * W)
    int32_t logW;          // log2 of words per row
    int32_t words_used;    // ceil(nf / 4)
    int32_t parts;         // CTAs of the histogram plan that work on this tile
    int32_t cta0;          // first of them
};

// Scalars produced and consumed on the device within one boosting iteration.
struct DevState {
    // the first three words are maximised over the ranks as they stand when the rows are sharded
    unsigned int gmax_bits;  // max |g| as float bits (non-negative floats order like uints)
    unsigned int hmax_bits;  // max h as float bits
    int bad_value;           // set when a gradient / hessian / bin code is out of domain (0 or 1)
    int kernel_error;        // set by a kernel that refused to run (checked at the next synchronising call)
    unsigned int part_nl;    // rows that went left in the last partition
    long long tot_g, tot_h;  // integer sums over all rows of the last quantization (adjacent: summed over the ranks together)
};
static_assert(offsetof(DevState, hmax_bits) == 4 && offsetof(DevState, bad_value) == 8 &&
              offsetof(DevState, tot_h) == offsetof(DevState, tot_g) + 8, "layout the rank exchanges rely on");

// Per-feature best candidate, then the leaf's best split (same fields as qgbdt_split).
struct SplitRec {
    double gain;
    long long gl, hl;
    int feature, bin;
    int valid, pad;
};

// Where a feature sits in the tiled matrix and in the histogram plan (one load instead of a
// chain through the tile table).
struct FeatRec {
    const uint32_t *col;   // the feature's word in row 0 of its tile
    int32_t logW, byte;    // words per row (log2) of the tile, byte of the word
    int32_t cta0, parts;   // partial-histogram slots of the tile
    int32_t fl, tile;      // feature number inside the tile, tile number
    const uint8_t *col8;   // the feature's column in the column-major copy (nullptr: there is none)
};

// Histogram CTAs per tile that take part in building a child of n rows during tree growth: one per
// `rows_min` rows, at most `parts`.  rows_min is 3072 for rows of up to 32 bytes (every CTA adds its
// whole local histogram into the leaf's sums) and 1024 per 32 bytes of the widest tile beyond (4096
// for 128-byte rows: a CTA of a wide tile writes a quarter of a megabyte of partial histogram that
// the finishing kernel has to read back, and has four times the work per row to make up for its
// fixed cost).
__device__ __host__ inline uint32_t qg_grow_parts(uint32_t parts, uint32_t n, uint32_t rows_min) {
    uint32_t want = (n + rows_min - 1) / rows_min;
    if (want < 1) want = 1;
    return want < parts ? want : parts;
}

// ---- leaf-wise growth on the device (grow.cu) --------------------------------------------------
// A tree grows in passes.  A pass splits up to GROW_MAX_JOBS leaves at once (row partition, the
// smaller child's histogram, the larger child's by subtraction, both children's best splits); the
// batch always holds the leaf that best-first growth (Sec. 3) would split next and is filled up with
// the known leaves of largest gain, also children of leaves whose own split has not been confirmed
// yet.  After the pass a commit step replays the best-first order: it takes the leaf with the
// largest gain, and if that leaf has been split already it numbers the children and records the
// node, until it meets a leaf that has not been split (which goes into the next batch) or the tree
// is full.  The result is the tree best-first growth builds, whatever the batches were.

constexpr int GROW_MAX_JOBS = 32;   // leaves split per pass, at most (a warp looks a job up with one ballot)
constexpr int GROW_SLACK = 96;      // leaves that may be split ahead of their confirmation at any time, at most
                                    // (a context allows three times its leaves per pass)

// A leaf with a number (confirmed by the commit step): what the refit and the score update read.
struct LeafRec {
    uint32_t off, n;     // its rows: entries [off, off + n) of pair buffer `buf`
    int32_t buf;         // 0 or 1; -1: the identity list of the root
    int32_t rec;         // its growth record
    uint32_t n_all;      // its rows over all ranks (= n unless the rows are sharded, Sec. 7.3)
    uint32_t pad;
};

// Growth record of a leaf the grower knows: confirmed or not, split or not.
struct NodeRec {
    uint32_t off, n;
    uint32_t n_all;          // rows of the leaf over all ranks (= n unless the rows are sharded, Sec. 7.3)
    int32_t buf;
    int32_t slot;            // histogram slot in the pool
    long long G, H;          // integer gradient / hessian totals
    SplitRec best;           // best split of the leaf
    int32_t state;           // 0: not split; 1: split (children in records child0, child0 + 1)
    int32_t child0;
    uint32_t nl;             // rows that went left when it was split
    int32_t parent_node, parent_side;   // position in the tree, valid once confirmed
};

// One leaf being split in the current pass.
// Tiles narrower than 2^this words per row: the histogram CTAs of a leaf being split add into one
// partial slot per tile; from this width on each CTA stores a partial slot of its own.
constexpr int QG_SHARED_PARTIAL_LOGW = 5;

struct GrowJob {
    int32_t rec;                     // its growth record
    int32_t feature, bin;            // the split
    int32_t logW, byte;              // tile width (log2 words per row) and byte of the split feature's word
    const uint32_t *col;             // that word in row 0 of the tile
    const uint8_t *col8;             // the split feature's column in the column-major copy, or nullptr
    uint32_t off, n;                 // rows of the leaf
    int32_t buf;                     // their pair buffer
    uint32_t nl;                     // rows that go left (written by the scatter kernel)
    uint32_t n_all;                  // rows of the leaf over all ranks
    long long gl, hl, PG, PH;        // left totals of the split, totals of the leaf
    int32_t parent_slot, small_slot; // histogram slots: the leaf's (becomes the larger child's), the smaller child's
    int32_t child0;                  // growth records of the children: child0 (left), child0 + 1 (right)
    int32_t pb0, pb;                 // blocks of the partition kernels: [pb0, pb0 + pb)
    int32_t cta0, parts;             // histogram CTAs per tile: x in [cta0, cta0 + parts) of the grid
    int32_t slot0;                   // partial-histogram slots: tile t, part p uses slot0 + t * parts + p
    unsigned int finish_count;       // blocks of the finishing kernel that are through
    unsigned int lb[2];              // largest lower bound on a gain seen so far over all features (smaller, larger
                                     // child), as order-preserving bits of a float; 0 = none yet
    int32_t pad;
};

// State of the growth of one tree, kept on the device so that the host never looks.
struct GrowState {
    int32_t n_jobs, done;
    int32_t n_leaves;                // confirmed leaves
    int32_t n_exec;                  // leaves split so far (confirmed or not)
    int32_t n_recs;                  // growth records in use
    int32_t tree_slot;               // slot of the tree being grown in the device-side model arrays
    GrowJob jobs[GROW_MAX_JOBS];
    unsigned long long hist_rows;    // rows of the smaller children of confirmed splits (all trees so far)
    unsigned long long hist_builds;  // confirmed splits (all trees so far)
    unsigned long long extra_rows, extra_builds;   // the same for splits made ahead that the tree did not use
    unsigned long long passes;
    long long nl_all[GROW_MAX_JOBS]; // per job: rows that go left over all ranks (the scatter kernel writes this
                                     // rank's count, a sharded run sums it over the ranks before the histograms)
};

// Per-leaf constants of the split search on 32-bit sums (the functions are in split_scan.cuh).
struct Admit32 {
    int G;                             // totals of the leaf
    uint32_t H, n_s, half;             // half = H / 2
    unsigned long long x_min, x_end;   // row estimate within [min_data, n_s - min_data]  <=>  x_min <= X < x_end
    uint32_t min_data;
    int const_h;
    float q_sure;                      // single-precision hessian sums from here on are certainly >= min_sum_h
    double min_sum_h, dh;
};

// Per leaf being split: what is the same for all its features in the finishing kernel.
struct JobPrep {
    double dg, dh;         // interval lengths of Eq. 5
    double tpS, tpL;       // the leaf's own term of Eq. 7 for the smaller and the larger child
    Admit32 aS, aL;
    uint32_t P;            // histogram CTAs per tile that took part
    int32_t small_is_left;
};

struct qgbdt_ctx {
    qgbdt_params prm;
    int device = 0;
    int sm_count = 0;
    int max_smem_optin = 0;
    bool coop_ok = false;   // the device supports cooperative launches
    // data
    int64_t N = 0;
    int F = 0, nb = 0;
    bool loaded = false;
    std::vector<TileDesc> tiles;
    TileDesc *d_tiles = nullptr;
    int hist_grid = 0, max_parts = 1;
    unsigned long long *d_partial = nullptr;  // [hist_grid][4][nb][32] partial histograms (only if max_parts > 1)
    std::vector<void *> tile_allocs;
    // quantized gradients
    uint8_t *d_codes = nullptr;  // [round_up(N, 16)] 16-bit codes, transposed inside blocks of 16 rows
    uint8_t *d_codes_nat = nullptr;  // [N] the same codes in row order (read through row lists)
    int code_bytes = 2;
    bool quantized = false;
    bool const_hess = false;
    float gmax = 0.f, hmax = 0.f;
    // leaves
    int n_leaves = 1;
    std::vector<int64_t> leaf_off, leaf_n;
    uint32_t *d_idx = nullptr, *d_idx_tmp = nullptr;
    bool idx_is_identity = false;
    int refit_leaves = 0;   // leaf count the last qgbdt_refit_leaves ran for (0: the leaves changed since)
    // scratch
    DevState *d_state = nullptr;
    uint32_t *d_part_counts = nullptr;  // per partition block: rows going left, then its exclusive scan
    uint32_t *d_part_bits = nullptr;    // one predicate bit per row of the leaf being split
    SplitRec *d_feat_best = nullptr;    // [F]
    SplitRec *d_split_out = nullptr;    // [2]
    long long *d_leaf_sums = nullptr;   // [L][2] fixed-point refit sums
    uint32_t *d_leaf_table = nullptr;   // [L][2] (offset, leaf) of the step-wise interface's leaves sorted by offset
    float *d_leaf_value = nullptr;      // [L]
    double *d_leaf_w = nullptr;         // [L]
    void *h_pinned = nullptr;           // small pinned staging area
    // training buffers (allocated on first qgbdt_train)
    float *d_g = nullptr, *d_h = nullptr;
    unsigned long long *d_hist_pool = nullptr;  // [L][F][nb]
    LeafRec *d_leaves = nullptr;                // [L] numbered leaves of the tree being grown
    NodeRec *d_recs = nullptr;                  // [qg_grow_max_recs] growth records
    double *d_rec_gain = nullptr;               // [qg_grow_max_recs] gain of a record's best split (-inf: none)
    int32_t *d_rec_child = nullptr;             // [qg_grow_max_recs] first child record of a split record, -1: not split
    int32_t *d_rec_pos = nullptr;               // [qg_grow_max_recs] (node << 1 | side) of a numbered record's parent, -1
    int32_t *d_rec_parent = nullptr;            // [qg_grow_max_recs] the record a record was split from
    int32_t *d_front = nullptr;                 // [L] growth record of every numbered leaf
    int grow_jobs = 1;                          // leaves split per pass (<= GROW_MAX_JOBS; fewer with thousands of features)
    int grow_pb_total = 0;                      // blocks of a partition launch
    int grow_xcap = 0;                          // histogram CTAs per tile of a growth launch
    int grow_rows_min = 1024;                   // rows per histogram CTA of tree growth, at least
    uint32_t *d_grow_bits = nullptr;            // [grow_jobs][bits_stride] predicate bits of the leaves being split
    size_t grow_bits_stride = 0;
    JobPrep *d_grow_prep = nullptr;                 // [GROW_MAX_JOBS]
    unsigned long long *d_grow_partial = nullptr;   // [grow_xcap * tiles][4][nb][32] partial histograms of growth
    uint2 *d_ent0 = nullptr, *d_ent1 = nullptr; // [N] (row, gradient code) pairs of the leaves, two buffers
    uint16_t *d_leaf_id = nullptr;              // [N] leaf of every row in the tree just grown
    GrowState *d_gs = nullptr;
    SplitRec *d_cand = nullptr;                 // [F][2] per-feature best candidates of the two children
    FeatRec *d_feat_rec = nullptr;              // [F] location of every feature
    uint8_t *d_colmajor = nullptr;              // [F][col_stride] column-major copy of the bin codes (training only)
    size_t col_stride = 0;
    // rows sharded over ranks (Sec. 7.3): this context holds rows [row_offset, row_offset + N) of total_rows
    int dist_rank = 0, dist_world = 1;
    int64_t row_offset = 0, total_rows = 0;
    qgbdt_allreduce_fn dist_reduce = nullptr;
    void *dist_user = nullptr;
    bool want_column_copy = true;               // QGBDT_OPT_COLUMN_COPY
    bool leaf_values_quantized = false;         // QGBDT_OPT_LEAF_VALUES: 1 = from the quantized sums (no refit)
    void *grow_graph_exec = nullptr;            // cudaGraphExec_t: the split loop of one tree
    int64_t grow_pass_launches = 0;             // kernel launches of one pass
    bool grow_graph_const_hess = false;         // objective it was captured for
    // trees of the current qgbdt_train call, on the device until the call ends
    int model_cap = 0;                          // trees the arrays below can hold
    int32_t *d_m_num_leaves = nullptr, *d_m_feature = nullptr, *d_m_bin = nullptr, *d_m_left = nullptr,
            *d_m_right = nullptr;
    double *d_m_gain = nullptr;
    float *d_m_leaf_value = nullptr;
    long long *d_m_leaf_count = nullptr;
    // counters
    int64_t n_launches = 0, n_hist_builds = 0, n_hist_row_features = 0;
    int64_t n_passes = 0, n_extra_builds = 0;   // commit steps run; leaves split ahead that their tree did not use
    // optional per-launch timing of the histogram kernel (event pairs on the launching stream)
    bool profile_hist = false;
    std::vector<cudaEvent_t> hist_events;  // start/stop pairs, reused
    std::vector<int> hist_event_phase;     // phase (QG_PHASE_*) of every pair
    size_t hist_events_used = 0;
    int64_t hist_prof_bytes = 0, hist_prof_launches = 0;
    char err[512] = {0};
};

int qg_fail(qgbdt_ctx *c, int code, const char *fmt, ...);

// Phases of a boosting iteration for the event timers (same order as qgbdt_get_timings reports them).
enum { QG_PHASE_GRADIENTS = 0, QG_PHASE_QUANTIZE, QG_PHASE_ROOT_HIST, QG_PHASE_PARTITION, QG_PHASE_CHILD_HIST,
       QG_PHASE_FINISH, QG_PHASE_COMMIT, QG_PHASE_REFIT, QG_PHASE_SCORES, QG_N_PHASES };
// With the timers on, records the start event of a phase on `st` (api.cu); qg_phase_end records the
// stop event of the phase begun last.  No-ops with the timers off.
int qg_phase_begin(qgbdt_ctx *c, int phase, cudaStream_t st);
int qg_phase_end(qgbdt_ctx *c, cudaStream_t st);

#define QG_CUDA(c, expr)                                                                       \
    do {                                                                                       \
        cudaError_t e_ = (expr);                                                               \
        if (e_ != cudaSuccess)                                                                 \
            return qg_fail((c), QGBDT_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

#define QG_LAUNCH_CHECK(c)                                                                    \
    do {                                                                                      \
        (c)->n_launches++;                                                                    \
        cudaError_t e_ = cudaGetLastError();                                                  \
        if (e_ != cudaSuccess)                                                                \
            return qg_fail((c), QGBDT_ERR_CUDA, "kernel launch failed at %s:%d: %s", __FILE__, \
                           __LINE__, cudaGetErrorString(e_));                                  \
    } while (0)

static inline int qg_levels_g(int bits) { return (1 << (bits - 1)) - 1; }
static inline int qg_levels_h(int bits, int mode) { return mode == 0 ? (1 << bits) - 2 : (1 << bits) - 1; }

// ---- launchers implemented in the kernel files (all asynchronous on `st`) ----

// load.cu
int qg_relayout(qgbdt_ctx *c, const uint8_t *d_bins, int layout, int64_t ld, cudaStream_t st);
int qg_iota(qgbdt_ctx *c, cudaStream_t st);
// Builds the column-major copy of the bin codes that the row partition of a split reads (one byte
// per row instead of a DRAM granule per row) and records the columns in the feature records.
// Without the memory for it the partition keeps reading the tiles.
int qg_build_columns(qgbdt_ctx *c, cudaStream_t st);

// quantize.cu
int qg_gradients(qgbdt_ctx *c, const float *d_scores, const float *d_labels, float *d_g, float *d_h,
                 bool reduce_max, bool clear_bad, cudaStream_t st);
int qg_absmax(qgbdt_ctx *c, const float *d_g, const float *d_h, cudaStream_t st);
int qg_quantize(qgbdt_ctx *c, const float *d_g, const float *d_h, uint32_t tree, int8_t *d_gq,
                uint8_t *d_hq, cudaStream_t st);

// hist.cu
int qg_hist(qgbdt_ctx *c, const uint32_t *d_rows, int64_t off, int64_t n, unsigned long long *d_hist,
            cudaStream_t st);
int qg_subtract(qgbdt_ctx *c, const unsigned long long *d_parent, const unsigned long long *d_small,
                unsigned long long *d_large, cudaStream_t st);

// hist_fp32.cu: Algorithm 1 with the original single-precision gradients (the unquantized baseline)
int qg_hist_fp32(qgbdt_ctx *c, const float *d_g, const float *d_h, const uint32_t *d_rows, int64_t n, float *d_hist,
                 cudaStream_t st);

// split.cu
int qg_find_split(qgbdt_ctx *c, const unsigned long long *d_hist, long long G, long long H, long long n_rows,
                  SplitRec *d_out, cudaStream_t st);

// partition.cu
int qg_partition(qgbdt_ctx *c, int64_t off, int64_t n, int feature, int bin, cudaStream_t st);

// refit.cu
int qg_refit(qgbdt_ctx *c, const float *d_g, const float *d_h, cudaStream_t st);
int qg_apply_leaf_values(qgbdt_ctx *c, float *d_scores, cudaStream_t st);
// the same two for a tree grown on the device (leaf table from the device leaf records)
int qg_refit_grown(qgbdt_ctx *c, const float *d_g, const float *d_h, float *d_scores, int tree_slot, cudaStream_t st);

// grow.cu: one tree by leaf-wise growth, every decision taken on the device
int qg_grow_tree(qgbdt_ctx *c, int tree_slot, cudaStream_t st);
// hist.cu: histograms of the smaller children of the leaves being split in the current pass
int qg_hist_grow(qgbdt_ctx *c, cudaStream_t st);
// api.cu: sums (kind QGBDT_REDUCE_SUM_I64) or maximises (QGBDT_REDUCE_MAX_U32) `count` words at d_buf over the
// ranks through the caller's callback; a no-op when the rows are not sharded
int qg_allreduce(qgbdt_ctx *c, void *d_buf, int64_t count, int kind, cudaStream_t st);
inline bool qg_sharded(const qgbdt_ctx *c) { return c->dist_world > 1 && c->dist_reduce != nullptr; }
int qg_grow_parts_cap(const qgbdt_ctx *c);   // grow.cu: histogram CTAs per tile one leaf may get
int qg_grow_slack(const qgbdt_ctx *c);       // grow.cu: leaves that may be split ahead of their confirmation
int qg_grow_max_recs(const qgbdt_ctx *c);    // grow.cu: growth records / histogram slots a tree may use
int qg_grow_max_slots(const qgbdt_ctx *c);
int qg_hist_grow_configure(qgbdt_ctx *c);   // function attributes of the kernels it launches (before a capture)
void qg_grow_graph_destroy(qgbdt_ctx *c);   // grow.cu: drops the captured split loop (buffers are about to change)

