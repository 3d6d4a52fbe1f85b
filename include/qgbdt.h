/*
 * qgbdt.h -- C ABI of the quantized-GBDT hot path for NVIDIA B200 (sm_100a).
 *
 * The library trains gradient-boosted trees from gradients quantized to 2..8 bits
 * by stochastic rounding, with integer histograms ("Quantized Training of Gradient
 * Boosting Decision Trees", arXiv 2207.09682).  Every step below runs in hand-written
 * CUDA kernels; there is no CPU fallback.
 *
 * Conventions
 *  - Every call returns 0 (QGBDT_OK) or a negative error code; qgbdt_last_error()
 *    gives the message of the last failure on that context.  Nothing throws or aborts.
 *  - Pointers named d_* are DEVICE pointers owned by the caller; they must stay valid
 *    until the stream work of the call has finished.  Pointers named h_* (and all
 *    scalar out-parameters) are HOST pointers owned by the caller.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *    that only take device pointers are asynchronous on that stream; calls that return
 *    host scalars synchronise the stream before returning (stated per call).
 *  - A context belongs to the CUDA device that was current when it was created, owns
 *    its work buffers (relaid bin matrix, row-index lists, packed gradient codes,
 *    histogram pool, scratch) and frees them in qgbdt_destroy().  A context is not
 *    thread-safe.
 *  - Histogram layout: hist[feature][bin], one 64-bit word per bin holding the hessian
 *    sum in the low 32 bits (unsigned) and the gradient sum in the high 32 bits
 *    (signed): word = (int64)G * 2^32 + H  (Sec. 6.2, packed gradient and hessian).
 *  - Leaf numbering: before any split there is one leaf, 0, holding all rows in
 *    ascending order.  Splitting leaf l keeps l as the left child (bin <= threshold)
 *    and gives the right child the next unused leaf number.
 */
#ifndef QGBDT_H
#define QGBDT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QGBDT_OK 0
#define QGBDT_ERR_ARG (-1)      /* null pointer, size or parameter out of range           */
#define QGBDT_ERR_STATE (-2)    /* call out of order (e.g. histogram before quantize)     */
#define QGBDT_ERR_OVERFLOW (-3) /* integer sums could exceed the 32+32-bit histogram word */
#define QGBDT_ERR_CUDA (-4)     /* a CUDA runtime call or kernel failed                   */
#define QGBDT_ERR_ALLOC (-5)    /* device or host allocation failed                       */
#define QGBDT_ERR_VALUE (-6)    /* non-finite gradient, negative hessian, |g| or h >= 256,
                                   or a bin code >= n_bins                                */

typedef struct qgbdt_ctx qgbdt_ctx;

/* Training parameters.  Defaults of the paper's runs: learning_rate 0.1, 255 leaves. */
typedef struct {
    int32_t bits;             /* B, gradient bits, 2..8 (Sec. 4.1)                              */
    int32_t objective;        /* 0: logistic loss, labels in {0,1}; 1: squared loss (hessian 1) */
    int32_t num_leaves;       /* leaves per tree, 1..4096 (leaf-wise growth, Sec. 3)            */
    int32_t num_trees;        /* informational; qgbdt_train takes its own count                */
    int32_t min_data_in_leaf; /* a split needs this many (estimated) rows on both sides         */
    double learning_rate;     /* leaf outputs are learning_rate * w* (Eq. 3)                    */
    double lambda_l2;         /* added to every hessian sum in Eq. 3 / Eq. 7 (paper: 0)         */
    double min_sum_hessian;   /* a split needs this much dequantized hessian on both sides      */
    double min_gain;          /* a split needs gain > min_gain                                  */
    uint64_t seed;            /* seed of the stochastic-rounding hash                           */
    int32_t hess_levels_mode; /* 0: delta_h = max h / (2^B - 2) (Eq. 5); 1: max h / (2^B - 1)   */
    int32_t rounding;         /* 0: stochastic rounding; 1: round to nearest (Eq. 8)            */
} qgbdt_params;

/* One histogram bin: little-endian view of the packed 64-bit word. */
typedef struct {
    uint32_t h; /* sum of quantized hessians */
    int32_t g;  /* sum of quantized gradients */
} qgbdt_bin;

/* Best split of one leaf (Eq. 7).  Rows with bin <= `bin` of `feature` go left. */
typedef struct {
    int32_t feature, bin;
    double gain;
    int64_t gl, hl, gr, hr; /* integer gradient / hessian sums of the two sides */
    int64_t nl_est, nr_est; /* rows per side estimated from hessian sums (exact for constant hessian) */
    int32_t valid;          /* 0: the leaf has no admissible split */
} qgbdt_split;

/* Trees written by qgbdt_train: HOST arrays allocated by the caller.  L = params.num_leaves.
 * Tree k uses node slots [k*(L-1), (k+1)*(L-1)) and leaf slots [k*L, (k+1)*L).
 * Node i of a tree is the i-th split made; a child c >= 0 is a node, c < 0 is leaf ~c. */
typedef struct {
    int32_t *num_leaves; /* [num_trees]                                   */
    int32_t *feature;    /* [num_trees * (L-1)]                           */
    int32_t *bin;        /* [num_trees * (L-1)] threshold bin             */
    int32_t *left;       /* [num_trees * (L-1)]                           */
    int32_t *right;      /* [num_trees * (L-1)]                           */
    double *gain;        /* [num_trees * (L-1)]                           */
    float *leaf_value;   /* [num_trees * L], already times learning_rate  */
    int64_t *leaf_count; /* [num_trees * L] rows per leaf                 */
} qgbdt_model;

/* Creates a context on the current CUDA device.  Fails with QGBDT_ERR_ARG on parameters
 * out of range and QGBDT_ERR_CUDA when no usable device is present. */
int qgbdt_create(qgbdt_ctx **ctx, const qgbdt_params *params);
int qgbdt_destroy(qgbdt_ctx *ctx);
/* Message of the last error on this context (owned by the context; "" if none). */
const char *qgbdt_last_error(const qgbdt_ctx *ctx);

/* Loads the bin matrix data[N][J] of Algorithm 1: one uint8 bin code per (row, feature),
 * every code < n_bins (2..256).  layout 0: row-major, element (i, j) at d_bins[i*ld + j];
 * layout 1: column-major, element (i, j) at d_bins[j*ld + i].  The matrix is copied into
 * an internal feature-tiled layout, so d_bins may be freed once the stream work is done.
 * Resets the leaf state to the single root leaf.  Synchronises (it checks the codes and
 * returns QGBDT_ERR_VALUE for a code >= n_bins).  n_rows < 2^31. */
int qgbdt_load_binned(qgbdt_ctx *ctx, const uint8_t *d_bins, int64_t n_rows, int32_t n_features,
                      int32_t n_bins, int32_t layout, int64_t ld, void *stream);
/* Same with the matrix in HOST memory (pinned or pageable); the copy to the device is part
 * of the call. */
int qgbdt_load_binned_host(qgbdt_ctx *ctx, const uint8_t *h_bins, int64_t n_rows, int32_t n_features,
                           int32_t n_bins, int32_t layout, int64_t ld, void *stream);

/* Eq. 1: gradients of the context's objective at the current scores.  d_h may be NULL for
 * the squared loss (constant hessian).  Asynchronous. */
int qgbdt_compute_gradients(qgbdt_ctx *ctx, const float *d_scores, const float *d_labels,
                            float *d_g, float *d_h, void *stream);

/* Eq. 5, 6, 8: quantizes the gradients of all rows for boosting iteration `tree`:
 * delta_g = max|g| / (2^(B-1) - 1), delta_h = max h / (2^B - 2), then stochastic rounding
 * with a counter hash of (seed, tree, row).  d_h == NULL: constant hessian, not quantized
 * (every row counts 1, delta_h = 1).  The packed per-row codes stay inside the context for
 * the histogram calls.  Optional outputs: d_gq [n_rows] int8, d_hq [n_rows] uint8 (device),
 * and the host scalars g_scale = delta_g, h_scale = delta_h, G_total, H_total (integer sums
 * over all rows).  Synchronises.  QGBDT_ERR_VALUE on bad gradient values. */
int qgbdt_quantize_gradients(qgbdt_ctx *ctx, const float *d_g, const float *d_h, uint32_t tree,
                             int8_t *d_gq, uint8_t *d_hq, double *g_scale, double *h_scale,
                             int64_t *G_total, int64_t *H_total, void *stream);

/* Algorithm 1 with integer gradients for the rows of `leaf`; d_hist [n_features][n_bins] is
 * overwritten.  Asynchronous. */
int qgbdt_build_histograms(qgbdt_ctx *ctx, int32_t leaf, qgbdt_bin *d_hist, void *stream);
/* The same for an explicit row list d_rows[n] (any order, duplicates counted twice). */
int qgbdt_build_histograms_rows(qgbdt_ctx *ctx, const uint32_t *d_rows, int64_t n, qgbdt_bin *d_hist,
                                void *stream);
/* Algorithm 1 as printed, without quantization: the histogram of the ORIGINAL single-precision
 * gradients (the floating-point baseline of Sec. 7.2's timing comparison), built on the same kernel
 * design as the integer one.  d_g, d_h [n_rows] (d_h == NULL: hessian 1); d_rows [n] a row list, or
 * NULL for all rows (then n must be n_rows); d_hist [n_features][n_bins][2] floats, gradient sum then
 * hessian sum, overwritten.  Float additions are order-dependent: the sums agree with a double-precision
 * sum to single-precision rounding error, not bit for bit.  Needs no quantize call.  Asynchronous. */
int qgbdt_build_histograms_fp32(qgbdt_ctx *ctx, const float *d_g, const float *d_h, const uint32_t *d_rows, int64_t n,
                                float *d_hist, void *stream);
/* Histogram subtraction: d_large = d_parent - d_small, bin by bin (the larger sibling's
 * histogram from its parent's and its smaller sibling's).  d_large may alias d_parent.
 * Asynchronous. */
int qgbdt_subtract_histograms(qgbdt_ctx *ctx, const qgbdt_bin *d_parent, const qgbdt_bin *d_small,
                              qgbdt_bin *d_large, void *stream);

/* Eq. 7: scans all (feature, threshold bin) candidates of a leaf whose integer totals are
 * G, H over n_rows rows, gain in double precision from the integer sums and the scales of
 * the last quantize call; ties go to the lowest (feature, bin).  Synchronises. */
int qgbdt_find_best_split(qgbdt_ctx *ctx, const qgbdt_bin *d_hist, int64_t G, int64_t H, int64_t n_rows,
                          qgbdt_split *h_out, void *stream);

/* The index sets I_s of Sec. 3: a split of leaf s by (feature, bin) divides I_s into the rows
 * with bin code <= bin, which stay in `leaf`, and the others, which form leaf *right_leaf
 * (a stable partition: relative order is kept on both sides).  Any (feature, bin) in range is
 * accepted, also one that leaves a side empty.  Synchronises. */
int qgbdt_split_leaf(qgbdt_ctx *ctx, int32_t leaf, int32_t feature, int32_t bin, int32_t *right_leaf,
                     int64_t *n_left, int64_t *n_right, void *stream);
/* Borrowed view of I_s (Sec. 3), the row list of a leaf: device memory inside the context,
 * valid until the next split or reset. */
int qgbdt_get_leaf_rows(qgbdt_ctx *ctx, int32_t leaf, const uint32_t **d_rows, int64_t *n);
/* Back to the state before any split (Sec. 3: the tree starts from a single root leaf whose
 * index set is all rows, ascending).  Asynchronous. */
int qgbdt_reset_leaves(qgbdt_ctx *ctx, void *stream);

/* Eq. 3 with the ORIGINAL gradients (leaf-value refitting, Sec. 4.2): for every current
 * leaf, w = -sum g / (sum h + lambda_l2) over its rows, sums taken in 2^-30 fixed point
 * (order-independent).  h_w [current leaves] receives w, h_value the leaf outputs
 * (float)(learning_rate * w); either may be NULL.  d_h == NULL: hessian 1.  Synchronises. */
int qgbdt_refit_leaves(qgbdt_ctx *ctx, const float *d_g, const float *d_h, double *h_w, float *h_value,
                       void *stream);

/* Fig. 1, last step of an iteration: adds to d_scores [n_rows] the output of the leaf every row
 * is in (the values of the last qgbdt_refit_leaves, which must have run for the current leaves:
 * QGBDT_ERR_STATE otherwise).  Asynchronous. */
int qgbdt_apply_leaf_values(qgbdt_ctx *ctx, float *d_scores, void *stream);

/* Fig. 1 workflow: trains boosting iterations first_tree .. first_tree + num_trees - 1
 * (gradients, quantization, leaf-wise growth with integer histograms and histogram
 * subtraction, refit, score update).  d_labels [n_rows]; d_scores [n_rows] holds the
 * current predictions on entry and the updated ones on return.  `model` (host) receives
 * the trees, tree k of this call in slot k.  Synchronises.
 * Memory: the first call after a load allocates the training workspaces, among them a
 * column-major copy of the bin codes (n_rows * n_features bytes) that the row partition
 * of a split reads; with option QGBDT_OPT_COLUMN_COPY set to 0, or if that allocation
 * fails, the partition reads the tiled matrix instead (same results, more memory
 * traffic); qgbdt_get_info(QGBDT_INFO_COLUMN_COPY) tells which path the last call took.
 * Gradients out of domain (QGBDT_ERR_VALUE) are reported when the call returns; the trees
 * from the offending iteration on are not grown (one leaf each). */
int qgbdt_train(qgbdt_ctx *ctx, const float *d_labels, float *d_scores, uint32_t first_tree,
                int32_t num_trees, qgbdt_model *model, void *stream);
/* Same with labels and scores in HOST memory; both copies are part of the call. */
int qgbdt_train_host(qgbdt_ctx *ctx, const float *h_labels, float *h_scores, uint32_t first_tree,
                     int32_t num_trees, qgbdt_model *model, void *stream);

/* Data-distributed training (Sec. 7.3: the rows are divided over the workers, the integer
 * histograms are summed across them).  This context holds rows [row_offset, row_offset + n_rows)
 * of a training set of total_rows rows (< 2^32, and total_rows * levels must fit the histogram
 * word like n_rows at load); rank in [0, world).  Every rank loads its shard, sets the same
 * parameters and calls qgbdt_train with its shard of labels and scores; the trees every rank
 * gets are identical, and identical to those one context trains on all rows: stochastic
 * rounding is keyed by the global row number, the two maxima of Eq. 5 are maximised and every
 * integer sum (totals, histograms of the root and of the smaller children, row counts, refit
 * sums) is added over the ranks, which is exact.  The exchange itself is the caller's:
 * `reduce` is called from the calling host thread whenever `count` words at device pointer d_buf
 * have to be combined in place over all ranks, kind QGBDT_REDUCE_SUM_I64 (64-bit integers, sum)
 * or QGBDT_REDUCE_MAX_U32 (32-bit unsigned integers, maximum); it must order the exchange after
 * the work already on `stream` and either finish it or enqueue it on `stream` (an NCCL all-reduce
 * on that stream does), and return 0, anything else aborts the train call with QGBDT_ERR_CUDA.
 * Every rank makes the same calls in the same order.  With ranks set, the passes of tree growth
 * run on the stream with the host following them.  world <= 1 or reduce == NULL switches the
 * mode off.  Set before qgbdt_train; model.leaf_count then holds global row counts. */
#define QGBDT_REDUCE_SUM_I64 0
#define QGBDT_REDUCE_MAX_U32 1
typedef int (*qgbdt_allreduce_fn)(void *user, void *d_buf, int64_t count, int32_t kind, void *stream);
int qgbdt_set_distributed(qgbdt_ctx *ctx, int32_t rank, int32_t world, int64_t row_offset, int64_t total_rows,
                          qgbdt_allreduce_fn reduce, void *user);

/* Options of a context (no counterpart in the paper).  Set them before qgbdt_load_binned /
 * qgbdt_train; unknown options and values out of range give QGBDT_ERR_ARG.
 *   QGBDT_OPT_COLUMN_COPY  1 (default): qgbdt_train keeps a column-major copy of the bin codes for
 *                          the row partition; 0: never (saves n_rows * n_features bytes).
 *   QGBDT_OPT_LEAF_VALUES  0 (default): qgbdt_train refits the leaf values from the original gradients
 *                          (Eq. 3, Sec. 4.2); 1: it takes them from the quantized sums of the leaves,
 *                          w~ = -(G~ delta_g) / (H~ delta_h + lambda_l2) (Sec. 4.2, first formula), and
 *                          skips the pass over the gradients.  May be changed between train calls. */
#define QGBDT_OPT_COLUMN_COPY 1
#define QGBDT_OPT_LEAF_VALUES 2
int qgbdt_set_option(qgbdt_ctx *ctx, int32_t option, int64_t value);
/* What the context is doing (host scalars, no synchronisation):
 *   QGBDT_INFO_COLUMN_COPY  1 when the training workspaces hold the column-major copy (the row
 *                           partition reads columns), 0 when they do not (it reads the tiles). */
#define QGBDT_INFO_COLUMN_COPY 1
int qgbdt_get_info(const qgbdt_ctx *ctx, int32_t what, int64_t *value);

/* Counters of the work done by qgbdt_train since the context was created:
 * kernel launches, histogram builds, and rows x features accumulated by them. */
int qgbdt_get_counters(const qgbdt_ctx *ctx, int64_t *kernel_launches, int64_t *hist_builds,
                       int64_t *hist_row_features);

/* Measurement aid (no counterpart in the paper): when enabled, every histogram build is
 * bracketed by a pair of CUDA events on its stream.  qgbdt_get_histogram_profile() waits for
 * them and returns the summed kernel time, the algorithmic bytes of those builds
 * (rows * (features + gradient-code bytes [+ 4 for a row list]) + features * bins * 8, with one
 * byte of packed gradient + hessian code per row up to 4 bits and two beyond) and their number,
 * then clears the record. */
int qgbdt_profile_histograms(qgbdt_ctx *ctx, int32_t enable);
int qgbdt_get_histogram_profile(qgbdt_ctx *ctx, double *total_ms, int64_t *total_bytes, int64_t *builds);
/* With the same switch on, qgbdt_train also brackets every phase of a boosting iteration (Fig. 1) with
 * events, and runs the passes of tree growth on the stream with the host following them (slower than
 * the graph it replays otherwise: this is for where the time goes, not for how long a tree takes).
 * h_ms [QGBDT_N_PHASES] receives the summed times since the switch was set or the record cleared,
 * h_intervals (may be NULL) the number of timed intervals; call it before
 * qgbdt_get_histogram_profile, which clears the record.  Phases, in order: gradients (Eq. 1),
 * quantization (Eq. 5, 6, 8), root histogram, row partition, children's histograms (Algorithm 1),
 * finish (merge, subtraction, Eq. 7), commit (best-first order and next batch), leaf values (Eq. 3),
 * score update. */
#define QGBDT_N_PHASES 9
int qgbdt_get_timings(qgbdt_ctx *ctx, double *h_ms, int64_t *h_intervals);

/* Histogram build that allocates nothing (the paper has no counterpart; it exists for callers
 * that are not allowed to call cudaMalloc: code running inside a memory pool that owns the
 * device, inside a loop where an allocation would stall the GPU, or in a plug-in whose host
 * bans allocator calls).  It needs no context.  It computes the same histogram as
 * qgbdt_build_histograms / qgbdt_build_histograms_rows from the caller's own arrays:
 *   d_bins  row-major bin matrix, element (i, j) at d_bins[i*ld + j], codes < n_bins
 *   d_gq    [n_rows] int8 quantized gradients, d_hq [n_rows] uint8 quantized hessians
 *           (the optional outputs of qgbdt_quantize_gradients)
 *   d_rows  [n] row list, or NULL for all rows (then n must equal n_rows)
 *   d_hist  [n_features][n_bins], overwritten
 *   d_status  optional device word the caller clears: set to 1 when a row index (>= n_rows), a bin
 *           code (>= n_bins) or a gradient code (-128) was out of range (such entries are skipped)
 * All pointers are device pointers owned by the caller.  The per-CTA partial histograms live in
 * a fixed 4 MiB array inside the library image (every GPU that loads the library holds it until
 * the process ends), so n_features * n_bins may be at most 16384; larger problems are refused
 * with QGBDT_ERR_ARG and need a context.  The call knows no bit width, so it bounds the sums by the
 * widest codes: n (entries of the list, or n_rows) may be at most 16 843 009 (n * 255 must fit the
 * 32-bit hessian field); more gives QGBDT_ERR_OVERFLOW.  The call makes no cudaMalloc / cudaFree and calls no
 * allocating routine.  The first call on a device looks up the array's device address; make
 * that first call outside any stream capture.  All calls share the one array, which keeps the
 * previous call's sums (each call clears what it uses): two calls whose kernels overlap on the
 * GPU -- different streams, or different host threads on different streams -- race; keep them on
 * one stream or order them with events.  Asynchronous on `stream`.  On failure
 * qgbdt_noalloc_last_error() gives the reason (per host thread). */
int qgbdt_build_histograms_noalloc(const uint8_t *d_bins, int64_t n_rows, int32_t n_features, int32_t n_bins,
                                   int64_t ld, const int8_t *d_gq, const uint8_t *d_hq, const uint32_t *d_rows,
                                   int64_t n, qgbdt_bin *d_hist, int32_t *d_status, void *stream);
const char *qgbdt_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* QGBDT_H */
