// Eq. 3 with the original gradients (leaf-value refitting, Sec. 4.2) and the score update.
// Sums are taken in 2^-30 fixed point: each term is rounded once, the 64-bit integer sum is
// exact, so the result does not depend on the order in which rows are added.
#include "qgbdt_internal.cuh"

namespace {

constexpr int REFIT_THREADS = 256;
constexpr int REFIT_ITEMS = 16;
constexpr int REFIT_BLOCK = REFIT_THREADS * REFIT_ITEMS;
constexpr int REFIT_LOCAL = 64;  // leaf slots a block can accumulate in shared memory

// Slot (index into the offset-sorted leaf table) of position p: last slot with offs[s] <= p.
__device__ inline int slot_of(const uint32_t *offs, int n_leaves, uint32_t p) {
    int lo = 0, hi = n_leaves - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (offs[mid] <= p) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__device__ inline long long to_fixed(float v) { return __double2ll_rn(__dmul_rn((double)v, 1073741824.0)); }

// The step-wise interface: table: [n_leaves] offsets ascending, then [n_leaves] leaf ids; the leaf
// of position p of the row list is the last table entry whose offset is <= p.  sums: [leaves][2].
__global__ void __launch_bounds__(REFIT_THREADS) k_refit_sums(const uint32_t *__restrict__ idx, uint32_t n,
                                                              const uint32_t *__restrict__ table, int n_leaves,
                                                              const float *__restrict__ g, const float *__restrict__ h,
                                                              long long *__restrict__ sums) {
    extern __shared__ uint32_t offs[];  // n_leaves offsets
    __shared__ unsigned long long acc[REFIT_LOCAL][2];
    for (int i = threadIdx.x; i < n_leaves; i += REFIT_THREADS) offs[i] = table[i];
    for (int i = threadIdx.x; i < REFIT_LOCAL * 2; i += REFIT_THREADS) (&acc[0][0])[i] = 0ull;
    __syncthreads();
    const uint32_t p0 = blockIdx.x * REFIT_BLOCK;
    const uint32_t p1 = min(n, p0 + REFIT_BLOCK);
    const int s_lo = slot_of(offs, n_leaves, p0);
    const int lane = threadIdx.x & 31;
#pragma unroll 4
    for (int j = 0; j < REFIT_ITEMS; ++j) {
        const uint32_t p = p0 + j * REFIT_THREADS + threadIdx.x;
        const bool ok = p < p1;
        int s = -1;
        long long gf = 0, hf = 0;
        if (ok) {
            s = slot_of(offs, n_leaves, p);
            const uint32_t row = idx[p];
            gf = to_fixed(g[row]);
            hf = h ? to_fixed(h[row]) : 1073741824LL;
        }
        const int s0 = __shfl_sync(0xffffffffu, s, 0);
        if (__all_sync(0xffffffffu, s == s0)) {
            if (s0 < 0) continue;  // whole warp past the end
            for (int o = 16; o > 0; o >>= 1) {
                gf += __shfl_xor_sync(0xffffffffu, gf, o);
                hf += __shfl_xor_sync(0xffffffffu, hf, o);
            }
            if (lane == 0) {
                if (s0 - s_lo < REFIT_LOCAL) {
                    atomicAdd(&acc[s0 - s_lo][0], (unsigned long long)gf);
                    atomicAdd(&acc[s0 - s_lo][1], (unsigned long long)hf);
                } else {
                    const uint32_t leaf = table[n_leaves + s0];
                    atomicAdd(reinterpret_cast<unsigned long long *>(&sums[2 * leaf]), (unsigned long long)gf);
                    atomicAdd(reinterpret_cast<unsigned long long *>(&sums[2 * leaf + 1]), (unsigned long long)hf);
                }
            }
        } else if (ok) {
            if (s - s_lo < REFIT_LOCAL) {
                atomicAdd(&acc[s - s_lo][0], (unsigned long long)gf);
                atomicAdd(&acc[s - s_lo][1], (unsigned long long)hf);
            } else {
                const uint32_t leaf = table[n_leaves + s];
                atomicAdd(reinterpret_cast<unsigned long long *>(&sums[2 * leaf]), (unsigned long long)gf);
                atomicAdd(reinterpret_cast<unsigned long long *>(&sums[2 * leaf + 1]), (unsigned long long)hf);
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < REFIT_LOCAL; i += REFIT_THREADS) {
        if (s_lo + i < n_leaves && (acc[i][0] | acc[i][1]) != 0ull) {
            const uint32_t leaf = table[n_leaves + s_lo + i];
            atomicAdd(reinterpret_cast<unsigned long long *>(&sums[2 * leaf]), acc[i][0]);
            atomicAdd(reinterpret_cast<unsigned long long *>(&sums[2 * leaf + 1]), acc[i][1]);
        }
    }
}

// w = -sum g / (sum h + lambda); output (float)(learning_rate * w); sums and outputs by leaf id.
__global__ void k_leaf_values(const long long *__restrict__ sums, int n_leaves, const GrowState *gs, double lambda,
                              double lr, double *__restrict__ w_out, float *__restrict__ v_out) {
    if (gs) n_leaves = gs->n_leaves;
    for (int leaf = blockIdx.x * blockDim.x + threadIdx.x; leaf < n_leaves; leaf += gridDim.x * blockDim.x) {
        const double den = __dadd_rn((double)sums[2 * leaf + 1], __dmul_rn(lambda, 1073741824.0));
        const double w = den > 0.0 ? __ddiv_rn(-(double)sums[2 * leaf], den) : 0.0;
        w_out[leaf] = w;
        v_out[leaf] = __double2float_rn(__dmul_rn(lr, w));
    }
}

// Sec. 4.2, leaf values without refitting: w~ = -(G~ delta_g) / (H~ delta_h + lambda) from the integer
// totals of every numbered leaf of a tree grown on the device; output (float)(learning_rate * w~).
__global__ void k_leaf_values_quantized(const LeafRec *__restrict__ leaves, const NodeRec *__restrict__ recs,
                                        const GrowState *gs, const DevState *state, int kg, int kh, int const_h,
                                        double lambda, double lr, double *__restrict__ w_out, float *__restrict__ v_out) {
    const int n_leaves = gs->n_leaves;
    const double dg = __ddiv_rn((double)__uint_as_float(state->gmax_bits), (double)kg);
    const double dh = const_h ? 1.0 : __ddiv_rn((double)__uint_as_float(state->hmax_bits), (double)kh);
    for (int leaf = blockIdx.x * blockDim.x + threadIdx.x; leaf < n_leaves; leaf += gridDim.x * blockDim.x) {
        const NodeRec *q = recs + leaves[leaf].rec;
        const double gd = __dmul_rn((double)q->G, dg);
        const double hd = __dadd_rn(__dmul_rn((double)q->H, dh), lambda);
        const double w = hd > 0.0 ? __ddiv_rn(-gd, hd) : 0.0;
        w_out[leaf] = w;
        v_out[leaf] = __double2float_rn(__dmul_rn(lr, w));
    }
}

// The step-wise interface.  Dynamic shared memory: [n_leaves] offsets, [n_leaves] values, so that a
// row costs a search in shared memory and two global accesses (its index, its score).  Four rows
// per thread are in flight.
__global__ void __launch_bounds__(REFIT_THREADS) k_apply_values(const uint32_t *__restrict__ idx, uint32_t n,
                                                                const uint32_t *__restrict__ table, int n_leaves,
                                                                const float *__restrict__ values,
                                                                float *__restrict__ scores) {
    extern __shared__ uint32_t offs[];
    float *vals = reinterpret_cast<float *>(offs + n_leaves);
    for (int i = threadIdx.x; i < n_leaves; i += REFIT_THREADS) {
        offs[i] = table[i];
        vals[i] = values[table[n_leaves + i]];
    }
    __syncthreads();
    const uint32_t stride = gridDim.x * REFIT_THREADS;
    for (uint32_t p0 = blockIdx.x * REFIT_THREADS + threadIdx.x; p0 < n; p0 += 4 * stride) {
        uint32_t row[4];
        float add[4], old[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t p = p0 + k * stride;
            row[k] = 0xFFFFFFFFu;
            add[k] = 0.f;
            if (p < n) {
                add[k] = vals[slot_of(offs, n_leaves, p)];
                row[k] = idx[p];
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) old[k] = row[k] != 0xFFFFFFFFu ? scores[row[k]] : 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (row[k] != 0xFFFFFFFFu) scores[row[k]] = __fadd_rn(old[k], add[k]);
    }
}

// ---- trees grown on the device: rows find their leaf by walking the finished tree -------------
//
// The growth kernels may have partitioned rows further than the finished tree goes (leaves split
// ahead of the best-first order that the tree did not use), so the leaf of a row is not read from
// the row lists: every row walks the tree's nodes with its own bin codes (bin <= threshold: left).
// Rows are visited in row order: the row's codes, its gradients and its score are read and
// written in streams, and the leaf number is kept (16 bits per row) for the score update.

struct WalkNode {           // a node of the tree being walked, in shared memory (16 bytes: one load)
    int32_t left, right;    // children: a node >= 0, or ~leaf
    uint8_t logW, shift, bin, byte;   // tile width, bit position in the word, threshold; byte of a 32-byte row
    int32_t feature;
};

// The same for a matrix of one tile of 32-byte rows, in 8 bytes (32 lanes at 32 different nodes: half the
// shared-memory wavefronts of the 16-byte node): children in 16 bits each (a context takes at most 4096
// leaves), then the threshold and the byte of the row.
__device__ __forceinline__ uint2 pack_node8(int left, int right, int bin, int byte) {
    return make_uint2(((uint32_t)left & 0xFFFFu) | ((uint32_t)right << 16), (uint32_t)(bin & 0xFF) | ((uint32_t)(byte & 0xFF) << 8));
}

constexpr int WALK_THREADS = 256;

// *p (two adjacent 32-bit shared words, low then high) += v, with 32-bit atomics.
__device__ __forceinline__ void add64(uint32_t *p, unsigned long long v) {
    const uint32_t lo = (uint32_t)v, hi = (uint32_t)(v >> 32);
    const uint32_t old = atomicAdd(p, lo);
    const uint32_t carry = old + lo < old ? 1u : 0u;
    if (hi + carry) atomicAdd(p + 1, hi + carry);
}

// nodes, then the refit sums of the block, then (32-byte rows) the block's rows, nine words apart
__host__ __device__ inline size_t walk_smem_bytes(int L, bool sums, bool rows) {
    return (size_t)(L > 1 ? L - 1 : 1) * sizeof(WalkNode) + (sums ? (size_t)L * 2 * sizeof(unsigned long long) : 0) +
           (rows ? (size_t)WALK_THREADS * 9 * sizeof(uint32_t) : 0);
}

// Stores the tree's leaf count and rows per leaf, and zeroes the refit sums.  One block.
__global__ void __launch_bounds__(256) k_tree_prepare(const LeafRec *__restrict__ leaves, const GrowState *gs, int max_leaves,
                                                      long long *__restrict__ sums, int32_t *__restrict__ m_num_leaves,
                                                      long long *__restrict__ m_leaf_count) {
    const int L = gs->n_leaves;
    for (int i = threadIdx.x; i < L; i += 256) m_leaf_count[i] = leaves[i].n_all;
    for (int i = threadIdx.x; i < 2 * max_leaves; i += 256) sums[i] = 0;   // all: a sharded run adds the whole array over the ranks
    if (threadIdx.x == 0) *m_num_leaves = L;
}

// SUMS: also adds the row's gradients (2^-30 fixed point) to its leaf's sums (Eq. 3).
// ROW_LOGW == 3: the matrix is one tile of 32-byte rows: a thread loads its whole row once
// (consecutive threads, consecutive rows: a coalesced stream) into shared memory, nine words from
// row to row so that the threads' accesses never share a bank, and reads the code of every node it
// passes as one byte from there.  -1: any tiling, one global load per node passed.
template <bool SUMS, int ROW_LOGW>
__global__ void __launch_bounds__(WALK_THREADS) k_walk(const GrowState *gs, const FeatRec *__restrict__ feat_rec,
                                                       const int32_t *__restrict__ m_feature, const int32_t *__restrict__ m_bin,
                                                       const int32_t *__restrict__ m_left, const int32_t *__restrict__ m_right,
                                                       uint32_t n, const float *__restrict__ g, const float *__restrict__ h,
                                                       uint16_t *__restrict__ leaf_id, long long *__restrict__ sums) {
    extern __shared__ __align__(16) unsigned char wsm[];
    const int L = gs->n_leaves, n_nodes = L - 1;
    WalkNode *nodes = reinterpret_cast<WalkNode *>(wsm);
    unsigned long long *acc = reinterpret_cast<unsigned long long *>(wsm + (size_t)(n_nodes > 0 ? n_nodes : 1) * sizeof(WalkNode));
    uint32_t *srow = reinterpret_cast<uint32_t *>(acc + (SUMS ? 2 * L : 0)) + threadIdx.x * 9;   // this thread's row
    uint2 *nodes8 = reinterpret_cast<uint2 *>(wsm);   // ROW_LOGW == 3: 8-byte nodes in the same place
    for (int i = threadIdx.x; i < n_nodes; i += WALK_THREADS) {
        const int f = m_feature[i];
        const FeatRec fr = feat_rec[f];
        if (ROW_LOGW == 3) {
            nodes8[i] = pack_node8(m_left[i], m_right[i], m_bin[i], fr.fl);
            continue;
        }
        WalkNode w;
        w.left = m_left[i]; w.right = m_right[i];
        w.logW = (uint8_t)fr.logW; w.shift = (uint8_t)(8 * fr.byte); w.bin = (uint8_t)m_bin[i]; w.byte = (uint8_t)fr.fl;
        w.feature = f;
        nodes[i] = w;
    }
    uint32_t *acc32 = reinterpret_cast<uint32_t *>(acc);   // [L][g lo, g hi, h lo, h hi]
    if (SUMS)
        for (int i = threadIdx.x; i < 4 * L; i += WALK_THREADS) acc32[i] = 0u;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    for (uint32_t base = blockIdx.x * WALK_THREADS + (threadIdx.x & ~31u); base < n; base += gridDim.x * WALK_THREADS) {
        const uint32_t r = base + lane;
        const bool active = r < n;
        int leaf = 0;
        if (active && n_nodes > 0) {
            if (ROW_LOGW == 3) {
                const uint4 *row = reinterpret_cast<const uint4 *>(feat_rec[0].col + ((size_t)r << 3));   // feature 0: word 0 of the tile
                const uint4 v0 = row[0], v1 = row[1];
                srow[0] = v0.x; srow[1] = v0.y; srow[2] = v0.z; srow[3] = v0.w;
                srow[4] = v1.x; srow[5] = v1.y; srow[6] = v1.z; srow[7] = v1.w;
            }
            int node = 0;
            for (;;) {
                int next;
                if (ROW_LOGW == 3) {
                    const uint2 w = nodes8[node];
                    const uint32_t code = reinterpret_cast<const uint8_t *>(srow)[(w.y >> 8) & 0xFFu];
                    next = code <= (w.y & 0xFFu) ? (int)(short)(w.x & 0xFFFFu) : (int)w.x >> 16;
                } else {
                    const WalkNode w = nodes[node];
                    const FeatRec fr = feat_rec[w.feature];
                    const uint32_t code = (fr.col[(size_t)r << w.logW] >> w.shift) & 0xFFu;
                    next = code <= w.bin ? w.left : w.right;
                }
                if (next < 0) { leaf = ~next; break; }
                node = next;
            }
        }
        if (active) leaf_id[r] = (uint16_t)leaf;
        if (SUMS) {
            // Consecutive rows often share a leaf (a few leaves hold most rows), and lanes adding to
            // one shared word serialise: up to two rounds in which the lanes of one leaf add up
            // their terms with shuffles and one lane adds the sum; what is left adds on its own.
            // 64-bit sums are two 32-bit shared atomics each (the low word's old value tells the
            // carry); a constant hessian only counts rows.
            const long long gf = active ? to_fixed(g[r]) : 0;
            const long long hf = (active && h) ? to_fixed(h[r]) : 0;
            unsigned rem = __ballot_sync(0xffffffffu, active);
            for (int round = 0; round < 2 && rem; ++round) {
                const int src = __ffs(rem) - 1;
                const int l0 = __shfl_sync(0xffffffffu, leaf, src);
                const bool mine = ((rem >> lane) & 1u) && leaf == l0;
                const unsigned m = __ballot_sync(0xffffffffu, mine);
                if (__popc(m) >= 4) {
                    long long gs_ = mine ? gf : 0, hs_ = mine ? hf : 0;
                    for (int o = 16; o > 0; o >>= 1) {
                        gs_ += __shfl_xor_sync(0xffffffffu, gs_, o);
                        if (h) hs_ += __shfl_xor_sync(0xffffffffu, hs_, o);
                    }
                    if (lane == src) {
                        add64(acc32 + 4 * l0, (unsigned long long)gs_);
                        if (h) add64(acc32 + 4 * l0 + 2, (unsigned long long)hs_);
                        else atomicAdd(acc32 + 4 * l0 + 2, (uint32_t)__popc(m));
                    }
                    rem &= ~m;
                } else {
                    break;   // the leaves of this warp are spread out: no gain in adding up first
                }
            }
            if ((rem >> lane) & 1u) {
                add64(acc32 + 4 * leaf, (unsigned long long)gf);
                if (h) add64(acc32 + 4 * leaf + 2, (unsigned long long)hf);
                else atomicAdd(acc32 + 4 * leaf + 2, 1u);
            }
        }
    }
    if (SUMS) {
        __syncthreads();
        for (int i = threadIdx.x; i < 2 * L; i += WALK_THREADS) {
            unsigned long long v = ((unsigned long long)acc32[2 * i + 1] << 32) | acc32[2 * i];
            if ((i & 1) && !h) v = (unsigned long long)acc32[2 * i] << 30;   // rows counted, each 2^30
            if (v != 0ull) atomicAdd(reinterpret_cast<unsigned long long *>(&sums[i]), v);
        }
    }
}

// scores[r] += value of r's leaf, in row order.
__global__ void __launch_bounds__(256) k_apply_ids(const uint16_t *__restrict__ leaf_id, const float *__restrict__ values,
                                                   uint32_t n, float *__restrict__ scores) {
    for (uint32_t r = blockIdx.x * 256 + threadIdx.x; r < n; r += gridDim.x * 256)
        scores[r] = __fadd_rn(scores[r], values[leaf_id[r]]);
}

// Writes the offset-sorted leaf table into pinned memory and queues its copy to the device.
int upload_table(qgbdt_ctx *c, cudaStream_t st) {
    const int L = c->n_leaves;
    uint32_t *tab = reinterpret_cast<uint32_t *>(c->h_pinned);
    std::vector<int> order(L);
    for (int i = 0; i < L; ++i) order[i] = i;
    // Order: offset, then empty leaves before the non-empty one that starts at the same offset (a
    // split that sends every row to one side leaves an empty leaf there; the search takes the last
    // slot whose offset is <= the position, which must be the leaf that owns the rows), then leaf
    // number.
    auto before = [&](int a, int b) {
        if (c->leaf_off[a] != c->leaf_off[b]) return c->leaf_off[a] < c->leaf_off[b];
        const bool ea = c->leaf_n[a] == 0, eb = c->leaf_n[b] == 0;
        if (ea != eb) return ea;
        return a < b;
    };
    for (int i = 1; i < L; ++i) {  // insertion sort (lists are short and nearly sorted)
        const int v = order[i];
        int j = i - 1;
        while (j >= 0 && before(v, order[j])) { order[j + 1] = order[j]; --j; }
        order[j + 1] = v;
    }
    for (int s = 0; s < L; ++s) {
        tab[s] = (uint32_t)c->leaf_off[order[s]];
        tab[L + s] = (uint32_t)order[s];
    }
    QG_CUDA(c, cudaMemcpyAsync(c->d_leaf_table, tab, sizeof(uint32_t) * 2 * L, cudaMemcpyHostToDevice, st));
    return QGBDT_OK;
}

}  // namespace

int qg_refit(qgbdt_ctx *c, const float *d_g, const float *d_h, cudaStream_t st) {
    const int L = c->n_leaves;
    int rc = upload_table(c, st);
    if (rc != QGBDT_OK) return rc;
    QG_CUDA(c, cudaMemsetAsync(c->d_leaf_sums, 0, sizeof(long long) * 2 * L, st));
    const unsigned blocks = (unsigned)((c->N + REFIT_BLOCK - 1) / REFIT_BLOCK);
    k_refit_sums<<<blocks, REFIT_THREADS, sizeof(uint32_t) * L, st>>>(c->d_idx, (uint32_t)c->N, c->d_leaf_table, L, d_g, d_h,
                                                                     c->d_leaf_sums);
    QG_LAUNCH_CHECK(c);
    k_leaf_values<<<(L + 255) / 256, 256, 0, st>>>(c->d_leaf_sums, L, nullptr, c->prm.lambda_l2, c->prm.learning_rate,
                                                   c->d_leaf_w, c->d_leaf_value);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

// Requires the leaf table uploaded by the preceding qg_refit on the same stream.
int qg_apply_leaf_values(qgbdt_ctx *c, float *d_scores, cudaStream_t st) {
    const int L = c->n_leaves;
    unsigned blocks = (unsigned)((c->N + REFIT_THREADS - 1) / REFIT_THREADS);
    if (blocks > (unsigned)c->sm_count * 16) blocks = (unsigned)c->sm_count * 16;
    k_apply_values<<<blocks, REFIT_THREADS, sizeof(uint32_t) * 2 * L, st>>>(c->d_idx, (uint32_t)c->N, c->d_leaf_table, L,
                                                                       c->d_leaf_value, d_scores);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

// Leaf values (Eq. 3 with the original gradients, or Sec. 4.2's values from the quantized sums)
// and score update for the tree just grown on the device; leaf values and counts go to slot
// `tree_slot` of the device-side model arrays.
int qg_refit_grown(qgbdt_ctx *c, const float *d_g, const float *d_h, float *d_scores, int tree_slot, cudaStream_t st) {
    const int L = c->prm.num_leaves;     // upper bound; the kernels read the real count from the grow state
    const size_t no = (size_t)tree_slot * (L > 1 ? L - 1 : 1);
    const bool refit = !c->leaf_values_quantized;
    int prc = qg_phase_begin(c, QG_PHASE_REFIT, st);
    if (prc != QGBDT_OK) return prc;
    k_tree_prepare<<<1, 256, 0, st>>>(c->d_leaves, c->d_gs, L, c->d_leaf_sums, c->d_m_num_leaves + tree_slot,
                                      c->d_m_leaf_count + (size_t)tree_slot * L);
    QG_LAUNCH_CHECK(c);
    // one tile of 32-byte rows (up to 32 features): the walk stages the row in shared memory
    const bool row8 = c->tiles.size() == 1 && c->tiles[0].logW == 3;
    const size_t smem = walk_smem_bytes(L, refit, row8);
    static bool configured[64] = {};
    if (smem > 48 * 1024 && (c->device < 0 || c->device >= 64 || !configured[c->device])) {
        const int cap_s = (int)walk_smem_bytes(4096, true, true), cap_n = (int)walk_smem_bytes(4096, false, true);
        QG_CUDA(c, cudaFuncSetAttribute(k_walk<true, -1>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap_s));
        QG_CUDA(c, cudaFuncSetAttribute(k_walk<false, -1>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap_n));
        QG_CUDA(c, cudaFuncSetAttribute(k_walk<true, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap_s));
        QG_CUDA(c, cudaFuncSetAttribute(k_walk<false, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap_n));
        if (c->device >= 0 && c->device < 64) configured[c->device] = true;
    }
    unsigned wb = (unsigned)((c->N + WALK_THREADS - 1) / WALK_THREADS);
    if (wb > (unsigned)c->sm_count * 8) wb = (unsigned)c->sm_count * 8;
    auto walk = [&](auto kern, const float *gg, const float *hh, long long *sums) {
        kern<<<wb, WALK_THREADS, smem, st>>>(c->d_gs, c->d_feat_rec, c->d_m_feature + no, c->d_m_bin + no, c->d_m_left + no,
                                             c->d_m_right + no, (uint32_t)c->N, gg, hh, c->d_leaf_id, sums);
    };
    if (refit) {
        if (row8) walk(k_walk<true, 3>, d_g, d_h, c->d_leaf_sums);
        else walk(k_walk<true, -1>, d_g, d_h, c->d_leaf_sums);
        QG_LAUNCH_CHECK(c);
        if ((prc = qg_allreduce(c, c->d_leaf_sums, 2 * (int64_t)L, QGBDT_REDUCE_SUM_I64, st)) != QGBDT_OK) return prc;
        k_leaf_values<<<(L + 255) / 256, 256, 0, st>>>(c->d_leaf_sums, L, c->d_gs, c->prm.lambda_l2, c->prm.learning_rate,
                                                       c->d_leaf_w, c->d_m_leaf_value + (size_t)tree_slot * L);
        QG_LAUNCH_CHECK(c);
    } else {
        if (row8) walk(k_walk<false, 3>, nullptr, nullptr, nullptr);
        else walk(k_walk<false, -1>, nullptr, nullptr, nullptr);
        QG_LAUNCH_CHECK(c);
        k_leaf_values_quantized<<<(L + 255) / 256, 256, 0, st>>>(
            c->d_leaves, c->d_recs, c->d_gs, c->d_state, qg_levels_g(c->prm.bits),
            qg_levels_h(c->prm.bits, c->prm.hess_levels_mode), c->const_hess ? 1 : 0, c->prm.lambda_l2,
            c->prm.learning_rate, c->d_leaf_w, c->d_m_leaf_value + (size_t)tree_slot * L);
        QG_LAUNCH_CHECK(c);
    }
    if ((prc = qg_phase_end(c, st)) != QGBDT_OK) return prc;
    if ((prc = qg_phase_begin(c, QG_PHASE_SCORES, st)) != QGBDT_OK) return prc;
    unsigned ab = (unsigned)((c->N + 255) / 256);
    if (ab > (unsigned)c->sm_count * 16) ab = (unsigned)c->sm_count * 16;
    k_apply_ids<<<ab, 256, 0, st>>>(c->d_leaf_id, c->d_m_leaf_value + (size_t)tree_slot * L, (uint32_t)c->N, d_scores);
    QG_LAUNCH_CHECK(c);
    return qg_phase_end(c, st);
}
