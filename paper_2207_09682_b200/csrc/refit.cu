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

// table: [n_slots] offsets ascending, then [n_slots] leaf ids.  A slot is a range of positions
// whose rows belong to one leaf; the step-wise interface has one slot per leaf.  sums: [leaves][2]
// by leaf id.  gs != nullptr: a tree grown on the device: the slot count comes from *gs (a leaf
// whose rows were partitioned further ahead of the best-first order is covered by several slots)
// and the table's third part [n_slots] says which (row, code) pair buffer holds a slot's rows
// (-1: the identity list).
__device__ inline uint32_t leaf_row(const uint32_t *idx, const uint2 *ent0, const uint2 *ent1, const uint32_t *table,
                                    int n_leaves, bool grown, int s, uint32_t p) {
    if (!grown) return idx[p];
    const int buf = (int)table[2 * n_leaves + s];
    return buf < 0 ? p : (buf ? ent1[p].x : ent0[p].x);
}

__global__ void __launch_bounds__(REFIT_THREADS) k_refit_sums(const uint32_t *__restrict__ idx,
                                                              const uint2 *__restrict__ ent0,
                                                              const uint2 *__restrict__ ent1, uint32_t n,
                                                              const uint32_t *__restrict__ table, int n_leaves,
                                                              const GrowState *gs, const float *__restrict__ g,
                                                              const float *__restrict__ h,
                                                              long long *__restrict__ sums) {
    extern __shared__ uint32_t offs[];  // n_leaves offsets
    const bool grown = gs != nullptr;
    if (grown) n_leaves = gs->n_segs;   // slots
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
            const uint32_t row = leaf_row(idx, ent0, ent1, table, n_leaves, grown, s, p);
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

// Dynamic shared memory: [n_slots] offsets, [n_slots] values, [n_slots] pair buffers, so that
// a row costs a search in shared memory and two global accesses (its pair, its score).  Four
// rows per thread are in flight.
__global__ void __launch_bounds__(REFIT_THREADS) k_apply_values(const uint32_t *__restrict__ idx,
                                                                const uint2 *__restrict__ ent0,
                                                                const uint2 *__restrict__ ent1, uint32_t n,
                                                                const uint32_t *__restrict__ table, int n_leaves,
                                                                const GrowState *gs,
                                                                const float *__restrict__ values,
                                                                float *__restrict__ scores) {
    extern __shared__ uint32_t offs[];
    const bool grown = gs != nullptr;
    if (grown) n_leaves = gs->n_segs;   // slots
    float *vals = reinterpret_cast<float *>(offs + n_leaves);
    int *bufs = reinterpret_cast<int *>(offs + 2 * n_leaves);
    for (int i = threadIdx.x; i < n_leaves; i += REFIT_THREADS) {
        offs[i] = table[i];
        vals[i] = values[table[n_leaves + i]];
        bufs[i] = grown ? (int)table[2 * n_leaves + i] : 0;
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
                const int sl = slot_of(offs, n_leaves, p);
                add[k] = vals[sl];
                if (!grown) row[k] = idx[p];
                else row[k] = bufs[sl] < 0 ? p : (bufs[sl] ? ent1[p].x : ent0[p].x);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) old[k] = row[k] != 0xFFFFFFFFu ? scores[row[k]] : 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (row[k] != 0xFFFFFFFFu) scores[row[k]] = __fadd_rn(old[k], add[k]);
    }
}

// Leaf table of a tree grown on the device.  A numbered leaf that was never split ahead of the
// best-first order is one slot: its range of its pair buffer.  A leaf that was split ahead without
// the tree using the split still owns the same rows, but only the deepest ranges written hold
// them intact (the scatter of a grandchild reuses the leaf's own buffer), so such a leaf is
// covered by the slots of its descendants: a record none of whose children has been split is
// intact in its own buffer.  Slots are ranked by (offset, empty first, order of discovery);
// [S] offsets, [S] leaf numbers, [S] pair buffers.  Also zeroes the sums and stores the tree's leaf
// count and rows per leaf.  One block; `seg` is scratch for 4 S words.
__global__ void __launch_bounds__(256) k_leaf_table(const LeafRec *__restrict__ leaves, const NodeRec *__restrict__ recs,
                                                    GrowState *gs, uint32_t *__restrict__ table, uint32_t *__restrict__ seg,
                                                    int max_segs, int max_leaves, long long *__restrict__ sums,
                                                    int32_t *__restrict__ m_num_leaves,
                                                    long long *__restrict__ m_leaf_count, DevState *state) {
    const int L = gs->n_leaves;
    __shared__ int n_segs;
    if (threadIdx.x == 0) n_segs = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < L; i += 256) {
        int stack[GROW_SLACK + GROW_MAX_JOBS + 4];
        int sp = 0;
        stack[sp++] = leaves[i].rec;
        while (sp > 0) {
            const int r = stack[--sp];
            const NodeRec q = recs[r];
            const bool deeper = q.state == 1 && (recs[q.child0].state == 1 || recs[q.child0 + 1].state == 1);
            if (deeper && sp + 2 <= GROW_SLACK + GROW_MAX_JOBS + 4) {
                stack[sp++] = q.child0 + 1;
                stack[sp++] = q.child0;
            } else {
                if (deeper) atomicExch(&state->kernel_error, 1);   // deeper than the slack allows: cannot happen
                const int k = atomicAdd(&n_segs, 1);
                if (k < max_segs) {
                    seg[4 * k] = q.off;
                    seg[4 * k + 1] = q.n;
                    seg[4 * k + 2] = (uint32_t)q.buf;
                    seg[4 * k + 3] = (uint32_t)i;
                }
            }
        }
        m_leaf_count[i] = leaves[i].n_all;
    }
    for (int i = threadIdx.x; i < 2 * max_leaves; i += 256) sums[i] = 0;   // all of them: a sharded run adds the whole array over the ranks
    __syncthreads();
    int S = n_segs;
    if (S > max_segs) {
        if (threadIdx.x == 0) atomicExch(&state->kernel_error, 1);
        S = max_segs;
    }
    __threadfence_block();
    for (int i = threadIdx.x; i < S; i += 256) {
        const uint32_t off = seg[4 * i], n = seg[4 * i + 1];
        int rank = 0;
        for (int j = 0; j < S; ++j) {
            const uint32_t oj = seg[4 * j], nj = seg[4 * j + 1];
            const bool before = oj < off || (oj == off && ((nj == 0) > (n == 0) || ((nj == 0) == (n == 0) && j < i)));
            rank += before ? 1 : 0;
        }
        table[rank] = off;
        table[S + rank] = seg[4 * i + 3];
        table[2 * S + rank] = seg[4 * i + 2];
    }
    if (threadIdx.x == 0) {
        *m_num_leaves = L;
        gs->n_segs = S;
    }
}

// Writes the offset-sorted leaf table into pinned memory and queues its copy to the device.
int upload_table(qgbdt_ctx *c, cudaStream_t st) {
    const int L = c->n_leaves;
    uint32_t *tab = reinterpret_cast<uint32_t *>(c->h_pinned);
    std::vector<int> order(L);
    for (int i = 0; i < L; ++i) order[i] = i;
    // Order: offset, then empty leaves before the non-empty one that starts at the same offset (a
    // split that sends every row to one side leaves an empty leaf there; the search below takes the
    // last slot whose offset is <= the position, which must be the leaf that owns the rows), then
    // leaf number: the same ranking as k_leaf_table.
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
    k_refit_sums<<<blocks, REFIT_THREADS, sizeof(uint32_t) * L, st>>>(c->d_idx, nullptr, nullptr, (uint32_t)c->N,
                                                                     c->d_leaf_table, L, nullptr, d_g, d_h,
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
    k_apply_values<<<blocks, REFIT_THREADS, sizeof(uint32_t) * 3 * L, st>>>(c->d_idx, nullptr, nullptr, (uint32_t)c->N,
                                                                       c->d_leaf_table, L, nullptr, c->d_leaf_value,
                                                                       d_scores);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

// Refit (Eq. 3 with the original gradients) and score update for the tree just grown on the
// device; leaf values and counts go to slot `tree_slot` of the device-side model arrays.
int qg_refit_grown(qgbdt_ctx *c, const float *d_g, const float *d_h, float *d_scores, int tree_slot, cudaStream_t st) {
    const int L = c->prm.num_leaves;     // upper bound; the kernels read the real counts from the grow state
    const int S = qg_leaf_table_slots(L);
    int prc = qg_phase_begin(c, QG_PHASE_REFIT, st);
    if (prc != QGBDT_OK) return prc;
    k_leaf_table<<<1, 256, 0, st>>>(c->d_leaves, c->d_recs, c->d_gs, c->d_leaf_table, c->d_leaf_table + 3 * (size_t)S, S, L,
                                    c->d_leaf_sums, c->d_m_num_leaves + tree_slot,
                                    c->d_m_leaf_count + (size_t)tree_slot * L, c->d_state);
    QG_LAUNCH_CHECK(c);
    if (c->leaf_values_quantized) {
        k_leaf_values_quantized<<<(L + 255) / 256, 256, 0, st>>>(
            c->d_leaves, c->d_recs, c->d_gs, c->d_state, qg_levels_g(c->prm.bits),
            qg_levels_h(c->prm.bits, c->prm.hess_levels_mode), c->const_hess ? 1 : 0, c->prm.lambda_l2,
            c->prm.learning_rate, c->d_leaf_w, c->d_m_leaf_value + (size_t)tree_slot * L);
        QG_LAUNCH_CHECK(c);
    } else {
        const unsigned blocks = (unsigned)((c->N + REFIT_BLOCK - 1) / REFIT_BLOCK);
        k_refit_sums<<<blocks, REFIT_THREADS, sizeof(uint32_t) * S, st>>>(nullptr, c->d_ent0, c->d_ent1, (uint32_t)c->N,
                                                                         c->d_leaf_table, S, c->d_gs, d_g, d_h,
                                                                         c->d_leaf_sums);
        QG_LAUNCH_CHECK(c);
        if ((prc = qg_allreduce(c, c->d_leaf_sums, 2 * (int64_t)L, QGBDT_REDUCE_SUM_I64, st)) != QGBDT_OK) return prc;
        k_leaf_values<<<(L + 255) / 256, 256, 0, st>>>(c->d_leaf_sums, L, c->d_gs, c->prm.lambda_l2, c->prm.learning_rate,
                                                       c->d_leaf_w, c->d_m_leaf_value + (size_t)tree_slot * L);
        QG_LAUNCH_CHECK(c);
    }
    if ((prc = qg_phase_end(c, st)) != QGBDT_OK) return prc;
    if ((prc = qg_phase_begin(c, QG_PHASE_SCORES, st)) != QGBDT_OK) return prc;
    unsigned ab = (unsigned)((c->N + REFIT_THREADS - 1) / REFIT_THREADS);
    if (ab > (unsigned)c->sm_count * 16) ab = (unsigned)c->sm_count * 16;
    k_apply_values<<<ab, REFIT_THREADS, sizeof(uint32_t) * 3 * S, st>>>(nullptr, c->d_ent0, c->d_ent1, (uint32_t)c->N,
                                                                   c->d_leaf_table, S, c->d_gs,
                                                                   c->d_m_leaf_value + (size_t)tree_slot * L, d_scores);
    QG_LAUNCH_CHECK(c);
    return qg_phase_end(c, st);
}

// Slots the leaf table of a grown tree may need: a leaf per slot, plus one per leaf split ahead.
int qg_leaf_table_slots(int L) { return L + GROW_SLACK + GROW_MAX_JOBS + 2; }
