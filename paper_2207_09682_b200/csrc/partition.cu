// Stable partition of a leaf's row list by (feature, threshold bin): rows with code <= bin
// first, the rest after, relative order kept (the index sets I_s of Sec. 3).
//
// Three passes: (1) one predicate bit per row by warp ballot and the number of left rows per
// block of 2048; (2) an exclusive scan of the block counts by one CTA; (3) a scatter into a
// second buffer at the stable destinations, copied back over the leaf's range.
#include "qgbdt_internal.cuh"

namespace {

constexpr int PART_THREADS = 256;
constexpr int PART_ITEMS = 8;
constexpr int PART_BLOCK = PART_THREADS * PART_ITEMS;  // 2048 rows
constexpr int PART_WORDS = PART_BLOCK / 32;            // 64 ballot words

__global__ void __launch_bounds__(PART_THREADS) k_part_flags(const uint32_t *__restrict__ idx, uint32_t off,
                                                             uint32_t n, const uint32_t *__restrict__ tile, int logW,
                                                             int wa, int byte, uint32_t thr,
                                                             uint32_t *__restrict__ bits,
                                                             uint32_t *__restrict__ counts) {
    const int lane = threadIdx.x & 31;
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < PART_ITEMS; ++j) {
        const uint32_t p = blockIdx.x * PART_BLOCK + j * PART_THREADS + threadIdx.x;
        bool left = false;
        if (p < n) {
            const uint32_t row = idx[off + p];
            const uint32_t w = tile[((size_t)row << logW) + wa];
            left = ((w >> (8 * byte)) & 0xFF) <= thr;
        }
        const uint32_t b = __ballot_sync(0xffffffffu, left);
        if (lane == 0) {
            bits[p >> 5] = b;
            mine += __popc(b);
        }
    }
    __shared__ uint32_t sm[PART_THREADS / 32];
    if (lane == 0) sm[threadIdx.x >> 5] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t s = 0;
        for (int w = 0; w < PART_THREADS / 32; ++w) s += sm[w];
        counts[blockIdx.x] = s;
    }
}

// In-place exclusive scan of the block counts; the total goes to state->part_nl.
__global__ void __launch_bounds__(1024) k_part_scan(uint32_t *counts, uint32_t nblocks, DevState *state) {
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t carry_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (uint32_t base = 0; base < nblocks; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t v = i < nblocks ? counts[i] : 0;
        uint32_t x = v;
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            uint32_t s = warp_sums[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += y;
            }
            warp_sums[lane] = s;  // inclusive over warps
        }
        __syncthreads();
        const uint32_t carry = carry_s;
        const uint32_t before = carry + (warp > 0 ? warp_sums[warp - 1] : 0) + (x - v);
        if (i < nblocks) counts[i] = before;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = carry + warp_sums[31];
        __syncthreads();
    }
    if (threadIdx.x == 0) state->part_nl = carry_s;
}

__global__ void __launch_bounds__(PART_THREADS) k_part_scatter(const uint32_t *__restrict__ idx, uint32_t off,
                                                               uint32_t n, const uint32_t *__restrict__ bits,
                                                               const uint32_t *__restrict__ counts,
                                                               const DevState *state, uint32_t *__restrict__ out) {
    __shared__ uint32_t words[PART_WORDS];
    __shared__ uint32_t prefix[PART_WORDS];
    const uint32_t blk0 = blockIdx.x * PART_BLOCK;
    if (threadIdx.x < PART_WORDS) {
        const uint32_t p = blk0 + threadIdx.x * 32;
        words[threadIdx.x] = p < n ? bits[p >> 5] : 0u;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t s = 0;
        for (int w = 0; w < PART_WORDS; ++w) { prefix[w] = s; s += __popc(words[w]); }
    }
    __syncthreads();
    const uint32_t nl_total = state->part_nl;
    const uint32_t left_before = counts[blockIdx.x];  // lefts in earlier blocks
    const uint32_t right_before = blk0 - left_before;
#pragma unroll
    for (int j = 0; j < PART_ITEMS; ++j) {
        const uint32_t local = j * PART_THREADS + threadIdx.x;
        const uint32_t p = blk0 + local;
        if (p >= n) continue;
        const uint32_t w = words[local >> 5];
        const uint32_t lane_bit = local & 31;
        const uint32_t lefts = prefix[local >> 5] + __popc(w & ((1u << lane_bit) - 1u));
        const bool left = (w >> lane_bit) & 1u;
        const uint32_t dest = left ? left_before + lefts : nl_total + right_before + (local - lefts);
        out[off + dest] = idx[off + p];
    }
}

__global__ void k_copy_u32(const uint32_t *__restrict__ src, uint32_t *__restrict__ dst, uint32_t n) {
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = src[i];
}

}  // namespace

int qg_partition(qgbdt_ctx *c, int64_t off, int64_t n, int feature, int bin, cudaStream_t st) {
    int ti = -1;
    for (size_t i = 0; i < c->tiles.size(); ++i)
        if (feature >= c->tiles[i].f0 && feature < c->tiles[i].f0 + c->tiles[i].nf) ti = (int)i;
    if (ti < 0) return qg_fail(c, QGBDT_ERR_ARG, "feature %d out of range", feature);
    const TileDesc &t = c->tiles[ti];
    const int fl = feature - t.f0;
    const unsigned nblocks = (unsigned)((n + PART_BLOCK - 1) / PART_BLOCK);
    k_part_flags<<<nblocks, PART_THREADS, 0, st>>>(c->d_idx, (uint32_t)off, (uint32_t)n, t.data, t.logW, fl / 4, fl % 4,
                                                   (uint32_t)bin, c->d_part_bits, c->d_part_counts);
    QG_LAUNCH_CHECK(c);
    k_part_scan<<<1, 1024, 0, st>>>(c->d_part_counts, nblocks, c->d_state);
    QG_LAUNCH_CHECK(c);
    k_part_scatter<<<nblocks, PART_THREADS, 0, st>>>(c->d_idx, (uint32_t)off, (uint32_t)n, c->d_part_bits,
                                                     c->d_part_counts, c->d_state, c->d_idx_tmp);
    QG_LAUNCH_CHECK(c);
    unsigned cb = (unsigned)((n + 1023) / 1024);
    if (cb > (unsigned)c->sm_count * 8) cb = (unsigned)c->sm_count * 8;
    k_copy_u32<<<cb, 256, 0, st>>>(c->d_idx_tmp + off, c->d_idx + off, (uint32_t)n);
    QG_LAUNCH_CHECK(c);
    c->idx_is_identity = false;
    return QGBDT_OK;
}
