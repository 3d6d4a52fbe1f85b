// Bin-matrix relayout into feature tiles, and the identity row list of the root leaf.
#include "qgbdt_internal.cuh"

// One thread per (row, word) of a tile: gathers four bin codes from the caller's matrix
// (row- or column-major), checks them against n_bins, and writes one packed word.
__global__ void k_relayout(const uint8_t *__restrict__ src, int layout, long long ld, long long n_rows,
                           int n_features, int n_bins, uint32_t *__restrict__ dst, int f0, int nf, int logW,
                           DevState *state) {
    const long long total = n_rows << logW;
    const int W = 1 << logW;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const long long row = t >> logW;
        const int a = (int)(t & (W - 1));
        uint32_t word = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int fl = 4 * a + k;
            if (fl < nf) {
                const int f = f0 + fl;
                const uint32_t code = layout == 0 ? src[row * ld + f] : src[(long long)f * ld + row];
                if (code >= (uint32_t)n_bins) {
                    state->bad_value = 1;
                } else {
                    word |= code << (8 * k);
                }
            }
        }
        dst[t] = word;
    }
}

__global__ void k_iota(uint32_t *idx, long long n) {
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < n;
         t += (long long)gridDim.x * blockDim.x)
        idx[t] = (uint32_t)t;
}

int qg_relayout(qgbdt_ctx *c, const uint8_t *d_bins, int layout, int64_t ld, cudaStream_t st) {
    for (const TileDesc &t : c->tiles) {
        const long long total = (long long)c->N << t.logW;
        const int threads = 256;
        long long blocks = (total + threads - 1) / threads;
        if (blocks > (long long)c->sm_count * 32) blocks = (long long)c->sm_count * 32;
        if (blocks < 1) blocks = 1;
        k_relayout<<<(unsigned)blocks, threads, 0, st>>>(d_bins, layout, ld, c->N, c->F, c->nb,
                                                         const_cast<uint32_t *>(t.data), t.f0, t.nf, t.logW,
                                                         c->d_state);
        QG_LAUNCH_CHECK(c);
    }
    return QGBDT_OK;
}

namespace {

// A block moves 256 rows of a tile at a time: coalesced words in (through shared memory, rows
// padded by one word against bank conflicts), 256 consecutive bytes of every column out.
__global__ void __launch_bounds__(256) k_to_columns(const uint32_t *__restrict__ tile, int logW, int nf, long long N,
                                                    uint8_t *__restrict__ cols, size_t stride) {
    extern __shared__ uint32_t sw[];   // [256][W + 1]
    const int W = 1 << logW;
    for (long long row0 = blockIdx.x * 256ll; row0 < N; row0 += (long long)gridDim.x * 256) {
        const int nrows = N - row0 < 256 ? (int)(N - row0) : 256;
        const uint32_t *src = tile + ((size_t)row0 << logW);
        for (int i = threadIdx.x; i < nrows * W; i += 256) sw[(i >> logW) * (W + 1) + (i & (W - 1))] = src[i];
        __syncthreads();
        if ((int)threadIdx.x < nrows) {
            for (int a = 0; 4 * a < nf; ++a) {
                const uint32_t w = sw[threadIdx.x * (W + 1) + a];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (4 * a + k < nf) cols[(size_t)(4 * a + k) * stride + row0 + threadIdx.x] = (uint8_t)(w >> (8 * k));
            }
        }
        __syncthreads();
    }
}

__global__ void k_set_columns(FeatRec *feat_rec, int F, uint8_t *cols, size_t stride) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f < F) feat_rec[f].col8 = cols + (size_t)f * stride;
}

}  // namespace

int qg_build_columns(qgbdt_ctx *c, cudaStream_t st) {
    if (c->d_colmajor) return QGBDT_OK;
    // switched off by the caller (qgbdt_set_option): training stays on the tiles alone, which saves
    // N x F bytes; the same path is taken when the allocation below fails
    if (!c->want_column_copy) return QGBDT_OK;
    const size_t stride = ((size_t)c->N + 127) / 128 * 128;
    void *p = nullptr;
    if (cudaMalloc(&p, stride * (size_t)c->F) != cudaSuccess) {
        cudaGetLastError();
        return QGBDT_OK;   // the feature records keep col8 == nullptr
    }
    c->d_colmajor = reinterpret_cast<uint8_t *>(p);
    c->col_stride = stride;
    for (const TileDesc &t : c->tiles) {
        long long bx = (c->N + 255) / 256;
        if (bx > (long long)c->sm_count * 32) bx = (long long)c->sm_count * 32;
        const size_t smem = (size_t)256 * ((1u << t.logW) + 1) * sizeof(uint32_t);
        k_to_columns<<<(unsigned)bx, 256, smem, st>>>(t.data, t.logW, t.nf, c->N, c->d_colmajor + (size_t)t.f0 * stride, stride);
        QG_LAUNCH_CHECK(c);
    }
    k_set_columns<<<(c->F + 255) / 256, 256, 0, st>>>(c->d_feat_rec, c->F, c->d_colmajor, stride);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

int qg_iota(qgbdt_ctx *c, cudaStream_t st) {
    long long blocks = (c->N + 255) / 256;
    if (blocks > (long long)c->sm_count * 16) blocks = (long long)c->sm_count * 16;
    if (blocks < 1) blocks = 1;
    k_iota<<<(unsigned)blocks, 256, 0, st>>>(c->d_idx, c->N);
    QG_LAUNCH_CHECK(c);
    c->idx_is_identity = true;
    return QGBDT_OK;
}
