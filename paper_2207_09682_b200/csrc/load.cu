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

int qg_iota(qgbdt_ctx *c, cudaStream_t st) {
    long long blocks = (c->N + 255) / 256;
    if (blocks > (long long)c->sm_count * 16) blocks = (long long)c->sm_count * 16;
    if (blocks < 1) blocks = 1;
    k_iota<<<(unsigned)blocks, 256, 0, st>>>(c->d_idx, c->N);
    QG_LAUNCH_CHECK(c);
    c->idx_is_identity = true;
    return QGBDT_OK;
}
