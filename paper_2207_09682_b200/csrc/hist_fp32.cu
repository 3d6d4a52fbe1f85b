// Floating-point histogram: Algorithm 1 as the paper prints it, with the original gradients
// g_i, h_i in single precision -- the unquantized baseline that Sec. 7.2 compares the integer
// histograms with.  It follows the integer kernel's design as far as floats allow: feature tiles,
// bank-private columns in shared memory (lane l of a warp only ever adds into column l), shared
// atomics (red.shared.add.f32), one local histogram per CTA.  A bin needs two 32-bit words (the
// gradient sum and the hessian sum), twice what a packed integer bin needs, so a CTA holds two of
// the four byte positions of a word and the rows are read twice, as with 32+32-bit integer bins;
// a row brings 8 bytes of gradients instead of a 2-byte code.  The CTAs add their local sums to
// the output with global atomics.  Float sums depend on the order of the additions: results agree
// with a double-precision sum to rounding error, not bit for bit.
#include "qgbdt_internal.cuh"

namespace {

constexpr int FP_THREADS = 1024;
constexpr int FP_WARPS = FP_THREADS / 32;
constexpr int FP_SMEM = 128 * 1024;   // [bin][2 byte positions][2 planes][32 lanes] floats

__device__ __forceinline__ void red_f32(float *p, float v) {
    asm volatile("red.shared.add.f32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "f"(v) : "memory");
}

// Grid (part, tile, pass).  rows == nullptr: rows 0 .. n-1.
__global__ void __launch_bounds__(FP_THREADS, 1) k_hist_fp32(const TileDesc *__restrict__ tiles, const float *__restrict__ g,
                                                             const float *__restrict__ h, const uint32_t *__restrict__ rows,
                                                             uint32_t n, int nb, float *__restrict__ hist) {
    extern __shared__ __align__(16) float lh[];
    const TileDesc td = tiles[blockIdx.y];
    const int pass = blockIdx.z;
    const uint32_t P = gridDim.x, part = blockIdx.x;
    for (int i = threadIdx.x; i < nb * 128; i += FP_THREADS) lh[i] = 0.f;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int logW = td.logW, logR = 5 - logW;
    const uint32_t R = 1u << logR, wa = (uint32_t)lane >> logR, slot = lane & (R - 1);
    const uint32_t e0 = (uint32_t)((unsigned long long)n * part / P), e1 = (uint32_t)((unsigned long long)n * (part + 1) / P);
    const uint32_t *tile = td.data + wa;
    float *col = lh + lane;
    const int sh0 = 16 * pass, sh1 = sh0 + 8;
    constexpr int U = 4;   // rows in flight per lane
    for (uint32_t i0 = e0 + warp * R + slot; i0 < e1; i0 += U * FP_WARPS * R) {
        uint32_t w[U];
        float gv[U], hv[U];
        bool on[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = i0 + u * FP_WARPS * R;
            on[u] = i < e1;
            if (on[u]) {
                const uint32_t row = rows ? rows[i] : i;
                w[u] = tile[(size_t)row << logW];
                gv[u] = g[row];
                hv[u] = h ? h[row] : 1.0f;
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (on[u]) {
                const uint32_t b0 = (w[u] >> sh0) & 0xFFu, b1 = (w[u] >> sh1) & 0xFFu;
                red_f32(col + b0 * 128, gv[u]);
                red_f32(col + b0 * 128 + 32, hv[u]);
                red_f32(col + b1 * 128 + 64, gv[u]);
                red_f32(col + b1 * 128 + 96, hv[u]);
            }
        }
    }
    __syncthreads();
    // the R replicas of a column are adjacent lanes; every (bin, byte position, word) goes to the output
    const int W = 1 << logW;
    for (int e = threadIdx.x; e < nb * 2 * W; e += FP_THREADS) {
        const int a = e & (W - 1), kk = (e >> logW) & 1, bin = e >> (logW + 1);
        const int fl = 4 * a + 2 * pass + kk;
        if (fl >= td.nf) continue;
        const float *p = lh + bin * 128 + kk * 64 + a * R;
        float sg = 0.f, shh = 0.f;
        for (uint32_t r = 0; r < R; ++r) {
            sg += p[r];
            shh += p[32 + r];
        }
        float *q = hist + ((size_t)(td.f0 + fl) * nb + bin) * 2;
        atomicAdd(q, sg);
        atomicAdd(q + 1, shh);
    }
}

}  // namespace

int qg_hist_fp32(qgbdt_ctx *c, const float *d_g, const float *d_h, const uint32_t *d_rows, int64_t n, float *d_hist,
                 cudaStream_t st) {
    QG_CUDA(c, cudaMemsetAsync(d_hist, 0, sizeof(float) * 2 * (size_t)c->F * c->nb, st));
    if (n <= 0) return QGBDT_OK;
    static bool configured[64] = {};
    if (c->device < 0 || c->device >= 64 || !configured[c->device]) {
        QG_CUDA(c, cudaFuncSetAttribute(k_hist_fp32, cudaFuncAttributeMaxDynamicSharedMemorySize, FP_SMEM));
        if (c->device >= 0 && c->device < 64) configured[c->device] = true;
    }
    const int T = (int)c->tiles.size();
    int parts = c->sm_count / (2 * T);          // (part, tile, pass): about one CTA per SM
    const int64_t want = (n + 2047) / 2048;
    if (parts > want) parts = (int)want;
    if (parts < 1) parts = 1;
    k_hist_fp32<<<dim3((unsigned)parts, (unsigned)T, 2), FP_THREADS, FP_SMEM, st>>>(c->d_tiles, d_g, d_h, d_rows, (uint32_t)n,
                                                                                     c->nb, d_hist);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}
