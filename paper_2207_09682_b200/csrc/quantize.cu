// Eq. 1 (gradients), Eq. 5 (scales), Eq. 6 + Eq. 8 (quantization with stochastic rounding).
#include "qgbdt_internal.cuh"

namespace {

__host__ __device__ inline uint32_t mix32(uint32_t x) {
    x ^= x >> 16;
    x *= 0x9E3779B9u;
    x ^= x >> 15;
    x *= 0xBB67AE85u;
    x ^= x >> 16;
    return x;
}

// Sigmoid from exactly rounded operations only, so that the bits do not depend on the
// machine: e = exp(-|s|) by range reduction and a degree-6 polynomial, then one divide.
__device__ inline float sigmoid_det(float s) {
    float a = fabsf(s);
    a = (a > 40.0f) ? 40.0f : a;
    const float x = -a;
    const float n = rintf(__fmul_rn(x, 0x1.715476p+0f));
    float r = __fmaf_rn(n, -0x1.62e400p-1f, x);
    r = __fmaf_rn(n, -0x1.7f7d1cp-20f, r);
    float p = 0x1.6c16c2p-10f;
    p = __fmaf_rn(p, r, 0x1.111112p-7f);
    p = __fmaf_rn(p, r, 0x1.555556p-5f);
    p = __fmaf_rn(p, r, 0x1.555556p-3f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    const float e = __int_as_float(__float_as_int(p) + (((int)n) << 23));
    const float d = __fadd_rn(1.0f, e);
    return s >= 0.0f ? __fdiv_rn(1.0f, d) : __fdiv_rn(e, d);
}

__device__ inline bool bad_g(float g) { return !isfinite(g) || fabsf(g) >= 256.0f; }
__device__ inline bool bad_h(float h) { return !isfinite(h) || h < 0.0f || h >= 256.0f; }

// Block-wide max of two non-negative floats (as bit patterns) and an OR of a flag, pushed to
// the device state with one atomic per block.
__device__ inline void block_max_to_state(float gabs, float hval, bool bad, DevState *state) {
    unsigned int gb = __float_as_uint(gabs), hb = __float_as_uint(hval);
    int bd = bad ? 1 : 0;
    for (int o = 16; o > 0; o >>= 1) {
        gb = max(gb, __shfl_xor_sync(0xffffffffu, gb, o));
        hb = max(hb, __shfl_xor_sync(0xffffffffu, hb, o));
        bd |= __shfl_xor_sync(0xffffffffu, bd, o);
    }
    __shared__ unsigned int sg[32], shh[32];
    __shared__ int sb[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sg[warp] = gb; shh[warp] = hb; sb[warp] = bd; }
    __syncthreads();
    if (warp == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        gb = lane < nw ? sg[lane] : 0u;
        hb = lane < nw ? shh[lane] : 0u;
        bd = lane < nw ? sb[lane] : 0;
        for (int o = 16; o > 0; o >>= 1) {
            gb = max(gb, __shfl_xor_sync(0xffffffffu, gb, o));
            hb = max(hb, __shfl_xor_sync(0xffffffffu, hb, o));
            bd |= __shfl_xor_sync(0xffffffffu, bd, o);
        }
        if (lane == 0) {
            if (gb) atomicMax(&state->gmax_bits, gb);
            if (hb) atomicMax(&state->hmax_bits, hb);
            if (bd) atomicOr(&state->bad_value, 1);
        }
    }
}

// Eq. 1.  objective 0: p = sigmoid(s), g = p - y, h = p (1 - p); objective 1: g = s - y.
// Also reduces max |g| and max h (Eq. 5) when `state` is given.
__global__ void k_gradients(int objective, const float *__restrict__ scores, const float *__restrict__ labels,
                            long long n, float *__restrict__ g, float *__restrict__ h, DevState *state) {
    float gm = 0.f, hm = 0.f;
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x) {
        const float s = scores[i], y = labels[i];
        float gi, hi = 0.f;
        if (objective == 0) {
            const float p = sigmoid_det(s);
            gi = __fsub_rn(p, y);
            hi = __fmul_rn(p, __fsub_rn(1.0f, p));
            h[i] = hi;
            bad |= bad_h(hi);
        } else {
            gi = __fsub_rn(s, y);
        }
        g[i] = gi;
        bad |= bad_g(gi);
        gm = fmaxf(gm, fabsf(gi));
        hm = fmaxf(hm, hi);
    }
    if (state) block_max_to_state(gm, hm, bad, state);
}

// Eq. 5: max |g| and max h of caller-provided gradients, with the domain checks.
__global__ void k_absmax(const float *__restrict__ g, const float *__restrict__ h, long long n, DevState *state) {
    float gm = 0.f, hm = 0.f;
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x) {
        const float gi = g[i];
        bad |= bad_g(gi);
        gm = fmaxf(gm, fabsf(gi));
        if (h) {
            const float hi = h[i];
            bad |= bad_h(hi);
            hm = fmaxf(hm, hi);
        }
    }
    block_max_to_state(gm, hm, bad, state);
}

// Eq. 8 on a value already scaled and clamped: floor(x) + [u < floor(frac * 2^24)] (SR),
// or floor(x) + [frac >= 1/2] (RN).
__device__ inline int round_level(float x, int rounding, uint32_t u) {
    const float f = floorf(x);
    const float frac = __fsub_rn(x, f);
    if (rounding == 1) return (int)f + (frac >= 0.5f ? 1 : 0);
    const uint32_t t = __float2uint_rz(__fmul_rn(frac, 16777216.0f));
    return (int)f + (u < t ? 1 : 0);
}

// Eq. 6 + Eq. 8 for every row; writes the packed 16-bit per-row code, optional unpacked copies,
// and adds the integer totals (one atomic pair per block).
__global__ void k_quantize(const float *__restrict__ g, const float *__restrict__ h, long long n, int kg, int kh,
                           int rounding, uint32_t key, uint32_t row_offset, DevState *state, uint8_t *__restrict__ codes,
                           uint16_t *__restrict__ codes_nat, int8_t *__restrict__ gq_out, uint8_t *__restrict__ hq_out) {
    const float gmax = __uint_as_float(state->gmax_bits);
    const float hmax = h ? __uint_as_float(state->hmax_bits) : 1.0f;
    const float inv_g = gmax > 0.f ? __fdiv_rn((float)kg, gmax) : 0.f;
    const float inv_h = hmax > 0.f ? __fdiv_rn((float)kh, hmax) : 0.f;
    long long sg = 0, sh = 0;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x) {
        const uint32_t r = mix32(key ^ ((uint32_t)i + row_offset));   // the row's number in the whole training set
        float x = __fmul_rn(g[i], inv_g);
        x = x > (float)kg ? (float)kg : x;
        x = x < -(float)kg ? -(float)kg : x;
        const int gq = round_level(x, rounding, mix32(r) >> 8);
        int hq = 1;
        if (h) {
            float y = __fmul_rn(h[i], inv_h);
            y = y > (float)kh ? (float)kh : y;
            y = y < 0.f ? 0.f : y;
            hq = round_level(y, rounding, mix32(r + 0x6A09E667u) >> 8);
        }
        // 4 x 4 transposed inside blocks of 16 rows (see the layout notes of the internal header)
        const long long pos = (i & ~15LL) | ((i & 3) << 2) | ((i >> 2) & 3);
        const uint16_t code = (uint16_t)(((gq & 0xFF) << 8) | hq);
        reinterpret_cast<uint16_t *>(codes)[pos] = code;
        codes_nat[i] = code;
        if (gq_out) gq_out[i] = (int8_t)gq;
        if (hq_out) hq_out[i] = (uint8_t)hq;
        sg += gq;
        sh += hq;
    }
    for (int o = 16; o > 0; o >>= 1) {
        sg += __shfl_xor_sync(0xffffffffu, sg, o);
        sh += __shfl_xor_sync(0xffffffffu, sh, o);
    }
    __shared__ long long wg[32], wh[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { wg[warp] = sg; wh[warp] = sh; }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        long long a = 0, b = 0;
        for (int w = 0; w < nw; ++w) { a += wg[w]; b += wh[w]; }
        atomicAdd(reinterpret_cast<unsigned long long *>(&state->tot_g), (unsigned long long)a);
        atomicAdd(reinterpret_cast<unsigned long long *>(&state->tot_h), (unsigned long long)b);
    }
}

// The out-of-domain flag is sticky over the trees of one train call: only the caller-facing
// quantize call and the start of a train call clear it.
__global__ void k_reset_state(DevState *state, int clear_bad) {
    state->gmax_bits = 0;
    state->hmax_bits = 0;
    if (clear_bad) state->bad_value = 0;
    state->tot_g = 0;
    state->tot_h = 0;
}

inline unsigned grid_for(const qgbdt_ctx *c, long long n, int threads, int per_sm) {
    long long blocks = (n + threads - 1) / threads;
    const long long cap = (long long)c->sm_count * per_sm;
    if (blocks > cap) blocks = cap;
    return (unsigned)(blocks < 1 ? 1 : blocks);
}

}  // namespace

int qg_gradients(qgbdt_ctx *c, const float *d_scores, const float *d_labels, float *d_g, float *d_h,
                 bool reduce_max, bool clear_bad, cudaStream_t st) {
    if (reduce_max) {
        k_reset_state<<<1, 1, 0, st>>>(c->d_state, clear_bad ? 1 : 0);
        QG_LAUNCH_CHECK(c);
    }
    k_gradients<<<grid_for(c, c->N, 256, 8), 256, 0, st>>>(c->prm.objective, d_scores, d_labels, c->N, d_g, d_h,
                                                            reduce_max ? c->d_state : nullptr);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

int qg_absmax(qgbdt_ctx *c, const float *d_g, const float *d_h, cudaStream_t st) {
    k_reset_state<<<1, 1, 0, st>>>(c->d_state, 1);
    QG_LAUNCH_CHECK(c);
    k_absmax<<<grid_for(c, c->N, 256, 8), 256, 0, st>>>(d_g, d_h, c->N, c->d_state);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

int qg_quantize(qgbdt_ctx *c, const float *d_g, const float *d_h, uint32_t tree, int8_t *d_gq, uint8_t *d_hq,
                cudaStream_t st) {
    const uint32_t seed_lo = (uint32_t)(c->prm.seed & 0xFFFFFFFFu), seed_hi = (uint32_t)(c->prm.seed >> 32);
    const uint32_t key = mix32(mix32(mix32(seed_lo ^ 0x6A09E667u) + seed_hi) ^ tree);
    const int kg = qg_levels_g(c->prm.bits), kh = qg_levels_h(c->prm.bits, c->prm.hess_levels_mode);
    const unsigned grid = grid_for(c, c->N, 256, 8);
    k_quantize<<<grid, 256, 0, st>>>(d_g, d_h, c->N, kg, kh, c->prm.rounding, key,
                                     qg_sharded(c) ? (uint32_t)c->row_offset : 0u, c->d_state, c->d_codes,
                                     reinterpret_cast<uint16_t *>(c->d_codes_nat), d_gq, d_hq);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}
