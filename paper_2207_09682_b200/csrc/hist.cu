// Algorithm 1 with integer gradients: per-CTA shared-memory histograms with packed
// gradient+hessian bins (Sec. 6.1 hierarchical buffers, Sec. 6.2 packing), merged into the
// leaf's 32+32-bit histogram with 64-bit global atomics; and histogram subtraction.
//
// Shared-memory layout (the part that differs from the paper's V100 design): the local
// histogram is indexed [byte k of the word][bin][lane].  Lane l of a warp always adds into
// column l, i.e. bank l, so the 32 shared atomics of one warp instruction never collide,
// whatever the bin codes are (uniform or 90 % in one bin).  A lane owns word a = l % W of
// row slot b = l / W; column l of slab k therefore holds feature 4a+k of the tile, and the
// R = 32/W row slots are R private replicas that the flush adds up.
//
// Local bin width: B <= 4 uses one 32-bit word per bin, gradient sum in the high 16 bits
// (signed), hessian sum in the low 16 bits; the CTA flushes before any lane slot has added
// more rows than fit (flush_rows).  B >= 5 uses two 32-bit words per bin (32+32 local).
#include "qgbdt_internal.cuh"

namespace {

constexpr int HIST_THREADS = 1024;
constexpr int HIST_WARPS = HIST_THREADS / 32;
constexpr int ROW_BLOCK = 2048;  // rows per work unit
constexpr int UNROLL = 8;

struct HistArgs {
    const TileDesc *tiles;
    int n_tiles;
    const uint8_t *codes;
    const uint32_t *rows;  // row list, or nullptr: rows off .. off+n-1
    uint32_t off, n;
    int nb;
    unsigned long long *hist;  // [F][nb]
    uint32_t flush_rows;       // rows one lane slot may add between flushes (16+16 local only)
    int k0;                    // first byte of the word handled by this launch
};

template <int CODE_BYTES>
__device__ inline uint32_t load_code(const uint8_t *codes, uint32_t row) {
    if (CODE_BYTES == 1) return codes[row];
    return reinterpret_cast<const uint16_t *>(codes)[row];
}

// Adds the CTA's local histogram of the current tile into the leaf histogram and clears it.
template <bool WIDE, int KC>
__device__ inline void flush_local(int *sh, const TileDesc &td, int nb, int k0, unsigned long long *hist) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = 1 << td.logW;
    for (int r = warp; r < KC * nb; r += HIST_WARPS) {
        const int kk = r / nb, bin = r - kk * nb;
        int G;
        unsigned int H;
        if (!WIDE) {
            const int v = sh[r * 32 + lane];
            sh[r * 32 + lane] = 0;
            G = v >> 16;
            H = (unsigned int)(v & 0xFFFF);
        } else {
            G = sh[(2 * r) * 32 + lane];
            H = (unsigned int)sh[(2 * r + 1) * 32 + lane];
            sh[(2 * r) * 32 + lane] = 0;
            sh[(2 * r + 1) * 32 + lane] = 0;
        }
        for (int o = W; o < 32; o <<= 1) {
            G += __shfl_xor_sync(0xffffffffu, G, o);
            H += __shfl_xor_sync(0xffffffffu, H, o);
        }
        const int fl = 4 * lane + k0 + kk;
        if (lane < W && fl < td.nf && (G != 0 || H != 0u)) {
            const long long packed = (long long)G * 4294967296LL + (long long)H;
            atomicAdd(&hist[(size_t)(td.f0 + fl) * nb + bin], (unsigned long long)packed);
        }
    }
}

// Persistent CTAs over work units (tile, block of ROW_BLOCK rows), tile-major, split evenly
// and contiguously, so a CTA changes tile (and flushes for that) at most a few times.
template <int CODE_BYTES, bool WIDE, int KC>
__global__ void __launch_bounds__(HIST_THREADS, 1) k_hist(HistArgs a) {
    extern __shared__ int sh[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_words = KC * a.nb * 32 * (WIDE ? 2 : 1);
    for (int i = threadIdx.x; i < n_words; i += HIST_THREADS) sh[i] = 0;
    __syncthreads();

    const uint32_t n = a.n;
    const uint32_t nblk = (n + ROW_BLOCK - 1) / ROW_BLOCK;
    const unsigned long long units = (unsigned long long)nblk * a.n_tiles;
    const uint32_t u0 = (uint32_t)(units * blockIdx.x / gridDim.x);
    const uint32_t u1 = (uint32_t)(units * (blockIdx.x + 1) / gridDim.x);

    int cur_tile = -1;
    TileDesc td = {};
    uint32_t slot_rows = 0;
    bool dirty = false;
    int *const my_col = sh + lane;

    for (uint32_t u = u0; u < u1; ++u) {
        const int t = (int)(u / nblk);
        const uint32_t blk = u - (uint32_t)t * nblk;
        if (t != cur_tile) {
            if (dirty) {
                __syncthreads();
                flush_local<WIDE, KC>(sh, td, a.nb, a.k0, a.hist);
                __syncthreads();
                dirty = false;
            }
            td = a.tiles[t];
            cur_tile = t;
            slot_rows = 0;
        }
        const int logW = td.logW;
        const int logR = 5 - logW;
        const uint32_t row0 = blk * ROW_BLOCK;
        const uint32_t rows_here = min((uint32_t)ROW_BLOCK, n - row0);
        const uint32_t groups = (rows_here + (1u << logR) - 1) >> logR;
        if (!WIDE) {
            if (slot_rows + groups > a.flush_rows) {
                __syncthreads();
                flush_local<WIDE, KC>(sh, td, a.nb, a.k0, a.hist);
                __syncthreads();
                slot_rows = 0;
            }
            slot_rows += groups;
        }
        dirty = true;
        const uint32_t wa = lane & ((1u << logW) - 1);  // word of the row held by this lane
        const uint32_t slot = lane >> logW;             // row slot of this lane
        const bool lane_used = wa < (uint32_t)td.words_used;
        const uint32_t *tile = td.data;

        for (uint32_t g0 = warp; g0 < groups; g0 += HIST_WARPS * UNROLL) {
            uint32_t row[UNROLL];
            bool ok[UNROLL];
#pragma unroll
            for (int j = 0; j < UNROLL; ++j) {
                const uint32_t gi = g0 + j * HIST_WARPS;
                const uint32_t p = row0 + (gi << logR) + slot;
                ok[j] = lane_used && gi < groups && p < n;
                row[j] = 0;
                if (ok[j]) row[j] = a.rows ? a.rows[a.off + p] : a.off + p;
            }
            uint32_t word[UNROLL], code[UNROLL];
#pragma unroll
            for (int j = 0; j < UNROLL; ++j) {
                word[j] = 0;
                code[j] = 0;
                if (ok[j]) {
                    word[j] = tile[((size_t)row[j] << logW) + wa];
                    code[j] = load_code<CODE_BYTES>(a.codes, row[j]);
                }
            }
#pragma unroll
            for (int j = 0; j < UNROLL; ++j) {
                if (!ok[j]) continue;
                const uint32_t w = word[j] >> (8 * a.k0);
                if (!WIDE) {
                    // 4-bit codes: gradient in the high nibble (signed), hessian in the low nibble
                    int gq, hq;
                    if (CODE_BYTES == 1) {
                        gq = ((int)(int8_t)code[j]) >> 4;
                        hq = (int)(code[j] & 0xF);
                    } else {
                        gq = (int)(int8_t)(code[j] >> 8);
                        hq = (int)(code[j] & 0xFF);
                    }
                    const int inc = gq * 65536 + hq;
#pragma unroll
                    for (int k = 0; k < KC; ++k) {
                        const uint32_t bin = (w >> (8 * k)) & 0xFF;
                        atomicAdd(my_col + (k * a.nb + bin) * 32, inc);
                    }
                } else {
                    int gq, hq;
                    if (CODE_BYTES == 1) {
                        gq = ((int)(int8_t)code[j]) >> 4;
                        hq = (int)(code[j] & 0xF);
                    } else {
                        gq = (int)(int8_t)(code[j] >> 8);
                        hq = (int)(code[j] & 0xFF);
                    }
#pragma unroll
                    for (int k = 0; k < KC; ++k) {
                        const uint32_t bin = (w >> (8 * k)) & 0xFF;
                        atomicAdd(my_col + (2 * (k * a.nb + bin)) * 32, gq);
                        atomicAdd(my_col + (2 * (k * a.nb + bin) + 1) * 32, hq);
                    }
                }
            }
        }
    }
    if (dirty) {
        __syncthreads();
        flush_local<WIDE, KC>(sh, td, a.nb, a.k0, a.hist);
    }
}

__global__ void k_subtract(const unsigned long long *__restrict__ parent, const unsigned long long *__restrict__ small,
                           unsigned long long *__restrict__ large, long long n) {
    // hessian fields never borrow (child <= parent in every bin), so one 64-bit subtract is exact
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        large[i] = parent[i] - small[i];
}

template <int CODE_BYTES, bool WIDE, int KC>
int launch_hist(qgbdt_ctx *c, const HistArgs &args, unsigned grid, cudaStream_t st) {
    const size_t smem = (size_t)KC * c->nb * 32 * 4 * (WIDE ? 2 : 1);
    auto kern = k_hist<CODE_BYTES, WIDE, KC>;
    static size_t configured = 48 * 1024;  // per instantiation: largest opt-in size set so far
    if (smem > configured) {
        QG_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured = smem;
    }
    kern<<<grid, HIST_THREADS, smem, st>>>(args);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

}  // namespace

int qg_hist(qgbdt_ctx *c, const uint32_t *d_rows, int64_t off, int64_t n, unsigned long long *d_hist,
            cudaStream_t st) {
    const size_t hist_bytes = (size_t)c->F * c->nb * sizeof(unsigned long long);
    QG_CUDA(c, cudaMemsetAsync(d_hist, 0, hist_bytes, st));
    c->n_hist_builds++;
    c->n_hist_row_features += n * c->F;
    if (n <= 0) return QGBDT_OK;

    const int bits = c->prm.bits;
    const int kg = qg_levels_g(bits);
    const int kh = c->const_hess ? 1 : qg_levels_h(bits, c->prm.hess_levels_mode);
    const bool wide = c->code_bytes == 2;

    HistArgs a;
    a.tiles = c->d_tiles;
    a.n_tiles = (int)c->tiles.size();
    a.codes = c->d_codes;
    a.rows = d_rows;
    a.off = (uint32_t)off;
    a.n = (uint32_t)n;
    a.nb = c->nb;
    a.hist = d_hist;
    a.k0 = 0;
    const uint32_t by_h = 65535u / (uint32_t)kh, by_g = 32767u / (uint32_t)kg;
    a.flush_rows = by_h < by_g ? by_h : by_g;

    const unsigned long long units = (unsigned long long)((n + ROW_BLOCK - 1) / ROW_BLOCK) * a.n_tiles;
    unsigned grid = (unsigned)(units < (unsigned long long)c->sm_count ? units : (unsigned long long)c->sm_count);

    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if (c->profile_hist) {
        if (c->hist_events_used + 2 > c->hist_events.size()) {
            for (int i = 0; i < 2; ++i) {
                cudaEvent_t e;
                QG_CUDA(c, cudaEventCreate(&e));
                c->hist_events.push_back(e);
            }
        }
        ev0 = c->hist_events[c->hist_events_used++];
        ev1 = c->hist_events[c->hist_events_used++];
        // algorithmic bytes of this build: bin codes + packed gradient code (+ row index) per row, histogram out
        c->hist_prof_bytes += n * (c->F + c->code_bytes + (d_rows ? 4 : 0)) + (int64_t)hist_bytes;
        c->hist_prof_launches++;
        QG_CUDA(c, cudaEventRecord(ev0, st));
    }
    int rc;
    if (!wide) {
        rc = launch_hist<1, false, 4>(c, a, grid, st);
    } else {
        // 32+32 local bins: two words per bin; all four bytes fit only for small bin counts
        const size_t full = (size_t)4 * c->nb * 32 * 4 * 2;
        if (full <= (size_t)c->max_smem_optin) {
            rc = launch_hist<2, true, 4>(c, a, grid, st);
        } else {
            rc = launch_hist<2, true, 2>(c, a, grid, st);
            if (rc == QGBDT_OK) {
                a.k0 = 2;
                rc = launch_hist<2, true, 2>(c, a, grid, st);
            }
        }
    }
    if (rc == QGBDT_OK && ev1) QG_CUDA(c, cudaEventRecord(ev1, st));
    return rc;
}

int qg_subtract(qgbdt_ctx *c, const unsigned long long *d_parent, const unsigned long long *d_small,
                unsigned long long *d_large, cudaStream_t st) {
    const long long n = (long long)c->F * c->nb;
    long long blocks = (n + 255) / 256;
    if (blocks > (long long)c->sm_count * 8) blocks = (long long)c->sm_count * 8;
    k_subtract<<<(unsigned)blocks, 256, 0, st>>>(d_parent, d_small, d_large, n);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}
