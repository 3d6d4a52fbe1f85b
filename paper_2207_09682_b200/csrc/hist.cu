// Algorithm 1 with integer gradients: per-CTA shared-memory histograms with packed
// gradient+hessian bins (Sec. 6.1 hierarchical buffers, Sec. 6.2 packing), merged into the
// leaf's 32+32-bit histogram in two stages; and histogram subtraction.
//
// What differs from the paper's V100 design (one 16+16 local histogram per CUDA block, merged
// with atomics):
//
//  * Bank-private columns.  The local histogram is indexed [bin][byte k of the word][lane].
//    Lane l of a warp always adds into column l, i.e. shared-memory bank l, so the 32 atomics
//    of one warp instruction never collide, whatever the bin codes are (uniform, or 90 % in
//    one bin).  A lane owns word a = l / R of row slot l % R; the R = 32/W row slots are R
//    private replicas in adjacent words that the flush adds up.  Measured: one conflict-free warp atomic per
//    clock per SM.
//  * One-instruction addressing.  The local histogram starts on a 64 KB boundary of the shared
//    window and a bin is 256 bytes apart from the next, so the address of (bin, lane) is the
//    lane's base address with its second byte replaced by the bin code: a single byte permute
//    of the loaded word yields the atomic's address, and the per-row increment (gradient << 16
//    + hessian) is one more permute of the row's 16-bit code.
//  * Rolling prefetch.  Every lane keeps U units of four rows in flight in registers and
//    refills a slot as soon as it has been consumed.
//  * Two-stage merge.  A CTA stores its partial histogram with plain coalesced stores; after a
//    grid-wide barrier the CTAs of a tile share the sums of its entries (cooperative launch), or a
//    small kernel does, or the kernel that finishes a split during tree growth.  (64-bit global
//    atomics from 148 CTAs on the same 7 k bins cost about as much as half of the whole build.)
//
// Local bin width: B <= 5 uses one 32-bit word per bin, gradient sum in the high bits (signed),
// hessian sum in the low bits (16+16; 18+14 with a constant hessian, which only counts rows).
// Before any column can have added more rows than fit, a CTA of a narrow tile flushes its local
// histogram; a CTA of a wide tile moves only the words that are about to overflow.  B >= 6 uses
// two 32-bit words per bin (32+32, a hessian plane and a gradient plane) and two passes over the
// rows, each pass taking two of the four bytes of a word; in a stand-alone build the two passes
// run side by side in pairs of CTAs that read the same rows at the same time.
#include <cooperative_groups.h>

#include <mutex>

#include "hist_cta.cuh"

namespace {

// Guards the per-instantiation "attribute set on this device" flags below: they are shared by all
// contexts of the process, and two contexts may be driven from two host threads.
std::mutex g_configure_mutex;

// Row shares of a tile when its CTAs work in pairs (one pass of the 32+32 mode each).
__device__ __host__ inline uint32_t paired_parts(uint32_t P) { return P > 1 ? P >> 1 : 1; }

// Stand-alone build: the grid is (part, tile - tile0).
template <int LOGW_T, int MODE, int LIST>
__global__ void __launch_bounds__(HIST_THREADS, 1) k_hist(HistArgs a) {
    extern __shared__ __align__(1024) int sh[];
    const TileDesc td = a.tiles[a.tile0 + blockIdx.y];
    const uint32_t P = effective_parts((uint32_t)td.parts, a.n);
    if (MODE == 1 && a.pass < 0) {
        // 32+32 local bins, both passes side by side: CTAs 2i and 2i + 1 take the same rows, one
        // pass each, at the same time, so that the second reader of a row finds it in L2
        const uint32_t P2 = paired_parts(P);
        if ((blockIdx.x >> 1) >= P2) return;
        a.pass = (int)(blockIdx.x & 1u);
        hist_cta<HIST_THREADS, LOGW_T, MODE, LIST>(a, td, blockIdx.x >> 1, P2, sh);
        return;
    }
    if (blockIdx.x >= P) return;
    hist_cta<HIST_THREADS, LOGW_T, MODE, LIST>(a, td, blockIdx.x, P, sh);
}

// Stand-alone build with the merge inside the kernel: a cooperative launch (every CTA resident),
// a grid-wide barrier after the partial histograms, then the P CTAs of a tile share the sums of
// its entries.  Saves the merge kernel and the gap before it.  Narrow local bins only.
template <int LOGW_T, int MODE, int LIST>
__global__ void __launch_bounds__(HIST_THREADS, 1) k_hist_coop(HistArgs a) {
    extern __shared__ __align__(1024) int sh[];
    const TileDesc td = a.tiles[a.tile0 + blockIdx.y];
    const uint32_t P = effective_parts((uint32_t)td.parts, a.n), part = blockIdx.x;
    if (part < P) hist_cta<HIST_THREADS, LOGW_T, MODE, LIST>(a, td, part, P, sh);
    __threadfence();
    cooperative_groups::this_grid().sync();
    if (part >= P || P <= 1) return;
    const int W = 1 << td.logW, nb = a.nb;
    const uint32_t total = 4u * nb * W;
    const size_t stride = (size_t)4 * nb * 32;
    const uint32_t e0 = (uint32_t)((unsigned long long)total * part / P), e1 = (uint32_t)((unsigned long long)total * (part + 1) / P);
    const unsigned long long *pbase = a.partial + (size_t)td.cta0 * stride;
    auto store = [&](uint32_t e, unsigned long long v) {
        const uint32_t wa = e & (W - 1), kb = e >> td.logW, k = kb / nb, bin = kb - k * nb, fl = 4 * wa + k;
        if (fl < (uint32_t)td.nf) a.hist[(size_t)(td.f0 + fl) * nb + bin] = v;
    };
    if (P <= 16) {
        for (uint32_t e = e0 + threadIdx.x; e < e1; e += HIST_THREADS) {
            unsigned long long x[16], v = 0;
#pragma unroll
            for (int k = 0; k < 16; ++k) x[k] = (uint32_t)k < P ? __ldcg(pbase + (size_t)k * stride + e) : 0ull;
#pragma unroll
            for (int k = 0; k < 16; ++k) v += x[k];
            store(e, v);
        }
    } else {
        // 16 groups of 64 threads: group g adds partials g, g + 16, ... of 64 entries at a time
        unsigned long long *acc = reinterpret_cast<unsigned long long *>(sh);   // [16][64], the local histogram is done with
        const uint32_t eg = threadIdx.x & 63, pg = threadIdx.x >> 6;
        for (uint32_t eb = e0; eb < e1; eb += 64) {
            const uint32_t e = eb + eg;
            unsigned long long x[10], v = 0;
#pragma unroll
            for (int k = 0; k < 10; ++k) {
                const uint32_t i = pg + 16u * k;
                x[k] = (e < e1 && i < P) ? __ldcg(pbase + (size_t)i * stride + e) : 0ull;
            }
#pragma unroll
            for (int k = 0; k < 10; ++k) v += x[k];
            for (uint32_t i = pg + 160u; e < e1 && i < P; i += 16) v += __ldcg(pbase + (size_t)i * stride + e);
            __syncthreads();
            acc[pg * 64 + eg] = v;
            __syncthreads();
            if (pg == 0 && e < e1) {
                for (int g = 1; g < 16; ++g) v += acc[g * 64 + eg];
                store(e, v);
            }
        }
    }
}

// Tree growth: a launch builds the histograms of the smaller children (ties: the left one) of all
// leaves being split in the current pass.  The rows are (row, code) pairs in the buffer the scatter
// kernel wrote; a job owns the CTAs x in [cta0, cta0 + parts) of every tile and the partial slots
// slot0 + tile * parts + part.  One CTA for a child: the histogram goes straight to the job's pool
// slot.  Several: on rows of up to 64 bytes they all add into the tile's first partial slot (zero
// before the launch, cleared by its reader), on 128-byte rows each stores a slot of its own; the
// finishing kernel moves the sums to the pool slot.  The grid is (CTAs per tile, tile - tile0).
struct GrowHist {
    const GrowState *gs;
    const uint2 *ent0, *ent1;
    unsigned long long *pool;
    size_t hist_words;
    uint32_t rows_min;   // rows per CTA, at least (qg_grow_parts)
};

template <int LOGW_T, int MODE>
__global__ void __launch_bounds__(HIST_THREADS, 1) k_hist_grow(HistArgs a, GrowHist g) {
    extern __shared__ __align__(1024) int sh[];
    const GrowState *gs = g.gs;
    // the job table and the tile at once (one round trip to memory), then the early exits: lane i of
    // every warp looks at job i
    const int done = gs->done, n_jobs = gs->n_jobs;
    const int li = threadIdx.x & 31;
    const int c0 = gs->jobs[li].cta0, np = gs->jobs[li].parts;
    TileDesc td = a.tiles[a.tile0 + blockIdx.y];
    if (done) return;
    const unsigned hit = __ballot_sync(0xffffffffu, li < n_jobs && (int)blockIdx.x >= c0 && (int)blockIdx.x < c0 + np);
    if (!hit) return;
    const int j = __ffs(hit) - 1;
    const int jc0 = __shfl_sync(0xffffffffu, c0, j);
    const GrowJob *job = gs->jobs + j;
    const int buf = job->buf, parts = job->parts, slot0 = job->slot0, small_slot = job->small_slot;
    const uint32_t nl = job->nl, n = job->n, off = job->off, n_all = job->n_all, nl_all = (uint32_t)gs->nl_all[j];
    const uint32_t nr = n - nl;
    const bool small_is_left = nl_all <= n_all - nl_all;   // by the rows over all ranks (the same child on every rank)
    a.ents = buf == 0 ? g.ent1 : g.ent0;
    a.off = small_is_left ? off : off + nl;
    a.n = small_is_left ? nl : nr;
    a.hist = g.pool + (size_t)small_slot * g.hist_words;
    td.cta0 = slot0 + (a.tile0 + (int)blockIdx.y) * parts;
    const uint32_t P = qg_grow_parts((uint32_t)parts, a.n, g.rows_min), part = blockIdx.x - (uint32_t)jc0;
    if (part >= P) return;
    hist_cta<HIST_THREADS, LOGW_T, MODE, 2>(a, td, part, P, sh);
}

// Sums the partial histograms of every tile that was built by more than one CTA.  A block takes
// 32 consecutive partial entries; its eight thread groups each add every eighth partial.
__global__ void __launch_bounds__(256) k_hist_reduce(const TileDesc *__restrict__ tiles, uint32_t n, int nb,
                                                     const unsigned long long *__restrict__ partial,
                                                     unsigned long long *__restrict__ hist, int paired) {
    const TileDesc td = tiles[blockIdx.y];
    const uint32_t P = paired ? paired_parts(effective_parts((uint32_t)td.parts, n)) : effective_parts((uint32_t)td.parts, n);
    if (P <= 1) return;
    const int W = 1 << td.logW;
    const uint32_t total = 4u * nb * W;
    const size_t stride = (size_t)4 * nb * 32;
    __shared__ unsigned long long acc[8][32];
    const uint32_t ex = threadIdx.x & 31, pg = threadIdx.x >> 5;
    for (uint32_t e0 = blockIdx.x * 32; e0 < total; e0 += gridDim.x * 32) {
        const uint32_t e = e0 + ex;
        unsigned long long s = 0;
        if (e < total) {
            const unsigned long long *p = partial + (size_t)td.cta0 * stride + e;
            // all of a thread's loads are independent and issued together (P <= 8 * 24)
            unsigned long long x[24];
#pragma unroll
            for (int k = 0; k < 24; ++k) {
                const uint32_t i = pg + 8u * k;
                x[k] = i < P ? p[(size_t)i * stride] : 0ull;
            }
#pragma unroll
            for (int k = 0; k < 24; ++k) s += x[k];
            for (uint32_t i = pg + 192u; i < P; i += 8) s += p[(size_t)i * stride];
        }
        acc[pg][ex] = s;
        __syncthreads();
        if (pg == 0 && e < total) {
            for (int g = 1; g < 8; ++g) s += acc[g][ex];
            const uint32_t a = e & (W - 1);
            const uint32_t kb = e >> td.logW;          // k * nb + bin
            const uint32_t k = kb / nb, bin = kb - k * nb;
            const uint32_t fl = 4 * a + k;
            if (fl < (uint32_t)td.nf) hist[(size_t)(td.f0 + fl) * nb + bin] = s;
        }
        __syncthreads();
    }
}

__global__ void k_subtract(const unsigned long long *__restrict__ parent, const unsigned long long *__restrict__ small,
                           unsigned long long *__restrict__ large, long long n) {
    // hessian fields never borrow (child <= parent in every bin), so one 64-bit subtract is exact
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        large[i] = parent[i] - small[i];
}

template <int LOGW_T, int MODE, int LIST>
int launch_one(qgbdt_ctx *c, const HistArgs &args, int n_tiles, cudaStream_t st) {
    auto kern = k_hist<LOGW_T, MODE, LIST>;
    static bool configured[64] = {};   // per instantiation and device (the attribute belongs to the device's context)
    {
        std::lock_guard<std::mutex> lock(g_configure_mutex);
        if (c->device < 0 || c->device >= 64 || !configured[c->device]) {
            QG_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_SMEM));
            if (c->device >= 0 && c->device < 64) configured[c->device] = true;
        }
    }
    int group_parts = 1;
    for (int t = args.tile0; t < args.tile0 + n_tiles; ++t)
        if (c->tiles[t].parts > group_parts) group_parts = c->tiles[t].parts;
    uint32_t gx = effective_parts((uint32_t)group_parts, args.n);
    if (MODE == 1 && args.pass < 0) gx = 2 * paired_parts(gx);
    const dim3 grid(gx, (unsigned)n_tiles);
    kern<<<grid, HIST_THREADS, HIST_SMEM, st>>>(args);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

template <int LOGW_T, int MODE, int LIST>
int launch_one_coop(qgbdt_ctx *c, HistArgs &args, int n_tiles, cudaStream_t st) {
    const void *kern = reinterpret_cast<const void *>(k_hist_coop<LOGW_T, MODE, LIST>);
    static bool configured[64] = {};   // per instantiation and device (the attribute belongs to the device's context)
    {
        std::lock_guard<std::mutex> lock(g_configure_mutex);
        if (c->device < 0 || c->device >= 64 || !configured[c->device]) {
            QG_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_SMEM));
            if (c->device >= 0 && c->device < 64) configured[c->device] = true;
        }
    }
    int group_parts = 1;
    for (int t = args.tile0; t < args.tile0 + n_tiles; ++t)
        if (c->tiles[t].parts > group_parts) group_parts = c->tiles[t].parts;
    const dim3 grid(effective_parts((uint32_t)group_parts, args.n), (unsigned)n_tiles);
    void *params[] = {&args};
    QG_CUDA(c, cudaLaunchCooperativeKernel(kern, grid, dim3(HIST_THREADS), params, HIST_SMEM, st));
    c->n_launches++;
    return QGBDT_OK;
}

// Cooperative variant of launch_hist: the merge happens inside the kernels.
template <int MODE, int LIST>
int launch_hist_coop(qgbdt_ctx *c, HistArgs args, cudaStream_t st) {
    const int T = (int)c->tiles.size();
    for (int t0 = 0; t0 < T;) {
        int t1 = t0 + 1;
        while (t1 < T && c->tiles[t1].logW == c->tiles[t0].logW) ++t1;
        args.tile0 = t0;
        int rc;
        switch (c->tiles[t0].logW) {
            case 5: rc = launch_one_coop<5, MODE, LIST>(c, args, t1 - t0, st); break;
            case 3: rc = launch_one_coop<3, MODE, LIST>(c, args, t1 - t0, st); break;
            default: rc = launch_one_coop<-1, MODE, LIST>(c, args, t1 - t0, st); break;
        }
        if (rc != QGBDT_OK) return rc;
        t0 = t1;
    }
    return QGBDT_OK;
}

// One launch per run of tiles of equal width (the full 128-feature tiles, then the remainder).
template <int MODE, int LIST>
int launch_hist(qgbdt_ctx *c, HistArgs args, cudaStream_t st) {
    const int T = (int)c->tiles.size();
    for (int t0 = 0; t0 < T;) {
        int t1 = t0 + 1;
        while (t1 < T && c->tiles[t1].logW == c->tiles[t0].logW) ++t1;
        args.tile0 = t0;
        int rc;
        switch (c->tiles[t0].logW) {
            case 5: rc = launch_one<5, MODE, LIST>(c, args, t1 - t0, st); break;
            case 3: rc = launch_one<3, MODE, LIST>(c, args, t1 - t0, st); break;
            default: rc = launch_one<-1, MODE, LIST>(c, args, t1 - t0, st); break;
        }
        if (rc != QGBDT_OK) return rc;
        t0 = t1;
    }
    return QGBDT_OK;
}

// Narrow local bins: where to split the 32-bit word between the gradient sum (above) and the
// hessian sum (below) so that a column can take the most rows before it must be flushed.  The
// 16+16 split has the one-instruction decode and is kept unless another split at least doubles
// the rows (a constant hessian counts rows in the low field: 14 bits are enough for 16383 of them).
void pick_field_split(int kg, int kh, int &shift, uint32_t &rows) {
    auto rows_at = [&](int s) {
        const uint32_t by_h = ((1u << s) - 1u) / (uint32_t)kh, by_g = ((1u << (31 - s)) - 1u) / (uint32_t)kg;
        return by_h < by_g ? by_h : by_g;
    };
    shift = 16;
    rows = rows_at(16);
    for (int s = 10; s <= 22; ++s)
        if (rows_at(s) >= 2 * rows_at(16) && rows_at(s) > rows) {
            shift = s;
            rows = rows_at(s);
        }
}

}  // namespace

int qg_hist(qgbdt_ctx *c, const uint32_t *d_rows, int64_t off, int64_t n, unsigned long long *d_hist,
            cudaStream_t st) {
    const size_t hist_bytes = (size_t)c->F * c->nb * sizeof(unsigned long long);
    c->n_hist_builds++;
    c->n_hist_row_features += n * c->F;
    if (n <= 0) {
        QG_CUDA(c, cudaMemsetAsync(d_hist, 0, hist_bytes, st));
        return QGBDT_OK;
    }
    if (!d_rows && off != 0) return qg_fail(c, QGBDT_ERR_ARG, "a contiguous build starts at row 0");

    const int bits = c->prm.bits;
    const int kg = qg_levels_g(bits);
    const int kh = c->const_hess ? 1 : qg_levels_h(bits, c->prm.hess_levels_mode);
    const bool wide = bits >= 6;

    HistArgs a;
    a.tiles = c->d_tiles;
    a.codes = reinterpret_cast<const uint16_t *>(c->d_codes);
    a.codes_nat = reinterpret_cast<const uint16_t *>(c->d_codes_nat);
    a.tile0 = 0;
    a.ents = nullptr;
    a.rows = d_rows;
    a.off = (uint32_t)off;
    a.n = (uint32_t)n;
    a.nb = c->nb;
    a.hist = d_hist;
    a.partial = c->d_partial;
    pick_field_split(kg, kh, a.shift, a.flush_rows);
    a.pass = 0;
    a.state = c->d_state;

    if (c->profile_hist) {
        // algorithmic bytes of this build: bin codes + gradient code (+ row index) per row, histogram out
        c->hist_prof_bytes += n * (c->F + c->code_bytes + (d_rows ? 4 : 0)) + (int64_t)hist_bytes;
        c->hist_prof_launches++;
        const int prc = qg_phase_begin(c, d_rows ? QG_PHASE_CHILD_HIST : QG_PHASE_ROOT_HIST, st);
        if (prc != QGBDT_OK) return prc;
    }
    int rc;
    const bool merge_needed = c->max_parts > 1 && effective_parts((uint32_t)c->max_parts, (uint32_t)n) > 1;
    // with at most one CTA per SM in every launch, the merge can follow a grid barrier in the same kernel
    const bool coop = !wide && merge_needed && c->coop_ok && (int)c->tiles.size() <= c->sm_count;
    if (coop && a.shift == 16) {
        rc = d_rows ? launch_hist_coop<0, 1>(c, a, st) : launch_hist_coop<0, 0>(c, a, st);
    } else if (coop) {
        rc = d_rows ? launch_hist_coop<2, 1>(c, a, st) : launch_hist_coop<2, 0>(c, a, st);
    } else if (!wide && a.shift == 16) {
        rc = d_rows ? launch_hist<0, 1>(c, a, st) : launch_hist<0, 0>(c, a, st);
    } else if (!wide) {
        rc = d_rows ? launch_hist<2, 1>(c, a, st) : launch_hist<2, 0>(c, a, st);
    } else {
        a.pass = -1;   // both passes in one launch, by pairs of CTAs
        rc = d_rows ? launch_hist<1, 1>(c, a, st) : launch_hist<1, 0>(c, a, st);
    }
    if (rc != QGBDT_OK) return rc;
    if (merge_needed && !coop) {
        const dim3 grid((unsigned)((4 * c->nb * 32 + 31) / 32), (unsigned)c->tiles.size());
        k_hist_reduce<<<grid, 256, 0, st>>>(c->d_tiles, (uint32_t)n, c->nb, c->d_partial, d_hist, wide ? 1 : 0);
        QG_LAUNCH_CHECK(c);
    }
    return qg_phase_end(c, st);
}

namespace {

template <int LOGW_T, int MODE>
int launch_grow_one(qgbdt_ctx *c, const HistArgs &args, const GrowHist &g, int n_tiles, cudaStream_t st,
                    bool configure_only) {
    auto kern = k_hist_grow<LOGW_T, MODE>;
    static bool configured[64] = {};   // per instantiation and device (the attribute belongs to the device's context)
    {
        std::lock_guard<std::mutex> lock(g_configure_mutex);
        if (c->device < 0 || c->device >= 64 || !configured[c->device]) {
            QG_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_SMEM));
            if (c->device >= 0 && c->device < 64) configured[c->device] = true;
        }
    }
    if (configure_only) return QGBDT_OK;
    kern<<<dim3((unsigned)c->grow_xcap, (unsigned)n_tiles), HIST_THREADS, HIST_SMEM, st>>>(args, g);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

template <int MODE>
int launch_grow(qgbdt_ctx *c, HistArgs args, const GrowHist &g, cudaStream_t st, bool configure_only = false) {
    const int T = (int)c->tiles.size();
    for (int t0 = 0; t0 < T;) {
        int t1 = t0 + 1;
        while (t1 < T && c->tiles[t1].logW == c->tiles[t0].logW) ++t1;
        args.tile0 = t0;
        int rc;
        switch (c->tiles[t0].logW) {
            case 5: rc = launch_grow_one<5, MODE>(c, args, g, t1 - t0, st, configure_only); break;
            case 3: rc = launch_grow_one<3, MODE>(c, args, g, t1 - t0, st, configure_only); break;
            default: rc = launch_grow_one<-1, MODE>(c, args, g, t1 - t0, st, configure_only); break;
        }
        if (rc != QGBDT_OK) return rc;
        t0 = t1;
    }
    return QGBDT_OK;
}

}  // namespace

// Sets the function attributes of the kernels qg_hist_grow launches for this context (stream
// captures must not meet a first-use configuration).
int qg_hist_grow_configure(qgbdt_ctx *c) {
    const int bits = c->prm.bits;
    const int kh = c->const_hess ? 1 : qg_levels_h(bits, c->prm.hess_levels_mode);
    HistArgs a = {};
    GrowHist g = {};
    pick_field_split(qg_levels_g(bits), kh, a.shift, a.flush_rows);
    if (bits >= 6) return launch_grow<1>(c, a, g, nullptr, true);
    return a.shift == 16 ? launch_grow<0>(c, a, g, nullptr, true) : launch_grow<2>(c, a, g, nullptr, true);
}

// Histograms of the smaller children of the leaves being split in the current pass (sizes known
// only on the device): sums in partial slots or, for a child that one CTA builds, the finished
// histogram in its pool slot.
int qg_hist_grow(qgbdt_ctx *c, cudaStream_t st) {
    const int bits = c->prm.bits;
    const int kg = qg_levels_g(bits);
    const int kh = c->const_hess ? 1 : qg_levels_h(bits, c->prm.hess_levels_mode);
    HistArgs a;
    a.tiles = c->d_tiles;
    a.codes = reinterpret_cast<const uint16_t *>(c->d_codes);
    a.codes_nat = reinterpret_cast<const uint16_t *>(c->d_codes_nat);
    a.tile0 = 0;
    a.rows = nullptr;
    a.ents = nullptr;
    a.off = 0;
    a.n = 0;
    a.nb = c->nb;
    a.hist = nullptr;
    a.partial = c->d_grow_partial;
    pick_field_split(kg, kh, a.shift, a.flush_rows);
    a.pass = 0;
    a.state = c->d_state;
    GrowHist g;
    g.gs = c->d_gs;
    g.ent0 = c->d_ent0;
    g.ent1 = c->d_ent1;
    g.pool = c->d_hist_pool;
    g.hist_words = (size_t)c->F * c->nb;
    g.rows_min = (uint32_t)c->grow_rows_min;
    int prc = qg_phase_begin(c, QG_PHASE_CHILD_HIST, st);
    if (prc != QGBDT_OK) return prc;
    int rc;
    if (bits < 6 && a.shift == 16) {
        rc = launch_grow<0>(c, a, g, st);
    } else if (bits < 6) {
        rc = launch_grow<2>(c, a, g, st);
    } else {
        rc = launch_grow<1>(c, a, g, st);
        if (rc == QGBDT_OK) {
            a.pass = 1;
            rc = launch_grow<1>(c, a, g, st);
        }
    }
    if (rc == QGBDT_OK) rc = qg_phase_end(c, st);
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
