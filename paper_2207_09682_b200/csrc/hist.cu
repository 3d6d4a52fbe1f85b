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
//  * Two-stage merge.  A CTA stores its partial histogram with plain coalesced stores; a small
//    kernel sums the partials of each feature tile.  (64-bit global atomics from 148 CTAs on
//    the same 7 k bins cost about as much as half of the whole build.)
//
// Local bin width: B <= 5 uses one 32-bit word per bin, gradient sum in the high 16 bits
// (signed), hessian sum in the low 16 bits; the CTA flushes before any column can have added
// more rows than fit.  B >= 6 uses two 32-bit words per bin (32+32, a hessian plane and a gradient
// plane) and two passes over the rows, each pass taking two of the four bytes of a word.
#include "qgbdt_internal.cuh"

namespace {

constexpr int HIST_THREADS = 1024;
constexpr int HIST_WARPS = HIST_THREADS / 32;
constexpr int HIST_SMEM = 192 * 1024;     // 128 KB histogram on a 64 KB boundary + the room below it
constexpr uint32_t MIN_ROWS_PER_CTA = 4096;
constexpr int U_ROOT = 4;                 // units in flight per lane, contiguous rows
constexpr int U_LIST = 2;                 // units in flight per lane, row list (plus as many index units)

struct HistArgs {
    const TileDesc *tiles;
    const uint16_t *codes;         // per-row code (g8 << 8 | h8), transposed inside blocks of 16 rows
    const uint16_t *codes_nat;     // the same codes in row order (row lists and leftover rows)
    int tile0;                     // first tile of this launch
    // tree growth: the rows are the smaller child of the split recorded in *gs (nullptr otherwise)
    const GrowState *gs;
    const uint32_t *idx0, *idx1;   // the two row-index buffers
    unsigned long long *pool;      // histogram pool, slot stride F * nb words
    size_t hist_words;
    const uint32_t *rows;          // row list, or nullptr: rows 0 .. n-1
    uint32_t off, n;               // list: entries rows[off .. off+n)
    int nb;
    unsigned long long *hist;      // [F][nb]
    unsigned long long *partial;   // [CTA][4][nb][32]
    uint32_t flush_rows;           // rows one column may add between flushes (16+16 local only)
    int pass;                      // 32+32 local only: bytes 2*pass, 2*pass+1 of every word
    DevState *state;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t s) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(s));
    return d;
}

template <int IMM>
__device__ __forceinline__ void red32(uint32_t addr, int v) {
    asm volatile("red.shared.add.u32 [%0+%1], %2;" ::"r"(addr), "n"(IMM), "r"(v) : "memory");
}

__device__ __forceinline__ uint32_t ldg32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ uint2 ldg64(const uint2 *p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t ldg16(const uint16_t *p) {
    uint32_t v;
    asm volatile("{ .reg .u16 t; ld.global.nc.L1::no_allocate.u16 t, [%1]; cvt.u32.u16 %0, t; }" : "=r"(v) : "l"(p));
    return v;
}

// One row's word: its bin codes -> shared atomics.  `half` selects the 16-bit code in the low
// or high half of c.
template <bool WIDE>
__device__ __forceinline__ void add_word(uint32_t base, uint32_t w, uint32_t c, int half, int pass) {
    if (!WIDE) {
        // inc = g * 65536 + h: byte 0 = h, byte 1 = 0, byte 2 = g, byte 3 = sign of g
        const int inc = (int)prmt(c, 0u, half ? 0xB342u : 0x9140u);
        red32<0>(prmt(w, base, 0x7604u), inc);
        red32<128>(prmt(w, base, 0x7614u), inc);
        red32<65536>(prmt(w, base, 0x7624u), inc);
        red32<65536 + 128>(prmt(w, base, 0x7634u), inc);
    } else {
        // 32+32 local bins: the hessian plane at +0 and the gradient plane at +128 of a bin's 256 bytes
        const int h = (int)prmt(c, 0u, half ? 0x4442u : 0x4440u);
        const int g = (int)prmt(c, 0u, half ? 0xBBB3u : 0x9991u);   // sign-extended
        const uint32_t s0 = 0x7604u | ((uint32_t)(2 * pass) << 4), s1 = s0 + 0x10u;
        const uint32_t a0 = prmt(w, base, s0), a1 = prmt(w, base, s1);
        red32<0>(a0, h);
        red32<128>(a0, g);
        red32<65536>(a1, h);
        red32<65536 + 128>(a1, g);
    }
}

struct Out {
    unsigned long long *ptr;   // partial slot of this CTA, or the final histogram
    bool direct;               // final layout hist[f][bin] instead of partial [k][bin][a]
    bool first;                // nothing stored yet: store instead of accumulate
};

// Adds the CTA's local histogram into its output and clears it.  The R replicas of a column
// (the row slots of word a) are R adjacent shared words, so one thread sums them from vector
// loads and writes one packed 64-bit bin.
template <bool WIDE>
__device__ inline void flush_local(int *hp, const TileDesc &td, const int logW, int nb, int pass, Out &out) {
    const int W = 1 << logW, R = 32 >> logW;
    const int per_k = nb << logW;                                   // outputs per byte position k
    for (int kk = 0; kk < (WIDE ? 2 : 4); ++kk) {
        const int k = WIDE ? 2 * pass + kk : kk;
        for (int e = threadIdx.x; e < per_k; e += HIST_THREADS) {
            const int a = e & (W - 1), bin = e >> logW;
            unsigned long long v;
            if (!WIDE) {
                int *p = hp + (kk >> 1) * 16384 + bin * 64 + (kk & 1) * 32 + a * R;
                int G = 0, H = 0;
                if (R >= 4) {
                    for (int r = 0; r < R; r += 4) {
                        const int4 x = *reinterpret_cast<const int4 *>(p + r);
                        *reinterpret_cast<int4 *>(p + r) = make_int4(0, 0, 0, 0);
                        G += (x.x >> 16) + (x.y >> 16) + (x.z >> 16) + (x.w >> 16);
                        H += (x.x & 0xFFFF) + (x.y & 0xFFFF) + (x.z & 0xFFFF) + (x.w & 0xFFFF);
                    }
                } else {
                    for (int r = 0; r < R; ++r) {
                        const int x = p[r];
                        p[r] = 0;
                        G += x >> 16;
                        H += x & 0xFFFF;
                    }
                }
                v = (unsigned long long)((long long)G * 4294967296LL + (long long)H);
            } else {
                // two 32-bit planes per bin; no field can overflow (checked at load time)
                int *p = hp + kk * 16384 + bin * 64 + a * R;
                long long G = 0;
                unsigned long long H = 0;
                for (int r = 0; r < R; ++r) {
                    H += (unsigned int)p[r];
                    G += p[32 + r];
                    p[r] = 0;
                    p[32 + r] = 0;
                }
                v = (unsigned long long)(G * 4294967296LL + (long long)H);
            }
            const int fl = 4 * a + k;
            if (fl < td.nf) {
                unsigned long long *q = out.direct ? out.ptr + (size_t)(td.f0 + fl) * nb + bin
                                                   : out.ptr + (size_t)k * nb * W + e;
                if (!out.first) v += *q;
                *q = v;
            }
        }
    }
    out.first = false;
}

// CTAs of the static plan that take part in a build of n rows of a tile.
__device__ __host__ inline uint32_t effective_parts(uint32_t parts, uint32_t n) {
    uint32_t want = (n + MIN_ROWS_PER_CTA - 1) / MIN_ROWS_PER_CTA;
    if (want < 1) want = 1;
    return want < parts ? want : parts;
}

// The work of a lane is cut into units of four rows.  Contiguous rows: unit v covers rows
// 16 (v / 4) + 4 j + v % 4, j = 0..3, whose codes are the four adjacent 16-bit values codes[4v ..].
// Row list: warp-unit q covers list entries 4 R q .. 4 R (q + 1) - 1, entry 4 R q + R j + slot for
// the lane's j-th row.  A warp instruction spans R units (one per row slot): a "warp-unit".
//
// LOGW_T >= 0 fixes the tile width at compile time (all strides become immediates); -1 reads it
// from the tile.  The grid is (part, tile - tile0).
template <int LOGW_T, bool WIDE, bool LIST>
__global__ void __launch_bounds__(HIST_THREADS, 1) k_hist(HistArgs a) {
    extern __shared__ __align__(1024) int sh[];
    const TileDesc td = a.tiles[a.tile0 + blockIdx.y];
    if (LIST && a.gs) {
        // the smaller child (ties: the left one) in the buffer the scatter kernel wrote; its
        // histogram goes to the pool slot numbered like the leaf about to be created
        const GrowState *gs = a.gs;
        if (gs->done) return;
        const uint32_t nl = gs->nl, nr = gs->n - nl;
        a.rows = gs->buf == 0 ? a.idx1 : a.idx0;
        a.off = nl <= nr ? gs->off : gs->off + nl;
        a.n = nl <= nr ? nl : nr;
        a.hist = a.pool + (size_t)gs->n_leaves * a.hist_words;
    }
    const uint32_t n = a.n;
    const uint32_t P = effective_parts((uint32_t)td.parts, n);
    const uint32_t part = blockIdx.x;
    if (part >= P) return;

    const uint32_t sbase = smem_u32(sh);
    const uint32_t h0 = (sbase + 65535u) & ~65535u;
    uint32_t dyn_size;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_size));
    if (h0 + 131072u > sbase + dyn_size) {   // the launch below leaves room; never write out of bounds
        if (threadIdx.x == 0) atomicExch(&a.state->kernel_error, 1);
        return;
    }
    int *hp = sh + (h0 - sbase) / 4;
    const int lane = threadIdx.x & 31;
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform for the compiler
    for (int i = threadIdx.x; i < a.nb * 64; i += HIST_THREADS) {
        hp[i] = 0;
        hp[16384 + i] = 0;
    }
    __syncthreads();

    const int logW = LOGW_T >= 0 ? LOGW_T : td.logW;
    const int logR = 5 - logW;
    const uint32_t R = 1u << logR;
    const uint32_t wa = lane >> logR;           // word of the row held by this lane
    const uint32_t slot = lane & (R - 1);       // row slot of this lane (adjacent lanes: replicas of a column)
    const uint32_t base = h0 + lane * 4;
    const uint32_t *tile = td.data;
    const int pass = a.pass;

    Out out;
    out.direct = P == 1;
    out.first = true;   // the two passes of the 32+32 mode write different features
    out.ptr = out.direct ? a.hist : a.partial + (size_t)(td.cta0 + part) * 4 * a.nb * 32;

    // ---- range of this part in warp-units [0, q1) from its first unit, and the leftover rows /
    //      entries [s0, s1) that are done one by one
    uint32_t q1, s0, s1, first_unit = 0, first_q = 0;
    if (!LIST) {
        const uint32_t B = n >> 4;                                   // full blocks of 16 rows
        const uint32_t b0 = (uint32_t)((unsigned long long)B * part / P);
        const uint32_t b1 = (uint32_t)((unsigned long long)B * (part + 1) / P);
        first_unit = b0 << 2;
        if (logR >= 2) {                                             // a warp-unit is R / 4 whole blocks
            const int lb = logR >= 2 ? logR - 2 : 0;                 // log2 of blocks per warp-unit
            q1 = (b1 - b0) >> lb;
            s0 = (b0 + (q1 << lb)) << 4;
        } else {                                                     // 4 / R warp-units per block
            q1 = (b1 - b0) << (2 - logR);
            s0 = b1 << 4;
        }
        s1 = part + 1 == P ? n : b1 << 4;
    } else {
        const uint32_t per = 4u << logR;                             // entries per warp-unit
        const uint32_t Q = n / per;                                  // full warp-units
        first_q = (uint32_t)((unsigned long long)Q * part / P);
        q1 = (uint32_t)((unsigned long long)Q * (part + 1) / P) - first_q;
        s0 = part + 1 == P ? Q * per : 0;
        s1 = part + 1 == P ? n : 0;
    }

    // ---- leftover rows first (the column counters are still zero): R rows per warp instruction
    uint32_t col_rows = 0;   // rows any one column may hold since the last flush
    if (s1 > s0) {
        for (uint32_t i = s0 + warp * R + slot; i < s1; i += HIST_WARPS * R) {
            const uint32_t row = LIST ? a.rows[a.off + i] : i;
            const uint32_t w = tile[((size_t)row << logW) + wa];
            const uint32_t c = a.codes_nat[row];
            add_word<WIDE>(base, w, c, 0, pass);
        }
        col_rows = (s1 - s0 + R - 1) >> logR;
    }

    // ---- fast warp-units, in epochs that keep every 16+16 column below its limit
    constexpr int U = LIST ? U_LIST : U_ROOT;
    uint32_t q = 0;
    while (q < q1) {
        uint32_t epoch = q1 - q;   // warp-units of this epoch, all warps together
        if (!WIDE) {
            const uint32_t room = a.flush_rows > col_rows ? a.flush_rows - col_rows : 0;
            const uint32_t fit = room >> 2;                          // every warp-unit adds 4 rows to each column
            if (fit == 0) {
                __syncthreads();
                flush_local<WIDE>(hp, td, logW, a.nb, pass, out);
                __syncthreads();
                col_rows = 0;
                continue;
            }
            if (fit < epoch) epoch = fit;
        }
        // this warp's warp-units: q + warp, q + warp + 32, ... < q + epoch
        const uint32_t nq = epoch > (uint32_t)warp ? (epoch - warp + HIST_WARPS - 1) / HIST_WARPS : 0;
        if (!LIST) {
            const uint32_t v = first_unit + ((q + warp) << logR) + slot;         // first unit of this lane
            const uint32_t row0 = ((v >> 2) << 4) + (v & 3u);
            const uint32_t *pw = tile + ((size_t)row0 << logW) + wa;
            const uint2 *pc = reinterpret_cast<const uint2 *>(a.codes) + v;
            const uint32_t jstride = 4u << logW;                                  // words between rows 4 apart
            constexpr uint32_t QW = 32 * 128;                                     // words per 32 warp-units
            const uint32_t qc = 32u << logR;                                      // units per 32 warp-units
            uint32_t w[U][4];
            uint2 c[U];
#define QG_LOAD_UNIT(u)                                                                  \
    {                                                                                    \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) w[u][j] = ldg32(pw + (u) * QW + j * jstride); \
        c[u] = ldg64(pc + (u) * qc);                                                     \
    }
#define QG_USE_UNIT(u)                                       \
    {                                                        \
        add_word<WIDE>(base, w[u][0], c[u].x, 0, pass);      \
        add_word<WIDE>(base, w[u][1], c[u].x, 1, pass);      \
        add_word<WIDE>(base, w[u][2], c[u].y, 0, pass);      \
        add_word<WIDE>(base, w[u][3], c[u].y, 1, pass);      \
    }
#pragma unroll
            for (int u = 0; u < U; ++u)
                if ((uint32_t)u < nq) QG_LOAD_UNIT(u)
            pw += U * QW;
            pc += U * qc;
            uint32_t i = 0;
            for (; i + 2 * U <= nq; i += U) {   // units i .. i+U-1 are in registers, the next U exist
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    QG_USE_UNIT(u)
                    QG_LOAD_UNIT(u)
                }
                pw += U * QW;
                pc += U * qc;
            }
            for (; i < nq; i += U) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (i + u < nq) {
                        QG_USE_UNIT(u)
                        if (i + u + U < nq) QG_LOAD_UNIT(u)
                    }
                }
                pw += U * QW;
                pc += U * qc;
            }
#undef QG_LOAD_UNIT
#undef QG_USE_UNIT
        } else {
            // entry of (warp-unit wu, j): off + (4 wu << logR) + (j << logR) + slot
            const uint32_t *pr = a.rows + a.off + ((size_t)(first_q + q + warp) << (logR + 2)) + slot;
            const uint32_t qs = 128u << logR;                                     // entries per 32 warp-units
            const uint32_t *tw = tile + wa;
            uint32_t idx[U][4], w[U][4], c[U][4];
#define QG_LOAD_IDX(u)                                                                              \
    {                                                                                               \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) idx[u][j] = pr[(u) * qs + ((uint32_t)j << logR)]; \
    }
#define QG_LOAD_DATA(u)                                                \
    {                                                                  \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) {                \
            w[u][j] = ldg32(tw + ((size_t)idx[u][j] << logW));         \
            c[u][j] = ldg16(a.codes_nat + idx[u][j]);                  \
        }                                                              \
    }
#define QG_USE_DATA(u)                                                                           \
    {                                                                                            \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) add_word<WIDE>(base, w[u][j], c[u][j], 0, pass); \
    }
#pragma unroll
            for (int u = 0; u < U; ++u)
                if ((uint32_t)u < nq) QG_LOAD_IDX(u)
            pr += U * qs;
#pragma unroll
            for (int u = 0; u < U; ++u)
                if ((uint32_t)u < nq) {
                    QG_LOAD_DATA(u)
                    if ((uint32_t)u + U < nq) QG_LOAD_IDX(u)
                }
            pr += U * qs;
            uint32_t i = 0;
            for (; i + 3 * U <= nq; i += U) {   // data of units i .. i+U-1 and indices of the next U are in registers
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    QG_USE_DATA(u)
                    QG_LOAD_DATA(u)
                    QG_LOAD_IDX(u)
                }
                pr += U * qs;
            }
            for (; i < nq; i += U) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (i + u < nq) {
                        QG_USE_DATA(u)
                        if (i + u + U < nq) {
                            QG_LOAD_DATA(u)
                            if (i + u + 2 * U < nq) QG_LOAD_IDX(u)
                        }
                    }
                }
                pr += U * qs;
            }
#undef QG_LOAD_IDX
#undef QG_LOAD_DATA
#undef QG_USE_DATA
        }
        q += epoch;
        col_rows += 4 * epoch;
    }
    __syncthreads();
    flush_local<WIDE>(hp, td, logW, a.nb, pass, out);
}

// Sums the partial histograms of every tile that was built by more than one CTA.  A block takes
// 32 consecutive partial entries; its eight thread groups each add every eighth partial.
__global__ void __launch_bounds__(256) k_hist_reduce(const TileDesc *__restrict__ tiles, uint32_t n, int nb,
                                                     const unsigned long long *__restrict__ partial,
                                                     unsigned long long *__restrict__ hist) {
    const TileDesc td = tiles[blockIdx.y];
    const uint32_t P = effective_parts((uint32_t)td.parts, n);
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
            uint32_t i = pg;
            for (; i + 24 < P; i += 32) {
                const unsigned long long x0 = p[(size_t)i * stride], x1 = p[(size_t)(i + 8) * stride];
                const unsigned long long x2 = p[(size_t)(i + 16) * stride], x3 = p[(size_t)(i + 24) * stride];
                s += (x0 + x1) + (x2 + x3);
            }
            for (; i < P; i += 8) s += p[(size_t)i * stride];
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

template <int LOGW_T, bool WIDE, bool LIST>
int launch_one(qgbdt_ctx *c, const HistArgs &args, int n_tiles, cudaStream_t st) {
    auto kern = k_hist<LOGW_T, WIDE, LIST>;
    static bool configured = false;   // per instantiation
    if (!configured) {
        QG_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, HIST_SMEM));
        configured = true;
    }
    int group_parts = 1;
    for (int t = args.tile0; t < args.tile0 + n_tiles; ++t)
        if (c->tiles[t].parts > group_parts) group_parts = c->tiles[t].parts;
    const dim3 grid(args.gs ? (unsigned)group_parts : effective_parts((uint32_t)group_parts, args.n), (unsigned)n_tiles);
    kern<<<grid, HIST_THREADS, HIST_SMEM, st>>>(args);
    QG_LAUNCH_CHECK(c);
    return QGBDT_OK;
}

// One launch per run of tiles of equal width (the full 128-feature tiles, then the remainder).
template <bool WIDE, bool LIST>
int launch_hist(qgbdt_ctx *c, HistArgs args, cudaStream_t st) {
    const int T = (int)c->tiles.size();
    for (int t0 = 0; t0 < T;) {
        int t1 = t0 + 1;
        while (t1 < T && c->tiles[t1].logW == c->tiles[t0].logW) ++t1;
        args.tile0 = t0;
        int rc;
        switch (c->tiles[t0].logW) {
            case 5: rc = launch_one<5, WIDE, LIST>(c, args, t1 - t0, st); break;
            case 3: rc = launch_one<3, WIDE, LIST>(c, args, t1 - t0, st); break;
            default: rc = launch_one<-1, WIDE, LIST>(c, args, t1 - t0, st); break;
        }
        if (rc != QGBDT_OK) return rc;
        t0 = t1;
    }
    return QGBDT_OK;
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
    a.gs = nullptr;
    a.idx0 = a.idx1 = nullptr;
    a.pool = nullptr;
    a.hist_words = 0;
    a.rows = d_rows;
    a.off = (uint32_t)off;
    a.n = (uint32_t)n;
    a.nb = c->nb;
    a.hist = d_hist;
    a.partial = c->d_partial;
    const uint32_t by_h = 65535u / (uint32_t)kh, by_g = 32767u / (uint32_t)kg;
    a.flush_rows = by_h < by_g ? by_h : by_g;
    a.pass = 0;
    a.state = c->d_state;

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
        // algorithmic bytes of this build: bin codes + gradient code (+ row index) per row, histogram out
        c->hist_prof_bytes += n * (c->F + c->code_bytes + (d_rows ? 4 : 0)) + (int64_t)hist_bytes;
        c->hist_prof_launches++;
        QG_CUDA(c, cudaEventRecord(ev0, st));
    }
    int rc;
    if (!wide) {
        rc = d_rows ? launch_hist<false, true>(c, a, st) : launch_hist<false, false>(c, a, st);
    } else {
        rc = d_rows ? launch_hist<true, true>(c, a, st) : launch_hist<true, false>(c, a, st);
        if (rc == QGBDT_OK) {
            a.pass = 1;
            rc = d_rows ? launch_hist<true, true>(c, a, st) : launch_hist<true, false>(c, a, st);
        }
    }
    if (rc != QGBDT_OK) return rc;
    if (c->max_parts > 1 && effective_parts((uint32_t)c->max_parts, (uint32_t)n) > 1) {
        const dim3 grid((unsigned)((4 * c->nb * 32 + 31) / 32), (unsigned)c->tiles.size());
        k_hist_reduce<<<grid, 256, 0, st>>>(c->d_tiles, (uint32_t)n, c->nb, c->d_partial, d_hist);
        QG_LAUNCH_CHECK(c);
    }
    if (ev1) QG_CUDA(c, cudaEventRecord(ev1, st));
    return QGBDT_OK;
}

// Histogram of the smaller child of the split recorded in the grow state (sizes known only on
// the device): partial histograms or, for a small child, the finished histogram in its pool slot.
int qg_hist_grow(qgbdt_ctx *c, cudaStream_t st) {
    const int bits = c->prm.bits;
    const int kg = qg_levels_g(bits);
    const int kh = c->const_hess ? 1 : qg_levels_h(bits, c->prm.hess_levels_mode);
    HistArgs a;
    a.tiles = c->d_tiles;
    a.codes = reinterpret_cast<const uint16_t *>(c->d_codes);
    a.codes_nat = reinterpret_cast<const uint16_t *>(c->d_codes_nat);
    a.tile0 = 0;
    a.gs = c->d_gs;
    a.idx0 = c->d_idx;
    a.idx1 = c->d_idx_tmp;
    a.pool = c->d_hist_pool;
    a.hist_words = (size_t)c->F * c->nb;
    a.rows = nullptr;
    a.off = 0;
    a.n = 0;
    a.nb = c->nb;
    a.hist = nullptr;
    a.partial = c->d_partial;
    const uint32_t by_h = 65535u / (uint32_t)kh, by_g = 32767u / (uint32_t)kg;
    a.flush_rows = by_h < by_g ? by_h : by_g;
    a.pass = 0;
    a.state = c->d_state;
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
        QG_CUDA(c, cudaEventRecord(ev0, st));
    }
    int rc;
    if (bits < 6) {
        rc = launch_hist<false, true>(c, a, st);
    } else {
        rc = launch_hist<true, true>(c, a, st);
        if (rc == QGBDT_OK) {
            a.pass = 1;
            rc = launch_hist<true, true>(c, a, st);
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
