// Device code of the histogram build (Algorithm 1 with integer gradients), shared by the
// stand-alone kernel and by the tree-growing kernel.  See hist.cu for the design notes.
#pragma once

#include "qgbdt_internal.cuh"

namespace {

constexpr int HIST_THREADS = 1024;
constexpr int HIST_WARPS = HIST_THREADS / 32;
constexpr int HIST_SMEM = 192 * 1024;     // 128 KB histogram on a 64 KB boundary + the room below it
constexpr uint32_t MIN_ROWS_PER_CTA = 1024;
// Wide tiles with at least this many bins look for hot words instead of flushing everything (a
// look comes twice as often as a flush would; with few bins a flush is cheap and wins).
constexpr int SELECTIVE_MIN_BINS = 128;
// A word is hot from 2^-SELECTIVE_T of a field's range on: an eighth in stand-alone builds (fewer
// looks); a half in the builds of tree growth, whose CTAs rarely see enough rows for a look and
// whose kernel came out 4 % slower per tree of the 2000-feature workload with the other test
// compiled in.
template <int LIST> struct SelectiveT { static constexpr int value = LIST == 2 ? 1 : 3; };

template <int T>
__device__ __forceinline__ uint32_t hot_bits(uint32_t x, uint32_t gm, uint32_t hm, int lsh) {
    if (T == 1) return ((x + 0x40000000u) | (x << lsh)) & 0x80000000u;   // the same test in fewer operations
    return ((x ^ (x << 1)) & gm) | (x & hm);
}
// Units of four rows in flight per lane.  A CTA of 512 threads (the tree-growing kernel) has twice
// the registers per thread and keeps more in flight per lane to make up for the fewer warps.
template <int NT> struct Units { static constexpr int root = NT >= 1024 ? 4 : 6, list = NT >= 1024 ? 2 : 4; };

struct HistArgs {
    const TileDesc *tiles;
    const uint16_t *codes;         // per-row code (g8 << 8 | h8), transposed inside blocks of 16 rows
    const uint16_t *codes_nat;     // the same codes in row order (row lists and leftover rows)
    int tile0;                     // first tile of this launch
    const uint32_t *rows;          // row list (LIST 1), or nullptr: rows 0 .. n-1 (LIST 0)
    const uint2 *ents;             // (row, code) pairs written by the tree-growing scatter (LIST 2)
    uint32_t off, n;               // list: entries rows[off .. off+n)
    int nb;
    unsigned long long *hist;      // [F][nb]
    unsigned long long *partial;   // [CTA][4][nb][32]
    uint32_t flush_rows;           // rows of the extreme levels a zeroed column can add (narrow local bins only)
    int shift;                     // narrow local bins: bit position of the gradient field (16: the 16+16 split)
    int pass;                      // 32+32 local only: bytes 2*pass, 2*pass+1 of every word (-1 at launch: the
                                   // CTA takes its pass from its number)
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
template <int MODE>
__device__ __forceinline__ void add_word(uint32_t base, uint32_t w, uint32_t c, int half, int pass, int shift) {
    if (MODE == 2) {
        // gradient field above bit `shift`, hessian below: inc = g * 2^shift + h
        const int h = (int)prmt(c, 0u, half ? 0x4442u : 0x4440u);
        const int g = (int)prmt(c, 0u, half ? 0xBBB3u : 0x9991u);   // sign-extended
        const int inc = g * (1 << shift) + h;
        red32<0>(prmt(w, base, 0x7604u), inc);
        red32<128>(prmt(w, base, 0x7614u), inc);
        red32<65536>(prmt(w, base, 0x7624u), inc);
        red32<65536 + 128>(prmt(w, base, 0x7634u), inc);
    } else if (MODE != 1) {
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
    bool shared_out;           // several CTAs add into the same (zeroed) output: reductions instead of stores
};

// Adds the CTA's local histogram into its output and clears it.  The R replicas of a column
// (the row slots of word a) are R adjacent shared words, so one thread sums them from vector
// loads and writes one packed 64-bit bin.
template <int NT, int MODE>
__device__ inline void flush_local(int *hp, const TileDesc &td, const int logW, int nb, int pass, int shift, Out &out) {
    const int hmask = (1 << shift) - 1;   // narrow bins: hessian field below bit `shift` (16 unless MODE 2)
    const int W = 1 << logW, R = 32 >> logW;
    const int per_k = nb << logW;                                   // outputs per byte position k
    for (int kk = 0; kk < (MODE == 1 ? 2 : 4); ++kk) {
        const int k = MODE == 1 ? 2 * pass + kk : kk;
        for (int e = threadIdx.x; e < per_k; e += NT) {
            const int a = e & (W - 1), bin = e >> logW;
            unsigned long long v;
            if (MODE != 1) {
                int *p = hp + (kk >> 1) * 16384 + bin * 64 + (kk & 1) * 32 + a * R;
                int G = 0, H = 0;
                if (R >= 4) {
                    for (int r = 0; r < R; r += 4) {
                        const int4 x = *reinterpret_cast<const int4 *>(p + r);
                        *reinterpret_cast<int4 *>(p + r) = make_int4(0, 0, 0, 0);
                        G += (x.x >> shift) + (x.y >> shift) + (x.z >> shift) + (x.w >> shift);
                        H += (x.x & hmask) + (x.y & hmask) + (x.z & hmask) + (x.w & hmask);
                    }
                } else {
                    for (int r = 0; r < R; ++r) {
                        const int x = p[r];
                        p[r] = 0;
                        G += x >> shift;
                        H += x & hmask;
                    }
                }
                v = (unsigned long long)((long long)G * 4294967296LL + (long long)H);
            } else {
                // two 32-bit planes per bin; no field can overflow (rows x levels is checked against the word at load time and for every row list)
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
                if (out.shared_out) {
                    if (v) atomicAdd(q, v);
                } else {
                    if (!out.first) v += *q;
                    *q = v;
                }
            }
        }
    }
    out.first = false;
}

// Wide tiles (one or two row slots per column: a flush moves up to 32 k bins through global
// memory) avoid most flushes: a column only adds 7/8 of `flush_rows` rows at a time, after which
// the CTA looks at every local word.  One whose hessian field has reached an eighth of its range,
// or whose gradient field has left the middle eighth of its range, is "hot": its sums move to the
// output (a reduction on the word's 64-bit bin) and the word restarts from zero; all other words
// can take another 7/8 of `flush_rows` rows as they are.  With bin codes spread over many bins
// almost no word is hot.  Before the first flush the output holds nothing that could be added
// to: then a hot word asks for a full flush (return value, CTA-uniform).  Callers synchronise
// before the call; the call ends with a barrier.
template <int NT, int MODE, int LOGW_T, int SELECTIVE_T>
__device__ __forceinline__ bool relieve_local(int *hp, const TileDesc &td, const int logW_rt, int nb, int shift,
                                              const Out &out) {
    static_assert(MODE != 1, "32+32 local bins never overflow");
    const int logW = LOGW_T >= 0 ? LOGW_T : logW_rt;
    const int logR = 5 - logW, W = 1 << logW;
    // hot: any of the top SELECTIVE_T bits of the hessian field set, or the top SELECTIVE_T + 1 bits
    // of the word (the gradient field's sign and the bits below it) not all equal
    const uint32_t hm = ((1u << SELECTIVE_T) - 1u) << (shift - SELECTIVE_T);
    const uint32_t gm = ~0u << (32 - SELECTIVE_T);
    const int lsh = 32 - shift;
    const int hmask = (1 << shift) - 1;
    bool want_full = false;
    const int n4 = nb * 16;                       // 16-byte groups per half of the local histogram
    for (int half = 0; half < 2; ++half) {
        for (int i = threadIdx.x; i < n4; i += NT) {
            int4 *p = reinterpret_cast<int4 *>(hp + half * 16384) + i;
            const int4 x = *p;
            // bit 31: gradient field outside [-2^(30-shift), 2^(30-shift)), or top bit of the hessian field set
            const uint32_t m = hot_bits<SELECTIVE_T>((uint32_t)x.x, gm, hm, lsh) | hot_bits<SELECTIVE_T>((uint32_t)x.y, gm, hm, lsh) |
                               hot_bits<SELECTIVE_T>((uint32_t)x.z, gm, hm, lsh) | hot_bits<SELECTIVE_T>((uint32_t)x.w, gm, hm, lsh);
            if (m) {
                if (out.first) {
                    want_full = true;
                } else {
                    int xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (hot_bits<SELECTIVE_T>((uint32_t)xs[j], gm, hm, lsh)) {
                            const int w = i * 4 + j;                      // word inside this half
                            const int bin = w >> 6, k = half * 2 + ((w >> 5) & 1), a = (w & 31) >> logR;
                            const int fl = 4 * a + k;
                            if (fl < td.nf) {
                                const long long G = xs[j] >> shift, H = xs[j] & hmask;
                                unsigned long long *q = out.direct ? out.ptr + (size_t)(td.f0 + fl) * nb + bin
                                                                   : out.ptr + (size_t)k * nb * W + (bin << logW) + a;
                                atomicAdd(q, (unsigned long long)(G * 4294967296LL + H));
                            }
                            xs[j] = 0;
                        }
                    }
                    *p = make_int4(xs[0], xs[1], xs[2], xs[3]);
                }
            }
        }
    }
    return __syncthreads_or(want_full ? 1 : 0) != 0;
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
// One CTA's share (part `part` of P) of the histogram of a.n rows for tile td.  `sh` is the
// CTA's dynamic shared memory (HIST_SMEM bytes).  Ends with the CTA's local histogram flushed.
template <int NT, int LOGW_T, int MODE, int LIST>
__device__ __forceinline__ void hist_cta(const HistArgs &a, const TileDesc &td, const uint32_t part, const uint32_t P,
                                         int *sh) {
    const uint32_t n = a.n;

    const uint32_t sbase = smem_u32(sh);
    const uint32_t h0 = (sbase + 65535u) & ~65535u;
    uint32_t dyn_size;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_size));
    if (h0 + 131072u > sbase + dyn_size) {   // the launches leave room; never write out of bounds
        if (threadIdx.x == 0) atomicExch(&a.state->kernel_error, 1);
        return;
    }
    int *hp = sh + (h0 - sbase) / 4;
    const int lane = threadIdx.x & 31;
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform for the compiler
    for (int i = threadIdx.x; i < a.nb * 64; i += NT) {
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
    const int shift = MODE == 2 ? a.shift : 16;

    Out out;
    out.direct = P == 1;
    // tree growth, rows of up to 64 bytes: the CTAs of a leaf's tile all add into the tile's first partial
    // slot, which is zero before the launch (whoever reads it clears it); integer sums come out the same
    // in any order.  (128-byte rows: 32 k reductions per CTA cost more than the partial slots' stores.)
    out.shared_out = LIST == 2 && P > 1 && logW < QG_SHARED_PARTIAL_LOGW;
    out.first = !out.shared_out;   // the two passes of the 32+32 mode write different features
    out.ptr = out.direct ? a.hist : a.partial + (size_t)(td.cta0 + (out.shared_out ? 0u : part)) * 4 * a.nb * 32;

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
        for (uint32_t i = s0 + warp * R + slot; i < s1; i += (NT / 32) * R) {
            uint32_t row, c;
            if (LIST == 2) {
                const uint2 e = __ldcg(a.ents + a.off + i);
                row = e.x;
                c = e.y;
            } else {
                row = LIST ? a.rows[a.off + i] : i;
                c = a.codes_nat[row];
            }
            const uint32_t w = tile[((size_t)row << logW) + wa];
            add_word<MODE>(base, w, c, 0, pass, shift);
        }
        col_rows = (s1 - s0 + R - 1) >> logR;
    }

    // ---- fast warp-units.  This warp takes warp-units warp, warp + NWARPS, ... of the part, in
    //      groups of U; every lane keeps its loads for the next group in flight in registers.
    //      Every 16+16 column must stay below its limit: after `kg` groups (4 U NWARPS kg rows per
    //      column) all warps meet, and the CTA flushes, or looks for hot words.  The loads in
    //      flight stay in flight across that meeting.
    constexpr int U = LIST ? Units<NT>::list : Units<NT>::root;
    constexpr int NWARPS = NT / 32;
    constexpr int SELECTIVE_T = SelectiveT<LIST>::value;
    const bool selective = logR <= 1 && a.nb >= SELECTIVE_MIN_BINS;   // wide tiles: look for hot words instead of flushing everything
    const uint32_t nq = q1 > (uint32_t)warp ? (q1 - warp + NWARPS - 1) / NWARPS : 0;   // this warp's units
    const uint32_t groups = ((q1 + NWARPS - 1) / NWARPS + U - 1) / U;                  // of warp 0: the same in every warp
    uint32_t kg = 0xFFFFFFFFu;                                                         // groups between two meetings
    if (MODE != 1) {
        // after a look every field has at least 1 - 2^-SELECTIVE_T of its range left
        const uint32_t limit = !selective ? a.flush_rows
                               : (SELECTIVE_T == 1 ? a.flush_rows >> 1 : a.flush_rows - (a.flush_rows >> SELECTIVE_T) - 1);
        kg = (limit > col_rows ? limit - col_rows : 0) / (4u * U * NWARPS);
        if (kg == 0) {   // the host picks wide local bins before the limit gets this small
            if (threadIdx.x == 0) atomicExch(&a.state->kernel_error, 1);
            return;
        }
    }
    uint32_t since = 0;   // groups since the last meeting
#define QG_MEET(grp)                                                                                          \
    if (MODE != 1 && since == kg && (grp) < groups) {                                                         \
        since = 0;                                                                                            \
        __syncthreads();                                                                                      \
        if (!selective || relieve_local<NT, MODE == 1 ? 0 : MODE, LOGW_T, SELECTIVE_T>(hp, td, logW, a.nb, shift, out)) { \
            flush_local<NT, MODE>(hp, td, logW, a.nb, pass, shift, out);                                      \
            __syncthreads();                                                                                  \
        }                                                                                                     \
    }
    if (!LIST) {
        const uint32_t v = first_unit + ((uint32_t)warp << logR) + slot;      // first unit of this lane
        const uint32_t row0 = ((v >> 2) << 4) + (v & 3u);
        const uint32_t *pw = tile + ((size_t)row0 << logW) + wa;
        const uint2 *pc = reinterpret_cast<const uint2 *>(a.codes) + v;
        const uint32_t jstride = 4u << logW;                                  // words between rows 4 apart
        constexpr uint32_t QW = NWARPS * 128;                                 // words per round of the CTA's warps
        const uint32_t qc = (uint32_t)NWARPS << logR;                         // units per round of the CTA's warps
        uint32_t w[U][4];
        uint2 c[U];
#define QG_LOAD_UNIT(u)                                                                  \
    {                                                                                    \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) w[u][j] = ldg32(pw + (u) * QW + j * jstride); \
        c[u] = ldg64(pc + (u) * qc);                                                     \
    }
#define QG_USE_UNIT(u)                                       \
    {                                                        \
        add_word<MODE>(base, w[u][0], c[u].x, 0, pass, shift);      \
        add_word<MODE>(base, w[u][1], c[u].x, 1, pass, shift);      \
        add_word<MODE>(base, w[u][2], c[u].y, 0, pass, shift);      \
        add_word<MODE>(base, w[u][3], c[u].y, 1, pass, shift);      \
    }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if ((uint32_t)u < nq) QG_LOAD_UNIT(u)
        pw += U * QW;
        pc += U * qc;
        uint32_t i = 0, grp = 0;
        while (grp < groups) {
            // groups that can run without a test: units in registers and the next U exist, until the next meeting
            uint32_t run = i + 2 * U <= nq ? (nq - i - 2 * U) / U + 1 : 0;
            run = run < kg - since ? run : kg - since;
            if (run) {
                for (uint32_t r = 0; r < run; ++r) {
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        QG_USE_UNIT(u)
                        QG_LOAD_UNIT(u)
                    }
                    pw += U * QW;
                    pc += U * qc;
                }
            } else {
                run = 1;
                if (i < nq) {
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (i + u < nq) {
                            QG_USE_UNIT(u)
                            if (i + u + U < nq) QG_LOAD_UNIT(u)
                        }
                    }
                }
                pw += U * QW;
                pc += U * qc;
            }
            i += run * U;
            grp += run;
            since += run;
            QG_MEET(grp)
        }
#undef QG_LOAD_UNIT
#undef QG_USE_UNIT
    } else {
        // entry of (warp-unit wu, j): off + (4 wu << logR) + (j << logR) + slot
        const size_t e0 = a.off + ((size_t)(first_q + warp) << (logR + 2)) + slot;
        const uint32_t *pr = LIST == 2 ? nullptr : a.rows + e0;
        const uint2 *pe = LIST == 2 ? a.ents + e0 : nullptr;
        const uint32_t qs = (uint32_t)(4 * NWARPS) << logR;                   // entries per round of the CTA's warps
        const uint32_t *tw = tile + wa;
        uint32_t idx[U][4], w[U][4], c[U][4];
        uint32_t cn[LIST == 2 ? U : 1][4];   // codes that came with the indices (pair entries)
#define QG_LOAD_IDX(u)                                                                \
    {                                                                                 \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) {                               \
            if (LIST == 2) {                                                          \
                const uint2 e = __ldcg(pe + (u) * qs + ((uint32_t)j << logR));        \
                idx[u][j] = e.x;                                                      \
                cn[LIST == 2 ? (u) : 0][j] = e.y;                                     \
            } else {                                                                  \
                idx[u][j] = pr[(u) * qs + ((uint32_t)j << logR)];                     \
            }                                                                         \
        }                                                                             \
    }
#define QG_LOAD_DATA(u)                                                \
    {                                                                  \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) {                \
            w[u][j] = ldg32(tw + ((size_t)idx[u][j] << logW));         \
            if (LIST == 2) c[u][j] = cn[LIST == 2 ? (u) : 0][j];       \
            else c[u][j] = ldg16(a.codes_nat + idx[u][j]);             \
        }                                                              \
    }
#define QG_USE_DATA(u)                                                                           \
    {                                                                                            \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) add_word<MODE>(base, w[u][j], c[u][j], 0, pass, shift); \
    }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if ((uint32_t)u < nq) QG_LOAD_IDX(u)
        if (LIST == 2) pe += U * qs; else pr += U * qs;
#pragma unroll
        for (int u = 0; u < U; ++u)
            if ((uint32_t)u < nq) {
                QG_LOAD_DATA(u)
                if ((uint32_t)u + U < nq) QG_LOAD_IDX(u)
            }
        if (LIST == 2) pe += U * qs; else pr += U * qs;
        uint32_t i = 0;
        for (uint32_t grp = 0; grp < groups; i += U) {
            if (i + 3 * U <= nq) {   // data of units i .. i+U-1 and indices of the next U are in registers, U more exist
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    QG_USE_DATA(u)
                    QG_LOAD_DATA(u)
                    QG_LOAD_IDX(u)
                }
            } else if (i < nq) {
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
            }
            if (LIST == 2) pe += U * qs; else pr += U * qs;
            ++grp;
            ++since;
            QG_MEET(grp)
        }
#undef QG_LOAD_IDX
#undef QG_LOAD_DATA
#undef QG_USE_DATA
    }
#undef QG_MEET
    __syncthreads();
    flush_local<NT, MODE>(hp, td, logW, a.nb, pass, shift, out);
}

}  // namespace
