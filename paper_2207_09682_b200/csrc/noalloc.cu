// Histogram build for callers that may not allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a memory pool that
// owns the whole device, in a latency-critical loop where an allocation would synchronise the
// device, or in a plug-in whose host forbids allocator calls.  qgbdt_build_histograms needs a
// context, and a context allocates (tiled copy of the bin matrix, partial-histogram scratch).
// The entry point below needs neither: it reads the caller's own arrays and keeps the one
// piece of scratch it needs -- the per-CTA partial histograms of the two-stage merge -- in a
// fixed array that is part of the library image.  Every GPU that loads the library carries
// that array (NOALLOC_SLOTS * NOALLOC_MAX_BINS * 8 bytes = 4 MiB) until the process exits.
//
// It is a plain kernel (global atomics into the CTA's own slot, then a sum over the slots), not
// the tuned shared-memory kernel of hist.cu: it trades speed for having no state.
#include <mutex>

#include "qgbdt_internal.cuh"

namespace {

constexpr int NOALLOC_SLOTS = 32;            // CTAs of the first stage, one partial histogram each
constexpr int NOALLOC_MAX_BINS = 16384;      // n_features * n_bins may not exceed this
constexpr int NOALLOC_MAX_DEVICES = 64;
constexpr long long NOALLOC_MAX_ENTRIES = 4294967295ll / 255;   // 16 843 009: n * 255 still fits the unsigned hessian field

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; the
// address a kernel can use is looked up once per device below.
static __device__ __align__(256) unsigned long long g_noalloc_scratch[NOALLOC_SLOTS * NOALLOC_MAX_BINS];

unsigned long long *g_scratch_addr[NOALLOC_MAX_DEVICES];   // per device, filled on first use
std::mutex g_setup_mutex;
thread_local char g_noalloc_err[256] = {0};

int na_fail(int code, const char *msg) {
    snprintf(g_noalloc_err, sizeof(g_noalloc_err), "%s", msg);
    return code;
}

// Stage 1: CTA p clears its slot, then adds the rows of its share with atomics that only its own
// threads contend for.  rows == nullptr: rows 0 .. n-1.
__global__ void __launch_bounds__(256) k_na_partial(const uint8_t *__restrict__ bins, long long ld, int F, int nb,
                                                    const int8_t *__restrict__ gq, const uint8_t *__restrict__ hq,
                                                    const uint32_t *__restrict__ rows, long long n, long long n_rows,
                                                    unsigned long long *__restrict__ scratch, int *__restrict__ bad) {
    unsigned long long *slot = scratch + (size_t)blockIdx.x * NOALLOC_MAX_BINS;
    const int total = F * nb;
    for (int i = threadIdx.x; i < total; i += blockDim.x) slot[i] = 0ull;   // the array keeps the last call's sums
    __syncthreads();
    const long long e0 = n * blockIdx.x / gridDim.x, e1 = n * (blockIdx.x + 1) / gridDim.x;
    const long long work = (e1 - e0) * F;
    for (long long t = threadIdx.x; t < work; t += blockDim.x) {
        const long long e = e0 + t / F;
        const int f = (int)(t % F);
        const long long row = rows ? (long long)rows[e] : e;
        if (row >= n_rows) { if (bad) *bad = 1; continue; }
        const int bin = bins[row * ld + f];
        if (bin >= nb) { if (bad) *bad = 1; continue; }
        if (gq[row] == -128) { if (bad) *bad = 1; continue; }   // outside every level range (|g| <= 127); the overflow bound assumes it
        const long long packed = (long long)gq[row] * 4294967296LL + (long long)hq[row];
        atomicAdd(&slot[(size_t)f * nb + bin], (unsigned long long)packed);
    }
}

// Stage 2: the histogram is the sum of the slots (packed 32+32 words add up as they are).
__global__ void __launch_bounds__(256) k_na_reduce(const unsigned long long *__restrict__ scratch, int slots, int total,
                                                   unsigned long long *__restrict__ hist) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        unsigned long long s = 0;
        for (int p = 0; p < slots; ++p) s += scratch[(size_t)p * NOALLOC_MAX_BINS + i];
        hist[i] = s;
    }
}

}  // namespace

extern "C" {

const char *qgbdt_noalloc_last_error(void) { return g_noalloc_err; }

int qgbdt_build_histograms_noalloc(const uint8_t *d_bins, int64_t n_rows, int32_t n_features, int32_t n_bins,
                                   int64_t ld, const int8_t *d_gq, const uint8_t *d_hq, const uint32_t *d_rows,
                                   int64_t n, qgbdt_bin *d_hist, int32_t *d_status, void *stream) {
    if (!d_bins || !d_gq || !d_hq || !d_hist) return na_fail(QGBDT_ERR_ARG, "null pointer");
    if (n_rows < 1 || n_rows >= (1ll << 31) || n_features < 1 || n_bins < 2 || n_bins > 256 || ld < n_features)
        return na_fail(QGBDT_ERR_ARG, "n_rows, n_features, n_bins or ld out of range");
    if (n < 0 || (d_rows == nullptr && n != n_rows)) return na_fail(QGBDT_ERR_ARG, "n must be n_rows when d_rows is NULL");
    if ((int64_t)n_features * n_bins > NOALLOC_MAX_BINS) {
        snprintf(g_noalloc_err, sizeof(g_noalloc_err),
                 "n_features * n_bins = %lld exceeds the fixed scratch of %d bins; use a context (qgbdt_build_histograms)",
                 (long long)n_features * n_bins, NOALLOC_MAX_BINS);
        return QGBDT_ERR_ARG;
    }
    // the caller's codes may be anything in [-127, 127] x [0, 255]: n entries can reach n * 255 in a hessian field
    if (n > NOALLOC_MAX_ENTRIES)
        return na_fail(QGBDT_ERR_OVERFLOW, "more than 16843009 entries: the sums could exceed the 32+32-bit histogram word");
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) {
        cudaGetLastError();
        return na_fail(QGBDT_ERR_CUDA, "no usable current CUDA device");
    }
    // Set-up, once per device, with that device current: the device address of the scratch array.
    unsigned long long *scratch;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_scratch_addr[dev]) {
            void *p = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (e != cudaSuccess || !p) {
                cudaGetLastError();
                snprintf(g_noalloc_err, sizeof(g_noalloc_err), "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
                return QGBDT_ERR_CUDA;
            }
            g_scratch_addr[dev] = reinterpret_cast<unsigned long long *>(p);
        }
        scratch = g_scratch_addr[dev];
    }
    cudaStream_t st = (cudaStream_t)stream;
    const int total = n_features * n_bins;
    long long want = (n * n_features + 65535) / 65536;
    const int slots = (int)(want < 1 ? 1 : (want > NOALLOC_SLOTS ? NOALLOC_SLOTS : want));
    k_na_partial<<<slots, 256, 0, st>>>(d_bins, ld, n_features, n_bins, d_gq, d_hq, d_rows, n, n_rows, scratch, d_status);
    k_na_reduce<<<(total + 255) / 256, 256, 0, st>>>(scratch, slots, total, reinterpret_cast<unsigned long long *>(d_hist));
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(g_noalloc_err, sizeof(g_noalloc_err), "kernel launch failed: %s", cudaGetErrorString(e));
        return QGBDT_ERR_CUDA;
    }
    return QGBDT_OK;
}

}  // extern "C"
