// Measurement probes for the secondary bounds of the gather kernels (no counterpart in the paper).
//
// SpMM, SDDMM and MTTKRP fetch one dense row per stored entry (Sections 6.2, 6.3: the inner loop
// over the dense dimension), so next to the HBM bound on their compulsory bytes they are bounded
// by how fast an SM can pull randomly chosen rows of a table that sits in L2 (or L1), and by the
// f64 multiply-add rate.  These two kernels measure those rates on the device at hand; the caller
// times them with events on the stream it passes.
#include "common.cuh"

namespace {

constexpr int kPThreads = 256;
constexpr int kInFlight = 8;   // independent row fetches a lane group issues before using any

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// A group of LPR lanes fetches whole rows of `row_elems` doubles (16 bytes per lane per load,
// NL loads per lane per row) at uniformly random row numbers.
template <int LPR, int NL>
__global__ void __launch_bounds__(kPThreads)
k_probe_gather(const double* __restrict__ table, uint32_t rows, int64_t per_group, uint64_t seed,
               double* __restrict__ sink) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t group = t / LPR;
    const int hl = (int)(t % LPR);
    constexpr int row_elems = LPR * 2 * NL;
    double acc0 = 0.0, acc1 = 0.0;
    for (int64_t it = 0; it < per_group; it += kInFlight) {
        double2 v[kInFlight][NL];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const uint32_t r = (uint32_t)(mix64(seed + (uint64_t)(group * per_group + it + u) * 0x9E3779B97F4A7C15ull) % rows);
            const double* p = table + (int64_t)r * row_elems + 2 * hl;
#pragma unroll
            for (int n = 0; n < NL; ++n) v[u][n] = *reinterpret_cast<const double2*>(p + n * 2 * LPR);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u)
#pragma unroll
            for (int n = 0; n < NL; ++n) { acc0 += v[u][n].x; acc1 += v[u][n].y; }
    }
    sink[t] = acc0 + acc1;
}

// Every lane fetches single 8-byte elements at uniformly random positions (what SpMV does with x).
__global__ void __launch_bounds__(kPThreads)
k_probe_gather_elems(const double* __restrict__ table, uint32_t n, int64_t per_lane, uint64_t seed,
                     double* __restrict__ sink) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    double acc = 0.0;
    for (int64_t it = 0; it < per_lane; it += kInFlight) {
        double v[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u)
            v[u] = table[mix64(seed + (uint64_t)(t * per_lane + it + u) * 0x9E3779B97F4A7C15ull) % n];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) acc += v[u];
    }
    sink[t] = acc;
}

constexpr int kChains = 8;

__global__ void __launch_bounds__(kPThreads)
k_probe_dfma(int64_t iters, double a, double b, double* __restrict__ sink) {
    double x[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) x[c] = (double)(threadIdx.x + c);
    for (int64_t i = 0; i < iters; ++i)
#pragma unroll
        for (int c = 0; c < kChains; ++c) x[c] = fma(x[c], a, b);
    double s = 0.0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += x[c];
    sink[blockIdx.x * (int64_t)blockDim.x + threadIdx.x] = s;
}

}  // namespace

extern "C" sp_status sp_probe_gather(const double* table, int64_t rows, int64_t row_elems, int64_t blocks,
                                     int64_t rows_per_group, uint64_t seed, double* sink, int64_t* fetched,
                                     void* stream_) {
    if (!table || !sink || rows < 1 || rows > 0xffffffffll || blocks < 1 || blocks > 0x7fffffff || rows_per_group < 1)
        return SP_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(table) % 16) return SP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t per = sp_ceil_div(rows_per_group, kInFlight) * kInFlight;
    int lpr = 0;
    if (row_elems == 1) {      // single elements: one fetch per lane
        k_probe_gather_elems<<<(unsigned)blocks, kPThreads, 0, stream>>>(table, (uint32_t)rows, per, seed, sink);
        SP_LAUNCH_CHECK();
        sp_count_launches(1);
        if (fetched) *fetched = blocks * kPThreads * per;
        return SP_OK;
    }
    switch (row_elems) {
#define SP_PROBE_CASE(E, LPR, NL)                                                                              \
    case E:                                                                                                    \
        lpr = LPR;                                                                                             \
        k_probe_gather<LPR, NL><<<(unsigned)blocks, kPThreads, 0, stream>>>(table, (uint32_t)rows, per, seed, sink); \
        break;
        SP_PROBE_CASE(16, 8, 1)     // 128-byte rows
        SP_PROBE_CASE(32, 8, 2)     // 256-byte rows (MTTKRP, R = 32; SpMM, N = 32)
        SP_PROBE_CASE(64, 16, 2)    // 512-byte rows (SpMM, N = 64)
        SP_PROBE_CASE(128, 32, 2)   // 1-KiB rows (SDDMM, K = 128)
#undef SP_PROBE_CASE
        default: return SP_ERR_UNSUPPORTED;
    }
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    if (fetched) *fetched = blocks * kPThreads / lpr * per;
    return SP_OK;
}

extern "C" sp_status sp_probe_dfma(int64_t blocks, int64_t iters, double* sink, int64_t* fmas, void* stream_) {
    if (!sink || blocks < 1 || blocks > 0x7fffffff || iters < 1) return SP_ERR_INVALID_ARG;
    k_probe_dfma<<<(unsigned)blocks, kPThreads, 0, static_cast<cudaStream_t>(stream_)>>>(iters, 0.999999, 1e-9, sink);
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    if (fmas) *fmas = blocks * kPThreads * kChains * iters;
    return SP_OK;
}
