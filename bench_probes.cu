// Measurement aids of bench.py (see bench_probes.h).  Built into libbench_probes.so together with
// a second compilation of the product's packer (csrc/pack.cu with SP_BENCH_BUILD), never into
// the product library.
#include "bench_probes.h"

#include <cuda_runtime.h>

namespace {

constexpr int kThreads = 256;
constexpr int kInFlight = 8;   // independent row fetches a lane group issues before using any

// A group of LPR lanes fetches whole rows of LPR * 2 * NL doubles (16 bytes per lane per load, NL
// loads per lane per row).  The warp owns per_warp consecutive row numbers; it reads 32 of them
// with one coalesced load (the next 32 are requested before the current ones are used), and group
// g takes numbers g, g + G, g + 2G, ... of the batch by shuffle, 8 rows at a time.
template <int LPR, int NL>
__global__ void __launch_bounds__(kThreads)
k_gather_rows(const double* __restrict__ table, const uint32_t* __restrict__ ids, int64_t per_warp,
              double* __restrict__ sink) {
    constexpr int G = 32 / LPR;
    constexpr int row_elems = LPR * 2 * NL;
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31, g = lane / LPR, hl = lane % LPR;
    const uint32_t* my = ids + (t >> 5) * per_warp;
    double acc0 = 0.0, acc1 = 0.0;
    uint32_t id_n = my[lane];
    for (int64_t base = 0; base < per_warp; base += 32) {
        const uint32_t id = id_n;
        if (base + 32 < per_warp) id_n = my[base + 32 + lane];
#pragma unroll
        for (int u0 = 0; u0 < LPR; u0 += kInFlight) {
            double2 v[kInFlight][NL];
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const uint32_t r = __shfl_sync(0xffffffffu, id, (u0 + u) * G + g);
                const double* p = table + (size_t)r * row_elems + 2 * hl;
#pragma unroll
                for (int n = 0; n < NL; ++n) v[u][n] = *reinterpret_cast<const double2*>(p + n * 2 * LPR);
            }
#pragma unroll
            for (int u = 0; u < kInFlight; ++u)
#pragma unroll
                for (int n = 0; n < NL; ++n) { acc0 += v[u][n].x; acc1 += v[u][n].y; }
        }
    }
    sink[t] = acc0 + acc1;
}

// Every lane fetches single 8-byte elements (what SpMV does with x), 8 in flight.
__global__ void __launch_bounds__(kThreads)
k_gather_elems(const double* __restrict__ table, const uint32_t* __restrict__ ids, int64_t per_warp,
               double* __restrict__ sink) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    const uint32_t* my = ids + (t >> 5) * per_warp;
    double acc = 0.0;
    for (int64_t base = 0; base < per_warp; base += 32 * kInFlight) {
        uint32_t id[kInFlight];
        double v[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) id[u] = my[base + u * 32 + lane];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) v[u] = table[id[u]];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) acc += v[u];
    }
    sink[t] = acc;
}

constexpr int kChains = 8;

__global__ void __launch_bounds__(kThreads)
k_dfma(int64_t iters, double a, double b, double* __restrict__ sink) {
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

extern "C" int spb_gather_rows(const double* table, int64_t rows, int64_t row_elems, const uint32_t* row_ids,
                               int64_t n_ids, int64_t blocks, double* sink, void* stream_) {
    if (!table || !row_ids || !sink || rows < 1 || rows > 0xffffffffll || blocks < 1 || blocks > 0x7fffffff)
        return SP_ERR_INVALID_ARG;
    const int64_t warps = blocks * (kThreads / 32);
    if (n_ids < 1 || n_ids % (warps * 32 * kInFlight) != 0) return SP_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(table) % 16) return SP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t per_warp = n_ids / warps;
    switch (row_elems) {
        case 1: k_gather_elems<<<(unsigned)blocks, kThreads, 0, stream>>>(table, row_ids, per_warp, sink); break;
        case 16: k_gather_rows<8, 1><<<(unsigned)blocks, kThreads, 0, stream>>>(table, row_ids, per_warp, sink); break;    // 128 B
        case 32: k_gather_rows<8, 2><<<(unsigned)blocks, kThreads, 0, stream>>>(table, row_ids, per_warp, sink); break;    // 256 B
        case 64: k_gather_rows<16, 2><<<(unsigned)blocks, kThreads, 0, stream>>>(table, row_ids, per_warp, sink); break;   // 512 B
        case 128: k_gather_rows<32, 2><<<(unsigned)blocks, kThreads, 0, stream>>>(table, row_ids, per_warp, sink); break;  // 1 KiB
        default: return SP_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? SP_OK : SP_ERR_CUDA;
}

extern "C" int spb_dfma(int64_t blocks, int64_t iters, double* sink, void* stream_) {
    if (!sink || blocks < 1 || blocks > 0x7fffffff || iters < 1) return SP_ERR_INVALID_ARG;
    k_dfma<<<(unsigned)blocks, kThreads, 0, static_cast<cudaStream_t>(stream_)>>>(iters, 0.999999, 1e-9, sink);
    return cudaGetLastError() == cudaSuccess ? SP_OK : SP_ERR_CUDA;
}
