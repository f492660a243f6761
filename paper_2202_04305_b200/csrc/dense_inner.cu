// SpMV over encodings whose inner level is dense: (compressed, dense) - the paper's "CDR" of
// Section 6.2, the best format for its row-band matrices - and (dense, dense), in either order.
//
// values holds one full inner slice per stored outer index q (explicit zeros included), so the
// loops are dense:  row-major   y[i_q] = sum_k val[q, k] * x[k]        (one dot product per slice)
//                   col-major   y[i]  += val[q, i] * x[k_q]            (one axpy per slice)
// with i_q / k_q = crd[0][q], or q itself when the outer level is dense.
#include "common.cuh"

namespace {

constexpr int kDThreads = 256;
constexpr int kDUnroll = 8;

// One group of TPR threads per stored slice: strided dot product with kDUnroll loads in flight.
template <typename I, int TPR>
__global__ void __launch_bounds__(kDThreads)
k_spmv_dense_rows(const double* __restrict__ val, const I* __restrict__ outer, int64_t nslices, int64_t inner,
                  const double* __restrict__ x, double* __restrict__ y) {
    __shared__ double s_part[kDThreads / 32];
    constexpr int kGroups = kDThreads / TPR;
    const int g = threadIdx.x / TPR, tl = threadIdx.x % TPR;
    for (int64_t q = (int64_t)blockIdx.x * kGroups + g; q < nslices; q += (int64_t)gridDim.x * kGroups) {
        const double* row = val + q * inner;
        double s = 0.0;
        int64_t k = tl;
        if (TPR == kDThreads && (inner & 1) == 0 && (reinterpret_cast<uintptr_t>(row) & 15) == 0 &&
            (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
            // long, aligned slices: 16-byte loads, kDUnroll of them in flight per thread
            const double2* row2 = reinterpret_cast<const double2*>(row);
            const double2* x2 = reinterpret_cast<const double2*>(x);
            const int64_t half = inner >> 1;
            int64_t h = tl;
            for (; h + (int64_t)(kDUnroll - 1) * TPR < half; h += (int64_t)kDUnroll * TPR) {
                double2 a[kDUnroll], b[kDUnroll];
#pragma unroll
                for (int u = 0; u < kDUnroll; ++u) { a[u] = __ldcs(row2 + h + u * TPR); b[u] = __ldg(x2 + h + u * TPR); }
#pragma unroll
                for (int u = 0; u < kDUnroll; ++u) { s = fma(a[u].x, b[u].x, s); s = fma(a[u].y, b[u].y, s); }
            }
            for (; h < half; h += TPR) { const double2 a = row2[h], b = __ldg(x2 + h); s = fma(a.x, b.x, s); s = fma(a.y, b.y, s); }
            k = inner;                    // everything consumed
        }
        for (; k + (int64_t)(kDUnroll - 1) * TPR < inner; k += (int64_t)kDUnroll * TPR) {
            double a[kDUnroll], b[kDUnroll];
#pragma unroll
            for (int u = 0; u < kDUnroll; ++u) { a[u] = __ldcs(row + k + u * TPR); b[u] = __ldg(x + k + u * TPR); }
#pragma unroll
            for (int u = 0; u < kDUnroll; ++u) s = fma(a[u], b[u], s);
        }
        for (; k < inner; k += TPR) s = fma(row[k], __ldg(x + k), s);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (TPR == 32) {
            if (tl == 0) y[outer ? (int64_t)outer[q] : q] = s;
        } else {                                  // TPR == kDThreads: the whole block works on slice q
            if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = s;
            __syncthreads();
            if (threadIdx.x == 0) {
                double tot = s_part[0];
#pragma unroll
                for (int i = 1; i < kDThreads / 32; ++i) tot += s_part[i];
                y[outer ? (int64_t)outer[q] : q] = tot;
            }
            __syncthreads();
        }
    }
}

// Column-major: thread = output row i, blockIdx.y = a chunk of stored slices; y was zeroed.
constexpr int kDChunk = 32;
template <typename I>
__global__ void __launch_bounds__(kDThreads)
k_spmv_dense_cols(const double* __restrict__ val, const I* __restrict__ outer, int64_t nslices, int64_t inner,
                  const double* __restrict__ x, double* __restrict__ y) {
    const int64_t i = (int64_t)blockIdx.x * kDThreads + threadIdx.x;
    if (i >= inner) return;
    const int64_t q0 = (int64_t)blockIdx.y * kDChunk;
    const int64_t q1 = q0 + kDChunk < nslices ? q0 + kDChunk : nslices;
    double s = 0.0;
    for (int64_t q = q0; q < q1; ++q) s = fma(__ldcs(val + q * inner + i), __ldg(x + (outer ? (int64_t)outer[q] : q)), s);
    atomicAdd(y + i, s);
}

}  // namespace

// Called by sp_spmv for rank-2 handles whose level 1 is dense.
sp_status sp_spmv_dense_inner(const sp_tensor* A, const double* x, double* y, cudaStream_t stream) {
    const bool rowmajor = A->ord[0] == 0;
    const bool outer_c = A->lt[0] == SP_COMPRESSED;
    const int64_t inner = A->dims[A->ord[1]];
    const int64_t nslices = outer_c ? A->ncrd[0] : A->dims[A->ord[0]];
    const int64_t m = A->dims[0];
    if (!rowmajor || outer_c) SP_CUDA(cudaMemsetAsync(y, 0, (size_t)m * sizeof(double), stream));
    if (nslices == 0 || inner == 0) return SP_OK;
#define SP_DENSE_LAUNCH(I)                                                                                           \
    do {                                                                                                             \
        const I* outer = outer_c ? static_cast<const I*>(A->crd[0]) : nullptr;                                       \
        if (rowmajor) {                                                                                              \
            if (inner >= 1024) {                                                                                     \
                const unsigned blocks = (unsigned)(nslices < 148 * 16 ? nslices : 148 * 16);                         \
                k_spmv_dense_rows<I, kDThreads><<<blocks, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, x, y); \
            } else {                                                                                                 \
                const int64_t need = sp_ceil_div(nslices, kDThreads / 32);                                           \
                const unsigned blocks = (unsigned)(need < 148 * 16 ? need : 148 * 16);                               \
                k_spmv_dense_rows<I, 32><<<blocks, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, x, y);     \
            }                                                                                                        \
        } else {                                                                                                     \
            const int64_t chunks = sp_ceil_div(nslices, kDChunk);                                                    \
            if (chunks > 65535) return SP_ERR_UNSUPPORTED;                                                           \
            dim3 grid((unsigned)sp_ceil_div(inner, kDThreads), (unsigned)chunks);                                    \
            k_spmv_dense_cols<I><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, x, y);               \
        }                                                                                                            \
    } while (0)
    if (A->crdBits == 32) SP_DENSE_LAUNCH(uint32_t); else SP_DENSE_LAUNCH(uint64_t);
#undef SP_DENSE_LAUNCH
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    return SP_OK;
}
