// SpMV and SpMM over encodings whose inner level is dense: (compressed, dense) - the paper's "CDR" of
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

// SpMM with a dense inner level: C[i,:] = sum_k A[i,k] * B[k,:] where A's stored slices are dense.
// A block owns kRT output rows and one 32-column tile of C and walks the contraction index in steps of
// kKT: the kRT x kKT tile of A is staged in shared memory (stored [k][row], so a warp reads its four
// row values with one 32-byte broadcast), each warp owns 4 rows, lane = column, and every B row is
// loaded once per warp and used for 4 rows.
//   row-major    : output row = stored slice q (i = crd[0][q]), k = inner index,  A[q,k]  = val[q*inner + k]
//   column-major : output row = inner index i,  k = stored slice q (crd[0][q]),   A[i,q]  = val[q*inner + i]
constexpr int kRT = 32, kKT = 32;

template <typename I, bool ROWMAJOR>
__global__ void __launch_bounds__(kDThreads)
k_spmm_dense_inner(const double* __restrict__ val, const I* __restrict__ outer, int64_t nslices, int64_t inner,
                   const double* __restrict__ B, int64_t N, int64_t ldb, double* __restrict__ C, int64_t ldc,
                   int64_t kchunk) {
    __shared__ double s_a[kKT][kRT + 4];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t nrows = ROWMAJOR ? nslices : inner;     // output rows this kernel produces
    const int64_t nk = ROWMAJOR ? inner : nslices;        // length of the contraction
    const int64_t r0 = (int64_t)blockIdx.x * kRT;
    const int64_t col = (int64_t)blockIdx.y * 32 + lane;
    const bool on = col < N;
    const double* Bc = B + (on ? col : (int64_t)blockIdx.y * 32);
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    // blockIdx.z owns the contraction range [kbeg, kend); with more than one range the partial
    // products are added into C (zeroed by the caller) with atomics
    const int64_t kbeg = (int64_t)blockIdx.z * kchunk;
    const int64_t kend = kbeg + kchunk < nk ? kbeg + kchunk : nk;
    for (int64_t k0 = kbeg; k0 < kend; k0 += kKT) {
        __syncthreads();
        // stage A[r0 .. r0+kRT) x [k0 .. k0+kKT), zero outside
        for (int e = threadIdx.x; e < kRT * kKT; e += kDThreads) {
            // the fast index of the load follows the contiguous index of val
            const int rr = ROWMAJOR ? e / kKT : e % kRT;
            const int kk = ROWMAJOR ? e % kKT : e / kRT;
            const int64_t r = r0 + rr, k = k0 + kk;
            double a = 0.0;
            if (r < nrows && k < kend) a = ROWMAJOR ? __ldcs(val + r * inner + k) : __ldcs(val + k * inner + r);
            s_a[kk][rr] = a;
        }
        __syncthreads();
        const int kmax = (int)(kend - k0 < kKT ? kend - k0 : kKT);
        double b[kKT / 4];
        for (int kb = 0; kb < kmax; kb += kKT / 4) {      // 8 B rows in flight per warp
#pragma unroll
            for (int u = 0; u < kKT / 4; ++u) {
                const int64_t k = k0 + kb + u;
                const int64_t krow = k < nk ? (ROWMAJOR ? k : (outer ? (int64_t)outer[k] : k)) : 0;
                b[u] = __ldg(Bc + krow * ldb);
            }
#pragma unroll
            for (int u = 0; u < kKT / 4; ++u) {
                if (kb + u < kmax) {
#pragma unroll
                    for (int r = 0; r < 4; ++r) acc[r] = fma(s_a[kb + u][4 * w + r], b[u], acc[r]);
                }
            }
        }
    }
    if (on) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int64_t row = r0 + 4 * w + r;
            if (row < nrows) {
                double* dst = C + (ROWMAJOR ? (outer ? (int64_t)outer[row] : row) : row) * ldc + col;
                if (gridDim.z > 1) atomicAdd(dst, acc[r]); else *dst = acc[r];
            }
        }
    }
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

// Called by sp_spmm for rank-2 handles whose level 1 is dense.
sp_status sp_spmm_dense_inner(const sp_tensor* A, const double* B, int64_t N, int64_t ldb, double* C, int64_t ldc,
                              cudaStream_t stream) {
    const bool rowmajor = A->ord[0] == 0;
    const bool outer_c = A->lt[0] == SP_COMPRESSED;
    const int64_t inner = A->dims[A->ord[1]];
    const int64_t nslices = outer_c ? A->ncrd[0] : A->dims[A->ord[0]];
    const int64_t m = A->dims[0];
    if (nslices == 0 || inner == 0) {                  // nothing stored: the product is zero
        if (ldc == N) SP_CUDA(cudaMemsetAsync(C, 0, (size_t)m * N * sizeof(double), stream));
        else SP_CUDA(cudaMemset2DAsync(C, (size_t)ldc * sizeof(double), 0, (size_t)N * sizeof(double), (size_t)m, stream));
        return SP_OK;
    }
    const int64_t nrows = rowmajor ? nslices : inner;
    const int64_t nk = rowmajor ? inner : nslices;
    const int64_t rb = sp_ceil_div(nrows, kRT), cb = sp_ceil_div(N, 32);
    // few row blocks and a long contraction (a row band): split the contraction so every SM has work
    int64_t ksplit = 1;
    if (rb * cb < 4 * 148) {
        ksplit = sp_ceil_div(4 * 148, rb * cb);
        const int64_t most = sp_ceil_div(nk, 8 * kKT);
        if (ksplit > most) ksplit = most;
        if (ksplit > 65535) ksplit = 65535;
        if (ksplit < 1) ksplit = 1;
    }
    const int64_t kchunk = sp_ceil_div(sp_ceil_div(nk, ksplit), kKT) * kKT;
    ksplit = sp_ceil_div(nk, kchunk);
    if ((rowmajor && outer_c) || ksplit > 1) {          // rows not stored are zero; split sums start at zero
        if (ldc == N) SP_CUDA(cudaMemsetAsync(C, 0, (size_t)m * N * sizeof(double), stream));
        else SP_CUDA(cudaMemset2DAsync(C, (size_t)ldc * sizeof(double), 0, (size_t)N * sizeof(double), (size_t)m, stream));
    }
    if (cb > 65535) return SP_ERR_UNSUPPORTED;
    dim3 grid((unsigned)rb, (unsigned)cb, (unsigned)(ksplit > 0 ? ksplit : 1));
#define SP_DENSE_MM(I)                                                                                                  \
    do {                                                                                                                \
        const I* outer = outer_c ? static_cast<const I*>(A->crd[0]) : nullptr;                                          \
        if (rowmajor) k_spmm_dense_inner<I, true><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, B, N, ldb, C, ldc, kchunk); \
        else k_spmm_dense_inner<I, false><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, B, N, ldb, C, ldc, kchunk);       \
    } while (0)
    if (A->crdBits == 32) SP_DENSE_MM(uint32_t); else SP_DENSE_MM(uint64_t);
#undef SP_DENSE_MM
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    return SP_OK;
}
