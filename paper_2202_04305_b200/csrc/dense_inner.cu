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

// SpMM with a dense inner level: C[i,:] = sum_k A[i,k] * B[k,:] where A's stored slices are dense,
// i.e. a plain f64 contraction - the one place on this path where tensor cores apply.  A block owns
// a kRT x kCT tile of C and walks the contraction index in steps of kKT; each of its 8 warps owns
// 32 rows x 32 columns as 4 x 4 tiles of the 8 x 8 x 4 f64 matrix instruction.  The kRT x kKT tile
// of A (stored [k][row]) and the kKT x kCT tile of B sit in shared memory, double buffered: the
// next tiles are fetched into registers before the current ones are used and written to the other
// buffer afterwards, so one barrier per step suffices.  Operand fragments are one double per lane
// (A: row lane/4, k lane%4; B: k lane%4, column lane/4), read with 8-byte shared loads; the row
// strides are chosen so that the four k of a fragment fall on distinct banks.
//   row-major    : output row = stored slice q (i = crd[0][q]), k = inner index,  A[q,k]  = val[q*inner + k]
//   column-major : output row = inner index i,  k = stored slice q (crd[0][q]),   A[i,q]  = val[q*inner + i]
constexpr int kRT = 256, kKT = 8, kCT = 32;
constexpr int kAStride = kRT + 4;               // doubles per k-row of the A tile: 520 words = 8 (mod 32 banks)
constexpr int kBStride = kCT + 4;               // ... of the B tile: 72 words = 8 (mod 32)
static_assert(kDThreads == kRT && kDThreads == kKT * kCT && kRT == 32 * (kDThreads / 32) && kCT == 32, "tile/thread layout");

__device__ __forceinline__ void dmma_8x8x4(double& c0, double& c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

template <typename I, bool ROWMAJOR>
__global__ void __launch_bounds__(kDThreads, 2)
k_spmm_dense_inner(const double* __restrict__ val, const I* __restrict__ outer, int64_t nslices, int64_t inner,
                   const double* __restrict__ B, int64_t N, int64_t ldb, double* __restrict__ C, int64_t ldc,
                   int64_t kchunk, int vec_a) {
    __shared__ __align__(16) double s_a[2][kKT][kAStride];
    __shared__ __align__(16) double s_b[2][kKT][kBStride];
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int64_t nrows = ROWMAJOR ? nslices : inner;     // output rows this kernel produces
    const int64_t nk = ROWMAJOR ? inner : nslices;        // length of the contraction
    const int64_t r0 = (int64_t)blockIdx.x * kRT, c0 = (int64_t)blockIdx.y * kCT;
    // blockIdx.z owns the contraction range [kbeg, kend); with more than one range the partial
    // products are added into C (zeroed by the caller) with atomics
    const int64_t kbeg = (int64_t)blockIdx.z * kchunk;
    const int64_t kend = kbeg + kchunk < nk ? kbeg + kchunk : nk;

    // Loader roles.  Row-major with 16-byte aligned rows: four lanes cover the kKT values (64 bytes)
    // of one row, a warp instruction covers 8 rows, a thread fetches a k-pair of 4 rows.
    // Otherwise thread t fetches the kKT values of tile row t one by one (column-major: coalesced
    // along the rows).  Every thread also fetches one element of the B tile.
    double a_reg[kKT], b_reg;
    const bool quad = ROWMAJOR && vec_a;
    const int bk = t / kCT, bc = t % kCT;
    auto load_tile = [&](int64_t k0) {
        if (quad && k0 + kKT <= kend) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t r = r0 + w * 32 + j * 8 + (lane >> 2);
                double2 v = make_double2(0.0, 0.0);
                if (r < nrows) v = __ldcs(reinterpret_cast<const double2*>(val + r * inner + k0) + (lane & 3));
                a_reg[2 * j] = v.x; a_reg[2 * j + 1] = v.y;
            }
        } else if (quad) {                                     // ragged last step of the range
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t r = r0 + w * 32 + j * 8 + (lane >> 2), k = k0 + 2 * (lane & 3);
                a_reg[2 * j] = (r < nrows && k < kend) ? __ldg(val + r * inner + k) : 0.0;
                a_reg[2 * j + 1] = (r < nrows && k + 1 < kend) ? __ldg(val + r * inner + k + 1) : 0.0;
            }
        } else {
            const int64_t lr = r0 + t;
#pragma unroll
            for (int kk = 0; kk < kKT; ++kk) {
                const int64_t k = k0 + kk;
                a_reg[kk] = (lr < nrows && k < kend) ? (ROWMAJOR ? __ldg(val + lr * inner + k) : __ldcs(val + k * inner + lr)) : 0.0;
            }
        }
        const int64_t k = k0 + bk, c = c0 + bc;
        b_reg = 0.0;
        if (k < kend && c < N) b_reg = __ldg(B + (ROWMAJOR ? k : (outer ? (int64_t)outer[k] : k)) * ldb + c);
    };
    auto store_tile = [&](int buf) {
        if (quad) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = w * 32 + j * 8 + (lane >> 2), kk = 2 * (lane & 3);
                s_a[buf][kk][r] = a_reg[2 * j];
                s_a[buf][kk + 1][r] = a_reg[2 * j + 1];
            }
        } else {
#pragma unroll
            for (int kk = 0; kk < kKT; ++kk) s_a[buf][kk][t] = a_reg[kk];
        }
        s_b[buf][bk][bc] = b_reg;
    };

    double acc[4][4][2];                        // [row tile][column tile][the lane's two columns]
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j][0] = 0.0; acc[i][j][1] = 0.0; }

    int buf = 0;
    if (kbeg < kend) {
        load_tile(kbeg);
        store_tile(0);
    }
    __syncthreads();
    const int fk = lane & 3, fr = lane >> 2;    // this lane's k and row/column inside a fragment
    for (int64_t k0 = kbeg; k0 < kend; k0 += kKT) {
        const bool more = k0 + kKT < kend;
        if (more) load_tile(k0 + kKT);
#pragma unroll
        for (int k4 = 0; k4 < kKT; k4 += 4) {
            double a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = s_a[buf][k4 + fk][w * 32 + i * 8 + fr];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = s_b[buf][k4 + fk][j * 8 + fr];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) dmma_8x8x4(acc[i][j][0], acc[i][j][1], a[i], b[j]);
        }
        if (more) store_tile(buf ^ 1);
        __syncthreads();
        buf ^= 1;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t row = r0 + w * 32 + i * 8 + fr;
        if (row >= nrows) continue;
        double* dst = C + (ROWMAJOR ? (outer ? (int64_t)outer[row] : row) : row) * ldc;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t col = c0 + j * 8 + 2 * fk + h;
                if (col < N) {
                    if (gridDim.z > 1) atomicAdd(dst + col, acc[i][j][h]); else dst[col] = acc[i][j][h];
                }
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
    const int64_t rb = sp_ceil_div(nrows, kRT), cb = sp_ceil_div(N, kCT);
    // few row blocks and a long contraction (a row band): split the contraction so every SM has work
    int64_t ksplit = 1;
    if (rb * cb < 2 * 148) {
        ksplit = sp_ceil_div(2 * 148, rb * cb);
        const int64_t most = sp_ceil_div(nk, 16 * kKT);
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
    // 16-byte loads along a stored row need every row to start on a 16-byte boundary
    const int vec_a = (inner % 2 == 0 && reinterpret_cast<uintptr_t>(A->val) % 16 == 0) ? 1 : 0;
#define SP_DENSE_MM(I)                                                                                                  \
    do {                                                                                                                \
        const I* outer = outer_c ? static_cast<const I*>(A->crd[0]) : nullptr;                                          \
        if (rowmajor) k_spmm_dense_inner<I, true><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, B, N, ldb, C, ldc, kchunk, vec_a); \
        else k_spmm_dense_inner<I, false><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, B, N, ldb, C, ldc, kchunk, vec_a);       \
    } while (0)
    if (A->crdBits == 32) SP_DENSE_MM(uint32_t); else SP_DENSE_MM(uint64_t);
#undef SP_DENSE_MM
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    return SP_OK;
}
