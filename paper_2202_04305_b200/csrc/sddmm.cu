// sp_sddmm: X[i,j] = S[i,j] * sum_k A[i,k] * B[k,j] over the stored (i,j) of S
// (Section 6.2), S in any two-dimensional encoding, row- or column-major.
//
// Compressed inner level (CSR, DCSR, CSC, DCSC):
// Loop shape: for each stored row i, for each p in pos[1][q]..pos[1][q+1]:
// j = crd[1][p]; x[p] = S.val[p] * dot(A[i,:], B[:,j]).  B is given K x n row-major,
// so a column is K elements a whole row apart; it is transposed once per call into
// a workspace so each entry reads one contiguous K-vector.  The (row end, entry)
// merge path is cut into equal pieces, one per warp; a warp keeps A[i,:] in
// registers across the entries of a row and reduces each dot product with shuffles.
#include "common.cuh"

namespace {

// Warps share nothing, so blocks are kept small (two warps): 0.328 ms on the 2,000,000-entry sample against
// 0.331 ms with four warps and 0.337 ms with eight.
#ifndef SP_SDDMM_THREADS
#define SP_SDDMM_THREADS 64
#endif
constexpr int kSThreads = SP_SDDMM_THREADS;
constexpr int kSItems = 64;   // merge items per warp

__global__ void __launch_bounds__(256)
k_transpose(const double* __restrict__ B, int64_t ldb, int64_t K, int64_t n, double* __restrict__ Bt, int64_t ldt) {
    __shared__ double tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
    const int64_t j0 = (int64_t)blockIdx.x * 32, k0 = (int64_t)blockIdx.y * 32;
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        int64_t k = k0 + r, j = j0 + tx;
        tile[r][tx] = (k < K && j < n) ? B[k * ldb + j] : 0.0;
    }
    __syncthreads();
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        int64_t j = j0 + r, k = k0 + tx;
        if (j < n && k < K) Bt[j * ldt + k] = tile[tx][r];
    }
}

template <int V>
__device__ __forceinline__ void ld2(const double* p, double* a) {
    if (V == 4) {           // one 32-byte load (p is 32-byte aligned)
        asm volatile("ld.global.nc.v4.f64 {%0,%1,%2,%3}, [%4];"
                     : "=d"(a[0]), "=d"(a[V > 1 ? 1 : 0]), "=d"(a[V > 2 ? 2 : 0]), "=d"(a[V > 3 ? 3 : 0]) : "l"(p));
    } else if (V == 2) { double2 q = *reinterpret_cast<const double2*>(p); a[0] = q.x; a[V - 1] = q.y; }
    else a[0] = *p;
}

// NCH > 0: A[i,:] lives in NCH register chunks of 32*V columns (K <= NCH*32*V).
// NCH == 0: any K, A is re-read (from L1) for every entry.
template <typename P, typename I, int V, int NCH>
__global__ void __launch_bounds__(kSThreads)
k_sddmm(const P* __restrict__ pos, const I* __restrict__ crd, const double* __restrict__ sval,
        const I* __restrict__ outer, const double* __restrict__ A, int64_t lda, const double* __restrict__ Bt,
        int64_t ldt, int64_t K, double* __restrict__ xv, const int64_t* __restrict__ prow,
        const int64_t* __restrict__ pnz, int64_t nchunks, int64_t na, int64_t nb) {
    // na, nb: rows of A and of Bt (used by the bounds-checking debug build only)
    sp_wait_for_previous_kernel();      // the transpose that wrote Bt
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    if (w >= nchunks) return;
    const int lane = threadIdx.x & 31;
    const int64_t i0 = prow[w], j0 = pnz[w], i1 = prow[w + 1], j1 = pnz[w + 1];
    if (j1 == j0) return;

    constexpr int NA = NCH > 0 ? NCH : 1;
    double a[NA][V];
    bool a_ready = false;
    int64_t row = i0, p = j0, rbase = i0, nzbase = j0;
    int64_t E = (rbase + lane < i1) ? (int64_t)pos[rbase + lane + 1] : j1;
    I c_l = (nzbase + lane < j1) ? crd[nzbase + lane] : (I)0;
    double v_l = (nzbase + lane < j1) ? sval[nzbase + lane] : 0.0;
    double res = 0.0;

    while (true) {
        const int64_t rend = row < i1 ? __shfl_sync(0xffffffffu, E, (int)(row - rbase)) : j1;
        const double* arow = nullptr;
        if (p < rend) {
            arow = A + SP_IDX(outer ? (int64_t)outer[row] : row, na) * lda;
            if (NCH > 0 && !a_ready) {
#pragma unroll
                for (int ch = 0; ch < NA; ++ch) {
                    const int64_t kk = (int64_t)ch * 32 * V + lane * V;
#pragma unroll
                    for (int q = 0; q < V; ++q) a[ch][q] = 0.0;
                    if (kk < K) ld2<V>(arow + kk, a[ch]);
                }
                a_ready = true;
            }
        }
        while (p < rend) {
            int off = (int)(p - nzbase);
            if (off == 32) {
                if (nzbase + lane < j1) xv[nzbase + lane] = v_l * res;
                nzbase += 32;
                c_l = (nzbase + lane < j1) ? crd[nzbase + lane] : (I)0;
                v_l = (nzbase + lane < j1) ? sval[nzbase + lane] : 0.0;
                off = 0;
            }
            const int cnt = (int)min(rend - p, (int64_t)(32 - off));
#ifndef SP_SDDMM_BATCH
#define SP_SDDMM_BATCH 2
#endif
            if (NCH > 0) {
                // kB entries at a time: all their operand loads are requested before the first of the
                // (dependent) warp reductions starts; a batch's tail repeats its last entry
                constexpr int kB = SP_SDDMM_BATCH;
                for (int t = 0; t < cnt; t += kB) {
                    double b[kB][NA][V];
#pragma unroll
                    for (int u = 0; u < kB; ++u) {
                        const int tt = t + u < cnt ? t + u : cnt - 1;
                        const int64_t j = SP_IDX(__shfl_sync(0xffffffffu, c_l, off + tt), nb);
                        const double* brow = Bt + j * ldt;
#pragma unroll
                        for (int ch = 0; ch < NA; ++ch) {
                            const int64_t kk = (int64_t)ch * 32 * V + lane * V;
#pragma unroll
                            for (int q = 0; q < V; ++q) b[u][ch][q] = 0.0;
                            if (kk < K) ld2<V>(brow + kk, b[u][ch]);
                        }
                    }
                    double part[kB];
#pragma unroll
                    for (int u = 0; u < kB; ++u) {
                        part[u] = 0.0;
#pragma unroll
                        for (int ch = 0; ch < NA; ++ch)
#pragma unroll
                            for (int q = 0; q < V; ++q) part[u] = fma(a[ch][q], b[u][ch][q], part[u]);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                        for (int u = 0; u < kB; ++u) part[u] += __shfl_xor_sync(0xffffffffu, part[u], o);
#pragma unroll
                    for (int u = 0; u < kB; ++u)
                        if (t + u < cnt && lane == off + t + u) res = part[u];
                }
            } else {
                for (int t = 0; t < cnt; ++t) {
                    const int64_t j = SP_IDX(__shfl_sync(0xffffffffu, c_l, off + t), nb);
                    const double* brow = Bt + j * ldt;
                    double part = 0.0;
                    for (int64_t kk = (int64_t)lane * V; kk < K; kk += 32 * V) {
                        double b[V], aa[V];
                        ld2<V>(brow + kk, b);
                        ld2<V>(arow + kk, aa);
#pragma unroll
                        for (int q = 0; q < V; ++q) part = fma(aa[q], b[q], part);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                    if (lane == off + t) res = part;
                }
            }
            p += cnt;
        }
        if (row >= i1) break;
        ++row;
        a_ready = false;
        if (row - rbase == 32) {
            rbase += 32;
            E = (rbase + lane < i1) ? (int64_t)pos[rbase + lane + 1] : j1;
        }
    }
    if (nzbase + lane < j1) xv[nzbase + lane] = v_l * res;
}

// S with a dense inner level ((dense|compressed, dense), either ordering): every cell of a stored
// outer index is a stored value, so x[q * ninner + c] = S.val[..] * sum_k Out[o,k] * In[k,c] with
// o the outer coordinate of stored row q.  One thread per inner coordinate c (loads of In[k, c..]
// coalesce, Out[o,k] is a broadcast), kDQ stored outer rows per block share each load of In.
constexpr int kDQ = 4;

template <typename I>
__global__ void __launch_bounds__(256)
k_sddmm_dense_inner(const I* __restrict__ outer, int64_t nouter, int64_t ninner, const double* __restrict__ sval,
                    const double* __restrict__ Out, int64_t out_row_stride, int64_t out_k_stride,
                    const double* __restrict__ In, int64_t ldin, int64_t K, double* __restrict__ xv, int64_t nouter_dim) {
    const int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    for (int64_t q0 = (int64_t)blockIdx.y * kDQ; q0 < nouter; q0 += (int64_t)gridDim.y * kDQ) {
        const double* orow[kDQ];
        double acc[kDQ];
#pragma unroll
        for (int r = 0; r < kDQ; ++r) {
            const int64_t q = q0 + r < nouter ? q0 + r : nouter - 1;
            orow[r] = Out + SP_IDX(outer ? (int64_t)outer[q] : q, nouter_dim) * out_row_stride;
            acc[r] = 0.0;
        }
        if (c < ninner) {
            for (int64_t k = 0; k < K; ++k) {
                const double b = In[k * ldin + c];
#pragma unroll
                for (int r = 0; r < kDQ; ++r) acc[r] = fma(orow[r][k * out_k_stride], b, acc[r]);
            }
#pragma unroll
            for (int r = 0; r < kDQ; ++r) {
                const int64_t p = (q0 + r) * ninner + c;
                if (q0 + r < nouter) xv[p] = sval[p] * acc[r];
            }
        }
    }
}

sp_status sddmm_dense_inner(sp_tensor* S, const double* A, int64_t lda, const double* B, int64_t ldb, int64_t K,
                            double* x_vals, cudaStream_t stream) {
    if (S->nval == 0) return SP_OK;
    if (!x_vals) return SP_ERR_INVALID_ARG;
    const bool colmajor = S->ord[0] == 1;
    const bool dbl = S->lt[0] == SP_COMPRESSED;
    const int64_t ninner = S->dims[S->ord[1]];
    const int64_t nouter = dbl ? S->ncrd[0] : S->dims[S->ord[0]];
    if (nouter == 0 || ninner == 0) return SP_OK;
    sp_workspace ws(stream);
    const double *Out = A, *In = B;
    int64_t out_row = lda, out_k = 1, ldin = ldb;
    if (colmajor) {
        // outer = column j: Out[j,k] = B[k,j]; inner = row i: In[k,i] = A[i,k], transposed once so that
        // neighbouring threads read neighbouring addresses
        const int64_t m = S->dims[0];
        double* At = ws.get<double>((size_t)K * m);
        if (ws.failed) return SP_ERR_ALLOC;
        dim3 tg((unsigned)sp_ceil_div(K, 32), (unsigned)sp_ceil_div(m, 32));
        k_transpose<<<tg, 256, 0, stream>>>(A, lda, m, K, At, m);
        SP_LAUNCH_CHECK();
        sp_count_launches(1);
        Out = B; out_row = 1; out_k = ldb;
        In = At; ldin = m;
    }
    dim3 grid((unsigned)sp_ceil_div(ninner, 256), (unsigned)std::min<int64_t>(sp_ceil_div(nouter, kDQ), 32768));
    if (S->crdBits == 32)
        k_sddmm_dense_inner<uint32_t><<<grid, 256, 0, stream>>>(dbl ? static_cast<const uint32_t*>(S->crd[0]) : nullptr, nouter,
                                                               ninner, S->val, Out, out_row, out_k, In, ldin, K, x_vals, S->dims[S->ord[0]]);
    else
        k_sddmm_dense_inner<uint64_t><<<grid, 256, 0, stream>>>(dbl ? static_cast<const uint64_t*>(S->crd[0]) : nullptr, nouter,
                                                               ninner, S->val, Out, out_row, out_k, In, ldin, K, x_vals, S->dims[S->ord[0]]);
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    return SP_OK;
}

}  // namespace

extern "C" sp_status sp_sddmm(sp_tensor* S, const double* A, int64_t lda, const double* B, int64_t ldb, int64_t K,
                              double* x_vals, void* stream_) {
    SP_API_RANGE("sp_sddmm");
    if (!S || !A || !B || K < 1 || lda < K) return SP_ERR_INVALID_ARG;
    if (sp_check_device(S) != SP_OK) return SP_ERR_INVALID_ARG;
    {   // 8- and 16-bit storage is read through its 32-bit shadow
        sp_tensor* wide_ = nullptr;
        const sp_status ws_ = sp_widened(S, static_cast<cudaStream_t>(stream_), &wide_);
        if (ws_ != SP_OK) return ws_;
        S = wide_;
    }
    if (S->rank != 2 || S->ord[0] == S->ord[1]) return SP_ERR_UNSUPPORTED;
    if (ldb < S->dims[1]) return SP_ERR_INVALID_ARG;
    if (S->lt[1] == SP_DENSE) return sddmm_dense_inner(S, A, lda, B, ldb, K, x_vals, static_cast<cudaStream_t>(stream_));
    const bool colmajor = S->ord[0] == 1;      // S stored by columns (CSC, DCSC)
    const int64_t n = S->dims[1];
    if (ldb < n) return SP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t nnz = S->ncrd[1];
    if (nnz == 0) return SP_OK;
    if (!x_vals) return SP_ERR_INVALID_ARG;
    const bool dbl = S->lt[0] == SP_COMPRESSED;

    sp_workspace ws(stream);
    const int64_t ldt = (K + 1) & ~(int64_t)1;   // even, so rows stay 16-byte aligned
    int64_t ldt_k = ldt;                         // leading dimension of the gathered operand in the kernel
    double* Bt = ws.get<double>((size_t)n * ldt);
    if (ws.failed) return SP_ERR_ALLOC;
    dim3 tg((unsigned)sp_ceil_div(n, 32), (unsigned)sp_ceil_div(K, 32));
    k_transpose<<<tg, 256, 0, stream>>>(B, ldb, K, n, Bt, ldt);
    SP_LAUNCH_CHECK();

    sp_partition part;
    sp_status st = sp_get_merge_partition(S, kSItems, stream, &part);
    if (st != SP_OK) return st;
    const bool vec2 = (K % 2 == 0) && (lda % 2 == 0) && (reinterpret_cast<uintptr_t>(A) % 16 == 0) &&
                      (reinterpret_cast<uintptr_t>(Bt) % 16 == 0);
    // 32-byte loads when every operand row starts on a 32-byte boundary and K is a multiple of four
    const bool vec4 = vec2 && (K % 4 == 0) && (lda % 4 == 0) && (ldt % 4 == 0) && (reinterpret_cast<uintptr_t>(A) % 32 == 0) &&
                      (reinterpret_cast<uintptr_t>(Bt) % 32 == 0);
    const unsigned blocks = (unsigned)sp_ceil_div(part.nchunks * 32, kSThreads);
    // The kernel keeps the operand row of the outer (segment) index in registers and gathers the
    // row of the inner index: for column-major S the two operands simply trade places
    // (segment = column j -> row j of B^T; inner coordinate = row i -> row i of A).
    if (colmajor) {
        const double* ta = A; A = Bt; Bt = const_cast<double*>(ta);
        const int64_t tl = lda; lda = ldt; ldt_k = tl;
    }
#define SP_SDDMM_LAUNCH(V, NCH)                                                                                     \
    sddmm_launch_st = sp_launch_dependent(k_sddmm<P, I, V, NCH>, dim3(blocks), dim3(kSThreads), 0, stream, pos, crd,  \
                                          (const double*)S->val, outer, (const double*)A, lda, (const double*)Bt, ldt_k, K, \
                                          x_vals, (const int64_t*)part.row, (const int64_t*)part.nz, part.nchunks,        \
                                          S->dims[S->ord[0]], S->dims[S->ord[1]])
    cudaError_t sddmm_launch_st = cudaSuccess;
    SP_DISPATCH_WIDTHS(S, {
        const P* pos = static_cast<const P*>(S->pos[1]);
        const I* crd = static_cast<const I*>(S->crd[1]);
        const I* outer = dbl ? static_cast<const I*>(S->crd[0]) : nullptr;
        if (vec4 && K > 64 && K <= 512) {
            if (K <= 128) SP_SDDMM_LAUNCH(4, 1);
            else if (K <= 256) SP_SDDMM_LAUNCH(4, 2);
            else SP_SDDMM_LAUNCH(4, 4);
        } else if (vec2) {
            if (K <= 64) SP_SDDMM_LAUNCH(2, 1);
            else if (K <= 128) SP_SDDMM_LAUNCH(2, 2);
            else if (K <= 256) SP_SDDMM_LAUNCH(2, 4);
            else SP_SDDMM_LAUNCH(2, 0);
        } else {
            SP_SDDMM_LAUNCH(1, 0);
        }
    });
#undef SP_SDDMM_LAUNCH
    SP_CUDA(sddmm_launch_st);
    SP_LAUNCH_CHECK();
    sp_count_launches(2);
    SP_BOUNDS_RETURN(stream);
    return SP_OK;
}
