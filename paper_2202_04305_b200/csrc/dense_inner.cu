// SpMV and SpMM over encodings whose inner level is dense: (compressed, dense) - the paper's "CDR" of
// Section 6.2, the best format for its row-band matrices - and (dense, dense), in either order.
//
// values holds one full inner slice per stored outer index q (explicit zeros included), so the
// loops are dense:  row-major   y[i_q] = sum_k val[q, k] * x[k]        (one dot product per slice)
//                   col-major   y[i]  += val[q, i] * x[k_q]            (one axpy per slice)
// with i_q / k_q = crd[0][q], or q itself when the outer level is dense.
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace {

constexpr int kDThreads = 256;
constexpr int kDUnroll = 8;

// One group of TPR threads per stored slice: strided dot product with kDUnroll loads in flight.
// four blocks per SM: 64 registers, room for the sixteen 16-byte loads a thread keeps in flight
#ifndef SP_LB_DENSE_SPMV
#define SP_LB_DENSE_SPMV 4
#endif
#define SP_DENSE_SPMV_BOUNDS __launch_bounds__(kDThreads, SP_LB_DENSE_SPMV)
template <typename I, int TPR>
__global__ void SP_DENSE_SPMV_BOUNDS
k_spmv_dense_rows(const double* __restrict__ val, const I* __restrict__ outer, int64_t nslices, int64_t inner,
                  const double* __restrict__ x, double* __restrict__ y, int64_t douter) {
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
            if (tl == 0) y[SP_IDX(outer ? (int64_t)outer[q] : q, douter)] = s;
        } else {                                  // TPR == kDThreads: the whole block works on slice q
            if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = s;
            __syncthreads();
            if (threadIdx.x == 0) {
                double tot = s_part[0];
#pragma unroll
                for (int i = 1; i < kDThreads / 32; ++i) tot += s_part[i];
                y[SP_IDX(outer ? (int64_t)outer[q] : q, douter)] = tot;
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
                  const double* __restrict__ x, double* __restrict__ y, int64_t douter) {
    const int64_t i = (int64_t)blockIdx.x * kDThreads + threadIdx.x;
    if (i >= inner) return;
    const int64_t q0 = (int64_t)blockIdx.y * kDChunk;
    const int64_t q1 = q0 + kDChunk < nslices ? q0 + kDChunk : nslices;
    double s = 0.0;
    for (int64_t q = q0; q < q1; ++q) s = fma(__ldcs(val + q * inner + i), __ldg(x + SP_IDX(outer ? (int64_t)outer[q] : q, douter)), s);
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
                   int64_t kchunk, int vec_a, int64_t douter) {
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
        if (k < kend && c < N) b_reg = __ldg(B + (ROWMAJOR ? k : SP_IDX(outer ? (int64_t)outer[k] : k, douter)) * ldb + c);
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
        double* dst = C + (ROWMAJOR ? SP_IDX(outer ? (int64_t)outer[row] : row, douter) : row) * ldc;
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

// Row-major SpMM over a dense inner level with the operand tiles brought into shared memory by the
// tensor memory accelerator: the same 256 x 32 tile per block and 8 x 8 x 4 f64 matrix
// instruction as k_spmm_dense_inner, but no thread touches an operand before it is a fragment.
//
// One elected thread issues, per stage of kTK contraction indices, kTK/4 boxes of A
// ([kRT rows][4 k], 32 bytes per row, so a box lands as rows of four doubles: the eight rows x four
// k of a fragment are 256 consecutive bytes - no bank conflict and no padding) and four boxes of B
// ([kTK k][8 columns], 64 bytes per k: the four k x eight columns of a fragment are again 256
// consecutive bytes).  Rows, columns and k beyond the tensor are filled with zeros by the copy
// engine, so there is no ragged-edge code.  The stages form a ring: a stage is refilled by the
// elected thread right after the barrier that ends the step which consumed it, and its arrival is
// signalled on an mbarrier whose waits are bounded - a wait that runs out records the fact in a
// host-visible word, drains what is still in flight (bounded again) and leaves the block; the next
// call on the path reports SP_ERR_TIMEOUT.  The tensor maps cover this device's memory only and no
// copy is multicast.
constexpr int kTThreads = 256;
constexpr int kTRT = 256, kTCT = 32;           // tile of C per block
#ifndef SP_TMA_K
#define SP_TMA_K 16
#endif
#ifndef SP_TMA_STAGES
#define SP_TMA_STAGES 2
#endif
#ifndef SP_TMA_BLOCKS
#define SP_TMA_BLOCKS 2
#endif
constexpr int kTK = SP_TMA_K;                  // contraction indices per stage
constexpr int kTStages = SP_TMA_STAGES;
constexpr int kABox = kTRT * 4;                // doubles in one box of A
constexpr int kBBox = kTK * 8;                 // doubles in one box of B
constexpr int kStageDoubles = (kTK / 4) * kABox + 4 * kBBox;
constexpr uint32_t kStageBytes = kStageDoubles * sizeof(double);
constexpr size_t kTmaSmem = (size_t)kTStages * kStageBytes + kTStages * sizeof(uint64_t) + 128;
constexpr uint32_t kWaitPollNs = 2000;         // one poll of an mbarrier may sleep this long ...
constexpr int kWaitLimit = 1 << 19;            // ... and a block gives up after this many polls: about a second

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity), "r"(kWaitPollNs) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (int it = 0; it < kWaitLimit; ++it)
        if (mbar_try(bar, parity)) return true;
    return false;
}
// one box of a rank-2 tensor map: x = innermost coordinate (elements), y = row
__device__ __forceinline__ void tma_box(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_addr(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_addr(bar)) : "memory");
}

template <typename I>
__global__ void __launch_bounds__(kTThreads, SP_TMA_BLOCKS)
k_spmm_dense_inner_tma(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       const I* __restrict__ outer, int64_t nrows, int64_t nk, int64_t N, double* __restrict__ C,
                       int64_t ldc, int64_t kchunk, int* __restrict__ gave_up, int64_t douter) {
    extern __shared__ __align__(128) unsigned char s_raw[];
    double* s_stage = reinterpret_cast<double*>((reinterpret_cast<uintptr_t>(s_raw) + 127) & ~(uintptr_t)127);
    uint64_t* s_full = reinterpret_cast<uint64_t*>(s_stage + (size_t)kTStages * kStageDoubles);
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int r0 = (int)blockIdx.x * kTRT, c0 = (int)blockIdx.y * kTCT;
    const int64_t kbeg = (int64_t)blockIdx.z * kchunk;
    const int64_t kend = kbeg + kchunk < nk ? kbeg + kchunk : nk;
    const int nsteps = kbeg < kend ? (int)((kend - kbeg + kTK - 1) / kTK) : 0;

    if (t == 0) {
#pragma unroll
        for (int s = 0; s < kTStages; ++s) mbar_init(&s_full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto issue = [&](int step) {                 // elected thread only
        const int s = step % kTStages;
        double* dst = s_stage + (size_t)s * kStageDoubles;
        const int k0 = (int)(kbeg + (int64_t)step * kTK);
        mbar_expect(&s_full[s], kStageBytes);
#pragma unroll
        for (int g = 0; g < kTK / 4; ++g) tma_box(dst + g * kABox, &map_a, k0 + 4 * g, r0, &s_full[s]);
#pragma unroll
        for (int j = 0; j < 4; ++j) tma_box(dst + (kTK / 4) * kABox + j * kBBox, &map_b, c0 + 8 * j, k0, &s_full[s]);
    };
    int issued = 0;
    if (t == 0)
        for (; issued < kTStages - 1 && issued < nsteps; ++issued) issue(issued);

    double acc[4][4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j][0] = 0.0; acc[i][j][1] = 0.0; }

    const int fk = lane & 3, fr = lane >> 2;
    bool lost = false;
    int step = 0;
    for (; step < nsteps; ++step) {
        // the stage refilled here was read in step - 1; the barrier that ended that step freed it
        if (t == 0 && issued < nsteps) { issue(issued); ++issued; }
        const int s = step % kTStages;
        const bool here = mbar_wait_bounded(&s_full[s], (uint32_t)(step / kTStages) & 1u);
        if (here) {
            const double* sa = s_stage + (size_t)s * kStageDoubles;
            const double* sb = sa + (kTK / 4) * kABox;
#pragma unroll
            for (int g = 0; g < kTK / 4; ++g) {
                double a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) a[i] = sa[g * kABox + (w * 32 + i * 8 + fr) * 4 + fk];
#pragma unroll
                for (int j = 0; j < 4; ++j) b[j] = sb[j * kBBox + (4 * g + fk) * 8 + fr];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) dmma_8x8x4(acc[i][j][0], acc[i][j][1], a[i], b[j]);
            }
        }
        // the barrier that frees this stage also carries the verdict of every thread's wait, so the
        // whole block leaves the loop together
        if (__syncthreads_or(here ? 0 : 1)) { lost = true; break; }
    }
    if (lost) {
        // some wait ran out: say so, let the copies already issued land (bounded) and write nothing
        if (t == 0) {
            *gave_up = 1;
            __threadfence_system();
            for (int p = step; p < issued; ++p) mbar_wait_bounded(&s_full[p % kTStages], (uint32_t)(p / kTStages) & 1u);
        }
        __syncthreads();
        return;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t row = (int64_t)r0 + w * 32 + i * 8 + fr;
        if (row >= nrows) continue;
        double* dst = C + SP_IDX(outer ? (int64_t)outer[row] : row, douter) * ldc;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t col = (int64_t)c0 + j * 8 + 2 * fk + h;
                if (col < N) {
                    if (gridDim.z > 1) atomicAdd(dst + col, acc[i][j][h]); else dst[col] = acc[i][j][h];
                }
            }
        }
    }
}


// ---- host side of the TMA-fed kernel ----------------------------------------------------------
// cuTensorMapEncodeTiled is fetched through the runtime, so the library does not link the driver.
using encode_tiled_fn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                     const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TmaHost {
    encode_tiled_fn encode = nullptr;
    int* gave_up_host = nullptr;       // pinned, mapped: written by a block whose wait ran out
    int* gave_up_dev = nullptr;
    bool ready = false;
};

TmaHost& tma_host() {
    static TmaHost h;
    static std::once_flag once;
    std::call_once(once, [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess || fn == nullptr) {
            (void)cudaGetLastError();
            return;
        }
        void* word = nullptr;
        if (cudaHostAlloc(&word, sizeof(int), cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess) { (void)cudaGetLastError(); return; }
        *static_cast<int*>(word) = 0;
        void* dev = nullptr;
        if (cudaHostGetDevicePointer(&dev, word, 0) != cudaSuccess) { (void)cudaGetLastError(); cudaFreeHost(word); return; }
        h.encode = reinterpret_cast<encode_tiled_fn>(fn);
        h.gave_up_host = static_cast<int*>(word);
        h.gave_up_dev = static_cast<int*>(dev);
        h.ready = true;
    });
    return h;
}

// rank-2 f64 tensor map: `cols` contiguous elements per row, rows `ld` elements apart
bool encode_f64_2d(const TmaHost& h, CUtensorMap* map, const double* base, uint64_t cols, uint64_t rows, uint64_t ld,
                   uint32_t box_cols, uint32_t box_rows) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * sizeof(double)};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return h.encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 2, const_cast<double*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Whether the TMA-fed kernel can take this product: row-major storage, every row of A and of B
// starting on a 16-byte boundary (a tensor map's stride rule), extents inside the 32-bit coordinates
// of a copy.  Returns SP_OK after the launch, SP_ERR_UNSUPPORTED when the caller should use the
// register-staged kernel, anything else as an error.
sp_status spmm_dense_inner_tma(const sp_tensor* A, const void* outer, int64_t nslices, int64_t inner, const double* B,
                               int64_t N, int64_t ldb, double* C, int64_t ldc, int64_t ksplit_hint, cudaStream_t stream) {
    constexpr int64_t kLim = (int64_t)1 << 31;
    if (inner % 2 || ldb % 2 || reinterpret_cast<uintptr_t>(A->val) % 16 || reinterpret_cast<uintptr_t>(B) % 16)
        return SP_ERR_UNSUPPORTED;
    if (N <= 0 || ldb < N || inner >= kLim - kTK || nslices >= kLim - kTRT || N >= kLim - kTCT) return SP_ERR_UNSUPPORTED;
    TmaHost& h = tma_host();
    if (!h.ready) return SP_ERR_UNSUPPORTED;
    if (*static_cast<volatile int*>(h.gave_up_host) != 0) return SP_ERR_TIMEOUT;   // an earlier launch gave up
    CUtensorMap map_a, map_b;
    if (!encode_f64_2d(h, &map_a, A->val, (uint64_t)inner, (uint64_t)nslices, (uint64_t)inner, 4, kTRT) ||
        !encode_f64_2d(h, &map_b, B, (uint64_t)N, (uint64_t)inner, (uint64_t)ldb, 8, kTK))
        return SP_ERR_UNSUPPORTED;
    const int64_t rb = sp_ceil_div(nslices, kTRT), cb = sp_ceil_div(N, kTCT);
    if (cb > 65535) return SP_ERR_UNSUPPORTED;
    int64_t ksplit = ksplit_hint;
    const int64_t most = sp_ceil_div(inner, 16 * kTK);
    if (ksplit > most) ksplit = most;
    if (ksplit < 1) ksplit = 1;
    const int64_t kchunk = sp_ceil_div(sp_ceil_div(inner, ksplit), kTK) * kTK;
    ksplit = sp_ceil_div(inner, kchunk);
    if (outer != nullptr || ksplit > 1) {               // rows not stored are zero; split sums start at zero
        const int64_t m = A->dims[0];
        if (ldc == N) SP_CUDA(cudaMemsetAsync(C, 0, (size_t)m * N * sizeof(double), stream));
        else SP_CUDA(cudaMemset2DAsync(C, (size_t)ldc * sizeof(double), 0, (size_t)N * sizeof(double), (size_t)m, stream));
    }
    dim3 grid((unsigned)rb, (unsigned)cb, (unsigned)ksplit);
    // the dynamic shared-memory limit is a per-device attribute of the function: raised once per device
    static std::mutex attr_mutex;
    static uint64_t attr_done[2] = {0, 0};          // [coordinate width], one bit per device
    const int wi = A->crdBits == 32 ? 0 : 1;
    {
        std::lock_guard<std::mutex> lock(attr_mutex);
        if (A->device < 0 || A->device >= 64 || !((attr_done[wi] >> A->device) & 1)) {
            SP_CUDA(wi == 0 ? cudaFuncSetAttribute(k_spmm_dense_inner_tma<uint32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTmaSmem)
                            : cudaFuncSetAttribute(k_spmm_dense_inner_tma<uint64_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTmaSmem));
            if (A->device >= 0 && A->device < 64) attr_done[wi] |= (uint64_t)1 << A->device;
        }
    }
    if (wi == 0)
        k_spmm_dense_inner_tma<uint32_t><<<grid, kTThreads, kTmaSmem, stream>>>(map_a, map_b, static_cast<const uint32_t*>(outer), nslices,
                                                                                inner, N, C, ldc, kchunk, h.gave_up_dev, A->dims[A->ord[0]]);
    else
        k_spmm_dense_inner_tma<uint64_t><<<grid, kTThreads, kTmaSmem, stream>>>(map_a, map_b, static_cast<const uint64_t*>(outer), nslices,
                                                                                inner, N, C, ldc, kchunk, h.gave_up_dev, A->dims[A->ord[0]]);
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    SP_BOUNDS_RETURN(stream);
    return SP_OK;
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
                k_spmv_dense_rows<I, kDThreads><<<blocks, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, x, y, A->dims[A->ord[0]]); \
            } else {                                                                                                 \
                const int64_t need = sp_ceil_div(nslices, kDThreads / 32);                                           \
                const unsigned blocks = (unsigned)(need < 148 * 16 ? need : 148 * 16);                               \
                k_spmv_dense_rows<I, 32><<<blocks, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, x, y, A->dims[A->ord[0]]);     \
            }                                                                                                        \
        } else {                                                                                                     \
            const int64_t chunks = sp_ceil_div(nslices, kDChunk);                                                    \
            if (chunks > 65535) return SP_ERR_UNSUPPORTED;                                                           \
            dim3 grid((unsigned)sp_ceil_div(inner, kDThreads), (unsigned)chunks);                                    \
            k_spmv_dense_cols<I><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, x, y, A->dims[A->ord[0]]);               \
        }                                                                                                            \
    } while (0)
    if (A->crdBits == 32) SP_DENSE_LAUNCH(uint32_t); else SP_DENSE_LAUNCH(uint64_t);
#undef SP_DENSE_LAUNCH
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    SP_BOUNDS_RETURN(stream);
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
    if (rowmajor) {
        // the TMA-fed kernel takes every row-major product whose operands meet a tensor map's rules
        const int64_t tiles = rb * cb;
        const sp_status st = spmm_dense_inner_tma(A, outer_c ? A->crd[0] : nullptr, nslices, inner, B, N, ldb, C, ldc,
                                                  tiles < SP_TMA_BLOCKS * 148 ? sp_ceil_div(SP_TMA_BLOCKS * 148, tiles) : 1, stream);
        if (st != SP_ERR_UNSUPPORTED) return st;
    }
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
        if (rowmajor) k_spmm_dense_inner<I, true><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, B, N, ldb, C, ldc, kchunk, vec_a, A->dims[A->ord[0]]); \
        else k_spmm_dense_inner<I, false><<<grid, kDThreads, 0, stream>>>(A->val, outer, nslices, inner, B, N, ldb, C, ldc, kchunk, vec_a, A->dims[A->ord[0]]);       \
    } while (0)
    if (A->crdBits == 32) SP_DENSE_MM(uint32_t); else SP_DENSE_MM(uint64_t);
#undef SP_DENSE_MM
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    SP_BOUNDS_RETURN(stream);
    return SP_OK;
}
