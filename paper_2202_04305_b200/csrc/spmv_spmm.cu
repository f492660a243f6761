// sp_spmv and sp_spmm over (dense|compressed, compressed) storage in either
// dimension order (CSR, DCSR, CSC, DCSC).
//
// The loops are the ones the paper's sparsification yields for
// x[i] = A[i,j] * b[j] (Section 6.2) and C[i,j] = A[i,k] * B[k,j] (Section 1):
// an outer loop over the level-0 index (all of it, or the stored ones through
// crd[0]) and an inner loop over pos[1][q] .. pos[1][q+1].  Here the two loops
// are flattened into one merge path over (segment ends, entries) and cut into
// equal pieces, so a piece costs the same whatever the row-length skew.
//
// Row-major encodings reduce into rows: pieces write the rows that end inside
// them and hand the open last row to a fix-up pass as a carry (no atomics).
// Column-major encodings scatter into the output with f64 atomic adds.
#include "common.cuh"

#include <limits.h>

namespace {

// ===================================================================== SpMV
constexpr int kVThreads = 256;
constexpr int kVIpt = 8;
constexpr int kVTile = kVThreads * kVIpt;   // merge items per CTA

// Five blocks per SM (48 registers, 40 warps): on the 65.5M-entry row band 0.161 ms against 0.173 ms with
// the 58 registers and four blocks the compiler picks on its own, and 0.189 ms with six (40 registers, spills).
#ifndef SP_LB_SPMV
#define SP_LB_SPMV 5
#endif
template <typename P, typename I, bool SCATTER>
__global__ void __launch_bounds__(kVThreads, SP_LB_SPMV)
k_spmv(const P* __restrict__ pos, const I* __restrict__ crd, const double* __restrict__ val,
       const I* __restrict__ outer, const double* __restrict__ x, double* __restrict__ y,
       const int64_t* __restrict__ prow, const int64_t* __restrict__ pnz, int64_t nseg,
       double* __restrict__ carry_val, int64_t* __restrict__ carry_row, int64_t m, int64_t n) {
    // m, n: lengths of y and x (used by the bounds-checking debug build only)
    // a thread walks kVIpt consecutive products; one pad slot per kVIpt keeps those walks on distinct banks
    __shared__ int s_end[kVTile + 1];
    __shared__ double s_prod[kVTile + kVTile / kVIpt];
    __shared__ I s_dst[SCATTER ? kVTile + kVTile / kVIpt : 1];
#define SP_PAD(i) ((i) + ((i) / kVIpt))
    __shared__ double s_wv[kVThreads / 32];
    __shared__ int s_wf[kVThreads / 32];

    const int t = threadIdx.x;
    const int64_t i0 = prow[blockIdx.x], j0 = pnz[blockIdx.x];
    const int64_t i1 = prow[blockIdx.x + 1], j1 = pnz[blockIdx.x + 1];
    const int nrows = (int)(i1 - i0), nnzs = (int)(j1 - j0);

    // All loads of the tile are issued before anything consumes them: kVIpt coordinates and values
    // per thread, then the kVIpt gathered x entries (out-of-range slots re-read entry 0 and are dropped).
    I cc[kVIpt];
    double vv[kVIpt], xx[kVIpt];
    if (nnzs > 0) {
#pragma unroll
        for (int it = 0; it < kVIpt; ++it) {
            const int jj = t + it * kVThreads;
            const int64_t g = j0 + (jj < nnzs ? jj : 0);
            cc[it] = crd[g];
            vv[it] = val[g];
        }
        if (!SCATTER) {
#pragma unroll
            for (int it = 0; it < kVIpt; ++it) xx[it] = __ldg(x + SP_IDX(cc[it], n));
        }
    }
    if (!SCATTER && nrows == 0) {
        // The whole tile lies inside one long row: no row ends to merge with, so the tile is a
        // plain dot product - registers and one block reduction, no staging.
        double s = 0.0;
#pragma unroll
        for (int it = 0; it < kVIpt; ++it)
            if (t + it * kVThreads < nnzs) s = fma(vv[it], xx[it], s);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if ((t & 31) == 0) s_wv[t >> 5] = s;
        __syncthreads();
        if (t == 0) {
            double tot = s_wv[0];
#pragma unroll
            for (int i = 1; i < kVThreads / 32; ++i) tot += s_wv[i];
            carry_val[blockIdx.x] = tot;
            carry_row[blockIdx.x] = (i1 < nseg && j1 > j0) ? i1 : -1;
        }
        return;
    }
    for (int r = t; r < nrows; r += kVThreads) s_end[r] = (int)((int64_t)pos[i0 + r + 1] - j0);
    if (nnzs > 0) {
#pragma unroll
        for (int it = 0; it < kVIpt; ++it) {
            const int jj = t + it * kVThreads;
            if (jj < nnzs) {
                if (SCATTER) { s_prod[SP_PAD(jj)] = vv[it]; s_dst[SP_PAD(jj)] = cc[it]; }
                else s_prod[SP_PAD(jj)] = vv[it] * xx[it];
            }
        }
    }
    __syncthreads();

    const int total = nrows + nnzs;
    const int d0 = min(t * kVIpt, total), d1 = min(d0 + kVIpt, total);
    int lo = max(0, d0 - nnzs), hi = min(d0, nrows);
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (s_end[mid] <= d0 - mid - 1) lo = mid + 1; else hi = mid;
    }
    int ti = lo, tj = d0 - lo;

    if (SCATTER) {
        // segment = a column of A; every entry adds val * x[col] into y[row]
        int64_t seg = i0 + ti;
        double xc = seg < nseg ? x[SP_IDX(outer ? (int64_t)outer[seg] : seg, n)] : 0.0;
        for (int s = d0; s < d1; ++s) {
            if (ti < nrows && s_end[ti] <= tj) {
                ++ti; ++seg;
                xc = seg < nseg ? x[SP_IDX(outer ? (int64_t)outer[seg] : seg, n)] : 0.0;
            } else {
                atomicAdd(y + SP_IDX(s_dst[SP_PAD(tj)], m), s_prod[SP_PAD(tj)] * xc);
                ++tj;
            }
        }
        return;
    }

    double run = 0.0, first_val = 0.0;
    int first_row = -1;
    for (int s = d0; s < d1; ++s) {
        if (ti < nrows && s_end[ti] <= tj) {
            if (first_row < 0) { first_row = ti; first_val = run; }
            else {
                const int64_t r = i0 + ti;
                y[SP_IDX(outer ? (int64_t)outer[r] : r, m)] = run;
            }
            run = 0.0;
            ++ti;
        } else {
            run += s_prod[SP_PAD(tj)];
            ++tj;
        }
    }
    // carry chain across threads: out = flag ? run : in + run
    int f = first_row >= 0;
    double v = run;
    const int lane = t & 31, w = t >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int fu = __shfl_up_sync(0xffffffffu, f, o);
        double vu = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) { if (!f) v += vu; f |= fu; }
    }
    int fe = __shfl_up_sync(0xffffffffu, f, 1);
    double ve = __shfl_up_sync(0xffffffffu, v, 1);
    if (lane == 0) { fe = 0; ve = 0.0; }
    if (lane == 31) { s_wf[w] = f; s_wv[w] = v; }
    __syncthreads();
    int pf = 0;
    double pv = 0.0;
    for (int i = 0; i < w; ++i) {
        if (s_wf[i]) { pf = 1; pv = s_wv[i]; } else pv += s_wv[i];
    }
    const double in = fe ? ve : pv + ve;
    (void)pf;
    if (first_row >= 0) {
        const int64_t r = i0 + first_row;
        y[SP_IDX(outer ? (int64_t)outer[r] : r, m)] = first_val + in;
    }
    if (t == kVThreads - 1) {
        const double outv = (first_row >= 0) ? run : in + run;
        carry_val[blockIdx.x] = outv;
        carry_row[blockIdx.x] = (i1 < nseg && j1 > j0) ? i1 : -1;
    }
#undef SP_PAD
}

template <typename I>
__global__ void k_spmv_fixup(const double* __restrict__ carry_val, const int64_t* __restrict__ carry_row,
                             int64_t ntiles, const I* __restrict__ outer, double* __restrict__ y, int64_t m) {
    sp_wait_for_previous_kernel();
    int64_t w = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (w >= ntiles) return;
    const int64_t r = carry_row[w];
    if (r < 0 || (w > 0 && carry_row[w - 1] == r)) return;
    double s = 0.0;
    for (int64_t u = w; u < ntiles && carry_row[u] == r; ++u) s += carry_val[u];
    y[SP_IDX(outer ? (int64_t)outer[r] : r, m)] += s;
}

// Row-major SpMV for matrices of short rows: G lanes per stored row, no staging, no carries.
// Every lane issues its (up to four) coordinate and value loads, then the gathered x entries,
// before the first multiply-add; the row's sum is folded over the group's lanes and written once.
// Rows without entries (CSR) are written as zeros here; when level 0 is compressed the group of
// stored row q also writes the zeros of the rows that storage elides between stored rows q - 1 and q
// (the last group those after its row too), so y needs no clearing pass.
#ifndef SP_SPMV_ROWS_THREADS
#define SP_SPMV_ROWS_THREADS 64
#endif
template <typename P, typename I, int G>
__global__ void __launch_bounds__(SP_SPMV_ROWS_THREADS)
k_spmv_rows(const P* __restrict__ pos, const I* __restrict__ crd, const double* __restrict__ val,
            const I* __restrict__ outer, const double* __restrict__ x, double* __restrict__ y, int64_t nseg,
            int64_t m, int64_t n, int64_t nnz) {
    constexpr int kU = 4;
    const int64_t q = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x % G;
    const bool live = q < nseg;
    const int64_t p0 = live ? (int64_t)pos[q] : 0, p1 = live ? (int64_t)pos[q + 1] : 0;
    double s = 0.0;
    for (int64_t p = p0 + gl; p < p1; p += kU * G) {
        I c[kU];
        double v[kU], xx[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int64_t pp = p + u * G;
            const bool ok = pp < p1;
            c[u] = ok ? crd[SP_IDX(pp, nnz)] : (I)0;
            v[u] = ok ? val[SP_IDX(pp, nnz)] : 0.0;
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) xx[u] = (p + u * G < p1) ? __ldg(x + SP_IDX(c[u], n)) : 0.0;
#pragma unroll
        for (int u = 0; u < kU; ++u) s = fma(v[u], xx[u], s);
    }
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (!live) return;
    const int64_t row = SP_IDX(outer ? (int64_t)outer[q] : q, m);
    if (gl == 0) y[row] = s;
    if (outer) {
        const int64_t gap0 = q > 0 ? SP_IDX(outer[q - 1], m) + 1 : 0;
        for (int64_t r = gap0 + gl; r < row; r += G) y[r] = 0.0;
        if (q == nseg - 1)
            for (int64_t r = row + 1 + gl; r < m; r += G) y[r] = 0.0;
    }
}

// ===================================================================== SpMM
// The merge-path and scatter kernels work warp by warp; four warps per block measured 1 to 5 % faster than eight.
#ifndef SP_SPMM_THREADS
#define SP_SPMM_THREADS 128
#endif
constexpr int kMThreads = SP_SPMM_THREADS;
constexpr int kMItems = 128;   // merge items per warp

template <int V> struct vec_t;
template <> struct vec_t<1> { double a[1]; };
template <> struct __align__(16) vec_t<2> { double a[2]; };

template <int V>
__device__ __forceinline__ vec_t<V> ld_vec(const double* p) {
    vec_t<V> r;
    if (V == 2) { double2 q = *reinterpret_cast<const double2*>(p); r.a[0] = q.x; r.a[V - 1] = q.y; }
    else r.a[0] = *p;
    return r;
}
template <int V>
__device__ __forceinline__ void st_vec(double* p, const double* a) {
    if (V == 2) *reinterpret_cast<double2*>(p) = make_double2(a[0], a[V - 1]);
    else *p = a[0];
}

// Row-major SpMM (CSR, DCSR).  A warp walks its merge-path piece 32 entries at a time; lane = output
// column(s).  The ends of the rows that fall inside a batch come from a 32-row window of pos[] as a
// bit mask, so the loads of the batch do not depend on the row structure: B rows are fetched in
// groups of kGather independent loads, then accumulated in order, and a row is stored when its end
// bit comes up (rows without entries that end at the same place are stored as zeros).
constexpr int kGather = 8;

// 1024 threads per SM (64 registers): 0.0755 ms on the power-law matrix with N = 64, against 0.0785 ms at
// the 72 registers the compiler takes unasked, 0.079 at 80-96, 0.0895 at 48
#ifndef SP_LB_GATHER
#define SP_LB_GATHER (1024 / SP_SPMM_THREADS)
#endif
#define SP_GATHER_BOUNDS __launch_bounds__(kMThreads, SP_LB_GATHER)
template <typename P, typename I, int V>
__global__ void SP_GATHER_BOUNDS
k_spmm_gather(const P* __restrict__ pos, const I* __restrict__ crd, const double* __restrict__ val,
              const I* __restrict__ outer, const double* __restrict__ B, int64_t N, int64_t ldb,
              double* __restrict__ C, int64_t ldc, const int64_t* __restrict__ prow,
              const int64_t* __restrict__ pnz, int64_t nchunks, int64_t nseg, double* __restrict__ carry,
              int64_t* __restrict__ carry_row, int64_t m, int64_t n) {
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    if (w >= nchunks) return;
    const int lane = threadIdx.x & 31;
    const int64_t i0 = prow[w], j0 = pnz[w], i1 = prow[w + 1], j1 = pnz[w + 1];
    constexpr int64_t kInf = INT64_MAX;
    constexpr int kG = V == 2 ? kGather / 2 : kGather;   // same bytes in flight either way
    int64_t pstart = j0;

    for (int64_t cbase = 0; cbase < N; cbase += 32 * V) {
        const int64_t col = cbase + (int64_t)lane * V;
        const bool on = col < N;
        const double* Bc = B + (on ? col : cbase);        // idle lanes read a valid column and never write
        double acc[V];
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] = 0.0;
        int64_t row = i0, p = j0, rbase = i0;
        pstart = j0;
        int64_t E = (rbase + lane < i1) ? (int64_t)pos[rbase + lane + 1] : kInf;
        I c_n = (p + lane < j1) ? crd[p + lane] : (I)0;
        double v_n = (p + lane < j1) ? val[p + lane] : 0.0;

        // stores `acc` as row `row`, then zero rows for the other rows of the window that end at `pe`
        auto close_rows = [&](int64_t pe) {
            const int same = __popc(__ballot_sync(0xffffffffu, E == pe));
            for (int r = 0; r < same; ++r) {
                if (on) st_vec<V>(C + SP_IDX(outer ? (int64_t)outer[row] : row, m) * ldc + col, acc);
#pragma unroll
                for (int q = 0; q < V; ++q) acc[q] = 0.0;
                ++row;
            }
            pstart = pe;
        };

        // every turn of this loop either closes at least one row or consumes at least one entry;
        // `budget` bounds the turns all the same, so a malformed pos[] cannot spin a warp for ever
        for (int64_t budget = (i1 - i0) + (j1 - j0) + 2; budget > 0; --budget) {
            if (row - rbase >= 32) {              // the window is used up (also when row == i1)
                rbase += 32;
                E = (rbase + lane < i1) ? (int64_t)pos[rbase + lane + 1] : kInf;
            }
            // rows that end exactly here: the open row if it is complete, and rows without entries
            if (row < i1 && __shfl_sync(0xffffffffu, E, (int)(row - rbase)) == p) {
                close_rows(p);
                continue;
            }
            if (p >= j1) break;
            const int64_t elast = __shfl_sync(0xffffffffu, E, 31);
            int64_t lim = j1 - p;
            if (elast - p < lim) lim = elast - p;
            const int cnt = lim < 32 ? (int)lim : 32;
            if (cnt <= 0) break;                  // cannot happen for a well-formed pos[]
            const I c_l = c_n;
            const double v_l = v_n;
            {
                const int64_t pn = p + cnt;
                c_n = (pn + lane < j1) ? crd[pn + lane] : (I)0;
                v_n = (pn + lane < j1) ? val[pn + lane] : 0.0;
            }
            const int64_t rel = E - p - 1;
            const unsigned endmask = __reduce_or_sync(0xffffffffu, (rel >= 0 && rel < cnt) ? (1u << (int)rel) : 0u);

            for (int g = 0; g < cnt; g += kG) {
                vec_t<V> b[kG];
#pragma unroll
                for (int u = 0; u < kG; ++u) {
                    if (g + u < cnt) {
                        const int64_t k = SP_IDX(__shfl_sync(0xffffffffu, c_l, g + u), n);
                        b[u] = ld_vec<V>(Bc + k * ldb);
                    }
                }
#pragma unroll
                for (int u = 0; u < kG; ++u) {
                    if (g + u < cnt) {
                        const double vv = __shfl_sync(0xffffffffu, v_l, g + u);
#pragma unroll
                        for (int q = 0; q < V; ++q) acc[q] = fma(vv, b[u].a[q], acc[q]);
                        if ((endmask >> (g + u)) & 1u) close_rows(p + g + u + 1);
                    }
                }
            }
            p += cnt;
        }
        if (on && j1 > pstart) st_vec<V>(carry + w * N + col, acc);
    }
    if (lane == 0) carry_row[w] = (j1 > pstart && i1 < nseg) ? i1 : -1;
}

// Row-major SpMM for matrices whose rows are of similar, moderate length: L lanes own a stored row
// and V = N / L output columns each, so nothing has to be reduced across lanes and nothing is
// carried between rows.  The lanes of a group read whole 16 * L-byte runs of a B row per load
// instruction (lane gl holds column pairs gl, gl + L, ...), and a lane has the loads of kU entries
// (16 loads of 16 bytes) in flight before the first multiply-add - the access pattern that fetches
// random rows fastest on this GPU.  Rows without entries are written as zeros; when level 0 is
// compressed the group of stored row q also writes the zeros of the rows that storage elides between
// stored rows q - 1 and q (the last group those after its row too), so that C needs no clearing pass.
#ifndef SP_SPMM_ROWS_THREADS
#define SP_SPMM_ROWS_THREADS 64
#endif
#ifdef SP_LB_ROWS
#define SP_ROWS_BOUNDS __launch_bounds__(SP_SPMM_ROWS_THREADS, SP_LB_ROWS)
#else
#define SP_ROWS_BOUNDS __launch_bounds__(SP_SPMM_ROWS_THREADS)
#endif
template <typename P, typename I, int L, int V>
__global__ void SP_ROWS_BOUNDS
k_spmm_rows(const P* __restrict__ pos, const I* __restrict__ crd, const double* __restrict__ val,
            const I* __restrict__ outer, const double* __restrict__ B, int64_t ldb, double* __restrict__ C,
            int64_t ldc, int64_t nseg, int64_t m, int64_t n) {
    constexpr int kU = 32 / V;                      // entries in flight: kU * V / 2 = 16 loads per lane
    const int64_t q = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) / L;
    const int gl = threadIdx.x % L;
    if (q >= nseg) return;                          // no warp-wide operation below: groups are independent
    const int64_t p0 = (int64_t)pos[q], p1 = (int64_t)pos[q + 1];
    const double* Bl = B + 2 * gl;
    double acc[V];
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] = 0.0;
    // coordinates and values are fetched one turn ahead, so that a turn's B rows can be requested at once
    I kn[kU];
    double vn[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {                  // the group's lanes read the same word: one transaction
        const bool ok = p0 + u < p1;
        kn[u] = ok ? crd[p0 + u] : (I)0;
        vn[u] = ok ? val[p0 + u] : 0.0;
    }
    for (int64_t p = p0; p < p1; p += kU) {
        int64_t k[kU];
        double v[kU];
        double2 b[kU][V / 2];
#pragma unroll
        for (int u = 0; u < kU; ++u) { k[u] = (int64_t)SP_IDX(kn[u], n); v[u] = vn[u]; }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
#pragma unroll
            for (int j = 0; j < V / 2; ++j)
                b[u][j] = (p + u < p1) ? *reinterpret_cast<const double2*>(Bl + k[u] * ldb + j * 2 * L) : make_double2(0.0, 0.0);
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const bool ok = p + kU + u < p1;
            kn[u] = ok ? crd[p + kU + u] : (I)0;
            vn[u] = ok ? val[p + kU + u] : 0.0;
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
#pragma unroll
            for (int j = 0; j < V / 2; ++j) {
                acc[2 * j] = fma(v[u], b[u][j].x, acc[2 * j]);
                acc[2 * j + 1] = fma(v[u], b[u][j].y, acc[2 * j + 1]);
            }
        }
    }
    const int64_t row = SP_IDX(outer ? (int64_t)outer[q] : q, m);
    double* crow = C + row * ldc + 2 * gl;
#pragma unroll
    for (int j = 0; j < V / 2; ++j) *reinterpret_cast<double2*>(crow + j * 2 * L) = make_double2(acc[2 * j], acc[2 * j + 1]);
    if (outer) {
        const int64_t gap0 = q > 0 ? SP_IDX(outer[q - 1], m) + 1 : 0;
        for (int64_t r = gap0; r < row; ++r)
#pragma unroll
            for (int j = 0; j < V / 2; ++j) *reinterpret_cast<double2*>(C + r * ldc + 2 * gl + j * 2 * L) = make_double2(0.0, 0.0);
        if (q == nseg - 1)
            for (int64_t r = row + 1; r < m; ++r)
#pragma unroll
                for (int j = 0; j < V / 2; ++j) *reinterpret_cast<double2*>(C + r * ldc + 2 * gl + j * 2 * L) = make_double2(0.0, 0.0);
    }
}

// Column-major SpMM (CSC, DCSC): C[i,:] += A[i,k] * B[k,:] for every stored entry, as a flat loop
// over entries.  seg[p] is the column k of entry p (expanded once per handle), crd[p] its row i.
// A warp takes kScatPer consecutive entries, 32 at a time; lane = output column.  Entries of one
// column are adjacent, so the B row they share is read from DRAM once and then from L1; C is
// updated with f64 atomic adds (it was zeroed by the caller).
constexpr int kScatPer = 256;

template <typename I, int V>
__global__ void __launch_bounds__(kMThreads)
k_spmm_scatter(const uint32_t* __restrict__ seg, const I* __restrict__ crd, const double* __restrict__ val,
               int64_t nnz, const double* __restrict__ B, int64_t N, int64_t ldb, double* __restrict__ C,
               int64_t ldc, int64_t m, int64_t n) {
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int64_t p0 = w * kScatPer;
    if (p0 >= nnz) return;
    const int64_t p1 = p0 + kScatPer < nnz ? p0 + kScatPer : nnz;
    for (int64_t cbase = 0; cbase < N; cbase += 32 * V) {
        const int64_t col = cbase + (int64_t)lane * V;
        const bool on = col < N;
        const double* Bc = B + (on ? col : cbase);
        double* Cc = C + (on ? col : cbase);
        for (int64_t p = p0; p < p1; p += 32) {
            const int cnt = p1 - p < 32 ? (int)(p1 - p) : 32;
            const uint32_t k_l = lane < cnt ? seg[p + lane] : 0u;
            const I i_l = lane < cnt ? crd[p + lane] : (I)0;
            const double v_l = lane < cnt ? val[p + lane] : 0.0;
            for (int g = 0; g < cnt; g += kGather) {
                vec_t<V> b[kGather];
#pragma unroll
                for (int u = 0; u < kGather; ++u) {
                    if (g + u < cnt) {
                        const int64_t k = SP_IDX(__shfl_sync(0xffffffffu, k_l, g + u), n);
                        b[u] = ld_vec<V>(Bc + k * ldb);
                    }
                }
#pragma unroll
                for (int u = 0; u < kGather; ++u) {
                    if (g + u < cnt) {
                        const int64_t i = SP_IDX(__shfl_sync(0xffffffffu, i_l, g + u), m);
                        const double vv = __shfl_sync(0xffffffffu, v_l, g + u);
                        if (on) {
#pragma unroll
                            for (int q = 0; q < V; ++q) atomicAdd(Cc + i * ldc + q, vv * b[u].a[q]);
                        }
                    }
                }
            }
        }
    }
}

template <typename I>
__global__ void k_spmm_fixup(const double* __restrict__ carry, const int64_t* __restrict__ carry_row,
                             int64_t nchunks, const I* __restrict__ outer, int64_t N, double* __restrict__ C,
                             int64_t ldc, int64_t m) {
    sp_wait_for_previous_kernel();
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    if (w >= nchunks) return;
    const int lane = threadIdx.x & 31;
    const int64_t r = carry_row[w];
    if (r < 0 || (w > 0 && carry_row[w - 1] == r)) return;
    int64_t end = w + 1;
    while (end < nchunks && carry_row[end] == r) ++end;
    double* crow = C + SP_IDX(outer ? (int64_t)outer[r] : r, m) * ldc;
    for (int64_t col = lane; col < N; col += 32) {
        double s = 0.0;
        for (int64_t u = w; u < end; ++u) s += carry[u * N + col];
        crow[col] += s;
    }
}

bool matrix_encoding_ok(const sp_tensor* A) {
    return A && A->rank == 2 && A->lt[1] == SP_COMPRESSED &&
           ((A->ord[0] == 0 && A->ord[1] == 1) || (A->ord[0] == 1 && A->ord[1] == 0));
}

}  // namespace

extern "C" sp_status sp_spmv(sp_tensor* A, const double* x, double* y, void* stream_) {
    SP_API_RANGE("sp_spmv");
    if (!A || !x || !y) return SP_ERR_INVALID_ARG;
    if (sp_check_device(A) != SP_OK) return SP_ERR_INVALID_ARG;
    {   // 8- and 16-bit storage is read through its 32-bit shadow
        sp_tensor* wide_ = nullptr;
        const sp_status ws_ = sp_widened(A, static_cast<cudaStream_t>(stream_), &wide_);
        if (ws_ != SP_OK) return ws_;
        A = wide_;
    }
    if (A->rank == 2 && A->lt[1] == SP_DENSE && A->ord[0] != A->ord[1])
        return sp_spmv_dense_inner(A, x, y, static_cast<cudaStream_t>(stream_));
    if (!matrix_encoding_ok(A)) return SP_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const bool rowmajor = A->ord[0] == 0;
    const bool dbl = A->lt[0] == SP_COMPRESSED;
    const int64_t m = A->dims[0];
    const int64_t nseg = A->npos[1] - 1;
    if (nseg <= 0 || A->ncrd[1] == 0 || (dbl && A->ncrd[0] == 0)) {
        SP_CUDA(cudaMemsetAsync(y, 0, (size_t)m * sizeof(double), stream));
        return SP_OK;
    }
    // Short rows (mean <= 256 entries, none longer than 4096): a lane group per row, one launch.
    // Anything skewed or long goes through the merge path below, whose cost does not depend on the
    // row lengths.
    if (rowmajor && A->ncrd[1] <= 256 * nseg) {
        int64_t max_seg = 0;
        const sp_status ms = sp_get_max_segment(A, stream, &max_seg);
        if (ms != SP_OK) return ms;
        if (max_seg <= 4096) {
            const int64_t mean = A->ncrd[1] / nseg;
            // About six entries per lane on average and at most 32 for the longest row.  Measured: rows of
            // 48 +- 7 entries, 8 lanes 0.040 ms, 16 lanes 0.042, 32 lanes 0.052, 4 lanes 0.044; power-law
            // rows of mean 16 and up to 435 entries, 16 lanes 0.023 ms, 4 lanes 0.031.
            const int64_t want = std::max<int64_t>(mean / 6, max_seg / 32);
            const int G = want <= 4 ? 4 : (want <= 8 ? 8 : (want <= 16 ? 16 : 32));
            const unsigned blocks = (unsigned)sp_ceil_div(nseg * G, SP_SPMV_ROWS_THREADS);
            SP_DISPATCH_WIDTHS(A, {
                const P* pos = static_cast<const P*>(A->pos[1]);
                const I* crd = static_cast<const I*>(A->crd[1]);
                const I* outer = dbl ? static_cast<const I*>(A->crd[0]) : nullptr;
                if (G == 4) k_spmv_rows<P, I, 4><<<blocks, SP_SPMV_ROWS_THREADS, 0, stream>>>(pos, crd, A->val, outer, x, y, nseg, m, A->dims[1], A->ncrd[1]);
                else if (G == 8) k_spmv_rows<P, I, 8><<<blocks, SP_SPMV_ROWS_THREADS, 0, stream>>>(pos, crd, A->val, outer, x, y, nseg, m, A->dims[1], A->ncrd[1]);
                else if (G == 16) k_spmv_rows<P, I, 16><<<blocks, SP_SPMV_ROWS_THREADS, 0, stream>>>(pos, crd, A->val, outer, x, y, nseg, m, A->dims[1], A->ncrd[1]);
                else k_spmv_rows<P, I, 32><<<blocks, SP_SPMV_ROWS_THREADS, 0, stream>>>(pos, crd, A->val, outer, x, y, nseg, m, A->dims[1], A->ncrd[1]);
            });
            SP_LAUNCH_CHECK();
            sp_count_launches(1);
            SP_BOUNDS_RETURN(stream);
            return SP_OK;
        }
    }
    if (!rowmajor || dbl) SP_CUDA(cudaMemsetAsync(y, 0, (size_t)m * sizeof(double), stream));
    sp_partition part;
    sp_status st = sp_get_merge_partition(A, kVTile, stream, &part);
    if (st != SP_OK) return st;
    // the open row of every tile: its partial sum and its row number, scratch of this call alone
    sp_workspace ws(stream);
    double* cval = rowmajor ? ws.get<double>((size_t)part.nchunks) : nullptr;
    int64_t* crow = rowmajor ? ws.get<int64_t>((size_t)part.nchunks) : nullptr;
    if (ws.failed) return SP_ERR_ALLOC;
    SP_DISPATCH_WIDTHS(A, {
        const P* pos = static_cast<const P*>(A->pos[1]);
        const I* crd = static_cast<const I*>(A->crd[1]);
        const I* outer = dbl ? static_cast<const I*>(A->crd[0]) : nullptr;
        if (rowmajor) {
            k_spmv<P, I, false><<<(unsigned)part.nchunks, kVThreads, 0, stream>>>(pos, crd, A->val, outer, x, y, part.row,
                                                                                  part.nz, nseg, cval, crow, m, A->dims[1]);
            SP_CUDA(sp_launch_dependent(k_spmv_fixup<I>, dim3((unsigned)sp_ceil_div(part.nchunks, 256)), dim3(256), 0, stream,
                                        (const double*)cval, (const int64_t*)crow, part.nchunks, outer, y, m));
            sp_count_launches(2);
        } else {
            k_spmv<P, I, true><<<(unsigned)part.nchunks, kVThreads, 0, stream>>>(pos, crd, A->val, outer, x, y, part.row,
                                                                                 part.nz, nseg, cval, crow, m, A->dims[1]);
            sp_count_launches(1);
        }
    });
    SP_LAUNCH_CHECK();
    SP_BOUNDS_RETURN(stream);
    return SP_OK;
}

extern "C" sp_status sp_spmm(sp_tensor* A, const double* B, int64_t N, int64_t ldb, double* C, int64_t ldc,
                             void* stream_) {
    SP_API_RANGE("sp_spmm");
    if (!A || !B || !C || N < 1 || ldb < N || ldc < N) return SP_ERR_INVALID_ARG;
    if (sp_check_device(A) != SP_OK) return SP_ERR_INVALID_ARG;
    if (N >= (1 << 20)) return SP_ERR_UNSUPPORTED;
    {   // 8- and 16-bit storage is read through its 32-bit shadow
        sp_tensor* wide_ = nullptr;
        const sp_status ws_ = sp_widened(A, static_cast<cudaStream_t>(stream_), &wide_);
        if (ws_ != SP_OK) return ws_;
        A = wide_;
    }
    if (A->rank == 2 && A->lt[1] == SP_DENSE && A->ord[0] != A->ord[1])
        return sp_spmm_dense_inner(A, B, N, ldb, C, ldc, static_cast<cudaStream_t>(stream_));
    if (!matrix_encoding_ok(A)) return SP_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const bool rowmajor = A->ord[0] == 0;
    const bool dbl = A->lt[0] == SP_COMPRESSED;
    const int64_t m = A->dims[0];
    auto clear_C = [&]() -> sp_status {
        if (ldc == N) SP_CUDA(cudaMemsetAsync(C, 0, (size_t)m * N * sizeof(double), stream));
        else SP_CUDA(cudaMemset2DAsync(C, (size_t)ldc * sizeof(double), 0, (size_t)N * sizeof(double), (size_t)m, stream));
        return SP_OK;
    };
    const int64_t nseg = A->npos[1] - 1;
    if (nseg <= 0 || A->ncrd[1] == 0 || (dbl && A->ncrd[0] == 0)) return clear_C();
    // column-major storage runs as a flat loop over entries with their column ids expanded once
    // (32-bit ids: a column-major matrix with 2^32 or more columns is refused)
    if (!rowmajor && A->dims[1] >= ((int64_t)1 << 32)) return SP_ERR_UNSUPPORTED;
    const uint32_t* segs = nullptr;
    sp_status st = SP_OK;
    // Rows of similar, moderate length (the longest at most four mean lengths + 32, and no more than
    // 4096 entries), N = 16, 32, 64 or 128 and 16-byte aligned operands: a lane group per row.
    // Skewed matrices stay on the merge path, whose pieces cost the same whatever the row lengths.
    // Measured on power-law rows (mean 16, up to 435 long, N = 64): merge path 0.091 ms, a lane group per
    // row 0.23 ms, lane groups for the rows up to 96 long plus a block for each longer one 0.16 ms.
    if (rowmajor && (N == 16 || N == 32 || N == 64 || N == 128) && ldb % 2 == 0 && ldc % 2 == 0 &&
        reinterpret_cast<uintptr_t>(B) % 16 == 0 && reinterpret_cast<uintptr_t>(C) % 16 == 0) {
        int64_t max_seg = 0;
        st = sp_get_max_segment(A, stream, &max_seg);
        if (st != SP_OK) return st;
        const int64_t mean = A->ncrd[1] / nseg;
        if (max_seg <= 4096 && max_seg <= 4 * mean + 32) {
#define SP_SPMM_ROWS(L, V)                                                                                              \
    k_spmm_rows<P, I, L, V><<<(unsigned)sp_ceil_div(nseg * L, SP_SPMM_ROWS_THREADS), SP_SPMM_ROWS_THREADS, 0, stream>>>( \
        pos, crd, A->val, outer, B, ldb, C, ldc, nseg, m, A->dims[1])
            SP_DISPATCH_WIDTHS(A, {
                const P* pos = static_cast<const P*>(A->pos[1]);
                const I* crd = static_cast<const I*>(A->crd[1]);
                const I* outer = dbl ? static_cast<const I*>(A->crd[0]) : nullptr;
                if (N == 16) SP_SPMM_ROWS(4, 4);
                else if (N == 32) SP_SPMM_ROWS(8, 4);
                else if (N == 64) SP_SPMM_ROWS(8, 8);
                else SP_SPMM_ROWS(16, 8);
            });
#undef SP_SPMM_ROWS
            SP_LAUNCH_CHECK();
            sp_count_launches(1);
            SP_BOUNDS_RETURN(stream);
            return SP_OK;
        }
    }
    if (!rowmajor || dbl) {            // rows that storage elides, and scatter targets, start from zero
        st = clear_C();
        if (st != SP_OK) return st;
    }
    sp_partition part;
    sp_workspace ws(stream);
    double* carry = nullptr;
    int64_t* crow = nullptr;
    if (!rowmajor) {
        st = sp_get_segment_ids(A, stream, &segs);
        if (st != SP_OK) return st;
    } else {
        st = sp_get_merge_partition(A, kMItems, stream, &part);
        if (st != SP_OK) return st;
        // the open row of every warp's piece: N partial sums and the row number, scratch of this call alone
        carry = ws.get<double>((size_t)part.nchunks * N);
        crow = ws.get<int64_t>((size_t)part.nchunks);
        if (ws.failed) return SP_ERR_ALLOC;
    }
    const bool vec2 = N > 32 && (N % 2 == 0) && (ldb % 2 == 0) && (ldc % 2 == 0) &&
                      (reinterpret_cast<uintptr_t>(B) % 16 == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0) &&
                      (reinterpret_cast<uintptr_t>(carry) % 16 == 0);
    const unsigned blocks = (unsigned)sp_ceil_div(part.nchunks * 32, kMThreads);
    SP_DISPATCH_WIDTHS(A, {
        const P* pos = static_cast<const P*>(A->pos[1]);
        const I* crd = static_cast<const I*>(A->crd[1]);
        const I* outer = dbl ? static_cast<const I*>(A->crd[0]) : nullptr;
        if (rowmajor) {
            if (vec2)
                k_spmm_gather<P, I, 2><<<blocks, kMThreads, 0, stream>>>(pos, crd, A->val, outer, B, N, ldb, C, ldc, part.row,
                                                                         part.nz, part.nchunks, nseg, carry, crow, m, A->dims[1]);
            else
                k_spmm_gather<P, I, 1><<<blocks, kMThreads, 0, stream>>>(pos, crd, A->val, outer, B, N, ldb, C, ldc, part.row,
                                                                         part.nz, part.nchunks, nseg, carry, crow, m, A->dims[1]);
            SP_CUDA(sp_launch_dependent(k_spmm_fixup<I>, dim3(blocks), dim3(kMThreads), 0, stream, (const double*)carry,
                                        (const int64_t*)crow, part.nchunks, outer, N, C, ldc, m));
            sp_count_launches(2);
        } else {
            (void)pos;
            const int64_t nnz = A->ncrd[1];
            const unsigned sblocks = (unsigned)sp_ceil_div(sp_ceil_div(nnz, kScatPer) * 32, kMThreads);
            if (nnz > 0) {
                if (vec2) k_spmm_scatter<I, 2><<<sblocks, kMThreads, 0, stream>>>(segs, crd, A->val, nnz, B, N, ldb, C, ldc, m, A->dims[1]);
                else k_spmm_scatter<I, 1><<<sblocks, kMThreads, 0, stream>>>(segs, crd, A->val, nnz, B, N, ldb, C, ldc, m, A->dims[1]);
                sp_count_launches(1);
            }
        }
    });
    SP_LAUNCH_CHECK();
    SP_BOUNDS_RETURN(stream);
    return SP_OK;
}

// ------------------------------------------------------------------ sp_spmv_static
// SpMV whose scratch (merge-path partition table and row carries) is a fixed device array
// compiled into the library instead of memory obtained at run time.
namespace {

constexpr int64_t kStaticMaxTiles = SP_SPMV_STATIC_MAX_ITEMS / kVTile;

struct SpmvStaticScratch {
    int64_t row[kStaticMaxTiles + 1];
    int64_t nz[kStaticMaxTiles + 1];
    double carry_val[kStaticMaxTiles];
    int64_t carry_row[kStaticMaxTiles];
};

// About 2 MiB, resident on every GPU that loads the library until the process exits.
static __device__ __align__(256) unsigned char g_spmv_static_scratch[sizeof(SpmvStaticScratch)];

// In host code the symbol above is only a handle; the device address has to be asked for,
// once per device, with that device current.
std::mutex g_static_mu;
void* g_static_addr[64] = {nullptr};

sp_status spmv_static_scratch(SpmvStaticScratch** out) {
    int dev = 0;
    SP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_addr[dev]) {
        void* p = nullptr;
        SP_CUDA(cudaGetSymbolAddress(&p, g_spmv_static_scratch));
        g_static_addr[dev] = p;
    }
    *out = static_cast<SpmvStaticScratch*>(g_static_addr[dev]);
    return SP_OK;
}

// Same merge-path split as the cached partition tables, written into the fixed scratch.
template <typename P>
__global__ void k_static_partition(const P* __restrict__ pos, int64_t nseg, int64_t nnz, int64_t ntiles,
                                   int64_t* __restrict__ row, int64_t* __restrict__ nz) {
    const int64_t w = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (w > ntiles) return;
    const int64_t total = nseg + nnz;
    int64_t d = w * kVTile;
    if (d > total) d = total;
    int64_t lo = d > nnz ? d - nnz : 0;
    int64_t hi = d < nseg ? d : nseg;
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)pos[mid + 1] <= d - mid - 1) lo = mid + 1; else hi = mid;
    }
    row[w] = lo;
    nz[w] = d - lo;
}

}  // namespace

extern "C" sp_status sp_spmv_static(const sp_tensor* A, const double* x, double* y, void* stream_) {
    SP_API_RANGE("sp_spmv_static");
    if (!A || !x || !y) return SP_ERR_INVALID_ARG;
    if (sp_check_device(A) != SP_OK) return SP_ERR_INVALID_ARG;
    if (!matrix_encoding_ok(A)) return SP_ERR_UNSUPPORTED;
    if (A->posBits < 32 || A->crdBits < 32) return SP_ERR_UNSUPPORTED;   // a widened copy would need an allocation
    const int64_t nseg = A->npos[1] - 1;
    const int64_t nnz = A->ncrd[1];
    if (nseg + nnz > (int64_t)SP_SPMV_STATIC_MAX_ITEMS) return SP_ERR_TOO_LARGE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    SpmvStaticScratch* sc = nullptr;
    sp_status st = spmv_static_scratch(&sc);
    if (st != SP_OK) return st;
    const bool rowmajor = A->ord[0] == 0;
    const bool dbl = A->lt[0] == SP_COMPRESSED;
    if (!rowmajor || dbl) SP_CUDA(cudaMemsetAsync(y, 0, (size_t)A->dims[0] * sizeof(double), stream));
    if (nseg <= 0) return SP_OK;
    int64_t ntiles = sp_ceil_div(nseg + nnz, kVTile);
    if (ntiles < 1) ntiles = 1;
    // Every scratch word read below is written earlier in this same call (the partition kernel
    // fills row/nz for all tiles, each SpMV block writes its own carry slot), so nothing left by
    // an earlier call is ever consumed and no clearing pass is needed.
    SP_DISPATCH_WIDTHS(A, {
        const P* pos = static_cast<const P*>(A->pos[1]);
        const I* crd = static_cast<const I*>(A->crd[1]);
        const I* outer = dbl ? static_cast<const I*>(A->crd[0]) : nullptr;
        k_static_partition<P><<<(unsigned)sp_ceil_div(ntiles + 1, 256), 256, 0, stream>>>(pos, nseg, nnz, ntiles, sc->row,
                                                                                          sc->nz);
        if (rowmajor) {
            k_spmv<P, I, false><<<(unsigned)ntiles, kVThreads, 0, stream>>>(pos, crd, A->val, outer, x, y, sc->row, sc->nz,
                                                                            nseg, sc->carry_val, sc->carry_row, A->dims[0], A->dims[1]);
            k_spmv_fixup<I><<<(unsigned)sp_ceil_div(ntiles, 256), 256, 0, stream>>>(sc->carry_val, sc->carry_row, ntiles,
                                                                                    outer, y, A->dims[0]);
            sp_count_launches(3);
        } else {
            k_spmv<P, I, true><<<(unsigned)ntiles, kVThreads, 0, stream>>>(pos, crd, A->val, outer, x, y, sc->row, sc->nz,
                                                                           nseg, sc->carry_val, sc->carry_row, A->dims[0], A->dims[1]);
            sp_count_launches(2);
        }
    });
    SP_LAUNCH_CHECK();
    return SP_OK;
}
