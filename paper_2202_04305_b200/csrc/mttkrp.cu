// sp_mttkrp: M[i,r] = sum_{j,k} T[i,j,k] * B[j,r] * C[k,r]  (Section 6.3).
//
// T is stored (compressed|dense, compressed, compressed) with logical dimension 0
// at level 0.  The derived loop nest walks slices (level 0), fibres (level 1) and
// entries (level 2); the entry loop accumulates val * F2[c2, r] per fibre, the
// fibre's sum is scaled by F1[c1, r] into the slice, and the slice's sum is row i
// of M.  F1 / F2 are B / C, or C / B when the two inner dimensions are stored
// interchanged (the paper's alternative ordering).
//
// The innermost entries are cut into equal ranges, one per warp; lane = column r.
// Slices that start and end inside a range are stored directly; the open slice at
// either end of a range is added into M (zeroed first) with one atomic add per
// column - no atomics in the entry or fibre loops.
#include "common.cuh"

namespace {

constexpr int kTThreads = 256;
constexpr int kTPer = 512;   // entries per warp

template <typename P, typename I>
__global__ void __launch_bounds__(kTThreads)
k_mttkrp(const P* __restrict__ pos1, const I* __restrict__ crd0, const P* __restrict__ pos2,
         const I* __restrict__ crd1, const I* __restrict__ crd2, const double* __restrict__ val,
         const double* __restrict__ F1, const double* __restrict__ F2, int64_t R, double* __restrict__ M,
         const int64_t* __restrict__ pfiber, const int64_t* __restrict__ pnz, const int64_t* __restrict__ pslice,
         int64_t nchunks, int64_t nslice, int64_t nfiber) {
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    if (w >= nchunks) return;
    const int lane = threadIdx.x & 31;
    const int64_t p0 = pnz[w], p1 = pnz[w + 1];
    if (p1 <= p0) return;

    for (int64_t rb = 0; rb < R; rb += 32) {
        const int64_t r = rb + lane;
        const bool on = r < R;
        int64_t f = pfiber[w], s = pslice[w], p = p0, nzbase = p0;
        int64_t fend = (int64_t)pos2[f + 1], send = (int64_t)pos1[s + 1];
        double bj = on ? F1[(int64_t)crd1[f] * R + r] : 0.0;
        double accf = 0.0, accs = 0.0;
        bool first = true, pending = false;
        I k_l = (nzbase + lane < p1) ? crd2[nzbase + lane] : (I)0;
        double v_l = (nzbase + lane < p1) ? val[nzbase + lane] : 0.0;

        while (p < p1) {
            const int64_t segend = fend < p1 ? fend : p1;
            while (p < segend) {
                int off = (int)(p - nzbase);
                if (off == 32) {
                    nzbase += 32;
                    k_l = (nzbase + lane < p1) ? crd2[nzbase + lane] : (I)0;
                    v_l = (nzbase + lane < p1) ? val[nzbase + lane] : 0.0;
                    off = 0;
                }
                const int cnt = (int)min(segend - p, (int64_t)(32 - off));
                for (int t = 0; t < cnt; t += 4) {
                    double c[4], vv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        c[u] = 0.0; vv[u] = 0.0;
                        if (t + u < cnt) {
                            const int64_t k = (int64_t)__shfl_sync(0xffffffffu, k_l, off + t + u);
                            vv[u] = __shfl_sync(0xffffffffu, v_l, off + t + u);
                            if (on) c[u] = F2[k * R + r];
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) accf = fma(vv[u], c[u], accf);
                }
                p += cnt;
                pending = true;
            }
            if (p == fend) {                       // the fibre is complete
                accs = fma(bj, accf, accs);
                accf = 0.0;
                ++f;
                if (f == send) {                   // and so is the slice
                    const int64_t i = crd0 ? (int64_t)crd0[s] : s;
                    if (on) {
                        if (first) atomicAdd(M + i * R + r, accs);
                        else M[i * R + r] = accs;
                    }
                    first = false;
                    pending = false;
                    accs = 0.0;
                    ++s;
                    while (s < nslice && (int64_t)pos1[s + 1] == f) ++s;   // slices with no fibres
                    send = s < nslice ? (int64_t)pos1[s + 1] : nfiber + 1;
                }
                if (f < nfiber) {
                    fend = (int64_t)pos2[f + 1];
                    bj = on ? F1[(int64_t)crd1[f] * R + r] : 0.0;
                }
            }
        }
        if (pending && on) {
            accs = fma(bj, accf, accs);
            const int64_t i = crd0 ? (int64_t)crd0[s] : s;
            atomicAdd(M + i * R + r, accs);
        }
    }
}

}  // namespace

extern "C" sp_status sp_mttkrp(sp_tensor* T, const double* B, const double* C, int64_t R, double* M, void* stream_) {
    if (!T || !B || !C || !M || R < 1) return SP_ERR_INVALID_ARG;
    if (T->rank != 3 || T->ord[0] != 0 || T->lt[1] != SP_COMPRESSED || T->lt[2] != SP_COMPRESSED)
        return SP_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    SP_CUDA(cudaMemsetAsync(M, 0, (size_t)T->dims[0] * R * sizeof(double), stream));
    const int64_t nnz = T->ncrd[2];
    if (nnz == 0) return SP_OK;
    const double* F1 = T->ord[1] == 1 ? B : C;   // factor of the dimension kept at level 1
    const double* F2 = T->ord[1] == 1 ? C : B;
    sp_partition part;
    sp_status st = sp_get_mttkrp_partition(T, kTPer, stream, &part);
    if (st != SP_OK) return st;
    const unsigned blocks = (unsigned)sp_ceil_div(part.nchunks * 32, kTThreads);
    SP_DISPATCH_WIDTHS(T, {
        k_mttkrp<P, I><<<blocks, kTThreads, 0, stream>>>(
            static_cast<const P*>(T->pos[1]), T->lt[0] == SP_COMPRESSED ? static_cast<const I*>(T->crd[0]) : nullptr,
            static_cast<const P*>(T->pos[2]), static_cast<const I*>(T->crd[1]), static_cast<const I*>(T->crd[2]),
            T->val, F1, F2, R, M, part.row, part.nz, part.aux, part.nchunks, T->npos[1] - 1, T->ncrd[1]);
    });
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    return SP_OK;
}
