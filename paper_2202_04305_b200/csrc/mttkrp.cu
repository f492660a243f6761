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

#include <limits.h>

namespace {

constexpr int kTThreads = 256;
constexpr int kTPer = 512;   // entries per warp

// One nnz batch = up to 32 consecutive entries held one per lane (coordinate, value).
// The ends of the fibres that fall inside the batch are turned into a 32-bit mask, so the
// per-entry loop is fully unrolled with static lane indices: all factor-row loads of a group
// of kGroup entries (and the level-1 factor row of every fibre that ends in the group) are
// issued before the first multiply-add that needs them.
constexpr int kGroup = 8;

template <typename P, typename I>
__global__ void __launch_bounds__(kTThreads)
k_mttkrp(const P* __restrict__ pos1, const I* __restrict__ crd0, const P* __restrict__ pos2,
         const I* __restrict__ crd1, const I* __restrict__ crd2, const double* __restrict__ val,
         const double* __restrict__ F1, const double* __restrict__ F2, int64_t R, double* __restrict__ M,
         const int64_t* __restrict__ pfiber, const int64_t* __restrict__ pnz, const int64_t* __restrict__ pslice,
         int64_t nchunks, int64_t nslice, int64_t nfiber, int64_t d0, int64_t d1, int64_t d2) {
    // d0, d1, d2: rows of M, F1, F2 (used by the bounds-checking debug build only)
    // open-slice sums of the block's warps: slot 2*warp = the slice the warp's range starts in,
    // slot 2*warp+1 = the slice it ends in (when different); equal neighbours are added here so
    // that a slice spanning the whole block costs one atomic add per column, not one per warp
    __shared__ double s_car[2 * kTThreads / 32][32];
    __shared__ long long s_id[2 * kTThreads / 32];
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    const bool live = w < nchunks;
    const int64_t p0 = live ? pnz[w] : 0, p1 = live ? pnz[w + 1] : 0;
    constexpr int64_t kInf = INT64_MAX;

    for (int64_t rb = 0; rb < R; rb += 32) {
        const bool on = rb + lane < R;
        const int64_t r = on ? rb + lane : rb;      // idle lanes read column rb and never write
        const double* F1r = F1 + r;
        const double* F2r = F2 + r;
        int64_t f = live ? pfiber[w] : 0, s = live ? pslice[w] : 0, p = p0, fb = f;
        int64_t send = (p1 > p0) ? (int64_t)pos1[s + 1] : kInf;
        long long head_id = -1, tail_id = -1;
        double head_v = 0.0, tail_v = 0.0;
        int64_t last_flush = p0;                    // entries before this index are already in M
        double accf = 0.0, accs = 0.0;
        bool first = true;
        int64_t fe_l = (p1 > p0 && fb + lane < nfiber) ? (int64_t)pos2[fb + lane + 1] : kInf;
        I j_l = (p1 > p0 && fb + lane < nfiber) ? crd1[fb + lane] : (I)0;

        while (p < p1) {
            const int64_t fe_last = __shfl_sync(0xffffffffu, fe_l, 31);
            int64_t lim = p1 - p;
            if (fe_last - p < lim) lim = fe_last - p;
            const int cnt = lim < 32 ? (int)lim : 32;
            const I k_l = (lane < cnt) ? crd2[p + lane] : (I)0;
            const double v_l = (lane < cnt) ? val[p + lane] : 0.0;
            const int64_t rel = fe_l - p - 1;
            const unsigned endmask = __reduce_or_sync(0xffffffffu, (rel >= 0 && rel < cnt) ? (1u << (int)rel) : 0u);
            const int fi0 = (int)(f - fb);          // fibre (within the register batch) of the batch's first entry

#pragma unroll
            for (int g = 0; g < 32 / kGroup; ++g) {
                if (g * kGroup < cnt) {
                    double c[kGroup], b[kGroup];
#pragma unroll
                    for (int u = 0; u < kGroup; ++u) {
                        const int t = g * kGroup + u;
                        c[u] = 0.0; b[u] = 0.0;
                        if (t < cnt) {
                            const int64_t k = SP_IDX(__shfl_sync(0xffffffffu, k_l, t), d2);
                            c[u] = F2r[k * R];
                            if ((endmask >> t) & 1u) {
                                const int fi = fi0 + __popc(endmask & ((1u << t) - 1u));
                                const int64_t j = SP_IDX(__shfl_sync(0xffffffffu, j_l, fi), d1);
                                b[u] = F1r[j * R];
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < kGroup; ++u) {
                        const int t = g * kGroup + u;
                        if (t < cnt) {
                            const double v = __shfl_sync(0xffffffffu, v_l, t);
                            accf = fma(v, c[u], accf);
                            if ((endmask >> t) & 1u) {              // the fibre is complete
                                accs = fma(b[u], accf, accs);
                                accf = 0.0;
                                ++f;
                                if (f == send) {                    // and so is the slice
                                    const int64_t i = SP_IDX(crd0 ? (int64_t)crd0[s] : s, d0);
                                    if (first) { head_id = i; head_v = accs; }
                                    else if (on) M[i * R + r] = accs;
                                    first = false;
                                    last_flush = p + t + 1;
                                    accs = 0.0;
                                    ++s;
                                    while (s < nslice && (int64_t)pos1[s + 1] == f) ++s;   // slices with no fibres
                                    send = s < nslice ? (int64_t)pos1[s + 1] : kInf;
                                }
                            }
                        }
                    }
                }
            }
            p += cnt;
            if (f - fb == 32) {
                fb = f;
                fe_l = (fb + lane < nfiber) ? (int64_t)pos2[fb + lane + 1] : kInf;
                j_l = (fb + lane < nfiber) ? crd1[fb + lane] : (I)0;
            }
        }
        if (p1 > last_flush) {                      // the range ends inside slice s
            if (f < nfiber && (int64_t)pos2[f] < p1) {   // ... and inside fibre f
                const double bj = F1r[SP_IDX(crd1[f], d1) * R];
                accs = fma(bj, accf, accs);
            }
            const int64_t i = SP_IDX(crd0 ? (int64_t)crd0[s] : s, d0);
            if (first) { head_id = i; head_v = accs; }
            else { tail_id = i; tail_v = accs; }
        }
        s_car[2 * wi][lane] = head_v;
        s_car[2 * wi + 1][lane] = tail_v;
        if (lane == 0) { s_id[2 * wi] = head_id; s_id[2 * wi + 1] = tail_id; }
        __syncthreads();
        constexpr int kSlots = 2 * kTThreads / 32;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e = 2 * wi + h;
            const long long id = s_id[e];
            if (id < 0) continue;
            int q = e - 1;
            while (q >= 0 && s_id[q] < 0) --q;
            if (q >= 0 && s_id[q] == id) continue;          // an earlier slot leads this run
            double sum = s_car[e][lane];
            for (int u = e + 1; u < kSlots; ++u) {
                const long long d = s_id[u];
                if (d < 0) continue;
                if (d != id) break;
                sum += s_car[u][lane];
            }
            if (on) atomicAdd(M + id * R + r, sum);
        }
        __syncthreads();
    }
}


// ---------------------------------------------------------------------------------------------
// Fast path (R a multiple of S, factor rows 16-byte aligned, dim * R < 2^31).
//
// A warp walks its entry range 32 entries at a time.  Each lane first prepares one entry of the
// batch - the element offset of its leaf factor row, the element offset of the level-1 factor row
// of the fibre it lies in, and whether a fibre sum must be closed after it - and parks that in
// shared memory.  The warp then splits into S groups of 32/S lanes; group g consumes the 32/S
// consecutive entries g*32/S .. of the batch, and a lane owns S adjacent output columns, so a
// group fetches a whole 32-column factor row with one (S = 2) or two (S = 4) 16-byte loads per
// lane.  Closing a fibre is accs += F1[j,:] * accf, written branch-free (a row of zeros when no
// close is due).  Every group closes its open partial sum at the end of its entries - sums are
// linear, so a fibre may be closed in pieces - which keeps the inner loop free of any cross-batch
// fibre state.  Batches never straddle a slice end.
struct __align__(16) Staged {
    uint32_t koff;   // leaf factor row offset (elements)
    uint32_t bw;     // (level-1 factor row offset << 1) | close-after-this-entry
    double v;
};

constexpr int kFastPer = 1024;   // entries per warp

// A lane's S columns are S/2 pairs; pair n sits at column offset coff[n] of the 32-column tile,
// laid out so that the lanes of a group read one contiguous run per 16-byte load.
// W256 (S = 4, all 32 columns in use, 32-byte aligned rows): the lane's four columns are adjacent and
// come with one 32-byte load, which halves the load instructions and their address arithmetic.
template <int S, bool W256>
__device__ __forceinline__ void ld_cols(const double* p, const int* coff, double* a) {
    if (W256) {
        asm volatile("ld.global.nc.v4.f64 {%0,%1,%2,%3}, [%4];"
                     : "=d"(a[0]), "=d"(a[1]), "=d"(a[S > 2 ? 2 : 0]), "=d"(a[S > 3 ? 3 : 0])
                     : "l"(p + coff[0]));
        return;
    }
#pragma unroll
    for (int q = 0; q < S; q += 2) {
        const double2 t = *reinterpret_cast<const double2*>(p + coff[q / 2]);
        a[q] = t.x;
        a[q + 1] = t.y;
    }
}

// Two warps per block, eight blocks per SM: the same 16 warps per SM as 256 x 2 (126 registers a thread
// either way), but a block's warps share nothing until the final combine of their open slices, and
// small blocks finish and are replaced more evenly: 0.527 ms against 0.555 ms on the 20,000,000-entry
// tensor (128 x 4: 0.533, 32 x 16: 0.528, 512 x 1: 0.583).
#ifndef SP_MTTKRP_FAST_THREADS
#define SP_MTTKRP_FAST_THREADS 64
#endif
#ifndef SP_LB_MTTKRP
#define SP_LB_MTTKRP (512 / SP_MTTKRP_FAST_THREADS)
#endif
constexpr int kFThreads = SP_MTTKRP_FAST_THREADS;
template <typename P, typename I, int S, bool W256>
__global__ void __launch_bounds__(kFThreads, SP_LB_MTTKRP)
k_mttkrp_fast(const P* __restrict__ pos1, const I* __restrict__ crd0, const P* __restrict__ pos2,
              const I* __restrict__ crd1, const I* __restrict__ crd2, const double* __restrict__ val,
              const double* __restrict__ F1, const double* __restrict__ F2, int64_t R, double* __restrict__ M,
              const int64_t* __restrict__ pfiber, const int64_t* __restrict__ pnz,
              const int64_t* __restrict__ pslice, int64_t nchunks, int64_t nslice, int64_t nfiber,
              int64_t d0, int64_t d1, int64_t d2) {
    constexpr int GL = 32 / S;      // lanes per group = entries per group and batch
    constexpr int kStepGroup = S == 2 ? 4 : 2;
    constexpr int kWarps = kFThreads / 32;
    __shared__ Staged s_st[kWarps][32];
    __shared__ double s_car[2 * kWarps][32];
    __shared__ long long s_id[2 * kWarps];
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5, g = lane / GL, hl = lane % GL;
    const bool live = w < nchunks;
    const int64_t p0 = live ? pnz[w] : 0, p1 = live ? pnz[w + 1] : 0;
    const bool work = p1 > p0;
    constexpr int64_t kInf = INT64_MAX;
    const uint32_t Ru = (uint32_t)R;

    for (int64_t rb = 0; rb < R; rb += 32) {
        int coff[S / 2];
        bool on[S / 2];
#pragma unroll
        for (int n = 0; n < S / 2; ++n) {
            const int c0 = W256 ? 4 * hl + 2 * n : n * 2 * GL + 2 * hl;
            on[n] = rb + c0 < R;
            coff[n] = on[n] ? c0 : 0;          // idle lanes read column rb and never write
        }
        const double* F1g = F1 + rb;
        const double* F2g = F2 + rb;
        int64_t f = work ? pfiber[w] : 0, s = work ? pslice[w] : 0, p = p0, fb = f;
        int64_t send = work ? (int64_t)pos1[s + 1] : 0;
        int64_t slice_end = work ? (int64_t)pos2[send] : kInf;   // entry index at which slice s ends
        long long head_id = -1, tail_id = -1;
        double head_v[S], tail_v[S], accs[S];
#pragma unroll
        for (int q = 0; q < S; ++q) { head_v[q] = 0.0; tail_v[q] = 0.0; accs[q] = 0.0; }
        bool first = true;
        int64_t last_flush = p0;
        // three windows of 32 fibres: ends and level-1 coordinates (the third is a prefetch)
        int64_t feA = kInf, feB = kInf, feC = kInf;
        I jA = 0, jB = 0, jC = 0;
        if (work) {
            if (fb + lane < nfiber) { feA = (int64_t)pos2[fb + lane + 1]; jA = crd1[fb + lane]; }
            if (fb + 32 + lane < nfiber) { feB = (int64_t)pos2[fb + 32 + lane + 1]; jB = crd1[fb + 32 + lane]; }
            if (fb + 64 + lane < nfiber) { feC = (int64_t)pos2[fb + 64 + lane + 1]; jC = crd1[fb + 64 + lane]; }
        }
        uint32_t k_n = (p + lane < p1) ? (uint32_t)crd2[p + lane] : 0u;
        double v_n = (p + lane < p1) ? val[p + lane] : 0.0;

        auto fold_groups = [&]() {       // add the S groups' slice sums into group 0's lanes
#pragma unroll
            for (int o = GL; o < 32; o <<= 1)
#pragma unroll
                for (int q = 0; q < S; ++q) accs[q] += __shfl_xor_sync(0xffffffffu, accs[q], o);
        };

        while (p < p1) {
            int64_t lim = p1 - p;
            if (slice_end - p < lim) lim = slice_end - p;
            const int cnt = lim < 32 ? (int)lim : 32;
            const uint32_t k_l = k_n;
            const double v_l = v_n;
            {
                const int64_t pn = p + cnt;
                k_n = (pn + lane < p1) ? (uint32_t)crd2[pn + lane] : 0u;
                v_n = (pn + lane < p1) ? val[pn + lane] : 0.0;
            }
            const int64_t relA = feA - p - 1, relB = feB - p - 1;
            const unsigned endmask = __reduce_or_sync(
                0xffffffffu, ((relA >= 0 && relA < cnt) ? (1u << (int)relA) : 0u) |
                                 ((relB >= 0 && relB < cnt) ? (1u << (int)relB) : 0u));
            const int fi = (int)(f - fb) + __popc(endmask & ((1u << lane) - 1u));
            const I ja = __shfl_sync(0xffffffffu, jA, fi & 31);
            const I jb = __shfl_sync(0xffffffffu, jB, fi & 31);
            const uint32_t j = (uint32_t)SP_IDX(fi < 32 ? ja : jb, d1);
            const bool valid = lane < cnt;
            const bool close = valid && (((endmask >> lane) & 1u) || lane == cnt - 1 || hl == GL - 1);
            Staged st;
            st.koff = valid ? (uint32_t)SP_IDX(k_l, d2) * Ru : 0u;
            st.bw = valid ? (((j * Ru) << 1) | (close ? 1u : 0u)) : 0u;
            st.v = valid ? v_l : 0.0;
            // entry e = g * GL + t is parked at slot t * S + g: the S groups read step t's entries from one
            // 16 * S-byte run (one shared-memory wavefront, where slots g * GL + t cost S: same banks)
            s_st[wi][(lane % GL) * S + lane / GL] = st;
            __syncwarp();

            double accf[S];
#pragma unroll
            for (int q = 0; q < S; ++q) accf[q] = 0.0;
            const Staged* mine = &s_st[wi][g];
#pragma unroll
            for (int t0 = 0; t0 < GL; t0 += kStepGroup) {
                // Note: no double is set to a constant zero in this loop.  Zeroing a 64-bit register
                // pair is issued on a narrow pipe that saturates long before the loads do; a closed
                // sum is cleared by masking its bits with integer ops instead, and the level-1 row is
                // read only under the same predicate that consumes it.
                Staged e[kStepGroup];
                double c[kStepGroup][S], b[kStepGroup][S];
#pragma unroll
                for (int u = 0; u < kStepGroup; ++u) {
                    e[u] = mine[(t0 + u) * S];
                    ld_cols<S, W256>(F2g + e[u].koff, coff, c[u]);
                    if (e[u].bw & 1u) ld_cols<S, W256>(F1g + (e[u].bw >> 1), coff, b[u]);
                }
#pragma unroll
                for (int u = 0; u < kStepGroup; ++u) {
                    const bool cl = e[u].bw & 1u;
                    const long long keep = (long long)(int)((e[u].bw & 1u) - 1u);   // all ones, or 0 after a close
#pragma unroll
                    for (int q = 0; q < S; ++q) {
                        accf[q] = fma(e[u].v, c[u][q], accf[q]);
                        if (cl) accs[q] = fma(b[u][q], accf[q], accs[q]);
                        accf[q] = __longlong_as_double(__double_as_longlong(accf[q]) & keep);
                    }
                }
            }
            __syncwarp();
            f += __popc(endmask);
            p += cnt;
            if (p == slice_end) {                    // slice s is complete: all groups' sums -> row i
                fold_groups();
                const int64_t i = SP_IDX(crd0 ? (int64_t)crd0[s] : s, d0);
                if (first) {
                    head_id = i;
#pragma unroll
                    for (int q = 0; q < S; ++q) head_v[q] = accs[q];
                } else if (g == 0) {
#pragma unroll
                    for (int q = 0; q < S; q += 2)
                        if (on[q / 2])
                            *reinterpret_cast<double2*>(M + i * R + rb + coff[q / 2]) = make_double2(accs[q], accs[q + 1]);
                }
                first = false;
                last_flush = p;
#pragma unroll
                for (int q = 0; q < S; ++q) accs[q] = 0.0;
                ++s;
                while (s < nslice && (int64_t)pos1[s + 1] == f) ++s;   // slices with no fibres
                if (s < nslice) { send = (int64_t)pos1[s + 1]; slice_end = (int64_t)pos2[send]; }
                else slice_end = kInf;
            }
            if (f - fb >= 32) {
                fb += 32;
                feA = feB; jA = jB; feB = feC; jB = jC;
                feC = kInf; jC = 0;
                if (fb + 64 + lane < nfiber) { feC = (int64_t)pos2[fb + 64 + lane + 1]; jC = crd1[fb + 64 + lane]; }
            }
        }
        if (p1 > last_flush) {                       // the range ends inside slice s
            fold_groups();
            const int64_t i = SP_IDX(crd0 ? (int64_t)crd0[s] : s, d0);
            if (first) {
                head_id = i;
#pragma unroll
                for (int q = 0; q < S; ++q) head_v[q] = accs[q];
            } else {
                tail_id = i;
#pragma unroll
                for (int q = 0; q < S; ++q) tail_v[q] = accs[q];
            }
        }
        if (g == 0) {
#pragma unroll
            for (int q = 0; q < S; ++q) {
                const int cc = (W256 ? 4 * hl + 2 * (q / 2) : (q / 2) * 2 * GL + 2 * hl) + (q & 1);
                s_car[2 * wi][cc] = head_v[q];
                s_car[2 * wi + 1][cc] = tail_v[q];
            }
        }
        if (lane == 0) { s_id[2 * wi] = head_id; s_id[2 * wi + 1] = tail_id; }
        __syncthreads();
        constexpr int kSlots = 2 * kWarps;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e = 2 * wi + h;
            const long long id = s_id[e];
            if (id < 0) continue;
            int q = e - 1;
            while (q >= 0 && s_id[q] < 0) --q;
            if (q >= 0 && s_id[q] == id) continue;
            double sum = s_car[e][lane];
            for (int u = e + 1; u < kSlots; ++u) {
                const long long d = s_id[u];
                if (d < 0) continue;
                if (d != id) break;
                sum += s_car[u][lane];
            }
            if (rb + lane < R) atomicAdd(M + id * R + rb + lane, sum);
        }
        __syncthreads();
    }
}

}  // namespace

// F1 / F2: factor matrices of the dimensions stored at levels 1 / 2; M: rows of the level-0 dimension.
static sp_status mttkrp_levels(sp_tensor* T, const double* F1, const double* F2, int64_t R, double* M, cudaStream_t stream);

extern "C" sp_status sp_mttkrp(sp_tensor* T, const double* B, const double* C, int64_t R, double* M, void* stream_) {
    SP_API_RANGE("sp_mttkrp");
    if (!T || !B || !C || !M || R < 1) return SP_ERR_INVALID_ARG;
    if (T->rank != 3 || T->ord[0] != 0 || T->lt[1] != SP_COMPRESSED || T->lt[2] != SP_COMPRESSED)
        return SP_ERR_UNSUPPORTED;
    return mttkrp_levels(T, T->ord[1] == 1 ? B : C, T->ord[1] == 1 ? C : B, R, M, static_cast<cudaStream_t>(stream_));
}

extern "C" sp_status sp_mttkrp_mode(sp_tensor* T, int mode, const double* const* factors, int64_t R, double* M,
                                    void* stream_) {
    SP_API_RANGE("sp_mttkrp_mode");
    if (!T || !factors || !M || R < 1 || mode < 0 || mode > 2) return SP_ERR_INVALID_ARG;
    if (T->rank != 3 || T->ord[0] != mode || T->lt[1] != SP_COMPRESSED || T->lt[2] != SP_COMPRESSED)
        return SP_ERR_UNSUPPORTED;
    const double* F1 = factors[T->ord[1]];
    const double* F2 = factors[T->ord[2]];
    if (!F1 || !F2) return SP_ERR_INVALID_ARG;
    return mttkrp_levels(T, F1, F2, R, M, static_cast<cudaStream_t>(stream_));
}

static sp_status mttkrp_levels(sp_tensor* T, const double* F1, const double* F2, int64_t R, double* M, cudaStream_t stream) {
    if (sp_check_device(T) != SP_OK) return SP_ERR_INVALID_ARG;
    {   // 8- and 16-bit storage is read through its 32-bit shadow
        sp_tensor* wide_ = nullptr;
        const sp_status ws_ = sp_widened(T, stream, &wide_);
        if (ws_ != SP_OK) return ws_;
        T = wide_;
    }
    const double* B = F1;
    const double* C = F2;
    SP_CUDA(cudaMemsetAsync(M, 0, (size_t)T->dims[T->ord[0]] * R * sizeof(double), stream));
    const int64_t nnz = T->ncrd[2];
    if (nnz == 0) return SP_OK;
    const int64_t d1 = T->dims[T->ord[1]], d2 = T->dims[T->ord[2]];
    const int64_t maxdim = d1 > d2 ? d1 : d2;
    const bool fast = (R % 2 == 0) && maxdim * R < ((int64_t)1 << 31) && reinterpret_cast<uintptr_t>(B) % 16 == 0 &&
                      reinterpret_cast<uintptr_t>(C) % 16 == 0 && reinterpret_cast<uintptr_t>(M) % 16 == 0;
    sp_partition part;
    sp_status st = sp_get_mttkrp_partition(T, fast ? kFastPer : kTPer, stream, &part);
    if (st != SP_OK) return st;
    const unsigned blocks = (unsigned)sp_ceil_div(part.nchunks * 32, fast ? kFThreads : kTThreads);
    if (fast) {
#define SP_MTTKRP_FAST(S, W)                                                                                           \
    k_mttkrp_fast<P, I, S, W><<<blocks, kFThreads, 0, stream>>>(                                                       \
        static_cast<const P*>(T->pos[1]), T->lt[0] == SP_COMPRESSED ? static_cast<const I*>(T->crd[0]) : nullptr,      \
        static_cast<const P*>(T->pos[2]), static_cast<const I*>(T->crd[1]), static_cast<const I*>(T->crd[2]), T->val,  \
        F1, F2, R, M, part.row, part.nz, part.aux, part.nchunks, T->npos[1] - 1, T->ncrd[1], T->dims[T->ord[0]], d1, d2)
        // one 32-byte load per lane and factor row when every lane has its four columns and rows are 32-byte aligned
        const bool w256 = R % 32 == 0 && reinterpret_cast<uintptr_t>(F1) % 32 == 0 && reinterpret_cast<uintptr_t>(F2) % 32 == 0;
        SP_DISPATCH_WIDTHS(T, {
            if (w256) SP_MTTKRP_FAST(4, true);
            else if (R % 4 == 0) SP_MTTKRP_FAST(4, false);
            else SP_MTTKRP_FAST(2, false);
        });
#undef SP_MTTKRP_FAST
        SP_LAUNCH_CHECK();
        sp_count_launches(1);
        SP_BOUNDS_RETURN(stream);
        return SP_OK;
    }
    SP_DISPATCH_WIDTHS(T, {
        k_mttkrp<P, I><<<blocks, kTThreads, 0, stream>>>(
            static_cast<const P*>(T->pos[1]), T->lt[0] == SP_COMPRESSED ? static_cast<const I*>(T->crd[0]) : nullptr,
            static_cast<const P*>(T->pos[2]), static_cast<const I*>(T->crd[1]), static_cast<const I*>(T->crd[2]),
            T->val, F1, F2, R, M, part.row, part.nz, part.aux, part.nchunks, T->npos[1] - 1, T->ncrd[1],
            T->dims[T->ord[0]], d1, d2);
    });
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    SP_BOUNDS_RETURN(stream);
    return SP_OK;
}
