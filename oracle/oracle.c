/*
 * CPU oracle: test infrastructure only.
 *
 * A plain, slow, single-threaded restatement of what the sparse path computes,
 * written from the paper (arXiv 2202.04305) and sharing nothing with the CUDA
 * library.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it; no product code path does.
 *
 *   - orc_pack / orc_unpack follow Section 4.1: per-level "dense" or
 *     "compressed" types, a dimension ordering, and the storage scheme of
 *     pointers[l][*], indices[l][*], values[*] that the section's five worked
 *     examples spell out (sparse vector, CSR, compressed-dense, DCSC, 3-d
 *     all-compressed), reached through a coordinate list as Section 4.2 says
 *     conversions are.
 *   - orc_spmv / orc_spmm / orc_sddmm / orc_mttkrp evaluate the tensor index
 *     expressions of Sections 1, 6.2 and 6.3 term by term over the coordinate
 *     list (the sparse code only skips terms that are zero, Section 2.1), in
 *     x87 extended precision, together with the per-entry bound sum |a*b|
 *     against which the f64 result of any summation order is judged.
 *
 *   - orc_par_* are the same products written as the loop nests Section 4.3
 *     derives over packed storage (outer loop over stored rows / slices, inner
 *     loops over pos[l][p] .. pos[l][p+1]), with the outer loop split over all
 *     host cores by OpenMP: the "oracle, N cores" leg of the CPU baseline.  They
 *     are pinned by the coordinate-loop functions above them.
 *
 * Readings where the paper is silent:
 *   - dimOrdering: result l of the affine map names the logical dimension
 *     stored at level l ("parity unpinned" by the paper for 3-cycles: all its
 *     examples are swaps; pinned here only by round trip and dense brute force).
 *   - duplicate coordinates are summed in input order; explicit zeros are kept.
 *   - bit widths are not modelled: every position and coordinate is int64.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORC_MAX_RANK 8
enum { ORC_DENSE = 0, ORC_COMPRESSED = 1 };

typedef struct {
    int rank;
    int64_t npos[ORC_MAX_RANK];   /* 0 for dense levels */
    int64_t ncrd[ORC_MAX_RANK];
    int64_t *pos[ORC_MAX_RANK];
    int64_t *crd[ORC_MAX_RANK];
    int64_t nval;
    double *val;
    int64_t *entry_pos;           /* storage position of each input entry */
} orc_storage;

/* ---- step 2 of the packer: lexicographic order of level coordinates ---- */
static int g_rank;
static const int64_t *g_lvl[ORC_MAX_RANK];

static int cmp_entries(const void *pa, const void *pb)
{
    int64_t a = *(const int64_t *)pa, b = *(const int64_t *)pb;
    for (int l = 0; l < g_rank; ++l) {
        int64_t ca = g_lvl[l][a], cb = g_lvl[l][b];
        if (ca != cb) return ca < cb ? -1 : 1;
    }
    return a < b ? -1 : (a > b ? 1 : 0);   /* equal coordinates keep input order */
}

void orc_free_storage(orc_storage *s)
{
    if (!s) return;
    for (int l = 0; l < ORC_MAX_RANK; ++l) { free(s->pos[l]); free(s->crd[l]); }
    free(s->val); free(s->entry_pos);
    memset(s, 0, sizeof *s);
}

/*
 * Section 4.1 storage construction.
 * coords[d] = coordinate array of logical dimension d (nnz entries each).
 * lt[l], ord[l] are per level: ord[l] = logical dimension stored at level l.
 * Returns 0, or -1 bad argument, -2 coordinate out of range, -3 out of memory.
 */
int orc_pack(int rank, const int64_t *dims, int64_t nnz, const int64_t *const *coords,
             const double *vals, const int *lt, const int *ord, orc_storage *out)
{
    memset(out, 0, sizeof *out);
    if (rank < 1 || rank > ORC_MAX_RANK || nnz < 0) return -1;
    int seen[ORC_MAX_RANK] = {0};
    for (int l = 0; l < rank; ++l) {
        if (ord[l] < 0 || ord[l] >= rank || seen[ord[l]]) return -1;
        seen[ord[l]] = 1;
        if (lt[l] != ORC_DENSE && lt[l] != ORC_COMPRESSED) return -1;
    }
    int64_t sz[ORC_MAX_RANK];
    for (int l = 0; l < rank; ++l) {          /* step 1: level sizes and level coordinates */
        sz[l] = dims[ord[l]];
        g_lvl[l] = coords[ord[l]];
        for (int64_t e = 0; e < nnz; ++e)
            if (g_lvl[l][e] < 0 || g_lvl[l][e] >= sz[l]) return -2;
    }
    out->rank = rank;
    int64_t *perm = malloc(sizeof(int64_t) * (size_t)(nnz + 1));
    int64_t *ppos = malloc(sizeof(int64_t) * (size_t)(nnz + 1));   /* per sorted entry */
    int64_t *npp  = malloc(sizeof(int64_t) * (size_t)(nnz + 1));
    double  *sval = malloc(sizeof(double)  * (size_t)(nnz + 1));
    int64_t *rep  = malloc(sizeof(int64_t) * (size_t)(nnz + 1));   /* merged entry of each sorted entry */
    out->entry_pos = malloc(sizeof(int64_t) * (size_t)(nnz + 1));
    if (!perm || !ppos || !npp || !sval || !rep || !out->entry_pos) return -3;
    for (int64_t e = 0; e < nnz; ++e) perm[e] = e;
    g_rank = rank;
    qsort(perm, (size_t)nnz, sizeof(int64_t), cmp_entries);   /* step 2 */
    int64_t *order = malloc(sizeof(int64_t) * (size_t)(nnz + 1));
    if (!order) return -3;
    memcpy(order, perm, sizeof(int64_t) * (size_t)nnz);

    /* step 3: entries with identical coordinates become one, summed in input order */
    int64_t u = 0;
    for (int64_t e = 0; e < nnz; ++e) {
        int same = e > 0;
        for (int l = 0; same && l < rank; ++l)
            same = g_lvl[l][perm[e]] == g_lvl[l][perm[e - 1]];
        if (same) { sval[u - 1] += vals[perm[e]]; }
        else { perm[u] = perm[e]; sval[u] = vals[perm[e]]; ++u; }
        rep[e] = u - 1;
    }
    /* perm[0..u) now lists one representative per distinct coordinate, sorted;
       order[] keeps the full sorted list and rep[e] the merged slot of order[e]. */

    /* step 4: levels top-down */
    int64_t parents = 1;
    for (int64_t e = 0; e < u; ++e) ppos[e] = 0;
    for (int l = 0; l < rank; ++l) {
        const int64_t *c = g_lvl[l];
        if (lt[l] == ORC_DENSE) {
            for (int64_t e = 0; e < u; ++e) ppos[e] = ppos[e] * sz[l] + c[perm[e]];
            parents *= sz[l];
        } else {
            int64_t *pos = calloc((size_t)(parents + 1), sizeof(int64_t));
            int64_t *crd = malloc(sizeof(int64_t) * (size_t)(u + 1));
            if (!pos || !crd) return -3;
            int64_t nodes = 0;
            for (int64_t e = 0; e < u; ++e) {
                int fresh = e == 0 || ppos[e] != ppos[e - 1] || c[perm[e]] != c[perm[e - 1]];
                if (fresh) {
                    crd[nodes] = c[perm[e]];
                    pos[ppos[e] + 1] += 1;          /* one more node under this parent */
                    ++nodes;
                }
                npp[e] = nodes - 1;
            }
            for (int64_t p = 0; p < parents; ++p) pos[p + 1] += pos[p];   /* counts -> offsets */
            for (int64_t e = 0; e < u; ++e) ppos[e] = npp[e];
            out->pos[l] = pos; out->npos[l] = parents + 1;
            out->crd[l] = crd; out->ncrd[l] = nodes;
            parents = nodes;
        }
    }
    /* step 5: values */
    out->nval = parents;
    out->val = calloc((size_t)(parents + 1), sizeof(double));
    if (!out->val) return -3;
    for (int64_t e = 0; e < u; ++e) out->val[ppos[e]] = sval[e];

    /* storage position of every original entry */
    for (int64_t e = 0; e < nnz; ++e) out->entry_pos[order[e]] = ppos[rep[e]];
    free(order);
    free(perm); free(ppos); free(npp); free(sval); free(rep);
    return 0;
}

/*
 * Inverse of the storage scheme: enumerate stored positions depth-first and
 * emit logical coordinates with the stored value (explicit zeros included).
 * coords_out[d] must hold nval entries each.  Returns the number emitted.
 */
static int64_t unpack_rec(const orc_storage *s, const int64_t *dims, const int *lt, const int *ord,
                          int l, int64_t ppos, int64_t *lvlc, int64_t *const *coords_out,
                          double *vals_out, int64_t n)
{
    if (l == s->rank) {
        for (int k = 0; k < s->rank; ++k) coords_out[ord[k]][n] = lvlc[k];
        vals_out[n] = s->val[ppos];
        return n + 1;
    }
    if (lt[l] == ORC_DENSE) {
        int64_t size = dims[ord[l]];
        for (int64_t c = 0; c < size; ++c) {
            lvlc[l] = c;
            n = unpack_rec(s, dims, lt, ord, l + 1, ppos * size + c, lvlc, coords_out, vals_out, n);
        }
    } else {
        for (int64_t q = s->pos[l][ppos]; q < s->pos[l][ppos + 1]; ++q) {
            lvlc[l] = s->crd[l][q];
            n = unpack_rec(s, dims, lt, ord, l + 1, q, lvlc, coords_out, vals_out, n);
        }
    }
    return n;
}

int64_t orc_unpack(const orc_storage *s, const int64_t *dims, const int *lt, const int *ord,
                   int64_t *const *coords_out, double *vals_out)
{
    int64_t lvlc[ORC_MAX_RANK];
    return unpack_rec(s, dims, lt, ord, 0, 0, lvlc, coords_out, vals_out, 0);
}

/* ------------------------------------------------------------------------
 * Kernels: the index expression, one term per coordinate-list entry.
 * "slot" maps an output row to a slot of the (possibly sampled) result, or -1
 * to skip it; NULL means every row, slot = row.  Results and bounds are f64
 * roundings of extended-precision sums.
 * ---------------------------------------------------------------------- */

/* C[i,j] = sum_k A[i,k] * B[k,j]  (Section 1; matvec of Section 6.2 is N = 1). */
int orc_spmm(int64_t nnz, const int64_t *ai, const int64_t *ak, const double *av,
             const double *B, int64_t N, int64_t ldb,
             const int64_t *slot, int64_t nslots, double *C, double *bound)
{
    size_t tot = (size_t)nslots * (size_t)N;
    long double *acc = calloc(tot + 1, sizeof(long double));
    long double *bnd = calloc(tot + 1, sizeof(long double));
    if (!acc || !bnd) { free(acc); free(bnd); return -3; }
    for (int64_t e = 0; e < nnz; ++e) {
        int64_t s = slot ? slot[ai[e]] : ai[e];
        if (s < 0) continue;
        const double *brow = B + ak[e] * ldb;
        for (int64_t j = 0; j < N; ++j) {
            long double t = (long double)av[e] * (long double)brow[j];
            acc[s * N + j] += t;
            bnd[s * N + j] += fabsl(t);
        }
    }
    for (size_t q = 0; q < tot; ++q) { C[q] = (double)acc[q]; bound[q] = (double)bnd[q]; }
    free(acc); free(bnd);
    return 0;
}

/* X[i,j] = S[i,j] * sum_k A[i,k] * B[k,j] for the listed entries of S (Section 6.2). */
int orc_sddmm(int64_t nnz, const int64_t *si, const int64_t *sj, const double *sv,
              const double *A, int64_t lda, const double *B, int64_t ldb, int64_t K,
              double *x, double *bound)
{
    for (int64_t e = 0; e < nnz; ++e) {
        long double dot = 0.0L, ab = 0.0L;
        for (int64_t k = 0; k < K; ++k) {
            long double t = (long double)A[si[e] * lda + k] * (long double)B[k * ldb + sj[e]];
            dot += t;
            ab += fabsl(t);
        }
        x[e] = (double)((long double)sv[e] * dot);
        bound[e] = (double)(fabsl((long double)sv[e]) * ab);
    }
    return 0;
}

/* M[i,r] = sum_{j,k} T[i,j,k] * B[j,r] * C[k,r]  (Section 6.3, with the paper's
   A, B, C, D renamed M, T, C(middle mode), and last-mode factor). */
int orc_mttkrp(int64_t nnz, const int64_t *ti, const int64_t *tj, const int64_t *tk, const double *tv,
               const double *B, const double *Cf, int64_t R,
               const int64_t *slot, int64_t nslots, double *M, double *bound)
{
    size_t tot = (size_t)nslots * (size_t)R;
    long double *acc = calloc(tot + 1, sizeof(long double));
    long double *bnd = calloc(tot + 1, sizeof(long double));
    if (!acc || !bnd) { free(acc); free(bnd); return -3; }
    for (int64_t e = 0; e < nnz; ++e) {
        int64_t s = slot ? slot[ti[e]] : ti[e];
        if (s < 0) continue;
        for (int64_t r = 0; r < R; ++r) {
            long double t = (long double)tv[e] * (long double)B[tj[e] * R + r] * (long double)Cf[tk[e] * R + r];
            acc[s * R + r] += t;
            bnd[s * R + r] += fabsl(t);
        }
    }
    for (size_t q = 0; q < tot; ++q) { M[q] = (double)acc[q]; bound[q] = (double)bnd[q]; }
    free(acc); free(bnd);
    return 0;
}

/* ------------------------------------------------------------------------
 * SpMSpM: C[i,j] = sum_k A[i,k] * B[k,j] with A, B and C all sparse (Section 4.3's
 * kernel; Section 6.2, Table 2).  Inputs are coordinate lists; the result is returned
 * row by row in increasing (i, j) order: every (i, j) for which some k has both
 * A[i,k] and B[k,j] stored is an entry of C, even if its value cancels to zero.
 * Pass 1 (crd_out == NULL) only counts; pass 2 fills.  Returns the entry count or -3.
 * ---------------------------------------------------------------------- */
static int cmp_i64(const void *a, const void *b)
{
    int64_t x = *(const int64_t *)a, y = *(const int64_t *)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}

int64_t orc_spmspm(int64_t m, int64_t kdim, int64_t n,
                   int64_t annz, const int64_t *ai, const int64_t *ak, const double *av,
                   int64_t bnnz, const int64_t *bk, const int64_t *bj, const double *bv,
                   int64_t *pos_out /* m+1 */, int64_t *crd_out, double *val_out, double *bound_out)
{
    /* bucket the entries of A by row and of B by row (= k), keeping input order inside a bucket */
    int64_t *astart = calloc((size_t)m + 2, sizeof(int64_t)), *bstart = calloc((size_t)kdim + 2, sizeof(int64_t));
    int64_t *aord = malloc(sizeof(int64_t) * (size_t)(annz + 1)), *bord = malloc(sizeof(int64_t) * (size_t)(bnnz + 1));
    long double *ws = calloc((size_t)n + 1, sizeof(long double)), *wb = calloc((size_t)n + 1, sizeof(long double));
    char *mark = calloc((size_t)n + 1, 1);
    int64_t *added = malloc(sizeof(int64_t) * (size_t)(n + 1));
    if (!astart || !bstart || !aord || !bord || !ws || !wb || !mark || !added) return -3;
    for (int64_t e = 0; e < annz; ++e) astart[ai[e] + 1]++;
    for (int64_t e = 0; e < bnnz; ++e) bstart[bk[e] + 1]++;
    for (int64_t r = 0; r < m; ++r) astart[r + 1] += astart[r];
    for (int64_t r = 0; r < kdim; ++r) bstart[r + 1] += bstart[r];
    {
        int64_t *fill = calloc((size_t)(m > kdim ? m : kdim) + 1, sizeof(int64_t));
        if (!fill) return -3;
        for (int64_t e = 0; e < annz; ++e) aord[astart[ai[e]] + fill[ai[e]]++] = e;
        memset(fill, 0, sizeof(int64_t) * (size_t)((m > kdim ? m : kdim) + 1));
        for (int64_t e = 0; e < bnnz; ++e) bord[bstart[bk[e]] + fill[bk[e]]++] = e;
        free(fill);
    }
    int64_t total = 0;
    pos_out[0] = 0;
    for (int64_t i = 0; i < m; ++i) {
        int64_t count = 0;
        for (int64_t p = astart[i]; p < astart[i + 1]; ++p) {
            const int64_t ea = aord[p], k = ak[ea];
            for (int64_t q = bstart[k]; q < bstart[k + 1]; ++q) {
                const int64_t eb = bord[q], j = bj[eb];
                const long double t = (long double)av[ea] * (long double)bv[eb];
                if (!mark[j]) { mark[j] = 1; added[count++] = j; }     /* access pattern expansion */
                ws[j] += t;
                wb[j] += fabsl(t);
            }
        }
        qsort(added, (size_t)count, sizeof(int64_t), cmp_i64);          /* insertion in index order */
        for (int64_t c = 0; c < count; ++c) {
            const int64_t j = added[c];
            if (crd_out) { crd_out[total + c] = j; val_out[total + c] = (double)ws[j]; bound_out[total + c] = (double)wb[j]; }
            ws[j] = 0; wb[j] = 0; mark[j] = 0;
        }
        total += count;
        pos_out[i + 1] = total;
    }
    free(astart); free(bstart); free(aord); free(bord); free(ws); free(wb); free(mark); free(added);
    return total;
}

/* ------------------------------------------------------------------------
 * Sparse-sparse inner product x = sum_i a[i] * b[i] of two compressed vectors, by the
 * co-iteration of Section 4.3: both coordinate lists (sorted, as storage keeps them) are
 * walked together, the smaller index advances, and a product is formed only where the two
 * indices meet.  Returns the f64 rounding of the extended-precision sum; *bound = sum|a*b|.
 * ---------------------------------------------------------------------- */
double orc_vec_dot(int64_t na, const int64_t *ai, const double *av, int64_t nb, const int64_t *bi, const double *bv,
                   double *bound)
{
    long double acc = 0.0L, bnd = 0.0L;
    int64_t ia = 0, ib = 0;
    while (ia < na && ib < nb) {
        const int64_t ixa = ai[ia], ixb = bi[ib];
        const int64_t i = ixa < ixb ? ixa : ixb;
        if (ixa == i && ixb == i) {
            const long double t = (long double)av[ia] * (long double)bv[ib];
            acc += t;
            bnd += fabsl(t);
        }
        if (ixa == i) ++ia;
        if (ixb == i) ++ib;
    }
    if (bound) *bound = (double)bnd;
    return (double)acc;
}

/* ------------------------------------------------------------------------
 * The same products as loop nests over packed storage, outer loop in parallel
 * (OpenMP, static blocks of rows; rows are independent, so no atomics).
 * rowid: crd[0] when level 0 is compressed (stored row q is row rowid[q]), NULL
 * when it is dense (q is the row).  Outputs must be zero-filled by the caller
 * for rows that store nothing.  Each returns the number of threads used.
 * ---------------------------------------------------------------------- */
#ifdef _OPENMP
#include <omp.h>
#endif

static int threads_used(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* C[i,:] = sum_p val[p] * B[crd1[p],:] over p in pos1[q] .. pos1[q+1]  (Section 1's matmul, row-major A) */
int orc_par_spmm(int64_t nstored, const int64_t *rowid, const int64_t *pos1, const int64_t *crd1,
                 const double *val, const double *B, int64_t N, int64_t ldb, double *C, int64_t ldc)
{
#pragma omp parallel
    {
        long double *acc = malloc(sizeof(long double) * (size_t)(N + 1));
#pragma omp for schedule(static)
        for (int64_t q = 0; q < nstored; ++q) {
            for (int64_t j = 0; j < N; ++j) acc[j] = 0.0L;
            for (int64_t p = pos1[q]; p < pos1[q + 1]; ++p) {
                const double *brow = B + crd1[p] * ldb;
                for (int64_t j = 0; j < N; ++j) acc[j] += (long double)val[p] * (long double)brow[j];
            }
            double *crow = C + (rowid ? rowid[q] : q) * ldc;
            for (int64_t j = 0; j < N; ++j) crow[j] = (double)acc[j];
        }
        free(acc);
    }
    return threads_used();
}

/* x[p] = S.val[p] * sum_k A[i,k] * B[k,crd1[p]] for the stored entries of row-major S (Section 6.2) */
int orc_par_sddmm(int64_t nstored, const int64_t *rowid, const int64_t *pos1, const int64_t *crd1,
                  const double *sval, const double *A, int64_t lda, const double *B, int64_t ldb, int64_t K,
                  double *x)
{
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < nstored; ++q) {
        const double *arow = A + (rowid ? rowid[q] : q) * lda;
        for (int64_t p = pos1[q]; p < pos1[q + 1]; ++p) {
            long double dot = 0.0L;
            for (int64_t k = 0; k < K; ++k) dot += (long double)arow[k] * (long double)B[k * ldb + crd1[p]];
            x[p] = (double)((long double)sval[p] * dot);
        }
    }
    return threads_used();
}

/* M[i,:] = sum over fibres f of slice q, entries p of fibre f of val[p] * B[crd1[f],:] * C[crd2[p],:]
   (Section 6.3 over all-compressed storage; the three scalars are multiplied per entry, as in the expression) */
int orc_par_mttkrp(int64_t nslices, const int64_t *crd0, const int64_t *pos1, const int64_t *crd1,
                   const int64_t *pos2, const int64_t *crd2, const double *val,
                   const double *B, const double *Cf, int64_t R, double *M)
{
#pragma omp parallel
    {
        long double *acc = malloc(sizeof(long double) * (size_t)(R + 1));
#pragma omp for schedule(dynamic, 16)
        for (int64_t q = 0; q < nslices; ++q) {
            for (int64_t r = 0; r < R; ++r) acc[r] = 0.0L;
            for (int64_t f = pos1[q]; f < pos1[q + 1]; ++f) {
                const double *brow = B + crd1[f] * R;
                for (int64_t p = pos2[f]; p < pos2[f + 1]; ++p) {
                    const double *crow = Cf + crd2[p] * R;
                    for (int64_t r = 0; r < R; ++r)
                        acc[r] += (long double)val[p] * (long double)brow[r] * (long double)crow[r];
                }
            }
            double *mrow = M + (crd0 ? crd0[q] : q) * R;
            for (int64_t r = 0; r < R; ++r) mrow[r] = (double)acc[r];
        }
        free(acc);
    }
    return threads_used();
}
