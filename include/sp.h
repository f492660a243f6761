/*
 * sp.h - C ABI of the sparse tensor library (CUDA, sm_100a, one GPU).
 *
 * The calls follow the statement of the problem in "Compiler Support for Sparse
 * Tensor Computations in MLIR" (arXiv 2202.04305): a tensor is stored according
 * to an encoding (Section 4.1: per-level type dense | compressed, a dimension
 * ordering, and bit widths for pointers and indices) as the arrays
 * pointers[l][*], indices[l][*] and values[*]; storage is built from a
 * coordinate list (Section 4.2: conversions go through an intermediate
 * coordinate scheme); and the kernels are the tensor index expressions the
 * paper runs over that storage (Sections 1, 6.2, 6.3).
 *
 * Naming: "positions" = the paper's pointers, "coordinates" = its indices.
 * A "level" l is a storage level; dimOrdering[l] is the logical dimension kept
 * at level l.
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers owned by the caller unless the
 *     parameter says "host".  The library owns only what lives inside an
 *     sp_tensor (released by sp_free) and transient workspaces that it obtains
 *     and returns through the allocator (sp_set_allocator).
 *   - Dense operands are row-major f64 with a leading dimension in elements.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Kernel calls are asynchronous on it.  sp_pack synchronises the stream
 *     (the sizes of the level arrays depend on the data).
 *   - Kernels OVERWRITE their output.
 *   - Every call returns an sp_status; nothing throws across the boundary.
 *     An encoding a kernel does not handle yields SP_ERR_UNSUPPORTED, never a
 *     different algorithm on the host.
 *   - A handle is immutable after sp_pack.  Kernels cache read-only work-partition
 *     tables inside it on first use (under the handle's lock; that first call
 *     waits for the stream once, so the tables are complete for every stream
 *     afterwards); everything a call writes
 *     besides its output is scratch it takes from the allocator for that call, so
 *     calls on different streams or host threads may share a handle.  The handle
 *     must be used with the device it was packed on current
 *     (SP_ERR_INVALID_ARG otherwise).
 *   - CUDA graphs: once a kernel call has run on a handle (so its cached tables
 *     exist), later sp_spmv / sp_spmm / sp_sddmm / sp_mttkrp calls on it only
 *     enqueue stream-ordered work (kernels, memsets and allocator calls for
 *     their scratch) and may be stream-captured, provided the installed
 *     allocator is itself legal during capture (a stream-ordered or caching
 *     pool).  sp_pack, sp_convert, sp_unpack and sp_spmspm read sizes back to
 *     the host and cannot be captured.
 */
#ifndef SP_H
#define SP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SP_MAX_RANK 5

typedef struct sp_tensor sp_tensor;   /* opaque; owns device arrays */

typedef enum { SP_DENSE = 0, SP_COMPRESSED = 1 } sp_level_type;

typedef enum {
    SP_OK = 0,
    SP_ERR_INVALID_ARG = 1,     /* null pointer, bad rank, dimOrdering not a permutation, bad width */
    SP_ERR_UNSUPPORTED = 2,     /* encoding / shape not handled by this call */
    SP_ERR_OUT_OF_RANGE = 3,    /* a coordinate is < 0 or >= its dimension */
    SP_ERR_WIDTH_OVERFLOW = 4,  /* a position or coordinate does not fit the requested width */
    SP_ERR_DUPLICATE = 5,       /* SP_DUP_ERROR was set and two entries share coordinates */
    SP_ERR_ALLOC = 6,           /* the allocator returned NULL */
    SP_ERR_CUDA = 7,            /* a CUDA runtime call failed */
    SP_ERR_TIMEOUT = 8,         /* a bounded device-side wait ran out: an earlier sp_spmm launch whose operand
                                   tiles arrive by asynchronous copy gave up waiting for one; see sp_spmm */
    SP_ERR_TOO_LARGE = 9        /* the problem does not fit a fixed-capacity entry point (sp_spmv_static) */
} sp_status;

/* flags of sp_pack */
#define SP_DUP_SUM   0u   /* entries with equal coordinates are added, in input order (default) */
#define SP_DUP_ERROR 1u   /* ... are reported as SP_ERR_DUPLICATE instead */

const char* sp_status_string(sp_status s);

/*
 * Workspace and storage allocator.  alloc(bytes, stream, ctx) returns device
 * memory usable on `stream`; dealloc returns it.  Both NULL restores the
 * default (the device's stream-ordered pool: cudaMallocAsync / cudaFreeAsync).
 * Process-wide; set it before the first sp_pack and do not change it while
 * handles are alive.  When alloc returns NULL the call in progress gives back
 * everything it had taken and returns SP_ERR_ALLOC.
 */
sp_status sp_set_allocator(void* (*alloc)(size_t bytes, void* stream, void* ctx),
                           void (*dealloc)(void* ptr, void* stream, void* ctx), void* ctx);

/*
 * sp_pack - build the storage of Section 4.1 from an unsorted coordinate list
 * (Section 4.2: the sparse constant given as index tuples plus values, and
 * conversion through a coordinate scheme).
 *
 *   rank            1..SP_MAX_RANK
 *   dims            host, rank logical extents (each >= 1)
 *   nnz             number of entries (>= 0, < 2^32)
 *   coo_coords      host array of `rank` DEVICE pointers; coo_coords[d][e] is
 *                   entry e's coordinate in logical dimension d
 *   coo_coord_bits  32 (int32) or 64 (int64) element type of those arrays
 *   coo_vals        device, nnz doubles
 *   dimLevelType    host, per level
 *   dimOrdering     host, per level: logical dimension stored at level l; NULL = identity
 *   posBits/crdBits 0 (= 64, the "native" width), 8, 16, 32 or 64 (Section 4.1); stored
 *                   unsigned.  A width too small for the largest position (the entry
 *                   count of a level) or for a compressed level's largest possible
 *                   coordinate (its size - 1) yields SP_ERR_WIDTH_OVERFLOW.  The compute
 *                   kernels read 8- and 16-bit arrays through a 32-bit copy that the
 *                   handle builds (through the allocator) on the first such call and
 *                   keeps until sp_free; the accessors always return the narrow arrays.
 *   flags           SP_DUP_SUM or SP_DUP_ERROR
 *   out             receives the handle; release with sp_free
 *
 * Stored entries appear in lexicographic order of their level coordinates;
 * empty parents repeat their position; trailing dense levels materialise
 * explicit zeros (the paper's five storage examples).  Explicit zeros in the
 * input are kept.  The inputs are not modified.
 */
sp_status sp_pack(int rank, const int64_t* dims, int64_t nnz,
                  const void* const* coo_coords, int coo_coord_bits, const double* coo_vals,
                  const sp_level_type* dimLevelType, const int* dimOrdering,
                  int posBits, int crdBits, unsigned flags, void* stream, sp_tensor** out);

/* Releases the handle and its device arrays (NULL is allowed). */
sp_status sp_free(sp_tensor* t);

/*
 * Accessors - the paper's pointers / indices / values operations (Section 4.2),
 * each returning one level's array as a device pointer plus its length in
 * elements.  Dense levels have no arrays: *dev_ptr = NULL, *len = 0.
 * Element type is uint32_t or uint64_t according to the handle's widths.
 * Any output pointer of sp_info may be NULL.
 */
sp_status sp_info(const sp_tensor* t, int* rank, int64_t* dims /* host, rank */,
                  sp_level_type* dimLevelType, int* dimOrdering, int* posBits, int* crdBits);
sp_status sp_positions(const sp_tensor* t, int level, const void** dev_ptr, int64_t* len);
sp_status sp_coordinates(const sp_tensor* t, int level, const void** dev_ptr, int64_t* len);
sp_status sp_values(const sp_tensor* t, const double** dev_ptr, int64_t* len);

/*
 * sp_unpack - storage back to a coordinate list (the other half of
 * Section 4.2's conversion through coordinates).  Emits every stored value in
 * storage order with its LOGICAL coordinates, explicit zeros included.
 * coo_coords_out: host array of `rank` device pointers to int64 arrays with
 * room for sp_values' len entries each; vals_out likewise.  *nnz_out (host)
 * receives the count.
 */
sp_status sp_unpack(const sp_tensor* t, void* const* coo_coords_out, double* vals_out,
                    int64_t* nnz_out, void* stream);

/*
 * sp_convert - re-encode a tensor (the convert operation of Section 4.2, which
 * the paper implements through an intermediate coordinate scheme, as here:
 * sp_unpack followed by sp_pack, all on the device).  Every stored value of the
 * source, explicit zeros included, becomes a stored entry of the result.
 * Synchronises the stream as sp_pack does.  *out: a new handle.
 */
sp_status sp_convert(const sp_tensor* t, const sp_level_type* dimLevelType, const int* dimOrdering,
                     int posBits, int crdBits, void* stream, sp_tensor** out);

/*
 * sp_spmv - y[i] = sum_k A[i,k] * x[k]  (the matvec of Section 6.2).
 * A: rank 2, any of the eight encodings: level types (dense, compressed) or
 * (compressed, compressed) in either ordering (CSR, DCSR, CSC, DCSC), and
 * (compressed, dense) - the "CDR" of Section 6.2 - or (dense, dense) in either
 * ordering.  x has dims[1] entries, y dims[0].
 * Rows without stored entries are written as 0.  Column-major encodings
 * accumulate with floating-point atomics: the summation order, and so the
 * last bits, may differ from run to run.
 */
sp_status sp_spmv(sp_tensor* A, const double* x, double* y, void* stream);

/*
 * sp_spmm - C[i,j] = sum_k A[i,k] * B[k,j], A sparse, B and C dense
 * (Sections 1 and 5.2).  B is dims[1] x N with leading dimension ldb, C is
 * dims[0] x N with ldc.  Encodings (all eight two-dimensional ones, the set the
 * search loop of Section 5.2 enumerates) and the atomics remark as for sp_spmv.
 * With a dense inner level the product is a dense contraction and runs on the
 * f64 matrix instruction (the one place in this library where tensor cores
 * apply; the sparse kernels are gathers and use none); when it has few output
 * rows its contraction index is split over thread blocks and the partial sums
 * meet in C through atomics too (row-major included).  Row-major, with the
 * stored slices and every row of B starting on 16-byte boundaries (even slice
 * length, even ldb, aligned pointers), the operand tiles are brought in by the
 * copy engine (tensor maps over this device's memory, built per call on the
 * host); otherwise threads stage them.  The kernel's waits for those copies
 * are bounded: if one runs out, the blocks concerned write nothing, a flag is
 * raised, and this and every later such call returns SP_ERR_TIMEOUT instead of
 * launching (the contents of that earlier C are then undefined).  A
 * column-major matrix with 2^32 or more columns is refused (SP_ERR_UNSUPPORTED).
 */
sp_status sp_spmm(sp_tensor* A, const double* B, int64_t N, int64_t ldb,
                  double* C, int64_t ldc, void* stream);

/*
 * sp_sddmm - X[i,j] = S[i,j] * sum_k A[i,k] * B[k,j] for the stored (i,j) of
 * S (Section 6.2).  S: rank 2, any of the eight encodings (for a dense inner
 * level every cell of a stored row or column counts as stored, explicit zeros
 * included).  A is dims[0] x K (lda), B is K x dims[1] (ldb).  x_vals receives
 * one value per stored entry of S, in S's storage order (X shares S's
 * positions and coordinates); its length is sp_values' len.
 */
sp_status sp_sddmm(sp_tensor* S, const double* A, int64_t lda, const double* B, int64_t ldb,
                   int64_t K, double* x_vals, void* stream);

/*
 * sp_mttkrp - M[i,r] = sum_{j,k} T[i,j,k] * B[j,r] * C[k,r]  (Section 6.3,
 * where the same expression is written A[i,j] = B[i,k,l] * D[l,j] * C[k,j]).
 * T: rank 3, level types (compressed|dense, compressed, compressed) with
 * logical dimension 0 at level 0 and the other two in either order.
 * B is dims[1] x R, C is dims[2] x R, M is dims[0] x R, all contiguous
 * row-major.  Slices without stored entries give zero rows.
 */
sp_status sp_mttkrp(sp_tensor* T, const double* B, const double* C, int64_t R,
                    double* M, void* stream);

/*
 * sp_mttkrp_mode - the same product for any output dimension:
 *   M[c_mode, r] = sum over the other two coordinates of T[c0,c1,c2] * F_a[c_a, r] * F_b[c_b, r]
 * (Section 6.3 gives the mode-0 case).  T must store logical dimension `mode` at
 * level 0 (pack it with that dimOrdering), levels 1 and 2 compressed.
 * factors: host array of 3 device pointers, factors[d] being the dims[d] x R
 * matrix of dimension d; factors[mode] is ignored.  M is dims[mode] x R.
 */
sp_status sp_mttkrp_mode(sp_tensor* T, int mode, const double* const* factors, int64_t R,
                         double* M, void* stream);

/*
 * sp_scale - x[..] *= c over the stored values only, in place (Section 4.3's first example:
 * the loop body runs only for stored entries).  Any rank and encoding.  This is the one call
 * that changes a handle's values; cached work partitions stay valid (structure is untouched).
 */
sp_status sp_scale(sp_tensor* x, double c, void* stream);

/*
 * sp_vec_dot - *result = sum_i a[i] * b[i] for two compressed vectors (rank 1, level type
 * compressed) of equal length and equal coordinate width: the co-iteration example of
 * Section 4.3 (a product only where both store the index).  result: device, one double.
 * Partial sums are combined with atomic adds.
 */
sp_status sp_vec_dot(const sp_tensor* a, const sp_tensor* b, double* result, void* stream);

/*
 * sp_spmspm - C[i,j] = sum_k A[i,k] * B[k,j] with all three matrices sparse and
 * stored row-wise as (dense, compressed) with identity ordering - the SpMSpM
 * kernel of Section 4.3 (access pattern expansion per row, insertion in index
 * order), measured in Section 6.2.  A and B must share their bit widths;
 * posBits / crdBits (0, 8, 16, 32, 64) are those of the result.  *out receives a new
 * handle (release with sp_free) usable by every other call.  An (i,j) is stored
 * in C when some k has both A[i,k] and B[k,j] stored, even if the sum cancels.
 * Synchronises the stream once (the size of C depends on the data).  Sums are
 * accumulated with floating-point atomics (order, and so the last bits, may
 * vary from run to run).
 */
sp_status sp_spmspm(const sp_tensor* A, const sp_tensor* B, int posBits, int crdBits, void* stream,
                    sp_tensor** out);

/*
 * sp_spmv_static - y = A * x exactly as sp_spmv computes it (same kernels, same
 * results; the four encodings with a compressed inner level: CSR, DCSR, CSC, DCSC),
 * for callers that are not allowed to allocate device memory.
 * The paper has no counterpart; this is a deployment variant of sp_spmv.
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a real-time or
 * safety-qualified loop whose memory must all be reserved at start-up, a plug-in
 * living inside a host application that owns the GPU heap and forbids foreign
 * allocations, or a service whose allocator may block or fail under memory
 * pressure at exactly the moment the product is needed.  sp_spmv obtains its
 * work-partition table (on a handle's first use) and its row-carry buffer (on
 * every call) through the allocator; this call never does.  It calls neither the installed allocator nor
 * cudaMalloc / cudaFree, and caches nothing in the handle.
 *
 * Its scratch is a fixed array compiled into the library (about 2 MiB of device
 * memory on every GPU that loads the library, held until the process exits).
 * Handles with 8- or 16-bit arrays are refused with SP_ERR_UNSUPPORTED (reading
 * them would need the allocated 32-bit copy).
 * Capacity: rows-or-columns stored at the compressed level plus stored entries,
 * i.e. (sp_positions(A, 1) len - 1) + (sp_coordinates(A, 1) len), must not exceed
 * SP_SPMV_STATIC_MAX_ITEMS; larger inputs are refused with SP_ERR_TOO_LARGE and
 * nothing is launched.
 *
 * The first call on each device looks up the array's device address (a CUDA
 * runtime query, no allocation); make that first call during set-up, before any
 * stream capture is begun.  All calls share the one array: two calls whose
 * kernels may overlap on the GPU (different streams, or different host threads
 * on one device) race on it and give wrong results - serialise them.  The array
 * keeps whatever the last call left; every word a call reads it has written
 * itself earlier in that call, so no clearing is needed between calls.
 * The partition is recomputed on every call (one small extra kernel).
 * x, y, stream, errors and the atomics remark are as for sp_spmv; A is not modified.
 */
#define SP_SPMV_STATIC_MAX_ITEMS 134217728   /* 65,536 tiles of 2,048 (row end + entry) items */
sp_status sp_spmv_static(const sp_tensor* A, const double* x, double* y, void* stream);

/*
 * sp_launch_count: number of kernels this library has launched in this process (no
 * counterpart in the paper; lets a caller check that work ran on the device).
 */
int64_t sp_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SP_H */
