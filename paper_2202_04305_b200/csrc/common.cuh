// Shared host/device declarations of the sparse tensor library (internal).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <mutex>
#include <vector>

#include "sp.h"

// ---------------------------------------------------------------------------
// Handle
// ---------------------------------------------------------------------------

// Work-partition table cached in a handle: chunk w covers merge-path
// coordinates [(row[w], nz[w]), (row[w+1], nz[w+1])).  The arrays are written once, when the table
// is created (the creating call waits for that work before it publishes the table, so any stream
// may read it afterwards), and only read from then on.  Scratch that a call writes (row carries)
// is never kept here: every call takes its own from the allocator, so calls on different streams
// share nothing writable.
struct sp_partition {
    int64_t nchunks = 0;
    int64_t* row = nullptr;   // nchunks + 1 entries (device)
    int64_t* nz = nullptr;    // nchunks + 1 entries (device)
    int64_t* aux = nullptr;   // kernel-specific (MTTKRP: slice of each chunk start)
};

struct sp_tensor {
    int rank = 0;
    int64_t dims[SP_MAX_RANK] = {};
    int lt[SP_MAX_RANK] = {};
    int ord[SP_MAX_RANK] = {};
    int posBits = 64, crdBits = 64;
    void* pos[SP_MAX_RANK] = {};
    int64_t npos[SP_MAX_RANK] = {};
    void* crd[SP_MAX_RANK] = {};
    int64_t ncrd[SP_MAX_RANK] = {};
    double* val = nullptr;
    int64_t nval = 0;
    int device = 0;
    std::mutex mu;
    std::map<uint64_t, sp_partition> parts;   // key = (kind << 56) | items per chunk
    // For handles stored with 8- or 16-bit positions/coordinates: a copy of the overhead arrays
    // widened to 32 bits that the compute kernels read (values shared, not copied).  Built on
    // first use by sp_widened(), owned by this handle.
    int64_t max_seg = -1;      // longest segment of the last level (entries under one parent); -1 = not measured yet
    sp_tensor* wide = nullptr;
    bool owns_val = true;
    void* block = nullptr;   // when set: pos[], crd[] and val are pieces of this one allocation
};

// SP_ERR_INVALID_ARG unless the handle's arrays live on the current device.
sp_status sp_check_device(const sp_tensor* t);
// Waits for the work that fills a cached table, so that the table can be published to every stream.
sp_status sp_partition_built(cudaStream_t stream);

// The handle the compute kernels should read: t itself when its widths are 32 or 64 bits,
// otherwise its (cached) 32-bit shadow.
sp_status sp_widened(sp_tensor* t, cudaStream_t stream, sp_tensor** out);

// ---------------------------------------------------------------------------
// Allocation through the installed allocator
// ---------------------------------------------------------------------------
void* sp_dev_alloc(size_t bytes, cudaStream_t stream);
void sp_dev_free(void* p, cudaStream_t stream);

// Frees everything it handed out when it goes out of scope.
struct sp_workspace {
    cudaStream_t stream;
    std::vector<void*> ptrs;
    bool failed = false;
    char* pool = nullptr;          // what is left of a reserve()d block
    size_t pool_left = 0;
    explicit sp_workspace(cudaStream_t s) : stream(s) {}
    ~sp_workspace() {
        for (void* p : ptrs) sp_dev_free(p, stream);
    }
    static size_t padded(size_t bytes) { return (bytes + 255) & ~(size_t)255; }
    template <typename T>
    static size_t bytes_for(size_t count) { return padded((count ? count : 1) * sizeof(T)); }
    // One trip to the allocator for buffers whose sizes are known up front (an allocator call can cost
    // microseconds of host time while the GPU idles): the get()s that follow carve 256-byte aligned
    // pieces out of this block and go to the allocator themselves only once it is used up.
    void reserve(size_t bytes) {
        if (bytes == 0) return;
        void* p = sp_dev_alloc(bytes, stream);
        if (!p) { failed = true; return; }
        ptrs.push_back(p);
        pool = static_cast<char*>(p);
        pool_left = bytes;
    }
    template <typename T>
    T* get(size_t count) {
        const size_t need = bytes_for<T>(count);
        if (pool && need <= pool_left) {
            T* r = reinterpret_cast<T*>(pool);
            pool += need;
            pool_left -= need;
            return r;
        }
        void* p = sp_dev_alloc((count ? count : 1) * sizeof(T), stream);
        if (!p) { failed = true; return nullptr; }
        ptrs.push_back(p);
        return static_cast<T*>(p);
    }
    // Hands ownership of p to the caller (it will not be freed here).
    void release(void* p) {
        for (auto& q : ptrs) if (q == p) { q = nullptr; }
    }
};

void sp_count_launches(int n);

// One NVTX range per API call (visible in Nsight Systems / Compute timelines; a no-op costing a
// few nanoseconds when no tool is attached).
#include <nvtx3/nvToolsExt.h>
struct sp_nvtx_range {
    explicit sp_nvtx_range(const char* name) { nvtxRangePushA(name); }
    ~sp_nvtx_range() { nvtxRangePop(); }
};
#define SP_API_RANGE(name) sp_nvtx_range nvtx_range__(name)

#define SP_CUDA(call)                                   \
    do {                                                \
        cudaError_t e__ = (call);                       \
        if (e__ != cudaSuccess) return SP_ERR_CUDA;     \
    } while (0)

#define SP_LAUNCH_CHECK() SP_CUDA(cudaGetLastError())

static inline int64_t sp_ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline bool sp_valid_width(int bits) { return bits == 8 || bits == 16 || bits == 32 || bits == 64; }
static inline uint64_t sp_width_max(int bits) { return bits >= 64 ? ~0ull : ((1ull << bits) - 1ull); }

// ---------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------
#ifdef __CUDACC__

// Element i of an unsigned array whose element width (8, 16, 32 or 64 bits) is known at run time.
__device__ __forceinline__ uint64_t sp_load_uint(const void* base, int64_t i, int bits) {
    switch (bits) {
        case 64: return static_cast<const uint64_t*>(base)[i];
        case 32: return static_cast<const uint32_t*>(base)[i];
        case 16: return static_cast<const uint16_t*>(base)[i];
        default: return static_cast<const uint8_t*>(base)[i];
    }
}
__device__ __forceinline__ void sp_store_uint(void* base, int64_t i, uint64_t v, int bits) {
    switch (bits) {
        case 64: static_cast<uint64_t*>(base)[i] = v; break;
        case 32: static_cast<uint32_t*>(base)[i] = static_cast<uint32_t>(v); break;
        case 16: static_cast<uint16_t*>(base)[i] = static_cast<uint16_t>(v); break;
        default: static_cast<uint8_t*>(base)[i] = static_cast<uint8_t>(v); break;
    }
}

__device__ __forceinline__ unsigned sp_lane() { return threadIdx.x & 31u; }

// Debug build (-DSP_DEBUG_BOUNDS): every index that a kernel derives from stored positions or
// coordinates is checked against the array it addresses.  A bad index is recorded (source line of the
// check, in this translation unit's device word) and replaced by a valid one, so the kernel finishes
// without a fault; the API call then reads the word back and returns SP_ERR_OUT_OF_RANGE.  In the
// normal build SP_IDX(i, n) is just i.
#ifdef SP_DEBUG_BOUNDS
static __device__ unsigned long long sp_bounds_word = 0;
__device__ __forceinline__ int64_t sp_checked_index(int64_t i, int64_t n, int line) {
    if (i >= 0 && i < n) return i;
    atomicMax(&sp_bounds_word, ((unsigned long long)line << 32) | 1ull);
    return (n > 0 && i >= n) ? n - 1 : 0;
}
#define SP_IDX(i, n) sp_checked_index((int64_t)(i), (int64_t)(n), __LINE__)
#else
#define SP_IDX(i, n) (i)
#endif

// Chains of short kernels in which each needs the one before it (the packer's passes, a kernel and
// its fix-up) are launched as programmatic dependents: the next kernel may be set up on the device
// while its predecessor drains, and its first statement waits until that predecessor has completed
// and its writes are visible.  Nothing triggers early: the only thing overlapped is the launch itself.
// In a kernel launched the ordinary way the wait returns at once.
__device__ __forceinline__ void sp_wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t sp_launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ double sp_shfl(double v, int src) {
    return __shfl_sync(0xffffffffu, v, src);
}

#endif  // __CUDACC__

#if defined(SP_DEBUG_BOUNDS) && defined(__CUDACC__)
// Host side of the debug build: waits for the stream, reads and clears this translation unit's word.
static inline sp_status sp_bounds_result(cudaStream_t stream) {
    unsigned long long w = 0, zero = 0;
    SP_CUDA(cudaStreamSynchronize(stream));
    SP_CUDA(cudaMemcpyFromSymbol(&w, sp_bounds_word, sizeof w));
    if (w) SP_CUDA(cudaMemcpyToSymbol(sp_bounds_word, &zero, sizeof zero));
    return w ? SP_ERR_OUT_OF_RANGE : SP_OK;
}
#define SP_BOUNDS_RETURN(stream) do { const sp_status b__ = sp_bounds_result(stream); if (b__ != SP_OK) return b__; } while (0)
#else
#define SP_BOUNDS_RETURN(stream) do {} while (0)
#endif

// Calls f(P{}, I{}) with the unsigned types matching the handle's widths.
#define SP_DISPATCH_WIDTHS(t, ...)                                              \
    do {                                                                        \
        if ((t)->posBits == 32 && (t)->crdBits == 32) { using P = uint32_t; using I = uint32_t; __VA_ARGS__ } \
        else if ((t)->posBits == 32) { using P = uint32_t; using I = uint64_t; __VA_ARGS__ }                 \
        else if ((t)->crdBits == 32) { using P = uint64_t; using I = uint32_t; __VA_ARGS__ }                 \
        else { using P = uint64_t; using I = uint64_t; __VA_ARGS__ }                                        \
    } while (0)

// Partition tables (partition.cu).  kind distinguishes the position array used.
enum { SP_PART_MERGE_LAST = 1, SP_PART_MTTKRP = 2, SP_PART_SEGIDS = 3 };
// For rank-2 (x, compressed) storage: the logical level-0 coordinate of every stored entry
// (the expanded "outer" index), uint32, cached in the handle.  Needs dims < 2^32.
sp_status sp_get_segment_ids(sp_tensor* t, cudaStream_t stream, const uint32_t** out);
sp_status sp_get_merge_partition(sp_tensor* t, int64_t items_per_chunk, cudaStream_t stream, sp_partition* out);
// Length of the longest last-level segment (row of CSR, stored row of DCSR, ...), measured on the
// device on first use (one small kernel and one read-back, which waits for the stream) and kept.
sp_status sp_get_max_segment(sp_tensor* t, cudaStream_t stream, int64_t* out);
sp_status sp_get_mttkrp_partition(sp_tensor* t, int64_t nnz_per_chunk, cudaStream_t stream, sp_partition* out);

// SpMV for rank-2 handles whose inner level is dense (dense_inner.cu).
sp_status sp_spmv_dense_inner(const sp_tensor* A, const double* x, double* y, cudaStream_t stream);
sp_status sp_spmm_dense_inner(const sp_tensor* A, const double* B, int64_t N, int64_t ldb, double* C, int64_t ldc,
                              cudaStream_t stream);
