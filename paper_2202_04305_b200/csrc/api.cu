// Handle management, allocator plumbing and the accessor calls of sp.h.
#include "common.cuh"

#include <atomic>

namespace {
void* (*g_alloc)(size_t, void*, void*) = nullptr;
void (*g_dealloc)(void*, void*, void*) = nullptr;
void* g_ctx = nullptr;
std::atomic<int64_t> g_launches{0};
}  // namespace

void sp_count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Default allocator: the device's stream-ordered pool, so that the per-call scratch of the compute
// calls costs neither a device synchronisation nor a trip to the driver's heap.
void* sp_dev_alloc(size_t bytes, cudaStream_t stream) {
    if (g_alloc) return g_alloc(bytes, stream, g_ctx);
    void* p = nullptr;
    if (cudaMallocAsync(&p, bytes, stream) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return p;
}

// stream == nullptr (sp_free): release after everything enqueued so far has finished.
void sp_dev_free(void* p, cudaStream_t stream) {
    if (!p) return;
    if (g_dealloc) { g_dealloc(p, stream, g_ctx); return; }
    if (stream) cudaFreeAsync(p, stream); else cudaFree(p);
}

sp_status sp_check_device(const sp_tensor* t) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SP_ERR_CUDA;
    return dev == t->device ? SP_OK : SP_ERR_INVALID_ARG;
}

sp_status sp_partition_built(cudaStream_t stream) {
    SP_CUDA(cudaStreamSynchronize(stream));
    return SP_OK;
}

extern "C" {

int64_t sp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* sp_status_string(sp_status s) {
    switch (s) {
        case SP_OK: return "ok";
        case SP_ERR_INVALID_ARG: return "invalid argument";
        case SP_ERR_UNSUPPORTED: return "unsupported encoding or shape";
        case SP_ERR_OUT_OF_RANGE: return "coordinate out of range";
        case SP_ERR_WIDTH_OVERFLOW: return "position or coordinate does not fit the requested bit width";
        case SP_ERR_DUPLICATE: return "duplicate coordinates";
        case SP_ERR_ALLOC: return "device allocation failed";
        case SP_ERR_CUDA: return "CUDA runtime error";
        case SP_ERR_TIMEOUT: return "a bounded device-side wait for an asynchronous copy ran out in an earlier launch";
        case SP_ERR_TOO_LARGE: return "problem exceeds the fixed scratch capacity of this entry point";
    }
    return "unknown status";
}

sp_status sp_set_allocator(void* (*alloc)(size_t, void*, void*), void (*dealloc)(void*, void*, void*), void* ctx) {
    if ((alloc == nullptr) != (dealloc == nullptr)) return SP_ERR_INVALID_ARG;
    g_alloc = alloc;
    g_dealloc = dealloc;
    g_ctx = ctx;
    return SP_OK;
}

sp_status sp_free(sp_tensor* t) {
    if (!t) return SP_OK;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(t->device);
    if (t->block) {
        sp_dev_free(t->block, nullptr);
    } else {
        for (int l = 0; l < SP_MAX_RANK; ++l) {
            sp_dev_free(t->pos[l], nullptr);
            sp_dev_free(t->crd[l], nullptr);
        }
        if (t->owns_val) sp_dev_free(t->val, nullptr);
    }
    if (t->wide) sp_free(t->wide);
    for (auto& kv : t->parts) {
        sp_dev_free(kv.second.row, nullptr);
        sp_dev_free(kv.second.nz, nullptr);
        sp_dev_free(kv.second.aux, nullptr);
    }
    delete t;
    cudaSetDevice(prev);
    return SP_OK;
}

sp_status sp_info(const sp_tensor* t, int* rank, int64_t* dims, sp_level_type* lt, int* ord, int* posBits, int* crdBits) {
    if (!t) return SP_ERR_INVALID_ARG;
    if (rank) *rank = t->rank;
    for (int l = 0; l < t->rank; ++l) {
        if (dims) dims[l] = t->dims[l];
        if (lt) lt[l] = static_cast<sp_level_type>(t->lt[l]);
        if (ord) ord[l] = t->ord[l];
    }
    if (posBits) *posBits = t->posBits;
    if (crdBits) *crdBits = t->crdBits;
    return SP_OK;
}

sp_status sp_positions(const sp_tensor* t, int level, const void** dev_ptr, int64_t* len) {
    if (!t || !dev_ptr || !len || level < 0 || level >= t->rank) return SP_ERR_INVALID_ARG;
    *dev_ptr = t->pos[level];
    *len = t->npos[level];
    return SP_OK;
}

sp_status sp_coordinates(const sp_tensor* t, int level, const void** dev_ptr, int64_t* len) {
    if (!t || !dev_ptr || !len || level < 0 || level >= t->rank) return SP_ERR_INVALID_ARG;
    *dev_ptr = t->crd[level];
    *len = t->ncrd[level];
    return SP_OK;
}

sp_status sp_values(const sp_tensor* t, const double** dev_ptr, int64_t* len) {
    if (!t || !dev_ptr || !len) return SP_ERR_INVALID_ARG;
    *dev_ptr = t->val;
    *len = t->nval;
    return SP_OK;
}

}  // extern "C"
