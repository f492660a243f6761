// Work partitions cached in a handle.
//
// Merge-path partition over the innermost compressed level: the list of segment
// ends pos[1..S] (S segments = rows of a CSR matrix, stored rows of DCSR, columns
// of CSC ...) is merged with the list of entry indices 0..nnz-1; chunk w starts at
// the point of that merge path lying on diagonal w * items.  Every chunk then owns
// the same number of (segment end + entry) items whatever the row-length skew.
#include "common.cuh"

namespace {

template <typename P>
__global__ void k_merge_partition(const P* __restrict__ pos, int64_t nseg, int64_t nnz, int64_t items,
                                  int64_t nchunks, int64_t* __restrict__ row, int64_t* __restrict__ nz) {
    int64_t w = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (w > nchunks) return;
    const int64_t total = nseg + nnz;
    int64_t d = w * items;
    if (d > total) d = total;
    int64_t lo = d > nnz ? d - nnz : 0;
    int64_t hi = d < nseg ? d : nseg;
    while (lo < hi) {
        int64_t mid = (lo + hi) >> 1;
        // segment end `mid` precedes entry (d - mid - 1) when all its entries are consumed
        if ((int64_t)pos[mid + 1] <= d - mid - 1) lo = mid + 1; else hi = mid;
    }
    row[w] = lo;
    nz[w] = d - lo;
}

// MTTKRP: equal ranges of innermost entries; for each range start the fibre
// (level-1 node) and slice (level-0 node or index) that contain it.
template <typename P>
__global__ void k_mttkrp_partition(const P* __restrict__ pos1, int64_t nslice, const P* __restrict__ pos2,
                                   int64_t nfiber, int64_t nnz, int64_t per, int64_t nchunks,
                                   int64_t* __restrict__ fiber, int64_t* __restrict__ nz, int64_t* __restrict__ slice) {
    int64_t w = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (w > nchunks) return;
    int64_t p = w * per;
    if (p >= nnz) { nz[w] = nnz; fiber[w] = nfiber; slice[w] = nslice; return; }
    int64_t lo = 0, hi = nfiber;            // last f with pos2[f] <= p
    while (hi - lo > 1) { int64_t mid = (lo + hi) >> 1; if ((int64_t)pos2[mid] <= p) lo = mid; else hi = mid; }
    const int64_t f = lo;
    lo = 0; hi = nslice;                    // last s with pos1[s] <= f
    while (hi - lo > 1) { int64_t mid = (lo + hi) >> 1; if ((int64_t)pos1[mid] <= f) lo = mid; else hi = mid; }
    nz[w] = p; fiber[w] = f; slice[w] = lo;
}

// One thread per stored entry: the segment (level-0 node) that holds it, by binary search in pos[1],
// mapped through crd[0] when level 0 is compressed.
template <typename P, typename I>
__global__ void k_segment_ids(const P* __restrict__ pos, int64_t nseg, int64_t nnz, const I* __restrict__ outer,
                              uint32_t* __restrict__ seg) {
    const int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p >= nnz) return;
    int64_t lo = 0, hi = nseg;              // last q with pos[q] <= p  (pos[nseg] = nnz > p)
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)pos[mid] <= p) lo = mid; else hi = mid;
    }
    seg[p] = outer ? (uint32_t)outer[lo] : (uint32_t)lo;
}

// Longest segment: grid-stride maximum of pos[q+1] - pos[q], one atomicMax per block.
template <typename P>
__global__ void k_max_segment(const P* __restrict__ pos, int64_t nseg, unsigned long long* __restrict__ out) {
    unsigned long long m = 0;
    for (int64_t q = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; q < nseg; q += (int64_t)gridDim.x * blockDim.x) {
        const unsigned long long len = (unsigned long long)pos[q + 1] - (unsigned long long)pos[q];
        m = len > m ? len : m;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long u = __shfl_xor_sync(0xffffffffu, m, o);
        m = u > m ? u : m;
    }
    if ((threadIdx.x & 31) == 0 && m > 0) atomicMax(out, m);
}

}  // namespace

sp_status sp_get_max_segment(sp_tensor* t, cudaStream_t stream, int64_t* out) {
    std::lock_guard<std::mutex> lock(t->mu);
    if (t->max_seg >= 0) { *out = t->max_seg; return SP_OK; }
    const int last = t->rank - 1;
    const int64_t nseg = t->npos[last] - 1;
    if (nseg <= 0 || t->ncrd[last] == 0) { t->max_seg = 0; *out = 0; return SP_OK; }
    sp_workspace ws(stream);
    unsigned long long* d = ws.get<unsigned long long>(1);
    if (ws.failed) return SP_ERR_ALLOC;
    SP_CUDA(cudaMemsetAsync(d, 0, sizeof *d, stream));
    const unsigned blocks = (unsigned)std::min<int64_t>(sp_ceil_div(nseg, 256), 148 * 8);
    if (t->posBits == 32) k_max_segment<uint32_t><<<blocks, 256, 0, stream>>>(static_cast<const uint32_t*>(t->pos[last]), nseg, d);
    else k_max_segment<uint64_t><<<blocks, 256, 0, stream>>>(static_cast<const uint64_t*>(t->pos[last]), nseg, d);
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    unsigned long long h = 0;
    SP_CUDA(cudaMemcpyAsync(&h, d, sizeof h, cudaMemcpyDeviceToHost, stream));
    SP_CUDA(cudaStreamSynchronize(stream));
    t->max_seg = (int64_t)h;
    *out = t->max_seg;
    return SP_OK;
}

sp_status sp_get_segment_ids(sp_tensor* t, cudaStream_t stream, const uint32_t** out) {
    std::lock_guard<std::mutex> lock(t->mu);
    const uint64_t key = (uint64_t)SP_PART_SEGIDS << 56;
    auto it = t->parts.find(key);
    if (it != t->parts.end()) { *out = reinterpret_cast<const uint32_t*>(it->second.aux); return SP_OK; }
    const int64_t nseg = t->npos[1] - 1, nnz = t->ncrd[1];
    sp_partition p;
    p.aux = static_cast<int64_t*>(sp_dev_alloc((size_t)(nnz ? nnz : 1) * sizeof(uint32_t), stream));
    if (!p.aux) return SP_ERR_ALLOC;
    uint32_t* seg = reinterpret_cast<uint32_t*>(p.aux);
    if (nnz > 0) {
        const unsigned blocks = (unsigned)sp_ceil_div(nnz, 256);
        SP_DISPATCH_WIDTHS(t, {
            k_segment_ids<P, I><<<blocks, 256, 0, stream>>>(static_cast<const P*>(t->pos[1]), nseg, nnz,
                                                           t->lt[0] == SP_COMPRESSED ? static_cast<const I*>(t->crd[0]) : nullptr,
                                                           seg);
        });
        if (cudaGetLastError() != cudaSuccess) { sp_dev_free(p.aux, stream); return SP_ERR_CUDA; }
        sp_count_launches(1);
    }
    if (sp_partition_built(stream) != SP_OK) { sp_dev_free(p.aux, stream); return SP_ERR_CUDA; }
    t->parts[key] = p;
    *out = seg;
    return SP_OK;
}

sp_status sp_get_merge_partition(sp_tensor* t, int64_t items, cudaStream_t stream, sp_partition* out) {
    std::lock_guard<std::mutex> lock(t->mu);
    const uint64_t key = ((uint64_t)SP_PART_MERGE_LAST << 56) | (uint64_t)items;
    auto it = t->parts.find(key);
    if (it != t->parts.end()) { *out = it->second; return SP_OK; }
    const int last = t->rank - 1;
    const int64_t nseg = t->npos[last] - 1;
    const int64_t nnz = t->ncrd[last];
    sp_partition p;
    p.nchunks = sp_ceil_div(nseg + nnz, items);
    if (p.nchunks < 1) p.nchunks = 1;
    p.row = static_cast<int64_t*>(sp_dev_alloc((size_t)(p.nchunks + 1) * sizeof(int64_t), stream));
    p.nz = static_cast<int64_t*>(sp_dev_alloc((size_t)(p.nchunks + 1) * sizeof(int64_t), stream));
    auto drop = [&](sp_status s) { sp_dev_free(p.row, stream); sp_dev_free(p.nz, stream); return s; };
    if (!p.row || !p.nz) return drop(SP_ERR_ALLOC);
    const unsigned blocks = (unsigned)sp_ceil_div(p.nchunks + 1, 256);
    if (t->posBits == 32)
        k_merge_partition<uint32_t><<<blocks, 256, 0, stream>>>(static_cast<const uint32_t*>(t->pos[last]), nseg, nnz,
                                                                 items, p.nchunks, p.row, p.nz);
    else
        k_merge_partition<uint64_t><<<blocks, 256, 0, stream>>>(static_cast<const uint64_t*>(t->pos[last]), nseg, nnz,
                                                                 items, p.nchunks, p.row, p.nz);
    if (cudaGetLastError() != cudaSuccess) return drop(SP_ERR_CUDA);
    sp_count_launches(1);
    if (sp_partition_built(stream) != SP_OK) return drop(SP_ERR_CUDA);
    t->parts[key] = p;
    *out = p;
    return SP_OK;
}

// ------------------------------------------------------------------ widened shadow ---
namespace {
template <typename S>
__global__ void k_widen(const S* __restrict__ src, uint32_t* __restrict__ dst, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = (uint32_t)src[i];
}

// A 32-bit (or, for bits >= 32, plain) copy of an overhead array.
sp_status widen_array(const void* src, int64_t n, int bits, cudaStream_t stream, void** out) {
    *out = nullptr;
    if (!src) return SP_OK;
    const int obits = bits < 32 ? 32 : bits;
    void* d = sp_dev_alloc((size_t)(n ? n : 1) * (obits / 8), stream);
    if (!d) return SP_ERR_ALLOC;
    *out = d;
    if (n == 0) return SP_OK;
    if (bits >= 32) {
        SP_CUDA(cudaMemcpyAsync(d, src, (size_t)n * (bits / 8), cudaMemcpyDeviceToDevice, stream));
        return SP_OK;
    }
    const unsigned blocks = (unsigned)std::min<int64_t>(sp_ceil_div(n, 256), 148 * 8);
    if (bits == 16) k_widen<uint16_t><<<blocks, 256, 0, stream>>>(static_cast<const uint16_t*>(src), static_cast<uint32_t*>(d), n);
    else k_widen<uint8_t><<<blocks, 256, 0, stream>>>(static_cast<const uint8_t*>(src), static_cast<uint32_t*>(d), n);
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    return SP_OK;
}
}  // namespace

sp_status sp_widened(sp_tensor* t, cudaStream_t stream, sp_tensor** out) {
    if (t->posBits >= 32 && t->crdBits >= 32) { *out = t; return SP_OK; }
    std::lock_guard<std::mutex> lock(t->mu);
    if (t->wide) {
        *out = t->wide;
        return SP_OK;
    }
    sp_tensor* w = new sp_tensor();
    w->rank = t->rank;
    w->device = t->device;
    w->posBits = t->posBits < 32 ? 32 : t->posBits;
    w->crdBits = t->crdBits < 32 ? 32 : t->crdBits;
    w->val = t->val;
    w->nval = t->nval;
    w->owns_val = false;
    sp_status st = SP_OK;
    for (int l = 0; l < t->rank; ++l) {
        w->dims[l] = t->dims[l]; w->lt[l] = t->lt[l]; w->ord[l] = t->ord[l];
        w->npos[l] = t->npos[l]; w->ncrd[l] = t->ncrd[l];
        if (st == SP_OK) st = widen_array(t->pos[l], t->npos[l], t->posBits, stream, &w->pos[l]);
        if (st == SP_OK) st = widen_array(t->crd[l], t->ncrd[l], t->crdBits, stream, &w->crd[l]);
    }
    if (st != SP_OK) { sp_free(w); return st; }
    if (sp_partition_built(stream) != SP_OK) { sp_free(w); return SP_ERR_CUDA; }
    t->wide = w;
    *out = w;
    return SP_OK;
}

sp_status sp_get_mttkrp_partition(sp_tensor* t, int64_t per, cudaStream_t stream, sp_partition* out) {
    std::lock_guard<std::mutex> lock(t->mu);
    const uint64_t key = ((uint64_t)SP_PART_MTTKRP << 56) | (uint64_t)per;
    auto it = t->parts.find(key);
    if (it != t->parts.end()) { *out = it->second; return SP_OK; }
    const int64_t nnz = t->ncrd[2];
    const int64_t nfiber = t->ncrd[1];
    const int64_t nslice = t->npos[1] - 1;
    sp_partition p;
    p.nchunks = sp_ceil_div(nnz, per);
    if (p.nchunks < 1) p.nchunks = 1;
    p.row = static_cast<int64_t*>(sp_dev_alloc((size_t)(p.nchunks + 1) * sizeof(int64_t), stream));
    p.nz = static_cast<int64_t*>(sp_dev_alloc((size_t)(p.nchunks + 1) * sizeof(int64_t), stream));
    p.aux = static_cast<int64_t*>(sp_dev_alloc((size_t)(p.nchunks + 1) * sizeof(int64_t), stream));
    auto drop = [&](sp_status s) { sp_dev_free(p.row, stream); sp_dev_free(p.nz, stream); sp_dev_free(p.aux, stream); return s; };
    if (!p.row || !p.nz || !p.aux) return drop(SP_ERR_ALLOC);
    const unsigned blocks = (unsigned)sp_ceil_div(p.nchunks + 1, 256);
    if (t->posBits == 32)
        k_mttkrp_partition<uint32_t><<<blocks, 256, 0, stream>>>(
            static_cast<const uint32_t*>(t->pos[1]), nslice, static_cast<const uint32_t*>(t->pos[2]), nfiber, nnz, per,
            p.nchunks, p.row, p.nz, p.aux);
    else
        k_mttkrp_partition<uint64_t><<<blocks, 256, 0, stream>>>(
            static_cast<const uint64_t*>(t->pos[1]), nslice, static_cast<const uint64_t*>(t->pos[2]), nfiber, nnz, per,
            p.nchunks, p.row, p.nz, p.aux);
    if (cudaGetLastError() != cudaSuccess) return drop(SP_ERR_CUDA);
    sp_count_launches(1);
    if (sp_partition_built(stream) != SP_OK) return drop(SP_ERR_CUDA);
    t->parts[key] = p;
    *out = p;
    return SP_OK;
}
