// The two small examples of Section 4.3, over storage: scaling a sparse tensor's stored values in
// place (x[i] *= c visits only stored entries) and the inner product of two compressed vectors
// (co-iteration: a product is formed only where both vectors store the same index).
#include "common.cuh"

namespace {

__global__ void k_scale(double* __restrict__ val, int64_t n, double c) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < n) val[i] *= c;
}

// One thread per stored entry of the shorter vector; the matching index of the other vector is found
// by binary search in its sorted coordinates (the sequential merge of the paper, made data parallel).
template <typename I>
__global__ void __launch_bounds__(256)
k_vec_dot(const I* __restrict__ acrd, const double* __restrict__ aval, int64_t na, const I* __restrict__ bcrd,
          const double* __restrict__ bval, int64_t nb, double* __restrict__ result) {
    __shared__ double s_part[8];
    const int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    double t = 0.0;
    if (p < na) {
        const I want = acrd[p];
        int64_t lo = 0, hi = nb;             // first q with bcrd[q] >= want
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (bcrd[mid] < want) lo = mid + 1; else hi = mid;
        }
        if (lo < nb && bcrd[lo] == want) t = aval[p] * bval[lo];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = s_part[0];
#pragma unroll
        for (int i = 1; i < 8; ++i) tot += s_part[i];
        if (tot != 0.0) atomicAdd(result, tot);
    }
}

}  // namespace

extern "C" sp_status sp_scale(sp_tensor* x, double c, void* stream_) {
    SP_API_RANGE("sp_scale");
    if (!x) return SP_ERR_INVALID_ARG;
    if (x->nval > 0) {
        k_scale<<<(unsigned)sp_ceil_div(x->nval, 256), 256, 0, static_cast<cudaStream_t>(stream_)>>>(x->val, x->nval, c);
        SP_LAUNCH_CHECK();
        sp_count_launches(1);
    }
    return SP_OK;
}

extern "C" sp_status sp_vec_dot(const sp_tensor* a, const sp_tensor* b, double* result, void* stream_) {
    SP_API_RANGE("sp_vec_dot");
    if (!a || !b || !result) return SP_ERR_INVALID_ARG;
    if (a->rank != 1 || b->rank != 1 || a->lt[0] != SP_COMPRESSED || b->lt[0] != SP_COMPRESSED) return SP_ERR_UNSUPPORTED;
    if (a->crdBits != b->crdBits) return SP_ERR_UNSUPPORTED;
    if (a->dims[0] != b->dims[0]) return SP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    SP_CUDA(cudaMemsetAsync(result, 0, sizeof(double), stream));
    if (a->ncrd[0] > b->ncrd[0]) { const sp_tensor* t = a; a = b; b = t; }    // walk the shorter one
    if (a->ncrd[0] == 0) return SP_OK;
    const unsigned blocks = (unsigned)sp_ceil_div(a->ncrd[0], 256);
#define SP_VEC_DOT(I)                                                                                             \
    k_vec_dot<I><<<blocks, 256, 0, stream>>>(static_cast<const I*>(a->crd[0]), a->val, a->ncrd[0],                \
                                             static_cast<const I*>(b->crd[0]), b->val, b->ncrd[0], result)
    switch (a->crdBits) {
        case 8: SP_VEC_DOT(uint8_t); break;
        case 16: SP_VEC_DOT(uint16_t); break;
        case 32: SP_VEC_DOT(uint32_t); break;
        default: SP_VEC_DOT(uint64_t); break;
    }
#undef SP_VEC_DOT
    SP_LAUNCH_CHECK();
    sp_count_launches(1);
    return SP_OK;
}
