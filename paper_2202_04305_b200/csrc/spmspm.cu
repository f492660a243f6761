// sp_spmspm: C[i,j] = sum_k A[i,k] * B[k,j] with A, B and C all stored row-wise as
// (dense, compressed) - the SpMSpM kernel of Section 4.3, measured in Section 6.2 (Table 2).
//
// The paper's loop nest expands each row of C into a dense workspace (values + "filled" flags),
// records which columns were touched, and compresses the row back in index order.  Here a block
// owns a row at a time: its warps walk the entries A[i,k] (one per warp), lanes walk row k of B
// and add a*b into the block's workspace row with atomics, setting one bit per touched column in
// a bitmap.  Compression reads the bitmap words in order, so the columns come out sorted without
// a sort; a block-wide scan of the words' bit counts gives every column its slot.  The kernel runs
// twice: a symbolic pass that only counts (row lengths -> positions by a scan -> sizes of C's
// arrays, read back once), and a numeric pass that fills coordinates and values.
// Cost per row is proportional to its products plus dims[1]/32 bitmap words.
// When a dense row of C and its bitmap fit in shared memory (dims[1] up to about 25,000) the
// workspace lives there and the expansion's atomics never leave the SM; wider results use one
// workspace row per block in global memory (L2-resident).
#include "common.cuh"

namespace {

constexpr int kPThreads = 256;

__device__ __forceinline__ uint32_t block_excl_scan_u32(uint32_t v, uint32_t* sums, uint32_t* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += u;
    }
    if (lane == 31) sums[w] = incl;
    __syncthreads();
    uint32_t pre = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < kPThreads / 32; ++i) {
        const uint32_t s = sums[i];
        if (i < w) pre += s;
        tot += s;
    }
    __syncthreads();
    *total = tot;
    return incl - v + pre;
}

// NUMERIC = false: rowlen[i] = number of distinct columns of row i.
// NUMERIC = true : crd / val of C filled at cpos[i].. ; the workspace row is left zeroed.
template <typename P, typename I, bool NUMERIC, bool SMEM>
__global__ void __launch_bounds__(kPThreads)
k_spmspm(const P* __restrict__ apos, const I* __restrict__ acrd, const double* __restrict__ aval,
         const P* __restrict__ bpos, const I* __restrict__ bcrd, const double* __restrict__ bval, int64_t m,
         int64_t n, double* __restrict__ ws_all, uint32_t* __restrict__ bm_all, int64_t* __restrict__ rowlen,
         const void* __restrict__ cpos, int cposBits, void* __restrict__ ccrd, int ccrdBits,
         double* __restrict__ cval, int64_t kdim) {
    __shared__ uint32_t sums[kPThreads / 32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t words = (n + 31) >> 5;
    extern __shared__ __align__(16) unsigned char s_dyn[];
    double* ws;          // this block's dense row of C
    uint32_t* bm;        // ... and its "filled" flags, one bit per column
    if (SMEM) {          // [bitmap words, padded to 8 bytes][row of C, numeric pass only]; both start zeroed
        bm = reinterpret_cast<uint32_t*>(s_dyn);
        ws = reinterpret_cast<double*>(s_dyn + ((words * 4 + 7) & ~(int64_t)7));
        for (int64_t x = threadIdx.x; x < words; x += kPThreads) bm[x] = 0u;
        if (NUMERIC)
            for (int64_t x = threadIdx.x; x < n; x += kPThreads) ws[x] = 0.0;
        __syncthreads();
    } else {
        ws = ws_all + (int64_t)blockIdx.x * n;
        bm = bm_all + (int64_t)blockIdx.x * words;
    }

    for (int64_t i = blockIdx.x; i < m; i += gridDim.x) {
        // expand: every product of row i lands in the workspace
        const int64_t a0 = (int64_t)apos[i], a1 = (int64_t)apos[i + 1];
        for (int64_t p = a0 + w; p < a1; p += kPThreads / 32) {
            const int64_t k = SP_IDX((int64_t)acrd[p], kdim);
            const double a = aval[p];
            const int64_t b0 = (int64_t)bpos[k], b1 = (int64_t)bpos[k + 1];
            for (int64_t q = b0 + lane; q < b1; q += 32) {
                const int64_t j = SP_IDX((int64_t)bcrd[q], n);
                atomicOr(bm + (j >> 5), 1u << (j & 31));
                if (NUMERIC) atomicAdd(ws + j, a * bval[q]);
            }
        }
        __syncthreads();
        // compress: bitmap words in order give the columns in order
        uint32_t carry = 0;
        const int64_t base = NUMERIC ? (int64_t)sp_load_uint(cpos, i, cposBits) : 0;
        for (int64_t w0 = 0; w0 < words; w0 += kPThreads) {
            const int64_t wi = w0 + threadIdx.x;
            uint32_t bits = wi < words ? bm[wi] : 0u;
            uint32_t tot;
            const uint32_t ex = block_excl_scan_u32((uint32_t)__popc(bits), sums, &tot);
            if (wi < words && bits) bm[wi] = 0u;
            if (NUMERIC && tot >= 8u * kPThreads) {
                // well-filled words: a warp empties its 32 words one after the other, lane = bit, so the
                // workspace row is read (and cleared) 32 adjacent columns at a time and C is written in order
                const uint32_t below = (1u << lane) - 1u;
                for (uint32_t todo = __ballot_sync(0xffffffffu, bits != 0u); todo; todo &= todo - 1u) {
                    const int q = __ffs(todo) - 1;                      // next word of this warp that has columns
                    const uint32_t wbits = __shfl_sync(0xffffffffu, bits, q);
                    const uint32_t woff = __shfl_sync(0xffffffffu, ex, q);
                    if ((wbits >> lane) & 1u) {
                        const int64_t j = ((w0 + (int64_t)(w * 32 + q)) << 5) + lane;
                        const int64_t slot = base + carry + woff + __popc(wbits & below);
                        sp_store_uint(ccrd, slot, (uint64_t)j, ccrdBits);
                        cval[slot] = ws[j];
                        ws[j] = 0.0;
                    }
                }
            } else if (NUMERIC && wi < words && bits) {
                // sparse words: every thread walks the few columns of its own word
                int64_t slot = base + carry + ex;
                while (bits) {
                    const int bpos_ = __ffs(bits) - 1;
                    bits &= bits - 1;
                    const int64_t j = (wi << 5) + bpos_;
                    sp_store_uint(ccrd, slot, (uint64_t)j, ccrdBits);
                    cval[slot] = ws[j];
                    ws[j] = 0.0;
                    ++slot;
                }
            }
            carry += tot;
        }
        if (!NUMERIC && threadIdx.x == 0) rowlen[i] = (int64_t)carry;
        __syncthreads();
    }
}

// Single block: pos[0] = 0, pos[i+1] = rowlen[0] + .. + rowlen[i]; total to *count.
__global__ void __launch_bounds__(kPThreads)
k_row_offsets(const int64_t* __restrict__ rowlen, int64_t m, void* __restrict__ pos, int posBits, int64_t* __restrict__ count) {
    __shared__ unsigned long long s_w[kPThreads / 32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned long long run = 0;
    if (threadIdx.x == 0) sp_store_uint(pos, 0, 0, posBits);
    for (int64_t b = 0; b < m; b += kPThreads) {
        const int64_t i = b + threadIdx.x;
        unsigned long long v = i < m ? (unsigned long long)rowlen[i] : 0ull, incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long u = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += u;
        }
        if (lane == 31) s_w[w] = incl;
        __syncthreads();
        unsigned long long pre = 0, tot = 0;
        for (int q = 0; q < kPThreads / 32; ++q) { if (q < w) pre += s_w[q]; tot += s_w[q]; }
        __syncthreads();
        if (i < m) sp_store_uint(pos, i + 1, run + pre + incl, posBits);
        run += tot;
    }
    if (threadIdx.x == 0) *count = (int64_t)run;
}

}  // namespace

extern "C" sp_status sp_spmspm(const sp_tensor* A, const sp_tensor* B, int posBits, int crdBits, void* stream_,
                               sp_tensor** out) {
    SP_API_RANGE("sp_spmspm");
    if (!out) return SP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!A || !B) return SP_ERR_INVALID_ARG;
    if (posBits == 0) posBits = 64;
    if (crdBits == 0) crdBits = 64;
    if (!sp_valid_width(posBits) || !sp_valid_width(crdBits)) return SP_ERR_INVALID_ARG;
    {   // 8- and 16-bit operands are read through their 32-bit shadows (a cache inside the handle)
        sp_tensor *wa = nullptr, *wb = nullptr;
        sp_status ws_ = sp_widened(const_cast<sp_tensor*>(A), static_cast<cudaStream_t>(stream_), &wa);
        if (ws_ == SP_OK) ws_ = sp_widened(const_cast<sp_tensor*>(B), static_cast<cudaStream_t>(stream_), &wb);
        if (ws_ != SP_OK) return ws_;
        A = wa; B = wb;
    }
    auto is_csr = [](const sp_tensor* t) {
        return t->rank == 2 && t->lt[0] == SP_DENSE && t->lt[1] == SP_COMPRESSED && t->ord[0] == 0 && t->ord[1] == 1;
    };
    if (!is_csr(A) || !is_csr(B)) return SP_ERR_UNSUPPORTED;
    if (A->posBits != B->posBits || A->crdBits != B->crdBits) return SP_ERR_UNSUPPORTED;
    if (A->dims[1] != B->dims[0]) return SP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t m = A->dims[0], n = B->dims[1];
    if (n > 0 && (uint64_t)(n - 1) > sp_width_max(crdBits)) return SP_ERR_WIDTH_OVERFLOW;

    const int64_t words = (n + 31) >> 5;
    // shared-memory workspace if one row of C and its bitmap fit next to a second block's
    int dev = 0, sms = 0, smem_max = 0;
    SP_CUDA(cudaGetDevice(&dev));
    SP_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    SP_CUDA(cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    const size_t shm_sym = (size_t)((words * 4 + 7) & ~(int64_t)7);
    const size_t shm_num = shm_sym + (size_t)n * sizeof(double);
    const bool in_smem = shm_num + 2048 <= (size_t)smem_max;
    auto blocks_for = [&](size_t shm) {
        int64_t per_sm = (int64_t)((size_t)smem_max / (shm + 1024));
        if (per_sm > 8) per_sm = 8;
        if (per_sm < 1) per_sm = 1;
        int64_t b = per_sm * sms;
        if (b > m) b = m;
        return b < 1 ? (int64_t)1 : b;
    };
    int64_t nblocks = m < 148 * 4 ? m : 148 * 4;
    if (nblocks < 1) nblocks = 1;
    sp_workspace ws(stream);
    double* wsrow = nullptr;
    uint32_t* bm = nullptr;
    if (!in_smem) {
        wsrow = ws.get<double>((size_t)nblocks * n);
        bm = ws.get<uint32_t>((size_t)nblocks * words);
    }
    int64_t* rowlen = ws.get<int64_t>((size_t)m + 1);
    int64_t* d_count = ws.get<int64_t>(1);
    if (ws.failed) return SP_ERR_ALLOC;
    if (!in_smem) {
        SP_CUDA(cudaMemsetAsync(wsrow, 0, (size_t)nblocks * n * sizeof(double), stream));
        SP_CUDA(cudaMemsetAsync(bm, 0, (size_t)nblocks * words * sizeof(uint32_t), stream));
    }

    sp_tensor* C = new sp_tensor();
    cudaGetDevice(&C->device);
    C->rank = 2;
    C->dims[0] = m; C->dims[1] = n;
    C->lt[0] = SP_DENSE; C->lt[1] = SP_COMPRESSED;
    C->ord[0] = 0; C->ord[1] = 1;
    C->posBits = posBits; C->crdBits = crdBits;
    C->npos[1] = m + 1;
    C->pos[1] = sp_dev_alloc((size_t)(m + 1) * (posBits / 8), stream);
    if (!C->pos[1]) { sp_free(C); return SP_ERR_ALLOC; }
    auto fail = [&](sp_status s) { sp_free(C); return s; };

#define SP_SPMSPM_ARGS                                                                                            \
    static_cast<const P*>(A->pos[1]), static_cast<const I*>(A->crd[1]), A->val, static_cast<const P*>(B->pos[1]), \
        static_cast<const I*>(B->crd[1]), B->val, m, n, wsrow, bm, rowlen, C->pos[1], posBits, C->crd[1], crdBits, C->val, \
        B->dims[0]
#define SP_SPMSPM_LAUNCH(NUM)                                                                                     \
    SP_DISPATCH_WIDTHS(A, {                                                                                       \
        if (in_smem) {                                                                                            \
            const size_t shm = NUM ? shm_num : shm_sym;                                                           \
            if (cudaFuncSetAttribute(k_spmspm<P, I, NUM, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,      \
                                     (int)shm) != cudaSuccess)                                                    \
                return fail(SP_ERR_CUDA);                                                                         \
            k_spmspm<P, I, NUM, true><<<(unsigned)blocks_for(shm), kPThreads, shm, stream>>>(SP_SPMSPM_ARGS);     \
        } else {                                                                                                  \
            k_spmspm<P, I, NUM, false><<<(unsigned)nblocks, kPThreads, 0, stream>>>(SP_SPMSPM_ARGS);              \
        }                                                                                                         \
    })
    if (m > 0) SP_SPMSPM_LAUNCH(false);
    k_row_offsets<<<1, kPThreads, 0, stream>>>(rowlen, m, C->pos[1], posBits, d_count);
    if (cudaGetLastError() != cudaSuccess) return fail(SP_ERR_CUDA);
    sp_count_launches(2);
    int64_t count = 0;
    if (cudaMemcpyAsync(&count, d_count, sizeof count, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return fail(SP_ERR_CUDA);
    if ((uint64_t)count > sp_width_max(posBits)) return fail(SP_ERR_WIDTH_OVERFLOW);
    C->ncrd[1] = count;
    C->nval = count;
    C->crd[1] = sp_dev_alloc((size_t)(count ? count : 1) * (crdBits / 8), stream);
    C->val = static_cast<double*>(sp_dev_alloc((size_t)(count ? count : 1) * sizeof(double), stream));
    if (!C->crd[1] || !C->val) return fail(SP_ERR_ALLOC);
    if (m > 0 && count > 0) {
        SP_SPMSPM_LAUNCH(true);
        if (cudaGetLastError() != cudaSuccess) return fail(SP_ERR_CUDA);
        sp_count_launches(1);
    }
#undef SP_SPMSPM_LAUNCH
#undef SP_SPMSPM_ARGS
#ifdef SP_DEBUG_BOUNDS
    { const sp_status b = sp_bounds_result(stream); if (b != SP_OK) return fail(b); }
#endif
    *out = C;
    return SP_OK;
}
