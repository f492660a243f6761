// sp_pack / sp_unpack: coordinate list <-> per-level storage (Section 4.1 scheme,
// reached through coordinates as in Section 4.2).
//
// Pipeline of sp_pack, all on the caller's stream:
//   1. k_build_keys   level coordinates c_l = coord[dimOrdering[l]] fused into one
//                     lexicographic key (level 0 in the top bits), range check
//   2. radix sort     stable LSD, <= 8 bits per pass, (key, entry index) pairs;
//                     per pass: tile histograms -> per-digit scan -> ranked scatter
//   3. k_count_flags  for every level the flag "key prefix through this level
//                     differs from the previous entry" = a new stored node;
//                     per-tile counts, then a scan of the tile counts
//   4. (one read-back of the node counts: the array sizes depend on the data)
//   5. k_emit         node ids from the scanned flags; coordinates per node;
//                     first-child offsets per parent; values (duplicates summed
//                     in input order)
//   6. suffix-min     compressed levels under a dense level: parents without
//                     children take the next parent's offset
#include "common.cuh"

#include <string.h>

namespace {

constexpr int kErrRange = 1;
constexpr int kErrDup = 2;

// Phase timing of the packer: CUDA events on the caller's stream between its kernels.  The product
// library never asks for it (times == nullptr: no event is created); the benchmark's own library
// compiles this file a second time with SP_BENCH_BUILD and exports the timed variant.
enum { kPhKeys = 0, kPhUpsweep, kPhScan, kPhDownsweep, kPhCount, kPhEmit, kPhCount_ };
struct PackTimes {
    double ms[kPhCount_];
    int passes;
};

struct PhaseTimer {
    cudaStream_t stream;
    PackTimes* out;
    bool on;
    std::vector<cudaEvent_t> ev;
    std::vector<int> phase;
    PhaseTimer(cudaStream_t s, PackTimes* times) : stream(s), out(times), on(times != nullptr) { if (on) mark(-1); }
    // closes the interval that started at the previous mark and files it under `ph`
    void mark(int ph) {
        if (!on) return;
        cudaEvent_t e;
        cudaEventCreate(&e);
        cudaEventRecord(e, stream);
        ev.push_back(e);
        phase.push_back(ph);
    }
    void finish(int passes) {
        if (!on) return;
        cudaEventSynchronize(ev.back());
        for (int i = 0; i < kPhCount_; ++i) out->ms[i] = 0;
        for (size_t i = 1; i < ev.size(); ++i) {
            float ms = 0;
            cudaEventElapsedTime(&ms, ev[i - 1], ev[i]);
            if (phase[i] >= 0) out->ms[phase[i]] += ms;
        }
        out->passes = passes;
    }
    ~PhaseTimer() { for (auto e : ev) cudaEventDestroy(e); }
};

struct LevelPlan {
    int rank;
    int shift[SP_MAX_RANK];
    int bits[SP_MAX_RANK];
    int lt[SP_MAX_RANK];
    int src[SP_MAX_RANK];       // logical dimension stored at level l
    int64_t sz[SP_MAX_RANK];
};

// ------------------------------------------------------------------ keys ---
struct LevelCoords { const void* p[SP_MAX_RANK]; };   // coordinate array of the dimension stored at level l

constexpr int kSortThreads = 256;
// Sort tile: 256 threads x kIpt keys.  With a separate 32-bit payload (PAY: key and entry index as a
// pair, 24 bytes moved per entry and pass) 8 keys per thread and four tiles per SM are the faster shape
// (six scatter passes over 20,000,000 entries: 0.78 ms against 0.87 ms with 16 keys and three tiles);
// with the index inside the key (8-byte words) 16 keys per thread and three tiles per SM are
// (5,000,000 entries: pack 0.48 ms against 0.50 ms).  Every kernel of one sort uses the same shape.
#ifndef SP_SORT_PAY_IPT
#define SP_SORT_PAY_IPT 8
#endif
#ifndef SP_SORT_PAY_BLOCKS
#define SP_SORT_PAY_BLOCKS 4
#endif
template <bool PAY>
struct SortShape {
    static constexpr int kIpt = PAY ? SP_SORT_PAY_IPT : 16;
    static constexpr int kTile = kSortThreads * kIpt;
    static constexpr int kMinBlocks = PAY ? SP_SORT_PAY_BLOCKS : 3;
};
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kMaxRadix = 256;

// A block builds the keys of one sort tile and, while it has them in registers, the tile's digit
// histogram for the first radix pass (digit = (key >> shift0) & mask0), so that pass needs no
// counting sweep of its own.
// idx_bits > 0: the entry index rides in the low idx_bits bits of the key itself (the sort then
// moves 8 bytes per entry).  Otherwise the entry's value travels beside its key from the first
// pass on (which reads it from the input, where value e belongs to key e), so no index exists.
template <typename CT, bool PAY>
__global__ void __launch_bounds__(kSortThreads)
k_build_keys(LevelCoords lc, int64_t n, LevelPlan p, uint64_t* keys, int idx_bits, int* err,
             int shift0, uint32_t mask0, uint32_t* __restrict__ tilehist, int64_t ntiles) {
    constexpr int kSortIpt = SortShape<PAY>::kIpt, kSortTile = SortShape<PAY>::kTile;
    __shared__ uint32_t hist[kSortWarps][kMaxRadix];
    const int t = threadIdx.x, w = t >> 5;
    for (int i = t; i < kSortWarps * kMaxRadix; i += kSortThreads) (&hist[0][0])[i] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
    CT c[kSortIpt / 2][SP_MAX_RANK];
    bool bad = false;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
#pragma unroll
        for (int i = 0; i < kSortIpt / 2; ++i) {       // the loads of half a thread's entries first
            const int64_t e = base + (int64_t)(half * (kSortIpt / 2) + i) * kSortThreads + t;
#pragma unroll
            for (int l = 0; l < SP_MAX_RANK; ++l)
                if (l < p.rank) c[i][l] = e < n ? static_cast<const CT*>(lc.p[l])[e] : (CT)0;
        }
#pragma unroll
        for (int i = 0; i < kSortIpt / 2; ++i) {
            const int64_t e = base + (int64_t)(half * (kSortIpt / 2) + i) * kSortThreads + t;
            if (e >= n) continue;
            uint64_t key = 0;
#pragma unroll
            for (int l = 0; l < SP_MAX_RANK; ++l) {
                if (l < p.rank) {
                    CT v = c[i][l];
                    if (v < 0 || (int64_t)v >= p.sz[l]) { bad = true; v = 0; }
                    key |= (uint64_t)v << p.shift[l];
                }
            }
            if (idx_bits > 0) key = (key << idx_bits) | (uint64_t)e;
            keys[e] = key;
            atomicAdd(&hist[w][(uint32_t)(key >> shift0) & mask0], 1u);
        }
    }
    if (bad) atomicOr(err, kErrRange);
    __syncthreads();
    for (uint32_t d = t; d <= mask0; d += kSortThreads) {
        uint32_t s = 0;
#pragma unroll
        for (int i = 0; i < kSortWarps; ++i) s += hist[i][d];
        tilehist[(int64_t)d * ntiles + blockIdx.x] = s;
    }
}

// ------------------------------------------------------------ radix sort ---
// Digits are up to kMaxDigitBits wide: the 42-bit keys of a 16,384^3 tensor sort in six passes of
// 7 bits.  (9-bit digits - five passes - were measured: each pass then costs 0.174 ms instead of
// 0.145 ms on 20,000,000 entries and its histogram 0.039 ms instead of 0.034 ms, so nothing is won.)
// The kernels are instantiated per digit width so that the ranking needs exactly that many ballots.
#ifndef SP_SORT_MAX_BITS
#define SP_SORT_MAX_BITS 8
#endif
constexpr int kMaxDigitBits = SP_SORT_MAX_BITS;
static_assert((1 << kMaxDigitBits) <= kMaxRadix, "the key-building kernel's histogram holds kMaxRadix bins");

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t u = __shfl_up_sync(0xffffffffu, v, o);
        if ((int)sp_lane() >= o) v += u;
    }
    return v;
}

// Exclusive scan over the NT threads of a block (NT a multiple of 32, at most 1024); `sums` has NT / 32 entries.
template <int NT>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* sums, uint32_t* total) {
    const int w = threadIdx.x >> 5;
    uint32_t incl = warp_incl_scan(v);
    if (sp_lane() == 31) sums[w] = incl;
    __syncthreads();
    uint32_t pre = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < NT / 32; ++i) {
        uint32_t s = sums[i];
        if (i < w) pre += s;
        tot += s;
    }
    __syncthreads();
    *total = tot;
    return incl - v + pre;
}
__device__ __forceinline__ uint32_t block256_excl_scan(uint32_t v, uint32_t* sums, uint32_t* total) {
    return block_excl_scan<256>(v, sums, total);
}

// Tile histograms of one digit (passes after the first; the first pass's come from k_build_keys).
// Counting them inside the previous pass's scatter, with global atomics where the keys land, was
// measured: skewed digits pile onto few counters and the 20,000,000-entry scatter went from 0.145 ms
// to 0.59 ms per pass.
template <int BITS, bool PAY>
__global__ void __launch_bounds__(kSortThreads)
k_sort_upsweep(const uint64_t* __restrict__ keys, int64_t n, int shift, uint32_t* __restrict__ tilehist, int64_t ntiles) {
    sp_wait_for_previous_kernel();
    constexpr int kSortIpt = SortShape<PAY>::kIpt, kSortTile = SortShape<PAY>::kTile;
    constexpr int RADIX = 1 << BITS;
    constexpr uint32_t mask = RADIX - 1;
    __shared__ uint32_t hist[kSortWarps][RADIX];     // one histogram per warp: conflicts only inside a warp
    const int t = threadIdx.x, w = t >> 5;
    for (int i = t; i < kSortWarps * RADIX; i += kSortThreads) (&hist[0][0])[i] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
    uint64_t k[kSortIpt];
#pragma unroll
    for (int i = 0; i < kSortIpt; ++i) {             // all loads first
        const int64_t e = base + (int64_t)i * kSortThreads + t;
        k[i] = e < n ? keys[e] : 0;
    }
#pragma unroll
    for (int i = 0; i < kSortIpt; ++i) {
        const int64_t e = base + (int64_t)i * kSortThreads + t;
        if (e < n) atomicAdd(&hist[w][(uint32_t)(k[i] >> shift) & mask], 1u);
    }
    __syncthreads();
    for (int d = t; d < RADIX; d += kSortThreads) {
        uint32_t c = 0;
#pragma unroll
        for (int i = 0; i < kSortWarps; ++i) c += hist[i][d];
        tilehist[(int64_t)d * ntiles + blockIdx.x] = c;
    }
}

// Lanes of the warp whose NB-bit value equals this lane's, by one ballot per bit.  The hardware
// match instruction does the same but costs more per call the more distinct values the warp holds:
// with uniform 8-bit digits the scatter pass ran 0.31 ms per five passes over 5 M entries with it and
// 0.24 ms with the ballots.  NB is a compile-time count: a run-time bound made the loop slower.
template <int NB>
__device__ __forceinline__ uint32_t same_value_lanes(uint32_t d) {
    uint32_t peers = 0xffffffffu;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        const bool bit = (d >> b) & 1u;
        const uint32_t bal = __ballot_sync(0xffffffffu, bit);
        peers &= bit ? bal : ~bal;
    }
    return peers;
}

// Exclusive scan of every digit's tile counts, in place, in two small launches: the counts of a digit
// are cut into chunks of kScanChunk tiles; k_sort_chunk_totals adds up each chunk, k_sort_scan scans a
// chunk starting from the sum of the chunks before it (a handful of values, added up by every block
// for itself).  Grid (digits, chunks): all SMs take part however many tiles there are.
constexpr int kScanChunk = 2048;

__global__ void __launch_bounds__(256)
k_sort_chunk_totals(const uint32_t* __restrict__ tilehist, int64_t ntiles, int64_t nchunks, uint32_t* __restrict__ chunk_tot) {
    sp_wait_for_previous_kernel();
    __shared__ uint32_t sums[8];
    const uint32_t* row = tilehist + (int64_t)blockIdx.x * ntiles;
    const int64_t base = (int64_t)blockIdx.y * kScanChunk;
    uint32_t local = 0;
#pragma unroll
    for (int i = 0; i < kScanChunk / 256; ++i) {
        const int64_t q = base + i * 256 + threadIdx.x;
        if (q < ntiles) local += row[q];
    }
    uint32_t tot;
    block256_excl_scan(local, sums, &tot);
    if (threadIdx.x == 0) chunk_tot[(int64_t)blockIdx.x * nchunks + blockIdx.y] = tot;
}

__global__ void __launch_bounds__(256)
k_sort_scan(uint32_t* tilehist, int64_t ntiles, int64_t nchunks, const uint32_t* __restrict__ chunk_tot,
            uint32_t* __restrict__ digit_total) {
    sp_wait_for_previous_kernel();
    __shared__ uint32_t stage[kScanChunk];
    __shared__ uint32_t sums[8];
    uint32_t* row = tilehist + (int64_t)blockIdx.x * ntiles;
    const int64_t base = (int64_t)blockIdx.y * kScanChunk;
    const int cnt = (int)min((int64_t)kScanChunk, ntiles - base);
    constexpr int kPer = kScanChunk / 256;
    uint32_t before = 0;                               // sum of the chunks before this one
    for (int64_t c = 0; c < (int64_t)blockIdx.y; ++c) before += chunk_tot[(int64_t)blockIdx.x * nchunks + c];
    for (int i = threadIdx.x; i < cnt; i += 256) stage[i] = row[base + i];
    __syncthreads();
    uint32_t local = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int q = threadIdx.x * kPer + i;
        if (q < cnt) local += stage[q];
    }
    uint32_t tot;
    uint32_t run = block256_excl_scan(local, sums, &tot) + before;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int q = threadIdx.x * kPer + i;
        if (q < cnt) { const uint32_t v = stage[q]; stage[q] = run; run += v; }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < cnt; i += 256) row[base + i] = stage[i];
    if (threadIdx.x == 0 && blockIdx.y == nchunks - 1) digit_total[blockIdx.x] = before + tot;
}

constexpr size_t down_smem(bool pay, int bits) {
    return (size_t)(pay ? SortShape<true>::kTile : SortShape<false>::kTile) * (pay ? 16 : 8) + (size_t)kSortWarps * ((1 << bits) + 1) * 4 +
           (size_t)(1 << bits) * 4 + 64;
}

// Ranks the warp's rounds of 32 keys: rank i = number of earlier keys of this warp with the same
// digit (below 512, so two ranks share a register: round i sits in half i & 1 of rank[i / 2]); the
// per-warp digit counts end up in mycnt[].  NB = BITS, or BITS + 1 when the tile has padding slots
// (their digit is RADIX, which sorts after every real digit).
template <int BITS, int NB, int kSortIpt>
__device__ __forceinline__ void rank_rounds(const uint64_t (&key)[kSortIpt], int shift, int w, int lane, int tile_n,
                                            uint32_t* mycnt, uint32_t (&rank)[kSortIpt / 2]) {
    constexpr uint32_t RADIX = 1u << BITS;
    const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
    for (int i = 0; i < kSortIpt; ++i) {
        uint32_t d = (uint32_t)(key[i] >> shift) & (RADIX - 1);
        if (NB > BITS && w * (32 * kSortIpt) + i * 32 + lane >= tile_n) d = RADIX;
        const uint32_t peers = same_value_lanes<NB>(d);
        const int leader = __ffs(peers) - 1;
        uint32_t b = 0;
        if (lane == leader) { b = mycnt[d]; mycnt[d] = b + (uint32_t)__popc(peers); }
        b = __shfl_sync(0xffffffffu, b, leader);
        const uint32_t r = b + (uint32_t)__popc(peers & lt_mask);
        if (i & 1) rank[i / 2] |= r << 16; else rank[i / 2] = r;
        __syncwarp();                                 // rounds update the same counters: keep them in order
    }
}

// PAY: a 64-bit payload (the entry's value, moved as bits) travels beside every key.  Without it the
// entry index sits in the key's low bits; the last pass (split_bits >= 0) then separates the two again
// on the way out: keys_out gets key >> split_bits, idx_out the low split_bits bits.
template <bool PAY, int BITS>
__global__ void __launch_bounds__(kSortThreads, SortShape<PAY>::kMinBlocks)   // several tiles per SM hide the ranking chain's latency
k_sort_downsweep(const uint64_t* __restrict__ keys_in, const uint64_t* __restrict__ pay_in,
                 uint64_t* __restrict__ keys_out, uint64_t* __restrict__ pay_out, uint32_t* __restrict__ idx_out,
                 int64_t n, int shift,
                 const uint32_t* __restrict__ tilehist, int64_t ntiles,
                 const uint32_t* __restrict__ digit_total, int split_bits) {
    sp_wait_for_previous_kernel();
    constexpr int kSortIpt = SortShape<PAY>::kIpt, kSortTile = SortShape<PAY>::kTile;
    constexpr int RADIX = 1 << BITS;
    constexpr uint32_t mask = RADIX - 1;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* skeys = reinterpret_cast<uint64_t*>(smem_raw);
    uint64_t* spay = skeys + kSortTile;
    uint32_t* wcnt = reinterpret_cast<uint32_t*>(PAY ? spay + kSortTile : spay);   // [warps][RADIX + 1]
    uint32_t* goff = wcnt + kSortWarps * (RADIX + 1);         // [RADIX]: where the digit's keys go in the output minus where they start in the tile (mod 2^32)
    __shared__ uint32_t sums[kSortThreads / 32];

    const int t = threadIdx.x, w = t >> 5, lane = t & 31;
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
    const int tile_n = (int)min((int64_t)kSortTile, n - base);

    for (int i = t; i < kSortWarps * (RADIX + 1); i += kSortThreads) wcnt[i] = 0;
    __syncthreads();

    uint64_t key[kSortIpt];
    uint64_t pay[PAY ? kSortIpt : 1];
    uint32_t rank[kSortIpt / 2];
    uint32_t* mycnt = wcnt + w * (RADIX + 1);
#pragma unroll
    for (int i = 0; i < kSortIpt; ++i) {             // all key loads first
        const int li = w * (32 * kSortIpt) + i * 32 + lane;
        key[i] = li < tile_n ? keys_in[base + li] : 0;
#ifdef SP_SORT_PAY_EARLY
        if (PAY) pay[i] = li < tile_n ? pay_in[base + li] : 0;
#endif
    }
    if (tile_n == kSortTile) rank_rounds<BITS, BITS, kSortIpt>(key, shift, w, lane, tile_n, mycnt, rank);
    else rank_rounds<BITS, BITS + 1, kSortIpt>(key, shift, w, lane, tile_n, mycnt, rank);
#ifndef SP_SORT_PAY_EARLY
    if (PAY) {
        // the payloads are not needed before the exchange: requested here, they arrive during the
        // digit scans below without holding registers through the ranking
#pragma unroll
        for (int i = 0; i < kSortIpt; ++i) {
            const int li = w * (32 * kSortIpt) + i * 32 + lane;
            pay[i] = li < tile_n ? pay_in[base + li] : 0;
        }
    }
#endif
    __syncthreads();

    // per digit: exclusive scan over warps; then exclusive scan over digits (each thread owns
    // RADIX / 256 consecutive digits when RADIX > 256)
    constexpr int DPT = RADIX > kSortThreads ? RADIX / kSortThreads : 1;
    uint32_t tot_d[DPT], gtot_d[DPT];
    uint32_t mine = 0, gmine = 0;
#pragma unroll
    for (int q = 0; q < DPT; ++q) {
        const int d = t * DPT + q;
        tot_d[q] = 0; gtot_d[q] = 0;
        if (d < RADIX) {
            uint32_t run = 0;
            for (int ww = 0; ww < kSortWarps; ++ww) {
                const uint32_t c = wcnt[ww * (RADIX + 1) + d];
                wcnt[ww * (RADIX + 1) + d] = run;
                run += c;
            }
            tot_d[q] = run;
            gtot_d[q] = digit_total[d];
        }
        mine += tot_d[q];
        gmine += gtot_d[q];
    }
    if (t == 0) {   // the padding bin: invalid items sort after every real digit
        uint32_t r2 = 0;
        for (int ww = 0; ww < kSortWarps; ++ww) {
            const uint32_t c = wcnt[ww * (RADIX + 1) + RADIX];
            wcnt[ww * (RADIX + 1) + RADIX] = r2;
            r2 += c;
        }
    }
    uint32_t tot_all, gtot_all;
    uint32_t ex = block_excl_scan<kSortThreads>(mine, sums, &tot_all);
    uint32_t gex = block_excl_scan<kSortThreads>(gmine, sums, &gtot_all);
#pragma unroll
    for (int q = 0; q < DPT; ++q) {
        const int d = t * DPT + q;
        if (d < RADIX) {
            // the warps' offsets inside the digit become positions inside the tile, so that placing a
            // key needs one table look-up
            for (int ww = 0; ww < kSortWarps; ++ww) wcnt[ww * (RADIX + 1) + d] += ex;
            // global base of digit d = totals of smaller digits + this tile's prefix within the digit
            goff[d] = gex + tilehist[(int64_t)d * ntiles + blockIdx.x] - ex;
            ex += tot_d[q];
            gex += gtot_d[q];
        }
    }
    (void)tot_all;
    __syncthreads();

#pragma unroll
    for (int i = 0; i < kSortIpt; ++i) {
        const int li = w * (32 * kSortIpt) + i * 32 + lane;
        const bool valid = li < tile_n;
        const uint32_t d = valid ? ((uint32_t)(key[i] >> shift) & mask) : (uint32_t)RADIX;
        const uint32_t s = mycnt[d] + ((i & 1) ? rank[i / 2] >> 16 : rank[i / 2] & 0xffffu);
        if (valid) {
            skeys[s] = key[i];
            if (PAY) spay[s] = pay[i];
        }
    }
    __syncthreads();
    for (int s = t; s < tile_n; s += kSortThreads) {
        const uint64_t k = skeys[s];
        const uint32_t d = (uint32_t)(k >> shift) & mask;
        const uint32_t o = goff[d] + (uint32_t)s;
        if (PAY) {
            keys_out[o] = k;
            pay_out[o] = spay[s];
        } else if (split_bits >= 0) {
            keys_out[o] = split_bits < 64 ? k >> split_bits : 0;
            idx_out[o] = (uint32_t)(k & ((1ull << split_bits) - 1ull));
        } else {
            keys_out[o] = k;
        }
    }
}

// One radix pass (tile histograms unless they exist already, per-digit scans, ranked scatter) for a
// digit of BITS bits at `shift`.
template <int BITS>
sp_status sort_pass(const uint64_t* kin, const uint64_t* pin, uint64_t* kout, uint64_t* pout, uint32_t* iout, int64_t n, int shift,
                    uint32_t* tilehist, int64_t stiles, uint32_t* digit_total, uint32_t* chunk_tot, bool fused, int split_bits,
                    bool have_hist, cudaStream_t stream, PhaseTimer& timer) {
    if (!have_hist) {
        if (fused) SP_CUDA(sp_launch_dependent(k_sort_upsweep<BITS, false>, dim3((unsigned)stiles), dim3(kSortThreads), 0, stream, kin, n, shift, tilehist, stiles));
        else SP_CUDA(sp_launch_dependent(k_sort_upsweep<BITS, true>, dim3((unsigned)stiles), dim3(kSortThreads), 0, stream, kin, n, shift, tilehist, stiles));
        sp_count_launches(1);
    }
    timer.mark(kPhUpsweep);
    {
        const int64_t nchunks = sp_ceil_div(stiles, kScanChunk);
        dim3 grid(1u << BITS, (unsigned)nchunks);
        if (nchunks > 1) {
            SP_CUDA(sp_launch_dependent(k_sort_chunk_totals, grid, dim3(256), 0, stream, tilehist, stiles, nchunks, chunk_tot));
            sp_count_launches(1);
        }
        SP_CUDA(sp_launch_dependent(k_sort_scan, grid, dim3(256), 0, stream, tilehist, stiles, nchunks, chunk_tot, digit_total));
    }
    timer.mark(kPhScan);
    if (fused) {
        SP_CUDA(cudaFuncSetAttribute(k_sort_downsweep<false, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)down_smem(false, BITS)));
        SP_CUDA(sp_launch_dependent(k_sort_downsweep<false, BITS>, dim3((unsigned)stiles), dim3(kSortThreads), down_smem(false, BITS), stream,
                                 kin, (const uint64_t*)nullptr, kout, (uint64_t*)nullptr, iout, n, shift, (const uint32_t*)tilehist, stiles,
                                 (const uint32_t*)digit_total, split_bits));
    } else {
        SP_CUDA(cudaFuncSetAttribute(k_sort_downsweep<true, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)down_smem(true, BITS)));
        SP_CUDA(sp_launch_dependent(k_sort_downsweep<true, BITS>, dim3((unsigned)stiles), dim3(kSortThreads), down_smem(true, BITS), stream,
                                 kin, pin, kout, pout, (uint32_t*)nullptr, n, shift, (const uint32_t*)tilehist, stiles,
                                 (const uint32_t*)digit_total, -1));
    }
    SP_LAUNCH_CHECK();
    timer.mark(kPhDownsweep);
    sp_count_launches(2);
    return SP_OK;
}

// ------------------------------------------------- flags, counts, emit ---
constexpr int kCtThreads = 256;
constexpr int kCtIpt = 8;
constexpr int kCtTile = kCtThreads * kCtIpt;   // 2048
constexpr int kField = 12;                     // SP_MAX_RANK 12-bit counters (a tile has 2048 entries) in 64 bits
constexpr uint64_t kFieldMask = (1ull << kField) - 1;

__device__ __forceinline__ uint64_t warp_incl_scan64(uint64_t v) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint64_t u = __shfl_up_sync(0xffffffffu, v, o);
        if ((int)sp_lane() >= o) v += u;
    }
    return v;
}

// Exclusive scan of packed counters over a block of up to 512 threads.
__device__ __forceinline__ uint64_t block_excl_scan64(uint64_t v, uint64_t* sums, uint64_t* total) {
    const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    uint64_t incl = warp_incl_scan64(v);
    if (sp_lane() == 31) sums[w] = incl;
    __syncthreads();
    uint64_t pre = 0, tot = 0;
    for (int i = 0; i < nw; ++i) {
        uint64_t s = sums[i];
        if (i < w) pre += s;
        tot += s;
    }
    __syncthreads();
    *total = tot;
    return incl - v + pre;
}

// Per tile of kCtTile sorted entries: how many of them open a node at each level (packed 12-bit
// counters).  Same entry-to-lane layout and the same test as k_emit below: a warp reads 32
// consecutive keys per round, "opens a node at level l" is (significant bits of key ^ previous key)
// > shift[l], and a count is the population count of a ballot.
template <int RANK>
__global__ void __launch_bounds__(kCtThreads)
k_count_flags(const uint64_t* __restrict__ keys, int64_t n, LevelPlan p, uint64_t* __restrict__ tilesum) {
    sp_wait_for_previous_kernel();
    __shared__ uint32_t wtot[kCtThreads / 32][SP_MAX_RANK];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t chunk = (int64_t)blockIdx.x * kCtTile + (int64_t)w * (32 * kCtIpt);
    uint64_t k[kCtIpt];
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        const int64_t e = chunk + i * 32 + lane;
        k[i] = e < n ? keys[e] : 0;
    }
    const uint64_t kbefore = (chunk > 0 && chunk <= n) ? keys[chunk - 1] : 0;
    uint32_t tot[RANK];
#pragma unroll
    for (int l = 0; l < RANK; ++l) tot[l] = 0;
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        const int64_t e = chunk + i * 32 + lane;
        const uint64_t up = __shfl_up_sync(0xffffffffu, k[i], 1);
        const uint64_t wrap = i > 0 ? __shfl_sync(0xffffffffu, k[i > 0 ? i - 1 : 0], 31) : kbefore;
        const uint64_t x = k[i] ^ (lane ? up : wrap);
        const int hb = e >= n ? 0 : (e == 0 ? 64 : 64 - __clzll((long long)x));
#pragma unroll
        for (int l = 0; l < RANK; ++l) tot[l] += (uint32_t)__popc(__ballot_sync(0xffffffffu, hb > p.shift[l]));
    }
    if (lane == 0) {
#pragma unroll
        for (int l = 0; l < RANK; ++l) wtot[w][l] = tot[l];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint64_t packed = 0;
#pragma unroll
        for (int l = 0; l < RANK; ++l) {
            uint32_t c = 0;
            for (int ww = 0; ww < kCtThreads / 32; ++ww) c += wtot[ww][l];
            packed |= (uint64_t)c << (kField * l);
        }
        tilesum[blockIdx.x] = packed;
    }
}

static_assert(kField * SP_MAX_RANK <= 64 && (1 << kField) > kCtTile, "packed per-tile counters");

// One block (512 threads) per level: tilesum (packed) -> tileprefix[l][tile] (exclusive), counts[l].
// Across tiles the counts outgrow the packed fields, so each level is scanned on its own.  A thread
// owns a run of consecutive tiles, so the block scans once however many tiles there are.
__global__ void __launch_bounds__(512)
k_scan_tiles(const uint64_t* __restrict__ tilesum, int64_t ntiles, int rank, int64_t* __restrict__ tileprefix,
             int64_t* __restrict__ counts) {
    sp_wait_for_previous_kernel();
    __shared__ uint64_t sums[16];
    const int64_t per = (ntiles + 511) / 512;
    const int64_t q0 = (int64_t)threadIdx.x * per, q1 = q0 + per < ntiles ? q0 + per : ntiles;
    for (int l = blockIdx.x; l < rank; l += gridDim.x) {
        uint64_t local = 0;
        for (int64_t q = q0; q < q1; ++q) local += (tilesum[q] >> (kField * l)) & kFieldMask;
        uint64_t tot;
        uint64_t run = block_excl_scan64(local, sums, &tot);
        for (int64_t q = q0; q < q1; ++q) {
            tileprefix[(int64_t)l * ntiles + q] = (int64_t)run;
            run += (tilesum[q] >> (kField * l)) & kFieldMask;
        }
        if (threadIdx.x == 0) counts[l] = (int64_t)tot;
    }
}

struct EmitArgs {
    const uint64_t* keys;
    const uint32_t* idx;        // sorted position -> input entry (when the index rode in the key), else null
    const double* vals_in;      // values in input order (read through idx)
    const double* vals_sorted;  // values in sorted order (when they travelled with the keys), else null
    int64_t n;
    LevelPlan plan;
    const int64_t* tileprefix;
    int64_t ntiles;
    void* pos[SP_MAX_RANK];
    void* crd[SP_MAX_RANK];
    double* val;
    uint32_t* seg_out;   // optional: level-0 coordinate of every stored entry (column-major matrices)
    int posBits, crdBits;
    unsigned flags;
    int* err;
    int64_t last_pos[SP_MAX_RANK];   // index of the closing entry of pos[l] (its parents' count) ...
    int64_t last_val[SP_MAX_RANK];   // ... and what goes there: the level's node count
};

#ifdef SP_LB_EMIT
#define SP_EMIT_BOUNDS __launch_bounds__(kCtThreads, SP_LB_EMIT)
#else
#define SP_EMIT_BOUNDS __launch_bounds__(kCtThreads)
#endif
// Writes crd, first-child pos and values of one tile (the tiles of k_count_flags).  A warp owns 256
// consecutive sorted entries and reads them 32 at a time, so every load and - node ids being
// consecutive along the entries - every store of a warp instruction falls on consecutive addresses.
// "Entry e opens a node at level l" is a comparison of the number of significant bits of
// key[e] ^ key[e-1] with the level's shift, so a node id is a ballot and a population count: first
// the warps total their flags per level, then (the totals exchanged through shared memory) each entry
// gets its ids from the same ballots and walks its levels on its own.
// W32: positions and coordinates are stored as 32-bit words (plain stores instead of a width switch).
template <int RANK, bool W32>
__global__ void SP_EMIT_BOUNDS k_emit(EmitArgs a) {
    __shared__ uint32_t wtot[kCtThreads / 32][SP_MAX_RANK];
    const LevelPlan& p = a.plan;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t chunk = (int64_t)blockIdx.x * kCtTile + (int64_t)w * (32 * kCtIpt);
    const uint32_t le_mask = 0xffffffffu >> (31 - lane);          // lanes up to and including this one

    uint64_t k[kCtIpt];
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        const int64_t e = chunk + i * 32 + lane;
        k[i] = e < a.n ? a.keys[e] : 0;
    }
    if (blockIdx.x == 0 && threadIdx.x < RANK && p.lt[threadIdx.x] == SP_COMPRESSED)   // pos[l] ends with the node count
        sp_store_uint(a.pos[threadIdx.x], a.last_pos[threadIdx.x], (uint64_t)a.last_val[threadIdx.x], a.posBits);
    // this thread's values, requested before anything is computed
    double vin[kCtIpt];
    if (a.vals_sorted) {
#pragma unroll
        for (int i = 0; i < kCtIpt; ++i) { const int64_t e = chunk + i * 32 + lane; vin[i] = e < a.n ? a.vals_sorted[e] : 0.0; }
    } else {
        uint32_t id[kCtIpt];
#pragma unroll
        for (int i = 0; i < kCtIpt; ++i) { const int64_t e = chunk + i * 32 + lane; id[i] = e < a.n ? a.idx[e] : 0u; }
#pragma unroll
        for (int i = 0; i < kCtIpt; ++i) vin[i] = a.vals_in[id[i]];
    }
    const uint64_t kbefore = (chunk > 0 && chunk <= a.n) ? a.keys[chunk - 1] : 0;   // uniform per warp
    // key of the entry before entry (i, lane)
    auto prev_key = [&](int i) -> uint64_t {
        const uint64_t up = __shfl_up_sync(0xffffffffu, k[i], 1);
        const uint64_t wrap = i > 0 ? __shfl_sync(0xffffffffu, k[i > 0 ? i - 1 : 0], 31) : kbefore;
        return lane ? up : wrap;
    };
    // significant bits of key ^ previous key (64 for the very first entry, 0 past the end): the entry
    // opens a node at level l exactly when this exceeds shift[l]
    int hb[kCtIpt];
    uint32_t tot[RANK];
#pragma unroll
    for (int l = 0; l < RANK; ++l) tot[l] = 0;
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        const int64_t e = chunk + i * 32 + lane;
        const uint64_t x = k[i] ^ prev_key(i);
        hb[i] = e >= a.n ? 0 : (e == 0 ? 64 : 64 - __clzll((long long)x));
#pragma unroll
        for (int l = 0; l < RANK; ++l) tot[l] += (uint32_t)__popc(__ballot_sync(0xffffffffu, hb[i] > p.shift[l]));
    }
    if (lane == 0) {
#pragma unroll
        for (int l = 0; l < RANK; ++l) wtot[w][l] = tot[l];
    }

    __syncthreads();

    uint32_t run[RANK];                           // flagged entries at level l before this warp's round (< nnz < 2^32)
#pragma unroll
    for (int l = 0; l < RANK; ++l) {
        uint32_t r = (uint32_t)a.tileprefix[(int64_t)l * a.ntiles + blockIdx.x];
        for (int ww = 0; ww < w; ++ww) r += wtot[ww][l];
        run[l] = r;
    }
    const uint64_t knext = (chunk + 32 * kCtIpt < a.n) ? a.keys[chunk + 32 * kCtIpt] : ~0ull;   // uniform per warp
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        const int64_t e = chunk + i * 32 + lane;
        // does the entry after this one repeat its coordinates?  (its last-level flag is clear)
        int hb_next = __shfl_down_sync(0xffffffffu, hb[i], 1);
        const int hb_wrap = __shfl_sync(0xffffffffu, hb[i + 1 < kCtIpt ? i + 1 : i], 0);
        if (lane == 31) hb_next = i + 1 < kCtIpt ? hb_wrap : ((e + 1 < a.n && knext == k[i]) ? 0 : 64);
        // Walk the levels.  `parent` is the position of this entry's node one level up: a node id under a
        // compressed level, parent * size + coordinate under a dense one; it is a new position exactly
        // when the level above opened a node for this entry (its flag), or for the very first entry.
        int64_t parent = 0;
        bool parent_new = e == 0;
#pragma unroll
        for (int l = 0; l < RANK; ++l) {
            const bool fl = hb[i] > p.shift[l];                                           // never set past the end
            const uint64_t c = (k[i] >> p.shift[l]) & (((uint64_t)1 << p.bits[l]) - 1);   // bits[l] <= 63
            if (p.lt[l] == SP_DENSE) {                                                    // uniform branch
                parent = parent * p.sz[l] + (int64_t)c;
            } else {
                const uint32_t m = __ballot_sync(0xffffffffu, fl);
                const uint32_t nid = run[l] + (uint32_t)__popc(m & le_mask) - 1u;
                run[l] += (uint32_t)__popc(m);
                if (fl) {
                    if (W32) static_cast<uint32_t*>(a.crd[l])[nid] = (uint32_t)c;
                    else sp_store_uint(a.crd[l], nid, c, a.crdBits);
                    if (parent_new) {
                        if (W32) static_cast<uint32_t*>(a.pos[l])[parent] = nid;
                        else sp_store_uint(a.pos[l], parent, (uint64_t)nid, a.posBits);
                    }
                }
                parent = nid;
            }
            parent_new = fl;
        }
        const bool full = parent_new;
        const int64_t ppos = parent;
        if (e >= a.n) continue;
        if (full) {
            double s = vin[i];
            if (e + 1 < a.n && !(hb_next > p.shift[RANK - 1]))   // rare: the run of equal coordinates is summed by its first entry
                for (int64_t g = e + 1; g < a.n && a.keys[g] == k[i]; ++g) s += a.vals_sorted ? a.vals_sorted[g] : a.vals_in[a.idx[g]];
            a.val[ppos] = s;
            if (a.seg_out) a.seg_out[ppos] = (uint32_t)(k[i] >> p.shift[0]);
        } else if (a.flags & SP_DUP_ERROR) {
            atomicOr(a.err, kErrDup);
        }
    }
}

// --------------------------------------------- suffix-min fill of pos[] ---
// a[i] <- min(a[i..L-1]).  Written as a forward scan over r = L-1-i.
template <typename T>
__device__ __forceinline__ T tmin(T a, T b) { return a < b ? a : b; }

template <typename T>
__device__ __forceinline__ T block_excl_minscan(T v, T* sums, T* total, T ident) {
    const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    T incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T u = __shfl_up_sync(0xffffffffu, incl, o);
        if ((int)sp_lane() >= o) incl = tmin(incl, u);
    }
    T exw = __shfl_up_sync(0xffffffffu, incl, 1);
    if (sp_lane() == 0) exw = ident;
    if (sp_lane() == 31) sums[w] = incl;
    __syncthreads();
    T pre = ident, tot = ident;
    for (int i = 0; i < nw; ++i) {
        T s = sums[i];
        if (i < w) pre = tmin(pre, s);
        tot = tmin(tot, s);
    }
    __syncthreads();
    *total = tot;
    return tmin(pre, exw);
}

template <typename T>
__global__ void __launch_bounds__(kCtThreads) k_rmin_reduce(const T* __restrict__ a, int64_t L, T* __restrict__ tilemin) {
    __shared__ T sums[16];
    const T ident = ~(T)0;
    int64_t r0 = (int64_t)blockIdx.x * kCtTile + (int64_t)threadIdx.x * kCtIpt;
    T m = ident;
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        int64_t r = r0 + i;
        if (r < L) m = tmin(m, a[L - 1 - r]);
    }
    T tot;
    block_excl_minscan<T>(m, sums, &tot, ident);
    if (threadIdx.x == 0) tilemin[blockIdx.x] = tot;
}

template <typename T>
__global__ void __launch_bounds__(512) k_rmin_tiles(T* tilemin, int64_t ntiles) {
    sp_wait_for_previous_kernel();
    __shared__ T sums[16];
    const T ident = ~(T)0;
    T carry = ident;
    for (int64_t base = 0; base < ntiles; base += 512) {
        int64_t i = base + threadIdx.x;
        T v = i < ntiles ? tilemin[i] : ident;
        T tot;
        T ex = block_excl_minscan<T>(v, sums, &tot, ident);
        if (i < ntiles) tilemin[i] = tmin(ex, carry);
        carry = tmin(carry, tot);
    }
}

template <typename T>
__global__ void __launch_bounds__(kCtThreads) k_rmin_apply(T* __restrict__ a, int64_t L, const T* __restrict__ tilecarry) {
    sp_wait_for_previous_kernel();
    __shared__ T sums[16];
    const T ident = ~(T)0;
    int64_t r0 = (int64_t)blockIdx.x * kCtTile + (int64_t)threadIdx.x * kCtIpt;
    T v[kCtIpt];
    T m = ident;
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        int64_t r = r0 + i;
        v[i] = r < L ? a[L - 1 - r] : ident;
        m = tmin(m, v[i]);
    }
    T tot;
    T run = tmin(block_excl_minscan<T>(m, sums, &tot, ident), tilecarry[blockIdx.x]);
#pragma unroll
    for (int i = 0; i < kCtIpt; ++i) {
        int64_t r = r0 + i;
        run = tmin(run, v[i]);
        if (r < L) a[L - 1 - r] = run;
    }
}

template <typename T>
sp_status suffix_min_inplace(void* a, int64_t L, cudaStream_t stream) {
    if (L <= 0) return SP_OK;
    int64_t ntiles = sp_ceil_div(L, kCtTile);
    sp_workspace ws(stream);
    T* tm = ws.get<T>((size_t)ntiles);
    if (ws.failed) return SP_ERR_ALLOC;
    k_rmin_reduce<T><<<(unsigned)ntiles, kCtThreads, 0, stream>>>(static_cast<const T*>(a), L, tm);
    SP_CUDA(sp_launch_dependent(k_rmin_tiles<T>, dim3(1), dim3(512), 0, stream, tm, ntiles));
    SP_CUDA(sp_launch_dependent(k_rmin_apply<T>, dim3((unsigned)ntiles), dim3(kCtThreads), 0, stream, static_cast<T*>(a), L, (const T*)tm));
    sp_count_launches(3);
    SP_LAUNCH_CHECK();
    return SP_OK;
}

// ---------------------------------------------------------------- unpack ---
struct UnpackArgs {
    int rank;
    int lt[SP_MAX_RANK], ord[SP_MAX_RANK];
    int64_t sz[SP_MAX_RANK];
    const void* pos[SP_MAX_RANK];
    int64_t npos[SP_MAX_RANK];
    const void* crd[SP_MAX_RANK];
    const double* val;
    int64_t nval;
    int posBits, crdBits;
    int64_t* out[SP_MAX_RANK];
    double* vals_out;
};

__global__ void k_unpack(UnpackArgs a) {
    int64_t q = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (q >= a.nval) return;
    a.vals_out[q] = a.val[q];
    int64_t p = q;
    for (int l = a.rank - 1; l >= 0; --l) {
        int64_t c;
        if (a.lt[l] == SP_DENSE) {
            c = p % a.sz[l];
            p /= a.sz[l];
        } else {
            c = (int64_t)sp_load_uint(a.crd[l], p, a.crdBits);
            // parent = last index whose offset is <= p
            int64_t lo = 0, hi = a.npos[l] - 1;   // answer in [0, npos-2]
            while (hi - lo > 1) {
                int64_t mid = (lo + hi) >> 1;
                if ((int64_t)sp_load_uint(a.pos[l], mid, a.posBits) <= p) lo = mid; else hi = mid;
            }
            p = lo;
        }
        a.out[a.ord[l]][q] = c;
    }
}

int ceil_log2(int64_t v) {   // bits needed for coordinates 0..v-1
    int b = 0;
    while (b < 63 && ((int64_t)1 << b) < v) ++b;
    return b;
}

// ---------------------------------------------------------------------------
sp_status pack_impl(int rank, const int64_t* dims, int64_t nnz, const void* const* coo_coords,
                    int coo_coord_bits, const double* coo_vals, const sp_level_type* dimLevelType,
                    const int* dimOrdering, int posBits, int crdBits, unsigned flags, void* stream_,
                    sp_tensor** out, PackTimes* times) {
    if (!out) return SP_ERR_INVALID_ARG;
    *out = nullptr;
    if (rank < 1 || rank > SP_MAX_RANK || !dims || !dimLevelType || nnz < 0) return SP_ERR_INVALID_ARG;
    if (nnz > 0 && (!coo_coords || !coo_vals)) return SP_ERR_INVALID_ARG;
    if (coo_coord_bits != 32 && coo_coord_bits != 64) return SP_ERR_INVALID_ARG;
    if (posBits == 0) posBits = 64;
    if (crdBits == 0) crdBits = 64;
    if (!sp_valid_width(posBits) || !sp_valid_width(crdBits)) return SP_ERR_INVALID_ARG;
    if (flags > SP_DUP_ERROR) return SP_ERR_INVALID_ARG;
    if (nnz >= ((int64_t)1 << 32)) return SP_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    LevelPlan plan;
    memset(&plan, 0, sizeof plan);
    plan.rank = rank;
    bool seen[SP_MAX_RANK] = {};
    int total_bits = 0;
    for (int l = 0; l < rank; ++l) {
        int d = dimOrdering ? dimOrdering[l] : l;
        if (d < 0 || d >= rank || seen[d]) return SP_ERR_INVALID_ARG;
        seen[d] = true;
        if (dims[d] < 1) return SP_ERR_INVALID_ARG;
        if (dimLevelType[l] != SP_DENSE && dimLevelType[l] != SP_COMPRESSED) return SP_ERR_INVALID_ARG;
        if (nnz > 0 && !coo_coords[d]) return SP_ERR_INVALID_ARG;
        plan.src[l] = d;
        plan.sz[l] = dims[d];
        plan.lt[l] = dimLevelType[l];
        plan.bits[l] = ceil_log2(dims[d]);
        total_bits += plan.bits[l];
    }
    if (total_bits > 63) return SP_ERR_UNSUPPORTED;
    for (int l = 0, s = total_bits; l < rank; ++l) { s -= plan.bits[l]; plan.shift[l] = s; }

    const uint64_t max_pos = sp_width_max(posBits);
    const uint64_t max_crd = sp_width_max(crdBits);
    for (int l = 0; l < rank; ++l)
        if (plan.lt[l] == SP_COMPRESSED && (uint64_t)(plan.sz[l] - 1) > max_crd) return SP_ERR_WIDTH_OVERFLOW;

    sp_workspace ws(stream);
    PhaseTimer timer(stream, times);
    int npasses_done = 0;
    const int64_t n = nnz;
    int64_t counts[SP_MAX_RANK] = {};
    uint64_t* keys = nullptr;
    uint32_t* idx = nullptr;            // sorted position -> input entry (index-in-key sorts)
    const double* vals_sorted = nullptr;   // or the values in sorted order (value-beside-key sorts)
    int64_t* tileprefix = nullptr;
    int* d_err = nullptr;
    int64_t ct_tiles = 0;

    if (n > 0) {
        const int npasses = (total_bits + kMaxDigitBits - 1) / kMaxDigitBits;
        // the entry index rides inside the key when both fit in 64 bits; otherwise the values travel
        // beside the keys (one array per side of the ping-pong; the first pass reads the input's)
        int idx_bits = 0;
        while (((int64_t)1 << idx_bits) < n) ++idx_bits;
        const bool fused = npasses > 0 && idx_bits > 0 && total_bits + idx_bits <= 64;
        const int64_t stiles = sp_ceil_div(n, fused ? SortShape<false>::kTile : SortShape<true>::kTile);
        ct_tiles = sp_ceil_div(n, kCtTile);
        const size_t nscan = (size_t)sp_ceil_div(stiles, kScanChunk) << kMaxDigitBits;
        // every buffer of the pack in one allocation
        ws.reserve(2 * sp_workspace::bytes_for<uint64_t>((size_t)n) +
                   (fused ? sp_workspace::bytes_for<uint32_t>((size_t)n) : npasses > 0 ? 2 * sp_workspace::bytes_for<uint64_t>((size_t)n) : 0) +
                   sp_workspace::bytes_for<uint32_t>((size_t)stiles << kMaxDigitBits) +
                   sp_workspace::bytes_for<uint32_t>((size_t)1 << kMaxDigitBits) + sp_workspace::bytes_for<uint32_t>(nscan) +
                   sp_workspace::bytes_for<uint64_t>((size_t)ct_tiles) + sp_workspace::bytes_for<int64_t>((size_t)ct_tiles * SP_MAX_RANK) +
                   sp_workspace::bytes_for<int64_t>(SP_MAX_RANK + 1));
        uint64_t* kbuf[2] = {ws.get<uint64_t>((size_t)n), ws.get<uint64_t>((size_t)n)};
        uint64_t* pbuf[2] = {nullptr, nullptr};
        uint32_t* isorted = nullptr;
        if (fused) isorted = ws.get<uint32_t>((size_t)n);
        else if (npasses > 0) { pbuf[0] = ws.get<uint64_t>((size_t)n); pbuf[1] = ws.get<uint64_t>((size_t)n); }
        uint32_t* tilehist = ws.get<uint32_t>((size_t)stiles << kMaxDigitBits);
        uint32_t* digit_total = ws.get<uint32_t>((size_t)1 << kMaxDigitBits);
        uint32_t* chunk_tot = ws.get<uint32_t>(nscan);
        uint64_t* tilesum = ws.get<uint64_t>((size_t)ct_tiles);
        tileprefix = ws.get<int64_t>((size_t)ct_tiles * SP_MAX_RANK);
        int64_t* d_counts = ws.get<int64_t>(SP_MAX_RANK + 1);      // node counts per level, then the error word
        if (ws.failed) return SP_ERR_ALLOC;
        d_err = reinterpret_cast<int*>(d_counts + SP_MAX_RANK);
        SP_CUDA(cudaMemsetAsync(d_err, 0, sizeof(int64_t), stream));

        LevelCoords lc;
        for (int l = 0; l < SP_MAX_RANK; ++l) lc.p[l] = coo_coords[l < rank ? plan.src[l] : 0];
        // digit widths as even as possible, the wider ones first
        int widths[16], shifts[16];
        for (int ps = 0, kshift = 0; ps < npasses; ++ps) {
            const int left = npasses - ps;
            widths[ps] = (total_bits - kshift + left - 1) / left;
            shifts[ps] = kshift + (fused ? idx_bits : 0);
            kshift += widths[ps];
        }
        const int shift0 = npasses ? shifts[0] : 0;
        const uint32_t mask0 = npasses ? (1u << widths[0]) - 1u : 0u;
#define SP_BUILD_KEYS(CT, PAY)                                                                                       \
    k_build_keys<CT, PAY><<<(unsigned)stiles, kSortThreads, 0, stream>>>(lc, n, plan, kbuf[0], fused ? idx_bits : 0,         \
                                                                        d_err, shift0, mask0, tilehist, stiles)
        if (coo_coord_bits == 32) { if (fused) SP_BUILD_KEYS(int32_t, false); else SP_BUILD_KEYS(int32_t, true); }
        else { if (fused) SP_BUILD_KEYS(int64_t, false); else SP_BUILD_KEYS(int64_t, true); }
#undef SP_BUILD_KEYS
        SP_LAUNCH_CHECK();
        sp_count_launches(1);
        timer.mark(kPhKeys);
        int cur = 0;
        for (int ps = 0; ps < npasses; ++ps) {
            const bool last = ps == npasses - 1;
            const int split = (fused && last) ? idx_bits : -1;
            sp_status ps_st = SP_ERR_UNSUPPORTED;
#define SP_SORT_PASS(B)                                                                                             \
    case B:                                                                                                         \
        ps_st = sort_pass<B>(kbuf[cur], ps == 0 ? reinterpret_cast<const uint64_t*>(coo_vals) : pbuf[cur],          \
                             kbuf[cur ^ 1], pbuf[cur ^ 1], isorted, n, shifts[ps], tilehist, stiles,                 \
                             digit_total, chunk_tot, fused, split, ps == 0, stream, timer);                          \
        break;
            switch (widths[ps]) {
                SP_SORT_PASS(1) SP_SORT_PASS(2) SP_SORT_PASS(3) SP_SORT_PASS(4) SP_SORT_PASS(5)
                SP_SORT_PASS(6) SP_SORT_PASS(7) SP_SORT_PASS(8)
            }
#undef SP_SORT_PASS
            if (ps_st != SP_OK) return ps_st;
            cur ^= 1;
        }
        npasses_done = npasses;
        keys = kbuf[cur];
        if (fused) idx = isorted;
        else vals_sorted = npasses > 0 ? reinterpret_cast<const double*>(pbuf[cur]) : coo_vals;   // no pass: one cell

        switch (rank) {
            case 1: SP_CUDA(sp_launch_dependent(k_count_flags<1>, dim3((unsigned)ct_tiles), dim3(kCtThreads), 0, stream, (const uint64_t*)keys, n, plan, tilesum)); break;
            case 2: SP_CUDA(sp_launch_dependent(k_count_flags<2>, dim3((unsigned)ct_tiles), dim3(kCtThreads), 0, stream, (const uint64_t*)keys, n, plan, tilesum)); break;
            case 3: SP_CUDA(sp_launch_dependent(k_count_flags<3>, dim3((unsigned)ct_tiles), dim3(kCtThreads), 0, stream, (const uint64_t*)keys, n, plan, tilesum)); break;
            case 4: SP_CUDA(sp_launch_dependent(k_count_flags<4>, dim3((unsigned)ct_tiles), dim3(kCtThreads), 0, stream, (const uint64_t*)keys, n, plan, tilesum)); break;
            default: SP_CUDA(sp_launch_dependent(k_count_flags<5>, dim3((unsigned)ct_tiles), dim3(kCtThreads), 0, stream, (const uint64_t*)keys, n, plan, tilesum)); break;
        }
        SP_CUDA(sp_launch_dependent(k_scan_tiles, dim3(rank), dim3(512), 0, stream, (const uint64_t*)tilesum, ct_tiles, rank, tileprefix, d_counts));
        SP_LAUNCH_CHECK();
        timer.mark(kPhCount);
        sp_count_launches(3);
        int64_t h_back[SP_MAX_RANK + 1] = {};          // one read-back: the counts and the error word
        SP_CUDA(cudaMemcpyAsync(h_back, d_counts, sizeof h_back, cudaMemcpyDeviceToHost, stream));
        SP_CUDA(cudaStreamSynchronize(stream));
        for (int l = 0; l < SP_MAX_RANK; ++l) counts[l] = h_back[l];
        const int h_err = (int)(h_back[SP_MAX_RANK] & 0xffffffff);
        if (h_err & kErrRange) return SP_ERR_OUT_OF_RANGE;
        if ((flags & SP_DUP_ERROR) && counts[rank - 1] != n) return SP_ERR_DUPLICATE;
    }

    // sizes of the level arrays
    sp_tensor* t = new sp_tensor();
    cudaGetDevice(&t->device);
    t->rank = rank;
    t->posBits = posBits;
    t->crdBits = crdBits;
    const size_t pw = posBits / 8, cw = crdBits / 8;
    sp_status st = SP_OK;
    int64_t parents = 1;
    int64_t parents_at[SP_MAX_RANK] = {};
    for (int l = 0; l < rank && st == SP_OK; ++l) {
        t->dims[l] = dims[l];
        t->lt[l] = plan.lt[l];
        t->ord[l] = plan.src[l];
        parents_at[l] = parents;
        if (plan.lt[l] == SP_DENSE) {
            if (parents > 0 && plan.sz[l] > (((int64_t)1 << 62) / parents)) { st = SP_ERR_ALLOC; break; }
            parents *= plan.sz[l];
        } else {
            if ((uint64_t)counts[l] > max_pos) { st = SP_ERR_WIDTH_OVERFLOW; break; }
            t->npos[l] = parents + 1;
            t->ncrd[l] = counts[l];
            parents = counts[l];
        }
    }
    if (st == SP_OK) {
        // one allocation holds every array of the handle (each piece 256-byte aligned): an allocator
        // call costs host time during which the GPU, drained by the read-back above, has nothing to do
        t->nval = parents;
        size_t off_pos[SP_MAX_RANK] = {}, off_crd[SP_MAX_RANK] = {}, total = 0;
        for (int l = 0; l < rank; ++l) {
            if (plan.lt[l] != SP_COMPRESSED) continue;
            off_pos[l] = total; total += sp_workspace::padded((size_t)t->npos[l] * pw);
            off_crd[l] = total; total += sp_workspace::padded((size_t)(t->ncrd[l] ? t->ncrd[l] : 1) * cw);
        }
        const size_t off_val = total;
        total += sp_workspace::padded((size_t)(parents ? parents : 1) * sizeof(double));
        t->block = sp_dev_alloc(total, stream);
        if (!t->block) {
            st = SP_ERR_ALLOC;
        } else {
            char* base = static_cast<char*>(t->block);
            for (int l = 0; l < rank; ++l) {
                if (plan.lt[l] != SP_COMPRESSED) continue;
                t->pos[l] = base + off_pos[l];
                t->crd[l] = base + off_crd[l];
            }
            t->val = reinterpret_cast<double*>(base + off_val);
        }
    }
    if (st != SP_OK) { sp_free(t); return st; }

    auto fail = [&](sp_status s) { sp_free(t); return s; };
#define SP_CUDA_T(call) do { if ((call) != cudaSuccess) return fail(SP_ERR_CUDA); } while (0)

    const bool trailing_dense = plan.lt[rank - 1] == SP_DENSE;
    if (trailing_dense && t->nval > 0) SP_CUDA_T(cudaMemsetAsync(t->val, 0, (size_t)t->nval * sizeof(double), stream));
    bool needs_fill[SP_MAX_RANK] = {};
    for (int l = 0; l < rank; ++l) {
        if (plan.lt[l] != SP_COMPRESSED) continue;
        needs_fill[l] = n > 0 && l >= 1 && plan.lt[l - 1] == SP_DENSE;
        if (n == 0) SP_CUDA_T(cudaMemsetAsync(t->pos[l], 0, (size_t)t->npos[l] * pw, stream));
        else if (needs_fill[l]) SP_CUDA_T(cudaMemsetAsync(t->pos[l], 0xFF, (size_t)t->npos[l] * pw, stream));
    }
    if (n > 0) {
        EmitArgs a;
        a.keys = keys; a.idx = idx; a.vals_in = coo_vals; a.vals_sorted = vals_sorted; a.n = n; a.plan = plan;
        a.tileprefix = tileprefix; a.ntiles = ct_tiles;
        for (int l = 0; l < SP_MAX_RANK; ++l) { a.pos[l] = t->pos[l]; a.crd[l] = t->crd[l]; }
        a.val = t->val; a.posBits = posBits; a.crdBits = crdBits; a.flags = flags; a.err = d_err;
        for (int l = 0; l < SP_MAX_RANK; ++l) { a.last_pos[l] = parents_at[l]; a.last_val[l] = counts[l]; }
        // Column-major matrices run SpMM as a flat loop over entries and need each entry's column:
        // it is in the sorted key anyway, so it is written here instead of being searched for later.
        a.seg_out = nullptr;
        if (rank == 2 && plan.src[0] == 1 && plan.lt[1] == SP_COMPRESSED && plan.sz[0] < ((int64_t)1 << 32)) {
            sp_partition sg;
            sg.aux = static_cast<int64_t*>(sp_dev_alloc((size_t)(t->nval ? t->nval : 1) * sizeof(uint32_t), stream));
            if (!sg.aux) return fail(SP_ERR_ALLOC);
            a.seg_out = reinterpret_cast<uint32_t*>(sg.aux);
            t->parts[(uint64_t)SP_PART_SEGIDS << 56] = sg;
        }
        const bool w32 = posBits == 32 && crdBits == 32;
#define SP_EMIT(R)                                                                              \
    case R:                                                                                     \
        if (w32) k_emit<R, true><<<(unsigned)ct_tiles, kCtThreads, 0, stream>>>(a);             \
        else k_emit<R, false><<<(unsigned)ct_tiles, kCtThreads, 0, stream>>>(a);                \
        break;
        switch (rank) { SP_EMIT(1) SP_EMIT(2) SP_EMIT(3) SP_EMIT(4) SP_EMIT(5) }
#undef SP_EMIT
        sp_count_launches(1);
        for (int l = 0; l < rank; ++l) {
            if (plan.lt[l] != SP_COMPRESSED) continue;
            if (needs_fill[l]) {
                sp_status s2 = posBits == 64   ? suffix_min_inplace<uint64_t>(t->pos[l], t->npos[l], stream)
                               : posBits == 32 ? suffix_min_inplace<uint32_t>(t->pos[l], t->npos[l], stream)
                               : posBits == 16 ? suffix_min_inplace<uint16_t>(t->pos[l], t->npos[l], stream)
                                               : suffix_min_inplace<uint8_t>(t->pos[l], t->npos[l], stream);
                if (s2 != SP_OK) return fail(s2);
            }
        }
        SP_CUDA_T(cudaGetLastError());
        timer.mark(kPhEmit);
        timer.finish(npasses_done);
        // the workspace is released below; with the default allocator cudaFree waits for the stream
    }
#undef SP_CUDA_T
    *out = t;
    return SP_OK;
}

}  // namespace

#ifdef SP_BENCH_BUILD
// The benchmark's library: the same packer with its phases bracketed by events.
// phase_ms: host, 6 entries (key build, sort histograms, sort scans, sort scatters, node counting,
// emit + fill); npasses: host, number of radix passes.
extern "C" sp_status spb_pack_timed(int rank, const int64_t* dims, int64_t nnz, const void* const* coo_coords,
                                    int coo_coord_bits, const double* coo_vals, const sp_level_type* dimLevelType,
                                    const int* dimOrdering, int posBits, int crdBits, unsigned flags, void* stream_,
                                    sp_tensor** out, double* phase_ms, int* npasses) {
    if (!phase_ms) return SP_ERR_INVALID_ARG;
    PackTimes t = {};
    const sp_status st = pack_impl(rank, dims, nnz, coo_coords, coo_coord_bits, coo_vals, dimLevelType, dimOrdering,
                                   posBits, crdBits, flags, stream_, out, &t);
    for (int i = 0; i < kPhCount_; ++i) phase_ms[i] = t.ms[i];
    if (npasses) *npasses = t.passes;
    return st;
}
#else
extern "C" sp_status sp_pack(int rank, const int64_t* dims, int64_t nnz, const void* const* coo_coords,
                             int coo_coord_bits, const double* coo_vals, const sp_level_type* dimLevelType,
                             const int* dimOrdering, int posBits, int crdBits, unsigned flags, void* stream_,
                             sp_tensor** out) {
    SP_API_RANGE("sp_pack");
    return pack_impl(rank, dims, nnz, coo_coords, coo_coord_bits, coo_vals, dimLevelType, dimOrdering, posBits,
                     crdBits, flags, stream_, out, nullptr);
}

extern "C" sp_status sp_unpack(const sp_tensor* t, void* const* coo_coords_out, double* vals_out,
                               int64_t* nnz_out, void* stream_) {
    SP_API_RANGE("sp_unpack");
    if (!t || !coo_coords_out || !vals_out || !nnz_out) return SP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    UnpackArgs a;
    memset(&a, 0, sizeof a);
    a.rank = t->rank;
    for (int l = 0; l < t->rank; ++l) {
        if (!coo_coords_out[l]) return SP_ERR_INVALID_ARG;
        a.lt[l] = t->lt[l];
        a.ord[l] = t->ord[l];
        a.sz[l] = t->dims[t->ord[l]];
        a.pos[l] = t->pos[l];
        a.npos[l] = t->npos[l];
        a.crd[l] = t->crd[l];
        a.out[l] = static_cast<int64_t*>(coo_coords_out[l]);
    }
    a.val = t->val;
    a.nval = t->nval;
    a.posBits = t->posBits;
    a.crdBits = t->crdBits;
    a.vals_out = vals_out;
    *nnz_out = t->nval;
    if (t->nval > 0) {
        k_unpack<<<(unsigned)sp_ceil_div(t->nval, 256), 256, 0, stream>>>(a);
        sp_count_launches(1);
        SP_LAUNCH_CHECK();
    }
    return SP_OK;
}

// sp_convert: storage -> coordinates -> storage (Section 4.2: conversions between sparse formats go
// through an intermediate coordinate scheme rather than one direct converter per pair of formats).
extern "C" sp_status sp_convert(const sp_tensor* t, const sp_level_type* dimLevelType, const int* dimOrdering,
                                int posBits, int crdBits, void* stream_, sp_tensor** out) {
    SP_API_RANGE("sp_convert");
    if (!out) return SP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!t || !dimLevelType) return SP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    sp_workspace ws(stream);
    const int64_t n = t->nval;
    void* coords[SP_MAX_RANK] = {};
    for (int d = 0; d < t->rank; ++d) coords[d] = ws.get<int64_t>((size_t)n);
    double* vals = ws.get<double>((size_t)n);
    if (ws.failed) return SP_ERR_ALLOC;
    int64_t cnt = 0;
    sp_status st = sp_unpack(t, coords, vals, &cnt, stream_);
    if (st != SP_OK) return st;
    return sp_pack(t->rank, t->dims, cnt, coords, 64, vals, dimLevelType, dimOrdering, posBits, crdBits, SP_DUP_SUM,
                   stream_, out);
}
#endif  // SP_BENCH_BUILD
