/*
 * bench_probes.h - measurement aids of bench.py (libbench_probes.so).
 *
 * Not part of the product library and not declared in include/sp.h: the paper has no
 * counterpart for any of this.  The library holds
 *   - three microbenchmarks for the secondary bounds of the row-gather kernels (SpMM, SDDMM and
 *     MTTKRP fetch one dense row per stored entry): the rate at which all SMs together fetch
 *     rows of a table at caller-supplied row numbers, the same for single 8-byte elements (the
 *     access SpMV makes to x), and the register-only f64 multiply-add rate;
 *   - spb_pack_timed: the product's packer (the same source file, compiled a second time) with
 *     CUDA events between its phases, which is how bench.py times one radix scatter pass.
 * Every call enqueues on `stream` (a cudaStream_t as void*) and returns an sp_status value
 * (0 = ok); all data pointers are DEVICE pointers unless marked host.
 */
#ifndef BENCH_PROBES_H
#define BENCH_PROBES_H

#include <stdint.h>

#include "sp.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * spb_gather_rows: fetch n_ids whole rows of table[rows x row_elems] (row-major f64, 16-byte
 * aligned) at the row numbers row_ids[0..n_ids) (uint32, each < rows; the caller draws them, so
 * the timed loop holds no random-number arithmetic).  A warp reads 32 row numbers with one
 * coalesced load and hands them to its lane groups with shuffles - the way the gather kernels
 * obtain their coordinates - and a lane group keeps 8 row fetches (16 bytes per lane per load) in
 * flight.  row_elems: 16, 32, 64 or 128, or 1 for single elements (one per lane, 8 in flight).
 * n_ids must be a multiple of 32 * blocks * 8 (whole batches per warp).  sink (blocks * 256
 * doubles) receives per-thread sums so that no load can be dropped.  Bytes moved =
 * n_ids * row_elems * 8 (+ 4 * n_ids for the row numbers).
 */
int spb_gather_rows(const double* table, int64_t rows, int64_t row_elems, const uint32_t* row_ids,
                    int64_t n_ids, int64_t blocks, double* sink, void* stream);

/*
 * spb_dfma: blocks x 256 threads each run eight independent chains of `iters` dependent f64
 * fused multiply-adds held in registers; flops = 2 * blocks * 256 * 8 * iters.
 */
int spb_dfma(int64_t blocks, int64_t iters, double* sink, void* stream);

/*
 * spb_pack_timed: sp_pack with its phases timed.  Arguments as sp_pack; phase_ms (host, 6
 * entries): key build, sort histograms, sort scans, sort scatters, node counting, emit + fill;
 * npasses (host, may be NULL): number of radix passes.  The handle is a normal sp_tensor
 * (release it with sp_free).
 */
int spb_pack_timed(int rank, const int64_t* dims, int64_t nnz, const void* const* coo_coords,
                   int coo_coord_bits, const double* coo_vals, const sp_level_type* dimLevelType,
                   const int* dimOrdering, int posBits, int crdBits, unsigned flags, void* stream,
                   sp_tensor** out, double* phase_ms, int* npasses);

#ifdef __cplusplus
}
#endif
#endif /* BENCH_PROBES_H */
