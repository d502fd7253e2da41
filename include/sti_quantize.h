/*
 * sti_quantize.h - the shard quantizer of STI (arXiv 2207.05022: the outlier-aware quantization of
 * Section 6, which produces the K fidelity versions Section 4.2 stores per shard) on the device.
 *
 * The paper runs this step offline in the cloud (Python + scikit-learn, minutes per bitwidth);
 * here one call turns fp32 shard units that already sit in device memory into the upload format of
 * sti_shard_upload (sti.h), so that the N x M x K shard versions of a model can be produced where the
 * weights are.  Per unit, on its flat fp32 array of n_weights values:
 *   1. fit one Gaussian (maximum likelihood: mean, 1/n variance);
 *   2. weights with log-likelihood below -4 are outliers, kept verbatim as (offset, value), ascending offset;
 *   3. the others are sorted (equal values keep their original order) and cut into 2^bits clusters of equal
 *      population, cluster c = sorted[floor(c n'/2^bits) : floor((c+1) n'/2^bits));
 *   4. centroid = arithmetic mean of the cluster (fp64 sum, rounded once to fp32; 0 for an empty cluster);
 *   5. every weight gets its cluster's index, an outlier's slot the index of the nearest centroid (the
 *      lower index on a tie; the paper only says that outliers are "also" stored as k-bit integers);
 *   6. indexes are packed: index i at stream bits [i*bits, i*bits + bits), least-significant bit first,
 *      little-endian 32-bit words.  A unit's matrices all hold a multiple of 128 weights, so the stream of
 *      the flat array equals the concatenation of the per-matrix streams sti_shard_upload expects.
 * NaN weights are not supported.
 */
#ifndef STI_QUANTIZE_H_
#define STI_QUANTIZE_H_

#include <stddef.h>
#include <stdint.h>

#include "sti.h"

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

/* Bytes of device workspace sti_quantize_units needs for n_units units of n_weights weights each
 * (per unit 17 bytes per weight - two ping-pong (key, offset) buffers and one byte per index for the
 * sorting method, the gathered bin members for the selecting one - plus one byte per unit that says
 * which method did it). */
size_t sti_quantize_workspace_bytes(uint32_t n_units, uint32_t n_weights);

/* How step 3 is carried out.  Both give the same output (index streams, outlier lists and counts bit for
 * bit; centroids up to the order of their fp64 sums).
 *   STI_QUANTIZE_SELECT  no sort: clusters are equal-population slices of the sorted order, so only the
 *                        2^bits - 1 weights at the slice boundaries are looked for (a histogram over value
 *                        bins, then rank selection inside the few bins that hold a boundary); a unit this
 *                        cannot take (zero variance, very many equal values) is sorted instead
 *   STI_QUANTIZE_SORT    every unit: a stable radix sort of the (value, offset) pairs */
#define STI_QUANTIZE_SELECT 0
#define STI_QUANTIZE_SORT 1

/* Quantizes n_units units (one CTA per unit), asynchronously on `stream` (a cudaStream_t,
 * NULL = default stream) of `device`; the caller's current device is left as it was.  All pointers are
 * device pointers owned by the caller:
 *   w_dev            [n_units][n_weights] fp32, read only, 16-byte aligned
 *   codes_dev        [n_units][n_weights*bits/32] 32-bit words of the index stream
 *   centroids_dev    [n_units][2^bits] fp32, ascending where clusters are non-empty
 *   outlier_off_dev  [n_units][max_outliers] offsets within the unit, ascending; outlier_val_dev the values
 *   n_outliers_dev   [n_units] the number of outliers found; when it exceeds max_outliers only the first
 *                    max_outliers pairs were written (the index stream is complete either way) and the
 *                    caller repeats the call with larger lists
 *   workspace_dev    at least sti_quantize_workspace_bytes(n_units, n_weights) bytes, 16-byte aligned;
 *                    contents undefined afterwards; calls that share a workspace must not overlap
 * Errors: STI_ERR_ARG (NULL or misaligned pointer), STI_ERR_BITS (bits outside 2..6), STI_ERR_SHAPE
 * (n_weights not a positive multiple of 32 or above 2^26, n_units 0 or above 65535, max_outliers 0),
 * STI_ERR_SIZE (workspace too small), STI_ERR_CUDA (no such device, launch failure).  Nothing is launched
 * on error.  Uses STI_QUANTIZE_SELECT. */
sti_status sti_quantize_units(int device, void* stream, const float* w_dev, uint32_t n_units, uint32_t n_weights,
                              int bits, uint32_t* codes_dev, float* centroids_dev, uint32_t* outlier_off_dev,
                              float* outlier_val_dev, uint32_t max_outliers, uint32_t* n_outliers_dev,
                              void* workspace_dev, size_t workspace_bytes);

/* The same with the method chosen by the caller (STI_ERR_ARG for an unknown one).  sorted_units_dev, when
 * not NULL, is a device array of n_units bytes that receives 1 for every unit the sort did and 0 for the
 * others. */
sti_status sti_quantize_units_by(int device, void* stream, const float* w_dev, uint32_t n_units, uint32_t n_weights,
                                 int bits, uint32_t* codes_dev, float* centroids_dev, uint32_t* outlier_off_dev,
                                 float* outlier_val_dev, uint32_t max_outliers, uint32_t* n_outliers_dev,
                                 void* workspace_dev, size_t workspace_bytes, int method, uint8_t* sorted_units_dev);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif

#endif /* STI_QUANTIZE_H_ */
