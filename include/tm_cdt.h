/*
 * tm_cdt / tm_bfdt -- taxicab and chessboard distance transforms, and a brute-force distance transform, C ABI
 * (sm_100a).  Paper: Section 2.1 (operators) and Section 2.3.2 (its paragraphs on the chamfer transform and on
 * the brute-force transform).  Status codes, stream type and error helpers are those of tm_edt.h; every call enqueues on
 * `stream` of the current device and returns without synchronising; scratch comes from the library's memory pool.
 */
#ifndef TM_CDT_H
#define TM_CDT_H

#include "tm_edt.h"

#ifdef __cplusplus
extern "C" {
#endif

enum { TM_METRIC_EUCLIDEAN = 0, TM_METRIC_TAXICAB = 1, TM_METRIC_CHESSBOARD = 2 };

/*
 * Taxicab or chessboard distance of every voxel to the nearest zero voxel of its image, as
 * scipy.ndimage.distance_transform_cdt returns it (the chamfer transform of the paper is exact for these two
 * metrics, so the result is defined by the metric alone):
 *   taxicab     min_s sum_k |x_k - s_k|        chessboard  min_s max_k |x_k - s_k|
 *   input     device, uint8, contiguous (B, C, n_0 .. n_{ndim-1}); nonzero = foreground.  Read only.
 *   ndim      1..8;  shape: host, ndim + 2 entries (any entry 0: nothing is written, TM_EDT_OK).
 *   metric    TM_METRIC_TAXICAB or TM_METRIC_CHESSBOARD (no sampling argument, as in SciPy).
 *   out_dist  device, int32, same shape; -1 in every voxel of an image without background.
 * One pass per axis, g_k(x) = min_j op(g_{k-1}(x with x_k := j), |x_k - j|) with op = + (taxicab) or max
 * (chessboard), each voxel scanning outward until the step alone reaches its minimum.
 */
TM_EDT_API int tm_cdt(const uint8_t* input, int ndim, const int64_t* shape, int metric, int32_t* out_dist,
                      tm_edt_stream_t stream);

/*
 * Brute-force distance transform: every voxel against every background voxel of its image, background
 * coordinates staged through shared memory in tiles of 256.  Quadratic cost: meant for validating the separable
 * transforms on the device and for the one case they do not offer, taxicab / chessboard distances with sampling.
 *   metric    any TM_METRIC_*;  sampling: host, ndim entries > 0, or NULL for 1.0.
 *   ndim      1..4 (the coordinate loop is unrolled per rank);  at most 2^24 voxels per image.
 *   out_dist  device, float32: sqrt(sum (w_k d_k)^2), sum w_k |d_k| or max w_k |d_k|; +inf without background.
 */
TM_EDT_API int tm_bfdt(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, int metric,
                       float* out_dist, tm_edt_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif
