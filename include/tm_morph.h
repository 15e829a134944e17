/*
 * tm_morph -- greyscale and binary erosion / dilation on the GPU, C ABI (sm_100a).
 *
 * Operators (paper, Section 2.1 "Covered transforms"; kernel design: Section 2.3.1 "Fused morphology
 * kernel"), with the conventions of scipy.ndimage that the paper mirrors:
 *
 *   grey erosion    out(x) = min over active k of [ f(x + k - c) - s(k) ]
 *   grey dilation   out(x) = max over active k of [ f(x - k + c') + s(k) ]   (the element reflected through its centre)
 *   binary erosion  out(x) = AND over active k of f(x + k - c);   binary dilation: OR, reflected element
 *
 * c = size / 2 + origin per axis.  Positions outside the image are resolved by one of five border rules
 * (greyscale) or by a single border value (binary).  The structuring element is flattened on the host into its
 * active entries (per-axis offsets and the flat offset against the image's strides); a thread whose whole
 * neighbourhood lies inside the image adds flat offsets only, the others map every coordinate by the border rule.
 *
 * All calls enqueue on `stream` of the current device and return without synchronising (except that the entry
 * list, a few KB, is copied from host memory during the call).  Status codes, the stream type and the error
 * helpers are those of tm_edt.h.  On any error other than TM_EDT_ERR_CUDA nothing has been enqueued.
 */
#ifndef TM_MORPH_H
#define TM_MORPH_H

#include "tm_edt.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Border rules of the greyscale operators, named as in scipy.ndimage:
 *   CONSTANT  cval outside;  REFLECT  d c b a | a b c d | d c b a;  NEAREST  a a a | a b c d | d d d;
 *   MIRROR    d c b | a b c d | c b a;  WRAP  a b c d | a b c d | a b c d. */
enum { TM_MORPH_CONSTANT = 0, TM_MORPH_REFLECT = 1, TM_MORPH_NEAREST = 2, TM_MORPH_MIRROR = 3, TM_MORPH_WRAP = 4 };
enum { TM_MORPH_EROSION = 0, TM_MORPH_DILATION = 1 };

#define TM_MORPH_MAX_ENTRIES 4096 /* active positions of a structuring element */

/*
 * Greyscale erosion or dilation of float32 images.
 *   input      device, float32, contiguous (B, C, n_0 .. n_{ndim-1}).  Read only; must not overlap output.
 *   ndim       spatial dimensions, 1..8;  shape: host, ndim + 2 entries (any entry 0: nothing is written, OK).
 *   footprint  host, uint8, contiguous (m_0 .. m_{ndim-1}): nonzero = active position.  At least one active
 *              position, at most TM_MORPH_MAX_ENTRIES; every m_a in 1..255.
 *   structure  host, float32, same shape as footprint: the additive structuring function s, or NULL for a
 *              flat element (s = 0).
 *   fp_shape   host, ndim entries.   origin: host, ndim entries, or NULL for 0; the centre m_a / 2 + origin_a
 *              must lie inside the element (as SciPy requires).
 *   op         TM_MORPH_EROSION or TM_MORPH_DILATION;  mode: a border rule;  cval: the CONSTANT value.
 *   output     device, float32, same shape as input.
 * Arithmetic is float32: one subtraction (erosion) or addition (dilation) per active position, exact min / max.
 */
TM_EDT_API int tm_grey_morph(const float* input, int ndim, const int64_t* shape, const uint8_t* footprint,
                             const float* structure, const int64_t* fp_shape, const int64_t* origin, int op, int mode,
                             float cval, float* output, tm_edt_stream_t stream);

/*
 * Binary erosion or dilation of uint8 masks (nonzero = true); output holds 0 or 1.
 *   structure     host, uint8, (m_0 .. m_{ndim-1}): the structuring element (same limits as footprint above).
 *   border_value  0 or 1: the value of every position outside the image.
 * A thread stops combining as soon as its result is decided (a false for erosion, a true for dilation).
 * Every other argument as in tm_grey_morph.
 */
TM_EDT_API int tm_binary_morph(const uint8_t* input, int ndim, const int64_t* shape, const uint8_t* structure,
                               const int64_t* fp_shape, const int64_t* origin, int op, int border_value,
                               uint8_t* output, tm_edt_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif
