/*
 * tm_edt -- exact Euclidean distance transform on one NVIDIA B200 (sm_100a), C ABI.
 *
 * Operation (paper, Section 2.1 "Covered transforms", paragraph "Distance transforms", and
 * Section 2.3.2 "Distance-transform kernels"): every nonzero (foreground) element of a batched
 * mask is labelled with its Euclidean distance to the nearest zero (background) element of the
 * same image, with scipy.ndimage.distance_transform_edt semantics: per-axis sampling, optional
 * nearest-background index map (Section 2.3.2, closing paragraph: the index output is optional and
 * carried through the passes), inputs shaped (B, C, Spatial...) with 1 <= spatial rank <= 8 (Section 2.2.1
 * "API surface"), pre-allocated outputs, work issued on the caller's stream (Section 2.2.4,
 * runtime tests).
 *
 * For every image (b, c), with Z the set of its zero voxels and w_k the sampling of spatial axis k:
 *
 *     sq(x)   = min over z in Z of  sum_k ( w_k * (x_k - z_k) )^2
 *     dist(x) = sqrt(sq(x))                      -> out_dist   (float32)
 *     sq(x) with every w_k == 1                  -> out_sqdist (int64, exact)
 *     some z attaining the minimum               -> out_indices (int64, one plane per spatial axis)
 *
 * An image with no zero voxel has no nearest background: its out_dist is +inf, its out_sqdist is
 * INT64_MAX and every component of out_indices is -1.  This is decided per image.  (The paper
 * mentions SciPy's virtual out-of-bounds convention for that case; this library defines the
 * result as infinite instead.)  When several background voxels are equally near, which one
 * out_indices names is unspecified; it always names one at the minimal distance, and a background
 * voxel names itself.
 *
 * All entry points are thread-safe.  The only state kept between calls is, per device, a private
 * stream-ordered memory pool from which tm_edt and tm_edt_host take their scratch (so that one call's
 * memory is reused by the next; tm_edt_trim_memory() gives it back) and the address of the built-in
 * scratch array of tm_edt_noalloc.  Nothing is thrown and no device trap is ever raised: every problem is a return code,
 * and every argument check happens before any work is enqueued.
 */
#ifndef TM_EDT_H_
#define TM_EDT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define TM_EDT_API __attribute__((visibility("default")))
#else
#define TM_EDT_API
#endif

#define TM_EDT_MAX_DIMS 8      /* spatial rank bound (Section 2.2.1 / 2.2.2: compile-time bound of eight) */
#define TM_EDT_MAX_EXTENT 8192 /* largest supported extent of one spatial axis */

typedef enum {
    TM_EDT_OK = 0,
    TM_EDT_ERR_INVALID_ARG = 1, /* NULL input/shape, ndim outside 1..8, negative extent, sampling not finite
                                   and > 0, no output requested, an output not aligned to its element size,
                                   outputs overlapping each other or the input */
    TM_EDT_ERR_UNSUPPORTED = 2, /* extent > TM_EDT_MAX_EXTENT, out_sqdist with non-unit sampling, more than
                                   2^40 elements, or more than 2^31 - 1 voxels per image */
    TM_EDT_ERR_BAD_POINTER = 3, /* a device buffer is not device-accessible memory of the current device
                                   (or a host buffer of tm_edt_host is device memory) */
    TM_EDT_ERR_ALLOC = 4,       /* scratch allocation failed, or the supplied workspace is too small */
    TM_EDT_ERR_CUDA = 5,        /* a CUDA runtime call or launch failed; see tm_edt_last_cuda_error() */
    TM_EDT_ERR_TOO_LARGE = 6,   /* tm_edt_noalloc only: the problem needs more scratch than its built-in array */
    TM_EDT_ERR_DEBUG_CHECK = 7  /* debug build only (see tm_edt_debug_build): an index of a kernel left its range;
                                   the access was skipped, the outputs of the call are not to be trusted */
} tm_edt_status;

/* The stream argument is a cudaStream_t (NULL = the legacy default stream). */
typedef struct CUstream_st* tm_edt_stream_t;

/*
 * The transform.  Enqueues all work on `stream` of the current device and returns without
 * synchronising; outputs are complete once the stream reaches the end of that work.
 *
 *   input        device, uint8, contiguous row-major (B, C, n_0 .. n_{ndim-1}); nonzero = foreground
 *                (a bool tensor is passed as its bytes).  Read only.
 *   ndim         number of SPATIAL dimensions, 1..8.
 *   shape        host, ndim + 2 entries: B, C, n_0 .. n_{ndim-1}.  Any entry may be 0 (nothing is
 *                written, TM_EDT_OK); extents of 1 are legal.  Copied during the call.
 *   sampling     host, ndim entries, each finite and > 0, or NULL for 1.0 on every axis.  Copied.
 *   out_dist     device float32 (B, C, n...), or NULL.
 *   out_sqdist   device int64 (B, C, n...), or NULL.  Requires unit sampling (else UNSUPPORTED).
 *   out_indices  device int64 (B, C, ndim, n...), or NULL.  out_indices[b, c, a, x] is the coordinate
 *                along spatial axis a of the background voxel chosen for voxel x.
 *   At least one output must be non-NULL.  The caller owns every buffer; the library keeps no
 *   pointer once the enqueued work has run.  Scratch memory is taken from the library's private
 *   stream-ordered memory pool of the device (allocation and release are both ordered on `stream`).
 *
 * Returns a tm_edt_status.  On any error other than TM_EDT_ERR_CUDA nothing has been enqueued.
 */
TM_EDT_API int tm_edt(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
           int64_t* out_sqdist, int64_t* out_indices, tm_edt_stream_t stream);

/*
 * Variants of the transform behind a flags word (0 = exactly tm_edt / tm_edt_ws):
 *
 *   TM_EDT_FLAG_VIRTUAL_BACKGROUND  An image without any background voxel gets, instead of +inf / INT64_MAX /
 *       -1, the values of the virtual out-of-bounds convention the paper takes over from scipy.ndimage
 *       (Section 2.3.2, "Distance-transform kernels"): as if its only background voxel sat at coordinate -1
 *       on spatial axis 0 and 0 on every other axis, i.e.
 *       d(x) = sqrt((w_0 (x_0 + 1))^2 + sum_{k>=1} (w_k x_k)^2), indices (-1, 0, .., 0).
 *   TM_EDT_FLAG_FLAT_INDEX  out_indices is (B, C, n...) int64: the row-major linear index, inside its image,
 *       of the chosen background voxel (one value per voxel instead of ndim; -1 for an image without
 *       background, minus the stride of axis 0 under the virtual-background convention).  The paper's index
 *       map has one coordinate per axis; this layout is an extra of this library.
 *
 *   TM_EDT_FLAG_DIST_F64  out_dist is float64 (B, C, n...): the distance to the chosen background voxel,
 *       recomputed in double precision from its coordinates (exactly rounded under unit sampling).  The transform
 *       then always produces the site of every voxel (in out_indices if given, else as one linear index per voxel
 *       in scratch) and a second kernel turns sites into distances: a compatibility path, slower than float32.
 *
 *   in_strides   host, ndim + 2 entries, BYTE strides of the mask per array dimension (B, C, n_0 ..), each >= 0,
 *                or NULL for the contiguous layout.  A non-contiguous mask is first gathered into scratch
 *                (1 byte per voxel), then transformed: also a compatibility path.
 *   out_dist     float32, or float64 with TM_EDT_FLAG_DIST_F64 (8-byte aligned).
 *   workspace    device scratch of at least tm_edt_ex_workspace_bytes(...) bytes for the same arguments, 256-byte
 *                aligned, or NULL to take scratch from the library's memory pool as tm_edt does (workspace_bytes
 *                ignored).
 *   Every other argument, the ownership rules and the error behaviour are those of tm_edt; an unknown flag
 *   bit or a negative stride gives TM_EDT_ERR_INVALID_ARG.  With a workspace the call allocates nothing and only
 *   enqueues kernels.
 */
#define TM_EDT_FLAG_VIRTUAL_BACKGROUND 1u
#define TM_EDT_FLAG_FLAT_INDEX 2u
#define TM_EDT_FLAG_DIST_F64 4u
TM_EDT_API int tm_edt_ex(const uint8_t* input, int ndim, const int64_t* shape, const int64_t* in_strides,
                         const double* sampling, void* out_dist, int64_t* out_sqdist, int64_t* out_indices,
                         unsigned flags, void* workspace, size_t workspace_bytes, tm_edt_stream_t stream);

/* Scratch bytes tm_edt_ex needs: those of tm_edt_workspace_bytes, plus the gathered mask for a non-contiguous
 * input, plus one int64 per voxel for float64 distances without an index output ((size_t)-1 on invalid arguments). */
TM_EDT_API size_t tm_edt_ex_workspace_bytes(int ndim, const int64_t* shape, const int64_t* in_strides, unsigned flags,
                                            int with_distances, int with_indices);

/*
 * Scratch bytes that suffice for any tm_edt_ws call with this geometry, whatever its sampling and outputs
 * (0 for empty problems, and (size_t)-1 if ndim/shape are invalid or unsupported).  Depends only on ndim and
 * shape: it is the largest need over unit and other sampling, with the index output requested.
 */
TM_EDT_API size_t tm_edt_workspace_bytes(int ndim, const int64_t* shape);

/*
 * Scratch bytes of one particular call (paper, Section 2.2.1: outputs are optional and may be pre-allocated):
 * the geometry, its sampling (NULL = unit) and which outputs it requests (non-zero = requested).  Never more than
 * tm_edt_workspace_bytes(ndim, shape); less when no index output is requested on extents above 128 (the offsets
 * to the site are then not carried between the passes).  tm_edt_ws accepts a workspace of this size for that call.
 */
TM_EDT_API size_t tm_edt_workspace_bytes_for(int ndim, const int64_t* shape, const double* sampling, int want_dist,
                                             int want_sqdist, int want_indices);

/*
 * Debug build (compiled with -DTM_EDT_DEBUG=1, the stand-in for a device memory checker): the quad kernels check
 * every shared-memory and global index they use, skip an access that leaves its range and record it; every call
 * then waits for its own work and returns TM_EDT_ERR_DEBUG_CHECK if anything was recorded.  tm_edt_debug_build()
 * says whether this library is such a build; tm_edt_debug_last_violation() returns how many violations the calling
 * thread's last call recorded and, through the optional pointers, the site code, index and bound of the first one.
 * In a release build the first returns 0 and the second always 0.  (No counterpart in the paper.)
 */
TM_EDT_API int tm_edt_debug_build(void);
TM_EDT_API unsigned long long tm_edt_debug_last_violation(long long* code, long long* index, long long* limit);

/*
 * Debug and test switches (environment variables TM_EDT_FORCE_GENERIC, TM_EDT_NO_SCALED, TM_EDT_OLD_PLANE,
 * TM_EDT_NO_VALUE_CARRY, TM_EDT_NO_LEAN, TM_EDT_NO_NARROW_TILES, TM_EDT_CHUNK_VOXELS; they select kernel families
 * and change no exact result -- squared distances and sites stay the same, a float32 distance can differ in its last
 * bit between families) are read from the environment once, at the first call that plans a transform.  This call
 * reads them again.
 */
TM_EDT_API void tm_edt_reload_switches(void);

/*
 * Same transform with caller-provided scratch: `workspace` is device memory of at least
 * tm_edt_workspace_bytes_for(...) bytes for this call (tm_edt_workspace_bytes(ndim, shape) always suffices),
 * 256-byte aligned, private to this call until the
 * enqueued work has run.  Allocates nothing and only enqueues kernels, so the call can be captured into a
 * CUDA graph and replayed.  A too-small workspace gives TM_EDT_ERR_ALLOC.
 */
TM_EDT_API int tm_edt_ws(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
              int64_t* out_sqdist, int64_t* out_indices, void* workspace, size_t workspace_bytes,
              tm_edt_stream_t stream);

/*
 * Host-buffer convenience: `input` and the outputs are HOST memory (pinned memory makes the copies
 * asynchronous).  Device buffers come from the stream-ordered allocator; the input is copied to the
 * device, the transform runs, and the requested outputs are copied back, all ordered on `stream`.
 * Does not synchronise: the host outputs are valid after the caller synchronises the stream.
 */
TM_EDT_API int tm_edt_host(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
                int64_t* out_sqdist, int64_t* out_indices, tm_edt_stream_t stream);

/*
 * The transform for callers that must not allocate device memory.  (The paper has no counterpart to
 * this entry point; it exists for deployment, not for the method.)
 *
 * Some hosts of this library cannot let it call cudaMalloc or the stream-ordered allocator while they
 * run: a real-time or safety-certified loop that fixed its memory budget at start-up, a process whose
 * device memory is entirely owned by another allocator, a driver sandbox that forbids allocation after
 * initialisation.  tm_edt allocates its scratch, and tm_edt_ws pushes that job onto the caller; this
 * variant does neither.  Its scratch is a fixed array of TM_EDT_NOALLOC_MAX_SCRATCH bytes that is part
 * of the library's device image, so every GPU that loads the library holds that much memory until the
 * process exits, whether or not this function is ever called.
 *
 * Arguments, outputs, stream behaviour and return codes are those of tm_edt (inputs and outputs are
 * still the caller's device buffers).  Differences:
 *   - A problem whose scratch need, tm_edt_workspace_bytes_for(...) of the call, exceeds
 *     TM_EDT_NOALLOC_MAX_SCRATCH is refused with TM_EDT_ERR_TOO_LARGE before anything is enqueued.
 *   - The first call on each device looks up the device address of the array (cudaGetSymbolAddress, with
 *     that device current) and remembers it.  Make that first call during set-up, before any stream
 *     capture begins.  Later calls on the device only enqueue kernels.
 *   - No cudaMalloc, cudaFree, stream-ordered allocation or other allocating routine is called, on any
 *     path, success or failure.
 *   - All calls on one device share the one array.  It keeps whatever the previous call left in it;
 *     that is harmless, because each pass writes every scratch element before a later pass reads it, so
 *     nothing has to be cleared.  Two calls whose work overlaps on the GPU (different streams without
 *     ordering between them, or threads racing on one device) corrupt each other's scratch: order them
 *     on one stream or with events.  Calls on different devices do not interact.
 */
#define TM_EDT_NOALLOC_MAX_SCRATCH (16u * 1024u * 1024u)
TM_EDT_API int tm_edt_noalloc(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling,
                              float* out_dist, int64_t* out_sqdist, int64_t* out_indices, tm_edt_stream_t stream);

/* TM_EDT_NOALLOC_MAX_SCRATCH as the loaded library was built (bytes). */
TM_EDT_API size_t tm_edt_noalloc_max_scratch(void);

/*
 * Measurement aid: tm_edt_ws with a CUDA event recorded on `stream` before every kernel and after the
 * last, then a wait for the last event (this entry point DOES block the calling thread).  On return
 * kernel_ms[i] is the device time from the start of kernel i to the start of kernel i + 1 (or to the end
 * of the call) in milliseconds, kernel_bytes[i] the bytes that launch has to read and write once (its
 * inputs plus its outputs), kernel_names + 48 * i a NUL-terminated label, and *n_kernels how many
 * entries were written (at most max_kernels).  kernel_bytes and kernel_names may be NULL.  The transform's outputs are
 * written as by tm_edt_ws (same operation: Section 2.3.2; the timing protocol follows the paper's
 * Results, "Protocol": explicit synchronisation inside the timed region).
 */
TM_EDT_API int tm_edt_profile(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling,
                              float* out_dist, int64_t* out_sqdist, int64_t* out_indices, void* workspace,
                              size_t workspace_bytes, tm_edt_stream_t stream, int max_kernels, float* kernel_ms,
                              double* kernel_bytes, char* kernel_names, int* n_kernels);

/* tm_edt_profile for the variants of tm_edt_ex: the same measurement with a flags word (workspace required when the
 * geometry needs scratch). */
TM_EDT_API int tm_edt_profile_ex(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling,
                                 float* out_dist, int64_t* out_sqdist, int64_t* out_indices, unsigned flags,
                                 void* workspace, size_t workspace_bytes, tm_edt_stream_t stream, int max_kernels,
                                 float* kernel_ms, double* kernel_bytes, char* kernel_names, int* n_kernels);

/*
 * Returns to the driver whatever the library's private memory pool of the current device holds and no
 * enqueued work still uses (tm_edt and tm_edt_host keep their scratch pooled between calls).  No
 * counterpart in the paper, which leaves memory to PyTorch's caching allocator (Section 2.2, Fig. 2).
 */
TM_EDT_API int tm_edt_trim_memory(void);

/* Static description of a status code. Never NULL. */
TM_EDT_API const char* tm_edt_strerror(int status);

/* The cudaError_t value behind the calling thread's most recent TM_EDT_ERR_CUDA / TM_EDT_ERR_ALLOC (0 if none). */
TM_EDT_API int tm_edt_last_cuda_error(void);

/* Library version string, e.g. "tm_edt 0.1 (sm_100a)". */
TM_EDT_API const char* tm_edt_version(void);

/* Number of kernels the calling thread's most recent successful tm_edt* call enqueued. */
TM_EDT_API int tm_edt_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TM_EDT_H_ */
