// Host-side plan of one call and the helpers shared by the translation units that launch the distance-transform
// kernels.  Not exported.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "edt_common.cuh"
#include "edt_debug.cuh"

namespace tmedt {

// The contiguous (B, C, n_0 .. n_{d-1}) array is, for the pass along spatial axis a, a
// (outer, n_a, inner) array.  Axes of extent 1 are never processed (their pass is the identity).
// Processing order: last spatial axis first ("plane" p = p-th processed axis).
struct Plan {
    int ndim = 0;
    int64_t images = 0, V = 0, N = 0;
    int E = 0;
    int axis[kMaxDims];
    int plane_of_axis[kMaxDims];
    int ext[kMaxDims];
    int64_t inner[kMaxDims];
    double w[kMaxDims];
    bool unit = true;
    bool use_double = false;  // arithmetic type of the envelope passes
    bool wide = false;        // int16 offsets instead of int8
    bool fast = false;        // packed-entry kernels (extents <= 128, 2..5 processed axes)
    unsigned flags = 0;       // TM_EDT_FLAG_* of the call
    int64_t shape_sp[kMaxDims];  // spatial extents of the call
    double w_sp[kMaxDims];       // sampling per spatial axis
    bool long_lines = false;  // two or three axes, extents up to 8192: plain heights scanned through the cache
    bool small = false;       // every extent <= 8: register-resident lines, value (+ site index) carry
    bool scaled = false;      // fast path in exact integers: scale * w^2 is an integer for every processed axis
    int si[kMaxDims];         // those integers
    double scale = 1.0;
    bool vscaled = false;     // wide-key / long-line shapes, distances only: the value kernels in exact scaled integers
    int vsi[kMaxDims];        // scale * w^2 per processed axis
    double vscale = 1.0;
    bool wide_keys = false;      // unit sampling, contiguous extent % 16 == 0: two axes <= 1024 or three axes <= 512
    size_t ws_bytes = 0;
    size_t plane_bytes = 0;   // bytes of one offset plane, rounded up to 256
};

// Debug and test switches, read from the environment once (and again by tm_edt_reload_switches()).
struct Switches {
    bool force_generic = false;   // TM_EDT_FORCE_GENERIC=1: rank- and extent-generic kernels for every shape
    bool no_scaled = false;       // TM_EDT_NO_SCALED: no scaled-integer mode
    bool old_plane = false;       // TM_EDT_OLD_PLANE=1: byte-load plane kernel
    bool no_value_carry = false;  // TM_EDT_NO_VALUE_CARRY: offsets are carried even without an index output
    bool no_lean = false;         // TM_EDT_NO_LEAN: one-voxel-per-lane kernels instead of the quad kernels
    bool no_narrow_tiles = false; // TM_EDT_NO_NARROW_TILES: a single image with few columns stays on wide_axis_kernel
    long long chunk_voxels = 0;   // TM_EDT_CHUNK_VOXELS=n: image ranges of at most n voxels (0 = grid limit)
    bool debug_inject = false;    // TM_EDT_DEBUG_INJECT=1, debug build only: the bounds checks get a bound that is too small
};
const Switches& switches();

// Per-kernel timing of tm_edt_profile: records an event before the launch that follows.
// `bytes`: what that launch has to read and write once (its inputs plus its outputs).
void prof_mark(cudaStream_t st, const char* name, double bytes);
double out_bytes_per_voxel(const EpilogueParams& ep);

// Raises a kernel's dynamic shared-memory limit when `smem` needs it; remembered per (kernel, device), so the
// attribute is set once and not at every call.
cudaError_t ensure_smem(const void* kernel, size_t smem);

// Quad-per-lane kernels (edt_lean.cuh, launched from tm_edt_lean.cu): whether they cover a call, and the call itself.
bool lean_ok(const Plan& pl, const uint8_t* in, const EpilogueParams& ep);
cudaError_t run_lean(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws, cudaStream_t st, int& launches);

// One axis pass of the wide-key path on plain integer values with the quad kernels (see tm_edt_lean.cu).
bool lean_value_axis_ok(const Plan& pl, int k, const EpilogueParams& ep);
bool lean_value_long_axis_ok(const Plan& pl, int k, const EpilogueParams& ep);
bool lean_value_all_axes_ok(const Plan& pl, const EpilogueParams& ep);
cudaError_t run_lean_value_long_axis(const Plan& pl, int k, const void* in, void* out, const EpilogueParams& ep, bool fin,
                                     cudaStream_t st);
cudaError_t run_lean_value_axis(const Plan& pl, int k, const void* in, void* out, const EpilogueParams& ep, bool fin,
                                cudaStream_t st, bool dist16 = false);

// Debug build: what the kernels launched from tm_edt_lean.cu recorded (see edt_debug.cuh).
// First-axis distances as 16-bit values (>= 0xC000: no background in the row) for rows of a multiple of 32 up to 1024
// voxels and a 32-byte aligned mask: the word-per-lane row kernel of cdt.cuh (defined in tm_cdt.cu).
cudaError_t launch_row_dist16(const uint8_t* mask, uint16_t* out, int64_t rows, int n0, cudaStream_t st);
cudaError_t lean_debug_collect(cudaStream_t st, DebugRecord* out);

}  // namespace tmedt
