// Shared device-side types of the distance-transform kernels.
//
// Carry between passes ("offset planes"): after the p-th processed axis every voxel holds, for each
// processed axis q <= p, the signed offset  site_q - x_q  to the background voxel that is nearest
// with respect to the processed axes only.  Plane q is a contiguous array over all voxels of the batch.
// The squared distance is recomputed from the offsets, sum_q w_q^2 * off_q^2, so the index map comes for
// free and integer results stay exact.  "No site yet" is marked by the sentinel in plane 0.
// (Separable formulation: paper, Section 2.3.2 "Distance-transform kernels".)
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tmedt {

constexpr int kMaxDims = 8;

template <typename OT> struct OffTraits;
template <> struct OffTraits<int8_t> { static constexpr int kNone = -128; };
template <> struct OffTraits<int16_t> { static constexpr int kNone = -32768; };

// What the last pass writes, and how processed axes ("planes", in processing order: plane 0 is the
// contiguous axis) map back to the spatial axes of the call.
struct EpilogueParams {
    float* dist;        // (images, V) or nullptr
    int64_t* sq;        // (images, V) or nullptr
    int64_t* idx;       // (images, ndim, V), or (images, V) when flat, or nullptr
    int64_t V;          // voxels per image
    int ndim;           // spatial rank of the call
    int E;              // number of processed axes
    int axis[kMaxDims];          // spatial axis of plane p
    int plane_of_axis[kMaxDims]; // plane of spatial axis a, or -1 if its extent is 1 (never processed)
    int ext[kMaxDims];           // extent of plane p
    double w2[kMaxDims];         // squared sampling of plane p
    int flat;                    // 1: idx holds one value per voxel, the linear index of the site inside its image
    int idx_planes;              // index values per voxel: 1 when flat, else ndim
    int64_t pstride[kMaxDims];   // voxel stride of plane p inside an image
};

template <typename CT> __device__ __forceinline__ CT sqrt_ct(CT v);
template <> __device__ __forceinline__ float sqrt_ct<float>(float v) { return __fsqrt_rn(v); }
template <> __device__ __forceinline__ double sqrt_ct<double>(double v) { return sqrt(v); }

// Writes the requested outputs of one voxel from its final offsets.
//   img      image index, v voxel index inside the image
//   coord[p] own coordinate along plane p, off[p] final offset along plane p (p < E)
template <typename CT>
__device__ __forceinline__ void emit_outputs(const EpilogueParams& ep, int64_t img, int64_t v, const int* coord,
                                             const int* off, bool none) {
    const int64_t e = img * ep.V + v;
    if (none) {
        if (ep.dist) ep.dist[e] = __int_as_float(0x7f800000);
        if (ep.sq) ep.sq[e] = INT64_MAX;
        if (ep.idx && ep.flat) ep.idx[e] = -1;
        else if (ep.idx)
            for (int a = 0; a < ep.ndim; ++a) ep.idx[(img * ep.ndim + a) * ep.V + v] = -1;
        return;
    }
    if (ep.dist) {
        CT h = 0;
#pragma unroll
        for (int p = 0; p < kMaxDims; ++p)
            if (p < ep.E) h += (CT)ep.w2[p] * (CT)off[p] * (CT)off[p];
        ep.dist[e] = (float)sqrt_ct<CT>(h);
    }
    if (ep.sq) {
        int64_t s = 0;
#pragma unroll
        for (int p = 0; p < kMaxDims; ++p)
            if (p < ep.E) s += (int64_t)off[p] * (int64_t)off[p];
        ep.sq[e] = s;
    }
    if (ep.idx && ep.flat) {
        int64_t f = 0;
#pragma unroll
        for (int p = 0; p < kMaxDims; ++p)
            if (p < ep.E) f += (int64_t)(coord[p] + off[p]) * ep.pstride[p];
        ep.idx[e] = f;
    } else if (ep.idx) {
        for (int a = 0; a < ep.ndim; ++a) {
            const int p = ep.plane_of_axis[a];
            int64_t val = 0;
#pragma unroll
            for (int q = 0; q < kMaxDims; ++q)
                if (q == p) val = (int64_t)(coord[q] + off[q]);
            ep.idx[(img * ep.ndim + a) * ep.V + v] = val;
        }
    }
}

}  // namespace tmedt
