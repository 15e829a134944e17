// Virtual-background convention for images without any background voxel (paper, Section 2.3.2: such images are
// handled by the virtual out-of-bounds convention of scipy.ndimage): the image behaves as if one background
// voxel sat at coordinate -1 on spatial axis 0 and 0 on every other axis, so
//     d(x) = sqrt( (w_0 (x_0 + 1))^2 + sum_{k >= 1} (w_k x_k)^2 ),   index (-1, 0, .., 0).
// The transform itself marks such images (+inf, INT64_MAX, -1); these two kernels rewrite them afterwards.
// The marker is read at voxel 0 of the image, so the first kernel fills every other voxel and the second one
// voxel 0 itself: no scratch, no race.
#pragma once
#include "edt_common.cuh"

namespace tmedt {

struct VirtualParams {
    int64_t images, V;
    int ndim;
    int64_t shape[kMaxDims];   // spatial extents
    double w[kMaxDims];        // sampling
    int64_t stride0;           // voxel stride of spatial axis 0
};

__device__ __forceinline__ bool image_marked_empty(const EpilogueParams& ep, int64_t img) {
    if (ep.dist) return ep.dist[img * ep.V] == __int_as_float(0x7f800000);
    if (ep.sq) return ep.sq[img * ep.V] == INT64_MAX;
    return ep.idx[img * ep.idx_planes * ep.V] == -1;
}

__device__ __forceinline__ void virtual_fill(const VirtualParams& P, const EpilogueParams& ep, int64_t img, int64_t vox) {
    int64_t rr = vox;
    double h = 0.0;
    int64_t s = 0;
    for (int a = P.ndim - 1; a >= 0; --a) {
        int64_t x = rr % P.shape[a];
        rr /= P.shape[a];
        if (a == 0) x += 1;
        const double t = P.w[a] * (double)x;
        h += t * t;
        s += x * x;
    }
    const int64_t e = img * P.V + vox;
    if (ep.dist) ep.dist[e] = (float)sqrt(h);
    if (ep.sq) ep.sq[e] = s;
    if (ep.idx && ep.flat) ep.idx[e] = -P.stride0;
    else if (ep.idx)
        for (int a = 0; a < P.ndim; ++a) ep.idx[(img * P.ndim + a) * P.V + vox] = a == 0 ? -1 : 0;
}

// every voxel but voxel 0 of each image
__global__ void __launch_bounds__(256) virtual_background_kernel(const __grid_constant__ VirtualParams P,
                                                                 const __grid_constant__ EpilogueParams ep) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= P.images * P.V) return;
    const int64_t img = t / P.V, vox = t - img * P.V;
    if (vox == 0 || !image_marked_empty(ep, img)) return;
    virtual_fill(P, ep, img, vox);
}

// voxel 0 of each image
__global__ void __launch_bounds__(256) virtual_background_first_kernel(const __grid_constant__ VirtualParams P,
                                                                       const __grid_constant__ EpilogueParams ep) {
    const int64_t img = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (img >= P.images || !image_marked_empty(ep, img)) return;
    virtual_fill(P, ep, img, 0);
}

}  // namespace tmedt
