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
    uint32_t rr = (uint32_t)vox;  // an image has fewer than 2^31 voxels
    double h = 0.0;
    int64_t s = 0;
    for (int a = P.ndim - 1; a >= 0; --a) {
        const uint32_t n = (uint32_t)P.shape[a], q = rr / n;
        int64_t x = rr - q * n;
        rr = q;
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

// every voxel but voxel 0 of each image: a block takes kVirtualChunk voxels of one image and leaves at once unless
// the image is marked empty
constexpr int kVirtualChunk = 256 * 8;
__global__ void __launch_bounds__(256) virtual_background_kernel(const __grid_constant__ VirtualParams P,
                                                                 const __grid_constant__ EpilogueParams ep,
                                                                 const unsigned chunks_per_image) {
    const int64_t img = blockIdx.x / chunks_per_image;
    if (!image_marked_empty(ep, img)) return;
    const int64_t v0 = (int64_t)(blockIdx.x - img * chunks_per_image) * kVirtualChunk;
    for (int i = threadIdx.x; i < kVirtualChunk; i += 256) {
        const int64_t vox = v0 + i;
        if (vox != 0 && vox < P.V) virtual_fill(P, ep, img, vox);
    }
}

// voxel 0 of each image
__global__ void __launch_bounds__(256) virtual_background_first_kernel(const __grid_constant__ VirtualParams P,
                                                                       const __grid_constant__ EpilogueParams ep) {
    const int64_t img = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (img >= P.images || !image_marked_empty(ep, img)) return;
    virtual_fill(P, ep, img, 0);
}

// Gathers a strided mask (byte strides per array dimension, batch and channel included) into the contiguous
// row-major layout the transform reads.  dims = ndim + 2.
struct GatherParams {
    const uint8_t* in;
    uint8_t* out;
    int64_t total;
    int dims;
    int64_t shape[kMaxDims + 2];
    int64_t stride[kMaxDims + 2];
};

// PER voxels of one row per thread (PER = 4 needs a last extent that is a multiple of 4): one index split, PER
// loads, one PER-byte store.
template <int PER>
__global__ void __launch_bounds__(256) gather_strided_kernel(const __grid_constant__ GatherParams P) {
    const int64_t e = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * PER;
    if (e >= P.total) return;
    int64_t off = 0;
    if (P.total <= 0xffffffffll) {  // 32-bit index arithmetic whenever the element count allows it
        uint32_t rr = (uint32_t)e;
        for (int a = P.dims - 1; a >= 0; --a) {
            const uint32_t n = (uint32_t)P.shape[a], q = rr / n;
            off += (int64_t)(rr - q * n) * P.stride[a];
            rr = q;
        }
    } else {
        int64_t rr = e;
        for (int a = P.dims - 1; a >= 0; --a) {
            const int64_t q = rr / P.shape[a];
            off += (rr - q * P.shape[a]) * P.stride[a];
            rr = q;
        }
    }
    if (PER == 1) {
        P.out[e] = P.in[off];
    } else {
        const int64_t sl = P.stride[P.dims - 1];
        uint32_t v = 0;
#pragma unroll
        for (int k = 0; k < PER; ++k) v |= (uint32_t)P.in[off + k * sl] << (8 * k);
        *reinterpret_cast<uint32_t*>(P.out + e) = v;
    }
}

// float64 distances, recomputed from the chosen site of every voxel:
//     d(x) = sqrt( sum_k (w_k (x_k - s_k))^2 )   in double precision
// (exactly rounded under unit sampling, where the sum is an integer).  The site comes from the index output of
// the transform: coordinate planes (images, ndim, V) or one linear index per voxel (flat).  A negative linear
// index, or -1 in the last coordinate plane, marks an image without background (+inf) unless the virtual-background
// convention is on, where it names the virtual voxel (-1, 0, .., 0).
// Blocks enumerate (image, 256 voxels of it); an image has fewer than 2^31 voxels, so positions inside it are split
// with 32-bit divisions.
__global__ void __launch_bounds__(256) dist_f64_kernel(const __grid_constant__ VirtualParams P, const int64_t* idx,
                                                       const int flat, const int virtual_bg, double* out,
                                                       const unsigned blocks_per_image) {
    const int64_t img = blockIdx.x / blocks_per_image;
    const uint32_t vox = (blockIdx.x - (uint32_t)img * blocks_per_image) * 256u + threadIdx.x;
    if ((int64_t)vox >= P.V) return;
    const int64_t e = img * P.V + vox;
    const int64_t fs64 = flat ? idx[e] : 0;
    const bool neg = flat ? fs64 < 0 : idx[(img * P.ndim + (P.ndim - 1)) * P.V + vox] == -1 && !virtual_bg;
    if (neg && !virtual_bg) { out[e] = __longlong_as_double(0x7ff0000000000000ll); return; }
    uint32_t rr = vox, fs = (uint32_t)fs64;
    double h = 0.0;
    for (int a = P.ndim - 1; a >= 0; --a) {
        const uint32_t n = (uint32_t)P.shape[a], q = rr / n;
        const int x = (int)(rr - q * n);
        rr = q;
        int sa;
        if (!flat) sa = (int)idx[(img * P.ndim + a) * P.V + vox];
        else if (neg) sa = a == 0 ? -1 : 0;
        else { const uint32_t qs = fs / n; sa = (int)(fs - qs * n); fs = qs; }
        const double t = P.w[a] * (double)(x - sa);
        h += t * t;
    }
    out[e] = sqrt(h);
}

}  // namespace tmedt
