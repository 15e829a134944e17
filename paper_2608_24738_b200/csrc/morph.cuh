// Fused erosion / dilation kernels (paper, Section 2.3.1 "Fused morphology kernel").  The host flattens the
// structuring element into its active entries; each entry carries the per-axis offsets and the flat offset
// against the image's strides.  Interior voxels (whole neighbourhood inside the image, tested with the per-axis
// offset extrema) add flat offsets to their linear index and nothing else; voxels within reach of a face map every
// neighbour coordinate by the border rule.  The two kinds run as two launches, so that no warp executes both code
// paths.  One template covers erosion and dilation (identity and combine differ), greyscale and binary (the binary
// form stops as soon as the result is decided).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tmmorph {

constexpr int kMaxDims = 8;

struct Entry {
    int flat;             // sum_a off[a] * stride[a]
    float s;              // structuring function at this position (0 for a flat element)
    int16_t off[kMaxDims];
};

struct Params {
    const void* in;
    void* out;
    const Entry* entries;
    int n_entries;
    int ndim;
    int64_t total;         // images * V
    int V;                 // voxels per image
    int ext[kMaxDims];
    int stride[kMaxDims];  // voxel strides inside an image
    int lo[kMaxDims];      // smallest offset per axis over all entries
    int hi[kMaxDims];      // largest offset per axis
    int64_t flat_lo, flat_hi;  // bounds of the flat offsets: sum_a lo[a] * stride[a], sum_a hi[a] * stride[a]
    int mode;
    float cval;            // greyscale CONSTANT value
    int border_value;      // binary: value outside the image
};

enum { kConstant = 0, kReflect = 1, kNearest = 2, kMirror = 3, kWrap = 4 };

// Coordinate c of an axis of extent n under a border rule; returns false if the position takes the constant.
__device__ __forceinline__ bool map_coord(int& c, int n, int mode) {
    if (c >= 0 && c < n) return true;
    switch (mode) {
        case kConstant: return false;
        case kNearest: c = c < 0 ? 0 : n - 1; return true;
        case kWrap: c %= n; if (c < 0) c += n; return true;
        case kReflect: {  // d c b a | a b c d | d c b a : period 2n
            const int p = 2 * n;
            int m = c % p; if (m < 0) m += p;
            c = m < n ? m : p - 1 - m;
            return true;
        }
        default: {  // mirror: d c b | a b c d | c b a : period 2n - 2
            if (n == 1) { c = 0; return true; }
            const int p = 2 * n - 2;
            int m = c % p; if (m < 0) m += p;
            c = m < n ? m : p - m;
            return true;
        }
    }
}

// Interior kernel.  A warp takes 32 * VPT consecutive voxels of a row; lane l owns voxels l, l + 32, .. of them, so
// that every load and store of the warp is one contiguous 128-byte (float) request.  VPT = 8 or 4 needs a last extent
// that is a multiple of 256 or 128; the host falls back to VPT = 1 otherwise.  FLAT: every structuring value is 0.  A voxel whose whole neighbourhood lies
// inside the image adds flat offsets to its linear index and nothing else; the other voxels are left out here:
// they belong to the border slabs of morph_border_kernel.  The flat offsets and structuring values of the
// entries are staged in shared memory once per block.
template <typename T, bool MIN, bool BINARY, int VPT, bool FLAT>
__global__ void __launch_bounds__(256) morph_interior_kernel(const __grid_constant__ Params P) {
    extern __shared__ __align__(16) unsigned char sm_morph[];
    int* s_flat = reinterpret_cast<int*>(sm_morph);
    float* s_val = reinterpret_cast<float*>(sm_morph) + P.n_entries;
    for (int k = threadIdx.x; k < P.n_entries; k += blockDim.x) {
        s_flat[k] = P.entries[k].flat;
        s_val[k] = P.entries[k].s;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t e = warp * (32 * VPT) + lane;  // the lane's first voxel
    if (e >= P.total) return;
    const int64_t img = e / P.V;
    const int vox = (int)(e - img * P.V);
    bool live[VPT];
    {
        uint32_t rr = (uint32_t)vox;
        bool others = true;
        int xl = 0, nl = 1;
#pragma unroll
        for (int a = kMaxDims - 1; a >= 0; --a) {
            if (a < P.ndim) {
                const uint32_t n = (uint32_t)P.ext[a], q = rr / n;
                const int xa = (int)(rr - q * n);
                rr = q;
                if (a == P.ndim - 1) { xl = xa; nl = (int)n; }
                else others = others && xa + P.lo[a] >= 0 && xa + P.hi[a] < (int)n;
            }
        }
        bool any = false;
#pragma unroll
        for (int j = 0; j < VPT; ++j) {  // the lane's voxels differ along the last axis only
            live[j] = others && xl + 32 * j + P.lo[P.ndim - 1] >= 0 && xl + 32 * j + P.hi[P.ndim - 1] < nl;
            any = any || live[j];
        }
        if (!any) return;
    }
    const T* __restrict__ p0 = static_cast<const T*>(P.in) + e;
    // Voxels at the ends of a row are not live, but as long as the warp's whole span plus the element's reach stays
    // inside the tensor their loads are harmless (they read neighbouring rows): the whole warp then runs one loop
    // without per-voxel tests and only the stores are guarded ("safe" below).
    if (BINARY) {
        const int64_t span0 = warp * (32 * VPT);
        const bool safe = span0 + P.flat_lo >= 0 && span0 + 32 * VPT - 1 + P.flat_hi < P.total;
        // bit j of `acc`: running AND (erosion) or OR (dilation) of voxel j; a lane stops once all its voxels are decided
        unsigned acc = MIN ? (1u << VPT) - 1u : 0u;
        unsigned lv = 0;
#pragma unroll
        for (int j = 0; j < VPT; ++j) lv |= live[j] ? 1u << j : 0u;
        if (safe) {
            for (int k = 0; k < P.n_entries; ++k) {
                const T* __restrict__ p = p0 + s_flat[k];
                unsigned v = 0;
#pragma unroll
                for (int j = 0; j < VPT; ++j) v |= (p[32 * j] != 0 ? 1u : 0u) << j;
                acc = MIN ? acc & v : acc | v;
                if (acc == (MIN ? 0u : (1u << VPT) - 1u)) break;
            }
        } else {
            for (int k = 0; k < P.n_entries; ++k) {
                const T* __restrict__ p = p0 + s_flat[k];
                unsigned v = MIN ? (1u << VPT) - 1u : 0u;
#pragma unroll
                for (int j = 0; j < VPT; ++j)
                    if (live[j]) v = (v & ~(1u << j)) | ((p[32 * j] != 0 ? 1u : 0u) << j);
                acc = MIN ? acc & v : acc | v;
            }
        }
        uint8_t* o = static_cast<uint8_t*>(P.out) + e;
#pragma unroll
        for (int j = 0; j < VPT; ++j)
            if ((lv >> j) & 1u) o[32 * j] = (uint8_t)((acc >> j) & 1u);
    } else {
        float acc[VPT];
#pragma unroll
        for (int j = 0; j < VPT; ++j) acc[j] = MIN ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
        const int64_t span0 = warp * (32 * VPT);
        const bool safe = span0 + P.flat_lo >= 0 && span0 + 32 * VPT - 1 + P.flat_hi < P.total;
        if (safe) {
#pragma unroll 4
            for (int k = 0; k < P.n_entries; ++k) {
                const T* __restrict__ p = p0 + s_flat[k];
                const float sv = FLAT ? 0.f : s_val[k];
#pragma unroll
                for (int j = 0; j < VPT; ++j) {
                    const float v = FLAT ? (float)p[32 * j] : (MIN ? __fsub_rn((float)p[32 * j], sv) : __fadd_rn((float)p[32 * j], sv));
                    acc[j] = MIN ? fminf(acc[j], v) : fmaxf(acc[j], v);
                }
            }
        } else {
            for (int k = 0; k < P.n_entries; ++k) {
                const T* __restrict__ p = p0 + s_flat[k];
                const float sv = FLAT ? 0.f : s_val[k];
#pragma unroll
                for (int j = 0; j < VPT; ++j)
                    if (live[j]) acc[j] = MIN ? fminf(acc[j], __fsub_rn((float)p[32 * j], sv)) : fmaxf(acc[j], __fadd_rn((float)p[32 * j], sv));
            }
        }
        float* o = static_cast<float*>(P.out) + e;
#pragma unroll
        for (int j = 0; j < VPT; ++j)
            if (live[j]) o[32 * j] = acc[j];
    }
}

// Border kernel: the voxels within reach of a face, enumerated as at most two slabs per axis (a slab = the whole
// image with one axis cut down to [start, start + width)).  Slabs overlap at edges and corners; those voxels are
// computed more than once, to the same value.  Every neighbour coordinate is mapped by the border rule.
struct Slabs {
    int count;
    int axis[2 * kMaxDims], start[2 * kMaxDims], width[2 * kMaxDims];
    int64_t first[2 * kMaxDims + 1];  // running sum of slab sizes (voxels per image)
};

template <typename T, bool MIN, bool BINARY>
__global__ void __launch_bounds__(256) morph_border_kernel(const __grid_constant__ Params P,
                                                           const __grid_constant__ Slabs S, const int64_t items) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= items) return;
    const int64_t per_image = S.first[S.count];
    const int64_t img = t / per_image;
    int64_t li = t - img * per_image;
    int sl = 0;
    while (sl + 1 < S.count && li >= S.first[sl + 1]) ++sl;
    li -= S.first[sl];
    int x[kMaxDims];
    int vox = 0;
    {
        uint32_t rr = (uint32_t)li;
#pragma unroll
        for (int a = kMaxDims - 1; a >= 0; --a) {
            x[a] = 0;
            if (a < P.ndim) {
                const uint32_t n = a == S.axis[sl] ? (uint32_t)S.width[sl] : (uint32_t)P.ext[a], q = rr / n;
                x[a] = (int)(rr - q * n) + (a == S.axis[sl] ? S.start[sl] : 0);
                rr = q;
                vox += x[a] * P.stride[a];
            }
        }
    }
    const T* __restrict__ base = static_cast<const T*>(P.in) + img * P.V;
    float acc = MIN ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
    int bacc = MIN ? 1 : 0;
    for (int k = 0; k < P.n_entries; ++k) {
        const Entry en = P.entries[k];
        int lin = 0;
        bool inside = true;
#pragma unroll
        for (int a = 0; a < kMaxDims; ++a) {
            if (a < P.ndim) {
                int c = x[a] + en.off[a];
                inside = map_coord(c, P.ext[a], P.mode) && inside;
                lin += c * P.stride[a];
            }
        }
        if (BINARY) {
            const int v = inside ? (base[lin] != 0) : P.border_value;
            if (MIN ? !v : v) { bacc = v; break; }
        } else {
            const float v = inside ? (float)base[lin] : P.cval;
            acc = MIN ? fminf(acc, __fsub_rn(v, en.s)) : fmaxf(acc, __fadd_rn(v, en.s));
        }
    }
    const int64_t e = img * P.V + vox;
    if (BINARY) static_cast<uint8_t*>(P.out)[e] = (uint8_t)bacc;
    else static_cast<float*>(P.out)[e] = acc;
}

}  // namespace tmmorph
