// Fused erosion / dilation kernel (paper, Section 2.3.2 "Fused morphology kernel").  The host flattens the
// structuring element into its active entries; each entry carries the per-axis offsets and the flat offset
// against the image's strides.  A thread owns one output voxel.  If its whole neighbourhood lies inside the
// image (tested with the per-axis offset extrema) it adds flat offsets to its linear index and nothing else;
// otherwise every neighbour coordinate is mapped by the border rule.  One template covers erosion and dilation
// (identity and combine differ), greyscale and binary (the binary form stops as soon as the result is decided).
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

template <typename T, bool MIN, bool BINARY>
__global__ void __launch_bounds__(256) morph_kernel(const __grid_constant__ Params P) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= P.total) return;
    const int64_t img = e / P.V;
    const int vox = (int)(e - img * P.V);
    const T* __restrict__ base = static_cast<const T*>(P.in) + img * P.V;
    int x[kMaxDims];
    bool interior = true;
    {
        uint32_t rr = (uint32_t)vox;
#pragma unroll
        for (int a = kMaxDims - 1; a >= 0; --a) {
            x[a] = 0;
            if (a < P.ndim) {
                const uint32_t n = (uint32_t)P.ext[a], q = rr / n;
                x[a] = (int)(rr - q * n);
                rr = q;
                interior = interior && x[a] + P.lo[a] >= 0 && x[a] + P.hi[a] < (int)n;
            }
        }
    }
    float acc = MIN ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
    int bacc = MIN ? 1 : 0;
    if (interior) {
        for (int k = 0; k < P.n_entries; ++k) {
            const int fo = P.entries[k].flat;
            if (BINARY) {
                const int v = base[vox + fo] != 0;
                if (MIN ? !v : v) { bacc = v; break; }
            } else {
                const float s = P.entries[k].s;
                const float v = (float)base[vox + fo];
                acc = MIN ? fminf(acc, __fsub_rn(v, s)) : fmaxf(acc, __fadd_rn(v, s));
            }
        }
    } else {
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
    }
    if (BINARY) static_cast<uint8_t*>(P.out)[e] = (uint8_t)bacc;
    else static_cast<float*>(P.out)[e] = acc;
}

}  // namespace tmmorph
