// Binary erosion / dilation on bit-packed lines (paper, Section 2.3.1: the binary form of the fused kernel combines
// the neighbourhood with AND / OR and a single border value).  A mask needs one bit per voxel, so the combine of 32
// voxels with one neighbour position is one funnel shift and one logic instruction on 32-bit words:
//   1. binary_pack_kernel     mask bytes -> one bit per voxel (bit b of word w of a line = voxel 32 w + b is nonzero);
//                             a lane takes 32 consecutive voxels (one 32-byte load), N / 8 bytes of scratch.
//   2. binary_lines_kernel    the host groups the element's active positions by their offsets along all axes but the
//                             contiguous one; a group is a neighbouring line plus a 64-bit mask of offsets along
//                             the line.  A lane produces one output word: per group it reads three words of the
//                             neighbouring line (or takes the border value if that line lies outside the image), and
//                             per offset of the group shifts the 96-bit window into place and combines it; the result
//                             is expanded to bytes and leaves as one 32-byte store.
//   3. binary_fused2d_kernel  both steps in one launch for elements that reach over the last two axes only: a block
//                             packs its lines and those within reach into shared memory and combines from there.
// Requires at most 4 axes, a contiguous extent that is a multiple of 32 with 32-byte aligned buffers (256-bit accesses)
// or a multiple of 4 from 32 voxels on with 4-byte aligned buffers (the last word of a line is then ragged), and offsets
// along the line within +-31; everything else runs on the byte kernels of morph.cuh.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "morph.cuh"

namespace tmmorph {

struct LineGroup {
    int16_t off[kMaxDims];  // offsets along the axes before the contiguous one (entry ndim - 1 unused)
    int64_t line_offset;    // the same as a number of lines inside one image
    uint64_t mask;          // bit (dx + 31) set: offset dx along the line is active
};

constexpr int kMaxLineGroups = 96;  // groups travel as kernel arguments (no copy to the device, no extra latency)

struct BitsParams {
    const uint8_t* in;
    uint8_t* out;
    uint32_t* bits;          // (lines, words) packed mask
    LineGroup groups[kMaxLineGroups];
    int n_groups;
    int ndim;
    int64_t lines;           // images * lines per image
    int64_t lines_per_image;
    int words;               // words per line = last extent / 32
    int ext[kMaxDims];
    int border_value;
    int fast;                // the contiguous extent is a multiple of 32 and both buffers are 32-byte aligned: 256-bit accesses
};

__device__ __forceinline__ uint32_t nonzero_bits4(uint32_t v) {
    // bit i = byte i of v is nonzero
    const uint32_t m = (((v & 0x7f7f7f7fu) + 0x7f7f7f7fu) | v) & 0x80808080u;  // 0x80 in every nonzero byte
    return (((m >> 7) * 0x00204081u) >> 21) & 0xfu;
}

// Word w (32 voxels) of a line of W voxels as bits.  W is a multiple of 32 (fast: one 256-bit load; the buffer is
// 32-byte aligned) or of 4 (4-byte loads; the voxels of a ragged last word beyond the line take the border value, like
// every other position outside the image).
__device__ __forceinline__ uint32_t bits_load_word(const uint8_t* line, const int w, const int W, const bool fast,
                                                   const uint32_t fill) {
    uint32_t v[8];
    if (fast) {
        asm("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"  // read-only data: free to be scheduled early
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
            : "l"(line + 32 * w));
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            v[i] = 32 * w + 4 * i < W ? __ldg(reinterpret_cast<const uint32_t*>(line + 32 * w) + i) : (fill & 0x01010101u);
    }
    uint32_t bits = 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) bits |= nonzero_bits4(v[i]) << (4 * i);
    return bits;
}

// 32 result bits -> bytes (0 / 1) of word w of a line of W voxels.
__device__ __forceinline__ void bits_store_word(uint8_t* line, const int w, const int W, const bool fast, const uint32_t acc) {
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t nib = (acc >> (4 * i)) & 0xfu;
        o[i] = (nib * 0x00204081u) & 0x01010101u;
    }
    if (fast) {
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     :: "l"(line + 32 * w), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                     : "memory");
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (32 * w + 4 * i < W) reinterpret_cast<uint32_t*>(line + 32 * w)[i] = o[i];
    }
}

__global__ void __launch_bounds__(256) binary_pack_kernel(const __grid_constant__ BitsParams P) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;  // word index over the whole batch
    if (t >= P.lines * P.words) return;
    const int64_t line = t / P.words;
    const int w = (int)(t - line * P.words), W = P.ext[P.ndim - 1];
    P.bits[t] = bits_load_word(P.in + line * W, w, W, P.fast, P.border_value ? 0xffffffffu : 0u);
}

// Block = 8 x 32 lanes (threadIdx.y, threadIdx.x); a lane produces word w of L consecutive lines, which differ only in
// their coordinate along the axis before the contiguous one (the host picks L = 4 when that extent is a multiple of
// 4), so that a group's offsets are decoded once for L words.  Blocks enumerate (group of 8 L lines, chunk of 32
// words).  ND: number of axes (1 .. 4).
template <bool MIN, int L, int ND>
__global__ void __launch_bounds__(256) binary_lines_kernel(const __grid_constant__ BitsParams P, const unsigned chunks) {
    const unsigned lb = blockIdx.x / chunks, ch = blockIdx.x - lb * chunks;
    const int64_t line0 = ((int64_t)lb * 8 + threadIdx.y) * L;
    const int w = (int)(ch * 32 + threadIdx.x);
    if (line0 >= P.lines || w >= P.words) return;
    // coordinates of the first line along the axes before the contiguous one (fewer than 2^31 lines per image)
    int x[ND > 1 ? ND - 1 : 1];
    x[0] = 0;
    {
        uint32_t rr = (uint32_t)(line0 % P.lines_per_image);
#pragma unroll
        for (int a = ND - 2; a >= 0; --a) {
            const uint32_t n = (uint32_t)P.ext[a], q = rr / n;
            x[a] = (int)(rr - q * n);
            rr = q;
        }
    }
    const uint32_t fill = P.border_value ? 0xffffffffu : 0u;
    uint32_t acc[L];
#pragma unroll
    for (int j = 0; j < L; ++j) acc[j] = MIN ? 0xffffffffu : 0u;
    for (int g = 0; g < P.n_groups; ++g) {
        const LineGroup& G = P.groups[g];
        bool in_outer = true;
#pragma unroll
        for (int a = 0; a < ND - 2; ++a) in_outer = in_outer && (unsigned)(x[a] + G.off[a]) < (unsigned)P.ext[a];
        const uint32_t* row = P.bits + (line0 + G.line_offset) * P.words + w;
        uint32_t lo[L], mid[L], hi[L];  // words w - 1, w, w + 1 of the neighbouring lines
#pragma unroll
        for (int j = 0; j < L; ++j) {
            const bool inside = in_outer && (ND < 2 || (unsigned)(x[ND > 1 ? ND - 2 : 0] + j + G.off[ND > 1 ? ND - 2 : 0]) < (unsigned)P.ext[ND > 1 ? ND - 2 : 0]);
            lo[j] = fill; mid[j] = fill; hi[j] = fill;
            if (inside) {
                const uint32_t* r = row + (int64_t)j * P.words;
                mid[j] = r[0];
                if (w > 0) lo[j] = r[-1];
                if (w + 1 < P.words) hi[j] = r[1];
            }
        }
        // output bit i takes input bit i + dx: offsets to the left (dx = b - 31 <= 0), then to the right
        for (uint32_t m = (uint32_t)G.mask; m; m &= m - 1) {
            const int sh = 31 - (__ffs((int)m) - 1);  // -dx (a shift of 0 returns mid)
#pragma unroll
            for (int j = 0; j < L; ++j) {
                const uint32_t v = __funnelshift_l(lo[j], mid[j], sh);
                acc[j] = MIN ? acc[j] & v : acc[j] | v;
            }
        }
        for (uint32_t m = (uint32_t)(G.mask >> 32); m; m &= m - 1) {
            const int sh = __ffs((int)m);  // dx = bit + 1
#pragma unroll
            for (int j = 0; j < L; ++j) {
                const uint32_t v = __funnelshift_r(mid[j], hi[j], sh);
                acc[j] = MIN ? acc[j] & v : acc[j] | v;
            }
        }
        uint32_t all = acc[0];
#pragma unroll
        for (int j = 1; j < L; ++j) all = MIN ? all | acc[j] : all & acc[j];
        if (all == (MIN ? 0u : 0xffffffffu)) break;  // decided for every voxel of the lane
    }
    // expand 32 bits to 32 bytes (0 / 1): one 256-bit store per line
    const int W = P.ext[P.ndim - 1];
#pragma unroll
    for (int j = 0; j < L; ++j) bits_store_word(P.out + (line0 + j) * W, w, W, P.fast, acc[j]);
}

// Elements that reach over the last two axes only (every 2-D element): packing and combining in one kernel, without
// the packed copy of the mask in global memory.  A block takes 32 lines x 32 words; it packs those lines and the
// lines within reach above and below them (dy_lo .. dy_hi), with one word on either side, into shared memory, then
// every lane produces word w of four consecutive lines as binary_lines_kernel does.  H: extent of the axis before
// the contiguous one (1 for a 1-D image).
constexpr int kFusedReach = 8;  // |dy| of the element, at most

template <bool MIN, bool FAST>
__global__ void __launch_bounds__(256) binary_fused2d_kernel(const __grid_constant__ BitsParams P, const unsigned chunks,
                                                             const int H, const int dy_lo, const int dy_hi) {
    __shared__ uint32_t sbits[32 + 2 * kFusedReach][34];
    const unsigned lb = blockIdx.x / chunks, ch = blockIdx.x - lb * chunks;
    const int64_t l0 = (int64_t)lb * 32;
    const int w0 = (int)ch * 32;
    const uint32_t fill = P.border_value ? 0xffffffffu : 0u;
    const int rows = 32 + dy_hi - dy_lo;
    const int W = P.ext[P.ndim - 1];
#pragma unroll 3
    for (int t = threadIdx.x; t < rows * 34; t += 256) {
        const int r = t / 34, c = t - r * 34;
        const int64_t line = l0 + dy_lo + r;
        const int w = w0 - 1 + c;
        uint32_t bits = fill;  // words beyond the ends of a line hold the border value
        if (w >= 0 && w < P.words) {
            bits = 0u;
            if (line >= 0 && line < P.lines) bits = bits_load_word(P.in + line * W, w, W, FAST, fill);
        }
        sbits[r][c] = bits;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int w = w0 + lane;
    const int64_t line0 = l0 + 4 * ty;
    if (w >= P.words || line0 >= P.lines) return;
    const int y0 = (int)(line0 % H);
    uint32_t acc[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[j] = MIN ? 0xffffffffu : 0u;
    for (int g = 0; g < P.n_groups; ++g) {
        const LineGroup& G = P.groups[g];
        const int dy = P.ndim >= 2 ? G.off[P.ndim - 2] : 0;
        uint32_t lo[4], mid[4], hi[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int y = y0 + j;
            if (y >= H) y -= H * (y / H);  // the next image (H < 4: several images further)
            const bool inside = (unsigned)(y + dy) < (unsigned)H;
            const uint32_t* row = sbits[4 * ty + j + dy - dy_lo];
            lo[j] = inside ? row[lane] : fill;
            mid[j] = inside ? row[lane + 1] : fill;
            hi[j] = inside ? row[lane + 2] : fill;
        }
        for (uint32_t m = (uint32_t)G.mask; m; m &= m - 1) {
            const int sh = 31 - (__ffs((int)m) - 1);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t v = __funnelshift_l(lo[j], mid[j], sh);
                acc[j] = MIN ? acc[j] & v : acc[j] | v;
            }
        }
        for (uint32_t m = (uint32_t)(G.mask >> 32); m; m &= m - 1) {
            const int sh = __ffs((int)m);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t v = __funnelshift_r(mid[j], hi[j], sh);
                acc[j] = MIN ? acc[j] & v : acc[j] | v;
            }
        }
        const uint32_t all = MIN ? (acc[0] | acc[1] | acc[2] | acc[3]) : (acc[0] & acc[1] & acc[2] & acc[3]);
        if (all == (MIN ? 0u : 0xffffffffu)) break;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (line0 + j >= P.lines) break;
        bits_store_word(P.out + (line0 + j) * W, w, W, FAST, acc[j]);
    }
}

}  // namespace tmmorph
