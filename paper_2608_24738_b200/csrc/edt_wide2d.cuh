// Two-dimensional images with extents up to 1024 and unit sampling (the packed 8-bit entries of the fast
// path stop at 128).  Two kernels:
//   row_keys_kernel     first-axis pass, one warp per row, 16 or 32 voxels per lane (128-bit loads).
//                       Writes, per voxel, the scan key  (off^2 << SH) | row  (32 bit; SH = 9 row bits for
//                       extents up to 512, 10 up to 1024: 2 * 1023^2 << 10 still stays below 2^31) and the
//                       signed 16-bit offset to the nearest zero of the row.
//   wide_column_kernel  second-axis pass and epilogue: a block stages the keys of an (n1 x 32) column
//                       strip in shared memory and runs the grouped bounded scan on it (edt_fast.cuh);
//                       the first-axis offset of the chosen site is fetched from global memory only
//                       when indices are requested.
// Same mathematics as the fast path: g_1(y, x) = min_j [ off(j, x)^2 + (y - j)^2 ], exact in integers.
#pragma once
#include "edt_fast.cuh"

namespace tmedt {


struct WideParams {
    const uint8_t* in;   // (images, n1, n0)
    uint32_t* keys;      // (images, n1, n0)
    int16_t* offs;       // (images, n1, n0)
    int64_t rows;        // images * n1
    int n0, n1;
};

template <int VPL, int SH>  // voxels per lane (16 or 32), row bits of the key
__global__ void __launch_bounds__(256) row_keys_kernel(const __grid_constant__ WideParams P) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= P.rows) return;  // the whole warp leaves together
    const int n0 = P.n0;
    const int y = (int)(row % P.n1);
    const uint8_t* src = P.in + row * n0;
    constexpr int CH = VPL / 16;  // 16-byte chunks per lane
    uint32_t zb = 0u;             // bit b set: voxel b of this lane is zero
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        uint4 v = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
        if (VPL * lane + 16 * c < n0) v = *reinterpret_cast<const uint4*>(src + VPL * lane + 16 * c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t m = ~(((w[i] & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w[i]) & 0x80808080u;
            // gather the four flag bits (bits 7, 15, 23, 31) into bits 0..3
            zb |= ((((m >> 7) * 0x00204081u) >> 21) & 0xfu) << (16 * c + 4 * i);
        }
    }
    const unsigned any = __ballot_sync(0xffffffffu, zb != 0u);
    uint32_t keys[VPL];
    int16_t offs[VPL];
    if (any == 0u) {
#pragma unroll
        for (int b = 0; b < VPL; ++b) { keys[b] = kNoneKey16; offs[b] = (int16_t)-32768; }
    } else {
        const int lzin = zb ? 31 - __clz(zb) : 0;
        const int fzin = zb ? __ffs(zb) - 1 : 0;
        const unsigned ml = any & ((1u << lane) - 1u);
        const unsigned mr = lane < 31 ? any >> (lane + 1) : 0u;
        const int Ll = ml ? 31 - __clz(ml) : 0;
        const int Lr = mr ? lane + __ffs(mr) : 0;
        const int lz_l = __shfl_sync(0xffffffffu, lzin, Ll);
        const int fz_r = __shfl_sync(0xffffffffu, fzin, Lr);
        const int x0 = VPL * lane;
        int dl[VPL];
        int cur = ml ? VPL * Ll + lz_l : -4096;
#pragma unroll
        for (int b = 0; b < VPL; ++b) {
            if ((zb >> b) & 1u) cur = x0 + b;
            dl[b] = x0 + b - cur;
        }
        cur = mr ? VPL * Lr + fz_r : 8192;
#pragma unroll
        for (int b = VPL - 1; b >= 0; --b) {
            if ((zb >> b) & 1u) cur = x0 + b;
            const int dr = cur - (x0 + b);
            const int a = min(dl[b], dr);
            offs[b] = (int16_t)(dl[b] <= dr ? -a : a);
            keys[b] = ((uint32_t)(a * a) << SH) | (uint32_t)y;
        }
    }
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        if (VPL * lane + 16 * c < n0) {
            uint4* kdst = reinterpret_cast<uint4*>(P.keys + row * n0 + VPL * lane + 16 * c);
#pragma unroll
            for (int i = 0; i < 4; ++i)
                kdst[i] = make_uint4(keys[16 * c + 4 * i], keys[16 * c + 4 * i + 1], keys[16 * c + 4 * i + 2],
                                     keys[16 * c + 4 * i + 3]);
            uint32_t pk[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
                pk[i] = (uint32_t)(uint16_t)offs[16 * c + 2 * i] | ((uint32_t)(uint16_t)offs[16 * c + 2 * i + 1] << 16);
            uint4* odst = reinterpret_cast<uint4*>(P.offs + row * n0 + VPL * lane + 16 * c);
            odst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            odst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        }
    }
}

template <int SH>
__global__ void __launch_bounds__(512) wide_column_kernel(const __grid_constant__ WideParams P,
                                                          const __grid_constant__ EpilogueParams ep,
                                                          const int strips_per_image) {
    extern __shared__ __align__(16) uint8_t sm_wide[];
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_wide);  // [n1][32]
    const int n0 = P.n0, n1 = P.n1;
    const int64_t img = blockIdx.x / strips_per_image;
    const int c0 = (int)(blockIdx.x - img * strips_per_image) * 32;
    const uint32_t* src = P.keys + img * (int64_t)n1 * n0 + c0;
    // stage: 8 threads copy one row of 32 keys (n0 is a multiple of 16, so a strip is 16 or 32 columns wide)
    const int width = min(32, n0 - c0);
    for (int t = threadIdx.x; t < n1 * 8; t += blockDim.x) {
        const int y = t >> 3, ch = t & 7;
        if (4 * ch < width)
            *reinterpret_cast<uint4*>(val + y * 32 + 4 * ch) = *reinterpret_cast<const uint4*>(src + (int64_t)y * n0 + 4 * ch);
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if (lane >= width) return;
    const int c = c0 + lane;
    constexpr int R = 4;
    constexpr uint32_t kRowMask = (1u << SH) - 1u;
    const int64_t base = img * ep.V + c;   // voxel (row 0, column c) of this image
    for (int y0 = warp * R; y0 < n1; y0 += nwarps * R) {
        uint32_t best[R];
        scan_keys_group<32, R, SH>(val + lane, n1, y0, best);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int y = y0 + i;
            if (y >= n1) break;
            const uint32_t b = best[i];
            const bool none = b >= kNoneKey16;
            const int64_t p = base + (int64_t)y * n0;
            const int sq = (int)(b >> SH);
            if (ep.dist) ep.dist[p] = none ? TMEDT_INF : __fsqrt_rn(small_int_to_float(sq));
            if (ep.sq) ep.sq[p] = none ? INT64_MAX : (int64_t)sq;
            if (ep.idx) {
                // two processed axes: plane 0 = contiguous axis, plane 1 = this axis; other axes have extent 1
                const int j = (int)(b & kRowMask);
                const int off0 = none ? 0 : (int)P.offs[img * (int64_t)n1 * n0 + (int64_t)j * n0 + c];
                for (int a = 0; a < ep.ndim; ++a) {
                    int64_t v = 0;
                    if (a == ep.axis[0]) v = c + off0;
                    if (a == ep.axis[1]) v = j;
                    ep.idx[(img * ep.ndim + a) * ep.V + (int64_t)y * n0 + c] = none ? -1 : v;
                }
            }
        }
    }
}

}  // namespace tmedt
