// Packed-entry path without an index output: between passes a voxel carries its squared distance so far (an
// exact integer: squared voxel units under unit sampling, scale * sum_q w_q^2 off_q^2 in scaled-integer mode)
// instead of the offsets of its site.  The key of a pass is then the value itself, with no arithmetic on offsets,
// no tile of entries is kept in shared memory, and nothing is fetched for the output:
//     g_k(x) = min_j [ g_{k-1}(x with x_k := j) + (w_k (x_k - j))^2 ]      (paper, Section 2.3.2)
// is carried as g itself.  VT = uint16_t when every value fits 16 bits (unit sampling, up to four axes of extent
// 128: 4 * 127^2 = 64516), else uint32_t; the all-ones value means "no site yet".
#pragma once
#include "edt_fast.cuh"

namespace tmedt {

template <typename VT> struct ValueNone;
template <> struct ValueNone<uint16_t> { static constexpr uint32_t v = 0xffffu; };
template <> struct ValueNone<uint32_t> { static constexpr uint32_t v = 0xffffffffu; };

// One further axis on carried values.  SCALED: weighted addends (P.sk * d^2), else d^2.
//   FINAL == false  writes the new value (VT);  FINAL == true  writes float32 distances and / or int64 squared distances.
template <bool FINAL, typename VT, bool SCALED, int TX>
__global__ void __launch_bounds__(256) column_value_kernel(const __grid_constant__ FastParams P,
                                                           const __grid_constant__ EpilogueParams ep,
                                                           const int tiles_per_slab) {
    extern __shared__ __align__(16) uint8_t sm_val[];
    constexpr int G = TX / 32;
    constexpr int SH = 0;  // no site is needed afterwards: the key is the value itself, without row bits
    constexpr uint32_t NONE = kNoneKey16;
    constexpr uint32_t VNONE = ValueNone<VT>::v;
    const int n = P.n;
    uint32_t* val = reinterpret_cast<uint32_t*>(sm_val);  // [n][TX]
    const int64_t slab = blockIdx.x / tiles_per_slab;
    const int64_t i0 = (int64_t)(blockIdx.x - slab * tiles_per_slab) * TX;
    const int width = (int)min((int64_t)TX, P.inner - i0);
    const VT* src = reinterpret_cast<const VT*>(P.in) + slab * (int64_t)n * P.inner + i0;
    constexpr int PER16 = 16 / (int)sizeof(VT);
    if ((P.inner % PER16) == 0 && width == TX) {  // full tile, 16-byte aligned rows
        constexpr int FULL = TX / PER16;
        for (int t = threadIdx.x; t < n * FULL; t += blockDim.x) {
            const int y = t / FULL, ch = t - y * FULL;
            const uint4 v = *reinterpret_cast<const uint4*>(src + (int64_t)y * P.inner + ch * PER16);
            const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
            uint32_t kv[PER16];
#pragma unroll
            for (int i = 0; i < PER16; ++i) {
                const uint32_t word = wv[(i * (int)sizeof(VT)) >> 2];
                const uint32_t x = sizeof(VT) == 4 ? word : ((word >> (16 * (i & 1))) & 0xffffu);
                kv[i] = x == VNONE ? NONE : x;
            }
#pragma unroll
            for (int i = 0; i < PER16; i += 4)
                *reinterpret_cast<uint4*>(val + y * TX + ch * PER16 + i) = make_uint4(kv[i], kv[i + 1], kv[i + 2], kv[i + 3]);
        }
    } else {
        for (int t = threadIdx.x; t < n * width; t += blockDim.x) {
            const int y = t / width, x = t - y * width;
            const uint32_t v = (uint32_t)src[(int64_t)y * P.inner + x];
            val[y * TX + x] = v == VNONE ? NONE : v;
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = warp % G, r0 = warp / G, rstep = nwarps / G;
    const int c = g * 32 + lane;
    if (c >= width) return;
    const int64_t col = slab * (int64_t)n * P.inner + i0 + c;  // row 0 of this column (FINAL: the slab is the image)
    VT* __restrict__ out = reinterpret_cast<VT*>(P.out);
    constexpr int R = 4;
    for (int y0 = r0 * R; y0 < n; y0 += rstep * R) {
        uint32_t best[R];
        scan_keys_group<TX, R, SH>(val + c, n, y0, best, SCALED ? (uint32_t)P.sk : 1u);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int y = y0 + i;
            if (y >= n) break;
            const uint32_t b = best[i];
            const bool none = b >= NONE;
            const uint32_t v = b >> SH;
            const int64_t p = col + (int64_t)y * P.inner;
            if (!FINAL) {
                out[p] = (VT)(none ? VNONE : v);
            } else {
                if (ep.dist) {
                    const float sqv = SCALED ? __uint2float_rn(v) * P.inv_scale : small_int_to_float((int)v);
                    __stcs(ep.dist + p, none ? TMEDT_INF : fast_sqrt(sqv));
                }
                if (ep.sq) __stcs(reinterpret_cast<long long*>(ep.sq + p), none ? (long long)INT64_MAX : (long long)v);  // unit sampling only
            }
        }
    }
}

}  // namespace tmedt
