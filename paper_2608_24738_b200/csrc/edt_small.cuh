// Small extents (every processed axis <= 8), any rank up to 8.  The carry between kernels is the squared
// distance itself (float32; exact integers under unit sampling, where sum (n-1)^2 <= 8 * 49) plus, only
// when indices are requested, the linear index of the site inside its image.
//
// Consecutive axes are grouped while the product of their extents stays <= 256.  One kernel handles one
// group: a block stages a tile (all coordinates of the group's axes x 32 neighbours along the remaining
// index) in shared memory and runs the group's axes over it one after the other.  For one axis a thread
// owns one line, holds its <= 8 values in registers and takes the minimum over all pairs
//     g_k(x) = min_j [ g_{k-1}(x with x_k := j) + (w_k (x_k - j))^2 ]      (paper, Section 2.3.2)
// directly: 56 compare-and-select steps at most.  The first kernel reads the mask, the last one writes
// the outputs, so an 8-D transform of extent 6 takes three launches.
#pragma once
#include "edt_common.cuh"

namespace tmedt {

constexpr int kSmallProd = 256;   // largest product of extents in one group
constexpr int kSmallT = 32;       // neighbours per tile
constexpr int kSmallThreads = 512;

struct SmallParams {
    const uint8_t* mask;     // first group
    const float* in_val;     // later groups
    const int32_t* in_site;  // later groups, with indices
    float* out_val;          // all but the last group
    int32_t* out_site;       // all but the last group, with indices
    int64_t outer, inner;    // view (outer, prod, inner) of the whole batch
    int64_t V;               // voxels per image
    int prod;                // product of the group's extents
    int m;                   // axes in the group
    int n[kMaxDims];         // their extents, fastest first
    float w2[kMaxDims];      // their squared samplings
};

template <bool SITE, bool FIRST, bool FINAL, int NMAX>
__global__ void __launch_bounds__(kSmallThreads, (!SITE && NMAX <= 6) ? 4 : 1) small_group_kernel(const __grid_constant__ SmallParams P,
                                                          const __grid_constant__ EpilogueParams ep) {
    extern __shared__ __align__(16) unsigned char small_smem[];
    float* sv = reinterpret_cast<float*>(small_smem);
    int* ss = reinterpret_cast<int*>(small_smem) + P.prod * kSmallT;
    const float inf = __int_as_float(0x7f800000);
    const int prod = P.prod;
    // inner == 1: the tile is T consecutive outer indices, a contiguous run of global memory, kept in
    // that order (t * prod + c).  Otherwise: one outer index, T consecutive inner ones, kept as c * T + t.
    const bool contiguous = P.inner == 1;
    int64_t o, r0;
    int tcount;
    if (contiguous) {
        o = (int64_t)blockIdx.x * kSmallT; r0 = 0;
        tcount = (int)min((int64_t)kSmallT, P.outer - o);
    } else {
        const unsigned tpo = (unsigned)((P.inner + kSmallT - 1) / kSmallT);
        const unsigned ob = blockIdx.x / tpo;
        o = ob; r0 = (int64_t)(blockIdx.x - ob * tpo) * kSmallT;
        tcount = (int)min((int64_t)kSmallT, P.inner - r0);
    }
    const int elems = contiguous ? tcount * prod : prod * kSmallT;
    // element e of the tile sits at gbase + offset(e); offsets stay below the voxel count of one image
    // (inner > 1) or of T * prod (inner == 1), so 32 bits hold them
    const int64_t gbase = contiguous ? o * prod : o * prod * P.inner + r0;
    const int inner32 = (int)P.inner;
    auto global_of = [&](int e, bool& live) -> int64_t {
        if (contiguous) { live = true; return gbase + e; }
        const int c = (unsigned)e / (unsigned)kSmallT, t = e - c * kSmallT;
        live = t < tcount;
        return gbase + (c * inner32 + t);
    };
    for (int e = threadIdx.x; e < elems; e += blockDim.x) {
        bool live;
        const int64_t g = global_of(e, live);
        float v = inf;
        int s = -1;
        if (live) {
            if (FIRST) {
                const bool bg = P.mask[g] == 0;
                v = bg ? 0.f : inf;
                if (SITE) s = bg ? (int)(g % P.V) : -1;
            } else {
                v = P.in_val[g];
                if (SITE) s = P.in_site[g];
            }
        }
        sv[e] = v;
        if (SITE) ss[e] = s;
    }
    __syncthreads();
    int cs = 1;  // stride of the current axis inside the group's coordinate space
    for (int q = 0; q < P.m; ++q) {
        const int n = P.n[q];
        const float w2 = P.w2[q];
        const int rest = prod / n;  // lines per neighbour
        const int lines = rest * (contiguous ? tcount : kSmallT);
        for (int l = threadIdx.x; l < lines; l += blockDim.x) {
            int t, cp;
            if (contiguous) { t = (unsigned)l / (unsigned)rest; cp = l - t * rest; }
            else { cp = (unsigned)l / (unsigned)kSmallT; t = l - cp * kSmallT; }
            const int hi = (unsigned)cp / (unsigned)cs, lo = cp - hi * cs;
            const int c0 = lo + hi * cs * n;
            const int a0 = contiguous ? t * prod + c0 : c0 * kSmallT + t;
            const int as = contiguous ? cs : cs * kSmallT;
            float v[NMAX];
            int s[NMAX];
#pragma unroll
            for (int j = 0; j < NMAX; ++j) {
                v[j] = inf; s[j] = -1;
                if (j < n) { v[j] = sv[a0 + j * as]; if (SITE) s[j] = ss[a0 + j * as]; }
            }
#pragma unroll
            for (int i = 0; i < NMAX; ++i) {
                if (i >= n) break;
                float best = v[i];
                int bs = s[i];
#pragma unroll
                for (int j = 0; j < NMAX; ++j) {
                    if (j == i) continue;
                    const float c = v[j] + w2 * (float)((i - j) * (i - j));
                    if (SITE) { if (c < best) { best = c; bs = s[j]; } }
                    else best = fminf(best, c);
                }
                sv[a0 + i * as] = best;
                if (SITE) ss[a0 + i * as] = bs;
            }
        }
        __syncthreads();
        cs *= n;
    }
    for (int e = threadIdx.x; e < elems; e += blockDim.x) {
        bool live;
        const int64_t g = global_of(e, live);
        if (!live) continue;
        const float best = sv[e];
        if (!FINAL) {
            P.out_val[g] = best;
            if (SITE) P.out_site[g] = ss[e];
        } else {
            const bool none = best == inf;
            if (ep.dist) ep.dist[g] = __fsqrt_rn(best);
            if (ep.sq) ep.sq[g] = none ? INT64_MAX : (int64_t)best;  // unit sampling: an exact small integer
            if (SITE && ep.flat) {
                ep.idx[g] = none ? -1 : (int64_t)ss[e];  // the carried site index is the linear index inside the image
            } else if (SITE) {
                // site = linear index inside the image; planes in processing order, plane 0 fastest
                const int64_t img = g / P.V, vox = g - img * P.V;
                int coord[kMaxDims];
                int rr = none ? 0 : ss[e];
#pragma unroll
                for (int p = 0; p < kMaxDims; ++p) {
                    coord[p] = 0;
                    if (p < ep.E) { coord[p] = rr % ep.ext[p]; rr /= ep.ext[p]; }
                }
                for (int a = 0; a < ep.ndim; ++a) {
                    const int p = ep.plane_of_axis[a];
                    int64_t val = 0;
#pragma unroll
                    for (int q = 0; q < kMaxDims; ++q)
                        if (q == p) val = coord[q];
                    ep.idx[(img * ep.ndim + a) * ep.V + vox] = none ? -1 : val;
                }
            }
        }
    }
}

}  // namespace tmedt
