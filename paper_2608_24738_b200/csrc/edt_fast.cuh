// Fast path for extents up to 128 and at most five processed axes.
//
// Carry layout ("entries"): after p + 1 processed axes every voxel holds one little packed entry whose
// byte q (q <= p) is the signed offset  site_q - x_q  along processed axis q (plane order: contiguous
// axis first); 1, 2, 4 bytes for 1, 2, 3..4 axes.  Byte 0 == 0x80 marks "no site yet".  An entry of
// all zeros is a background voxel.  Entries make every load, gather and store of a voxel one access.
//
// Kernels:
//   plane_kernel   first axis + second axis fused: one thread block per (n_1 x n_0) plane.  The rows
//                  of the raw mask are bit-packed with warp ballots and turned into 1-byte offsets in
//                  shared memory (first-axis pass), then one thread per column runs the envelope pass
//                  along axis 1 on the shared tile and writes 2-byte entries or the final outputs.
//   column_kernel  one further axis: a block stages an (n x TX) tile of entries in shared memory
//                  (TX consecutive positions of the contiguous `inner` index), one thread per column
//                  runs the envelope pass, outputs go straight to global memory (a warp writes one
//                  contiguous run per row).
//
// Envelope pass of one column (lower envelope of parabolas, paper Section 2.3.2; here split at
// background voxels).  A background voxel has height 0, so no site beyond it can matter to the voxels
// before it: the column falls apart into independent runs of foreground voxels, each bounded by the
// background voxels next to it.  Background rows cost a load and a store.  Within a run the sites are
// pushed on a stack of row numbers (one byte each, in shared memory); site v between u and w is dropped
// when the parabola intersections are out of order, tested without division:
//     (H_v - H_u) (w - v) >= (H_w - H_v) (v - u),   H_s = h_s + w^2 s^2.
// The two top entries are cached in registers.  The query walks the surviving sites upward and moves
// to the next one past their intersection  x* = (H_next - H_cur) / (2 w^2 (next - cur)).
// All arithmetic is float32; for unit sampling every value is an integer below 2^24, hence exact.
#pragma once
#include "edt_common.cuh"

namespace tmedt {

template <int BYTES> struct EntryType;
template <> struct EntryType<1> { using type = uint8_t; };
template <> struct EntryType<2> { using type = uint16_t; };
template <> struct EntryType<4> { using type = uint32_t; };
__host__ __device__ constexpr int entry_bytes(int axes) { return axes <= 1 ? 1 : (axes == 2 ? 2 : 4); }

struct FastParams {
    const void* in;      // mask (plane kernel) or entries of K axes (column kernel)
    void* out;           // entries of K + 1 axes (unused when FINAL)
    int64_t outer;       // number of (outer) slabs; the array is (outer, n, inner)
    int64_t inner;
    int n;               // extent of the axis of this pass
    int n0;              // plane kernel: extent of the contiguous axis (== inner)
    float w2;            // squared sampling of this axis
    float inv2w2;        // 1 / (2 w2)
    float w2p[4];        // squared sampling of the earlier axes (plane order)
    int unit;            // all sampling == 1
};

__device__ __forceinline__ float small_int_to_float(int v) {  // exact for 0 <= v < 2^23, two full-rate ops
    return __int_as_float(v | 0x4B000000) - 8388608.0f;
}

template <int K> __device__ __forceinline__ bool entry_none(uint32_t e) { return (e & 0xffu) == 0x80u; }

template <int K>
__device__ __forceinline__ float entry_height(uint32_t e, const float* w2p, bool unit) {
    int o0 = (int)(int8_t)(e & 0xff);
    if (unit) {
        int s = o0 * o0;
        if (K > 1) { int o = (int)(int8_t)((e >> 8) & 0xff); s += o * o; }
        if (K > 2) { int o = (int)(int8_t)((e >> 16) & 0xff); s += o * o; }
        if (K > 3) { int o = (int)(int8_t)((e >> 24) & 0xff); s += o * o; }
        return small_int_to_float(s);
    }
    float h = w2p[0] * small_int_to_float(o0 * o0);
    if (K > 1) { int o = (int)(int8_t)((e >> 8) & 0xff); h = fmaf(w2p[1], small_int_to_float(o * o), h); }
    if (K > 2) { int o = (int)(int8_t)((e >> 16) & 0xff); h = fmaf(w2p[2], small_int_to_float(o * o), h); }
    if (K > 3) { int o = (int)(int8_t)((e >> 24) & 0xff); h = fmaf(w2p[3], small_int_to_float(o * o), h); }
    return h;
}

// Per-column output sink.
template <int K, bool FINAL>
struct ColumnOut {
    // non-final
    typename EntryType<entry_bytes(K + 1)>::type* out;  // &out[first voxel of the column]
    // final
    float* dist; int64_t* sq; int64_t* idx;  // &buf[image base + first voxel of the column]; idx: plane 0 of image
    int64_t stride;      // distance between consecutive rows of the column, in voxels
    int64_t V;           // voxels per image (index-plane stride)
    int coord[4];        // own coordinates along the earlier planes
    int axis[5];         // spatial axis of plane p
    int ndim;
    bool unit;
};

template <int K, bool FINAL>
__device__ __forceinline__ void emit(const ColumnOut<K, FINAL>& o, int y, uint32_t e, int offk, float h, bool none) {
    if (!FINAL) {
        using EO = typename EntryType<entry_bytes(K + 1)>::type;
        uint32_t v = none ? 0x80u : (e | ((uint32_t)(uint8_t)(int8_t)offk << (8 * (K & 3))));
        o.out[(int64_t)y * o.stride] = (EO)v;
        return;
    }
    const int64_t p = (int64_t)y * o.stride;
    if (none) {
        if (o.dist) o.dist[p] = __int_as_float(0x7f800000);
        if (o.sq) o.sq[p] = INT64_MAX;
        if (o.idx)
            for (int a = 0; a < o.ndim; ++a) o.idx[(int64_t)a * o.V + p] = -1;
        return;
    }
    if (o.dist) o.dist[p] = o.unit ? __fsqrt_rn(h) : sqrtf(h);
    int off[5];
#pragma unroll
    for (int q = 0; q < K; ++q) off[q] = (int)(int8_t)((e >> (8 * q)) & 0xff);
    off[K] = offk;
    if (o.sq) {
        int s = 0;
#pragma unroll
        for (int q = 0; q <= K; ++q) s += off[q] * off[q];
        o.sq[p] = (int64_t)s;
    }
    if (o.idx) {
        // axes of extent 1 keep index 0; processed axes get own coordinate + offset
        for (int a = 0; a < o.ndim; ++a) {
            int64_t val = 0;
#pragma unroll
            for (int q = 0; q <= K; ++q)
                if (o.axis[q] == a) val = (int64_t)((q == K ? y : o.coord[q]) + off[q]);
            o.idx[(int64_t)a * o.V + p] = val;
        }
    }
}

// One column of a shared-memory tile.  tile[y * tstride] is the entry of row y (ET = tile element type),
// stk[k * sstride] the k-th stack slot of this column (3n/2 + 2 slots).
//
// Two sweeps, both with all lanes of a warp on the same row, so that the row's loads and stores are one
// contiguous run per warp.  Sweep 1 builds, run by run, the surviving sites; the segments of successive
// runs follow one another on the stack, each run's last slot carrying an end mark (bit 7; rows are
// below 128).  Background rows that do not touch a run are not on the stack at all.  Sweep 2 emits the
// outputs: background rows directly, foreground rows by walking the segment of their run.
template <int K, bool FINAL, typename ET>
__device__ __forceinline__ void column_pass(const ET* __restrict__ tile, int tstride, uint8_t* __restrict__ stk,
                                            int sstride, int n, const FastParams& P,
                                            const ColumnOut<K, FINAL>& out) {
    const float w2 = P.w2, inv2w2 = P.inv2w2;
    const bool unit = P.unit != 0;
    float w2p[4] = {P.w2p[0], P.w2p[1], P.w2p[2], P.w2p[3]};

    // ---- sweep 1: build ----
    int k = -1;                 // top slot
    int base = 0;               // first slot of the open run
    int s1 = 0, s0 = 0;         // rows of the top and below-top entries of the open run
    float fs1 = 0.f, fs0 = 0.f, H1 = 0.f, H0 = 0.f, D10 = 0.f, d10 = 0.f;
    bool open = false;          // a run of foreground rows is open
    int lastbg = -1;            // most recent background row

    auto push = [&](int u, float fu, float Hu) {
        while (k > base) {
            if (D10 * (fu - fs1) >= (Hu - H1) * d10) {  // top is nowhere the minimum: pop
                --k; s1 = s0; fs1 = fs0; H1 = H0;
                if (k > base) {
                    s0 = stk[(k - 1) * sstride];
                    fs0 = small_int_to_float(s0);
                    H0 = fmaf(w2 * fs0, fs0, entry_height<K>((uint32_t)tile[s0 * tstride], w2p, unit));
                    D10 = H1 - H0; d10 = fs1 - fs0;
                }
            } else break;
        }
        ++k;
        stk[k * sstride] = (uint8_t)u;
        s0 = s1; fs0 = fs1; H0 = H1;
        s1 = u; fs1 = fu; H1 = Hu;
        D10 = H1 - H0; d10 = fs1 - fs0;
    };

    {
        float fy = 0.f;
        for (int y = 0; y < n; ++y, fy += 1.0f) {
            const uint32_t e = (uint32_t)tile[y * tstride];
            if (e == 0u) {  // background voxel
                if (open) {  // closes the run: it is the run's last site
                    push(y, fy, w2 * fy * fy);
                    stk[k * sstride] = (uint8_t)(y | 0x80);
                    open = false;
                }
                lastbg = y;
                continue;
            }
            if (!open) {  // first foreground row after background (or row 0): start a run
                open = true;
                base = k + 1;
                if (lastbg >= 0) {
                    k = base;
                    stk[k * sstride] = (uint8_t)lastbg;
                    s1 = lastbg; fs1 = small_int_to_float(lastbg); H1 = w2 * fs1 * fs1;
                }
            }
            if (entry_none<K>(e)) continue;  // foreground without a site so far: no site, still in the run
            push(y, fy, fmaf(w2 * fy, fy, entry_height<K>(e, w2p, unit)));
        }
    }
    const int ktop = k;  // last slot in use (-1: the column has no site at all)

    // ---- sweep 2: emit ----
    int kc = -1;                // slot of the current site
    bool in_run = false, last = true;   // `last`: the current site is the last of its run
    int sc = 0; uint32_t ec = 0; float fsc = 0.f, hc = 0.f, Hc = 0.f;
    int sn = 0; uint32_t en = 0; float fsn = 0.f, hn = 0.f, Hn = 0.f;
    bool nlast = true;
    float xb = __int_as_float(0x7f800000);
    auto load_site = [&](int slot, int& s, uint32_t& e, float& fs, float& h, float& H, bool& is_last) {
        const int raw = stk[slot * sstride];
        is_last = (raw & 0x80) != 0 || slot == ktop;
        s = raw & 0x7f;
        e = (uint32_t)tile[s * tstride];
        fs = small_int_to_float(s);
        h = entry_height<K>(e, w2p, unit);
        H = fmaf(w2 * fs, fs, h);
    };
    auto load_next = [&]() {
        if (!last) {
            load_site(kc + 1, sn, en, fsn, hn, Hn, nlast);
            xb = __fdividef((Hn - Hc) * inv2w2, fsn - fsc);
        } else {
            xb = __int_as_float(0x7f800000);
        }
    };
    float fy = 0.f;
    for (int y = 0; y < n; ++y, fy += 1.0f) {
        const uint32_t e = (uint32_t)tile[y * tstride];
        if (e == 0u) {
            emit<K, FINAL>(out, y, 0u, 0, 0.f, false);
            in_run = false;
            continue;
        }
        if (ktop < 0) {  // no site in the whole column
            emit<K, FINAL>(out, y, 0u, 0, 0.f, true);
            continue;
        }
        if (!in_run) {  // first row of a run: move to the first slot of its segment
            in_run = true;
            if (kc >= 0) {
                while (!last) { ++kc; last = (stk[kc * sstride] & 0x80) != 0 || kc == ktop; }
            }
            ++kc;
            load_site(kc, sc, ec, fsc, hc, Hc, last);
            load_next();
        }
        while (fy > xb) {
            ++kc; sc = sn; ec = en; fsc = fsn; hc = hn; Hc = Hn; last = nlast;
            load_next();
        }
        const float d = fsc - fy;
        emit<K, FINAL>(out, y, ec, sc - y, fmaf(w2 * d, d, hc), false);
    }
}

// ---------------------------------------------------------------------------------------------
// First-axis pass of one row of a plane into shared memory: 1-byte offsets (or 0x80).
// One warp per row at a time; n0 <= 128, i.e. at most four ballot words.  All branch conditions are
// warp-uniform (they depend on the ballot words only).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pass0_row_to_tile(const uint8_t* __restrict__ row, int n0, uint8_t* __restrict__ trow,
                                                  int lane) {
    unsigned Z[4];
    const int nw = (n0 + 31) >> 5;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        Z[w] = 0u;
        if (w < nw) {
            const int x = w * 32 + lane;
            const uint8_t b = x < n0 ? row[x] : (uint8_t)1;
            Z[w] = __ballot_sync(0xffffffffu, x < n0 && b == 0);
        }
    }
    int prevw[4], nextw[4];
    int last = -1000;
#pragma unroll
    for (int w = 0; w < 4; ++w) { prevw[w] = last; if (Z[w]) last = w * 32 + 31 - __clz(Z[w]); }
    int first = 1000;
#pragma unroll
    for (int w = 3; w >= 0; --w) { nextw[w] = first; if (Z[w]) first = w * 32 + __ffs(Z[w]) - 1; }
    const bool none = last < 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        if (w >= nw) break;
        const int x = w * 32 + lane;
        int off;
        if (none) off = -128;
        else if (Z[w] == 0xffffffffu) off = 0;
        else {
            const unsigned Zl = Z[w] & (0xffffffffu >> (31 - lane));
            const unsigned Zr = Z[w] >> lane;
            const int lp = Zl ? w * 32 + 31 - __clz(Zl) : prevw[w];
            const int rp = Zr ? x + __ffs(Zr) - 1 : nextw[w];
            off = (x - lp <= rp - x) ? (lp - x) : (rp - x);
        }
        if (x < n0) trow[x] = (uint8_t)(int8_t)off;
    }
}

template <bool FINAL>
__global__ void __launch_bounds__(128) plane_kernel(const __grid_constant__ FastParams P,
                                                    const __grid_constant__ EpilogueParams ep) {
    extern __shared__ __align__(16) uint8_t sm_plane[];
    const int n0 = P.n0, n1 = P.n;
    const int tstride = (n0 + 15) & ~15;
    uint8_t* tile = sm_plane;                       // [n1][tstride]
    uint8_t* stk = sm_plane + (size_t)n1 * tstride; // [3 n1 / 2 + 2][blockDim]
    const int64_t plane = blockIdx.x;               // planes = outer
    const uint8_t* src = reinterpret_cast<const uint8_t*>(P.in) + plane * (int64_t)n1 * n0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int y = warp; y < n1; y += nwarps) pass0_row_to_tile(src + (int64_t)y * n0, n0, tile + y * tstride, lane);
    __syncthreads();
    const int c = threadIdx.x;
    if (c >= n0) return;
    ColumnOut<1, FINAL> out;
    out.stride = n0;
    if (!FINAL) {
        out.out = reinterpret_cast<uint16_t*>(P.out) + plane * (int64_t)n1 * n0 + c;
    } else {
        // two processed axes: the plane is the image
        out.dist = ep.dist ? ep.dist + plane * ep.V + c : nullptr;
        out.sq = ep.sq ? ep.sq + plane * ep.V + c : nullptr;
        out.idx = ep.idx ? ep.idx + plane * ep.ndim * ep.V + c : nullptr;
        out.V = ep.V; out.ndim = ep.ndim; out.unit = P.unit != 0;
        out.coord[0] = c;
        out.axis[0] = ep.axis[0]; out.axis[1] = ep.axis[1];
    }
    column_pass<1, FINAL, uint8_t>(tile + c, tstride, stk + c, blockDim.x, n1, P, out);
}

template <int K, bool FINAL>
__global__ void __launch_bounds__(128) column_kernel(const __grid_constant__ FastParams P,
                                                     const __grid_constant__ EpilogueParams ep,
                                                     const int tiles_per_slab) {
    using EI = typename EntryType<entry_bytes(K)>::type;
    extern __shared__ __align__(16) uint8_t sm_col[];
    const int TX = blockDim.x, n = P.n;
    EI* tile = reinterpret_cast<EI*>(sm_col);                                  // [n][TX]
    uint8_t* stk = sm_col + (size_t)n * TX * sizeof(EI);                       // [3 n / 2 + 2][TX]
    const int64_t slab = blockIdx.x / tiles_per_slab;
    const int64_t i0 = (int64_t)(blockIdx.x - slab * tiles_per_slab) * TX;
    const int width = (int)min((int64_t)TX, P.inner - i0);
    const EI* src = reinterpret_cast<const EI*>(P.in) + slab * (int64_t)n * P.inner + i0;
    // stage the tile: 16-byte chunks when rows are 16-byte aligned, single entries otherwise
    constexpr int PER16 = 16 / (int)sizeof(EI);
    if ((P.inner % PER16) == 0 && (width % PER16) == 0) {
        const int chunks = width / PER16;
        for (int t = threadIdx.x; t < n * chunks; t += TX) {
            const int y = t / chunks, ch = t - y * chunks;
            const uint4 v = *reinterpret_cast<const uint4*>(src + (int64_t)y * P.inner + ch * PER16);
            *reinterpret_cast<uint4*>(tile + y * TX + ch * PER16) = v;
        }
    } else {
        for (int t = threadIdx.x; t < n * width; t += TX) {
            const int y = t / width, x = t - y * width;
            tile[y * TX + x] = src[(int64_t)y * P.inner + x];
        }
    }
    __syncthreads();
    const int c = threadIdx.x;
    if (c >= width) return;
    ColumnOut<K, FINAL> out;
    out.stride = P.inner;
    if (!FINAL) {
        using EO = typename EntryType<entry_bytes(K + 1)>::type;
        out.out = reinterpret_cast<EO*>(P.out) + slab * (int64_t)n * P.inner + i0 + c;
    } else {
        // last pass: the slab is the image; i0 + c enumerates the earlier planes, plane 0 fastest
        const int64_t v0 = i0 + c;
        out.dist = ep.dist ? ep.dist + slab * ep.V + v0 : nullptr;
        out.sq = ep.sq ? ep.sq + slab * ep.V + v0 : nullptr;
        out.idx = ep.idx ? ep.idx + slab * ep.ndim * ep.V + v0 : nullptr;
        out.V = ep.V; out.ndim = ep.ndim; out.unit = P.unit != 0;
        int64_t rr = v0;
#pragma unroll
        for (int q = 0; q < K; ++q) { out.coord[q] = (int)(rr % ep.ext[q]); rr /= ep.ext[q]; }
#pragma unroll
        for (int q = 0; q <= K; ++q) out.axis[q] = ep.axis[q];
    }
    column_pass<K, FINAL, EI>(tile + c, TX, stk + c, TX, n, P, out);
}

}  // namespace tmedt
