// Launch code of the quad-per-lane kernels (edt_lean.cuh): a translation unit of its own.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <mutex>

#include "edt_lean.cuh"
#include "host_plan.h"

namespace tmedt {

// Largest dynamic shared-memory size configured so far per (kernel, device): the attribute is set once, not per call.
struct SmemAttr { const void* fn; int dev; size_t bytes; };
static SmemAttr g_smem_attr[256];
static int g_smem_attr_count = 0;
static std::mutex g_smem_attr_mutex;

cudaError_t ensure_smem(const void* fn, size_t smem) {
    if (smem <= 48 * 1024) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(g_smem_attr_mutex);
    SmemAttr* slot = nullptr;
    for (int i = 0; i < g_smem_attr_count; ++i)
        if (g_smem_attr[i].fn == fn && g_smem_attr[i].dev == dev) { slot = &g_smem_attr[i]; break; }
    if (slot && slot->bytes >= smem) return cudaSuccess;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (!slot && g_smem_attr_count < 256) slot = &g_smem_attr[g_smem_attr_count++];
    if (slot) { slot->fn = fn; slot->dev = dev; slot->bytes = smem; }
    return cudaSuccess;
}

// Quad-per-lane kernels (edt_lean.cuh) for the shapes they cover: three or four processed axes, contiguous extent a
// multiple of 4, outputs aligned for 16-byte (float32) and 32-byte (int64) stores, exact integer keys (unit sampling, or scaled integers without index output),
// index output (coordinate planes or one linear index per voxel) with every spatial axis processed.
bool lean_ok(const Plan& pl, const uint8_t* in, const EpilogueParams& ep) {
    if (!pl.fast || pl.E < 3 || pl.E > 4 || pl.ext[0] % 4 != 0 || ((uintptr_t)in & 3u) != 0) return false;
    if (((uintptr_t)ep.dist & 15u) || ((uintptr_t)ep.sq & 31u) || ((uintptr_t)ep.idx & 31u)) return false;
    if (ep.idx) return pl.unit && pl.ndim == pl.E;
    return pl.unit || pl.scaled || pl.vscaled;  // (vscaled: a scale that fits plain 32-bit values, no index output)
}

template <int VS, typename VT>
static cudaError_t launch_lean_plane(const LeanParams& P, int64_t planes, cudaStream_t st) {
    const size_t smem = (size_t)(P.n + 2 * kLeanPad) * VS * 4;
    // full-width planes: three blocks per SM fit whatever their size, so each gets 16 warps (more resident warps to
    // cover the latencies of the first-axis pass and of long scans)
    if (VS == 128) {
        auto kern = lean_plane_kernel<VS, VT, 16>;
        cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)planes, 512, smem, st>>>(P);
        return cudaGetLastError();
    }
    auto kern = lean_plane_kernel<VS, VT, 8>;
    cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)planes, 256, smem, st>>>(P);
    return cudaGetLastError();
}

template <typename VT>
static cudaError_t launch_lean_plane_vs(const LeanParams& P, int64_t planes, cudaStream_t st) {
    if (P.n0 <= 32) return launch_lean_plane<32, VT>(P, planes, st);
    if (P.n0 <= 64) return launch_lean_plane<64, VT>(P, planes, st);
    return launch_lean_plane<128, VT>(P, planes, st);
}

// Columns per tile of a later axis: about 2048 to 4096 voxels per block.
static int lean_tile_columns(int n, int64_t inner) {
    int tx = n <= 32 ? 128 : (n <= 64 ? 64 : 32);
    while (tx > 32 && tx / 2 >= inner) tx >>= 1;
    return tx;
}

template <int K, bool FINAL, int TX>
static cudaError_t launch_lean_column_tx(LeanParams P, const EpilogueParams& ep, int64_t outer, cudaStream_t st) {
    const size_t smem = (size_t)(P.n + 2 * kLeanPad) * TX * 4 + (size_t)P.n * TX * entry_bytes(K);
    P.tiles_per_slab = (int)((P.inner + TX - 1) / TX);
    if (FINAL && ep.flat) {
        auto kern = lean_column_kernel<K, FINAL, TX, FINAL>;
        cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)(outer * P.tiles_per_slab), 256, smem, st>>>(P, ep);
        return cudaGetLastError();
    }
    auto kern = lean_column_kernel<K, FINAL, TX>;
    cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)(outer * P.tiles_per_slab), 256, smem, st>>>(P, ep);
    return cudaGetLastError();
}

template <int K, bool FINAL>
static cudaError_t launch_lean_column(const LeanParams& P, const EpilogueParams& ep, int64_t outer, cudaStream_t st) {
    const int tx = lean_tile_columns(P.n, P.inner);
    if (tx == 128) return launch_lean_column_tx<K, FINAL, 128>(P, ep, outer, st);
    if (tx == 64) return launch_lean_column_tx<K, FINAL, 64>(P, ep, outer, st);
    return launch_lean_column_tx<K, FINAL, 32>(P, ep, outer, st);
}

template <bool FINAL, typename VT, int TX>
static cudaError_t launch_lean_value_tx(LeanParams P, const EpilogueParams& ep, int64_t outer, cudaStream_t st) {
    const size_t smem = (size_t)(P.n + 2 * kLeanPad) * TX * 4;
    P.tiles_per_slab = (int)((P.inner + TX - 1) / TX);
    if (TX < 32 || P.n >= 384) {  // very long axes, narrow tiles: two blocks per SM, 32 warps each
        auto kern = lean_value_kernel<FINAL, VT, TX, 32>;
        cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)(outer * P.tiles_per_slab), 1024, smem, st>>>(P, ep);
        return cudaGetLastError();
    }
    if (TX == 32 && P.n > 128) {  // long axes: few blocks fit an SM, so each gets 16 warps
        auto kern = lean_value_kernel<FINAL, VT, TX, 16>;
        cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)(outer * P.tiles_per_slab), 512, smem, st>>>(P, ep);
        return cudaGetLastError();
    }
    auto kern = lean_value_kernel<FINAL, VT, TX>;
    cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)(outer * P.tiles_per_slab), 256, smem, st>>>(P, ep);
    return cudaGetLastError();
}

template <bool FINAL, typename VT>
static cudaError_t launch_lean_value(const LeanParams& P, const EpilogueParams& ep, int64_t outer, cudaStream_t st) {
    const int tx = lean_tile_columns(P.n, P.inner);
    if (tx == 128) return launch_lean_value_tx<FINAL, VT, 128>(P, ep, outer, st);
    if (tx == 64) return launch_lean_value_tx<FINAL, VT, 64>(P, ep, outer, st);
    return launch_lean_value_tx<FINAL, VT, 32>(P, ep, outer, st);
}

// One axis pass of the wide-key path on plain integer values (unit sampling, no index output, extents up to 1024)
// with the quad kernel lean_value_kernel: `in` / `out` hold one 32-bit value per voxel (2^31 = no site).
// Columns per tile on axis k: 32 where that gives every SM its blocks; with few columns (a single image) and 384
// rows or more, tiles of 16 or 8 columns; 0 = too few tiles even so (wide_axis_kernel splits its strips over several
// blocks instead) or too many rows.
static int lean_value_tile(const Plan& pl, int k) {
    const int n = pl.ext[k];
    const size_t smem = (size_t)(n + 2 * kLeanPad) * 32 * 4;
    if (smem > 136 * 1024) return 0;  // up to 1024 rows (one block of 32 warps per SM beyond 100 KB)
    const int64_t outer = pl.N / ((int64_t)n * pl.inner[k]);
    auto blocks = [&](int tx) { return outer * ((pl.inner[k] + tx - 1) / tx); };
    const int64_t resident = smem > 100 * 1024 ? 148 : 296;  // blocks of 32-column tiles the device holds at once
    const bool narrow = n >= 384 && !switches().no_narrow_tiles;
    // fewer than four rounds of 32-column tiles: the last, partly filled round weighs less with tiles of 16 columns
    // (32 images of 512 x 512: 0.0446 -> 0.0409 ms; 8 of 1024 x 1024: 0.068 -> 0.060 ms; with many rounds -- a 512^3
    // volume -- the wider tile wins, 0.49 against 0.61 ms)
    if (narrow && blocks(32) < 4 * resident && blocks(16) >= 148) return 16;
    if (blocks(32) >= resident) return 32;
    if (!narrow) return 0;
    if (blocks(8) >= 96) return 8;
    return 0;
}

bool lean_value_axis_ok(const Plan& pl, int k, const EpilogueParams& ep) {
    if ((!pl.unit && !pl.vscaled) || ep.idx || pl.ext[0] % 4 != 0) return false;
    if (((uintptr_t)ep.dist & 15u) || ((uintptr_t)ep.sq & 31u)) return false;
    return lean_value_tile(pl, k) != 0;
}

cudaError_t run_lean_value_axis(const Plan& pl, int k, const void* in, void* out, const EpilogueParams& ep, bool fin,
                                cudaStream_t st, bool dist16) {
    LeanParams P;
    memset(&P, 0, sizeof(P));
    P.in = in; P.out = out;
    P.in_elems = pl.N; P.out_elems = pl.N; P.images = pl.images;
    P.n = pl.ext[k]; P.inner = pl.inner[k];
    P.wk = pl.unit ? 1u : (uint32_t)pl.vsi[k]; P.w0 = pl.unit ? 1u : (uint32_t)pl.vsi[0];  // (scaled sampling: integer weights)
    P.inv_scale = pl.unit ? 1.0f : (float)(1.0 / pl.vscale);
    const int64_t outer = pl.N / ((int64_t)pl.ext[k] * pl.inner[k]);
    const int tx = lean_value_tile(pl, k);
    if (dist16) {  // 16-bit first-axis distances in; final outputs or 32-bit values out
        P.dist16 = 1;
        if (tx == 16) return fin ? launch_lean_value_tx<true, uint16_t, 16>(P, ep, outer, st)
                                 : launch_lean_value_tx<false, uint16_t, 16>(P, ep, outer, st);
        if (tx == 8) return fin ? launch_lean_value_tx<true, uint16_t, 8>(P, ep, outer, st)
                                : launch_lean_value_tx<false, uint16_t, 8>(P, ep, outer, st);
        return fin ? launch_lean_value_tx<true, uint16_t, 32>(P, ep, outer, st)
                   : launch_lean_value_tx<false, uint16_t, 32>(P, ep, outer, st);
    }
    if (tx == 16) return fin ? launch_lean_value_tx<true, uint32_t, 16>(P, ep, outer, st)
                             : launch_lean_value_tx<false, uint32_t, 16>(P, ep, outer, st);
    if (tx == 8) return fin ? launch_lean_value_tx<true, uint32_t, 8>(P, ep, outer, st)
                            : launch_lean_value_tx<false, uint32_t, 8>(P, ep, outer, st);
    return fin ? launch_lean_value_tx<true, uint32_t, 32>(P, ep, outer, st)
               : launch_lean_value_tx<false, uint32_t, 32>(P, ep, outer, st);
}

// The same pass on axes beyond 1024 rows: the whole column still fits a shared-memory tile if the tile is only 16, 8
// or 4 columns wide (one block of 32 warps per SM); 32-bit values in, values or final outputs out.
static int lean_value_long_tile(int n) {
    const size_t rows = (size_t)(n + 2 * kLeanPad);
    // one block per SM; narrower tiles that would let two blocks share an SM are not faster (4096 rows: 0.408 ms with
    // 4 columns and two blocks against 0.400 ms with 8 columns and one)
    if (rows * 16 * 4 <= 136 * 1024) return 16;
    if (rows * 8 * 4 <= 136 * 1024) return 8;
    if (rows * 4 * 4 <= 136 * 1024) return 4;
    return 0;
}

bool lean_value_long_axis_ok(const Plan& pl, int k, const EpilogueParams& ep) {
    if ((!pl.unit && !pl.vscaled) || ep.idx || pl.ext[0] % 4 != 0) return false;
    if (((uintptr_t)ep.dist & 15u) || ((uintptr_t)ep.sq & 31u)) return false;
    const int n = pl.ext[k], tx = lean_value_long_tile(n);
    if (n <= 1024 || tx == 0) return false;
    const int64_t blocks = pl.N / ((int64_t)n * pl.inner[k]) * ((pl.inner[k] + tx - 1) / tx);
    return blocks >= 148;
}

template <bool FINAL, int TX>
static cudaError_t launch_lean_value_long(LeanParams P, const EpilogueParams& ep, int64_t outer, cudaStream_t st) {
    const size_t smem = (size_t)(P.n + 2 * kLeanPad) * TX * 4;
    P.tiles_per_slab = (int)((P.inner + TX - 1) / TX);
    auto kern = lean_value_kernel<FINAL, uint32_t, TX, 32>;
    cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)(outer * P.tiles_per_slab), 1024, smem, st>>>(P, ep);
    return cudaGetLastError();
}

cudaError_t run_lean_value_long_axis(const Plan& pl, int k, const void* in, void* out, const EpilogueParams& ep, bool fin,
                                     cudaStream_t st) {
    LeanParams P;
    memset(&P, 0, sizeof(P));
    P.in = in; P.out = out;
    P.in_elems = pl.N; P.out_elems = pl.N; P.images = pl.images;
    P.n = pl.ext[k]; P.inner = pl.inner[k];
    P.wk = pl.unit ? 1u : (uint32_t)pl.vsi[k]; P.w0 = pl.unit ? 1u : (uint32_t)pl.vsi[0];  // (scaled sampling: integer weights)
    P.inv_scale = pl.unit ? 1.0f : (float)(1.0 / pl.vscale);
    const int64_t outer = pl.N / ((int64_t)pl.ext[k] * pl.inner[k]);
    const int tx = lean_value_long_tile(P.n);
    if (tx == 16)
        return fin ? launch_lean_value_long<true, 16>(P, ep, outer, st) : launch_lean_value_long<false, 16>(P, ep, outer, st);
    if (tx == 8)
        return fin ? launch_lean_value_long<true, 8>(P, ep, outer, st) : launch_lean_value_long<false, 8>(P, ep, outer, st);
    return fin ? launch_lean_value_long<true, 4>(P, ep, outer, st) : launch_lean_value_long<false, 4>(P, ep, outer, st);
}

// every axis pass after the first on one of the two forms above
bool lean_value_all_axes_ok(const Plan& pl, const EpilogueParams& ep) {
    for (int k = 1; k < pl.E; ++k)
        if (!lean_value_axis_ok(pl, k, ep) && !lean_value_long_axis_ok(pl, k, ep)) return false;
    return pl.E >= 2;
}

cudaError_t run_lean(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws, cudaStream_t st, int& launches) {
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    char* bufA = static_cast<char*>(ws);
    char* bufB = bufA + up((size_t)pl.N * 4);
    const double out_bpv = out_bytes_per_voxel(ep);
    const bool entries = ep.idx != nullptr;
    double sumsq = 0.0;
    for (int p = 0; p < pl.E; ++p) sumsq += (double)(pl.ext[p] - 1) * (pl.ext[p] - 1);
    const bool v16 = !entries && pl.unit && sumsq < 65535.0;
    const double carry = entries ? 2.0 : (v16 ? 2.0 : 4.0);  // bytes per voxel the plane kernel writes
    auto weight = [&](int p) { return pl.unit ? 1u : (uint32_t)(pl.scaled ? pl.si[p] : pl.vsi[p]); };
    LeanParams P;
    memset(&P, 0, sizeof(P));
    P.in = in; P.out = bufA;
    P.in_elems = pl.N; P.out_elems = pl.N; P.images = pl.images;
#ifdef TM_EDT_DEBUG
    // test hook of the debug build: a bound that is too small on purpose, so that the checks fire on valid accesses
    // (which are then skipped) and the reporting path can be tested without any invalid access
    if (switches().debug_inject) P.out_elems = 16;
#endif
    P.n0 = pl.ext[0]; P.n = pl.ext[1]; P.inner = pl.inner[1];
    P.w0 = weight(0); P.wk = weight(1);
    P.inv_scale = (float)(1.0 / (pl.unit || pl.scaled ? pl.scale : pl.vscale));
    for (int q = 0; q < 4; ++q) {
        P.shift[q] = -1;
        if (q < pl.E)
            for (int s = 0; s < 8; ++s)
                if (pl.ext[q] == (1 << s)) P.shift[q] = s;
    }
    const int64_t planes = pl.N / ((int64_t)pl.ext[0] * pl.ext[1]);
    prof_mark(st, "plane", (double)pl.N * (1.0 + carry));
    cudaError_t e = entries ? launch_lean_plane_vs<uint8_t>(P, planes, st)
                            : (v16 ? launch_lean_plane_vs<uint16_t>(P, planes, st) : launch_lean_plane_vs<uint32_t>(P, planes, st));
    ++launches;
    if (e != cudaSuccess) return e;
    char* src = bufA;
    char* dst = bufB;
    for (int k = 2; k < pl.E; ++k) {
        const bool fin = k == pl.E - 1;
        P.in = src; P.out = dst;
        P.n = pl.ext[k]; P.inner = pl.inner[k]; P.wk = weight(k);
        P.reverse = fin ? 0 : 1;  // a pass between the plane pass and the last one walks its blocks backwards
        const int64_t outer = pl.N / ((int64_t)pl.ext[k] * pl.inner[k]);
        if (entries) {
            const double eb = (double)entry_bytes(k);
            prof_mark(st, fin ? "column_final" : "column", (double)pl.N * (eb + (fin ? out_bpv : (double)entry_bytes(k + 1))));
            if (k == 2) e = fin ? launch_lean_column<2, true>(P, ep, outer, st) : launch_lean_column<2, false>(P, ep, outer, st);
            else e = launch_lean_column<3, true>(P, ep, outer, st);
        } else {
            prof_mark(st, fin ? "column_value_final" : "column_value", (double)pl.N * (carry + (fin ? out_bpv : carry)));
            if (v16) e = fin ? launch_lean_value<true, uint16_t>(P, ep, outer, st) : launch_lean_value<false, uint16_t>(P, ep, outer, st);
            else e = fin ? launch_lean_value<true, uint32_t>(P, ep, outer, st) : launch_lean_value<false, uint32_t>(P, ep, outer, st);
        }
        ++launches;
        if (e != cudaSuccess) return e;
        char* t = src; src = dst; dst = t;
    }
    return cudaSuccess;
}

// Debug build: violations recorded by the kernels of this translation unit (cleared by the call).
cudaError_t lean_debug_collect(cudaStream_t st, DebugRecord* out) {
#ifdef TM_EDT_DEBUG
    return debug_collect(st, out);
#else
    (void)st;
    out->count = 0;
    return cudaSuccess;
#endif
}

}  // namespace tmedt
