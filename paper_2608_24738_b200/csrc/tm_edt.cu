// C ABI of the distance-transform library: argument validation, the host-side plan
// (all geometry is resolved on the host: paper, Section 2.2.2 "Three layers") and kernel launches.
#include "../../include/tm_edt.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <mutex>

#include "edt_common.cuh"
#include "edt_generic.cuh"
#include "edt_fast.cuh"
#include "edt_wide.cuh"
#include "edt_small.cuh"
#include "edt_long.cuh"
#include "edt_compat.cuh"
#include "edt_value.cuh"
#include "host_shared.h"
#include "host_plan.h"
#include <stdlib.h>

namespace tmedt {

static thread_local int g_last_cuda_error = 0;
static thread_local int g_last_launches = 0;
static thread_local DebugRecord g_last_debug = {0ull, 0, 0, 0};  // debug build: record of this thread's last call

// Debug and test switches.  The environment is read once, at the first call that needs a switch, and again only
// when tm_edt_reload_switches() is called (the tests change switches inside one process).
static Switches g_switches;
static bool g_switches_loaded = false;
static std::mutex g_switches_mutex;

static void load_switches_locked() {
    auto on = [](const char* name) { const char* v = getenv(name); return v && v[0] == '1'; };
    auto set = [](const char* name) { return getenv(name) != nullptr; };
    Switches s;
    s.force_generic = on("TM_EDT_FORCE_GENERIC");
    s.no_scaled = set("TM_EDT_NO_SCALED");
    s.old_plane = on("TM_EDT_OLD_PLANE");
    s.no_value_carry = set("TM_EDT_NO_VALUE_CARRY");
    s.no_lean = set("TM_EDT_NO_LEAN");
    s.no_narrow_tiles = set("TM_EDT_NO_NARROW_TILES");
    s.debug_inject = on("TM_EDT_DEBUG_INJECT");
    s.chunk_voxels = 0;
    if (const char* lim = getenv("TM_EDT_CHUNK_VOXELS")) { const long long v = atoll(lim); if (v > 0) s.chunk_voxels = v; }
    g_switches = s;
    g_switches_loaded = true;
}

const Switches& switches() {
    std::lock_guard<std::mutex> lock(g_switches_mutex);
    if (!g_switches_loaded) load_switches_locked();
    return g_switches;
}

// Optional per-kernel timing (tm_edt_profile): an event is recorded on the stream before every launch
// and once after the last one.
constexpr int kProfMax = 32;
struct Profiler {
    bool active = false;
    int count = 0;
    cudaEvent_t ev[kProfMax + 1];
    const char* name[kProfMax];
    double bytes[kProfMax];
};
static thread_local Profiler g_prof;

// `bytes`: what this launch has to read and write once (its inputs plus its outputs).
void prof_mark(cudaStream_t st, const char* name, double bytes) {
    if (!g_prof.active || g_prof.count >= kProfMax) return;
    cudaEventRecord(g_prof.ev[g_prof.count], st);
    g_prof.name[g_prof.count] = name;
    g_prof.bytes[g_prof.count] = bytes;
    ++g_prof.count;
}

// Scratch layout of the wide-key and long-line paths: two 32-bit key (or height) buffers, and -- only when an index
// output is requested -- 16-bit offsets per processed axis; the long-line path adds its block minima.
struct WideLayout { size_t keysA, offsA, keysB, offsB, offsC, bm, total; };

static WideLayout wide_layout(int64_t N, int E, bool want_idx, bool block_minima) {
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    WideLayout L;
    size_t o = 0;
    L.keysA = o; o += up((size_t)N * 4);
    L.offsA = o; if (want_idx) o += up((size_t)N * 2);
    L.keysB = o; if (E >= 3) o += up((size_t)N * 4);
    L.offsB = o; if (E >= 3 && want_idx) o += up((size_t)N * 4);
    L.offsC = o; if (E == 4 && want_idx) o += up((size_t)N * 8);
    L.bm = o; if (block_minima) o += up((size_t)N / 4 + 1024);
    L.total = o;
    return L;
}

// want_idx: whether the call asks for the index output (scratch of the wide-key and long-line paths depends on it).
static int make_plan(int ndim, const int64_t* shape, const double* sampling, Plan& pl, bool want_idx = true) {
    if (!shape || ndim < 1 || ndim > kMaxDims) return TM_EDT_ERR_INVALID_ARG;
    for (int k = 0; k < ndim + 2; ++k)
        if (shape[k] < 0) return TM_EDT_ERR_INVALID_ARG;
    if (sampling)
        for (int k = 0; k < ndim; ++k)
            if (!(sampling[k] > 0.0) || isinf(sampling[k])) return TM_EDT_ERR_INVALID_ARG;
    pl.ndim = ndim;
    // element counts, guarding against overflow
    const int64_t kMaxElems = (int64_t)1 << 40;
    int64_t V = 1;
    bool empty = shape[0] == 0 || shape[1] == 0;
    for (int k = 0; k < ndim; ++k) {
        if (shape[2 + k] == 0) empty = true;
        if (shape[2 + k] > TM_EDT_MAX_EXTENT) return TM_EDT_ERR_UNSUPPORTED;
    }
    if (empty) { pl.images = 0; pl.V = 0; pl.N = 0; pl.E = 0; pl.ws_bytes = 0; return TM_EDT_OK; }
    for (int k = 0; k < ndim; ++k) {
        V *= shape[2 + k];
        if (V > (int64_t)INT32_MAX) return TM_EDT_ERR_UNSUPPORTED;
    }
    if (shape[0] > kMaxElems || shape[1] > kMaxElems) return TM_EDT_ERR_UNSUPPORTED;
    const int64_t images = shape[0] * shape[1];
    if (images > kMaxElems || images * V > kMaxElems) return TM_EDT_ERR_UNSUPPORTED;
    pl.images = images; pl.V = V; pl.N = images * V;

    pl.unit = true;
    if (sampling)
        for (int k = 0; k < ndim; ++k)
            if (sampling[k] != 1.0) pl.unit = false;

    for (int a = 0; a < ndim; ++a) pl.plane_of_axis[a] = -1;
    int E = 0;
    int64_t inner = 1;
    for (int a = ndim - 1; a >= 0; --a) {
        const int64_t n = shape[2 + a];
        if (n > 1) {
            pl.axis[E] = a; pl.ext[E] = (int)n; pl.inner[E] = inner;
            pl.w[E] = sampling ? sampling[a] : 1.0;
            pl.plane_of_axis[a] = E;
            ++E;
        }
        inner *= n;
    }
    if (E == 0) {  // a single voxel per image: keep the last axis so that one pass runs
        pl.axis[0] = ndim - 1; pl.ext[0] = 1; pl.inner[0] = 1;
        pl.w[0] = sampling ? sampling[ndim - 1] : 1.0;
        pl.plane_of_axis[ndim - 1] = 0;
        E = 1;
    }
    pl.E = E;
    int nmax = 1;
    double sumsq = 0.0;
    for (int p = 0; p < E; ++p) {
        nmax = pl.ext[p] > nmax ? pl.ext[p] : nmax;
        sumsq += (double)(pl.ext[p] - 1) * (double)(pl.ext[p] - 1);
    }
    pl.wide = nmax > 128;
    // float32 envelope arithmetic is exact for unit sampling while every value stays below 2^24 and the
    // interval starts keep a safe margin to the next integer; otherwise switch to float64.  Sampled
    // transforms are float32 throughout (their results are only defined up to rounding).
    pl.use_double = pl.unit && !(sumsq + (double)nmax * nmax < 16777216.0 && nmax <= 512);
    const size_t elem = pl.wide ? 2 : 1;
    pl.plane_bytes = (((size_t)pl.N * elem) + 255) & ~(size_t)255;
    pl.ws_bytes = E > 1 ? 2 * (size_t)(E - 1) * pl.plane_bytes : 0;
    const Switches& sw = switches();
    const bool force = sw.force_generic;
    pl.small = nmax <= 8 && !force;
    pl.fast = !pl.small && nmax <= 128 && E >= 2 && E <= 5 && !force;
    // unit sampling: integer keys (two axes up to extent 1024, three up to 512); other sampling: float heights
    // integer keys (value << sh | row, sh = 9 row bits up to extent 512, else 10): every real key must stay below the
    // "no site" key 2^31 and "no site" plus the largest addend below 2^32
    const double key_scale = nmax > 512 ? 1024.0 : 512.0;
    const bool keys_fit = sumsq * key_scale < 2147483648.0 && (double)(nmax + 4) * (nmax + 4) * key_scale < 2147483648.0;
    pl.wide_keys = !pl.small && !pl.fast && E >= 2 && E <= 4 && nmax <= 1024 && (!pl.unit || keys_fit) &&
                   !force;
    pl.long_lines = !pl.small && !pl.fast && !pl.wide_keys && (E == 2 || E == 3) && nmax <= 8192 &&
                    !force;
    if (pl.wide_keys || pl.long_lines) pl.ws_bytes = wide_layout(pl.N, E, want_idx, pl.long_lines).total;
    if (pl.small) pl.ws_bytes = E > 1 ? 4 * ((((size_t)pl.N * 4) + 255) & ~(size_t)255) : 0;  // 2 value + 2 site buffers
    static const int cand[] = {1, 4, 16, 25, 64, 100, 256, 400, 625, 1024, 2500, 10000};
    if ((pl.wide_keys || pl.long_lines || pl.fast) && !pl.unit && !want_idx && pl.ext[0] % 4 == 0 && !sw.no_scaled) {
        // a scale for the value-carrying kernels (no index output; the longer extents, and the quad kernels of the
        // packed-entry shapes when the narrower search below fails): plain 32-bit values, so the largest value and the
        // largest addend of a scan (a few rows beyond the extent) must stay below 2^31
        for (int S : cand) {
            bool ok = true;
            double total = 0.0, edge = 0.0;
            for (int p = 0; p < E && ok; ++p) {
                const double v = pl.w[p] * pl.w[p] * S, r = nearbyint(v);
                if (r < 1.0 || r > 1048576.0 || fabs(v - r) > 1e-9 * v) { ok = false; break; }
                pl.vsi[p] = (int)r;
                total += r * (double)(pl.ext[p] - 1) * (double)(pl.ext[p] - 1);
                const double e2 = r * (double)(pl.ext[p] + 8) * (double)(pl.ext[p] + 8);
                edge = e2 > edge ? e2 : edge;
            }
            if (ok && total < 2147483648.0 && edge < 2147483648.0) { pl.vscaled = true; pl.vscale = S; break; }
        }
    }
    if (pl.fast && !pl.unit && pl.ext[0] % 4 == 0 && !sw.no_scaled) {
        // sampling given with a few decimals: look for a scale that makes every w^2 an integer and keeps
        // the largest possible value below 2^24 (keys are value << 7 | row in 32 bits)
        for (int S : cand) {
            bool ok = true;
            double total = 0.0, edge = 0.0;
            for (int p = 0; p < E && ok; ++p) {
                const double v = pl.w[p] * pl.w[p] * S, r = nearbyint(v);
                if (r < 1.0 || r > 1048576.0 || fabs(v - r) > 1e-9 * v) { ok = false; break; }
                pl.si[p] = (int)r;
                total += r * (double)(pl.ext[p] - 1) * (double)(pl.ext[p] - 1);
                const double e2 = r * (double)(pl.ext[p] + 4) * (double)(pl.ext[p] + 4);
                edge = e2 > edge ? e2 : edge;
            }
            // total: largest true value; edge: largest addend.  Both below 2^24 keep every real key below the
            // "no site" key 2^31 and every key + addend below 2^32.
            if (ok && total < 16777216.0 && edge < 16777216.0) { pl.scaled = true; pl.scale = S; break; }
        }
    }
    if (pl.fast) {
        auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
        const size_t a = E >= 3 ? up((size_t)pl.N * 4) : 0;  // entries (2 or 4 B) or carried values (up to 4 B)
        const size_t b = E >= 4 ? up((size_t)pl.N * 4) : 0;
        pl.ws_bytes = a + b;
    }
    return TM_EDT_OK;
}

static void fill_epilogue(const Plan& pl, float* dist, int64_t* sq, int64_t* idx, EpilogueParams& ep) {
    memset(&ep, 0, sizeof(ep));
    ep.dist = dist; ep.sq = sq; ep.idx = idx;
    ep.V = pl.V; ep.ndim = pl.ndim; ep.E = pl.E;
    for (int p = 0; p < kMaxDims; ++p) {
        ep.axis[p] = p < pl.E ? pl.axis[p] : 0;
        ep.ext[p] = p < pl.E ? pl.ext[p] : 1;
        ep.w2[p] = p < pl.E ? pl.w[p] * pl.w[p] : 0.0;
    }
    for (int a = 0; a < kMaxDims; ++a) ep.plane_of_axis[a] = a < pl.ndim ? pl.plane_of_axis[a] : -1;
    ep.flat = (pl.flags & TM_EDT_FLAG_FLAT_INDEX) ? 1 : 0;
    ep.idx_planes = ep.flat ? 1 : pl.ndim;
    for (int p = 0; p < kMaxDims; ++p) ep.pstride[p] = p < pl.E ? pl.inner[p] : 0;
}

double out_bytes_per_voxel(const EpilogueParams& ep) {
    return (ep.dist ? 4.0 : 0.0) + (ep.sq ? 8.0 : 0.0) + (ep.idx ? 8.0 * ep.idx_planes : 0.0);
}

template <typename OT>
static cudaError_t launch_pass0(const Plan& pl, const uint8_t* in, void* out, bool final_pass,
                                const EpilogueParams& ep, cudaStream_t st) {
    Pass0Params P;
    P.in = in; P.out = out; P.n = pl.ext[0]; P.lines = pl.N / pl.ext[0]; P.w = pl.w[0];
    prof_mark(st, P.n <= 32 ? "pass0_short" : "pass0_long",
              (double)pl.N * (1.0 + (final_pass ? out_bytes_per_voxel(ep) : (double)sizeof(OT))));
    if (P.n <= 32) {
        const int per_warp = 32 / P.n;
        const int64_t warps = (P.lines + per_warp - 1) / per_warp;
        const int64_t blocks = (warps + 7) / 8;
        if (final_pass) pass0_short_kernel<OT, true><<<(unsigned)blocks, 256, 0, st>>>(P, ep);
        else pass0_short_kernel<OT, false><<<(unsigned)blocks, 256, 0, st>>>(P, ep);
    } else {
        const int nw = (P.n + 31) / 32;
        const size_t smem = (size_t)4 * 3 * nw * sizeof(int);
        const int64_t blocks = (P.lines + 3) / 4;
        if (final_pass) pass0_long_kernel<OT, true><<<(unsigned)blocks, 128, smem, st>>>(P, ep);
        else pass0_long_kernel<OT, false><<<(unsigned)blocks, 128, smem, st>>>(P, ep);
    }
    return cudaGetLastError();
}

template <typename CT, typename OT, int K, bool FINAL>
static cudaError_t launch_axis_k(const AxisParams& P, const EpilogueParams& ep, cudaStream_t st) {
    const int nw = (P.n + 31) / 32;
    const size_t per_thread = (size_t)2 * nw * sizeof(unsigned);
    int threads = 128;
    while (threads > 32 && per_thread * threads > 64 * 1024) threads >>= 1;
    const size_t smem = per_thread * threads;
    auto kern = axis_pass_kernel<CT, OT, K, FINAL>;
    {
        cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
    }
    const int64_t blocks = (P.lines + threads - 1) / threads;
    prof_mark(st, FINAL ? "axis_pass_final" : "axis_pass",
              (double)P.lines * P.n * (K * (double)sizeof(OT) + (FINAL ? out_bytes_per_voxel(ep) : (K + 1.0) * sizeof(OT))));
    kern<<<(unsigned)blocks, threads, smem, st>>>(P, ep);
    return cudaGetLastError();
}

template <typename CT, typename OT, bool FINAL>
static cudaError_t launch_axis(int K, const AxisParams& P, const EpilogueParams& ep, cudaStream_t st) {
    switch (K) {
        case 1: return launch_axis_k<CT, OT, 1, FINAL>(P, ep, st);
        case 2: return launch_axis_k<CT, OT, 2, FINAL>(P, ep, st);
        case 3: return launch_axis_k<CT, OT, 3, FINAL>(P, ep, st);
        case 4: return launch_axis_k<CT, OT, 4, FINAL>(P, ep, st);
        case 5: return launch_axis_k<CT, OT, 5, FINAL>(P, ep, st);
        case 6: return launch_axis_k<CT, OT, 6, FINAL>(P, ep, st);
        case 7: return launch_axis_k<CT, OT, 7, FINAL>(P, ep, st);
    }
    return cudaErrorInvalidValue;
}

template <typename CT, typename OT>
static cudaError_t run_generic(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws,
                               cudaStream_t st, int& launches) {
    cudaError_t e;
    char* bufA = static_cast<char*>(ws);
    char* bufB = bufA + (size_t)(pl.E > 1 ? pl.E - 1 : 0) * pl.plane_bytes;
    e = launch_pass0<OT>(pl, in, bufA, pl.E == 1, ep, st);
    ++launches;
    if (e != cudaSuccess) return e;
    char* src = bufA;
    char* dst = bufB;
    for (int k = 1; k < pl.E; ++k) {
        AxisParams P;
        memset(&P, 0, sizeof(P));
        P.in = src; P.out = dst;
        P.plane_elems = (int64_t)(pl.plane_bytes / sizeof(OT));
        P.n = pl.ext[k]; P.inner = pl.inner[k]; P.lines = pl.N / pl.ext[k];
        P.w2 = pl.w[k] * pl.w[k];
        for (int p = 0; p < k; ++p) P.w2p[p] = pl.w[p] * pl.w[p];
        const bool fin = k == pl.E - 1;
        e = fin ? launch_axis<CT, OT, true>(k, P, ep, st) : launch_axis<CT, OT, false>(k, P, ep, st);
        ++launches;
        if (e != cudaSuccess) return e;
        char* t = src; src = dst; dst = t;
    }
    return cudaSuccess;
}

template <bool UNIT>
static void fill_scan_tab(ScanTab& tab, double w, int shift) {
    for (int d = 0; d < 132; ++d) {
        if (UNIT) tab.add[d] = (uint32_t)(d * d) << shift;
        else { const float f = (float)(w * w) * (float)d * (float)d; memcpy(&tab.add[d], &f, 4); }
    }
}

template <int K, bool FINAL, bool UNIT, int TX>
static cudaError_t launch_column_tx(const FastParams& P, const EpilogueParams& ep, const ScanTab& tab, cudaStream_t st,
                                    double out_bpv) {
    const size_t eb = (size_t)entry_bytes(K);
    const size_t smem = (size_t)P.n * TX * (4 + eb);
    auto kern = column_kernel<K, FINAL, UNIT, TX>;
    {
        cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
    }
    const int tiles = (int)((P.inner + TX - 1) / TX);
    const int64_t blocks = P.outer * tiles;
    const double vox = (double)P.outer * P.n * (double)P.inner;
    prof_mark(st, FINAL ? "column_final" : "column", vox * ((double)eb + (FINAL ? out_bpv : (double)entry_bytes(K + 1))));
    kern<<<(unsigned)blocks, 256, smem, st>>>(P, ep, tab, tiles);
    return cudaGetLastError();
}

template <int K, bool FINAL, bool UNIT>
static cudaError_t launch_column(const FastParams& P, const EpilogueParams& ep, const ScanTab& tab, cudaStream_t st,
                                 double out_bpv) {
    // tile = n rows x (32 * G) columns, about 4096 voxels
    int G = 1;
    while (G < 4 && P.n * 32 * G * 2 <= 4096 && 32 * G < P.inner) G <<= 1;
    if (G == 1) return launch_column_tx<K, FINAL, UNIT, 32>(P, ep, tab, st, out_bpv);
    if (G == 2) return launch_column_tx<K, FINAL, UNIT, 64>(P, ep, tab, st, out_bpv);
    return launch_column_tx<K, FINAL, UNIT, 128>(P, ep, tab, st, out_bpv);
}

template <bool FINAL, bool UNIT>
static cudaError_t launch_column_any(int K, const FastParams& P, const EpilogueParams& ep, const ScanTab& tab,
                                     cudaStream_t st, double out_bpv) {
    switch (K) {
        case 2: return launch_column<2, FINAL, UNIT>(P, ep, tab, st, out_bpv);
        case 3: return launch_column<3, FINAL, UNIT>(P, ep, tab, st, out_bpv);
        case 4: if (FINAL) return launch_column<4, true, UNIT>(P, ep, tab, st, out_bpv);
    }
    return cudaErrorInvalidValue;
}

// A further axis on carried values (no index output requested): see edt_value.cuh.
template <bool FINAL, typename VT, bool SCALED>
static cudaError_t launch_column_value(const FastParams& P, const EpilogueParams& ep, cudaStream_t st, double out_bpv) {
    int G = 1;
    while (G < 4 && P.n * 32 * G * 2 <= 4096 && 32 * G < P.inner) G <<= 1;
    const int TX = 32 * G;
    const size_t smem = (size_t)P.n * TX * 4;
    const int tiles = (int)((P.inner + TX - 1) / TX);
    const int64_t blocks = P.outer * tiles;
    const double vox = (double)P.outer * P.n * (double)P.inner;
    prof_mark(st, FINAL ? "column_value_final" : "column_value", vox * ((double)sizeof(VT) + (FINAL ? out_bpv : (double)sizeof(VT))));
#define TM_LAUNCH_COLUMN_VALUE(TXV)                                                                            \
    do {                                                                                                       \
        auto kern = column_value_kernel<FINAL, VT, SCALED, TXV>;                                               \
        const cudaError_t ea = ensure_smem(reinterpret_cast<const void*>(kern), smem);                           \
        if (ea != cudaSuccess) return ea;                                                                      \
        kern<<<(unsigned)blocks, 256, smem, st>>>(P, ep, tiles);                                               \
    } while (0)
    if (G == 1) TM_LAUNCH_COLUMN_VALUE(32); else if (G == 2) TM_LAUNCH_COLUMN_VALUE(64); else TM_LAUNCH_COLUMN_VALUE(128);
#undef TM_LAUNCH_COLUMN_VALUE
    return cudaGetLastError();
}

// Packed-entry path: fused first + second axis, then one column kernel per further axis.
template <bool UNIT>
static cudaError_t run_fast(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws, cudaStream_t st,
                            int& launches) {
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    char* bufA = static_cast<char*>(ws);
    char* bufB = bufA + (pl.E >= 3 ? up((size_t)pl.N * 4) : 0);
    const double out_bpv = out_bytes_per_voxel(ep);
    auto fill = [&](FastParams& P, int k) {
        memset(&P, 0, sizeof(P));
        P.n = pl.ext[k]; P.inner = pl.inner[k]; P.outer = pl.N / ((int64_t)pl.ext[k] * pl.inner[k]);
        P.w2 = (float)(pl.w[k] * pl.w[k]);
        for (int p = 0; p < k && p < 4; ++p) P.w2p[p] = (float)(pl.w[p] * pl.w[p]);
    };
    FastParams P;
    ScanTab tab;
    fill(P, 1);
    fill_scan_tab<UNIT>(tab, pl.w[1], 8);
    P.in = in; P.out = bufA; P.n0 = pl.ext[0];
    // without an index output the passes carry squared distances instead of offsets (unit sampling, tile plane kernel)
    double sumsq = 0.0;
    for (int p = 0; p < pl.E; ++p) sumsq += (double)(pl.ext[p] - 1) * (pl.ext[p] - 1);
    const Switches& sw = switches();
    const bool vc = UNIT && !ep.idx && pl.E >= 3 && pl.ext[0] % 4 == 0 && ((uintptr_t)in & 3u) == 0 &&
                    !sw.old_plane && !sw.no_value_carry;
    const bool vc16 = vc && sumsq < 65535.0;
    P.value_carry = vc ? (vc16 ? 2 : 4) : 0;
    {
        const int threads = 256;
        const int tstride = (pl.ext[0] + 15) & ~15;
        const size_t smem = (((size_t)pl.ext[1] * tstride + 15) & ~(size_t)15) + (size_t)pl.ext[1] * 32 * 4;
        const bool fin = pl.E == 2;
        prof_mark(st, fin ? "plane_final" : "plane", (double)pl.N * (1.0 + (fin ? out_bpv : (P.value_carry == 4 ? 4.0 : 2.0))));
        if (UNIT && pl.ext[0] % 4 == 0 && ((uintptr_t)in & 3u) == 0 && !sw.old_plane) {
            // whole-plane key tile; row stride = extent rounded up to 32, 64 or 128 columns
            const int vs = pl.ext[0] <= 32 ? 32 : (pl.ext[0] <= 64 ? 64 : 128);
            const size_t smem_u = (size_t)pl.ext[1] * vs * 4;
#define TM_LAUNCH_PLANE_UNIT(FIN, VSV, VCV)                                                                    \
    do {                                                                                                       \
        auto kern = plane_unit_kernel<FIN, VSV, VCV>;                                                          \
        const cudaError_t ea = ensure_smem(reinterpret_cast<const void*>(kern), smem_u);                           \
        if (ea != cudaSuccess) return ea;                                                                      \
        kern<<<(unsigned)P.outer, threads, smem_u, st>>>(P, ep);                                               \
    } while (0)
#define TM_LAUNCH_PLANE_UNIT_VS(FIN, VCV)                                                                      \
    do {                                                                                                       \
        if (vs == 32) TM_LAUNCH_PLANE_UNIT(FIN, 32, VCV); else if (vs == 64) TM_LAUNCH_PLANE_UNIT(FIN, 64, VCV); else TM_LAUNCH_PLANE_UNIT(FIN, 128, VCV); \
    } while (0)
            if (fin && !ep.idx && !sw.no_value_carry) TM_LAUNCH_PLANE_UNIT_VS(true, 4);  // plain values: no site needed
            else if (fin) TM_LAUNCH_PLANE_UNIT_VS(true, 0);
            else if (P.value_carry == 2) TM_LAUNCH_PLANE_UNIT_VS(false, 2);
            else if (P.value_carry == 4) TM_LAUNCH_PLANE_UNIT_VS(false, 4);
            else TM_LAUNCH_PLANE_UNIT_VS(false, 0);
#undef TM_LAUNCH_PLANE_UNIT_VS
#undef TM_LAUNCH_PLANE_UNIT
        } else if (!UNIT && pl.ext[0] % 4 == 0 && ((uintptr_t)in & 3u) == 0 && !sw.old_plane) {
            const int vs = pl.ext[0] <= 32 ? 32 : (pl.ext[0] <= 64 ? 64 : 128);
            const size_t smem_s = (size_t)pl.ext[1] * vs * 5;
#define TM_LAUNCH_PLANE_SAMPLED(FIN, VSV)                                                                      \
    do {                                                                                                       \
        auto kern = plane_sampled_kernel<FIN, VSV>;                                                            \
        const cudaError_t ea = ensure_smem(reinterpret_cast<const void*>(kern), smem_s);                           \
        if (ea != cudaSuccess) return ea;                                                                      \
        kern<<<(unsigned)P.outer, 512, smem_s, st>>>(P, ep, tab);                                              \
    } while (0)
            if (fin) { if (vs == 32) TM_LAUNCH_PLANE_SAMPLED(true, 32); else if (vs == 64) TM_LAUNCH_PLANE_SAMPLED(true, 64); else TM_LAUNCH_PLANE_SAMPLED(true, 128); }
            else { if (vs == 32) TM_LAUNCH_PLANE_SAMPLED(false, 32); else if (vs == 64) TM_LAUNCH_PLANE_SAMPLED(false, 64); else TM_LAUNCH_PLANE_SAMPLED(false, 128); }
#undef TM_LAUNCH_PLANE_SAMPLED
        } else if (fin) plane_kernel<true, UNIT><<<(unsigned)P.outer, threads, smem, st>>>(P, ep, tab);
        else plane_kernel<false, UNIT><<<(unsigned)P.outer, threads, smem, st>>>(P, ep, tab);
        ++launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    char* src = bufA;
    char* dst = bufB;
    for (int k = 2; k < pl.E; ++k) {
        fill(P, k);
        fill_scan_tab<UNIT>(tab, pl.w[k], 8);
        P.in = src; P.out = dst;
        const bool fin = k == pl.E - 1;
        cudaError_t e;
        if (vc16) e = fin ? launch_column_value<true, uint16_t, false>(P, ep, st, out_bpv) : launch_column_value<false, uint16_t, false>(P, ep, st, out_bpv);
        else if (vc) e = fin ? launch_column_value<true, uint32_t, false>(P, ep, st, out_bpv) : launch_column_value<false, uint32_t, false>(P, ep, st, out_bpv);
        else e = fin ? launch_column_any<true, UNIT>(k, P, ep, tab, st, out_bpv)
                     : launch_column_any<false, UNIT>(k, P, ep, tab, st, out_bpv);
        ++launches;
        if (e != cudaSuccess) return e;
        char* t = src; src = dst; dst = t;
    }
    return cudaSuccess;
}

template <int K, bool FINAL>
static cudaError_t launch_column_scaled(const FastParams& P, const EpilogueParams& ep, cudaStream_t st, double out_bpv) {
    const size_t eb = (size_t)entry_bytes(K);
    int G = 1;
    while (G < 4 && P.n * 32 * G * 2 <= 4096 && 32 * G < P.inner) G <<= 1;
    const int TX = 32 * G;
    const size_t smem = (size_t)P.n * TX * (4 + eb);
    const int tiles = (int)((P.inner + TX - 1) / TX);
    const int64_t blocks = P.outer * tiles;
    const double vox = (double)P.outer * P.n * (double)P.inner;
    prof_mark(st, FINAL ? "column_scaled_final" : "column_scaled",
              vox * ((double)eb + (FINAL ? out_bpv : (double)entry_bytes(K + 1))));
#define TM_LAUNCH_COLUMN_SCALED(TXV)                                                                           \
    do {                                                                                                       \
        auto kern = column_scaled_kernel<K, FINAL, TXV>;                                                       \
        const cudaError_t ea = ensure_smem(reinterpret_cast<const void*>(kern), smem);                           \
        if (ea != cudaSuccess) return ea;                                                                      \
        kern<<<(unsigned)blocks, 256, smem, st>>>(P, ep, tiles);                                               \
    } while (0)
    if (G == 1) TM_LAUNCH_COLUMN_SCALED(32); else if (G == 2) TM_LAUNCH_COLUMN_SCALED(64); else TM_LAUNCH_COLUMN_SCALED(128);
#undef TM_LAUNCH_COLUMN_SCALED
    return cudaGetLastError();
}

// Packed-entry path in scaled integers (see edt_fast.cuh): fused plane kernel, then column kernels.
static cudaError_t run_scaled(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws, cudaStream_t st,
                              int& launches) {
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    char* bufA = static_cast<char*>(ws);
    char* bufB = bufA + (pl.E >= 3 ? up((size_t)pl.N * 4) : 0);
    const double out_bpv = out_bytes_per_voxel(ep);
    auto fill = [&](FastParams& P, int k) {
        memset(&P, 0, sizeof(P));
        P.n = pl.ext[k]; P.inner = pl.inner[k]; P.outer = pl.N / ((int64_t)pl.ext[k] * pl.inner[k]);
        for (int p = 0; p < k && p < 4; ++p) P.si[p] = pl.si[p];
        P.sk = pl.si[k];
        P.inv_scale = (float)(1.0 / pl.scale);
    };
    FastParams P;
    fill(P, 1);
    P.in = in; P.out = bufA; P.n0 = pl.ext[0];
    // without an index output the passes carry the scaled squared distance (32 bits) instead of offsets
    const Switches& sw = switches();
    const bool vc = !ep.idx && pl.E >= 3 && !sw.no_value_carry;
    P.value_carry = vc ? 4 : 0;
    {
        const bool fin = pl.E == 2;
        const int vs = pl.ext[0] <= 32 ? 32 : (pl.ext[0] <= 64 ? 64 : 128);
        const bool plain_fin = fin && !ep.idx && ep.dist && !sw.no_value_carry;
        const size_t smem = (size_t)pl.ext[1] * vs * (((vc && !fin) || plain_fin) ? 4 : 5);  // keys, plus a byte tile of first-axis offsets
        prof_mark(st, fin ? "plane_scaled_final" : "plane_scaled", (double)pl.N * (1.0 + (fin ? out_bpv : (vc ? 4.0 : 2.0))));
#define TM_LAUNCH_PLANE_SCALED(FIN, VSV, VCV)                                                                  \
    do {                                                                                                       \
        auto kern = plane_scaled_kernel<FIN, VSV, VCV>;                                                        \
        const cudaError_t ea = ensure_smem(reinterpret_cast<const void*>(kern), smem);                           \
        if (ea != cudaSuccess) return ea;                                                                      \
        kern<<<(unsigned)P.outer, 512, smem, st>>>(P, ep);                                                     \
    } while (0)
        if (plain_fin) { if (vs == 32) TM_LAUNCH_PLANE_SCALED(true, 32, true); else if (vs == 64) TM_LAUNCH_PLANE_SCALED(true, 64, true); else TM_LAUNCH_PLANE_SCALED(true, 128, true); }
        else if (fin) { if (vs == 32) TM_LAUNCH_PLANE_SCALED(true, 32, false); else if (vs == 64) TM_LAUNCH_PLANE_SCALED(true, 64, false); else TM_LAUNCH_PLANE_SCALED(true, 128, false); }
        else if (vc) { if (vs == 32) TM_LAUNCH_PLANE_SCALED(false, 32, true); else if (vs == 64) TM_LAUNCH_PLANE_SCALED(false, 64, true); else TM_LAUNCH_PLANE_SCALED(false, 128, true); }
        else { if (vs == 32) TM_LAUNCH_PLANE_SCALED(false, 32, false); else if (vs == 64) TM_LAUNCH_PLANE_SCALED(false, 64, false); else TM_LAUNCH_PLANE_SCALED(false, 128, false); }
#undef TM_LAUNCH_PLANE_SCALED
        ++launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    char* src = bufA;
    char* dst = bufB;
    for (int k = 2; k < pl.E; ++k) {
        fill(P, k);
        P.in = src; P.out = dst;
        const bool fin = k == pl.E - 1;
        cudaError_t e = cudaErrorInvalidValue;
        if (vc) {
            e = fin ? launch_column_value<true, uint32_t, true>(P, ep, st, out_bpv)
                    : launch_column_value<false, uint32_t, true>(P, ep, st, out_bpv);
        } else if (fin) {
            if (k == 2) e = launch_column_scaled<2, true>(P, ep, st, out_bpv);
            else if (k == 3) e = launch_column_scaled<3, true>(P, ep, st, out_bpv);
            else if (k == 4) e = launch_column_scaled<4, true>(P, ep, st, out_bpv);
        } else {
            if (k == 2) e = launch_column_scaled<2, false>(P, ep, st, out_bpv);
            else if (k == 3) e = launch_column_scaled<3, false>(P, ep, st, out_bpv);
        }
        ++launches;
        if (e != cudaSuccess) return e;
        char* t = src; src = dst; dst = t;
    }
    return cudaSuccess;
}

// Every extent <= 8: consecutive axes grouped while the product of their extents stays <= 256, one kernel
// per group, squared distances (and site indices) carried between kernels as plain arrays.
template <bool SITE>
static cudaError_t run_small(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws, cudaStream_t st,
                             int& launches) {
    const size_t buf = (((size_t)pl.N * 4) + 255) & ~(size_t)255;
    char* w = static_cast<char*>(ws);
    float* val[2] = {reinterpret_cast<float*>(w), reinterpret_cast<float*>(w + buf)};
    int32_t* site[2] = {reinterpret_cast<int32_t*>(w + 2 * buf), reinterpret_cast<int32_t*>(w + 3 * buf)};
    const double out_bpv = out_bytes_per_voxel(ep);
    int g = 0;
    for (int k = 0; k < pl.E; ++g) {
        SmallParams P;
        memset(&P, 0, sizeof(P));
        P.prod = 1;
        const int k0 = k;
        while (k < pl.E && (k == k0 || P.prod * pl.ext[k] <= kSmallProd)) {
            P.n[P.m] = pl.ext[k];
            P.w2[P.m] = (float)(pl.w[k] * pl.w[k]);
            P.prod *= pl.ext[k];
            ++P.m; ++k;
        }
        const bool first = k0 == 0, fin = k == pl.E;
        const size_t smem = (size_t)P.prod * kSmallT * (SITE ? 8 : 4);
        P.mask = in;
        P.in_val = val[(g + 1) & 1]; P.in_site = site[(g + 1) & 1];
        P.out_val = val[g & 1]; P.out_site = site[g & 1];
        P.inner = pl.inner[k0]; P.outer = pl.N / (P.inner * P.prod);
        P.V = pl.V;
        const double carry = SITE ? 8.0 : 4.0;
        prof_mark(st, fin ? "small_group_final" : first ? "small_group_first" : "small_group",
                  (double)pl.N * ((first ? 1.0 : carry) + (fin ? out_bpv : carry)));
        const int64_t tiles = P.inner == 1 ? (P.outer + kSmallT - 1) / kSmallT
                                           : P.outer * ((P.inner + kSmallT - 1) / kSmallT);
        const unsigned blocks = (unsigned)tiles;
#define TM_SMALL_LAUNCH3(FIRST, FIN, NM)                                                                         \
    do {                                                                                                         \
        auto kern = small_group_kernel<SITE, FIRST, FIN, NM>;                                                    \
        const cudaError_t ea = ensure_smem(reinterpret_cast<const void*>(kern), smem);                           \
        if (ea != cudaSuccess) return ea;                                                                      \
        kern<<<blocks, threads, smem, st>>>(P, ep);                                                        \
    } while (0)
#define TM_SMALL_LAUNCH(FIRST, FIN)                                                                              \
    do {                                                                                                         \
        if (nm <= 4) TM_SMALL_LAUNCH3(FIRST, FIN, 4);                                                            \
        else if (nm <= 6) TM_SMALL_LAUNCH3(FIRST, FIN, 6);                                                       \
        else TM_SMALL_LAUNCH3(FIRST, FIN, 8);                                                                    \
    } while (0)
        int nm = 0, nmin = 8;
        for (int q = 0; q < P.m; ++q) { nm = std::max(nm, P.n[q]); nmin = std::min(nmin, P.n[q]); }
        // one thread per line of the axis with the most lines, within [128, 512]
        const int max_lines = P.prod / nmin * kSmallT;
        const unsigned threads = (unsigned)std::min(kSmallThreads, std::max(128, (max_lines + 31) / 32 * 32));
        if (first && fin) TM_SMALL_LAUNCH(true, true);
        else if (first) TM_SMALL_LAUNCH(true, false);
        else if (fin) TM_SMALL_LAUNCH(false, true);
        else TM_SMALL_LAUNCH(false, false);
#undef TM_SMALL_LAUNCH3
#undef TM_SMALL_LAUNCH
        ++launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Unit sampling beyond extent 128 (two axes up to 1024, three up to 512): key rows, then strip scans.
// sh: row bits of the integer keys (9 or 10), or -1 for float heights
template <int K, bool FINAL, int CW>
static cudaError_t launch_wide_axis_cw(const WideAxisParams& A, const EpilogueParams& ep, int sh, cudaStream_t st) {
    const int strips = (int)((A.inner + CW - 1) / CW);
    const size_t smem = (size_t)A.n * CW * 4;
    auto kern = sh < 0 ? wide_axis_kernel<K, FINAL, -1, CW>
                       : (sh == 0 ? wide_axis_kernel<K, FINAL, 0, CW>
                                  : (sh == 10 ? wide_axis_kernel<K, FINAL, 10, CW> : wide_axis_kernel<K, FINAL, 9, CW>));
    {
        cudaError_t e = ensure_smem(reinterpret_cast<const void*>(kern), smem);
        if (e != cudaSuccess) return e;
    }
    // few strips (a single large image): several blocks share a strip, each taking a range of its rows, until
    // there are about two blocks per SM
    WideAxisParams B = A;
    const int64_t base_blocks = A.outer * strips;
    B.row_parts = (int)std::max<int64_t>(1, std::min<int64_t>(std::min(8, A.n / 64), 296 / base_blocks));
    // 16 warps per strip from 384 rows on (8 for the narrow strips): a strip's rows are independent work
    const int threads = A.n >= 384 ? (CW == 32 ? 512 : 256) : 256;
    kern<<<(unsigned)(base_blocks * B.row_parts), threads, smem, st>>>(B, ep, strips);
    return cudaGetLastError();
}

// sh: row bits of the integer keys (9 or 10), 0 for plain values, or -1 for float heights
template <int K, bool FINAL>
static cudaError_t launch_wide_axis(const WideAxisParams& A, const EpilogueParams& ep, int sh, cudaStream_t st) {
    // long axes: strips of 16 columns (half the shared memory per block, so more blocks are resident and the
    // grid divides more evenly over the SMs)
    const int cw = A.n > 256 && A.inner >= 32 ? 16 : 32;
    return cw == 16 ? launch_wide_axis_cw<K, FINAL, 16>(A, ep, sh, st) : launch_wide_axis_cw<K, FINAL, 32>(A, ep, sh, st);
}

static cudaError_t run_wide(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws, cudaStream_t st,
                              int& launches) {
    char* w = static_cast<char*>(ws);
    const WideLayout L = wide_layout(pl.N, pl.E, ep.idx != nullptr, false);
    uint32_t* keysA = reinterpret_cast<uint32_t*>(w + L.keysA);
    int16_t* offsA = reinterpret_cast<int16_t*>(w + L.offsA);
    uint32_t* keysB = reinterpret_cast<uint32_t*>(w + L.keysB);
    int16_t* offsB = reinterpret_cast<int16_t*>(w + L.offsB);
    const bool carry = ep.idx != nullptr;  // offsets are carried only for the index output
    WideParams P;
    P.in = in; P.keys = keysA; P.offs = carry ? offsA : nullptr;
    P.n0 = pl.ext[0]; P.n1 = pl.ext[1];
    P.rows = pl.N / pl.ext[0];
    P.w2x = (float)(pl.w[0] * pl.w[0]);
    P.w0i = 1u;  // (set below for scaled sampling)
    const double out_bpv = out_bytes_per_voxel(ep);
    // integer keys carry 9 row bits up to extent 512 and 10 up to 1024 (two axes only); general sampling uses float
    // heights.  A lane of the row kernel takes 16 voxels (rows up to 512) or 32.
    int nmax = 1;
    for (int p = 0; p < pl.E; ++p) nmax = pl.ext[p] > nmax ? pl.ext[p] : nmax;
    // without an index output no site is needed afterwards: plain values as keys (sh = 0)
    // sampling whose squares share an integer scale, distances only: the value kernels run in exact scaled integers if
    // every axis pass fits them (the first pass hands them 16-bit row distances or weighted integer values)
    const bool vs = !pl.unit && pl.vscaled && !carry && !switches().no_lean && lean_value_all_axes_ok(pl, ep);
    const int sh = vs ? 0 : (!pl.unit ? -1 : (!carry ? 0 : (nmax > 512 ? 10 : 9)));
    if (vs) P.w0i = (uint32_t)pl.vsi[0];
    // no index output, unit sampling: the first pass hands 16-bit row distances to the quad value kernel of the second axis
    const bool dist16 = sh == 0 && pl.ext[0] % 32 == 0 && pl.ext[0] <= 1024 && ((uintptr_t)in & 31u) == 0 &&
                        !switches().no_lean && lean_value_axis_ok(pl, 1, ep);
    prof_mark(st, "row_keys", (double)pl.N * (1.0 + (dist16 ? 2.0 : 4.0) + (carry ? 2.0 : 0.0)));
    const unsigned row_blocks = (unsigned)((P.rows + 7) / 8);
    if (dist16) {
        cudaError_t e16 = launch_row_dist16(in, reinterpret_cast<uint16_t*>(keysA), P.rows, pl.ext[0], st);
        if (e16 != cudaSuccess) return e16;
    } else if (pl.ext[0] % 16 != 0 || ((uintptr_t)in & 15u) != 0) {
        // rows that are not 16-byte aligned: one voxel per lane, ballot words
        if (sh < 0) long_row_any_kernel<-1><<<row_blocks, 256, 0, st>>>(P);
        else if (sh == 0) long_row_any_kernel<0><<<row_blocks, 256, 0, st>>>(P);
        else if (sh == 9) long_row_any_kernel<9><<<row_blocks, 256, 0, st>>>(P);
        else long_row_any_kernel<10><<<row_blocks, 256, 0, st>>>(P);
    } else if (pl.ext[0] <= 512) {
        if (sh < 0) row_keys_kernel<16, -1><<<row_blocks, 256, 0, st>>>(P);
        else if (sh == 0) row_keys_kernel<16, 0><<<row_blocks, 256, 0, st>>>(P);
        else if (sh == 9) row_keys_kernel<16, 9><<<row_blocks, 256, 0, st>>>(P);
        else row_keys_kernel<16, 10><<<row_blocks, 256, 0, st>>>(P);
    } else {
        if (sh < 0) row_keys_kernel<32, -1><<<row_blocks, 256, 0, st>>>(P);
        else if (sh == 0) row_keys_kernel<32, 0><<<row_blocks, 256, 0, st>>>(P);
        else row_keys_kernel<32, 10><<<row_blocks, 256, 0, st>>>(P);
    }
    ++launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    int16_t* offsC = reinterpret_cast<int16_t*>(w + L.offsC);
    WideAxisParams A;
    memset(&A, 0, sizeof(A));
    A.n0 = pl.ext[0]; A.n1 = pl.ext[1];
    // axis k reads what axis k - 1 wrote: keys ping-pong between the two key buffers, offsets grow by one per axis
    const uint32_t* keys_in[4] = {nullptr, keysA, keysB, keysA};
    uint32_t* keys_out[4] = {nullptr, keysB, keysA, nullptr};
    const int16_t* offs_in[4] = {nullptr, offsA, offsB, offsC};
    int16_t* offs_out[4] = {nullptr, offsB, offsC, nullptr};
    for (int k = 1; k < pl.E; ++k) {
        const bool fin = k == pl.E - 1;
        A.keys_in = keys_in[k]; A.offs_in = offs_in[k];
        A.keys_out = fin ? nullptr : keys_out[k]; A.offs_out = (fin || !carry) ? nullptr : offs_out[k];
        A.n = pl.ext[k]; A.inner = pl.inner[k]; A.outer = pl.N / ((int64_t)pl.ext[k] * pl.inner[k]);
        A.next_n = fin ? 0 : pl.ext[k + 1];
        A.w2 = (float)(pl.w[k] * pl.w[k]);
        const double offs_b = k == 3 ? 8.0 : 2.0 * k;  // bytes of offsets per voxel read by this axis
        if (fin) prof_mark(st, "wide_axis_final", (double)pl.N * ((dist16 && k == 1 ? 2.0 : 4.0) + out_bpv + (ep.idx ? offs_b : 0.0)));
        else prof_mark(st, "wide_axis", (double)pl.N * ((dist16 && k == 1 ? 2.0 : 4.0) + 4.0 + (carry ? offs_b + (k == 2 ? 8.0 : 4.0) : 0.0)));
        if (dist16 && k == 1) e = run_lean_value_axis(pl, 1, keysA, fin ? nullptr : keys_out[1], ep, fin, st, true);
        else if (sh == 0 && !switches().no_lean && lean_value_axis_ok(pl, k, ep))
            e = run_lean_value_axis(pl, k, keys_in[k], fin ? nullptr : keys_out[k], ep, fin, st);
        else if (k == 1) e = fin ? launch_wide_axis<1, true>(A, ep, sh, st) : launch_wide_axis<1, false>(A, ep, sh, st);
        else if (k == 2) e = fin ? launch_wide_axis<2, true>(A, ep, sh, st) : launch_wide_axis<2, false>(A, ep, sh, st);
        else e = launch_wide_axis<3, true>(A, ep, sh, st);
        ++launches;
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Two or three axes with extents up to 8192: heights and 16-bit offsets per voxel, scans through the cache.
template <bool FLT>
static cudaError_t run_long(const Plan& pl, const uint8_t* in, const EpilogueParams& ep, void* ws, cudaStream_t st,
                            int& launches) {
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    char* w = static_cast<char*>(ws);
    const WideLayout L = wide_layout(pl.N, pl.E, ep.idx != nullptr, true);
    uint32_t* hA = reinterpret_cast<uint32_t*>(w + L.keysA);
    int16_t* offsA = reinterpret_cast<int16_t*>(w + L.offsA);
    uint32_t* hB = reinterpret_cast<uint32_t*>(w + L.keysB);
    int16_t* offsB = reinterpret_cast<int16_t*>(w + L.offsB);
    uint32_t* blockmin = reinterpret_cast<uint32_t*>(w + L.bm);
    WideParams P;
    const bool carry = ep.idx != nullptr;  // offsets are carried only for the index output
    P.in = in; P.keys = hA; P.offs = carry ? offsA : nullptr;
    P.n0 = pl.ext[0]; P.n1 = pl.ext[1];
    P.rows = pl.N / pl.ext[0];
    P.w2x = (float)(pl.w[0] * pl.w[0]);
    P.w0i = pl.unit ? 1u : (uint32_t)pl.vsi[0];  // (integer heights under sampling: the scaled-integer value passes)
    const double out_bpv = out_bytes_per_voxel(ep);
    prof_mark(st, "long_row", (double)pl.N * (1.0 + 4.0 + (carry ? 2.0 : 0.0)));
    if (pl.ext[0] % 16 == 0 && ((uintptr_t)in & 15u) == 0) long_row_kernel<FLT><<<(unsigned)((P.rows + 7) / 8), 256, 0, st>>>(P);
    else long_row_any_kernel<FLT ? -1 : -2><<<(unsigned)((P.rows + 7) / 8), 256, 0, st>>>(P);
    ++launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    LongAxisParams A;
    memset(&A, 0, sizeof(A));
    auto set_axis = [&](int k) {
        A.n = pl.ext[k]; A.inner = pl.inner[k]; A.outer = pl.N / ((int64_t)pl.ext[k] * pl.inner[k]);
        A.n0 = pl.ext[0];
        A.w2 = (float)(pl.w[k] * pl.w[k]);
        A.strips_per_slab = (int)((A.inner + 31) / 32);
        A.row_blocks = (A.n + kLongRows - 1) / kLongRows;
        A.blockmin = A.n > 128 ? blockmin : nullptr;  // short axes: the row-by-row phase covers the column
        return (unsigned)(A.outer * A.strips_per_slab * A.row_blocks);
    };
    // block minima of the heights the next axis pass reads
    auto block_minima = [&]() -> cudaError_t {
        if (!A.blockmin) return cudaSuccess;
        const int64_t items = A.outer * ((A.n + 31) / 32) * A.inner;
        prof_mark(st, "long_blockmin", (double)pl.N * 4.0);
        long_blockmin_kernel<<<(unsigned)((items + 255) / 256), 256, 0, st>>>(A);
        ++launches;
        return cudaGetLastError();
    };
    // unit sampling without index output: every axis still fits a shared-memory tile (32 columns wide up to 1024
    // rows, 16, 8 or 4 beyond), and the quad value kernel takes the pass instead of the scans through the cache
    auto tile_axis = [&](int k) {
        if (FLT || carry || switches().no_lean) return 0;
        return lean_value_axis_ok(pl, k, ep) ? 1 : (lean_value_long_axis_ok(pl, k, ep) ? 2 : 0);
    };
    auto run_tile_axis = [&](int k, const void* src, void* dst, bool fin) -> cudaError_t {
        prof_mark(st, fin ? "long_tile_final" : "long_tile", (double)pl.N * (4.0 + (fin ? out_bpv : 4.0)));
        ++launches;
        return tile_axis(k) == 1 ? run_lean_value_axis(pl, k, src, dst, ep, fin, st) : run_lean_value_long_axis(pl, k, src, dst, ep, fin, st);
    };
    {
        const bool fin = pl.E == 2;
        if (tile_axis(1)) {
            e = run_tile_axis(1, hA, fin ? nullptr : hB, fin);
        } else {
            A.h_in = hA; A.offs_in = offsA; A.h_out = hB; A.offs_out = carry ? offsB : nullptr;
            const unsigned blocks = set_axis(1);
            e = block_minima();
            if (e != cudaSuccess) return e;
            if (fin) {
                prof_mark(st, "long_axis_final", (double)pl.N * (4.0 + out_bpv + (ep.idx ? 2.0 : 0.0)));
                long_axis_kernel<1, true, FLT><<<blocks, 256, 0, st>>>(A, ep);
            } else {
                prof_mark(st, "long_axis", (double)pl.N * (4.0 + 4.0 + (carry ? 2.0 + 4.0 : 0.0)));
                long_axis_kernel<1, false, FLT><<<blocks, 256, 0, st>>>(A, ep);
            }
            ++launches;
            e = cudaGetLastError();
        }
        if (e != cudaSuccess || fin) return e;
    }
    if (tile_axis(2)) return run_tile_axis(2, hB, nullptr, true);
    A.h_in = hB; A.offs_in = offsB; A.h_out = nullptr; A.offs_out = nullptr;
    const unsigned blocks = set_axis(2);
    e = block_minima();
    if (e != cudaSuccess) return e;
    prof_mark(st, "long_axis_final", (double)pl.N * (4.0 + out_bpv + (ep.idx ? 4.0 : 0.0)));
    long_axis_kernel<2, true, FLT><<<blocks, 256, 0, st>>>(A, ep);
    ++launches;
    return cudaGetLastError();
}

// Stream-ordered scratch of tm_edt and tm_edt_host comes from a memory pool of the library's own, one per
// device, created on first use.  Its release threshold is unlimited, so the memory of one call is reused by
// the next instead of going back to the driver at every synchronisation; tm_edt_trim_memory() returns it.
static cudaMemPool_t g_pool[64];
static bool g_pool_ready[64];
static std::mutex g_pool_mutex;

static cudaError_t scratch_alloc(void** p, size_t bytes, cudaStream_t st) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaMallocAsync(p, bytes, st);
    {
        std::lock_guard<std::mutex> lock(g_pool_mutex);
        if (!g_pool_ready[dev]) {
            cudaMemPoolProps props;
            memset(&props, 0, sizeof(props));
            props.allocType = cudaMemAllocationTypePinned;
            props.handleTypes = cudaMemHandleTypeNone;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            e = cudaMemPoolCreate(&g_pool[dev], &props);
            if (e != cudaSuccess) return e;
            uint64_t keep = UINT64_MAX;
            cudaMemPoolSetAttribute(g_pool[dev], cudaMemPoolAttrReleaseThreshold, &keep);
            g_pool_ready[dev] = true;
        }
    }
    return cudaMallocFromPoolAsync(p, bytes, g_pool[dev], st);
}

static bool is_device_ptr(const void* p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return false; }
    int dev = 0;
    cudaGetDevice(&dev);
    if (at.type == cudaMemoryTypeManaged) return true;
    return at.type == cudaMemoryTypeDevice && at.device == dev;
}

static bool is_host_ptr(const void* p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return true; }
    return at.type != cudaMemoryTypeDevice;
}

static bool overlap(const void* a, size_t na, const void* b, size_t nb) {
    if (!a || !b || na == 0 || nb == 0) return false;
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + nb && b0 < a0 + na;
}

cudaError_t shared_scratch_alloc(void** p, size_t bytes, cudaStream_t st) { return scratch_alloc(p, bytes, st); }
bool shared_is_device_ptr(const void* p) { return is_device_ptr(p); }
bool shared_overlap(const void* a, size_t na, const void* b, size_t nb) { return overlap(a, na, b, nb); }
void shared_record(int cuda_error, int launches) {
    if (cuda_error >= 0) g_last_cuda_error = cuda_error;
    g_last_launches = launches;
}

// Argument checks common to every entry point (no CUDA work).
static int check_call(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
                      int64_t* out_sq, int64_t* out_idx, Plan& pl, unsigned flags = 0) {
    if (!input) return TM_EDT_ERR_INVALID_ARG;
    if (flags & ~(unsigned)(TM_EDT_FLAG_VIRTUAL_BACKGROUND | TM_EDT_FLAG_FLAT_INDEX | TM_EDT_FLAG_DIST_F64))
        return TM_EDT_ERR_INVALID_ARG;
    // the float64 variant obtains the site of every voxel first, so it plans like a call with index output
    const bool want_idx = out_idx != nullptr || ((flags & TM_EDT_FLAG_DIST_F64) && out_dist != nullptr);
    const int rc = make_plan(ndim, shape, sampling, pl, want_idx);
    if (rc != TM_EDT_OK) return rc;
    pl.flags = flags;
    for (int a = 0; a < ndim; ++a) { pl.shape_sp[a] = shape[2 + a]; pl.w_sp[a] = sampling ? sampling[a] : 1.0; }
    if (!out_dist && !out_sq && !out_idx) return TM_EDT_ERR_INVALID_ARG;
    const bool f64 = (flags & TM_EDT_FLAG_DIST_F64) != 0;
    if (((uintptr_t)out_dist & (f64 ? 7u : 3u)) || ((uintptr_t)out_sq & 7u) || ((uintptr_t)out_idx & 7u)) return TM_EDT_ERR_INVALID_ARG;
    if (out_sq && !pl.unit) return TM_EDT_ERR_UNSUPPORTED;
    const size_t N = (size_t)pl.N;
    const size_t bi = N, bd = N * (f64 ? 8 : 4), bs = N * 8, bx = N * 8 * (size_t)((flags & TM_EDT_FLAG_FLAT_INDEX) ? 1 : ndim);
    if (overlap(input, bi, out_dist, bd) || overlap(input, bi, out_sq, bs) || overlap(input, bi, out_idx, bx) ||
        overlap(out_dist, bd, out_sq, bs) || overlap(out_dist, bd, out_idx, bx) || overlap(out_sq, bs, out_idx, bx))
        return TM_EDT_ERR_INVALID_ARG;
    return TM_EDT_OK;
}

static cudaError_t run_images(const Plan& pl, const uint8_t* input, float* out_dist, int64_t* out_sq, int64_t* out_idx,
                              void* ws, cudaStream_t st, int& launches) {
    EpilogueParams ep;
    fill_epilogue(pl, out_dist, out_sq, out_idx, ep);
    if (pl.small) return ep.idx ? run_small<true>(pl, input, ep, ws, st, launches) : run_small<false>(pl, input, ep, ws, st, launches);
    if (pl.wide_keys) return run_wide(pl, input, ep, ws, st, launches);
    if (pl.long_lines) {
        // sampling with an integer scale, distances only, every axis pass on the value kernels: integer heights too
        const bool ints = pl.unit || (pl.vscaled && !ep.idx && !switches().no_lean && lean_value_all_axes_ok(pl, ep));
        return ints ? run_long<false>(pl, input, ep, ws, st, launches) : run_long<true>(pl, input, ep, ws, st, launches);
    }
    if (!switches().no_lean && lean_ok(pl, input, ep)) return run_lean(pl, input, ep, ws, st, launches);
    if (pl.fast && pl.scaled && ((uintptr_t)input & 3u) == 0) return run_scaled(pl, input, ep, ws, st, launches);
    if (pl.fast)
        return pl.unit ? run_fast<true>(pl, input, ep, ws, st, launches) : run_fast<false>(pl, input, ep, ws, st, launches);
    if (pl.use_double)
        return pl.wide ? run_generic<double, int16_t>(pl, input, ep, ws, st, launches)
                       : run_generic<double, int8_t>(pl, input, ep, ws, st, launches);
    return pl.wide ? run_generic<float, int16_t>(pl, input, ep, ws, st, launches)
                   : run_generic<float, int8_t>(pl, input, ep, ws, st, launches);
}

// Images are independent, so a batch too large for one grid (no kernel uses more than one block per
// voxel; a grid holds 2^31 - 1 blocks) is run as consecutive image ranges on the same stream and scratch.
static int run_device(const Plan& pl, const uint8_t* input, float* out_dist, int64_t* out_sq, int64_t* out_idx,
                      void* ws, cudaStream_t st) {
    int64_t max_voxels = INT32_MAX;
    const long long lim = switches().chunk_voxels;  // test hook: smaller image ranges
    if (lim > 0 && lim < max_voxels) max_voxels = lim;
    const int64_t max_images = std::max<int64_t>(1, max_voxels / pl.V);
    int launches = 0;
    for (int64_t first = 0; first < pl.images; first += max_images) {
        Plan sub = pl;
        sub.images = std::min<int64_t>(max_images, pl.images - first);
        sub.N = sub.images * pl.V;
        sub.plane_bytes = (((size_t)sub.N * (pl.wide ? 2 : 1)) + 255) & ~(size_t)255;
        const int64_t v0 = first * pl.V;
        cudaError_t e = run_images(sub, input + v0, out_dist ? out_dist + v0 : nullptr, out_sq ? out_sq + v0 : nullptr,
                                   out_idx ? out_idx + v0 * ((pl.flags & TM_EDT_FLAG_FLAT_INDEX) ? 1 : pl.ndim) : nullptr, ws, st,
                                   launches);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return TM_EDT_ERR_CUDA; }
    }
    if (pl.flags & TM_EDT_FLAG_VIRTUAL_BACKGROUND) {
        // images the transform marked as having no background get the virtual-background values
        VirtualParams VP;
        memset(&VP, 0, sizeof(VP));
        VP.images = pl.images; VP.V = pl.V; VP.ndim = pl.ndim;
        for (int a = 0; a < pl.ndim; ++a) { VP.shape[a] = pl.shape_sp[a]; VP.w[a] = pl.w_sp[a]; }
        VP.stride0 = pl.V / pl.shape_sp[0];
        EpilogueParams ep;
        fill_epilogue(pl, out_dist, out_sq, out_idx, ep);
        const int64_t cpi = (pl.V + kVirtualChunk - 1) / kVirtualChunk;
        if (pl.images * cpi > (int64_t)INT32_MAX) return TM_EDT_ERR_UNSUPPORTED;
        prof_mark(st, "virtual_background", 0.0);
        virtual_background_kernel<<<(unsigned)(pl.images * cpi), 256, 0, st>>>(VP, ep, (unsigned)cpi);
        virtual_background_first_kernel<<<(unsigned)((pl.images + 255) / 256), 256, 0, st>>>(VP, ep);
        launches += 2;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return TM_EDT_ERR_CUDA; }
    }
    g_last_launches = launches;
#ifdef TM_EDT_DEBUG
    {   // debug build: wait for the call and turn a recorded bounds violation into a status
        DebugRecord rec = {0ull, 0, 0, 0};
        cudaError_t e = lean_debug_collect(st, &rec);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return TM_EDT_ERR_CUDA; }
        g_last_debug = rec;
        if (rec.count != 0ull) return TM_EDT_ERR_DEBUG_CHECK;
    }
#endif
    return TM_EDT_OK;
}

}  // namespace tmedt

using namespace tmedt;

extern "C" {

// Largest scratch any call on this shape can need with / without index output: the planner may pick different kernel
// families for unit and for other sampling, so both plans are made and the larger one reported.
static size_t worst_case_workspace(int ndim, const int64_t* shape, bool want_idx) {
    Plan unit_plan, sampled_plan;
    double other[kMaxDims];
    for (int k = 0; k < kMaxDims; ++k) other[k] = 1.37;
    if (make_plan(ndim, shape, nullptr, unit_plan, want_idx) != TM_EDT_OK) return (size_t)-1;
    if (make_plan(ndim, shape, other, sampled_plan, want_idx) != TM_EDT_OK) return (size_t)-1;
    return std::max(unit_plan.ws_bytes, sampled_plan.ws_bytes);
}

size_t tm_edt_workspace_bytes(int ndim, const int64_t* shape) { return worst_case_workspace(ndim, shape, true); }

size_t tm_edt_workspace_bytes_for(int ndim, const int64_t* shape, const double* sampling, int want_dist, int want_sqdist,
                                  int want_indices) {
    (void)want_dist; (void)want_sqdist;  // distances and squared distances need no scratch of their own
    Plan pl;
    if (make_plan(ndim, shape, sampling, pl, want_indices != 0) != TM_EDT_OK) return (size_t)-1;
    return pl.ws_bytes;
}

void tm_edt_reload_switches(void) {
    std::lock_guard<std::mutex> lock(g_switches_mutex);
    load_switches_locked();
}

int tm_edt_ws(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
              int64_t* out_sqdist, int64_t* out_indices, void* workspace, size_t workspace_bytes,
              tm_edt_stream_t stream) {
    Plan pl;
    int rc = check_call(input, ndim, shape, sampling, out_dist, out_sqdist, out_indices, pl);
    if (rc != TM_EDT_OK) return rc;
    if (pl.N == 0) { g_last_launches = 0; return TM_EDT_OK; }
    if (pl.ws_bytes > 0) {
        if (!workspace || workspace_bytes < pl.ws_bytes) return TM_EDT_ERR_ALLOC;
        if (((uintptr_t)workspace & 255u) != 0) return TM_EDT_ERR_INVALID_ARG;
        if (!is_device_ptr(workspace)) return TM_EDT_ERR_BAD_POINTER;
    }
    if (!is_device_ptr(input) || (out_dist && !is_device_ptr(out_dist)) || (out_sqdist && !is_device_ptr(out_sqdist)) ||
        (out_indices && !is_device_ptr(out_indices)))
        return TM_EDT_ERR_BAD_POINTER;
    return run_device(pl, input, out_dist, out_sqdist, out_indices, workspace, (cudaStream_t)stream);
}

int tm_edt(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
           int64_t* out_sqdist, int64_t* out_indices, tm_edt_stream_t stream) {
    Plan pl;
    int rc = check_call(input, ndim, shape, sampling, out_dist, out_sqdist, out_indices, pl);
    if (rc != TM_EDT_OK) return rc;
    if (pl.N == 0) { g_last_launches = 0; return TM_EDT_OK; }
    if (!is_device_ptr(input) || (out_dist && !is_device_ptr(out_dist)) || (out_sqdist && !is_device_ptr(out_sqdist)) ||
        (out_indices && !is_device_ptr(out_indices)))
        return TM_EDT_ERR_BAD_POINTER;
    cudaStream_t st = (cudaStream_t)stream;
    void* ws = nullptr;
    if (pl.ws_bytes > 0) {
        cudaError_t e = scratch_alloc(&ws, pl.ws_bytes, st);
        if (e != cudaSuccess) { cudaGetLastError(); g_last_cuda_error = (int)e; return TM_EDT_ERR_ALLOC; }
    }
    rc = run_device(pl, input, out_dist, out_sqdist, out_indices, ws, st);
    if (ws) cudaFreeAsync(ws, st);
    return rc;
}

// Contiguous byte strides of (B, C, n...), or the caller's; returns false if a stride is negative.
static bool resolve_strides(int ndim, const int64_t* shape, const int64_t* in_strides, int64_t* st, bool& strided,
                            size_t& span) {
    const int dims = ndim + 2;
    int64_t c = 1;
    strided = false;
    span = 1;
    for (int a = dims - 1; a >= 0; --a) {
        st[a] = in_strides ? in_strides[a] : c;
        if (st[a] < 0) return false;
        if (shape[a] > 1 && st[a] != c) strided = true;
        if (shape[a] > 0) span += (size_t)(shape[a] - 1) * (size_t)st[a];
        c *= shape[a];
    }
    return true;
}

struct ExLayout { size_t core, mask, fidx, total; };

static ExLayout ex_layout(const Plan& pl, bool strided, unsigned flags, bool with_indices, bool with_dist) {
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    ExLayout L;
    L.core = up(pl.ws_bytes);
    L.mask = strided ? up((size_t)pl.N) : 0;
    L.fidx = ((flags & TM_EDT_FLAG_DIST_F64) && with_dist && !with_indices) ? up((size_t)pl.N * 8) : 0;
    L.total = L.core + L.mask + L.fidx;
    if (L.mask == 0 && L.fidx == 0) L.total = pl.ws_bytes;
    return L;
}

size_t tm_edt_ex_workspace_bytes(int ndim, const int64_t* shape, const int64_t* in_strides, unsigned flags,
                                 int with_distances, int with_indices) {
    Plan pl;
    if (make_plan(ndim, shape, nullptr, pl) != TM_EDT_OK) return (size_t)-1;
    const bool want_idx = with_indices != 0 || ((flags & TM_EDT_FLAG_DIST_F64) && with_distances != 0);
    pl.ws_bytes = worst_case_workspace(ndim, shape, want_idx);
    int64_t st[kMaxDims + 2];
    bool strided = false;
    size_t span = 0;
    if (!resolve_strides(ndim, shape, in_strides, st, strided, span)) return (size_t)-1;
    return ex_layout(pl, strided, flags, with_indices != 0, with_distances != 0).total;
}

int tm_edt_ex(const uint8_t* input, int ndim, const int64_t* shape, const int64_t* in_strides, const double* sampling,
              void* out_dist, int64_t* out_sqdist, int64_t* out_indices, unsigned flags, void* workspace,
              size_t workspace_bytes, tm_edt_stream_t stream) {
    Plan pl;
    int rc = check_call(input, ndim, shape, sampling, static_cast<float*>(out_dist), out_sqdist, out_indices, pl, flags);
    if (rc != TM_EDT_OK) return rc;
    int64_t strides[kMaxDims + 2];
    bool strided = false;
    size_t span = 0;
    if (!resolve_strides(ndim, shape, in_strides, strides, strided, span)) return TM_EDT_ERR_INVALID_ARG;
    if (pl.N == 0) { g_last_launches = 0; return TM_EDT_OK; }
    if (strided) {  // the outputs must not overlap the bytes the strided mask spans
        const size_t N = (size_t)pl.N;
        if (overlap(input, span, out_dist, N * ((flags & TM_EDT_FLAG_DIST_F64) ? 8 : 4)) || overlap(input, span, out_sqdist, N * 8) ||
            overlap(input, span, out_indices, N * 8 * (size_t)((flags & TM_EDT_FLAG_FLAT_INDEX) ? 1 : ndim)))
            return TM_EDT_ERR_INVALID_ARG;
    }
    if (!is_device_ptr(input) || (out_dist && !is_device_ptr(out_dist)) || (out_sqdist && !is_device_ptr(out_sqdist)) ||
        (out_indices && !is_device_ptr(out_indices)))
        return TM_EDT_ERR_BAD_POINTER;
    const bool f64 = (flags & TM_EDT_FLAG_DIST_F64) && out_dist;
    const ExLayout L = ex_layout(pl, strided, flags, out_indices != nullptr, out_dist != nullptr);
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = static_cast<char*>(workspace);
    bool pooled = false;
    if (workspace) {
        if (workspace_bytes < L.total) return TM_EDT_ERR_ALLOC;
        if (((uintptr_t)workspace & 255u) != 0) return TM_EDT_ERR_INVALID_ARG;
        if (!is_device_ptr(workspace)) return TM_EDT_ERR_BAD_POINTER;
    } else if (L.total > 0) {
        cudaError_t e = scratch_alloc((void**)&ws, L.total, st);
        if (e != cudaSuccess) { cudaGetLastError(); g_last_cuda_error = (int)e; return TM_EDT_ERR_ALLOC; }
        pooled = true;
    }
    int extra_launches = 0;
    const uint8_t* mask = input;
    if (strided) {
        GatherParams G;
        memset(&G, 0, sizeof(G));
        G.in = input; G.out = reinterpret_cast<uint8_t*>(ws + L.core); G.total = pl.N; G.dims = ndim + 2;
        for (int a = 0; a < ndim + 2; ++a) { G.shape[a] = shape[a]; G.stride[a] = strides[a]; }
        if (pl.N > (int64_t)INT32_MAX * 128) rc = TM_EDT_ERR_UNSUPPORTED;
        else {
            prof_mark(st, "gather_strided", (double)pl.N * 2.0);
            if (shape[ndim + 1] % 4 == 0) gather_strided_kernel<4><<<(unsigned)((pl.N / 4 + 255) / 256), 256, 0, st>>>(G);
            else gather_strided_kernel<1><<<(unsigned)((pl.N + 255) / 256), 256, 0, st>>>(G);
            ++extra_launches;
            mask = G.out;
        }
    }
    if (rc == TM_EDT_OK) {
        if (!f64) {
            rc = run_device(pl, mask, static_cast<float*>(out_dist), out_sqdist, out_indices, ws, st);
        } else {
            // float64 distances: the transform delivers the site of every voxel (the caller's index output, or one
            // linear index per voxel in scratch), a second kernel turns sites into distances
            Plan p2 = pl;
            int64_t* site = out_indices;
            if (!site) { site = reinterpret_cast<int64_t*>(ws + L.core + L.mask); p2.flags |= TM_EDT_FLAG_FLAT_INDEX; }
            rc = run_device(p2, mask, nullptr, out_sqdist, site, ws, st);
            if (rc == TM_EDT_OK) {
                const int64_t bpi = (pl.V + 255) / 256;  // blocks per image
                if (pl.images * bpi > (int64_t)INT32_MAX) rc = TM_EDT_ERR_UNSUPPORTED;
                else {
                    VirtualParams VP;
                    memset(&VP, 0, sizeof(VP));
                    VP.images = pl.images; VP.V = pl.V; VP.ndim = pl.ndim;
                    for (int a = 0; a < pl.ndim; ++a) { VP.shape[a] = pl.shape_sp[a]; VP.w[a] = pl.w_sp[a]; }
                    prof_mark(st, "dist_f64", (double)pl.N * (8.0 + 8.0 * ((p2.flags & TM_EDT_FLAG_FLAT_INDEX) ? 1 : pl.ndim)));
                    dist_f64_kernel<<<(unsigned)(pl.images * bpi), 256, 0, st>>>(
                        VP, site, (p2.flags & TM_EDT_FLAG_FLAT_INDEX) ? 1 : 0, (flags & TM_EDT_FLAG_VIRTUAL_BACKGROUND) ? 1 : 0,
                        static_cast<double*>(out_dist), (unsigned)bpi);
                    ++extra_launches;
                    cudaError_t e = cudaGetLastError();
                    if (e != cudaSuccess) { g_last_cuda_error = (int)e; rc = TM_EDT_ERR_CUDA; }
                }
            }
        }
    }
    if (rc == TM_EDT_OK) g_last_launches += extra_launches;
    if (pooled) cudaFreeAsync(ws, st);
    return rc;
}

int tm_edt_host(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
                int64_t* out_sqdist, int64_t* out_indices, tm_edt_stream_t stream) {
    Plan pl;
    int rc = check_call(input, ndim, shape, sampling, out_dist, out_sqdist, out_indices, pl);
    if (rc != TM_EDT_OK) return rc;
    if (pl.N == 0) { g_last_launches = 0; return TM_EDT_OK; }
    if (!is_host_ptr(input) || (out_dist && !is_host_ptr(out_dist)) || (out_sqdist && !is_host_ptr(out_sqdist)) ||
        (out_indices && !is_host_ptr(out_indices)))
        return TM_EDT_ERR_BAD_POINTER;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t N = (size_t)pl.N;
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const size_t b_in = up(N), b_d = out_dist ? up(N * 4) : 0, b_s = out_sqdist ? up(N * 8) : 0,
                 b_x = out_indices ? up(N * 8 * (size_t)ndim) : 0, b_ws = up(pl.ws_bytes);
    char* dev = nullptr;
    cudaError_t e = scratch_alloc((void**)&dev, b_in + b_d + b_s + b_x + b_ws, st);
    if (e != cudaSuccess) { cudaGetLastError(); g_last_cuda_error = (int)e; return TM_EDT_ERR_ALLOC; }
    uint8_t* d_in = (uint8_t*)dev;
    float* d_d = out_dist ? (float*)(dev + b_in) : nullptr;
    int64_t* d_s = out_sqdist ? (int64_t*)(dev + b_in + b_d) : nullptr;
    int64_t* d_x = out_indices ? (int64_t*)(dev + b_in + b_d + b_s) : nullptr;
    void* d_ws = pl.ws_bytes ? (void*)(dev + b_in + b_d + b_s + b_x) : nullptr;
    e = cudaMemcpyAsync(d_in, input, N, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
        rc = run_device(pl, d_in, d_d, d_s, d_x, d_ws, st);
        if (rc == TM_EDT_OK && out_dist) e = cudaMemcpyAsync(out_dist, d_d, N * 4, cudaMemcpyDeviceToHost, st);
        if (rc == TM_EDT_OK && e == cudaSuccess && out_sqdist)
            e = cudaMemcpyAsync(out_sqdist, d_s, N * 8, cudaMemcpyDeviceToHost, st);
        if (rc == TM_EDT_OK && e == cudaSuccess && out_indices)
            e = cudaMemcpyAsync(out_indices, d_x, N * 8 * (size_t)ndim, cudaMemcpyDeviceToHost, st);
    }
    cudaFreeAsync(dev, st);
    if (e != cudaSuccess) { cudaGetLastError(); g_last_cuda_error = (int)e; return TM_EDT_ERR_CUDA; }
    return rc;
}

// ---- entry point that allocates nothing -------------------------------------------------------
// Scratch for tm_edt_noalloc: one fixed array in device memory, part of the library image, so every GPU
// that loads the library carries it until the process exits.
#define TM_EDT_NOALLOC_SCRATCH_BYTES ((size_t)TM_EDT_NOALLOC_MAX_SCRATCH)
static __device__ __align__(256) unsigned char g_noalloc_scratch[TM_EDT_NOALLOC_MAX_SCRATCH];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel could use:
// the device address is asked for once per device (with that device current) and remembered.
static void* g_noalloc_ptr[64];
static bool g_noalloc_ready[64];
static std::mutex g_noalloc_mutex;

static int noalloc_scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { cudaGetLastError(); g_last_cuda_error = (int)e; return TM_EDT_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return TM_EDT_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ready[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            g_last_cuda_error = (int)e;
            return TM_EDT_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = p;
        g_noalloc_ready[dev] = true;
    }
    *out = g_noalloc_ptr[dev];
    return TM_EDT_OK;
}

int tm_edt_noalloc(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
                   int64_t* out_sqdist, int64_t* out_indices, tm_edt_stream_t stream) {
    Plan pl;
    int rc = check_call(input, ndim, shape, sampling, out_dist, out_sqdist, out_indices, pl);
    if (rc != TM_EDT_OK) return rc;
    if (pl.N == 0) { g_last_launches = 0; return TM_EDT_OK; }
    if (pl.ws_bytes > TM_EDT_NOALLOC_SCRATCH_BYTES) return TM_EDT_ERR_TOO_LARGE;
    if (!is_device_ptr(input) || (out_dist && !is_device_ptr(out_dist)) || (out_sqdist && !is_device_ptr(out_sqdist)) ||
        (out_indices && !is_device_ptr(out_indices)))
        return TM_EDT_ERR_BAD_POINTER;
    void* scratch = nullptr;
    if (pl.ws_bytes > 0) {
        rc = noalloc_scratch_address(&scratch);
        if (rc != TM_EDT_OK) return rc;
    }
    return run_device(pl, input, out_dist, out_sqdist, out_indices, scratch, (cudaStream_t)stream);
}

int tm_edt_trim_memory(void) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return TM_EDT_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return TM_EDT_OK;
    std::lock_guard<std::mutex> lock(g_pool_mutex);
    if (g_pool_ready[dev]) {
        cudaError_t e = cudaMemPoolTrimTo(g_pool[dev], 0);
        if (e != cudaSuccess) { cudaGetLastError(); g_last_cuda_error = (int)e; return TM_EDT_ERR_CUDA; }
    }
    return TM_EDT_OK;
}

size_t tm_edt_noalloc_max_scratch(void) { return TM_EDT_NOALLOC_SCRATCH_BYTES; }

const char* tm_edt_strerror(int status) {
    switch (status) {
        case TM_EDT_OK: return "ok";
        case TM_EDT_ERR_INVALID_ARG: return "invalid argument";
        case TM_EDT_ERR_UNSUPPORTED: return "unsupported size or option";
        case TM_EDT_ERR_BAD_POINTER: return "buffer is not in the expected memory space";
        case TM_EDT_ERR_ALLOC: return "scratch allocation failed or workspace too small";
        case TM_EDT_ERR_CUDA: return "CUDA runtime error";
        case TM_EDT_ERR_TOO_LARGE: return "problem needs more scratch than the built-in array of tm_edt_noalloc holds";
        case TM_EDT_ERR_DEBUG_CHECK: return "debug build: a kernel index left its range (see tm_edt_debug_last_violation)";
    }
    return "unknown status";
}

int tm_edt_profile(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
                   int64_t* out_sqdist, int64_t* out_indices, void* workspace, size_t workspace_bytes,
                   tm_edt_stream_t stream, int max_kernels, float* kernel_ms, double* kernel_bytes, char* kernel_names,
                   int* n_kernels) {
    return tm_edt_profile_ex(input, ndim, shape, sampling, out_dist, out_sqdist, out_indices, 0u, workspace,
                             workspace_bytes, stream, max_kernels, kernel_ms, kernel_bytes, kernel_names, n_kernels);
}

int tm_edt_profile_ex(const uint8_t* input, int ndim, const int64_t* shape, const double* sampling, float* out_dist,
                      int64_t* out_sqdist, int64_t* out_indices, unsigned flags, void* workspace, size_t workspace_bytes,
                      tm_edt_stream_t stream, int max_kernels, float* kernel_ms, double* kernel_bytes,
                      char* kernel_names, int* n_kernels) {
    if (!kernel_ms || !n_kernels || max_kernels < 1) return TM_EDT_ERR_INVALID_ARG;
    *n_kernels = 0;
    cudaStream_t st = (cudaStream_t)stream;
    g_prof.count = 0;
    for (int i = 0; i <= kProfMax; ++i)
        if (cudaEventCreate(&g_prof.ev[i]) != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(g_prof.ev[j]);
            g_last_cuda_error = (int)cudaGetLastError();
            return TM_EDT_ERR_CUDA;
        }
    g_prof.active = true;
    int rc = flags ? tm_edt_ex(input, ndim, shape, nullptr, sampling, out_dist, out_sqdist, out_indices, flags, workspace,
                               workspace_bytes, stream)
                   : tm_edt_ws(input, ndim, shape, sampling, out_dist, out_sqdist, out_indices, workspace, workspace_bytes,
                               stream);
    g_prof.active = false;
    const int cnt = g_prof.count;
    if (rc == TM_EDT_OK && cnt > 0) {
        cudaEventRecord(g_prof.ev[cnt], st);
        cudaError_t e = cudaEventSynchronize(g_prof.ev[cnt]);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; rc = TM_EDT_ERR_CUDA; }
        for (int i = 0; rc == TM_EDT_OK && i < cnt && i < max_kernels; ++i) {
            float ms = 0.f;
            cudaEventElapsedTime(&ms, g_prof.ev[i], g_prof.ev[i + 1]);
            kernel_ms[i] = ms;
            if (kernel_bytes) kernel_bytes[i] = g_prof.bytes[i];
            if (kernel_names) {
                strncpy(kernel_names + (size_t)i * 48, g_prof.name[i], 47);
                kernel_names[(size_t)i * 48 + 47] = 0;
            }
        }
        if (rc == TM_EDT_OK) *n_kernels = cnt < max_kernels ? cnt : max_kernels;
    }
    for (int i = 0; i <= kProfMax; ++i) cudaEventDestroy(g_prof.ev[i]);
    return rc;
}

int tm_edt_debug_build(void) {
#ifdef TM_EDT_DEBUG
    return 1;
#else
    return 0;
#endif
}

unsigned long long tm_edt_debug_last_violation(long long* code, long long* index, long long* limit) {
    if (code) *code = g_last_debug.code;
    if (index) *index = g_last_debug.index;
    if (limit) *limit = g_last_debug.limit;
    return g_last_debug.count;
}

int tm_edt_last_cuda_error(void) { return g_last_cuda_error; }
int tm_edt_last_launch_count(void) { return g_last_launches; }
const char* tm_edt_version(void) { return "tm_edt 0.1 (sm_100a)"; }

}  // extern "C"
