// Bounds checks of the debug build (-DTM_EDT_DEBUG=1), the stand-in for a memory checker: an index that leaves
// its range is recorded in a device-side record and the access is skipped -- no trap, no assert, the context stays
// usable -- and the host turns a non-empty record into the status TM_EDT_ERR_DEBUG_CHECK after the call.  In the
// release build the checks are the constant `true` and cost nothing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tmedt {

struct DebugRecord {
    unsigned long long count;  // violations seen
    long long code;            // where the first one happened (a number unique to the access site)
    long long index, limit;    // its index and the exclusive upper bound it should have respected
};

#ifdef TM_EDT_DEBUG
// one record per translation unit that launches kernels; read and cleared by debug_collect() below
static __device__ DebugRecord g_debug_record;

__device__ __forceinline__ bool debug_in_range(long long index, long long limit, int code) {
    if (index >= 0 && index < limit) return true;
    if (atomicAdd(&g_debug_record.count, 1ull) == 0ull) {
        g_debug_record.code = code;
        g_debug_record.index = index;
        g_debug_record.limit = limit;
    }
    return false;
}
#define TM_EDT_IN_RANGE(index, limit, code) ::tmedt::debug_in_range((long long)(index), (long long)(limit), (code))

// Host side: waits for `st`, copies this translation unit's record out and clears it.
static inline cudaError_t debug_collect(cudaStream_t st, DebugRecord* out) {
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    e = cudaMemcpyFromSymbol(out, g_debug_record, sizeof(DebugRecord));
    if (e != cudaSuccess) return e;
    if (out->count != 0ull) {
        const DebugRecord zero = {0ull, 0, 0, 0};
        e = cudaMemcpyToSymbol(g_debug_record, &zero, sizeof(DebugRecord));
    }
    return e;
}
#else
#define TM_EDT_IN_RANGE(index, limit, code) (true)
#endif

}  // namespace tmedt
