// Host-side helpers of tm_edt.cu that the other entry points of the library use as well: the stream-ordered
// scratch pool, the device-pointer test and the per-thread error / launch-count records.  Not exported.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace tmedt {
cudaError_t shared_scratch_alloc(void** p, size_t bytes, cudaStream_t st);
bool shared_is_device_ptr(const void* p);
bool shared_overlap(const void* a, size_t na, const void* b, size_t nb);
void shared_record(int cuda_error, int launches);  // cuda_error < 0: leave the error record alone
}  // namespace tmedt
