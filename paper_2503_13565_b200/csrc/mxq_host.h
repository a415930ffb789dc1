// Host-side helpers: argument validation and launch plumbing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxq.h"

namespace mxq {

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool shape_ok(int64_t N, int64_t K) { return N >= 1 && K >= 32 && (K % 32) == 0; }
inline int launch_status() { return cudaGetLastError() == cudaSuccess ? MXQ_OK : MXQ_ERR_CUDA; }

// number of SMs of the current device (cached per device)
int sm_count();
// whether mxq_linear launches carry the programmatic-dependent-launch attribute
bool pdl_enabled();

}  // namespace mxq
