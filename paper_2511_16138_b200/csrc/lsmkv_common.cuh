// Shared device-side helpers: status block, error recording, small utilities.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "lsmkv.h"

namespace lsmkv {

// Mirrors lsmkv_status_t field for field (device copy, updated with atomics).
struct DevStatus {
    unsigned int flags;
    unsigned int reserved;
    unsigned long long first_bad;
    unsigned long long chunks_encoded;
    unsigned long long lookups;
    unsigned long long chunks_hit;
    unsigned long long empty_probes;
    unsigned long long chunks_decoded;
};
static_assert(sizeof(DevStatus) == sizeof(lsmkv_status_t), "status layouts must match");

__device__ __forceinline__ void st_flag(DevStatus *st, unsigned int flag, unsigned long long idx)
{
    atomicOr(&st->flags, flag);
    atomicMin(&st->first_bad, idx);
}

constexpr uint32_t kSkip = 0xFFFFFFFFu;  // plan entry of a chunk that must not be copied

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }

}  // namespace lsmkv
