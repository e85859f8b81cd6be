// Shared host/device helpers of the s3scan library: error reporting, status block, key packing.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/s3.h"

namespace s3 {

// ---- host-side error reporting -------------------------------------------------------------
void set_error(const char* fmt, ...);
s3_status fail(s3_status code, const char* fmt, ...);

#define S3_CUDA_TRY(expr)                                                                        \
    do {                                                                                         \
        cudaError_t e__ = (expr);                                                                \
        if (e__ != cudaSuccess)                                                                  \
            return ::s3::fail(S3_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), \
                              __FILE__, __LINE__);                                               \
    } while (0)

#define S3_REQUIRE(cond, code, ...)                      \
    do {                                                 \
        if (!(cond)) return ::s3::fail(code, __VA_ARGS__); \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int device_sm_count();      // SMs of the current device (cached per device)
int device_cc_major();      // compute capability major of the current device

// ---- device status block (first 64 bytes of every workspace) ---------------------------------
// word 0: sticky error code (0 = fine). Codes name the wait that gave up.
enum : uint32_t {
    DEV_OK = 0,
    DEV_TIMEOUT_TMA_FULL = 1,    // MMA warp: operand tile never arrived
    DEV_TIMEOUT_SMEM_EMPTY = 2,  // TMA warp: pipeline slot never freed
    DEV_TIMEOUT_ACC_FULL = 3,    // epilogue: accumulator never completed
    DEV_TIMEOUT_ACC_EMPTY = 4,   // MMA warp: accumulator never drained
    DEV_BAD_FEATURE_ID = 16,     // postings: id >= d_sae met in the input
    DEV_COMPACT_CAPACITY = 17,   // compact index: block or payload buffer too small (sizes[] has the need)
    DEV_DUPLICATE_ID = 18,       // postings: one token carries the same feature id twice
};

__device__ __forceinline__ void dev_set_error(uint32_t* status, uint32_t code) { atomicCAS(status, 0u, code); }

// ---- Top-k candidate keys ----------------------------------------------------------------------
// A candidate (value > 0, feature id) is one 64-bit key: value bits in the high word (positive
// floats order like unsigned ints) and ~id in the low word, so a larger key is a better candidate
// under (value descending, id ascending). Key 0 is "no candidate".
__host__ __device__ __forceinline__ uint64_t make_key(uint32_t value_bits, uint32_t id)
{
    return (static_cast<uint64_t>(value_bits) << 32) | static_cast<uint32_t>(~id);
}

}  // namespace s3
