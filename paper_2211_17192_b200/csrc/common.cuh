// Shared helpers of the CUDA library: status/error plumbing, warp primitives,
// the counter-based generator.  sm_100a only.
#pragma once

#include <atomic>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdarg>
#include <cstdio>

#include "spec_decode.h"

namespace spec {

// ---- per-thread error message ---------------------------------------------
char* error_buffer();  // 512 bytes, thread-local (defined in api.cu)

inline int fail(int status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(error_buffer(), 512, fmt, ap);
    va_end(ap);
    return status;
}

#define SPEC_CUDA_TRY(expr)                                                             \
    do {                                                                                \
        cudaError_t err__ = (expr);                                                     \
        if (err__ != cudaSuccess)                                                       \
            return ::spec::fail(SPEC_ERR_CUDA, "%s failed: %s (%s:%d)", #expr,          \
                                cudaGetErrorString(err__), __FILE__, __LINE__);         \
    } while (0)

// ---- programmatic dependent launch -------------------------------------------
// Every kernel of the decode path is launched with programmatic stream
// serialization and follows one rule: it may start while its predecessor in the
// stream is still running, it calls pdl_wait() before it reads or writes
// anything another kernel touches, and it calls pdl_trigger() as early as it
// can so that its successor can start its own independent prologue (for a GEMM:
// streaming the first weight tiles).  pdl_wait() returns once the predecessor
// grid has completed and its writes are visible; because every kernel waits,
// completion is transitive along the stream.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// SPEC_NO_PDL=1 in the environment launches every kernel fully serialised (for debugging; the one
// environment variable the library reads, documented in the public header).
bool pdl_enabled();  // api.cu

// True the first time it is called on the current device for this flag word (one bit per
// device ordinal below 64): per-device one-time setup such as a kernel's shared-memory opt-in,
// which a process that uses several GPUs has to repeat on each of them.
inline bool first_use_on_this_device(std::atomic<unsigned long long>& seen) {
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return true;
    const unsigned long long bit = 1ull << device;
    return (seen.fetch_or(bit) & bit) == 0;
}

template <typename... KArgs, typename... Args>
inline int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    if (err != cudaSuccess) return fail(SPEC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(err));
    return SPEC_OK;
}

// ---- warp / block primitives ----------------------------------------------
constexpr unsigned kFullMask = 0xffffffffu;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
    return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFullMask, v, o));
    return v;
}

// Inclusive prefix sum across the lanes of a warp.
__device__ __forceinline__ float warp_inclusive_scan(float v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        float up = __shfl_up_sync(kFullMask, v, o);
        if (lane >= o) v += up;
    }
    return v;
}

// ---- Philox4x32-10 (Salmon et al., SC'11) -----------------------------------
// key = 64-bit seed, counter = (position, sequence, purpose, 0); the first
// output word w becomes the uniform (2 * (w >> 9) + 1) / 2^24, which lies
// strictly inside (0, 1) and is exact in fp32.
__host__ __device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2,
                                                               uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = 0xD2511F53ull * c0;
        const uint64_t p1 = 0xCD9E8D57ull * c2;
        const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = static_cast<uint32_t>(p1);
        const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = static_cast<uint32_t>(p0);
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

__host__ __device__ __forceinline__ float method_uniform(uint64_t seed, uint32_t position,
                                                         uint32_t sequence, uint32_t purpose) {
    const uint32_t w = philox_first_word(position, sequence, purpose, 0u, static_cast<uint32_t>(seed),
                                         static_cast<uint32_t>(seed >> 32));
    return static_cast<float>(2u * (w >> 9) + 1u) * (1.0f / 16777216.0f);
}

enum : uint32_t { kPurposeDraft = 0, kPurposeAccept = 1, kPurposeFinal = 2 };

}  // namespace spec
