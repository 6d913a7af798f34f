// Shared device/host helpers of the CUDA library: status word, launch checks, Philox4x32-10 uniforms,
// warp reductions and 16-byte vector types.  Nothing here is shared with the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/spec.h"

namespace spec {

// ---- status word: int32[4] = {code, detail, 0, 0}; the first error wins --------------------------------------
__device__ __forceinline__ void set_status(int32_t* status, int code, int detail)
{
    if (status != nullptr && atomicCAS(status, 0, code) == 0) status[1] = detail;
}

#define SPEC_CUDA_OK(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) return SPEC_ERR_CUDA;        \
    } while (0)

// Number of kernels this library has launched in this process (every launcher reports through launch_status()).
std::atomic<long long>& launch_counter();
inline spec_status launch_status(int n_launched = 1)
{
    launch_counter() += n_launched;
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

// Kernel attributes (dynamic shared memory limits) are set per device: one bit per device ordinal records where a call site
// has done its one-time set-up, so a process that drives several devices configures each of them, and two host threads that
// arrive together at worst both do the (idempotent) set-up.
struct PerDeviceOnce {
    std::atomic<unsigned long long> seen{0};
    // true when the current device still needs the set-up; call done() after it succeeded
    bool needed(int* dev_out)
    {
        int dev = 0;
        cudaGetDevice(&dev);
        *dev_out = dev;
        return (seen.load(std::memory_order_acquire) & (1ull << (dev & 63))) == 0;
    }
    void done(int dev) { seen.fetch_or(1ull << (dev & 63), std::memory_order_release); }
};

// Programmatic dependent launch.  A kernel launched through launch_pdl may be scheduled before the kernel in front of it
// in the stream has finished (as soon as that one has called pdl_trigger, or has exited), which hides the launch latency
// between the many short dependent kernels of a step; it must call pdl_wait before it touches global memory (the wait
// returns once the kernel in front has completed and its writes are visible).  Both calls are no-ops in a kernel that
// was launched the ordinary way.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Per-thread scratch for split-K GEMMs, set by the context entry points (the stateless spec_gemm has none and never splits).
struct GemmScratch { void* ptr = nullptr; size_t bytes = 0; };
GemmScratch& gemm_scratch();

// ---- Philox4x32-10 (Salmon et al., SC'11).  key = (lo, hi) of the seed, counter = (step, seq, slot, stream);
// the uniform is the top 24 bits of the first output word scaled by 2^-24: in [0,1), exact in fp32. ------------
__device__ __forceinline__ uint32_t philox_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                 uint32_t k1)
{
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t h0 = __umulhi(M0, c0), l0 = M0 * c0;
        const uint32_t h1 = __umulhi(M1, c2), l1 = M1 * c2;
        const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
        c0 = n0; c1 = l1; c2 = n2; c3 = l0;
        k0 += W0; k1 += W1;
    }
    return c0;
}

__device__ __forceinline__ float philox_uniform(uint64_t seed, uint32_t step, uint32_t seq, uint32_t slot,
                                                uint32_t stream)
{
    const uint32_t w = philox_word0(step, seq, slot, stream, (uint32_t)seed, (uint32_t)(seed >> 32));
    return (float)(w >> 8) * (1.0f / 16777216.0f);
}

// ---- warp helpers ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ int warp_max(int v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_inclusive_scan(double v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// ---- element types ----------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <class T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

inline size_t dtype_bytes(int dtype) { return dtype == SPEC_DTYPE_F32 ? 4 : 2; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace spec
