// Test helper (not part of the library): the first output word of cuRAND's device Philox4x32-10 for the counters
// (step, sequence, slot, stream tag) under the key (lo, hi) of a seed.  The GPU tests compare the library's and the
// oracle's uniforms with (word >> 8) * 2^-24 computed from these words, which pins both to an implementation
// neither of them shares code with.
#include <cstdint>
#include <cuda_runtime.h>
#include <curand_kernel.h>

namespace {
__global__ void words_kernel(uint32_t lo, uint32_t hi, uint32_t step, uint32_t tag, int n_seq, int n_slots, uint32_t* out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_seq * n_slots) return;
    const uint4 r = curand_Philox4x32_10(make_uint4(step, (uint32_t)(i / n_slots), (uint32_t)(i % n_slots), tag), make_uint2(lo, hi));
    out[i] = r.x;
}
}  // namespace

extern "C" int curand_philox_words(uint64_t seed, uint32_t step, uint32_t tag, int n_seq, int n_slots, uint32_t* out_dev)
{
    const int n = n_seq * n_slots;
    if (n <= 0) return 0;
    words_kernel<<<(n + 255) / 256, 256>>>((uint32_t)seed, (uint32_t)(seed >> 32), step, tag, n_seq, n_slots, out_dev);
    return cudaDeviceSynchronize() == cudaSuccess ? 0 : -1;
}
