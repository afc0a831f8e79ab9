// Key caching (Section 3.5): the core's keys change only every q rounds, so sender and
// receiver keep them and a push / pull of the core carries the values plus a signature of the
// key list.  slimdp_core_signature computes that signature on the device:
//     sig = sum over j of mix64(((j << 32) | key_j) + 0x9E3779B97F4A7C15)   (mod 2^64)
// with mix64 the output function of the SplitMix64 generator.  The sum is order-free in its
// evaluation (any grouping of a wrapping sum gives the same value) but position-dependent in
// its terms, so a permuted list gets a different signature.
#include "common.cuh"

namespace slimdp {

namespace {

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__global__ void __launch_bounds__(256) signature_kernel(const uint32_t* __restrict__ keys, uint64_t count,
                                                        unsigned long long* __restrict__ sig) {
    __shared__ unsigned long long warp_part[8];
    unsigned long long part = 0;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += stride)
        part += mix64(((j << 32) | (unsigned long long)__ldg(keys + j)) + 0x9E3779B97F4A7C15ull);
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, d);
    if ((threadIdx.x & 31u) == 0) warp_part[threadIdx.x >> 5] = part;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long total = 0;
        for (int wdx = 0; wdx < 8; ++wdx) total += warp_part[wdx];
        if (total) atomicAdd(sig, total);
    }
}

}  // namespace

slimdp_status launch_signature(const uint32_t* keys, uint64_t count, unsigned long long* sig, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    if (cudaMemsetAsync(sig, 0, sizeof(unsigned long long), st) != cudaSuccess) return SLIMDP_ERR_CUDA;
    if (count == 0) return SLIMDP_OK;
    uint64_t grid = (count + 255) / 256;
    if (grid > (uint64_t)sms * 8) grid = (uint64_t)sms * 8;
    signature_kernel<<<(unsigned)grid, 256, 0, st>>>(keys, count, sig);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
