// Key caching (Section 3.5): the core's keys change only every q rounds, so sender and
// receiver keep them and a push / pull of the core carries the values plus a signature of the
// key list.  slimdp_core_signature computes that signature on the device:
//     sig = sum over j of mix64(((j << 32) | key_j) + 0x9E3779B97F4A7C15)   (mod 2^64)
// with mix64 the output function of the SplitMix64 generator.  The sum is order-free in its
// evaluation (any grouping of a wrapping sum gives the same value) but position-dependent in
// its terms, so a permuted list gets a different signature.
#include "common.cuh"

namespace slimdp {

slimdp_status launch_signature(const uint32_t* keys, uint64_t count, unsigned long long* sig, cudaStream_t st);

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

// ---- one worker's push as a message ----------------------------------------------------------
// Layout (little-endian, all fields 4-byte aligned; the message itself is 16-byte aligned):
//    0 u32 magic "SDPW"    4 u32 flags (bit 0: the core's keys are included)
//    8 u64 signature of the sender's core keys
//   16 u32 k_core   20 u32 k_exp   24 u32 worker   28 u32 round
//   32 [k_core x u32 keys]  k_core x f32 values  k_exp x (u32 key, f32 value)
constexpr uint32_t kWireMagic = 0x57504453u;
constexpr uint32_t kWireHeaderWords = 8;

__global__ void __launch_bounds__(256) wire_pack_kernel(const uint32_t* __restrict__ core_idx, uint64_t k_core,
                                                        const uint32_t* __restrict__ exp_idx, uint64_t k_exp,
                                                        const uint32_t* __restrict__ val,
                                                        const unsigned long long* __restrict__ sig, uint32_t worker,
                                                        uint32_t round, uint32_t with_keys,
                                                        uint32_t* __restrict__ msg) {
    const uint64_t gid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    if (gid == 0) {
        const unsigned long long s = *sig;
        msg[0] = kWireMagic;
        msg[1] = with_keys;
        msg[2] = (uint32_t)s;
        msg[3] = (uint32_t)(s >> 32);
        msg[4] = (uint32_t)k_core;
        msg[5] = (uint32_t)k_exp;
        msg[6] = worker;
        msg[7] = round;
    }
    uint32_t* p = msg + kWireHeaderWords;
    if (with_keys) {
        for (uint64_t j = gid; j < k_core; j += stride) p[j] = __ldg(core_idx + j);
        p += k_core;
    }
    for (uint64_t j = gid; j < k_core; j += stride) p[j] = __ldcs(val + j);
    p += k_core;
    for (uint64_t j = gid; j < k_exp; j += stride) {
        p[2 * j] = __ldg(exp_idx + j);
        p[2 * j + 1] = __ldcs(val + k_core + j);
    }
}

// status[0]: 0 = taken apart, 1 = keys wanted, -1 = malformed; status + 2 (as 64 bits): the
// signature of the k_core words after the header, computed by signature_kernel before this launch.
__global__ void __launch_bounds__(256) wire_unpack_kernel(const uint32_t* __restrict__ msg, uint64_t msg_bytes,
                                                          const unsigned long long* __restrict__ cached_sig,
                                                          uint64_t k_core, uint64_t k_exp,
                                                          uint32_t* __restrict__ core_idx,
                                                          uint32_t* __restrict__ exp_idx, uint32_t* __restrict__ val,
                                                          unsigned long long* __restrict__ sig_out,
                                                          int32_t* __restrict__ status) {
    const uint64_t gid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    int32_t verdict = 0;
    uint32_t flags = 0;
    unsigned long long sig = 0;
    if (msg_bytes < 32 || __ldg(msg) != kWireMagic) {
        verdict = -1;
    } else {
        flags = __ldg(msg + 1);
        sig = (unsigned long long)__ldg(msg + 2) | ((unsigned long long)__ldg(msg + 3) << 32);
        if (flags > 1u || __ldg(msg + 4) != k_core || __ldg(msg + 5) != k_exp ||
            msg_bytes != 32 + 4 * k_core * (flags ? 2 : 1) + 8 * k_exp)
            verdict = -1;
        else if (flags & 1u)
            verdict = (*reinterpret_cast<const unsigned long long*>(status + 2) == sig) ? 0 : -1;
        else
            verdict = (*cached_sig == sig) ? 0 : 1;
    }
    // every thread reached the same verdict from the same words; one of them reports it
    if (gid == 0) {
        status[0] = verdict;
        if (verdict == 0) *sig_out = sig;
    }
    if (verdict != 0) return;
    const uint32_t* p = msg + kWireHeaderWords;
    if (flags & 1u) {
        for (uint64_t j = gid; j < k_core; j += stride) core_idx[j] = __ldcs(p + j);
        p += k_core;
    }
    for (uint64_t j = gid; j < k_core; j += stride) val[j] = __ldcs(p + j);
    p += k_core;
    for (uint64_t j = gid; j < k_exp; j += stride) {
        exp_idx[j] = __ldcs(p + 2 * j);
        val[k_core + j] = __ldcs(p + 2 * j + 1);
    }
}

}  // namespace

slimdp_status launch_wire_pack(const uint32_t* core_idx, uint64_t k_core, const uint32_t* exp_idx, uint64_t k_exp,
                               const float* val, const unsigned long long* sig, uint32_t worker, uint32_t round,
                               bool with_keys, void* msg, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    uint64_t grid = (k_core + k_exp + 255) / 256;
    if (grid > (uint64_t)sms * 8) grid = (uint64_t)sms * 8;
    if (grid == 0) grid = 1;
    wire_pack_kernel<<<(unsigned)grid, 256, 0, st>>>(core_idx, k_core, exp_idx, k_exp,
                                                     reinterpret_cast<const uint32_t*>(val), sig, worker, round,
                                                     with_keys ? 1u : 0u, reinterpret_cast<uint32_t*>(msg));
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

slimdp_status launch_wire_unpack(const void* msg, size_t msg_bytes, const unsigned long long* cached_sig,
                                 uint64_t k_core, uint64_t k_exp, uint32_t* core_idx, uint32_t* exp_idx, float* val,
                                 unsigned long long* sig_out, int32_t* status, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    // signature of the words where a message with keys has them (unused if it turns out to have none)
    slimdp_status rc = launch_signature(reinterpret_cast<const uint32_t*>(msg) + kWireHeaderWords, k_core,
                                        reinterpret_cast<unsigned long long*>(status + 2), st);
    if (rc != SLIMDP_OK) return rc;
    uint64_t grid = (k_core + k_exp + 255) / 256;
    if (grid > (uint64_t)sms * 8) grid = (uint64_t)sms * 8;
    if (grid == 0) grid = 1;
    wire_unpack_kernel<<<(unsigned)grid, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(msg), msg_bytes, cached_sig,
                                                       k_core, k_exp, core_idx, exp_idx,
                                                       reinterpret_cast<uint32_t*>(val), sig_out, status);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

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
