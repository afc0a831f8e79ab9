// Shared declarations of the Slim-DP CUDA library (sm_100a).
#pragma once

#include <atomic>
#include <cuda_runtime.h>
#include <stdint.h>

#include "slimdp.h"

namespace slimdp {

constexpr uint32_t kBlock = SLIMDP_BLOCK;        // parameters per bitmap block
constexpr uint32_t kWordsPerBlock = kBlock / 32; // 32 bitmap words per block
constexpr uint32_t kDirStride = SLIMDP_DIR_STRIDE;      // parameters per directory entry
constexpr uint32_t kDirPerBlock = kBlock / kDirStride;  // 16 directory entries per bitmap block
constexpr uint32_t kWordsPerDir = kDirStride / 32;      // 2 bitmap words per directory entry
static_assert(kWordsPerDir == 2, "select0 walks exactly two bitmap words per directory entry");
constexpr uint32_t kSampleBits = 18;             // the selection's bracket is estimated from 2^18 sampled keys
constexpr uint64_t kBracketMinN = 1ull << 21;    // below this the selection reads the keys three more times instead
constexpr uint32_t kQ8Bucket = SLIMDP_Q8_BUCKET;   // packed entries that share one scale of the 8-bit codes
constexpr uint32_t kStageChunk = 512;            // entries per chunk of the staging area (see layout.cuh)

// K device pointers passed by value as a kernel argument (512 bytes).
template <typename T>
struct PtrArray {
    T* p[SLIMDP_MAX_WORKERS];
};

// First 256 bytes of every workspace.
struct WsHeader {
    int32_t status;      // sticky: SLIMDP_OK or SLIMDP_ERR_INTERNAL
    uint32_t prefix;     // radix prefix found so far; after the last pass the threshold key T
    uint32_t k_rem;      // rank still to resolve inside the prefix; after the last pass the tie quota r
    uint32_t ties;       // r: how many keys equal to T are admitted (smallest indices first)
    uint32_t n_def;      // bracket pass: keys in bins >= b_top (certainly in the core)
    uint32_t n_cand;     // bracket pass: keys inside the bracket (candidates)
    uint32_t b_top;      // first 18-bit bin (key >> 14) certainly above T (2^18: none)
    uint32_t b_bot;      // lowest 18-bit bin that may hold T
    uint32_t ticket[8];  // "last CTA done" counters, one per kernel that needs one
    uint32_t coarse_x[2];  // sample: coarse bins in which the two target ranks are crossed
    uint32_t next_block;   // fused scoring pass: the next 1024-parameter block to hand out
    uint32_t barrier;      // finishing kernel: arrivals at its grid barrier so far (all epochs)
    uint32_t abort;        // finishing kernel: a bounded wait ran out; every CTA leaves
    uint32_t next_chunk;   // fused scoring pass: the next free chunk of the staging area
    uint32_t stage_lost;   // fused scoring pass: the staging area ran out of chunks
    uint32_t threshold;    // what the finishing kernel hands the emitting kernel: the threshold key T ...
    uint32_t tie_quota;    // ... and how many keys equal to T belong to the core
    uint32_t reserved[39];
};
static_assert(sizeof(WsHeader) == 256, "header is 256 bytes");

// True when the selection's pass over all keys proved that the threshold lies inside the sampled
// bracket and every candidate was stored (k = k_core, cap = capacity of the candidate list).
__host__ __device__ __forceinline__ bool bracket_held(uint32_t n_def, uint32_t n_cand, uint32_t k, uint32_t cap) {
    return n_def < k && k - n_def <= n_cand && n_cand <= cap;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline uint64_t num_blocks(uint64_t n) { return (n + kBlock - 1) / kBlock; }

// Number of SMs of the current device (cached per device id).
int sm_count();

// Adds n to the process-wide count of launched kernels.
void count_launches(unsigned n);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

// Asks for the largest shared-memory share of the SM's L1 for `kernel`.  An SM keeps one split
// at a time, so kernels that are to run side by side on one SM ask for the same split.
template <typename Kernel>
inline bool prefer_max_shared(Kernel kernel) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                (int)cudaSharedmemCarveoutMaxShared) == cudaSuccess;
}

// Marks, per device (bit d = device d, devices above 63 are never marked), that a setting the device
// keeps has been made: kernel attributes are set on a kernel's first launch on a device, not on every call.
struct DeviceOnce {
    std::atomic<unsigned long long> done{0};
    bool needed() const {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
        return ((done.load(std::memory_order_relaxed) >> dev) & 1ull) == 0;
    }
    void mark() {
        int dev = -1;
        if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64)
            done.fetch_or(1ull << dev, std::memory_order_relaxed);
    }
};

// After a group of `count` kernel launches: fail on a launch error, else count them.
#define SLIMDP_LAUNCHED(count)                                          \
    do {                                                                \
        if (cudaGetLastError() != cudaSuccess) return SLIMDP_ERR_CUDA;  \
        count_launches(count);                                          \
    } while (0)

// ---- device helpers -------------------------------------------------------

// Position of the n-th (0-based) set bit of word; word must have more than n set bits.
__device__ __forceinline__ uint32_t nth_set_bit(uint32_t word, uint32_t n) {
    uint32_t pos = 0;
#pragma unroll
    for (int width = 16; width >= 1; width >>= 1) {
        uint32_t low = (word >> pos) & ((1u << width) - 1u);
        uint32_t c = __popc(low);
        if (n >= c) {
            n -= c;
            pos += width;
        }
    }
    return pos;
}

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31u; }

// Inclusive warp scan (all 32 lanes active).
__device__ __forceinline__ uint32_t warp_inclusive_scan(uint32_t v) {
    const uint32_t lane = lane_id();
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t t = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= (uint32_t)d) v += t;
    }
    return v;
}

__device__ __forceinline__ unsigned long long warp_inclusive_scan64(unsigned long long v) {
    const uint32_t lane = lane_id();
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= (uint32_t)d) v += t;
    }
    return v;
}

// Exclusive scan of one value per thread over a block of NWARPS * 32 threads.
// Returns the exclusive prefix; *total receives the block sum.  smem: 33 words.
template <int NWARPS>
__device__ __forceinline__ unsigned long long block_exclusive_scan64(unsigned long long v,
                                                                     unsigned long long* smem,
                                                                     unsigned long long* total) {
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned long long inc = warp_inclusive_scan64(v);
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned long long s = (lane < (uint32_t)NWARPS) ? smem[lane] : 0ull;
        unsigned long long sinc = warp_inclusive_scan64(s);
        smem[lane] = sinc - s;
        if (lane == 31) smem[32] = sinc;
    }
    __syncthreads();
    unsigned long long out = smem[warp] + inc - v;
    *total = smem[32];
    __syncthreads();
    return out;
}

__device__ __forceinline__ unsigned long long block_exclusive_scan64_1024(unsigned long long v,
                                                                          unsigned long long* smem,
                                                                          unsigned long long* total) {
    return block_exclusive_scan64<32>(v, smem, total);
}

// Significance of one parameter (Eq. 1): |w| + c |g| with one rounding, every NaN as the canonical quiet NaN.
__device__ __forceinline__ float score_one(float c, float g, float w) {
    float s = __fmaf_rn(c, fabsf(g), fabsf(w));
    return (s != s) ? __uint_as_float(0x7FC00000u) : s;
}

// A merged model value as it is stored (Section 3.3 step 3 defines the value only): IEEE 754 leaves the
// payload of a NaN that an operation passes on open, so every NaN result of an update is stored as the
// canonical quiet NaN, as scores are.  Once NaN a parameter stays NaN, so one check after the last of a
// chain of updates gives the same bits as a check after each.
__device__ __forceinline__ float stored_model_value(float x) { return (x != x) ? __uint_as_float(0x7FC00000u) : x; }

}  // namespace slimdp
