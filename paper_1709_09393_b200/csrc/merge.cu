// slimdp_merge: the server update of Section 3.3 step 3,
// w <- w - eta' * T_C(delta_k) for every worker, applied in ascending worker
// order so that the fp32 result is unique.
//
// Core segment: one thread owns one core parameter and folds the K pushed
// values into it in worker order (K coalesced value streams, one gather and
// one scatter).
// Explorer segments: different workers' explorers may contain the same
// parameter (never a core one), so the order across workers matters.  The
// parameter vector is cut into ranges; one CTA owns one range, finds each
// worker's entries inside it by binary search of the ascending index lists,
// and applies worker 0's entries, a block barrier, worker 1's entries, ...
// Inside one worker the indices are distinct, and no other CTA touches the
// range, so a parameter receives its updates in ascending k without atomics.
#include "common.cuh"

namespace slimdp {

namespace {

__global__ void __launch_bounds__(256) merge_core_kernel(float* __restrict__ w, const uint32_t* __restrict__ core_idx,
                                                         uint64_t k_core, PtrArray<const float> val, int K,
                                                         float neg_eta) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_core; j += stride) {
        const uint32_t i = __ldg(core_idx + j);
        float x = w[i];
        int k = 0;
        for (; k + 8 <= K; k += 8) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = __ldcs(val.p[k + q] + j);
#pragma unroll
            for (int q = 0; q < 8; ++q) x = __fmaf_rn(neg_eta, v[q], x);
        }
        for (; k < K; ++k) x = __fmaf_rn(neg_eta, __ldcs(val.p[k] + j), x);
        w[i] = x;
    }
}

// First position in a[0, len) whose value is >= x.
__device__ __forceinline__ uint32_t lower_bound(const uint32_t* __restrict__ a, uint32_t len, uint64_t x) {
    uint32_t lo = 0, hi = len;
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if ((uint64_t)__ldg(a + mid) < x)
            lo = mid + 1;
        else
            hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(256) merge_explore_kernel(float* w, uint64_t n, PtrArray<const uint32_t> exp,
                                                            uint32_t k_exp, PtrArray<const float> val,
                                                            uint64_t k_core, int K, float neg_eta,
                                                            uint32_t range_shift) {
    __shared__ uint32_t begin[SLIMDP_MAX_WORKERS], end[SLIMDP_MAX_WORKERS];
    const uint64_t first = (uint64_t)blockIdx.x << range_shift;
    const uint64_t last = first + (1ull << range_shift);
    for (int t = threadIdx.x; t < 2 * K; t += blockDim.x) {
        const int k = (t < K) ? t : t - K;
        const uint32_t pos = lower_bound(exp.p[k], k_exp, (t < K) ? first : last);
        if (t < K)
            begin[k] = pos;
        else
            end[k] = pos;
    }
    __syncthreads();
    for (int k = 0; k < K; ++k) {
        const uint32_t* __restrict__ idx = exp.p[k];
        const float* __restrict__ v = val.p[k] + k_core;
        const uint32_t b = end[k];
        for (uint32_t e = begin[k] + threadIdx.x; e < b; e += blockDim.x) {
            const uint32_t i = __ldg(idx + e);
            w[i] = __fmaf_rn(neg_eta, __ldcs(v + e), w[i]);
        }
        __syncthreads();   // worker k's updates are visible to the whole CTA before worker k+1 starts
    }
}

}  // namespace

slimdp_status launch_merge(float* w, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                           const PtrArray<const uint32_t>& exp, uint64_t k_exp, const PtrArray<const float>& val,
                           float eta, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const float neg_eta = -eta;
    if (k_core > 0) {
        uint64_t grid = (k_core + 255) / 256;
        if (grid > (uint64_t)sms * 32) grid = (uint64_t)sms * 32;
        merge_core_kernel<<<(unsigned)grid, 256, 0, st>>>(w, core_idx, k_core, val, (int)K, neg_eta);
        SLIMDP_LAUNCHED(1);
    }
    if (k_exp > 0) {
        // range length: a power of two with about 256 entries per worker per range, at least 1024 parameters
        uint32_t shift = 10;
        while (shift < 24 && ((k_exp << shift) / n) < 256) ++shift;
        const uint64_t ranges = (n + (1ull << shift) - 1) >> shift;
        merge_explore_kernel<<<(unsigned)ranges, 256, 0, st>>>(w, n, exp, (uint32_t)k_exp, val, k_core, (int)K,
                                                               neg_eta, shift);
        SLIMDP_LAUNCHED(1);
    }
    return SLIMDP_OK;
}

}  // namespace slimdp
