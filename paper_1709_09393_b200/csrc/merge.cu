// slimdp_merge: the server update of Section 3.3 step 3,
// w <- w - eta' * T_C(delta_k) for every worker, applied in ascending worker
// order so that the fp32 result is unique.
//
// Core segment: one thread owns one core parameter and folds the K pushed
// values into it in worker order (K coalesced value streams, one gather and
// one scatter).  Explorer segments: workers' explorers may collide with each
// other (never with the core), so they are applied as K stream-ordered
// launches; inside one worker the indices are distinct.
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
#pragma unroll 4
        for (int k = 0; k < K; ++k) x = __fmaf_rn(neg_eta, __ldcs(val.p[k] + j), x);
        w[i] = x;
    }
}

__global__ void __launch_bounds__(256) merge_explore_kernel(float* __restrict__ w, const uint32_t* __restrict__ exp_idx,
                                                            uint64_t k_exp, const float* __restrict__ val_exp,
                                                            float neg_eta) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_exp; j += stride) {
        const uint32_t i = __ldg(exp_idx + j);
        w[i] = __fmaf_rn(neg_eta, __ldcs(val_exp + j), w[i]);
    }
}

}  // namespace

slimdp_status launch_merge(float* w, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
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
        uint64_t grid = (k_exp + 255) / 256;
        if (grid > (uint64_t)sms * 32) grid = (uint64_t)sms * 32;
        for (uint32_t k = 0; k < K; ++k) {
            merge_explore_kernel<<<(unsigned)grid, 256, 0, st>>>(w, exp.p[k], k_exp, val.p[k] + k_core, neg_eta);
            SLIMDP_LAUNCHED(1);
        }
    }
    return SLIMDP_OK;
}

}  // namespace slimdp
