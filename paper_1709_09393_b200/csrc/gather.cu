// slimdp_pack / slimdp_pull: gather the values of the communication set
// T_C = core U explorer (Section 3.1) out of a full-length vector: the
// worker's updates for the push (the extraction step of Section 3.5), the
// merged global parameters for the pull (Section 3.3 step 4).
#include "common.cuh"

namespace slimdp {

namespace {

// grid.y = worker.  out[w][j] = src[w][core_idx[j]] (j < k_core), out[w][k_core + j] = src[w][exp[w][j]].
__global__ void __launch_bounds__(256) gather_kernel(PtrArray<const float> src, const uint32_t* __restrict__ core_idx,
                                                     uint64_t k_core, PtrArray<const uint32_t> exp, uint64_t k_exp,
                                                     PtrArray<float> out) {
    const uint32_t worker = blockIdx.y;
    const float* __restrict__ s = src.p[worker];
    const uint32_t* __restrict__ e = exp.p[worker];
    float* __restrict__ o = out.p[worker];
    const uint64_t m = k_core + k_exp;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x * 4;
    for (uint64_t j0 = ((uint64_t)blockIdx.x * blockDim.x) * 4 + threadIdx.x; j0 < m; j0 += stride) {
        uint32_t idx[4];
        float v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            if (j < m) idx[q] = (j < k_core) ? __ldg(core_idx + j) : __ldg(e + (j - k_core));
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            if (j < m) v[q] = __ldg(s + idx[q]);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            if (j < m) o[j] = v[q];
        }
    }
}

}  // namespace

slimdp_status launch_gather(const PtrArray<const float>& src, uint32_t workers, const uint32_t* core_idx,
                            uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                            const PtrArray<float>& out, cudaStream_t st) {
    const uint64_t m = k_core + k_exp;
    if (m == 0) return SLIMDP_OK;
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    uint64_t grid = (m + 1023) / 1024;
    const uint64_t cap = ((uint64_t)sms * 32 + workers - 1) / workers;
    if (grid > cap) grid = cap;
    gather_kernel<<<dim3((unsigned)grid, workers), 256, 0, st>>>(src, core_idx, k_core, exp, k_exp, out);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
