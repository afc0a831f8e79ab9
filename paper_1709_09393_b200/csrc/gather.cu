// slimdp_pack / slimdp_pull: gather the values of the communication set
// T_C = core U explorer (Section 3.1) out of a full-length vector: the
// worker's updates for the push (the extraction step of Section 3.5), the
// merged global parameters for the pull (Section 3.3 step 4).
//
// Core segment: the core keys are shared by all workers (Section 3.5, key
// caching), so one thread reads core_idx[j] once and serves all K workers:
// K independent gathers in flight for the push, a single gather written K
// times for the pull.  Explorer segments: one grid row per worker.
#include "common.cuh"

namespace slimdp {

namespace {

// Sparse 4-byte reads: ask L2 for its smallest fetch (64 B) instead of a whole 128-byte line.
__device__ __forceinline__ float ld_sparse(const float* p) {
    float v;
    asm volatile("ld.global.L2::64B.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

// out[k][j] = src[k][core_idx[j]] for every worker k.  SAME: all workers read the same source.
template <bool SAME>
__global__ void __launch_bounds__(256) gather_core_kernel(PtrArray<const float> src,
                                                          const uint32_t* __restrict__ core_idx, uint64_t k_core,
                                                          PtrArray<float> out, int K) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_core; j += stride) {
        const uint32_t i = __ldg(core_idx + j);
        if (SAME) {
            const float v = __ldg(src.p[0] + i);
#pragma unroll 8
            for (int k = 0; k < K; ++k) __stcs(out.p[k] + j, v);
        } else {
            int k = 0;
            for (; k + 8 <= K; k += 8) {
                float v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = __ldg(src.p[k + q] + i);
#pragma unroll
                for (int q = 0; q < 8; ++q) __stcs(out.p[k + q] + j, v[q]);
            }
            for (; k < K; ++k) __stcs(out.p[k] + j, __ldg(src.p[k] + i));
        }
    }
}

// grid.y = worker.  out[w][k_core + j] = src[w][exp[w][j]].
__global__ void __launch_bounds__(256) gather_explore_kernel(PtrArray<const float> src, PtrArray<const uint32_t> exp,
                                                             uint64_t k_exp, PtrArray<float> out, uint64_t k_core) {
    const uint32_t worker = blockIdx.y;
    const float* __restrict__ s = src.p[worker];
    const uint32_t* __restrict__ e = exp.p[worker];
    float* __restrict__ o = out.p[worker] + k_core;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x * 4;
    for (uint64_t j0 = ((uint64_t)blockIdx.x * blockDim.x) * 4 + threadIdx.x; j0 < k_exp; j0 += stride) {
        uint32_t idx[4];
        float v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            if (j < k_exp) idx[q] = __ldg(e + j);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            if (j < k_exp) v[q] = ld_sparse(s + idx[q]);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            if (j < k_exp) __stcs(o + j, v[q]);
        }
    }
}

// Worker-side Merge (Algorithm 1; Section 3.3 step 5): the pulled values replace the local
// model's values on the communication set.  Core segment: the shared key is read once and
// serves all K workers.
__global__ void __launch_bounds__(256) worker_merge_core_kernel(PtrArray<float> w_local,
                                                                const uint32_t* __restrict__ core_idx,
                                                                uint64_t k_core, PtrArray<const float> pulled,
                                                                int K) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_core; j += stride) {
        const uint32_t i = __ldg(core_idx + j);
        int k = 0;
        for (; k + 8 <= K; k += 8) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = __ldcs(pulled.p[k + q] + j);
#pragma unroll
            for (int q = 0; q < 8; ++q) w_local.p[k + q][i] = v[q];
        }
        for (; k < K; ++k) w_local.p[k][i] = __ldcs(pulled.p[k] + j);
    }
}

// Explorer segments: grid.y = worker.
__global__ void __launch_bounds__(256) worker_merge_explore_kernel(PtrArray<float> w_local,
                                                                   PtrArray<const uint32_t> exp, uint64_t k_exp,
                                                                   PtrArray<const float> pulled, uint64_t k_core) {
    const uint32_t worker = blockIdx.y;
    float* __restrict__ w = w_local.p[worker];
    const uint32_t* __restrict__ e = exp.p[worker];
    const float* __restrict__ v = pulled.p[worker] + k_core;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_exp; j += stride)
        w[__ldg(e + j)] = __ldcs(v + j);
}

}  // namespace

slimdp_status launch_worker_merge(const PtrArray<float>& w_local, uint32_t workers, const uint32_t* core_idx,
                                  uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                                  const PtrArray<const float>& pulled, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    if (k_core > 0) {
        uint64_t grid = (k_core + 255) / 256;
        if (grid > (uint64_t)sms * 32) grid = (uint64_t)sms * 32;
        worker_merge_core_kernel<<<(unsigned)grid, 256, 0, st>>>(w_local, core_idx, k_core, pulled, (int)workers);
        SLIMDP_LAUNCHED(1);
    }
    if (k_exp > 0) {
        uint64_t grid = (k_exp + 255) / 256;
        const uint64_t cap = ((uint64_t)sms * 32 + workers - 1) / workers;
        if (grid > cap) grid = cap;
        worker_merge_explore_kernel<<<dim3((unsigned)grid, workers), 256, 0, st>>>(w_local, exp, k_exp, pulled, k_core);
        SLIMDP_LAUNCHED(1);
    }
    return SLIMDP_OK;
}

slimdp_status launch_gather(const PtrArray<const float>& src, bool same_src, uint32_t workers,
                            const uint32_t* core_idx, uint64_t k_core, const PtrArray<const uint32_t>& exp,
                            uint64_t k_exp, const PtrArray<float>& out, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    if (k_core > 0) {
        uint64_t grid = (k_core + 255) / 256;
        if (grid > (uint64_t)sms * 32) grid = (uint64_t)sms * 32;
        if (same_src)
            gather_core_kernel<true><<<(unsigned)grid, 256, 0, st>>>(src, core_idx, k_core, out, (int)workers);
        else
            gather_core_kernel<false><<<(unsigned)grid, 256, 0, st>>>(src, core_idx, k_core, out, (int)workers);
        SLIMDP_LAUNCHED(1);
    }
    if (k_exp > 0) {
        uint64_t grid = (k_exp + 1023) / 1024;
        const uint64_t cap = ((uint64_t)sms * 32 + workers - 1) / workers;
        if (grid > cap) grid = cap;
        gather_explore_kernel<<<dim3((unsigned)grid, workers), 256, 0, st>>>(src, exp, k_exp, out, k_core);
        SLIMDP_LAUNCHED(1);
    }
    return SLIMDP_OK;
}

}  // namespace slimdp
