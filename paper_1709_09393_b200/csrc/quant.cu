// 8-bit codes for the pushed values.  Section 2.2 closes with the remark that the method can be
// combined with quantisation of what is sent; the paper defines no quantiser, so the library fixes a
// deterministic one: the packed buffer of a worker (core values, then explorer values) is cut into
// buckets of SLIMDP_Q8_BUCKET consecutive entries; a bucket's scale is its largest finite magnitude;
// a value v becomes the signed code rint(v * (127 / scale)) clamped to [-127, 127] (fp32 division,
// fp32 product, ties to even), 0 if the scale is 0 or v is a NaN, +-127 for an infinity.  The
// receiver reads code * (scale / 127).
//
// slimdp_pack_q8_batched is the extraction of Section 3.5 with that quantiser folded into its
// stores: one CTA per bucket and worker gathers the bucket's values, reduces their magnitudes and
// writes codes and scale; the fp32 packed buffer never exists.
#include <float.h>

#include "common.cuh"

namespace slimdp {

namespace {

static_assert(kQ8Bucket == 256, "one thread per entry of a bucket");

__global__ void __launch_bounds__(kQ8Bucket) pack_q8_kernel(PtrArray<const float> delta,
                                                            const uint32_t* __restrict__ core_idx, uint64_t k_core,
                                                            PtrArray<const uint32_t> exp, uint64_t k_exp,
                                                            PtrArray<int8_t> codes, PtrArray<float> scales) {
    __shared__ float warp_max[kQ8Bucket / 32];
    const uint32_t worker = blockIdx.y;
    const uint64_t j = (uint64_t)blockIdx.x * kQ8Bucket + threadIdx.x;
    const uint64_t m = k_core + k_exp;
    float v = 0.0f;
    if (j < m) {
        const uint32_t i = (j < k_core) ? __ldg(core_idx + j) : __ldg(exp.p[worker] + (j - k_core));
        v = __ldg(delta.p[worker] + i);
    }
    float a = fabsf(v);
    if (!(a <= FLT_MAX)) a = 0.0f;   // NaNs and infinities do not set the scale
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, d));
    if ((threadIdx.x & 31u) == 0) warp_max[threadIdx.x >> 5] = a;
    __syncthreads();
    float amax = warp_max[0];
#pragma unroll
    for (int x = 1; x < kQ8Bucket / 32; ++x) amax = fmaxf(amax, warp_max[x]);
    if (threadIdx.x == 0) scales.p[worker][blockIdx.x] = amax;
    if (j < m) {
        const float inv = (amax > 0.0f) ? __fdiv_rn(127.0f, amax) : 0.0f;
        float q;
        if (v != v)
            q = 0.0f;
        else if (fabsf(v) > FLT_MAX)
            q = (v > 0.0f) ? 127.0f : -127.0f;   // an infinity, whatever the scale
        else
            q = fminf(fmaxf(rintf(__fmul_rn(v, inv)), -127.0f), 127.0f);
        codes.p[worker][j] = (int8_t)q;
    }
}

}  // namespace

slimdp_status launch_pack_q8(const PtrArray<const float>& delta, uint32_t K, const uint32_t* core_idx,
                             uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                             const PtrArray<int8_t>& codes, const PtrArray<float>& scales, cudaStream_t st) {
    const uint64_t m = k_core + k_exp;
    if (m == 0) return SLIMDP_OK;
    const uint64_t buckets = (m + kQ8Bucket - 1) / kQ8Bucket;
    pack_q8_kernel<<<dim3((unsigned)buckets, K), kQ8Bucket, 0, st>>>(delta, core_idx, k_core, exp, k_exp, codes, scales);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
