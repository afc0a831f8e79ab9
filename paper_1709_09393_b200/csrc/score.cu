// slimdp_score: significance S_i = |w_i| + c |g_i| (Eq. 1, Section 3.2) as one
// streaming pass: 128-bit loads of w and of the K updates, fp32 left-to-right
// sum over workers, one fused multiply-add, 128-bit store.
#include <math.h>

#include "common.cuh"

namespace slimdp {

namespace {

// KT > 0: K known at compile time (all loads of one element group are issued
// before the first add).  KT == 0: K from the argument.
template <int KT>
__global__ void __launch_bounds__(256) score_vec4_kernel(const float4* __restrict__ w, PtrArray<const float> g,
                                                         int K, float c, uint64_t n4, uint64_t n,
                                                         float4* __restrict__ S) {
    const int kk = (KT > 0) ? KT : K;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 a = __ldcs(reinterpret_cast<const float4*>(g.p[0]) + i);
        if (KT > 0) {
            float4 b[KT > 1 ? KT - 1 : 1];
#pragma unroll
            for (int k = 1; k < KT; ++k) b[k - 1] = __ldcs(reinterpret_cast<const float4*>(g.p[k]) + i);
#pragma unroll
            for (int k = 1; k < KT; ++k) {
                a.x = __fadd_rn(a.x, b[k - 1].x);
                a.y = __fadd_rn(a.y, b[k - 1].y);
                a.z = __fadd_rn(a.z, b[k - 1].z);
                a.w = __fadd_rn(a.w, b[k - 1].w);
            }
        } else {
#pragma unroll 4
            for (int k = 1; k < kk; ++k) {
                float4 b = __ldcs(reinterpret_cast<const float4*>(g.p[k]) + i);
                a.x = __fadd_rn(a.x, b.x);
                a.y = __fadd_rn(a.y, b.y);
                a.z = __fadd_rn(a.z, b.z);
                a.w = __fadd_rn(a.w, b.w);
            }
        }
        float4 ww = __ldcs(w + i);
        float4 s;
        s.x = score_one(c, a.x, ww.x);
        s.y = score_one(c, a.y, ww.y);
        s.z = score_one(c, a.z, ww.z);
        s.w = score_one(c, a.w, ww.w);
        S[i] = s;
    }
    // ragged tail (n % 4 elements)
    if (blockIdx.x == 0 && threadIdx.x < (uint32_t)(n - 4 * n4)) {
        const uint64_t i = 4 * n4 + threadIdx.x;
        const float* ws = reinterpret_cast<const float*>(w);
        float a = g.p[0][i];
        for (int k = 1; k < kk; ++k) a = __fadd_rn(a, g.p[k][i]);
        reinterpret_cast<float*>(S)[i] = score_one(c, a, ws[i]);
    }
}

// Any 4-byte alignment.
__global__ void __launch_bounds__(256) score_scalar_kernel(const float* __restrict__ w, PtrArray<const float> g,
                                                           int K, float c, uint64_t n, float* __restrict__ S) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        float a = g.p[0][i];
        for (int k = 1; k < K; ++k) a = __fadd_rn(a, g.p[k][i]);
        S[i] = score_one(c, a, w[i]);
    }
}

// Dense push at a reselection boundary (Algorithm 1: Push(delta) when (t + 1) % q == 0, then
// Update, then Core-Selection on the updated model with the updates just pushed): one streaming
// pass applies every worker's whole update in worker order and, if S is given, scores the result.
template <bool VEC>
__global__ void __launch_bounds__(256) dense_merge_score_kernel(float* __restrict__ w, PtrArray<const float> g, int K,
                                                                float neg_eta, float c, uint64_t n,
                                                                float* __restrict__ S) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    if (VEC) {
        const uint64_t n4 = n / 4;
        float4* w4 = reinterpret_cast<float4*>(w);
        for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
            float4 x = w4[i];
            float4 a = __ldcs(reinterpret_cast<const float4*>(g.p[0]) + i);
            x.x = __fmaf_rn(neg_eta, a.x, x.x);
            x.y = __fmaf_rn(neg_eta, a.y, x.y);
            x.z = __fmaf_rn(neg_eta, a.z, x.z);
            x.w = __fmaf_rn(neg_eta, a.w, x.w);
#pragma unroll 4
            for (int k = 1; k < K; ++k) {
                const float4 b = __ldcs(reinterpret_cast<const float4*>(g.p[k]) + i);
                a.x = __fadd_rn(a.x, b.x);
                a.y = __fadd_rn(a.y, b.y);
                a.z = __fadd_rn(a.z, b.z);
                a.w = __fadd_rn(a.w, b.w);
                x.x = __fmaf_rn(neg_eta, b.x, x.x);
                x.y = __fmaf_rn(neg_eta, b.y, x.y);
                x.z = __fmaf_rn(neg_eta, b.z, x.z);
                x.w = __fmaf_rn(neg_eta, b.w, x.w);
            }
            x.x = stored_model_value(x.x);
            x.y = stored_model_value(x.y);
            x.z = stored_model_value(x.z);
            x.w = stored_model_value(x.w);
            w4[i] = x;
            if (S) {
                float4 s;
                s.x = score_one(c, a.x, x.x);
                s.y = score_one(c, a.y, x.y);
                s.z = score_one(c, a.z, x.z);
                s.w = score_one(c, a.w, x.w);
                reinterpret_cast<float4*>(S)[i] = s;
            }
        }
    }
    // scalar path: everything when not vectorised, else the ragged tail
    const uint64_t first = VEC ? (n / 4) * 4 : 0;
    for (uint64_t i = first + (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        float x = w[i];
        float a = g.p[0][i];
        x = __fmaf_rn(neg_eta, a, x);
        for (int k = 1; k < K; ++k) {
            const float b = g.p[k][i];
            a = __fadd_rn(a, b);
            x = __fmaf_rn(neg_eta, b, x);
        }
        x = stored_model_value(x);
        w[i] = x;
        if (S) S[i] = score_one(c, a, x);
    }
}

}  // namespace

slimdp_status launch_dense_merge_score(float* w, const PtrArray<const float>& g, uint32_t K, float eta, float c,
                                       uint64_t n, float* S, bool vec, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    uint64_t blocks = ((vec ? n / 4 : n) + 255) / 256;
    if (blocks > (uint64_t)sms * 32) blocks = (uint64_t)sms * 32;
    if (blocks == 0) blocks = 1;
    if (vec)
        dense_merge_score_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(w, g, (int)K, -eta, c, n, S);
    else
        dense_merge_score_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(w, g, (int)K, -eta, c, n, S);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

slimdp_status launch_score(const float* w, const PtrArray<const float>& g, uint32_t K, float c, uint64_t n,
                           float* S, bool vec, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    if (!vec) {
        uint64_t blocks = (n + 255) / 256;
        if (blocks > (uint64_t)sms * 32) blocks = (uint64_t)sms * 32;
        score_scalar_kernel<<<(unsigned)blocks, 256, 0, st>>>(w, g, (int)K, c, n, S);
        SLIMDP_LAUNCHED(1);
        return SLIMDP_OK;
    }
    const uint64_t n4 = n / 4;
    uint64_t blocks = (n4 + 255) / 256;
    if (blocks > (uint64_t)sms * 32) blocks = (uint64_t)sms * 32;
    if (blocks == 0) blocks = 1;
    const float4* w4 = reinterpret_cast<const float4*>(w);
    float4* S4 = reinterpret_cast<float4*>(S);
#define SLIMDP_SCORE_CASE(KK)                                                                        \
    case KK:                                                                                         \
        score_vec4_kernel<KK><<<(unsigned)blocks, 256, 0, st>>>(w4, g, (int)K, c, n4, n, S4);        \
        break;
    switch (K) {
        SLIMDP_SCORE_CASE(1)
        SLIMDP_SCORE_CASE(2)
        SLIMDP_SCORE_CASE(4)
        SLIMDP_SCORE_CASE(8)
        SLIMDP_SCORE_CASE(16)
        default:
            score_vec4_kernel<0><<<(unsigned)blocks, 256, 0, st>>>(w4, g, (int)K, c, n4, n, S4);
    }
#undef SLIMDP_SCORE_CASE
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
