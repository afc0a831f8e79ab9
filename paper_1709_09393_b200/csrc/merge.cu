// slimdp_merge: the server update of Section 3.3 step 3,
// w <- w - eta' * T_C(delta_k) for every worker, applied in ascending worker
// order so that the fp32 result is unique; and slimdp_exchange, which does the
// push (extraction), that update and the pull (Section 3.3 step 4) in one pass.
//
// Core segment: one thread owns one core parameter and folds the K pushed
// values into it in worker order (K coalesced value streams, one gather and
// one scatter).
// Explorer segments: different workers' explorers may contain the same
// parameter (never a core one), so the order across workers matters.  The
// parameter vector is cut into ranges; one warp owns one range, finds each
// worker's entries inside it by binary search of the ascending index lists,
// and applies worker 0's entries, a warp barrier, worker 1's entries, ...
// Inside one worker the indices are distinct, and no other warp touches the
// range, so a parameter receives its updates in ascending k without atomics.
#include "common.cuh"
#include "layout.cuh"
#include "select_dev.cuh"

namespace slimdp {

namespace {

constexpr int kMergeWarps = 8;

// Where the pushed values come from: fp32 buffers as slimdp_pack writes them, or 8-bit codes with
// one fp32 scale per bucket of kQ8Bucket packed entries (value = code * (scale / 127), fp32).
struct F32Vals {
    PtrArray<const float> p;
    __device__ __forceinline__ float get(int k, uint64_t j) const { return __ldcs(p.p[k] + j); }
};
struct Q8Vals {
    PtrArray<const int8_t> codes;
    PtrArray<const float> scales;
    __device__ __forceinline__ float get(int k, uint64_t j) const {
        const float step = __fdiv_rn(__ldg(scales.p[k] + j / kQ8Bucket), 127.0f);
        return __fmul_rn((float)__ldg(codes.p[k] + j), step);
    }
};

template <typename Vals>
__global__ void __launch_bounds__(256) merge_core_kernel(float* __restrict__ w, const uint32_t* __restrict__ core_idx,
                                                         uint64_t k_core, Vals val, int K, float neg_eta) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_core; j += stride) {
        const uint32_t i = __ldg(core_idx + j);
        float x = w[i];
        int k = 0;
        for (; k + 8 <= K; k += 8) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = val.get(k + q, j);
#pragma unroll
            for (int q = 0; q < 8; ++q) x = __fmaf_rn(neg_eta, v[q], x);
        }
        for (; k < K; ++k) x = __fmaf_rn(neg_eta, val.get(k, j), x);
        w[i] = stored_model_value(x);
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

// bound[k][r]: where the r-th of the CTA's 9 range boundaries falls in worker k's index list.
__device__ __forceinline__ void find_bounds(uint32_t (*bound)[kMergeWarps + 1], const PtrArray<const uint32_t>& exp,
                                            uint32_t k_exp, int K, uint32_t range_shift, uint64_t vblock) {
    const uint64_t first = (vblock * kMergeWarps) << range_shift;
    for (int t = threadIdx.x; t < K * (kMergeWarps + 1); t += blockDim.x) {
        const int k = t / (kMergeWarps + 1), r = t % (kMergeWarps + 1);
        bound[k][r] = lower_bound(exp.p[k], k_exp, first + ((uint64_t)r << range_shift));
    }
    __syncthreads();
}

// Sparse 4-byte accesses: ask L2 for the smallest fetch it offers (64 B) instead of a whole 128-byte line.
__device__ __forceinline__ float ld_sparse(const float* p) {
    float v;
    asm volatile("ld.global.L2::64B.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}
// Early request of a location that a later phase reads: a real load whose value is only
// folded into a sink.  The caller folds a whole batch after issuing it, so that the loads of a
// batch are all in flight together.
__device__ __forceinline__ uint32_t touch(const float* p) {
    uint32_t v;
    asm volatile("ld.global.L2::64B.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Requests, for every worker, the model values (and, if delta is given, the update values) of
// this warp's range ahead of the ordered phases: 8 workers' loads are issued back to back.
template <bool WITH_DELTA>
__device__ __forceinline__ uint32_t touch_range(const float* w, const PtrArray<const uint32_t>& exp,
                                                const PtrArray<const float>& delta,
                                                uint32_t (*bound)[kMergeWarps + 1], int K, uint32_t wid,
                                                uint32_t lane) {
    uint32_t sink = 0;
    for (int k0 = 0; k0 < K; k0 += 8) {
        uint32_t i[8], v[16];
        bool ok[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int k = k0 + q;
            const uint32_t e = (k < K) ? bound[k][wid] + lane : 0u;
            ok[q] = k < K && e < bound[k][wid + 1];
            i[q] = ok[q] ? __ldg(exp.p[k] + e) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            v[2 * q] = ok[q] ? touch(w + i[q]) : 0u;
            v[2 * q + 1] = (WITH_DELTA && ok[q]) ? touch(delta.p[k0 + q] + i[q]) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) sink ^= v[q];
        // the rare worker with more than 32 entries in this range
        for (int q = 0; q < 8 && k0 + q < K; ++q) {
            const int k = k0 + q;
            const uint32_t b = bound[k][wid + 1];
            for (uint32_t e = bound[k][wid] + lane + 32; e < b; e += 32) {
                const uint32_t j = __ldg(exp.p[k] + e);
                sink ^= touch(w + j);
                if (WITH_DELTA) sink ^= touch(delta.p[k] + j);
            }
        }
    }
    return sink;
}

// One CTA owns 8 consecutive ranges of 2^range_shift parameters, one per warp.  Every warp, on
// its own, first requests all lines it is going to touch (L2 prefetch), then applies worker 0's
// entries of its range, a warp barrier, worker 1's entries, ...
template <typename Vals>
__global__ void __launch_bounds__(kMergeWarps * 32) merge_explore_kernel(float* w, PtrArray<const uint32_t> exp,
                                                                         uint32_t k_exp, Vals val, uint64_t k_core,
                                                                         int K, float neg_eta, uint32_t range_shift) {
    __shared__ uint32_t bound[SLIMDP_MAX_WORKERS][kMergeWarps + 1];
    find_bounds(bound, exp, k_exp, K, range_shift, blockIdx.x);
    const uint32_t wid = threadIdx.x >> 5, lane = lane_id();
    PtrArray<const float> none;
    const uint32_t sink = touch_range<false>(w, exp, none, bound, K, wid, lane);
    for (int k = 0; k < K; ++k) {
        const uint32_t* __restrict__ idx = exp.p[k];
        const uint32_t b = bound[k][wid + 1];
        for (uint32_t e = bound[k][wid] + lane; e < b; e += 32) {
            const uint32_t i = __ldg(idx + e);
            w[i] = stored_model_value(__fmaf_rn(neg_eta, val.get(k, k_core + e), ld_sparse(w + i)));
        }
        __syncwarp();   // worker k's updates are visible to the whole warp before worker k+1 starts
    }
    if (sink == 0x9E3779B9u && lane >= 32) w[0] = 0.0f;   // never true: keeps the early requests alive
}

// ---- push + server update + pull in one pass (slimdp_exchange) -----------------------------

// Core segment: thread j gathers the K workers' updates of core parameter core_idx[j] (the
// push), folds them into the parameter in worker order (the update) and hands the merged value
// back to all K workers (the pull).  One read of the key, K gathers, one read-modify-write.
// The gathers ask for 64-byte fetches: where the core is dense both halves of a line are asked
// for anyway, where it is thin (one member per line) half the line stays in DRAM.
// One core parameter: i its index, j its place in the core.
__device__ __forceinline__ void exchange_core_one(float* __restrict__ w, uint32_t i, uint64_t j,
                                                  const PtrArray<const float>& delta, const PtrArray<float>& val,
                                                  const PtrArray<float>& pulled, int K, float neg_eta) {
    float x = ld_sparse(w + i);
    int k = 0;
    for (; k + 8 <= K; k += 8) {
        float v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = ld_sparse(delta.p[k + q] + i);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            __stcs(val.p[k + q] + j, v[q]);
            x = __fmaf_rn(neg_eta, v[q], x);
        }
    }
    for (; k < K; ++k) {
        const float v = ld_sparse(delta.p[k] + i);
        __stcs(val.p[k] + j, v);
        x = __fmaf_rn(neg_eta, v, x);
    }
    x = stored_model_value(x);
    w[i] = x;
#pragma unroll 8
    for (int q = 0; q < K; ++q) __stcs(pulled.p[q] + j, x);
}

__device__ __forceinline__ void exchange_core_body(float* __restrict__ w, const uint32_t* __restrict__ core_idx,
                                                   uint64_t k_core, const PtrArray<const float>& delta,
                                                   const PtrArray<float>& val, const PtrArray<float>& pulled, int K,
                                                   float neg_eta, uint64_t vblock, uint64_t vgrid) {
    const uint64_t stride = vgrid * blockDim.x;
    for (uint64_t j = vblock * blockDim.x + threadIdx.x; j < k_core; j += stride)
        exchange_core_one(w, __ldg(core_idx + j), j, delta, val, pulled, K, neg_eta);
}

// Explorer segments: warp-owned ranges as in merge_explore_kernel.  Per worker, in ascending
// order, the warp gathers the worker's updates inside its range, stores them as the pushed
// values and applies them; after the last worker it reads the merged values back for every
// worker's pull (they are still in cache).
__device__ __forceinline__ void exchange_explore_body(float* w, const PtrArray<const uint32_t>& exp, uint32_t k_exp,
                                                      const PtrArray<const float>& delta, const PtrArray<float>& val,
                                                      const PtrArray<float>& pulled, uint64_t k_core, int K,
                                                      float neg_eta, uint32_t range_shift, uint64_t vblock,
                                                      uint32_t (*bound)[kMergeWarps + 1]) {
    find_bounds(bound, exp, k_exp, K, range_shift, vblock);
    const uint32_t wid = threadIdx.x >> 5, lane = lane_id();
    const uint32_t sink = touch_range<true>(w, exp, delta, bound, K, wid, lane);
    for (int k = 0; k < K; ++k) {
        const uint32_t* __restrict__ idx = exp.p[k];
        const float* __restrict__ d = delta.p[k];
        float* __restrict__ v = val.p[k] + k_core;
        const uint32_t b = bound[k][wid + 1];
        for (uint32_t e = bound[k][wid] + lane; e < b; e += 32) {
            const uint32_t i = __ldg(idx + e);
            const float u = ld_sparse(d + i);
            __stcs(v + e, u);
            w[i] = stored_model_value(__fmaf_rn(neg_eta, u, ld_sparse(w + i)));
        }
        __syncwarp();   // worker k's updates are visible to the whole warp before worker k+1 starts
    }
    for (int k = 0; k < K; ++k) {
        const uint32_t* __restrict__ idx = exp.p[k];
        float* __restrict__ o = pulled.p[k] + k_core;
        const uint32_t b = bound[k][wid + 1];
        for (uint32_t e = bound[k][wid] + lane; e < b; e += 32) __stcs(o + e, ld_sparse(w + __ldg(idx + e)));
    }
    if (sink == 0x9E3779B9u && lane >= 32) w[0] = 0.0f;   // never true: keeps the early requests alive
}

// ---- explorer segments straight from the sorted ranks ---------------------------------------
//
// A worker's explorer is { select0(r) : r in its sorted ranks }, select0(r) the r-th parameter
// outside the core.  A warp that owns the parameter range [a, a + 2^shift) owns exactly the ranks
// in [dir(a), dir(a + 2^shift)), dir(x) the number of non-core parameters below x, which the
// core's directory holds for every multiple of 64.  Inside the range select0 is local: the
// range's directory entries (one per lane, at most 32 groups of 64 parameters) and bitmap words
// (two per lane) are all it needs.  So the warp turns its ranks into indices itself, writes them
// out as the explorer (ascending, since the ranks are) and goes on as exchange_explore_body; the
// separate pass that turns all ranks into indices, and the wait for it, fall away.
struct RankSource {
    const uint32_t* ranks;    // worker k's sorted ranks at ranks + k * stride
    uint64_t stride;
    const uint32_t* bitmap;   // core bitmap, 32 words per 1024-parameter block
    const uint32_t* dir;      // dir[d] = non-core parameters below 64 d, d <= nd; dir[nd] = n - k_core
    uint32_t nd;
    int32_t* status;          // the explorer workspace's status word
};

// First position in a[0, len) whose value is >= x (plain loads: `a` may have been written by this grid's predecessor only).
__device__ __forceinline__ uint32_t lower_bound_ranks(const uint32_t* __restrict__ a, uint32_t len, uint32_t x) {
    uint32_t lo = 0, hi = len;
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if (__ldg(a + mid) < x)
            lo = mid + 1;
        else
            hi = mid;
    }
    return lo;
}

// What a warp that owns a parameter range knows about it: lane l holds the range's l-th group of 64
// parameters (dl = non-core parameters below the group, words = its two words of the core bitmap).
struct RangeView {
    uint32_t groups;    // groups in the range, 1 .. 32
    uint32_t group0;    // the range's first group
    uint32_t dl;        // 0xFFFFFFFF: this lane has no group
    uint2 words;
};

__device__ __forceinline__ void explore_ranks_rest(float* w, const RankSource& src, const RangeView& rv,
                                                   const PtrArray<const uint32_t>& exp, uint32_t k_exp,
                                                   const PtrArray<const float>& delta, const PtrArray<float>& val,
                                                   const PtrArray<float>& pulled, uint64_t k_core, int K,
                                                   float neg_eta, uint32_t (*bound)[kMergeWarps + 1]);

__device__ __forceinline__ void exchange_explore_ranks_body(float* w, const RankSource& src,
                                                            const PtrArray<const uint32_t>& exp, uint32_t k_exp,
                                                            const PtrArray<const float>& delta,
                                                            const PtrArray<float>& val, const PtrArray<float>& pulled,
                                                            uint64_t k_core, int K, float neg_eta,
                                                            uint32_t range_shift, uint64_t vblock,
                                                            uint32_t (*bound)[kMergeWarps + 1]) {
    const uint32_t wid = threadIdx.x >> 5, lane = lane_id();
    const uint32_t groups = 1u << (range_shift - 6);   // 64-parameter groups per warp range, 1 .. 32
    const uint64_t first_group = (vblock * kMergeWarps) << (range_shift - 6);
    // where the CTA's 9 range boundaries fall in every worker's sorted ranks
    for (int t = threadIdx.x; t < K * (kMergeWarps + 1); t += blockDim.x) {
        const int k = t / (kMergeWarps + 1), r = t % (kMergeWarps + 1);
        const uint64_t d = first_group + (uint64_t)r * groups;
        const uint32_t rank_lo = __ldg(src.dir + (d < src.nd ? d : src.nd));
        bound[k][r] = lower_bound_ranks(src.ranks + (uint64_t)k * src.stride, k_exp, rank_lo);
    }
    __syncthreads();
    // this warp's piece of the directory and of the bitmap: lane l holds group l of the range
    const uint64_t my_group = first_group + (uint64_t)wid * groups + lane;
    const bool have_group = lane < groups && my_group < src.nd;
    RangeView rv;
    rv.groups = groups;
    rv.group0 = (uint32_t)(first_group + (uint64_t)wid * groups);
    rv.dl = have_group ? __ldg(src.dir + my_group) : 0xFFFFFFFFu;
    rv.words = have_group ? __ldg(reinterpret_cast<const uint2*>(src.bitmap) + my_group) : make_uint2(0u, 0u);
    explore_ranks_rest(w, src, rv, exp, k_exp, delta, val, pulled, k_core, K, neg_eta, bound);
}

__device__ __forceinline__ void explore_ranks_rest(float* w, const RankSource& src, const RangeView& rv,
                                                   const PtrArray<const uint32_t>& exp, uint32_t k_exp,
                                                   const PtrArray<const float>& delta, const PtrArray<float>& val,
                                                   const PtrArray<float>& pulled, uint64_t k_core, int K,
                                                   float neg_eta, uint32_t (*bound)[kMergeWarps + 1]) {
    const uint32_t wid = threadIdx.x >> 5, lane = lane_id();
    const uint32_t groups = rv.groups;
    const uint32_t dl = rv.dl;
    const uint2 words = rv.words;
    const uint32_t group0 = rv.group0;
    bool bad = false;
    // rank -> parameter index inside this warp's range; every lane takes part (shuffles), `ok` says
    // whether the lane's rank is real
    auto select0_local = [&](uint32_t r, bool ok) -> uint32_t {
        uint32_t lo = 0, hi = groups - 1;   // largest group g with dl[g] <= r
#pragma unroll
        for (int step = 0; step < 5; ++step) {
            const uint32_t mid = lo + ((hi - lo + 1) >> 1);
            const uint32_t v = __shfl_sync(0xFFFFFFFFu, dl, (int)mid);
            if (lo < hi) {
                if (v <= r)
                    lo = mid;
                else
                    hi = mid - 1;
            }
        }
        const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, dl, (int)lo);
        const uint32_t w0 = __shfl_sync(0xFFFFFFFFu, words.x, (int)lo);
        const uint32_t w1 = __shfl_sync(0xFFFFFFFFu, words.y, (int)lo);
        const uint32_t rem = r - d0;
        const uint32_t z0 = ~w0, z1 = ~w1;
        const uint32_t c0 = __popc(z0);
        const bool second = rem >= c0;
        const uint32_t z = second ? z1 : z0;
        const uint32_t rr = second ? rem - c0 : rem;
        // the directory and the bitmap disagree, or the rank does not belong to this range
        if (ok && (r < d0 || rr >= (uint32_t)__popc(z))) bad = true;
        return (group0 + lo) * 64u + (second ? 32u : 0u) + nth_set_bit(z, (ok && !bad) ? rr : 0u);
    };
    // indices of every worker's entries in the range, written out as the explorer; early requests of
    // the model and update values they name, 8 workers' worth in flight together
    uint32_t sink = 0;
    for (int k0 = 0; k0 < K; k0 += 8) {
        uint32_t i[8], v[16];
        bool ok[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int k = k0 + q;
            ok[q] = false;
            i[q] = 0;
            if (k < K) {   // warp-uniform
                const uint32_t e = bound[k][wid] + lane;
                ok[q] = e < bound[k][wid + 1];
                const uint32_t r = ok[q] ? __ldg(src.ranks + (uint64_t)k * src.stride + e) : 0u;
                i[q] = select0_local(r, ok[q]);
                ok[q] = ok[q] && !bad;
                if (ok[q]) const_cast<uint32_t*>(exp.p[k])[e] = i[q];
            }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            v[2 * q] = ok[q] ? touch(w + i[q]) : 0u;
            v[2 * q + 1] = ok[q] ? touch(delta.p[k0 + q] + i[q]) : 0u;
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) sink ^= v[q];
        // the rare worker with more than 32 entries in this range
        for (int q = 0; q < 8 && k0 + q < K; ++q) {
            const int k = k0 + q;
            const uint32_t hi = bound[k][wid + 1];
            for (uint32_t e0 = bound[k][wid] + 32; e0 < hi; e0 += 32) {   // warp-uniform bounds
                const uint32_t e = e0 + lane;
                const bool more = e < hi;
                const uint32_t r = more ? __ldg(src.ranks + (uint64_t)k * src.stride + e) : 0u;
                const uint32_t j = select0_local(r, more);
                if (more && !bad) {
                    const_cast<uint32_t*>(exp.p[k])[e] = j;
                    sink ^= touch(w + j);
                    sink ^= touch(delta.p[k] + j);
                }
            }
        }
    }
    if (__any_sync(0xFFFFFFFFu, bad)) {
        if (lane == 0) *src.status = SLIMDP_ERR_INTERNAL;
        return;   // the whole warp: nothing of this range is exchanged
    }
    __syncwarp();
    for (int k = 0; k < K; ++k) {
        const uint32_t* idx = exp.p[k];   // plain loads: this thread reads back the entries it wrote itself
        const float* __restrict__ d = delta.p[k];
        float* __restrict__ v = val.p[k] + k_core;
        const uint32_t b = bound[k][wid + 1];
        for (uint32_t e = bound[k][wid] + lane; e < b; e += 32) {
            const uint32_t i = idx[e];
            const float u = ld_sparse(d + i);
            __stcs(v + e, u);
            w[i] = stored_model_value(__fmaf_rn(neg_eta, u, ld_sparse(w + i)));
        }
        __syncwarp();   // worker k's updates are visible to the whole warp before worker k+1 starts
    }
    for (int k = 0; k < K; ++k) {
        const uint32_t* idx = exp.p[k];
        float* __restrict__ o = pulled.p[k] + k_core;
        const uint32_t b = bound[k][wid + 1];
        for (uint32_t e = bound[k][wid] + lane; e < b; e += 32) __stcs(o + e, ld_sparse(w + idx[e]));
    }
    if (sink == 0x9E3779B9u && lane >= 32) w[0] = 0.0f;   // never true: keeps the early requests alive
}

// ---- core segment from the staging area ------------------------------------------------------
//
// In the one-call round the pass over all parameters has set aside, for every parameter that is
// certainly in the core and for every candidate, its index and its K update values (chunks of
// kStageChunk entries, see layout.cuh).  The core segment then streams those chunks instead of
// gathering K + 1 scattered lines per core parameter: the entry's place in the core comes from
// the core's bitmap and directory (a candidate that did not make it has its bit clear and is
// skipped), the K values go out as the pushed values, the model value is read, updated in worker
// order and written back, and the merged value goes to all K workers' pulls.  Entries of one
// chunk are in ascending parameter order, so all of these accesses are runs.
struct StagedSource {
    const uint32_t* fill;      // null: nothing was staged, the core segment gathers
    const uint32_t* chunks;
    uint32_t max_chunks;
    const WsHeader* sel;       // the selection's header: staging is valid only if its bracket held
    uint32_t k, cap;
    const uint32_t* bitmap;    // the core's bitmap and directory (core_aux)
    const uint32_t* dir;
    int32_t* status;
};

__device__ __forceinline__ bool staged_valid(const StagedSource& s) {
    return s.fill != nullptr && s.sel->stage_lost == 0u && bracket_held(s.sel->n_def, s.sel->n_cand, s.k, s.cap);
}

__device__ __forceinline__ void exchange_core_staged_body(float* __restrict__ w, const StagedSource& src,
                                                          uint64_t k_core, const PtrArray<float>& val,
                                                          const PtrArray<float>& pulled, int K, float neg_eta,
                                                          uint32_t chunk) {
    const uint32_t f = __ldg(src.fill + chunk);
    const uint32_t* __restrict__ base = src.chunks + (size_t)chunk * (size_t)(K + 1) * kStageChunk;
    for (uint32_t e = threadIdx.x; e < f; e += blockDim.x) {
        const uint32_t i = __ldcs(base + e);
        const uint32_t d = i >> 6, bit = i & 63u;
        const uint2 words = __ldg(reinterpret_cast<const uint2*>(src.bitmap) + d);
        const uint32_t word = (bit < 32u) ? words.x : words.y;
        if (!((word >> (bit & 31u)) & 1u)) continue;   // a candidate below the threshold
        const uint32_t below = (bit < 32u) ? __popc(words.x & ((1u << bit) - 1u))
                                           : __popc(words.x) + __popc(words.y & ((1u << (bit - 32u)) - 1u));
        const uint64_t j = (uint64_t)d * 64u - __ldg(src.dir + d) + below;   // core parameters below i
        if (j >= k_core) {
            *src.status = SLIMDP_ERR_INTERNAL;
            continue;
        }
        float x = w[i];
        int k = 0;
        for (; k + 8 <= K; k += 8) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = __uint_as_float(__ldcs(base + (size_t)(k + q + 1) * kStageChunk + e));
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                __stcs(val.p[k + q] + j, v[q]);
                x = __fmaf_rn(neg_eta, v[q], x);
            }
        }
        for (; k < K; ++k) {
            const float v = __uint_as_float(__ldcs(base + (size_t)(k + 1) * kStageChunk + e));
            __stcs(val.p[k] + j, v);
            x = __fmaf_rn(neg_eta, v, x);
        }
        x = stored_model_value(x);
        w[i] = x;
#pragma unroll 8
        for (int q = 0; q < K; ++q) __stcs(pulled.p[q] + j, x);
    }
}

// One launch for both segments.  The core segment streams whole lines of the dense layers and is
// bound by DRAM bandwidth; the explorer segments issue sparse accesses and are bound by their
// latency and rate.  CTAs of both kinds are interleaved in the grid (core_ctas of every
// total_ctas, evenly spread), so both kinds are resident together and fill each other's gaps.
// The two segments touch disjoint parameters and disjoint parts of val / pulled.
__global__ void __launch_bounds__(256, 8) exchange_kernel(float* w, const uint32_t* __restrict__ core_idx,
                                                       uint64_t k_core, PtrArray<const uint32_t> exp, uint32_t k_exp,
                                                       PtrArray<const float> delta, PtrArray<float> val,
                                                       PtrArray<float> pulled, int K, float neg_eta,
                                                       uint32_t range_shift, uint64_t core_ctas, uint64_t total_ctas,
                                                       uint64_t gather_ctas, RankSource from_ranks,
                                                       StagedSource staged) {
    __shared__ uint32_t bound[SLIMDP_MAX_WORKERS][kMergeWarps + 1];
    const uint64_t b = blockIdx.x;
    const uint64_t core_before = b * core_ctas / total_ctas;            // core CTAs among blocks [0, b)
    const bool is_core = (b + 1) * core_ctas / total_ctas > core_before;
    if (is_core) {
        // core CTA number core_before: one staged chunk, or one slice of the gather
        if (staged_valid(staged)) {
            if (core_before < staged.max_chunks)
                exchange_core_staged_body(w, staged, k_core, val, pulled, K, neg_eta, (uint32_t)core_before);
        } else if (core_before < gather_ctas) {
            exchange_core_body(w, core_idx, k_core, delta, val, pulled, K, neg_eta, core_before, gather_ctas);
        }
    } else if (from_ranks.ranks != nullptr) {
        // the explorers are not there yet: `exp` is where this launch writes them
        exchange_explore_ranks_body(w, from_ranks, exp, k_exp, delta, val, pulled, k_core, K, neg_eta, range_shift,
                                    b - core_before, bound);
    } else {
        exchange_explore_body(w, exp, k_exp, delta, val, pulled, k_core, K, neg_eta, range_shift, b - core_before,
                              bound);
    }
}

// ---- the one-call round's exchange: no emit before it ------------------------------------------
//
// After the selection's finishing kernel every warp can place a block's core members by itself
// (block_selection: the "greater" / "equal" bitmaps, the per-block counts and their group prefixes).
// Core CTAs own eight blocks spread over the vector, a warp per block: the warp writes the block's part of the
// core bitmap and directory, lists the block's members in shared memory, and then takes them 32 at
// a time through the push, the update and the pull (consecutive places in the core, so the value
// stores are whole lines) and writes the index list as it goes.  Explorer CTAs work as in
// exchange_explore_ranks_body, except that a warp derives its range's piece of the directory and
// bitmap from the same sources instead of reading them: nothing here waits for an emit kernel.
struct RoundSource {
    const uint32_t* G;
    const uint32_t* E;
    const unsigned long long* cnt;
    const unsigned long long* super_pref;
    WsHeader* sel_hdr;
    uint32_t* bitmap;     // written here (core CTAs)
    uint32_t* dir;
    uint32_t* core_idx;
    uint64_t nb;
    uint64_t n;
};

__device__ __forceinline__ void round_core_body(float* __restrict__ w, const RoundSource& rs, uint32_t ties,
                                                uint64_t k_core, const PtrArray<const float>& delta,
                                                const PtrArray<float>& val, const PtrArray<float>& pulled, int K,
                                                float neg_eta, uint64_t cta, uint64_t core_ctas, uint16_t* list) {
    const uint32_t wid = threadIdx.x >> 5, lane = lane_id();
    // the CTA's eight blocks lie an eighth of the vector apart: the core clusters in some layers, and this
    // way every core CTA gets its share of the heavy blocks, all through the launch
    const uint64_t blk = (uint64_t)wid * core_ctas + cta;
    if (blk >= rs.nb) return;
    uint32_t sel, pos0;
    const uint32_t in_block = block_selection(rs.G, rs.E, rs.cnt, rs.super_pref, ties, blk, &sel, &pos0);
    write_block_aux(rs.bitmap, rs.dir, blk, sel, pos0);
    if (in_block == 0) return;
    const uint32_t base = __shfl_sync(0xFFFFFFFFu, pos0, 0);   // core parameters below the block
    uint16_t* mine = list + wid * kBlock;   // the members' offsets in the block, in index order
    const uint32_t first = (uint32_t)(blk * kBlock);
    uint32_t at = pos0 - base;
    for (uint32_t word = sel; word; word &= word - 1, ++at)
        if (at < kBlock) mine[at] = (uint16_t)(lane * 32u + (uint32_t)__ffs(word) - 1u);
    __syncwarp();
    for (uint32_t e = lane; e < in_block; e += 32) {
        const uint64_t j = (uint64_t)base + e;
        if (j >= k_core) {
            rs.sel_hdr->status = SLIMDP_ERR_INTERNAL;
            continue;
        }
        const uint32_t i = first + mine[e];
        rs.core_idx[j] = i;
        exchange_core_one(w, i, j, delta, val, pulled, K, neg_eta);
    }
}

__device__ __forceinline__ void round_explore_body(float* w, const RankSource& src, const RoundSource& rs,
                                                   uint32_t ties, const PtrArray<const uint32_t>& exp, uint32_t k_exp,
                                                   const PtrArray<const float>& delta, const PtrArray<float>& val,
                                                   const PtrArray<float>& pulled, uint64_t k_core, int K,
                                                   float neg_eta, uint32_t range_shift, uint64_t vblock,
                                                   uint32_t (*bound)[kMergeWarps + 1], uint32_t* range_lo) {
    const uint32_t wid = threadIdx.x >> 5, lane = lane_id();
    const uint32_t groups = 1u << (range_shift - 6);   // 64-parameter groups per warp range, 1 .. 32
    const uint64_t group0 = ((vblock * kMergeWarps + wid) << (range_shift - 6));   // this warp's first group
    const uint64_t nd = rs.nb * kDirPerBlock;
    const uint32_t all_noncore = (uint32_t)(rs.n - k_core);
    // the block(s) that hold the range (two only for ranges of 2048 parameters)
    const uint64_t blkA = group0 / kDirPerBlock;
    uint32_t selA = 0, posA = 0, selB = 0, posB = 0;
    if (blkA < rs.nb) block_selection(rs.G, rs.E, rs.cnt, rs.super_pref, ties, blkA, &selA, &posA);
    if (groups > kDirPerBlock && blkA + 1 < rs.nb)
        block_selection(rs.G, rs.E, rs.cnt, rs.super_pref, ties, blkA + 1, &selB, &posB);
    // lane l takes group l of the range: its two words and the core parameters below it
    const uint64_t my_group = group0 + lane;
    const uint32_t in_blk = (uint32_t)(my_group % kDirPerBlock) * 2u;   // first word of the group in its block
    const bool second = my_group / kDirPerBlock != blkA;
    const uint32_t a0 = __shfl_sync(0xFFFFFFFFu, selA, in_blk), a1 = __shfl_sync(0xFFFFFFFFu, selA, in_blk + 1);
    const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, selB, in_blk), b1 = __shfl_sync(0xFFFFFFFFu, selB, in_blk + 1);
    const uint32_t pa = __shfl_sync(0xFFFFFFFFu, posA, in_blk), pb = __shfl_sync(0xFFFFFFFFu, posB, in_blk);
    const bool have_group = lane < groups && my_group < nd;
    RangeView rv;
    rv.groups = groups;
    rv.group0 = (uint32_t)group0;
    rv.words = have_group ? make_uint2(second ? b0 : a0, second ? b1 : a1) : make_uint2(0u, 0u);
    rv.dl = have_group ? (uint32_t)(my_group * 64u) - (second ? pb : pa) : 0xFFFFFFFFu;
    // non-core parameters below the range's first parameter, and below the CTA's last one
    if (lane == 0) range_lo[wid] = have_group ? rv.dl : all_noncore;
    if (wid == kMergeWarps - 1 && lane == groups - 1)
        range_lo[kMergeWarps] =
            have_group ? rv.dl + 64u - (uint32_t)__popc(rv.words.x) - (uint32_t)__popc(rv.words.y) : all_noncore;
    __syncthreads();
    // where the CTA's 9 range boundaries fall in every worker's sorted ranks
    for (int t = threadIdx.x; t < K * (kMergeWarps + 1); t += blockDim.x) {
        const int k = t / (kMergeWarps + 1), r = t % (kMergeWarps + 1);
        bound[k][r] = lower_bound_ranks(src.ranks + (uint64_t)k * src.stride, k_exp, range_lo[r]);
    }
    __syncthreads();
    explore_ranks_rest(w, src, rv, exp, k_exp, delta, val, pulled, k_core, K, neg_eta, bound);
}

__global__ void __launch_bounds__(256) round_exchange_kernel(float* w, uint64_t k_core, PtrArray<const uint32_t> exp,
                                                             uint32_t k_exp, PtrArray<const float> delta,
                                                             PtrArray<float> val, PtrArray<float> pulled, int K,
                                                             float neg_eta, uint32_t range_shift, uint64_t core_ctas,
                                                             uint64_t total_ctas, RankSource from_ranks,
                                                             RoundSource rs) {
    __shared__ uint32_t bound[SLIMDP_MAX_WORKERS][kMergeWarps + 1];
    __shared__ uint32_t range_lo[kMergeWarps + 1];
    __shared__ uint16_t list[kMergeWarps * kBlock];
    if (rs.sel_hdr->abort != 0u) return;   // the finishing kernel gave up (its status word says so)
    const uint32_t ties = rs.sel_hdr->tie_quota;
    const uint64_t b = blockIdx.x;
    const uint64_t core_before = b * core_ctas / total_ctas;            // core CTAs among blocks [0, b)
    const bool is_core = (b + 1) * core_ctas / total_ctas > core_before;
    if (is_core)
        round_core_body(w, rs, ties, k_core, delta, val, pulled, K, neg_eta, core_before, core_ctas, list);
    else
        round_explore_body(w, from_ranks, rs, ties, exp, k_exp, delta, val, pulled, k_core, K, neg_eta, range_shift,
                           b - core_before, bound, range_lo);
}

// Range per warp: a power of two with 16 to 32 entries per worker on average, at least 32 parameters.
uint32_t explore_range_shift(uint64_t n, uint64_t k_exp) {
    uint32_t shift = 5;
    while (shift < 24 && ((k_exp << (shift + 1)) / n) <= 32) ++shift;
    return shift;
}

}  // namespace

template <typename Vals>
static slimdp_status launch_merge_with(float* w, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                                       const PtrArray<const uint32_t>& exp, uint64_t k_exp, const Vals& val, float eta,
                                       cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const float neg_eta = -eta;
    if (k_core > 0) {
        uint64_t grid = (k_core + 255) / 256;
        if (grid > (uint64_t)sms * 32) grid = (uint64_t)sms * 32;
        merge_core_kernel<Vals><<<(unsigned)grid, 256, 0, st>>>(w, core_idx, k_core, val, (int)K, neg_eta);
        SLIMDP_LAUNCHED(1);
    }
    if (k_exp > 0) {
        const uint32_t shift = explore_range_shift(n, k_exp);
        const uint64_t per_cta = (uint64_t)kMergeWarps << shift;
        const uint64_t ctas = (n + per_cta - 1) / per_cta;
        merge_explore_kernel<Vals><<<(unsigned)ctas, kMergeWarps * 32, 0, st>>>(w, exp, (uint32_t)k_exp, val, k_core,
                                                                                (int)K, neg_eta, shift);
        SLIMDP_LAUNCHED(1);
    }
    return SLIMDP_OK;
}

slimdp_status launch_merge(float* w, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                           const PtrArray<const uint32_t>& exp, uint64_t k_exp, const PtrArray<const float>& val,
                           float eta, cudaStream_t st) {
    return launch_merge_with(w, n, K, core_idx, k_core, exp, k_exp, F32Vals{val}, eta, st);
}

slimdp_status launch_merge_q8(float* w, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                              const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                              const PtrArray<const int8_t>& codes, const PtrArray<const float>& scales, float eta,
                              cudaStream_t st) {
    return launch_merge_with(w, n, K, core_idx, k_core, exp, k_exp, Q8Vals{codes, scales}, eta, st);
}

// Whether the exchange can turn sorted ranks into explorer indices itself: a warp's range must be
// made of 1 to 32 whole 64-parameter groups of the core's directory.
bool exchange_takes_ranks(uint64_t n, uint64_t k_exp) {
    if (k_exp == 0) return false;
    const uint32_t shift = explore_range_shift(n, k_exp);
    return shift >= 6 && shift <= 11;
}

// ranks / rank_stride / core_aux_* / explore_status non-null: the explorers `exp` do not exist yet;
// the launch computes them from every worker's sorted ranks and the core's bitmap and directory
// (exchange_takes_ranks must hold) and writes them to `exp`.  stage non-null: the core segment may
// stream the staging area that the selection's pass filled (core_bitmap / core_dir are needed then).
slimdp_status launch_exchange(float* w, uint64_t n, uint32_t K, const PtrArray<const float>& delta,
                              const uint32_t* core_idx, uint64_t k_core, const PtrArray<const uint32_t>& exp,
                              uint64_t k_exp, float eta, const PtrArray<float>& val, const PtrArray<float>& pulled,
                              const uint32_t* ranks, uint64_t rank_stride, const uint32_t* core_bitmap,
                              const uint32_t* core_dir, int32_t* explore_status, const ExchangeStage* stage,
                              cudaStream_t st) {
    static_assert(kMergeWarps * 32 == 256, "both kinds of CTA have 256 threads");
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    uint64_t core_ctas = 0, explore_ctas = 0, gather_ctas = 0;
    uint32_t shift = 0;
    StagedSource staged{};
    if (k_core > 0) {
        gather_ctas = (k_core + 255) / 256;   // one core parameter per thread: short CTAs interleave best
        core_ctas = gather_ctas;
        if (stage != nullptr && stage->fill != nullptr) {
            // which of the two ways the core segment takes is known on the device only (did the
            // selection's bracket hold?): the grid has room for either, the other's CTAs return at once
            staged = StagedSource{stage->fill, stage->chunks, stage->max_chunks, stage->select_hdr, (uint32_t)k_core,
                                  stage->cand_cap, core_bitmap, core_dir, &stage->select_hdr->status};
            if (stage->max_chunks > core_ctas) core_ctas = stage->max_chunks;
        }
    }
    if (k_exp > 0) {
        shift = explore_range_shift(n, k_exp);
        const uint64_t per_cta = (uint64_t)kMergeWarps << shift;
        explore_ctas = (n + per_cta - 1) / per_cta;
    }
    const uint64_t total = core_ctas + explore_ctas;
    if (total == 0) return SLIMDP_OK;
    RankSource src{};
    if (ranks != nullptr) {
        if (!exchange_takes_ranks(n, k_exp)) return SLIMDP_ERR_INTERNAL;
        src = RankSource{ranks, rank_stride, core_bitmap, core_dir, (uint32_t)(num_blocks(n) * kDirPerBlock),
                         explore_status};
    }
    exchange_kernel<<<(unsigned)total, 256, 0, st>>>(w, core_idx, k_core, exp, (uint32_t)k_exp, delta, val, pulled,
                                                     (int)K, -eta, shift, core_ctas, total, gather_ctas, src, staged);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

// Whether slimdp_round can hand the selection's bitmaps and counts straight to the exchange (no emit
// kernel, no separate explorer-index step): the explorers' warp ranges must line up with the directory.
bool round_exchange_applies(uint64_t n, uint64_t k_exp) { return k_exp == 0 || exchange_takes_ranks(n, k_exp); }

slimdp_status launch_round_exchange(float* w, uint64_t n, uint32_t K, const PtrArray<const float>& delta,
                                    uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp, float eta,
                                    const PtrArray<float>& val, const PtrArray<float>& pulled, const uint32_t* ranks,
                                    uint64_t rank_stride, int32_t* explore_status, const uint32_t* G,
                                    const uint32_t* E, const unsigned long long* cnt,
                                    const unsigned long long* super_pref, WsHeader* sel_hdr, uint32_t* core_idx,
                                    uint32_t* core_bitmap, uint32_t* core_dir, cudaStream_t st) {
    if (!round_exchange_applies(n, k_exp)) return SLIMDP_ERR_INTERNAL;
    const uint64_t nb = num_blocks(n);
    const uint64_t core_ctas = (nb + kMergeWarps - 1) / kMergeWarps;
    uint64_t explore_ctas = 0;
    uint32_t shift = 6;
    if (k_exp > 0) {
        shift = explore_range_shift(n, k_exp);
        const uint64_t per_cta = (uint64_t)kMergeWarps << shift;
        explore_ctas = (n + per_cta - 1) / per_cta;
    }
    const uint64_t total = core_ctas + explore_ctas;
    const RankSource src{ranks, rank_stride, core_bitmap, core_dir, (uint32_t)(nb * kDirPerBlock), explore_status};
    const RoundSource rs{G, E, cnt, super_pref, sel_hdr, core_bitmap, core_dir, core_idx, nb, n};
    round_exchange_kernel<<<(unsigned)total, 256, 0, st>>>(w, k_core, exp, (uint32_t)k_exp, delta, val, pulled, (int)K,
                                                           -eta, shift, core_ctas, total, src, rs);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
