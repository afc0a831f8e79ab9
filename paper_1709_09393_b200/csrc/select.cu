// slimdp_select_core: exact top-k_core of the scores (Section 3.2: rank by
// significance, keep the top), ties to the smaller index.
//
// Keys are the scores' 32-bit patterns compared as unsigned integers.  The
// result is defined by the k-th largest key T and the number r of keys equal
// to T that belong to the core (those with the smallest indices).
//
// Large inputs (n >= 2^21) take the bracketed path, which reads the scores once:
//   1. sample (two small kernels): 2^18 keys (sixteen at each of 2^14 evenly spaced places) are copied out and
//      counted by their top 8 bits, then, around the two target ranks, by their
//      top 16 bits; the last CTA of each kernel turns the counts into a
//      bracket of 16-bit bins [b_bot, b_top) that holds T with overwhelming
//      probability;
//   2. bracket pass (one read of all keys): keys in bins >= b_top are
//      certainly in the core and go straight into the "greater" bitmap; keys
//      inside the bracket are copied, with their indices, to a candidate list;
//   3. if the counts prove the bracket right (n_def < k <= n_def + n_cand and
//      the list did not overflow), three radix histogram passes over the
//      candidates alone find T and r exactly, and one pass over the
//      candidates adds them to the "greater" / "equal" bitmaps;
//   4. otherwise the full path below runs (its kernels are always enqueued and
//      return at once when the bracket held), so the result is exact for every input.
// Full path (small inputs, or a failed bracket, e.g. one score value repeated
// millions of times): three most-significant-digit-first histogram passes over
// all keys (12 + 10 + 10 bits), then one classifying pass that writes both bitmaps.
// Both paths end the same way: a two-kernel exclusive scan over per-1024-block
// counts and one pass over the bitmaps that admits the first r equal keys in
// index order and writes the core bitmap, the non-core rank directory and the
// ascending index list (ordered compaction, no atomic cursors, no spinning).
// Each histogram kernel's last CTA (found with an atomic ticket) also locates
// the bin of the wanted rank, so no separate single-CTA launches are needed.
#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

namespace {

constexpr int kHistThreads = 512;
constexpr uint32_t kBins0 = 4096;   // pass 0: bits 31..20
constexpr uint32_t kBins12 = 1024;  // pass 1: bits 19..10, pass 2: bits 9..0

enum Mode : int { kFullAlways = 0, kFullIfBracketFailed = 1, kCandidates = 2 };

__global__ void select_init_kernel(WsHeader* hdr, uint32_t k) {
    hdr->status = SLIMDP_OK;
    hdr->prefix = (k == 0) ? 0xFFFFFFFFu : 0u;   // k = 0: no key is greater than or (with r = 0) admitted at T
    hdr->k_rem = k;
    hdr->ties = 0;
}

// True when the bracket pass proved that T lies inside the bracket and every candidate was stored.
__device__ __forceinline__ bool bracket_ok(const WsHeader* hdr, uint32_t k, uint32_t cap) {
    const uint32_t n_def = hdr->n_def, n_cand = hdr->n_cand;
    return n_def < k && k - n_def <= n_cand && n_cand <= cap;
}

__device__ __forceinline__ bool mode_runs(int mode, const WsHeader* hdr, uint32_t k, uint32_t cap) {
    if (mode == kFullAlways) return true;
    const bool ok = bracket_ok(hdr, k, cap);
    return (mode == kCandidates) ? ok : !ok;
}

// ---- step 1: sample histogram and bracket ------------------------------------------------

// "Last CTA done": every CTA ends with this; it returns true in exactly one CTA, the last to
// arrive, and that CTA then sees all global writes and atomics the others made before arriving.
// The block barrier orders the CTA's own accesses before thread 0's device-wide fence, the
// fence orders them before the ticket.
__device__ __forceinline__ bool last_cta_done(uint32_t* ticket) {
    __shared__ bool last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        last = atomicAdd(ticket, 1u) == gridDim.x - 1;
        __threadfence();
    }
    __syncthreads();
    return last;
}

// The sample rank of T is about r = k * samples / n; the bracket keeps 6 standard deviations
// (+16) of the sample count on each side of it.
__device__ __forceinline__ void bracket_targets(uint32_t k, uint64_t n, long long* lo_target, long long* hi_target) {
    const double samples = (double)(1u << kSampleBits);
    const double p = (double)k / (double)n;
    const double r = p * samples;
    const double margin = 6.0 * sqrt(samples * p * (1.0 - p)) + 16.0;
    *lo_target = (long long)floor(r - margin);
    *hi_target = (long long)ceil(r + margin);
}

// Sample kernel A: 2^18 keys, sixteen at each of 2^14 evenly spaced places, are copied to `sample` and counted by their top 8
// bits (256 coarse bins: shared memory per CTA, then a few global atomics).  The last CTA finds
// the two coarse bins in which the count from the top crosses the two target ranks:
// coarse_x[0] for b_top (highest coarse bin whose inclusive count exceeds lo_target),
// coarse_x[1] for b_bot (highest coarse bin whose inclusive count reaches hi_target);
// 0xFFFFFFFF = no crossing.  coarse_incl[c] = samples in coarse bins >= c is kept for kernel B.
__global__ void __launch_bounds__(1024) sample_coarse_kernel(const uint32_t* __restrict__ keys, uint64_t n,
                                                             uint32_t k, WsHeader* hdr,
                                                             uint32_t* __restrict__ sample,
                                                             uint32_t* __restrict__ coarse_hist,
                                                             uint32_t* __restrict__ coarse_incl) {
    __shared__ unsigned long long smem[33];
    __shared__ uint32_t sh_coarse[256];
    __shared__ long long s_incl[257];
    const uint32_t t = threadIdx.x;
    if (t < 256) sh_coarse[t] = 0;
    __syncthreads();
    // sixteen consecutive keys (one 64-byte piece, the least DRAM hands out) at each of 2^14 evenly spaced places
    const uint32_t j = blockIdx.x * 1024 + t;   // sample number, < 2^18
    const uint32_t key = __ldg(keys + ((((uint64_t)(j >> 4) * (n / 16)) >> (kSampleBits - 4)) << 4) + (j & 15u));
    sample[j] = key;
    atomicAdd(&sh_coarse[key >> 24], 1u);
    __syncthreads();
    if (t < 256 && sh_coarse[t]) atomicAdd(&coarse_hist[t], sh_coarse[t]);
    if (!last_cta_done(&hdr->ticket[6])) return;
    long long lo_target, hi_target;
    bracket_targets(k, n, &lo_target, &hi_target);
    // coarse bins from the top down: thread t < 256 owns coarse bin 255 - t
    unsigned long long total;
    const unsigned long long c = (t < 256) ? __ldcg(coarse_hist + 255 - t) : 0ull;
    const long long c_above = (long long)block_exclusive_scan64<32>(c, smem, &total);
    if (t < 256) s_incl[255 - t] = c_above + (long long)c;
    if (t == 0) {
        s_incl[256] = 0;
        hdr->coarse_x[0] = 0xFFFFFFFFu;
        hdr->coarse_x[1] = 0xFFFFFFFFu;
    }
    __syncthreads();
    if (t < 256) {
        const long long incl = s_incl[t], above = s_incl[t + 1];
        coarse_incl[t] = (uint32_t)incl;
        if (incl > lo_target && above <= lo_target) hdr->coarse_x[0] = t;
        if (incl >= hi_target && above < hi_target) hdr->coarse_x[1] = t;
    }
}

// Sample kernel B: the members of the two crossing coarse bins are counted by their top 16 bits
// (2 x 256 fine bins); the last CTA resolves each crossing to a 16-bit bin:
// b_top = lowest bin b with (samples in bins >= b) <= lo_target, 65536 if there is none;
// b_bot = highest bin b with (samples in bins >= b) >= hi_target, 0 if there is none.
__global__ void __launch_bounds__(1024) sample_fine_kernel(const uint32_t* __restrict__ sample, uint64_t n,
                                                           uint32_t k, WsHeader* hdr,
                                                           uint32_t* __restrict__ fine_hist,
                                                           const uint32_t* __restrict__ coarse_incl) {
    __shared__ unsigned long long smem[33];
    __shared__ uint32_t sh_fine[2][256];
    __shared__ uint32_t s_val[2];
    const uint32_t t = threadIdx.x;
    const uint32_t cx0 = hdr->coarse_x[0], cx1 = hdr->coarse_x[1];
    if (t < 512) sh_fine[t >> 8][t & 255u] = 0;
    __syncthreads();
    const uint32_t key = sample[blockIdx.x * 1024 + t];
    const uint32_t cb = key >> 24, fb = (key >> 16) & 255u;
    if (cb == cx0) atomicAdd(&sh_fine[0][fb], 1u);
    if (cb == cx1) atomicAdd(&sh_fine[1][fb], 1u);
    __syncthreads();
    if (t < 512 && sh_fine[t >> 8][t & 255u]) atomicAdd(&fine_hist[t], sh_fine[t >> 8][t & 255u]);
    if (!last_cta_done(&hdr->ticket[7])) return;
    long long lo_target, hi_target;
    bracket_targets(k, n, &lo_target, &hi_target);
    for (int which = 0; which < 2; ++which) {
        const long long target = which ? hi_target : lo_target;
        const uint32_t cx = which ? cx1 : cx0;
        if (cx == 0xFFFFFFFFu) {
            // no crossing: which = 0: target < 0 (nothing is certain: 65536) or every bin qualifies (0);
            //              which = 1: target above the sample size: every bin may hold T (0)
            if (t == 0) s_val[which] = which ? 0u : ((target < 0) ? 65536u : 0u);
            __syncthreads();
            continue;
        }
        const long long above_cx = (cx == 255) ? 0 : (long long)coarse_incl[cx + 1];
        // fine bins of coarse bin cx from the top down: thread t < 256 owns fine bin cx * 256 + 255 - t
        unsigned long long total;
        const unsigned long long f = (t < 256) ? __ldcg(fine_hist + which * 256 + 255 - t) : 0ull;
        const long long f_above = (long long)block_exclusive_scan64<32>(f, smem, &total);
        if (t == 0) s_val[which] = which ? 0u : (cx + 1) * 256u;   // default when no fine bin of cx qualifies
        __syncthreads();
        if (t < 256) {
            const uint32_t b = cx * 256 + 255 - t;
            const long long incl = above_cx + f_above + (long long)f;
            if (which == 0) {
                if (incl <= target) atomicMin(&s_val[0], b);
            } else {
                if (incl >= target) atomicMax(&s_val[1], b);
            }
        }
        __syncthreads();
    }
    if (t == 0) {
        hdr->b_top = s_val[0];
        hdr->b_bot = s_val[1];
    }
}

// ---- step 2: one pass over all keys ------------------------------------------------------

constexpr uint32_t kFlushAt = 128;             // a warp appends its staged candidates once it holds this many
constexpr uint32_t kStage = kFlushAt + 256;    // staging capacity: below kFlushAt before a quarter block, +256 in it

// Warp per 1024-parameter block, a quarter block (8 words) at a time.  Candidates are staged per
// warp in shared memory and appended to the global list at least kFlushAt at a time, so the
// list cursor sees one atomic per kFlushAt candidates or more.
__global__ void __launch_bounds__(256, 8) bracket_pass_kernel(const uint32_t* __restrict__ keys, uint64_t n, uint64_t nb,
                                                           WsHeader* hdr, uint32_t cap, uint32_t* __restrict__ G,
                                                           uint32_t* __restrict__ E,
                                                           unsigned long long* __restrict__ cnt,
                                                           uint32_t* __restrict__ cand_key,
                                                           uint32_t* __restrict__ cand_idx) {
    __shared__ uint32_t st_key[8][kStage], st_idx[8][kStage];
    __shared__ uint32_t cta_def;
    const uint32_t b_top = hdr->b_top, b_bot = hdr->b_bot;
    const uint32_t lane = lane_id(), wid = threadIdx.x >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t* my_key = st_key[wid];
    uint32_t* my_idx = st_idx[wid];
    if (threadIdx.x == 0) cta_def = 0;
    __syncthreads();
    uint32_t staged = 0, def_acc = 0;
    auto flush = [&](uint32_t m) {
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(&hdr->n_cand, m);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if ((uint64_t)base + m <= cap) {   // else: overflow, n_cand > cap sends the call down the full path
            for (uint32_t e = lane; e < m; e += 32) {
                cand_key[base + e] = my_key[e];
                cand_idx[base + e] = my_idx[e];
            }
        }
        __syncwarp();
    };
    // keys >= top_key are certainly in the core; keys in [bot_key, top_key) are candidates
    const bool has_top = b_top < 65536u;
    const uint32_t top_key = has_top ? (b_top << 16) : 0xFFFFFFFFu;
    const uint32_t bot_key = b_bot << 16;
    const uint64_t warps = (uint64_t)gridDim.x * (blockDim.x >> 5);
    for (uint64_t blk = (uint64_t)blockIdx.x * (blockDim.x >> 5) + wid; blk < nb; blk += warps) {
        const uint64_t base = blk * kBlock;
        const uint32_t valid = (base + kBlock <= n) ? kBlock : (uint32_t)(n - base);   // parameters in this block
        const uint32_t* src = keys + base + lane;
        const uint32_t idx0 = (uint32_t)base + lane;
        uint32_t myG = 0;
        // a quarter block (8 rows of 32 keys) at a time; `full` blocks skip the end-of-vector tests
        auto quarter = [&](const int q, const bool full) {
            uint32_t key[8];
#pragma unroll
            for (int wd = 0; wd < 8; ++wd) {
                const uint32_t off = (q * 8 + wd) * 32;
                key[wd] = (full || off + lane < valid) ? __ldcs(src + off) : 0u;
            }
            uint32_t place = staged;
#pragma unroll
            for (int wd = 0; wd < 8; ++wd) {
                const uint32_t off = (q * 8 + wd) * 32;
                const bool in = full || off + lane < valid;
                const bool def = has_top && key[wd] >= top_key && in;
                const bool cand = key[wd] >= bot_key && !def && in;
                const uint32_t bg = __ballot_sync(0xFFFFFFFFu, def);
                const uint32_t bc = __ballot_sync(0xFFFFFFFFu, cand);
                if (lane == (uint32_t)(q * 8 + wd)) myG = bg;
                if (bc) {   // warp-uniform: most rows hold no candidate
                    if (cand) {
                        const uint32_t slot = place + __popc(bc & lt_mask);
                        my_key[slot] = key[wd];
                        my_idx[slot] = idx0 + off;
                    }
                    place += __popc(bc);
                }
            }
            staged = place;
            __syncwarp();
            if (staged >= kFlushAt) {
                flush(staged);
                staged = 0;
            }
        };
        if (valid == kBlock) {
#pragma unroll 1
            for (int q = 0; q < 4; ++q) quarter(q, true);
        } else {
#pragma unroll 1
            for (int q = 0; q < 4; ++q) quarter(q, false);
        }
        G[blk * kWordsPerBlock + lane] = myG;
        E[blk * kWordsPerBlock + lane] = 0u;
        const uint32_t cg = __reduce_add_sync(0xFFFFFFFFu, __popc(myG));
        if (lane == 0) cnt[blk] = cg;
        def_acc += cg;
    }
    if (staged) flush(staged);
    if (lane == 0 && def_acc) atomicAdd(&cta_def, def_acc);
    __syncthreads();
    if (threadIdx.x == 0 && cta_def) atomicAdd(&hdr->n_def, cta_def);
}

// ---- scoring fused into the bracketed path -----------------------------------------------
//
// When a whole round is enqueued at once the scores need not exist in memory: the sample is
// scored straight from the model and the updates, and the one pass over all parameters computes
// each score in registers and sorts it into "certainly core" / candidate / neither on the spot.
// The score array is written only if the bracket fails and the full path has to read it.

// Left-to-right fp32 sum of the K updates of four consecutive parameters, then their scores.
template <int KT>
__device__ __forceinline__ void score4(const float* __restrict__ w, const PtrArray<const float>& g, int K, float c,
                                       uint64_t i4, uint32_t key[4]) {
    const int kk = (KT > 0) ? KT : K;
    float4 a = __ldcs(reinterpret_cast<const float4*>(g.p[0]) + i4);
    if (KT > 0) {
        float4 b[KT > 1 ? KT - 1 : 1];
#pragma unroll
        for (int k = 1; k < KT; ++k) b[k - 1] = __ldcs(reinterpret_cast<const float4*>(g.p[k]) + i4);
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
            const float4 b = __ldcs(reinterpret_cast<const float4*>(g.p[k]) + i4);
            a.x = __fadd_rn(a.x, b.x);
            a.y = __fadd_rn(a.y, b.y);
            a.z = __fadd_rn(a.z, b.z);
            a.w = __fadd_rn(a.w, b.w);
        }
    }
    const float4 ww = __ldcs(reinterpret_cast<const float4*>(w) + i4);
    key[0] = __float_as_uint(score_one(c, a.x, ww.x));
    key[1] = __float_as_uint(score_one(c, a.y, ww.y));
    key[2] = __float_as_uint(score_one(c, a.z, ww.z));
    key[3] = __float_as_uint(score_one(c, a.w, ww.w));
}

__device__ __forceinline__ uint32_t score1(const float* __restrict__ w, const PtrArray<const float>& g, int K,
                                           float c, uint64_t i) {
    float a = g.p[0][i];
    for (int k = 1; k < K; ++k) a = __fadd_rn(a, g.p[k][i]);
    return __float_as_uint(score_one(c, a, w[i]));
}

// Sample kernel A of the fused path: 2^14 evenly spaced groups of sixteen consecutive parameters
// are scored (2^18 sampled keys, one 16-byte load per tensor and thread); the rest is
// sample_coarse_kernel's.  Needs n >= 16 and 16-byte aligned tensors.  1024 groups per CTA: the
// sampled keys fall into a handful of coarse bins, and every CTA adds to those few global
// counters, so few large CTAs queue up less there than many small ones.
__global__ void __launch_bounds__(1024) sample_score_coarse_kernel(const float* __restrict__ w,
                                                                    PtrArray<const float> g, int K, float c,
                                                                    uint64_t n, uint32_t k, WsHeader* hdr,
                                                                    uint32_t* __restrict__ sample,
                                                                    uint32_t* __restrict__ coarse_hist,
                                                                    uint32_t* __restrict__ coarse_incl) {
    __shared__ unsigned long long smem[33];
    __shared__ uint32_t sh_coarse[256];
    __shared__ long long s_incl[257];
    const uint32_t t = threadIdx.x;
    if (t < 256) sh_coarse[t] = 0;
    __syncthreads();
    // thread j scores four consecutive parameters; threads 4s .. 4s+3 together take sixteen consecutive
    // ones at the s-th of 2^14 evenly spaced places: one 64-byte piece per tensor and place, the least
    // DRAM hands out, so the sample costs a quarter of the fetches that 2^16 separate places would
    const uint32_t j = blockIdx.x * 1024 + t;   // < 2^16
    uint32_t key[4];
    score4<0>(w, g, K, c, ((((uint64_t)(j >> 2) * (n / 16)) >> (kSampleBits - 4)) << 2) + (j & 3u), key);
    reinterpret_cast<uint4*>(sample)[j] = make_uint4(key[0], key[1], key[2], key[3]);
    // most of a warp's keys share a coarse bin: one shared-memory atomic per distinct bin and warp
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint32_t bin = key[q] >> 24;
        const uint32_t peers = __match_any_sync(0xFFFFFFFFu, bin);
        if ((peers & ((1u << lane_id()) - 1u)) == 0) atomicAdd(&sh_coarse[bin], (uint32_t)__popc(peers));
    }
    __syncthreads();
    if (t < 256 && sh_coarse[t]) atomicAdd(&coarse_hist[t], sh_coarse[t]);
    if (!last_cta_done(&hdr->ticket[6])) return;
    long long lo_target, hi_target;
    bracket_targets(k, n, &lo_target, &hi_target);
    // coarse bins from the top down: thread t < 256 owns coarse bin 255 - t
    unsigned long long total;
    const unsigned long long cc = (t < 256) ? __ldcg(coarse_hist + 255 - t) : 0ull;
    const long long c_above = (long long)block_exclusive_scan64<32>(cc, smem, &total);
    if (t < 256) s_incl[255 - t] = c_above + (long long)cc;
    if (t == 0) {
        s_incl[256] = 0;
        hdr->coarse_x[0] = 0xFFFFFFFFu;
        hdr->coarse_x[1] = 0xFFFFFFFFu;
    }
    __syncthreads();
    if (t < 256) {
        const long long incl = s_incl[t], above = s_incl[t + 1];
        coarse_incl[t] = (uint32_t)incl;
        if (incl > lo_target && above <= lo_target) hdr->coarse_x[0] = t;
        if (incl >= hi_target && above < hi_target) hdr->coarse_x[1] = t;
    }
}

constexpr uint32_t kFusedStage = kFlushAt + 128;   // below kFlushAt before a row of 128 parameters, +128 in it

// The bracket pass with the scores computed in place of being read.  Warp per 1024-parameter
// block, a row of 128 parameters (one 16-byte load per lane and tensor) at a time; lane l holds
// parameters 4l .. 4l+3 of the row, so eight neighbouring lanes make one bitmap word.
template <int KT>
__global__ void __launch_bounds__(256, 4) score_bracket_kernel(const float* __restrict__ w, PtrArray<const float> g,
                                                               int K, float c, uint64_t n, uint64_t nb,
                                                               WsHeader* hdr, uint32_t cap,
                                                               uint32_t* __restrict__ G, uint32_t* __restrict__ E,
                                                               unsigned long long* __restrict__ cnt,
                                                               uint32_t* __restrict__ cand_key,
                                                               uint32_t* __restrict__ cand_idx) {
    __shared__ uint32_t st_key[8][kFusedStage], st_idx[8][kFusedStage];
    __shared__ uint32_t cta_def;
    const uint32_t b_top = hdr->b_top, b_bot = hdr->b_bot;
    const uint32_t lane = lane_id(), wid = threadIdx.x >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t* my_key = st_key[wid];
    uint32_t* my_idx = st_idx[wid];
    if (threadIdx.x == 0) cta_def = 0;
    __syncthreads();
    uint32_t staged = 0, def_acc = 0;
    auto flush = [&](uint32_t m) {
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(&hdr->n_cand, m);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if ((uint64_t)base + m <= cap) {   // else: overflow, n_cand > cap sends the call down the full path
            for (uint32_t e = lane; e < m; e += 32) {
                cand_key[base + e] = my_key[e];
                cand_idx[base + e] = my_idx[e];
            }
        }
        __syncwarp();
    };
    const bool has_top = b_top < 65536u;
    const uint32_t top_key = has_top ? (b_top << 16) : 0xFFFFFFFFu;
    const uint32_t bot_key = b_bot << 16;
    // Blocks are handed out on request, one at a time per warp: other kernels share the SMs while
    // this pass runs, so CTAs start at different times and a fixed split would leave a long tail.
    // The request for the block after this one is issued before the work on this one starts.
    auto next_block = [&]() {
        uint32_t b = 0;
        if (lane == 0) b = atomicAdd(&hdr->next_block, 1u);
        return b;
    };
    uint32_t ahead = next_block();
    for (;;) {
        const uint64_t blk = __shfl_sync(0xFFFFFFFFu, ahead, 0);
        if (blk >= nb) break;
        ahead = next_block();
        const uint64_t base = blk * kBlock;
        const bool full = base + kBlock <= n;
        uint32_t myG = 0;
#pragma unroll 1
        for (uint32_t r = 0; r < 8; ++r) {
            const uint64_t e0 = base + r * 128 + 4 * lane;   // this lane's first parameter of the row
            uint32_t key[4];
            uint32_t in = 0xFu;                               // which of the four exist
            if (full || e0 + 4 <= n) {
                score4<KT>(w, g, K, c, e0 / 4, key);
            } else {
                in = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    key[q] = 0;
                    if (e0 + q < n) {
                        key[q] = score1(w, g, K, c, e0 + q);
                        in |= 1u << q;
                    }
                }
            }
            uint32_t nib = 0, cm = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool ex = (in >> q) & 1u;
                const bool def = has_top && key[q] >= top_key && ex;
                const bool cand = key[q] >= bot_key && !def && ex;
                nib |= (uint32_t)def << q;
                cm |= (uint32_t)cand << q;
            }
            // the row's four bitmap words: lanes 8j .. 8j+7 assemble word j, lane 4r + j keeps it
            uint32_t word = nib << (4 * (lane & 7u));
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
            const uint32_t got = __shfl_sync(0xFFFFFFFFu, word, (lane & 3u) * 8);
            if ((lane >> 2) == r) myG = got;
            if (__any_sync(0xFFFFFFFFu, cm != 0)) {   // warp-uniform: most rows hold no candidate
                uint32_t place = staged;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const bool cand = (cm >> q) & 1u;
                    const uint32_t bc = __ballot_sync(0xFFFFFFFFu, cand);
                    if (cand) {
                        const uint32_t slot = place + __popc(bc & lt_mask);
                        my_key[slot] = key[q];
                        my_idx[slot] = (uint32_t)e0 + q;
                    }
                    place += __popc(bc);
                }
                staged = place;
                __syncwarp();
                if (staged >= kFlushAt) {
                    flush(staged);
                    staged = 0;
                }
            }
        }
        G[blk * kWordsPerBlock + lane] = myG;
        E[blk * kWordsPerBlock + lane] = 0u;
        const uint32_t cg = __reduce_add_sync(0xFFFFFFFFu, __popc(myG));
        if (lane == 0) cnt[blk] = cg;
        def_acc += cg;
    }
    if (staged) flush(staged);
    if (lane == 0 && def_acc) atomicAdd(&cta_def, def_acc);
    __syncthreads();
    if (threadIdx.x == 0 && cta_def) atomicAdd(&hdr->n_def, cta_def);
}

// ---- the same pass with its loads kept in flight in shared memory ---------------------------
//
// The pass above keeps a row's 16-byte loads in registers, so the bytes in flight per SM are
// bounded by the registers of its 32 resident warps, and it leaves other kernels no room on the
// SM.  Here every lane copies its 16 bytes of each tensor straight into a per-warp ring in
// shared memory (cp.async, no registers) and reads them back S rows later: 8 warps per SM keep
// S rows each in flight, which saturates the memory system with one CTA per SM and a fraction
// of the register file.  The rest of the SM is free for the kernels that run beside the pass.
// A lane reads only what it copied itself, so waiting for its own copy groups is all the
// synchronisation the ring needs.

// 16 bytes from global to shared memory without a register in between.  `policy` marks the line
// as the first to leave L2 (the pass reads every byte once), and the copy asks for whole 128-byte lines.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src, uint64_t policy) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global.L2::cache_hint.L2::128B [%0], [%1], 16, %2;" ::"r"(d), "l"(gmem_src),
                 "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
}

// Ring bytes per CTA: as many stages as fit the first budget, which leaves the kernels beside the
// pass about 100 KB of the SM's shared memory; with many workers, two stages within the second.
constexpr uint32_t kAsyncRingBudget = 112u * 1024u, kAsyncRingBudgetMax = 176u * 1024u;

// Candidate staging of a CTA of `warps` warps, as in the pass above.
inline uint32_t async_cand_bytes(uint32_t warps) { return warps * 2u * kFusedStage * 4u; }
// Bytes of one ring stage of a CTA: a row of 128 parameters of the model and the K updates per warp.
inline uint32_t async_stage_bytes(uint32_t K, uint32_t warps) { return warps * (K + 1u) * 512u; }
// Stages the ring gets for K workers and `warps` warps per CTA (0: this pass does not apply:
// a stage is too large, or the rows are too short to keep enough bytes in flight).
inline int async_stages(uint32_t K, uint32_t warps) {
    const uint32_t stage = async_stage_bytes(K, warps);
    uint32_t s = kAsyncRingBudget / stage;
    if (s < 2 && 2 * stage <= kAsyncRingBudgetMax) s = 2;
    if (s > 8) s = 8;   // the copies run at most one block ahead of the arithmetic
    if (s < 2 || s * stage < 64u * 1024u) return 0;
    return (int)s;
}

// S ring stages per warp, W warps per CTA.
template <int S, int W>
__global__ void __launch_bounds__(W * 32, 2)
    score_bracket_async_kernel(const float* __restrict__ w, PtrArray<const float> g, int K, float c, uint64_t n,
                               uint64_t nb, WsHeader* hdr, uint32_t cap, uint32_t* __restrict__ G,
                               uint32_t* __restrict__ E, unsigned long long* __restrict__ cnt,
                               uint32_t* __restrict__ cand_key, uint32_t* __restrict__ cand_idx) {
    static_assert(S >= 2 && S <= 8, "the copies stay within the block after the one being processed");
    extern __shared__ __align__(16) uint32_t async_smem[];
    __shared__ uint32_t cta_def;
    const uint32_t b_top = hdr->b_top, b_bot = hdr->b_bot;
    const uint32_t lane = lane_id(), wid = threadIdx.x >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t* my_key = async_smem + wid * kFusedStage;
    uint32_t* my_idx = async_smem + (W + wid) * kFusedStage;
    const uint32_t stage_f4 = (uint32_t)(K + 1) * 32u;   // 16-byte words of one stage of one warp
    float4* ring = reinterpret_cast<float4*>(async_smem + 2 * W * kFusedStage) + (size_t)wid * S * stage_f4;
    if (threadIdx.x == 0) cta_def = 0;
    __syncthreads();
    uint32_t staged = 0, def_acc = 0;
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    auto flush = [&](uint32_t m) {
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(&hdr->n_cand, m);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        if ((uint64_t)base + m <= cap) {   // else: overflow, n_cand > cap sends the call down the full path
            for (uint32_t e = lane; e < m; e += 32) {
                cand_key[base + e] = my_key[e];
                cand_idx[base + e] = my_idx[e];
            }
        }
        __syncwarp();
    };
    const bool has_top = b_top < 65536u;
    const uint32_t top_key = has_top ? (b_top << 16) : 0xFFFFFFFFu;
    const uint32_t bot_key = b_bot << 16;
    // Blocks are handed out on request, one at a time per warp (other kernels share the SMs, so
    // warps advance at different speeds).  A warp knows the block it works on and the next one;
    // the request for the one after that is in flight meanwhile.
    auto request_block = [&]() {
        uint32_t b = 0;
        if (lane == 0) b = atomicAdd(&hdr->next_block, 1u);
        return b;
    };
    uint64_t blk = __shfl_sync(0xFFFFFFFFu, request_block(), 0);
    uint64_t blk_next = __shfl_sync(0xFFFFFFFFu, request_block(), 0);
    uint32_t requested = request_block();
    // the copies: row `copy_row` of block (copy_ahead ? blk_next : blk) goes to stage `copy_slot`
    uint32_t copy_ahead = 0, copy_row = 0, copy_slot = 0, slot = 0;
    auto copy_next_row = [&]() {
        const uint64_t b = copy_ahead ? blk_next : blk;
        if (b < nb && (b + 1) * kBlock <= n) {   // whole blocks only; the ragged last block is loaded directly
            const uint64_t i4 = (b * kBlock + copy_row * 128u) / 4u + lane;
            float4* dst = ring + copy_slot * stage_f4 + lane;
            for (int k = 0; k < K; ++k)
                cp_async16(dst + k * 32, reinterpret_cast<const float4*>(g.p[k]) + i4, policy);
            cp_async16(dst + K * 32, reinterpret_cast<const float4*>(w) + i4, policy);
        }
        cp_async_commit();   // one group per row, empty or not, so that the group count tells the row
        copy_slot = (copy_slot + 1 == S) ? 0 : copy_slot + 1;
        if (++copy_row == 8) {
            copy_row = 0;
            ++copy_ahead;
        }
    };
#pragma unroll 1
    for (int s0 = 0; s0 < S; ++s0) copy_next_row();
    while (blk < nb) {
        const uint64_t base = blk * kBlock;
        const bool full = base + kBlock <= n;
        uint32_t myG = 0;
#pragma unroll 1
        for (uint32_t r = 0; r < 8; ++r) {
            const uint64_t e0 = base + r * 128 + 4 * lane;   // this lane's first parameter of the row
            uint32_t key[4];
            uint32_t in = 0xFu;                               // which of the four exist
            cp_async_wait<S - 1>();                           // this row's copies have landed
            if (full) {
                const float4* src = ring + slot * stage_f4 + lane;
                float4 a = src[0];
#pragma unroll 4
                for (int k = 1; k < K; ++k) {
                    const float4 b = src[k * 32];
                    a.x = __fadd_rn(a.x, b.x);
                    a.y = __fadd_rn(a.y, b.y);
                    a.z = __fadd_rn(a.z, b.z);
                    a.w = __fadd_rn(a.w, b.w);
                }
                const float4 ww = src[K * 32];
                key[0] = __float_as_uint(score_one(c, a.x, ww.x));
                key[1] = __float_as_uint(score_one(c, a.y, ww.y));
                key[2] = __float_as_uint(score_one(c, a.z, ww.z));
                key[3] = __float_as_uint(score_one(c, a.w, ww.w));
            } else if (e0 + 4 <= n) {
                score4<0>(w, g, K, c, e0 / 4, key);
            } else {
                in = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    key[q] = 0;
                    if (e0 + q < n) {
                        key[q] = score1(w, g, K, c, e0 + q);
                        in |= 1u << q;
                    }
                }
            }
            slot = (slot + 1 == S) ? 0 : slot + 1;
            copy_next_row();   // into the stage just read
            uint32_t nib = 0, cm = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool ex = (in >> q) & 1u;
                const bool def = has_top && key[q] >= top_key && ex;
                const bool cand = key[q] >= bot_key && !def && ex;
                nib |= (uint32_t)def << q;
                cm |= (uint32_t)cand << q;
            }
            // the row's four bitmap words: lanes 8j .. 8j+7 assemble word j, lane 4r + j keeps it
            uint32_t word = nib << (4 * (lane & 7u));
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
            const uint32_t got = __shfl_sync(0xFFFFFFFFu, word, (lane & 3u) * 8);
            if ((lane >> 2) == r) myG = got;
            if (__any_sync(0xFFFFFFFFu, cm != 0)) {   // warp-uniform: most rows hold no candidate
                uint32_t place = staged;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const bool cand = (cm >> q) & 1u;
                    const uint32_t bc = __ballot_sync(0xFFFFFFFFu, cand);
                    if (cand) {
                        const uint32_t at = place + __popc(bc & lt_mask);
                        my_key[at] = key[q];
                        my_idx[at] = (uint32_t)e0 + q;
                    }
                    place += __popc(bc);
                }
                staged = place;
                __syncwarp();
                if (staged >= kFlushAt) {
                    flush(staged);
                    staged = 0;
                }
            }
        }
        G[blk * kWordsPerBlock + lane] = myG;
        E[blk * kWordsPerBlock + lane] = 0u;
        const uint32_t cg = __reduce_add_sync(0xFFFFFFFFu, __popc(myG));
        if (lane == 0) cnt[blk] = cg;
        def_acc += cg;
        // on to the next block; the copies are S rows into it already
        blk = blk_next;
        blk_next = __shfl_sync(0xFFFFFFFFu, requested, 0);
        requested = request_block();
        --copy_ahead;
    }
    cp_async_wait<0>();
    if (staged) flush(staged);
    if (lane == 0 && def_acc) atomicAdd(&cta_def, def_acc);
    __syncthreads();
    if (threadIdx.x == 0 && cta_def) atomicAdd(&hdr->n_def, cta_def);
}

// The scores for the full path, written only when the bracket failed.
__global__ void __launch_bounds__(256) score_if_bracket_failed_kernel(const float* __restrict__ w,
                                                                      PtrArray<const float> g, int K, float c,
                                                                      uint64_t n, const WsHeader* __restrict__ hdr,
                                                                      uint32_t k, uint32_t cap,
                                                                      uint32_t* __restrict__ S) {
    if (bracket_ok(hdr, k, cap)) return;
    const uint64_t n4 = n / 4;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    const uint64_t gid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (uint64_t i = gid; i < n4; i += stride) {
        uint32_t key[4];
        score4<0>(w, g, K, c, i, key);
        reinterpret_cast<uint4*>(S)[i] = make_uint4(key[0], key[1], key[2], key[3]);
    }
    if (gid < n - 4 * n4) S[4 * n4 + gid] = score1(w, g, K, c, 4 * n4 + gid);
}

// ---- radix histogram passes (over all keys, or over the candidates) -----------------------

template <int PASS>
__device__ __forceinline__ void hist_key(uint32_t key, uint32_t prefix, uint32_t* sh) {
    if (PASS == 0) {
        atomicAdd(&sh[key >> 20], 1u);
    } else if (PASS == 1) {
        if ((key >> 20) == (prefix >> 20)) atomicAdd(&sh[(key >> 10) & 1023u], 1u);
    } else {
        if ((key >> 10) == (prefix >> 10)) atomicAdd(&sh[key & 1023u], 1u);
    }
}

// Histogram of one radix digit; the last CTA to finish then walks the histogram
// from the top bin down and records the bin that holds the wanted rank.
template <int PASS>
__global__ void __launch_bounds__(kHistThreads) hist_kernel(const uint32_t* __restrict__ all_keys, uint64_t n_all,
                                                            const uint32_t* __restrict__ cand_key, WsHeader* hdr,
                                                            uint32_t* __restrict__ hist, uint32_t k, uint32_t cap,
                                                            int mode) {
    constexpr uint32_t NB = (PASS == 0) ? kBins0 : kBins12;
    constexpr uint32_t PER = NB / kHistThreads;
    constexpr uint32_t SHIFT = (PASS == 0) ? 20 : (PASS == 1 ? 10 : 0);
    __shared__ uint32_t sh[NB];
    __shared__ unsigned long long smem[33];
    if (!mode_runs(mode, hdr, k, cap)) return;
    const uint32_t* keys = (mode == kCandidates) ? cand_key : all_keys;
    const uint64_t n = (mode == kCandidates) ? hdr->n_cand : n_all;
    for (uint32_t b = threadIdx.x; b < NB; b += kHistThreads) sh[b] = 0;
    __syncthreads();
    const uint32_t prefix = (PASS == 0) ? 0u : hdr->prefix;

    // scalar head up to 16-byte alignment, 128-bit body, scalar tail
    const uint64_t mis = (reinterpret_cast<uintptr_t>(keys) & 15u) / 4u;
    uint64_t head = (4u - mis) & 3u;
    if (head > n) head = n;
    const uint64_t body4 = (n - head) / 4;
    const uint64_t tail = n - head - 4 * body4;
    const uint64_t gid = (uint64_t)blockIdx.x * kHistThreads + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * kHistThreads;
    if (gid < head) hist_key<PASS>(keys[gid], prefix, sh);
    if (gid < tail) hist_key<PASS>(keys[head + 4 * body4 + gid], prefix, sh);
    const uint4* k4 = reinterpret_cast<const uint4*>(keys + head);
    for (uint64_t i = gid; i < body4; i += stride) {
        uint4 v = __ldg(k4 + i);
        hist_key<PASS>(v.x, prefix, sh);
        hist_key<PASS>(v.y, prefix, sh);
        hist_key<PASS>(v.z, prefix, sh);
        hist_key<PASS>(v.w, prefix, sh);
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < NB; b += kHistThreads) {
        uint32_t c = sh[b];
        if (c) atomicAdd(&hist[b], c);
    }
    if (!last_cta_done(&hdr->ticket[PASS + (mode == kCandidates ? 0 : 3)])) return;

    // rank wanted inside the current prefix
    uint32_t want;
    if (PASS == 0)
        want = (mode == kCandidates) ? k - hdr->n_def : k;
    else
        want = hdr->k_rem;
    const volatile uint32_t* gh = hist;
    const uint32_t top = NB - 1 - threadIdx.x * PER;   // this thread's highest bin
    uint32_t h[PER];
    unsigned long long sum = 0;
#pragma unroll
    for (uint32_t q = 0; q < PER; ++q) {
        h[q] = gh[top - q];
        sum += h[q];
    }
    unsigned long long total;
    unsigned long long above = block_exclusive_scan64<kHistThreads / 32>(sum, smem, &total);
    if (total < want) {
        if (threadIdx.x == 0) hdr->status = SLIMDP_ERR_INTERNAL;
        return;
    }
#pragma unroll
    for (uint32_t q = 0; q < PER; ++q) {
        if (above < want && (unsigned long long)want <= above + h[q]) {
            const uint32_t rem = want - (uint32_t)above;
            hdr->prefix = prefix | ((top - q) << SHIFT);
            hdr->k_rem = rem;
            if (PASS == 2) hdr->ties = rem;
        }
        above += h[q];
    }
}

// ---- step 3: candidates into the bitmaps --------------------------------------------------

__global__ void __launch_bounds__(256) mark_candidates_kernel(const uint32_t* __restrict__ cand_key,
                                                              const uint32_t* __restrict__ cand_idx,
                                                              const WsHeader* __restrict__ hdr, uint32_t k,
                                                              uint32_t cap, uint32_t* __restrict__ G,
                                                              uint32_t* __restrict__ E,
                                                              unsigned long long* __restrict__ cnt) {
    if (!bracket_ok(hdr, k, cap)) return;
    const uint32_t T = hdr->prefix, n_cand = hdr->n_cand;
    const uint32_t stride = gridDim.x * blockDim.x;
    for (uint32_t c = blockIdx.x * blockDim.x + threadIdx.x; c < n_cand; c += stride) {
        const uint32_t key = __ldg(cand_key + c);
        if (key < T) continue;
        const uint32_t i = __ldg(cand_idx + c);
        if (key > T) {
            atomicOr(&G[i >> 5], 1u << (i & 31u));
            atomicAdd(&cnt[i / kBlock], 1ull);
        } else {
            atomicOr(&E[i >> 5], 1u << (i & 31u));
            atomicAdd(&cnt[i / kBlock], 1ull << 32);
        }
    }
}

// ---- full path: classify every key against T ----------------------------------------------

// Warp per 1024-parameter block: two bitmap words per lane and the block's counts.
__global__ void __launch_bounds__(256) classify_kernel(const uint32_t* __restrict__ keys, uint64_t n, uint64_t nb,
                                                       const WsHeader* __restrict__ hdr, uint32_t k, uint32_t cap,
                                                       int mode, uint32_t* __restrict__ G, uint32_t* __restrict__ E,
                                                       unsigned long long* __restrict__ cnt) {
    if (!mode_runs(mode, hdr, k, cap)) return;
    const uint32_t T = hdr->prefix;
    const uint32_t lane = lane_id();
    const uint64_t warps = (uint64_t)gridDim.x * (blockDim.x >> 5);
    for (uint64_t blk = (uint64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); blk < nb; blk += warps) {
        const uint64_t base = blk * kBlock;
        uint32_t myG = 0, myE = 0;
        if (base + kBlock <= n) {
            uint32_t key[32];
#pragma unroll
            for (int wd = 0; wd < 32; ++wd) key[wd] = __ldcs(keys + base + wd * 32 + lane);
#pragma unroll
            for (int wd = 0; wd < 32; ++wd) {
                uint32_t bg = __ballot_sync(0xFFFFFFFFu, key[wd] > T);
                uint32_t be = __ballot_sync(0xFFFFFFFFu, key[wd] == T);
                if (lane == (uint32_t)wd) {
                    myG = bg;
                    myE = be;
                }
            }
        } else {
            for (int wd = 0; wd < 32; ++wd) {
                const uint64_t i = base + wd * 32 + lane;
                const bool in = i < n;
                const uint32_t key = in ? keys[i] : 0u;
                uint32_t bg = __ballot_sync(0xFFFFFFFFu, in && key > T);
                uint32_t be = __ballot_sync(0xFFFFFFFFu, in && key == T);
                if (lane == (uint32_t)wd) {
                    myG = bg;
                    myE = be;
                }
            }
        }
        G[blk * kWordsPerBlock + lane] = myG;
        E[blk * kWordsPerBlock + lane] = myE;
        uint32_t cg = __reduce_add_sync(0xFFFFFFFFu, __popc(myG));
        uint32_t ce = __reduce_add_sync(0xFFFFFFFFu, __popc(myE));
        if (lane == 0) cnt[blk] = (unsigned long long)cg | ((unsigned long long)ce << 32);
    }
}

// ---- last step: bitmaps to core bitmap, directory and ascending index list ----------------

// Warp per 1024-parameter block, bitmaps only.
__global__ void __launch_bounds__(256) emit_kernel(const uint32_t* __restrict__ G, const uint32_t* __restrict__ E,
                                                   const unsigned long long* __restrict__ pref,
                                                   const unsigned long long* __restrict__ totals, uint64_t n,
                                                   uint64_t nb, uint32_t k_core, WsHeader* hdr,
                                                   uint32_t* __restrict__ core_idx, uint32_t* __restrict__ bitmap,
                                                   uint32_t* __restrict__ dir) {
    const uint32_t ties = hdr->ties;
    const uint32_t lane = lane_id();
    const uint64_t warps = (uint64_t)gridDim.x * (blockDim.x >> 5);
    const uint64_t warp0 = (uint64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (warp0 == 0 && lane == 0) {
        // whole-vector check: (#greater) + min(#equal, r) must be k_core
        const unsigned long long t = totals[0];
        const uint32_t ng = (uint32_t)t, ne = (uint32_t)(t >> 32);
        if (ng + min(ne, ties) != k_core) hdr->status = SLIMDP_ERR_INTERNAL;
        dir[nb * kDirPerBlock] = (uint32_t)(n - k_core);
    }
    // the next block's words are requested before this block's are worked on
    uint32_t Gn = 0, En = 0;
    unsigned long long pn = 0;
    if (warp0 < nb) {
        Gn = __ldcs(G + warp0 * kWordsPerBlock + lane);
        En = __ldcs(E + warp0 * kWordsPerBlock + lane);
        pn = __ldcs(pref + warp0);
    }
    for (uint64_t blk = warp0; blk < nb; blk += warps) {
        const uint32_t Gw = Gn, Ew = En;
        const unsigned long long p = pn;
        if (blk + warps < nb) {
            Gn = __ldcs(G + (blk + warps) * kWordsPerBlock + lane);
            En = __ldcs(E + (blk + warps) * kWordsPerBlock + lane);
            pn = __ldcs(pref + blk + warps);
        }
        const uint32_t g_before = (uint32_t)p, e_before = (uint32_t)(p >> 32);
        // equal keys: admit those whose rank among all equal keys (index order) is below r
        const uint32_t pe = __popc(Ew);
        const uint32_t e_rank0 = e_before + warp_inclusive_scan(pe) - pe;
        uint32_t admit = (ties > e_rank0) ? min(ties - e_rank0, pe) : 0u;
        uint32_t Ea;
        if (admit == pe) {
            Ea = Ew;
        } else if (admit == 0) {
            Ea = 0;
        } else {
            Ea = Ew & ((1u << nth_set_bit(Ew, admit)) - 1u);
        }
        const uint32_t sel = Gw | Ea;
        const uint32_t ps = __popc(sel);
        const uint32_t sel_before = g_before + min(e_before, ties);
        const uint32_t ps_incl = warp_inclusive_scan(ps);
        const uint32_t out_base = sel_before + ps_incl - ps;
        bitmap[blk * kWordsPerBlock + lane] = sel;
        if ((lane & (kWordsPerDir - 1)) == 0)   // one directory entry per 64 parameters (2 words)
            dir[blk * kDirPerBlock + lane / kWordsPerDir] = (uint32_t)(blk * kBlock + lane * 32 - out_base);
        const uint32_t in_block = __shfl_sync(0xFFFFFFFFu, ps_incl, 31);
        if (in_block == 0) continue;
        const uint32_t first = (uint32_t)(blk * kBlock);
        if (in_block <= 256) {
            // sparse block: every lane writes out its own word's members
            uint32_t word = sel, pos = out_base;
            while (word) {
                const uint32_t bit = __ffs(word) - 1;
                word &= word - 1;
                if (pos < k_core)
                    core_idx[pos] = first + lane * 32 + bit;
                else
                    hdr->status = SLIMDP_ERR_INTERNAL;
                ++pos;
            }
        } else {
            // dense block: the warp writes one word's members at a time (coalesced)
            const uint32_t any = __ballot_sync(0xFFFFFFFFu, sel != 0);
            for (uint32_t m = any; m; m &= m - 1) {
                const int wd = __ffs(m) - 1;
                const uint32_t word = __shfl_sync(0xFFFFFFFFu, sel, wd);
                const uint32_t base = __shfl_sync(0xFFFFFFFFu, out_base, wd);
                if ((word >> lane) & 1u) {
                    const uint32_t pos = base + __popc(word & ((1u << lane) - 1u));
                    if (pos < k_core)
                        core_idx[pos] = first + wd * 32 + lane;
                    else
                        hdr->status = SLIMDP_ERR_INTERNAL;
                }
            }
        }
    }
}

}  // namespace

// One selection.  `fused` non-null: the scores are not in memory yet; they are computed from the
// model and the updates inside the bracketed path (which the caller has checked applies), and
// `scores` is written only if the full path has to run.
struct FusedScore {
    const float* w;
    const PtrArray<const float>* g;
    uint32_t K;
    float c;
    cudaEvent_t mark_begin, mark_end;   // recorded around the pass over all parameters when not null
    // called once the pass over all parameters is enqueued: what the caller enqueues on other
    // streams from here on finds the pass's CTAs already placed
    slimdp_status (*after_pass)(void*);
    void* after_arg;
    cudaEvent_t pass_ready;   // recorded just before the pass is enqueued when not null: work that is to run
                              // beside the pass, not before it, waits for this
};

// A second stream for the full path's kernels.  After the bracket pass exactly one of the two
// paths does any work (the other's kernels return at once), and the two write disjoint state, so
// they may run side by side; the idle one then costs no time on the critical path.
struct GateStream {
    cudaStream_t stream;
    cudaEvent_t fork, join;
};

static slimdp_status launch_select_impl(float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx,
                                        void* core_aux, void* ws, const FusedScore* fused, const GateStream* gate,
                                        cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const SelectWs L = select_ws_layout(ws, n);
    const uint64_t nb = num_blocks(n);
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(scores);
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(core_aux);
    uint32_t* dir = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(core_aux) + slimdp_core_aux_dir_offset(n));
    const uint32_t k = (uint32_t)k_core;
    const uint32_t cap = (uint32_t)L.cand_cap;

    // header, radix histograms and sample histograms are contiguous: one clear
    if (cudaMemsetAsync(L.hdr, 0, L.zero_bytes, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
    select_init_kernel<<<1, 1, 0, st>>>(L.hdr, k);
    SLIMDP_LAUNCHED(1);
    uint64_t cgrid = (nb + 7) / 8;
    if (cgrid > (uint64_t)sms * 8) cgrid = (uint64_t)sms * 8;
    const unsigned hgrid = (unsigned)sms * 4;
    const bool bracketed = k_core > 0 && n >= kBracketMinN;
    cudaStream_t fs = st;   // the stream of the full path's kernels
    if (bracketed) {
        if (fused)
            sample_score_coarse_kernel<<<(1u << (kSampleBits - 2)) / 1024, 1024, 0, st>>>(
                fused->w, *fused->g, (int)fused->K, fused->c, n, k, L.hdr, L.sample, L.coarse_hist, L.coarse_incl);
        else
            sample_coarse_kernel<<<(1u << kSampleBits) / 1024, 1024, 0, st>>>(keys, n, k, L.hdr, L.sample,
                                                                              L.coarse_hist, L.coarse_incl);
        sample_fine_kernel<<<(1u << kSampleBits) / 1024, 1024, 0, st>>>(L.sample, n, k, L.hdr, L.fine_hist,
                                                                        L.coarse_incl);
        if (fused) {
            if (fused->mark_begin && cudaEventRecord(fused->mark_begin, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
            if (fused->pass_ready && cudaEventRecord(fused->pass_ready, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
            constexpr uint32_t warps = 8;
            const int stages = async_stages(fused->K, warps);
            if (stages > 0) {
                // one CTA per SM, its loads in flight in shared memory (see score_bracket_async_kernel)
                const uint32_t smem = async_cand_bytes(warps) + (uint32_t)stages * async_stage_bytes(fused->K, warps);
                uint64_t agrid = (nb + warps - 1) / warps;
                if (agrid > (uint64_t)sms) agrid = (uint64_t)sms;
#define SLIMDP_ASYNC_CASE(SS)                                                                                       \
    case SS: {                                                                                                      \
        auto kern = score_bracket_async_kernel<SS, warps>;                                                          \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||    \
            !prefer_max_shared(kern))                                                                               \
            return SLIMDP_ERR_CUDA;                                                                                 \
        kern<<<(unsigned)agrid, warps * 32, smem, st>>>(fused->w, *fused->g, (int)fused->K, fused->c, n, nb, L.hdr, \
                                                        cap, L.G, L.E, L.cnt, L.cand_key, L.cand_idx);              \
    } break
                switch (stages) {
                    SLIMDP_ASYNC_CASE(2);
                    SLIMDP_ASYNC_CASE(3);
                    SLIMDP_ASYNC_CASE(4);
                    SLIMDP_ASYNC_CASE(5);
                    SLIMDP_ASYNC_CASE(6);
                    SLIMDP_ASYNC_CASE(7);
                    SLIMDP_ASYNC_CASE(8);
                    default: return SLIMDP_ERR_INTERNAL;
                }
#undef SLIMDP_ASYNC_CASE
            } else {
                // very many workers (a ring stage would not fit) or very few (too few bytes per row)
                uint64_t fgrid = (nb + 7) / 8;
                const uint64_t fmax = 4ull * (uint64_t)sms;
                if (fgrid > fmax) fgrid = fmax;
#define SLIMDP_FUSED_CASE(KK)                                                                                     \
    score_bracket_kernel<KK><<<(unsigned)fgrid, 256, 0, st>>>(fused->w, *fused->g, (int)fused->K, fused->c, n, nb, \
                                                              L.hdr, cap, L.G, L.E, L.cnt, L.cand_key, L.cand_idx)
                switch (fused->K) {
                    case 4: SLIMDP_FUSED_CASE(4); break;
                    case 8: SLIMDP_FUSED_CASE(8); break;
                    default: SLIMDP_FUSED_CASE(0);
                }
#undef SLIMDP_FUSED_CASE
            }
            if (fused->mark_end && cudaEventRecord(fused->mark_end, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
            if (fused->after_pass) {
                const slimdp_status hs = fused->after_pass(fused->after_arg);
                if (hs != SLIMDP_OK) return hs;
            }
        } else {
            bracket_pass_kernel<<<(unsigned)cgrid, 256, 0, st>>>(keys, n, nb, L.hdr, cap, L.G, L.E, L.cnt, L.cand_key,
                                                                 L.cand_idx);
        }
        if (gate) {   // the full path's kernels go to the second stream from here on
            if (cudaEventRecord(gate->fork, st) != cudaSuccess ||
                cudaStreamWaitEvent(gate->stream, gate->fork, 0) != cudaSuccess)
                return SLIMDP_ERR_CUDA;
            fs = gate->stream;
        }
        // T and r from the candidates (these return at once if the bracket failed) ...
        const unsigned cand_grid = (unsigned)sms;
        hist_kernel<0><<<cand_grid, kHistThreads, 0, st>>>(keys, n, L.cand_key, L.hdr, L.hist + 3 * kBins0, k, cap,
                                                           kCandidates);
        hist_kernel<1><<<cand_grid, kHistThreads, 0, st>>>(keys, n, L.cand_key, L.hdr, L.hist + 4 * kBins0, k, cap,
                                                           kCandidates);
        hist_kernel<2><<<cand_grid, kHistThreads, 0, st>>>(keys, n, L.cand_key, L.hdr, L.hist + 5 * kBins0, k, cap,
                                                           kCandidates);
        mark_candidates_kernel<<<(unsigned)sms * 4, 256, 0, st>>>(L.cand_key, L.cand_idx, L.hdr, k, cap, L.G, L.E,
                                                                  L.cnt);
        SLIMDP_LAUNCHED(7);
    }
    if (fused) {
        score_if_bracket_failed_kernel<<<(unsigned)sms * 8, 256, 0, fs>>>(fused->w, *fused->g, (int)fused->K, fused->c,
                                                                          n, L.hdr, k, cap,
                                                                          reinterpret_cast<uint32_t*>(scores));
        SLIMDP_LAUNCHED(1);
    }
    if (k_core > 0) {
        // ... or from all keys (these return at once if the bracket held)
        const int mode = bracketed ? kFullIfBracketFailed : kFullAlways;
        hist_kernel<0><<<hgrid, kHistThreads, 0, fs>>>(keys, n, L.cand_key, L.hdr, L.hist, k, cap, mode);
        hist_kernel<1><<<hgrid, kHistThreads, 0, fs>>>(keys, n, L.cand_key, L.hdr, L.hist + kBins0, k, cap, mode);
        hist_kernel<2><<<hgrid, kHistThreads, 0, fs>>>(keys, n, L.cand_key, L.hdr, L.hist + 2 * kBins0, k, cap, mode);
        SLIMDP_LAUNCHED(3);
    }
    classify_kernel<<<(unsigned)cgrid, 256, 0, fs>>>(keys, n, nb, L.hdr, k, cap,
                                                     bracketed ? kFullIfBracketFailed : kFullAlways, L.G, L.E, L.cnt);
    SLIMDP_LAUNCHED(1);
    if (fs != st) {   // join: the scan needs whichever path ran
        if (cudaEventRecord(gate->join, fs) != cudaSuccess || cudaStreamWaitEvent(st, gate->join, 0) != cudaSuccess)
            return SLIMDP_ERR_CUDA;
    }
    slimdp_status s = launch_block_scan(L.cnt, L.pref, L.tile_sums, L.totals, nb, 1, nb, num_scan_tiles(n), st);
    if (s != SLIMDP_OK) return s;
    emit_kernel<<<(unsigned)cgrid, 256, 0, st>>>(L.G, L.E, L.pref, L.totals, n, nb, k, L.hdr, core_idx, bitmap, dir);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

slimdp_status launch_select(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx, void* core_aux,
                            void* ws, cudaStream_t st) {
    return launch_select_impl(const_cast<float*>(scores), n, k_core, core_idx, core_aux, ws, nullptr, nullptr, st);
}

// Whether scoring can be folded into the selection for these sizes and alignments.
bool score_select_fusable(uint64_t n, uint64_t k_core, bool vec) { return vec && k_core > 0 && n >= kBracketMinN; }

slimdp_status launch_score_select(const float* w, const PtrArray<const float>& g, uint32_t K, float c, uint64_t n,
                                  float* scores, uint64_t k_core, uint32_t* core_idx, void* core_aux, void* ws,
                                  cudaEvent_t mark_begin, cudaEvent_t mark_end, cudaStream_t gate_stream,
                                  cudaEvent_t gate_fork, cudaEvent_t gate_join, slimdp_status (*after_pass)(void*),
                                  void* after_arg, cudaEvent_t pass_ready, cudaStream_t st) {
    const FusedScore f{w, &g, K, c, mark_begin, mark_end, after_pass, after_arg, pass_ready};
    const GateStream gs{gate_stream, gate_fork, gate_join};
    return launch_select_impl(scores, n, k_core, core_idx, core_aux, ws, &f, gate_stream ? &gs : nullptr, st);
}

}  // namespace slimdp
