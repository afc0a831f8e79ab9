// slimdp_select_core: exact top-k_core of the scores (Section 3.2: rank by
// significance, keep the top), ties to the smaller index.
//
// Keys are the scores' 32-bit patterns compared as unsigned integers.  The
// result is defined by the k-th largest key T and the number r of keys equal
// to T that belong to the core (those with the smallest indices).
//
// Large inputs (n >= 2^21) take the bracketed path, which reads the keys once:
//   1. sample (two small kernels): 2^18 keys (sixteen at each of 2^14 evenly
//      spaced places) are counted by their top 8 bits, then, around the two
//      target ranks, by their top 18 bits; the last CTA of each kernel turns
//      the counts into a bracket of 18-bit bins [b_bot, b_top) that holds T
//      with overwhelming probability;
//   2. bracket pass (one read of all keys): keys in bins >= b_top are
//      certainly in the core and go straight into the "greater" bitmap; keys
//      inside the bracket are copied, with their indices, to a candidate list
//      and counted by the top 12 bits of their offset in the bracket; the
//      pass's last CTA finds the 12-bit bin that holds T;
//   3. the finishing kernel (one cooperative launch, two CTAs per SM, phases
//      separated by a grid barrier): if the counts prove the bracket right
//      (n_def < k <= n_def + n_cand, list not overflowed) it resolves the
//      remaining low bits of T from the candidates alone (at most two more
//      counting rounds) and adds the candidates >= T to the "greater" /
//      "equal" bitmaps and to the per-block counts; otherwise (one score value
//      repeated millions of times, a defeated sample, small inputs) it takes the
//      full path: three most-significant-digit-first counting rounds over all
//      keys (12 + 10 + 10 bits) and one classifying round that writes both
//      bitmaps and the counts.  Either way it ends by turning the per-block
//      counts into prefixes per group of 64 blocks;
//   4. the emit kernel (select_dev.cuh; half a warp per 1024-parameter block, no
//      waiting between warps): admits the first r equal keys in index order
//      and writes the core bitmap, the non-core rank directory and the
//      ascending index list (ordered compaction, no atomic cursors).
// Every wait of the grid barrier is bounded: if it runs out the kernel records
// SLIMDP_ERR_INTERNAL in the workspace header and every CTA returns.
#include <atomic>

#include "common.cuh"
#include "layout.cuh"
#include "select_dev.cuh"

namespace slimdp {

namespace {

constexpr uint32_t kBins0 = 4096;       // full path, round 0: bits 31..20
constexpr uint32_t kDigitBits = 12;     // candidates: bits resolved per counting round
constexpr uint32_t kDigitBins = 1u << kDigitBits;

// True when the bracket pass proved that T lies inside the bracket and every candidate was stored.
__device__ __forceinline__ bool bracket_ok(const WsHeader* hdr, uint32_t k, uint32_t cap) {
    return bracket_held(hdr->n_def, hdr->n_cand, k, cap);
}

// The bracket's resolution: bins of 2^kBinShift consecutive keys (the keys' top 18 bits), found in two
// steps (8 bits, then kFineBits more inside the two coarse bins that matter).
constexpr uint32_t kFineBits = 10;
constexpr uint32_t kFineBins = 1u << kFineBits;
constexpr uint32_t kBinShift = 24 - kFineBits;
constexpr uint32_t kNoBin = 1u << (32 - kBinShift);   // b_top when no bin is certainly above T

// Candidates' keys lie in [b_bot << kBinShift, b_top << kBinShift).  Their offsets from the bottom of
// the bracket need `width` bits; the first counting round takes the top kDigitBits of them and leaves
// this many.
__host__ __device__ __forceinline__ uint32_t cand_low_bits(uint32_t b_top, uint32_t b_bot) {
    if (b_top <= b_bot) return 0;
    const unsigned long long span = (unsigned long long)(b_top - b_bot) << kBinShift;   // <= 2^32
    uint32_t width = kBinShift;
    while ((1ull << width) < span) ++width;
    return width > kDigitBits ? width - kDigitBits : 0;
}

// ---- step 1: sample histogram and bracket ------------------------------------------------

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

// Left-to-right fp32 sum of the K updates of four consecutive parameters, then their scores.
__device__ __forceinline__ void score4(const float* __restrict__ w, const PtrArray<const float>& g, int K, float c,
                                       uint64_t i4, uint32_t key[4]) {
    float4 a = __ldcs(reinterpret_cast<const float4*>(g.p[0]) + i4);
#pragma unroll 4
    for (int k = 1; k < K; ++k) {
        const float4 b = __ldcs(reinterpret_cast<const float4*>(g.p[k]) + i4);
        a.x = __fadd_rn(a.x, b.x);
        a.y = __fadd_rn(a.y, b.y);
        a.z = __fadd_rn(a.z, b.z);
        a.w = __fadd_rn(a.w, b.w);
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

// The sample's source: scores in memory (fused == nullptr semantics are the caller's), or the
// model and the updates, scored on the spot.
struct ScoreInputs {
    const float* w;
    PtrArray<const float> g;
    int K;
    float c;
};

// Sample kernel A: 2^18 keys, sixteen consecutive ones (one 64-byte piece, the least DRAM hands
// out) at each of 2^14 evenly spaced places, are copied to `sample` and counted by their top 8
// bits (256 coarse bins: shared memory per CTA, then a few global atomics).  Thread j takes four
// consecutive keys.  FUSED: the keys are scored from the model and the updates (16-byte aligned
// tensors); otherwise read from `keys` (any 4-byte alignment).  The last CTA finds the two coarse
// bins in which the count from the top crosses the two target ranks: coarse_x[0] for b_top
// (highest coarse bin whose inclusive count exceeds lo_target), coarse_x[1] for b_bot (highest
// coarse bin whose inclusive count reaches hi_target); 0xFFFFFFFF = no crossing.
// coarse_incl[c] = samples in coarse bins >= c is kept for kernel B.  1024 threads per CTA: the
// sampled keys fall into a handful of coarse bins, and every CTA adds to those few global
// counters, so few large CTAs queue up less there than many small ones.
template <bool FUSED>
__global__ void __launch_bounds__(1024) sample_coarse_kernel(const uint32_t* __restrict__ keys, ScoreInputs in,
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
    const uint32_t j = blockIdx.x * 1024 + t;   // < 2^16
    const uint64_t first = ((((uint64_t)(j >> 2) * (n / 16)) >> (kSampleBits - 4)) << 4) + 4 * (j & 3u);
    uint32_t key[4];
    if (FUSED) {
        score4(in.w, in.g, in.K, in.c, first / 4, key);
    } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) key[q] = __ldg(keys + first + q);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) sample[4 * j + q] = key[q];
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

// Sample kernel B: the members of the two crossing coarse bins are counted by the kFineBits key bits
// that follow (2 x kFineBins fine bins); the last CTA resolves each crossing to an 18-bit bin:
// b_top = lowest bin b with (samples in bins >= b) <= lo_target, kNoBin if there is none;
// b_bot = highest bin b with (samples in bins >= b) >= hi_target, 0 if there is none.
__global__ void __launch_bounds__(1024) sample_fine_kernel(const uint32_t* __restrict__ sample, uint64_t n,
                                                           uint32_t k, WsHeader* hdr,
                                                           uint32_t* __restrict__ fine_hist,
                                                           const uint32_t* __restrict__ coarse_incl) {
    __shared__ unsigned long long smem[33];
    __shared__ uint32_t sh_fine[2][kFineBins];
    __shared__ uint32_t s_val[2];
    constexpr uint32_t kPer = kFineBins / 1024;   // fine bins per thread of the last CTA
    const uint32_t t = threadIdx.x;
    const uint32_t cx0 = hdr->coarse_x[0], cx1 = hdr->coarse_x[1];
    for (uint32_t b = t; b < 2 * kFineBins; b += 1024) sh_fine[b / kFineBins][b % kFineBins] = 0;
    __syncthreads();
    const uint32_t key = sample[blockIdx.x * 1024 + t];
    const uint32_t cb = key >> 24, fb = (key >> kBinShift) & (kFineBins - 1u);
    if (cb == cx0) atomicAdd(&sh_fine[0][fb], 1u);
    if (cb == cx1) atomicAdd(&sh_fine[1][fb], 1u);
    __syncthreads();
    for (uint32_t b = t; b < 2 * kFineBins; b += 1024) {
        const uint32_t c = sh_fine[b / kFineBins][b % kFineBins];
        if (c) atomicAdd(&fine_hist[b], c);
    }
    if (!last_cta_done(&hdr->ticket[7])) return;
    long long lo_target, hi_target;
    bracket_targets(k, n, &lo_target, &hi_target);
    for (int which = 0; which < 2; ++which) {
        const long long target = which ? hi_target : lo_target;
        const uint32_t cx = which ? cx1 : cx0;
        if (cx == 0xFFFFFFFFu) {
            // no crossing: which = 0: target < 0 (nothing is certain: kNoBin) or every bin qualifies (0);
            //              which = 1: target above the sample size: every bin may hold T (0)
            if (t == 0) s_val[which] = which ? 0u : ((target < 0) ? kNoBin : 0u);
            __syncthreads();
            continue;
        }
        const long long above_cx = (cx == 255) ? 0 : (long long)coarse_incl[cx + 1];
        // fine bins of coarse bin cx from the top down: thread t owns fine bins
        // kFineBins - 1 - kPer t, ..., kFineBins - kPer (t + 1)
        uint32_t f[kPer];
        unsigned long long mine = 0;
#pragma unroll
        for (uint32_t q = 0; q < kPer; ++q) {
            f[q] = __ldcg(fine_hist + which * kFineBins + (kFineBins - 1u - (kPer * t + q)));
            mine += f[q];
        }
        unsigned long long total;
        long long run = above_cx + (long long)block_exclusive_scan64<32>(mine, smem, &total);
        if (t == 0) s_val[which] = which ? 0u : (cx + 1) * kFineBins;   // default when no fine bin of cx qualifies
        __syncthreads();
#pragma unroll
        for (uint32_t q = 0; q < kPer; ++q) {
            const uint32_t b = cx * kFineBins + (kFineBins - 1u - (kPer * t + q));
            run += (long long)f[q];   // samples in bins >= b
            if (which == 0) {
                if (run <= target) atomicMin(&s_val[0], b);
            } else {
                if (run >= target) atomicMax(&s_val[1], b);
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
//
// Both pass kernels (keys read from memory, or scored on the spot) work on rows of 128
// parameters, lane l holding parameters 4l .. 4l+3 of the row, and share everything that follows
// the keys: classification, the bitmap words, the candidate list and its counts.

constexpr uint32_t kFlushAt = 128;               // a warp appends its staged candidates once it holds this many
constexpr uint32_t kCandStage = kFlushAt + 128;  // staging capacity: below kFlushAt before a row of 128, +128 in it
constexpr int kPassWarps = 8;

// Where the pass's results go.
struct PassOut {
    WsHeader* hdr;
    uint32_t cap;
    uint32_t k;
    uint32_t* G;
    uint32_t* E;
    unsigned long long* tile_sum;   // members found, per tile of kEmitTile blocks
    uint32_t* cand_key;
    uint32_t* cand_idx;
    uint32_t* hist1;   // candidates by the top kDigitBits of their offset in the bracket
};

// A warp's view of the pass.
struct PassWarp {
    uint32_t* my_key;    // this warp's candidate staging in shared memory, kCandStage entries
    uint32_t* my_idx;
    uint32_t* sh_hist;   // the CTA's copy of hist1
    uint32_t top_key, bot_key, low_bits;
    bool has_top;
    uint32_t lane, lt_mask;
    uint32_t staged, def_acc;
};

__device__ __forceinline__ void pass_begin(PassWarp& pw, const PassOut& out, uint32_t* cand_smem, uint32_t* sh_hist) {
    const uint32_t b_top = out.hdr->b_top, b_bot = out.hdr->b_bot;
    const uint32_t wid = threadIdx.x >> 5;
    pw.lane = lane_id();
    pw.lt_mask = (1u << pw.lane) - 1u;
    pw.my_key = cand_smem + wid * kCandStage;
    pw.my_idx = cand_smem + (kPassWarps + wid) * kCandStage;
    pw.sh_hist = sh_hist;
    // keys >= top_key are certainly in the core; keys in [bot_key, top_key) are candidates
    pw.has_top = b_top < kNoBin;
    pw.top_key = pw.has_top ? (b_top << kBinShift) : 0xFFFFFFFFu;
    pw.bot_key = b_bot << kBinShift;
    pw.low_bits = cand_low_bits(b_top, b_bot);
    pw.staged = 0;
    pw.def_acc = 0;
    for (uint32_t b = threadIdx.x; b < kDigitBins; b += blockDim.x) sh_hist[b] = 0;
    __syncthreads();
}

// Appends the warp's first m staged candidates to the global list (one cursor atomic).
__device__ __forceinline__ void pass_flush(PassWarp& pw, const PassOut& out, uint32_t m) {
    uint32_t base = 0;
    if (pw.lane == 0) base = atomicAdd(&out.hdr->n_cand, m);
    base = __shfl_sync(0xFFFFFFFFu, base, 0);
    if ((uint64_t)base + m <= out.cap) {   // else: overflow, n_cand > cap sends the call down the full path
        for (uint32_t e = pw.lane; e < m; e += 32) {
            out.cand_key[base + e] = pw.my_key[e];
            out.cand_idx[base + e] = pw.my_idx[e];
        }
    }
    __syncwarp();
}

// One row: key[q] is the key of parameter e0 + q (this lane's four), `in` says which of them exist.
// Returns the lane's 4-bit masks: certainly-core members (*nib) and candidates (*cm).
__device__ __forceinline__ void pass_classify(const PassWarp& pw, const uint32_t key[4], uint32_t in, uint32_t* nib,
                                              uint32_t* cm) {
    uint32_t d = 0, c = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const bool ex = (in >> q) & 1u;
        const bool def = pw.has_top && key[q] >= pw.top_key && ex;
        const bool cand = key[q] >= pw.bot_key && !def && ex;
        d |= (uint32_t)def << q;
        c |= (uint32_t)cand << q;
    }
    *nib = d;
    *cm = c;
}

// The row's four bitmap words: lanes 8j .. 8j+7 assemble word j, lane 4r + j keeps it (r = row in the block).
__device__ __forceinline__ void pass_row_words(const PassWarp& pw, uint32_t nib, uint32_t r, uint32_t* myG) {
    uint32_t word = nib << (4 * (pw.lane & 7u));
    word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
    word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
    word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
    const uint32_t got = __shfl_sync(0xFFFFFFFFu, word, (pw.lane & 3u) * 8);
    if ((pw.lane >> 2) == r) *myG = got;
}

// The row's candidates: staged per warp, counted by their first digit, appended when enough are staged.
__device__ __forceinline__ void pass_candidates(PassWarp& pw, const PassOut& out, const uint32_t key[4], uint32_t cm,
                                                uint32_t e0) {
    if (!__any_sync(0xFFFFFFFFu, cm != 0)) return;   // warp-uniform: most rows hold no candidate
    uint32_t place = pw.staged;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const bool cand = (cm >> q) & 1u;
        const uint32_t bc = __ballot_sync(0xFFFFFFFFu, cand);
        if (cand) {
            const uint32_t at = place + __popc(bc & pw.lt_mask);
            pw.my_key[at] = key[q];
            pw.my_idx[at] = e0 + q;
            atomicAdd(&pw.sh_hist[(key[q] - pw.bot_key) >> pw.low_bits], 1u);
        }
        place += __popc(bc);
    }
    pw.staged = place;
    __syncwarp();
    if (pw.staged >= kFlushAt) {
        pass_flush(pw, out, pw.staged);
        pw.staged = 0;
    }
}

__device__ __forceinline__ void pass_end_block(PassWarp& pw, const PassOut& out, uint64_t blk, uint32_t myG) {
    out.G[blk * kWordsPerBlock + pw.lane] = myG;
    out.E[blk * kWordsPerBlock + pw.lane] = 0u;
    const uint32_t cg = __reduce_add_sync(0xFFFFFFFFu, __popc(myG));
    if (pw.lane == 0 && cg) atomicAdd(&out.tile_sum[blk / kEmitTile], (unsigned long long)cg);
    pw.def_acc += cg;
}

// End of the kernel: the warp's last candidates, the CTA's counts; the last CTA to finish finds the
// first digit of T's offset in the bracket (relative prefix and remaining rank in the header).
__device__ __forceinline__ void pass_end(PassWarp& pw, const PassOut& out, uint32_t* cta_def,
                                         unsigned long long* scan_smem, uint32_t* res) {
    if (pw.staged) pass_flush(pw, out, pw.staged);
    if (pw.lane == 0 && pw.def_acc) atomicAdd(cta_def, pw.def_acc);
    __syncthreads();
    if (threadIdx.x == 0 && *cta_def) atomicAdd(&out.hdr->n_def, *cta_def);
    for (uint32_t b = threadIdx.x; b < kDigitBins; b += blockDim.x) {
        const uint32_t c = pw.sh_hist[b];
        if (c) atomicAdd(&out.hist1[b], c);
    }
    if (!last_cta_done(&out.hdr->ticket[0])) return;
    const volatile WsHeader* vh = out.hdr;
    const uint32_t n_def = vh->n_def, n_cand = vh->n_cand;
    if (!bracket_held(n_def, n_cand, out.k, out.cap)) return;   // the full path will run
    uint32_t bin, rem;
    if (find_rank_bin<kPassWarps * 32>(out.hist1, kDigitBins, out.k - n_def, scan_smem, res, &bin, &rem)) {
        if (threadIdx.x == 0) {
            out.hdr->prefix = bin << pw.low_bits;   // relative to the bottom of the bracket
            out.hdr->k_rem = rem;
        }
    } else if (threadIdx.x == 0) {
        out.hdr->status = SLIMDP_ERR_INTERNAL;
    }
}

// Keys from memory.  Warp per 1024-parameter block; VEC: 16-byte aligned keys, a whole block's
// eight 16-byte loads per lane are issued before the first is used.
template <bool VEC>
__global__ void __launch_bounds__(kPassWarps * 32) bracket_pass_kernel(const uint32_t* __restrict__ keys, uint64_t n,
                                                                       uint64_t nb, PassOut out) {
    __shared__ uint32_t cand_smem[2 * kPassWarps * kCandStage];
    __shared__ uint32_t sh_hist[kDigitBins];
    __shared__ unsigned long long scan_smem[33];
    __shared__ uint32_t res[3];
    __shared__ uint32_t cta_def;
    PassWarp pw;
    if (threadIdx.x == 0) cta_def = 0;
    pass_begin(pw, out, cand_smem, sh_hist);
    const uint64_t warps = (uint64_t)gridDim.x * kPassWarps;
    for (uint64_t blk = (uint64_t)blockIdx.x * kPassWarps + (threadIdx.x >> 5); blk < nb; blk += warps) {
        const uint64_t base = blk * kBlock;
        const bool full = base + kBlock <= n;
        uint32_t myG = 0;
        uint4 rows[8];
        if (VEC && full) {
#pragma unroll
            for (int r = 0; r < 8; ++r) rows[r] = __ldcs(reinterpret_cast<const uint4*>(keys + base + r * 128) + pw.lane);
        }
#pragma unroll
        for (uint32_t r = 0; r < 8; ++r) {
            const uint64_t e0 = base + r * 128 + 4 * pw.lane;
            uint32_t key[4], in = 0xFu;
            if (VEC && full) {
                key[0] = rows[r].x;
                key[1] = rows[r].y;
                key[2] = rows[r].z;
                key[3] = rows[r].w;
            } else {
                in = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    key[q] = 0;
                    if (e0 + q < n) {
                        key[q] = __ldcs(keys + e0 + q);
                        in |= 1u << q;
                    }
                }
            }
            uint32_t nib, cm;
            pass_classify(pw, key, in, &nib, &cm);
            pass_row_words(pw, nib, r, &myG);
            pass_candidates(pw, out, key, cm, (uint32_t)e0);
        }
        pass_end_block(pw, out, blk, myG);
    }
    pass_end(pw, out, &cta_def, scan_smem, res);
}

// ---- the pass with the scores computed on the spot (one-call round) ------------------------
//
// When a whole round is enqueued at once the scores need not exist in memory: the sample is
// scored straight from the model and the updates, and the one pass over all parameters computes
// each score and sorts it into "certainly core" / candidate / neither on the spot.  The score
// array is written only if the bracket fails and the full path has to read it.
//
// Every lane copies its 16 bytes of each tensor straight into a per-warp ring in shared memory
// (cp.async, no registers) and reads them back S rows later: 8 warps per SM keep S rows each in
// flight, which saturates the memory system with one CTA per SM and a fraction of the register
// file.  The rest of the SM is free for the kernels that run beside the pass.  A lane reads only
// what it copied itself, so waiting for its own copy groups is all the synchronisation the ring
// needs.
//
// STAGE: while a row is in the ring, the update values of its certainly-core members and of its
// candidates are set aside in the staging area (see layout.cuh), so that the exchange can stream
// them instead of gathering them out of the K update vectors again.

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
constexpr uint32_t kAsyncRingBudget = 112u * 1024u, kAsyncRingBudgetMax = 160u * 1024u;

// Candidate staging of the CTA plus, per warp, the list of a row's staged positions.
inline uint32_t async_fixed_bytes() { return kPassWarps * 2u * kCandStage * 4u + kPassWarps * 128u; }
// Bytes of one ring stage of a CTA: a row of 128 parameters of the model and the K updates per warp.
inline uint32_t async_stage_bytes(uint32_t K) { return kPassWarps * (K + 1u) * 512u; }
// Stages the ring gets for K workers (0: this pass does not apply: a stage is too large, or the
// rows are too short to keep enough bytes in flight).
inline int async_stages(uint32_t K) {
    const uint32_t stage = async_stage_bytes(K);
    uint32_t s = kAsyncRingBudget / stage;
    if (s < 2 && 2 * stage <= kAsyncRingBudgetMax) s = 2;
    if (s > 8) s = 8;   // the copies run at most one block ahead of the arithmetic
    if (s < 2 || s * stage < 64u * 1024u) return 0;
    return (int)s;
}

struct StageOut {
    uint32_t* fill;
    uint32_t* chunks;
    uint32_t max_chunks;
};

// The warp's place in the staging area: the chunk being filled, how much of it is used, and a
// chunk in reserve that was asked for early (its number arrives while the warp works).
struct StageCursor {
    uint32_t chunk, used, spare_req;
};

__device__ __forceinline__ uint32_t stage_request_chunk(WsHeader* hdr, uint32_t lane) {
    uint32_t ch = 0;
    if (lane == 0) ch = atomicAdd(&hdr->next_chunk, 1u);
    return ch;
}

// After `total` entries went in at cur.used ..: on to the reserve chunk once this one is full.
__device__ __forceinline__ void stage_advance(StageCursor& cur, uint32_t total, uint32_t spare, const StageOut& stage,
                                              WsHeader* hdr, uint32_t lane) {
    cur.used += total;
    if (cur.used >= kStageChunk) {
        if (lane == 0) {
            if (cur.chunk < stage.max_chunks)
                stage.fill[cur.chunk] = kStageChunk;
            else
                hdr->stage_lost = 1u;
        }
        cur.chunk = spare;
        cur.used -= kStageChunk;
        cur.spare_req = stage_request_chunk(hdr, lane);
    }
}

__device__ __forceinline__ float f4_get(const float4& v, int q) { return q == 0 ? v.x : q == 1 ? v.y : q == 2 ? v.z : v.w; }

// S ring stages per warp.  KT > 0: K is known at compile time and a row's update values are kept
// in registers, so the row's ring stage is free for the next copy before anything is staged;
// KT == 0: any K, values are staged out of the ring before the stage is reused.
template <int S, int KT, bool STAGE>
__global__ void __launch_bounds__(kPassWarps * 32, 2)
    score_bracket_async_kernel(const float* __restrict__ w, PtrArray<const float> g, int K_arg, float c, uint64_t n,
                               uint64_t nb, PassOut out, StageOut stage) {
    static_assert(S >= 2 && S <= 8, "the copies stay within the block after the one being processed");
    extern __shared__ __align__(16) uint32_t async_smem[];
    __shared__ uint32_t sh_hist[kDigitBins];
    __shared__ unsigned long long scan_smem[33];
    __shared__ uint32_t res[3];
    __shared__ uint32_t cta_def;
    const int K = (KT > 0) ? KT : K_arg;
    constexpr int KR = (KT > 0) ? KT : 1;
    const uint32_t wid = threadIdx.x >> 5;
    PassWarp pw;
    if (threadIdx.x == 0) cta_def = 0;
    pass_begin(pw, out, async_smem, sh_hist);
    const uint32_t lane = pw.lane;
    uint8_t* pos_list = reinterpret_cast<uint8_t*>(async_smem + 2 * kPassWarps * kCandStage) + wid * 128;
    const uint32_t stage_f4 = (uint32_t)(K + 1) * 32u;   // 16-byte words of one stage of one warp
    float4* ring = reinterpret_cast<float4*>(async_smem + 2 * kPassWarps * kCandStage + kPassWarps * 32) +
                   (size_t)wid * S * stage_f4;
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    // Blocks are handed out on request, one at a time per warp (other kernels share the SMs, so
    // warps advance at different speeds).  A warp knows the block it works on and the next one;
    // the request for the one after that is in flight meanwhile.
    auto request_block = [&]() {
        uint32_t b = 0;
        if (lane == 0) b = atomicAdd(&out.hdr->next_block, 1u);
        return b;
    };
    uint64_t blk = __shfl_sync(0xFFFFFFFFu, request_block(), 0);
    uint64_t blk_next = __shfl_sync(0xFFFFFFFFu, request_block(), 0);
    uint32_t requested = request_block();
    StageCursor cur{0, 0, 0};
    const size_t chunk_words = (size_t)(K + 1) * kStageChunk;
    if (STAGE) {
        cur.chunk = __shfl_sync(0xFFFFFFFFu, stage_request_chunk(out.hdr, lane), 0);
        cur.spare_req = stage_request_chunk(out.hdr, lane);
    }
    // the copies: row `copy_row` of block (copy_ahead ? blk_next : blk) goes to stage `copy_slot`
    uint32_t copy_ahead = 0, copy_row = 0, copy_slot = 0, slot = 0;
    auto copy_next_row = [&]() {
        const uint64_t b = copy_ahead ? blk_next : blk;
        if (b < nb && (b + 1) * kBlock <= n) {   // whole blocks only; the ragged last block is loaded directly
            const uint64_t i4 = (b * kBlock + copy_row * 128u) / 4u + lane;
            float4* dst = ring + copy_slot * stage_f4 + lane;
            if (KT > 0) {
#pragma unroll
                for (int k = 0; k < KR; ++k)
                    cp_async16(dst + k * 32, reinterpret_cast<const float4*>(g.p[k]) + i4, policy);
            } else {
                for (int k = 0; k < K; ++k)
                    cp_async16(dst + k * 32, reinterpret_cast<const float4*>(g.p[k]) + i4, policy);
            }
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
            const uint32_t row0 = (uint32_t)base + r * 128;   // first parameter of the row
            const uint64_t e0 = base + r * 128 + 4 * lane;    // this lane's first parameter of the row
            uint32_t key[4];
            uint32_t in = 0xFu;                               // which of the four exist
            float4 v[KR];                                     // KT > 0: this lane's update values of the row
            cp_async_wait<S - 1>();                           // this row's copies have landed
            const float4* src = ring + slot * stage_f4 + lane;
            if (full) {
                float4 a;
                if (KT > 0) {
#pragma unroll
                    for (int k = 0; k < KR; ++k) v[k] = src[k * 32];
                    a = v[0];
#pragma unroll
                    for (int k = 1; k < KR; ++k) {
                        a.x = __fadd_rn(a.x, v[k].x);
                        a.y = __fadd_rn(a.y, v[k].y);
                        a.z = __fadd_rn(a.z, v[k].z);
                        a.w = __fadd_rn(a.w, v[k].w);
                    }
                } else {
                    a = src[0];
#pragma unroll 4
                    for (int k = 1; k < K; ++k) {
                        const float4 b = src[k * 32];
                        a.x = __fadd_rn(a.x, b.x);
                        a.y = __fadd_rn(a.y, b.y);
                        a.z = __fadd_rn(a.z, b.z);
                        a.w = __fadd_rn(a.w, b.w);
                    }
                }
                const float4 ww = src[K * 32];
                key[0] = __float_as_uint(score_one(c, a.x, ww.x));
                key[1] = __float_as_uint(score_one(c, a.y, ww.y));
                key[2] = __float_as_uint(score_one(c, a.z, ww.z));
                key[3] = __float_as_uint(score_one(c, a.w, ww.w));
            } else if (e0 + 4 <= n) {
                score4(w, g, K, c, e0 / 4, key);
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
            uint32_t nib, cm;
            pass_classify(pw, key, in, &nib, &cm);
            const uint32_t sm = nib | cm;   // to be staged
            const bool stage_row = STAGE && __any_sync(0xFFFFFFFFu, sm != 0);   // warp-uniform
            // order of the row's staged parameters = index order: lane-major, then q
            uint32_t before = 0, total = 0;
            if (stage_row) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t bq = __ballot_sync(0xFFFFFFFFu, (sm >> q) & 1u);
                    before += __popc(bq & pw.lt_mask);
                    total += __popc(bq);
                }
            }
            const bool from_regs = KT > 0 && full;
            if (stage_row && !from_regs) {
                // out of the ring (or, in the ragged last block, out of memory), entry by entry
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if ((sm >> q) & 1u) pos_list[before + __popc(sm & ((1u << q) - 1u))] = (uint8_t)(4 * lane + q);
                __syncwarp();
                const uint32_t spare = __shfl_sync(0xFFFFFFFFu, cur.spare_req, 0);
                const float* row = reinterpret_cast<const float*>(ring + slot * stage_f4);   // [k][128], model last
                for (uint32_t e = lane; e < total; e += 32) {
                    const uint32_t p = pos_list[e];
                    uint32_t at = cur.used + e, ch = cur.chunk;
                    if (at >= kStageChunk) {
                        at -= kStageChunk;
                        ch = spare;
                    }
                    if (ch < stage.max_chunks) {
                        uint32_t* dst = stage.chunks + (size_t)ch * chunk_words + at;
                        dst[0] = row0 + p;
                        if (full) {
#pragma unroll 4
                            for (int k = 0; k < K; ++k)
                                dst[(size_t)(k + 1) * kStageChunk] = __float_as_uint(row[k * 128 + p]);
                        } else {
                            for (int k = 0; k < K; ++k)
                                dst[(size_t)(k + 1) * kStageChunk] = __float_as_uint(g.p[k][(uint64_t)row0 + p]);
                        }
                    }
                }
                __syncwarp();
                stage_advance(cur, total, spare, stage, out.hdr, lane);
            }
            slot = (slot + 1 == S) ? 0 : slot + 1;
            copy_next_row();   // into the stage just read
            if (stage_row && from_regs) {
                // out of registers: every lane places its own members
                const uint32_t spare = __shfl_sync(0xFFFFFFFFu, cur.spare_req, 0);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (!((sm >> q) & 1u)) continue;
                    uint32_t at = cur.used + before + __popc(sm & ((1u << q) - 1u)), ch = cur.chunk;
                    if (at >= kStageChunk) {
                        at -= kStageChunk;
                        ch = spare;
                    }
                    if (ch < stage.max_chunks) {
                        uint32_t* dst = stage.chunks + (size_t)ch * chunk_words + at;
                        dst[0] = (uint32_t)e0 + q;
#pragma unroll
                        for (int k = 0; k < KR; ++k) dst[(size_t)(k + 1) * kStageChunk] = __float_as_uint(f4_get(v[k], q));
                    }
                }
                stage_advance(cur, total, spare, stage, out.hdr, lane);
            }
            pass_row_words(pw, nib, r, &myG);
            pass_candidates(pw, out, key, cm, (uint32_t)e0);
        }
        pass_end_block(pw, out, blk, myG);
        // on to the next block; the copies are S rows into it already
        blk = blk_next;
        blk_next = __shfl_sync(0xFFFFFFFFu, requested, 0);
        requested = request_block();
        --copy_ahead;
    }
    cp_async_wait<0>();
    if (STAGE && lane == 0 && cur.used > 0) {
        if (cur.chunk < stage.max_chunks)
            stage.fill[cur.chunk] = cur.used;
        else
            out.hdr->stage_lost = 1u;
    }
    pass_end(pw, out, &cta_def, scan_smem, res);
}

// ---- step 3: the finishing kernel ------------------------------------------------------------

struct FinishArgs {
    const uint32_t* keys;   // the scores: read by the full path (after this kernel wrote them, if fused)
    ScoreInputs in;         // fused: the model and the updates the scores come from
    int fused;
    int bracketed;
    int given;              // the threshold and the tie quota come with the call (range-sharded selection)
    uint32_t T_given, ties_given;
    uint64_t n, nb;
    uint32_t k, cap;
    WsHeader* hdr;
    uint32_t* hist;         // 6 x 4096: full path rounds 0..2, candidates' digits 1..3
    const uint32_t* cand_key;
    const uint32_t* cand_idx;
    uint32_t* G;
    uint32_t* E;
    unsigned long long* tile_sum;   // per tile of kEmitTile blocks: #greater | #equal << 32
    unsigned long long* super_pref; // per group of tiles: the counts below the group (written here)
    uint32_t* core_idx;
    uint32_t* bitmap;
    uint32_t* dir;
};

template <int ROUND>
__device__ __forceinline__ void full_hist_key(uint32_t key, uint32_t prefix, uint32_t* sh) {
    if (ROUND == 0) {
        atomicAdd(&sh[key >> 20], 1u);
    } else if (ROUND == 1) {
        if ((key >> 20) == (prefix >> 20)) atomicAdd(&sh[(key >> 10) & 1023u], 1u);
    } else {
        if ((key >> 10) == (prefix >> 10)) atomicAdd(&sh[key & 1023u], 1u);
    }
}

// One counting round of the full path over all keys: this CTA's share into shared memory, then
// into the global histogram.  Scalar head up to 16-byte alignment, 128-bit body, scalar tail.
template <int ROUND>
__device__ __forceinline__ void full_hist_round(const uint32_t* keys, uint64_t n, uint32_t prefix, uint32_t* sh,
                                                uint32_t* hist) {
    constexpr uint32_t NB = (ROUND == 0) ? kBins0 : 1024u;
    for (uint32_t b = threadIdx.x; b < NB; b += kFinishThreads) sh[b] = 0;
    __syncthreads();
    const uint64_t mis = (reinterpret_cast<uintptr_t>(keys) & 15u) / 4u;
    uint64_t head = (4u - mis) & 3u;
    if (head > n) head = n;
    const uint64_t body4 = (n - head) / 4;
    const uint64_t tail = n - head - 4 * body4;
    const uint64_t gid = (uint64_t)blockIdx.x * kFinishThreads + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * kFinishThreads;
    if (gid < head) full_hist_key<ROUND>(__ldcg(keys + gid), prefix, sh);
    if (gid < tail) full_hist_key<ROUND>(__ldcg(keys + head + 4 * body4 + gid), prefix, sh);
    const uint4* k4 = reinterpret_cast<const uint4*>(keys + head);
    for (uint64_t i = gid; i < body4; i += stride) {
        const uint4 v = __ldcg(k4 + i);
        full_hist_key<ROUND>(v.x, prefix, sh);
        full_hist_key<ROUND>(v.y, prefix, sh);
        full_hist_key<ROUND>(v.z, prefix, sh);
        full_hist_key<ROUND>(v.w, prefix, sh);
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < NB; b += kFinishThreads) {
        const uint32_t c = sh[b];
        if (c) atomicAdd(&hist[b], c);
    }
}

__global__ void __launch_bounds__(kFinishThreads, 2) finish_kernel(FinishArgs a) {
    __shared__ uint32_t sh[kDigitBins];   // a counting round's histogram
    __shared__ unsigned long long scan_smem[33];
    __shared__ uint32_t res[3];
    WsHeader* hdr = a.hdr;
    const uint32_t t = threadIdx.x, lane = lane_id(), wid = t >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint32_t k = a.k;
    uint32_t epoch = 0;
    const bool cand_mode = a.bracketed && bracket_ok(hdr, k, a.cap);
    uint32_t T = 0xFFFFFFFFu, ties = 0;
    bool failed = false;

    if (cand_mode) {
        // tile_sum holds what the pass counted (certainly-core members only so far)
        const uint32_t b_top = hdr->b_top, b_bot = hdr->b_bot;
        const uint32_t bot_key = b_bot << kBinShift;
        const uint32_t n_cand = hdr->n_cand;
        uint32_t low = cand_low_bits(b_top, b_bot);
        uint32_t prefix = hdr->prefix, rem = hdr->k_rem;   // first digit: found by the pass's last CTA
        const uint32_t gid = blockIdx.x * kFinishThreads + t, gstride = gridDim.x * kFinishThreads;
        int round = 0;
        while (low > 0) {
            const uint32_t d = low < kDigitBits ? low : kDigitBits, shift = low - d;
            uint32_t* hist = a.hist + (4 + round) * kBins0;
            for (uint32_t b = t; b < kDigitBins; b += kFinishThreads) sh[b] = 0;
            __syncthreads();
            // (the list is long on long flat vectors: four keys per load, two loads in flight per thread)
            auto count = [&](uint32_t key) {
                const uint32_t rel = key - bot_key;
                if ((rel >> low) == (prefix >> low)) atomicAdd(&sh[(rel >> shift) & ((1u << d) - 1u)], 1u);
            };
            const uint32_t n4 = n_cand / 4;
            const uint4* key4 = reinterpret_cast<const uint4*>(a.cand_key);
            for (uint32_t c = gid; c < n4; c += 2 * gstride) {
                const uint4 v0 = __ldcg(key4 + c);
                const bool two = c + gstride < n4;
                const uint4 v1 = two ? __ldcg(key4 + c + gstride) : make_uint4(0u, 0u, 0u, 0u);
                count(v0.x), count(v0.y), count(v0.z), count(v0.w);
                if (two) count(v1.x), count(v1.y), count(v1.z), count(v1.w);
            }
            if (gid < n_cand - 4 * n4) count(__ldcg(a.cand_key + 4 * n4 + gid));
            __syncthreads();
            for (uint32_t b = t; b < (1u << d); b += kFinishThreads)
                if (sh[b]) atomicAdd(&hist[b], sh[b]);
            if (!grid_barrier(hdr, &epoch)) return;
            uint32_t bin, r2;
            if (!find_rank_bin<kFinishThreads>(hist, 1u << d, rem, scan_smem, res, &bin, &r2)) {
                failed = true;
                break;
            }
            prefix |= bin << shift;
            rem = r2;
            low = shift;
            ++round;
        }
        T = bot_key + prefix;
        ties = rem;
        if (!failed) {
            // candidates at or above T into the bitmaps and the tile counts
            // (neighbours in the list come from neighbouring parameters: a warp adds to a tile's
            // counter once, not once per candidate)
            // (four stretches of the list per warp and turn, their loads in flight together)
            for (uint64_t c0 = gid - lane; c0 < n_cand; c0 += 4ull * gstride) {
                uint32_t key[4], idx[4];
                bool take[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint64_t c = c0 + (uint64_t)j * gstride + lane;
                    key[j] = (c < n_cand) ? __ldcg(a.cand_key + c) : 0u;
                    take[j] = c < n_cand && key[j] >= T;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    idx[j] = take[j] ? __ldcg(a.cand_idx + c0 + (uint64_t)j * gstride + lane) : 0xFFFFFFFFu;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (c0 + (uint64_t)j * gstride >= n_cand) break;   // warp-uniform
                    const uint32_t i = idx[j];
                    if (take[j]) atomicOr(((key[j] > T) ? a.G : a.E) + (i >> 5), 1u << (i & 31u));
                    const uint32_t tile = take[j] ? i / (kBlock * kEmitTile) : 0xFFFFFFFFu;
                    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, tile);
                    const uint32_t gt = __ballot_sync(0xFFFFFFFFu, take[j] && key[j] > T);
                    if (take[j] && (peers & lt_mask) == 0)   // the first lane of each group adds for the group
                        atomicAdd(&a.tile_sum[tile], (unsigned long long)__popc(peers & gt) |
                                                         ((unsigned long long)__popc(peers & ~gt) << 32));
                }
            }
        }
    } else {
        if (a.given) {
            T = a.T_given;
            ties = a.ties_given;
        } else if (k > 0) {
            if (a.fused) {
                // the scores did not exist yet: write them for the rounds below
                uint32_t* S = const_cast<uint32_t*>(a.keys);
                const uint64_t n4 = a.n / 4;
                const uint64_t stride = (uint64_t)gridDim.x * kFinishThreads;
                const uint64_t gid = (uint64_t)blockIdx.x * kFinishThreads + t;
                for (uint64_t i = gid; i < n4; i += stride) {
                    uint32_t key[4];
                    score4(a.in.w, a.in.g, a.in.K, a.in.c, i, key);
                    reinterpret_cast<uint4*>(S)[i] = make_uint4(key[0], key[1], key[2], key[3]);
                }
                if (gid < a.n - 4 * n4) S[4 * n4 + gid] = score1(a.in.w, a.in.g, a.in.K, a.in.c, 4 * n4 + gid);
                if (!grid_barrier(hdr, &epoch)) return;
            }
            uint32_t prefix = 0, rem = k, bin = 0, r2 = 0;
            full_hist_round<0>(a.keys, a.n, prefix, sh, a.hist);
            if (!grid_barrier(hdr, &epoch)) return;
            failed = !find_rank_bin<kFinishThreads>(a.hist, kBins0, rem, scan_smem, res, &bin, &r2);
            prefix = bin << 20;
            rem = r2;
            if (!failed) {
                full_hist_round<1>(a.keys, a.n, prefix, sh, a.hist + kBins0);
                if (!grid_barrier(hdr, &epoch)) return;
                failed = !find_rank_bin<kFinishThreads>(a.hist + kBins0, 1024u, rem, scan_smem, res, &bin, &r2);
                prefix |= bin << 10;
                rem = r2;
            }
            if (!failed) {
                full_hist_round<2>(a.keys, a.n, prefix, sh, a.hist + 2 * kBins0);
                if (!grid_barrier(hdr, &epoch)) return;
                failed = !find_rank_bin<kFinishThreads>(a.hist + 2 * kBins0, 1024u, rem, scan_smem, res, &bin, &r2);
                prefix |= bin;
                rem = r2;
            }
            T = prefix;
            ties = rem;
        }
        // every key against T: both bitmaps and the tile counts (warp per block).  A bracketed call
        // that ends up here had its tile counts started by the pass: they are rebuilt from zero.
        if (a.bracketed) {
            const uint64_t ntiles = (a.nb + kEmitTile - 1) / kEmitTile;
            for (uint64_t x = (uint64_t)blockIdx.x * kFinishThreads + t; x < ntiles; x += (uint64_t)gridDim.x * kFinishThreads)
                a.tile_sum[x] = 0ull;
            if (!grid_barrier(hdr, &epoch)) return;
        }
        if (!failed) {
            const uint64_t warps = (uint64_t)gridDim.x * (kFinishThreads / 32);
            for (uint64_t blk = (uint64_t)blockIdx.x * (kFinishThreads / 32) + wid; blk < a.nb; blk += warps) {
                const uint64_t base = blk * kBlock;
                uint32_t myG = 0, myE = 0;
                for (int wd = 0; wd < 32; ++wd) {
                    const uint64_t i = base + wd * 32 + lane;
                    const bool in = i < a.n;
                    const uint32_t key = in ? __ldcg(a.keys + i) : 0u;
                    const uint32_t bg = __ballot_sync(0xFFFFFFFFu, in && key > T);
                    const uint32_t be = __ballot_sync(0xFFFFFFFFu, in && key == T);
                    if (lane == (uint32_t)wd) {
                        myG = bg;
                        myE = be;
                    }
                }
                a.G[blk * kWordsPerBlock + lane] = myG;
                a.E[blk * kWordsPerBlock + lane] = myE;
                const uint32_t cg = __reduce_add_sync(0xFFFFFFFFu, __popc(myG));
                const uint32_t ce = __reduce_add_sync(0xFFFFFFFFu, __popc(myE));
                if (lane == 0 && (cg | ce))
                    atomicAdd(&a.tile_sum[blk / kEmitTile], (unsigned long long)cg | ((unsigned long long)ce << 32));
            }
        }
    }
    if (failed) {
        if (t == 0) hdr->status = SLIMDP_ERR_INTERNAL;
        return;
    }

    // the block counts are complete once every CTA is here: sums per group of blocks by all CTAs, then
    // one CTA turns them into the groups' prefixes
    if (!grid_barrier(hdr, &epoch)) return;
    super_sum_phase<kFinishThreads>(a.tile_sum, a.super_pref, a.nb);
    if (!grid_barrier(hdr, &epoch)) return;
    if (blockIdx.x != 0) return;
    if (t == 0) {   // for whoever places the core's members next, and for whoever reads the header afterwards
        hdr->threshold = T;
        hdr->tie_quota = ties;
    }
    tile_scan_phase<kFinishThreads>(a.super_pref, a.n, a.nb, k, ties, hdr, a.dir, scan_smem);
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
    void* stage;              // staging area for the exchange (may be null: nothing is staged)
    size_t stage_bytes;
};

// CTAs of the finishing kernel: one per SM (cooperative launch), fewer for short vectors.
static int finish_grid(uint64_t n, int sms) {
    static std::atomic<int> per_sm_cached[64];   // 0 = not asked yet, < 0 = no cooperative launch here
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    int f = per_sm_cached[dev].load(std::memory_order_relaxed);
    if (f == 0) {
        int per_sm = 0, coop = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, finish_kernel, kFinishThreads, 0) != cudaSuccess)
            return -1;
        f = (coop && per_sm >= 1) ? (per_sm > 2 ? 2 : per_sm) : -1;
        per_sm_cached[dev].store(f, std::memory_order_relaxed);
    }
    if (f < 0) return -1;
    uint64_t grid = (n + 16383) / 16384;
    if (grid > (uint64_t)sms * f) grid = (uint64_t)sms * f;
    return (int)(grid < 1 ? 1 : grid);
}

struct GivenThreshold {
    uint32_t T, ties;
};

// emit = false: the call ends with the finishing kernel; the caller places the core's members itself
// (block_selection on the workspace's bitmaps and counts) and writes core_idx and core_aux.
static slimdp_status launch_select_impl(float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx,
                                        void* core_aux, void* ws, const FusedScore* fused, bool* staged_out,
                                        const GivenThreshold* given, bool emit, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const SelectWs L = select_ws_layout(ws, n);
    const uint64_t nb = num_blocks(n);
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(scores);
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(core_aux);
    uint32_t* dir = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(core_aux) + slimdp_core_aux_dir_offset(n));
    const uint32_t k = (uint32_t)k_core;
    const uint32_t cap = (uint32_t)L.cand_cap;
    if (staged_out) *staged_out = false;

    // header, radix histograms and sample histograms are contiguous: one clear (status = SLIMDP_OK = 0)
    if (cudaMemsetAsync(L.hdr, 0, L.zero_bytes, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
    const bool bracketed = k_core > 0 && n >= kBracketMinN && given == nullptr;
    ScoreInputs in{};
    if (fused) {
        in.w = fused->w;
        in.g = *fused->g;
        in.K = (int)fused->K;
        in.c = fused->c;
    }
    if (bracketed) {
        PassOut out{L.hdr, cap, k, L.G, L.E, L.tile_sum, L.cand_key, L.cand_idx, L.hist + 3 * kBins0};
        if (fused)
            sample_coarse_kernel<true><<<(1u << (kSampleBits - 2)) / 1024, 1024, 0, st>>>(
                keys, in, n, k, L.hdr, L.sample, L.coarse_hist, L.coarse_incl);
        else
            sample_coarse_kernel<false><<<(1u << (kSampleBits - 2)) / 1024, 1024, 0, st>>>(
                keys, in, n, k, L.hdr, L.sample, L.coarse_hist, L.coarse_incl);
        sample_fine_kernel<<<(1u << kSampleBits) / 1024, 1024, 0, st>>>(L.sample, n, k, L.hdr, L.fine_hist,
                                                                        L.coarse_incl);
        SLIMDP_LAUNCHED(2);
        if (fused) {
            const int stages = async_stages(fused->K);
            if (stages <= 0) return SLIMDP_ERR_INTERNAL;   // the caller checked score_select_fusable
            // one CTA per SM, its loads in flight in shared memory (see score_bracket_async_kernel)
            uint64_t agrid = (nb + kPassWarps - 1) / kPassWarps;
            if (agrid > (uint64_t)sms) agrid = (uint64_t)sms;
            StageOut so{nullptr, nullptr, 0};
            bool stage_on = false;
            if (fused->stage != nullptr && 2 * k_core <= n) {
                const StageArea A = stage_layout(fused->stage, n, fused->K, k_core, (uint32_t)sms * kPassWarps);
                if (A.bytes <= fused->stage_bytes && A.max_chunks < 0xFFFFFFFFull) {
                    if (cudaMemsetAsync(A.fill, 0, A.fill_bytes, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
                    so = StageOut{A.fill, A.chunks, (uint32_t)A.max_chunks};
                    stage_on = true;
                }
            }
            if (fused->mark_begin && cudaEventRecord(fused->mark_begin, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
            if (fused->pass_ready && cudaEventRecord(fused->pass_ready, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
            const uint32_t smem = async_fixed_bytes() + (uint32_t)stages * async_stage_bytes(fused->K);
#define SLIMDP_ASYNC_LAUNCH(SS, KK, ST)                                                                             \
    {                                                                                                               \
        auto kern = score_bracket_async_kernel<SS, KK, ST>;                                                             \
        static DeviceOnce attributes;                                                                               \
        if (attributes.needed()) {                                                                                  \
            int dev = 0, optin = 0;                                                                                 \
            cudaFuncAttributes fa;                                                                                  \
            if (cudaGetDevice(&dev) != cudaSuccess ||                                                               \
                cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||      \
                cudaFuncGetAttributes(&fa, kern) != cudaSuccess ||                                                  \
                cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,                             \
                                     optin - (int)fa.sharedSizeBytes) != cudaSuccess ||                             \
                !prefer_max_shared(kern))                                                                           \
                return SLIMDP_ERR_CUDA;                                                                             \
            attributes.mark();                                                                                      \
        }                                                                                                           \
        kern<<<(unsigned)agrid, kPassWarps * 32, smem, st>>>(fused->w, *fused->g, (int)fused->K, fused->c, n, nb,   \
                                                             out, so);                                              \
    }
#define SLIMDP_ASYNC_CASE(SS, KK)                \
    if (stage_on)                                \
        SLIMDP_ASYNC_LAUNCH(SS, KK, true)        \
    else                                         \
        SLIMDP_ASYNC_LAUNCH(SS, KK, false)
            // the worker counts of the usual workloads get their own instantiation (values in registers)
            if (fused->K == 8 && stages == 3) {
                SLIMDP_ASYNC_CASE(3, 8)
            } else if (fused->K == 4 && stages == 5) {
                SLIMDP_ASYNC_CASE(5, 4)
            } else {
                switch (stages) {
                    case 2: SLIMDP_ASYNC_CASE(2, 0) break;
                    case 3: SLIMDP_ASYNC_CASE(3, 0) break;
                    case 4: SLIMDP_ASYNC_CASE(4, 0) break;
                    case 5: SLIMDP_ASYNC_CASE(5, 0) break;
                    case 6: SLIMDP_ASYNC_CASE(6, 0) break;
                    case 7: SLIMDP_ASYNC_CASE(7, 0) break;
                    case 8: SLIMDP_ASYNC_CASE(8, 0) break;
                    default: return SLIMDP_ERR_INTERNAL;
                }
            }
#undef SLIMDP_ASYNC_CASE
#undef SLIMDP_ASYNC_LAUNCH
            SLIMDP_LAUNCHED(1);
            if (staged_out) *staged_out = stage_on;
            if (fused->mark_end && cudaEventRecord(fused->mark_end, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
            if (fused->after_pass) {
                const slimdp_status hs = fused->after_pass(fused->after_arg);
                if (hs != SLIMDP_OK) return hs;
            }
        } else {
            // one wave of CTAs: as many as are resident at once
            const bool vec = aligned16(keys);
            int per_sm = 0;
            if ((vec ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bracket_pass_kernel<true>,
                                                                      kPassWarps * 32, 0)
                     : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bracket_pass_kernel<false>,
                                                                      kPassWarps * 32, 0)) != cudaSuccess ||
                per_sm < 1)
                return SLIMDP_ERR_CUDA;
            uint64_t cgrid = (nb + kPassWarps - 1) / kPassWarps;
            if (cgrid > (uint64_t)sms * per_sm) cgrid = (uint64_t)sms * per_sm;
            if (vec)
                bracket_pass_kernel<true><<<(unsigned)cgrid, kPassWarps * 32, 0, st>>>(keys, n, nb, out);
            else
                bracket_pass_kernel<false><<<(unsigned)cgrid, kPassWarps * 32, 0, st>>>(keys, n, nb, out);
            SLIMDP_LAUNCHED(1);
        }
    }
    const int fgrid = finish_grid(n, sms);
    if (fgrid <= 0) return SLIMDP_ERR_CUDA;
    FinishArgs fa{};
    fa.keys = keys;
    fa.in = in;
    fa.fused = fused != nullptr;
    fa.bracketed = bracketed;
    fa.given = given != nullptr;
    fa.T_given = given ? given->T : 0u;
    fa.ties_given = given ? given->ties : 0u;
    fa.n = n;
    fa.nb = nb;
    fa.k = k;
    fa.cap = cap;
    fa.hdr = L.hdr;
    fa.hist = L.hist;
    fa.cand_key = L.cand_key;
    fa.cand_idx = L.cand_idx;
    fa.G = L.G;
    fa.E = L.E;
    fa.tile_sum = L.tile_sum;
    fa.super_pref = L.super_pref;
    fa.core_idx = core_idx;
    fa.bitmap = bitmap;
    fa.dir = dir;
    void* args[] = {&fa};
    if (cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(finish_kernel), dim3((unsigned)fgrid),
                                    dim3(kFinishThreads), args, 0, st) != cudaSuccess)
        return SLIMDP_ERR_CUDA;
    SLIMDP_LAUNCHED(1);
    if (!emit) return SLIMDP_OK;
    return launch_emit(L.G, L.E, L.tile_sum, L.super_pref, n, k, L.hdr, core_idx, bitmap, dir, st);
}

slimdp_status launch_select(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx, void* core_aux,
                            void* ws, bool emit, cudaStream_t st) {
    return launch_select_impl(const_cast<float*>(scores), n, k_core, core_idx, core_aux, ws, nullptr, nullptr, nullptr,
                              emit, st);
}

// A shard's part of the core for a threshold and a tie quota that were found over all shards.
slimdp_status launch_select_given(const float* scores, uint64_t n, uint32_t T, uint32_t ties, uint64_t k_shard,
                                  uint32_t* core_idx, void* core_aux, void* ws, cudaStream_t st) {
    const GivenThreshold gt{T, ties};
    return launch_select_impl(const_cast<float*>(scores), n, k_shard, core_idx, core_aux, ws, nullptr, nullptr, &gt, true,
                              st);
}

// Whether scoring can be folded into the selection for these sizes and alignments.
bool score_select_fusable(uint64_t n, uint64_t k_core, uint32_t K, bool vec) {
    return vec && k_core > 0 && n >= kBracketMinN && async_stages(K) > 0;
}

// Bytes of staging area that let the one-call round set the core's update values aside during its pass
// (0: staging does not apply to these sizes).
size_t stage_bytes_for(uint64_t n, uint32_t K, uint64_t k_core) {
    const int sms = sm_count();
    if (sms <= 0 || n < kBracketMinN || k_core == 0 || 2 * k_core > n || async_stages(K) <= 0) return 0;
    return stage_layout(nullptr, n, K, k_core, (uint32_t)sms * kPassWarps).bytes;
}

slimdp_status launch_score_select(const float* w, const PtrArray<const float>& g, uint32_t K, float c, uint64_t n,
                                  float* scores, uint64_t k_core, uint32_t* core_idx, void* core_aux, void* ws,
                                  cudaEvent_t mark_begin, cudaEvent_t mark_end, slimdp_status (*after_pass)(void*),
                                  void* after_arg, cudaEvent_t pass_ready, void* stage, size_t stage_bytes,
                                  bool* staged, bool emit, cudaStream_t st) {
    const FusedScore f{w, &g, K, c, mark_begin, mark_end, after_pass, after_arg, pass_ready, stage, stage_bytes};
    return launch_select_impl(scores, n, k_core, core_idx, core_aux, ws, &f, staged, nullptr, emit, st);
}

}  // namespace slimdp
