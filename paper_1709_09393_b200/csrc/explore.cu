// slimdp_sample_explore: the exploration operator T_R^k (Section 3.1 item 2,
// Section 3.3 step 2): k_exp distinct parameters drawn uniformly from outside
// the core, anew for every worker and every communication round.
//
// The explorer is { select0(pi(j)) : j < k_exp }, ascending, where pi is the
// keyed permutation of the M non-core ranks and select0(r) the r-th non-core
// parameter.  select0 is monotone, so sorting the ranks sorts the indices, and
// the ranks are uniform on [0, M), so a bucket sort by the ranks' high bits
// is balanced:
//   1. setup: round keys (three Philox-4x32-10 blocks per worker);
//   2. rank: thread j evaluates pi(j) (10-round alternating Feistel network
//      with cycle walking), stores it and counts it into its bucket (rank >> s);
//   3. two-kernel exclusive scan of the bucket counts;
//   4. scatter: every rank goes to its bucket's slice (order inside a bucket
//      is arbitrary here and is fixed by the next step);
//   5. bucket: one CTA per (bucket, worker) marks its ranks in a 2^s-bit
//      shared-memory bitmap, which sorts them; a block scan of the popcounts
//      gives each rank its output position, and a select0 query (binary
//      search of the per-64 non-core directory inside the bucket's range,
//      seeded by interpolation, then the group's 2 bitmap words, skipped when
//      the group holds no core parameter) turns it into the parameter index.
// No global bitmap, no inter-CTA waiting; the result does not depend on the
// order in which atomics land.
#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

namespace {

constexpr int kBucketThreads = 256;
constexpr size_t kGroupSmemMax = 200 * 1024;   // shared memory the scatter step may use to group a chunk


__device__ __forceinline__ void philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1, uint32_t c2,
                                              uint32_t c3, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0;
        c1 = lo1;
        c2 = n2;
        c3 = lo0;
        if (r < 9) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

// Largest block b in [lo, hi] with dir[b] <= x (dir[lo] <= x is given).
__device__ __forceinline__ uint32_t find_block(const uint32_t* __restrict__ dir, uint32_t lo, uint32_t hi,
                                               uint32_t x) {
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo + 1) >> 1);
        if (__ldg(dir + mid) <= x)
            lo = mid;
        else
            hi = mid - 1;
    }
    return lo;
}

// Round keys per worker, and per rank bucket the directory entry (64-parameter group) that holds
// the bucket's first rank (bounds[buckets] = the group of the last rank M - 1).  The bounds
// depend on the core only.
__global__ void explore_setup_kernel(WsHeader* hdr, uint32_t* __restrict__ rk, uint32_t seed_lo, uint32_t seed_hi,
                                     uint32_t first_worker, uint32_t workers, uint32_t round,
                                     const uint32_t* __restrict__ dir, uint32_t nd, uint32_t M, uint32_t s,
                                     uint32_t buckets, uint32_t* __restrict__ bounds, int parts) {
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if ((parts & 1) && t == 0) hdr->status = SLIMDP_OK;
    if ((parts & 1) && t < workers * 3) {
        const uint32_t w = t / 3, b = t % 3;
        uint32_t out[4];
        philox4x32_10(seed_lo, seed_hi, b, first_worker + w, round, 0x534C494Du, out);
#pragma unroll
        for (int q = 0; q < 4; ++q) rk[w * 12 + b * 4 + q] = out[q];
    }
    // one warp per bucket boundary: a 32-way search (5 probes for 2^25 entries instead of 25)
    const uint32_t bnd = t >> 5, lane = t & 31u;
    if ((parts & 2) && M > 0 && bnd <= buckets) {
        const uint64_t first = (uint64_t)bnd << s;
        const uint32_t rank = (first < M) ? (uint32_t)first : M - 1;
        uint32_t lo = 0, hi = nd - 1;   // the answer is the largest d in [lo, hi] with dir[d] <= rank; dir[lo] <= rank
        while (hi > lo) {
            const uint32_t step = (hi - lo) / 32u + 1u;              // lane probes lo + lane * step
            const uint64_t p = (uint64_t)lo + (uint64_t)lane * step;
            const bool le = p <= hi && __ldg(dir + p) <= rank;       // true for a prefix of the lanes (lane 0 always)
            const uint32_t c = __popc(__ballot_sync(0xFFFFFFFFu, le));
            const uint32_t nlo = lo + (c - 1u) * step;
            const uint64_t nhi = (uint64_t)nlo + step - 1u;
            lo = nlo;
            hi = (nhi < hi) ? (uint32_t)nhi : hi;
        }
        if (lane == 0) bounds[bnd] = lo;
    }
}

// grid = (chunks, workers).  rho[w][j] = pi(j) for the CTA's chunk of j; cnt[w][rho >> s] += 1.
// Lanes whose walk has ended take the next j of their warp's range at once, so a
// long cycle walk in one lane does not idle the other 31.
template <bool SMEM_HIST>
__global__ void __launch_bounds__(1024) rank_kernel(uint32_t M, uint32_t k_exp, uint32_t chunk, uint32_t bits,
                                                    uint32_t s, uint32_t buckets,
                                                    const uint32_t* __restrict__ rk_all, uint32_t* __restrict__ rho,
                                                    uint64_t rho_stride, unsigned long long* __restrict__ cnt,
                                                    uint64_t cnt_stride, uint32_t* __restrict__ cta_hist) {
    extern __shared__ uint32_t sh_hist[];
    const uint32_t worker = blockIdx.y, lane = lane_id();
    if (SMEM_HIST) {
        for (uint32_t b = threadIdx.x; b < buckets; b += blockDim.x) sh_hist[b] = 0;
        __syncthreads();
    }
    uint32_t rk[10];
#pragma unroll
    for (int r = 0; r < 10; ++r) rk[r] = rk_all[worker * 12 + r];
    // x = A * 2^c + B, A of a = floor(bits / 2) bits, B of c = bits - a bits
    const uint32_t a = bits >> 1, c = bits - a;
    const uint32_t maskA = (1u << a) - 1u, maskB = (1u << c) - 1u;
    uint32_t* my_rho = rho + (uint64_t)worker * rho_stride;
    unsigned long long* my_cnt = cnt + (uint64_t)worker * cnt_stride;
    // this warp's contiguous range of j
    const uint64_t c0 = (uint64_t)blockIdx.x * chunk;
    const uint64_t c1 = (c0 + chunk < k_exp) ? c0 + chunk : k_exp;
    const uint32_t warps = blockDim.x >> 5, wid = threadIdx.x >> 5;
    const uint64_t span = (c1 > c0) ? (c1 - c0 + warps - 1) / warps : 0;
    uint64_t next = c0 + (uint64_t)wid * span;
    const uint64_t stop = (next + span < c1) ? next + span : c1;
    bool have = false;
    uint32_t x = 0, j = 0;
    while (true) {
        const uint32_t want = __ballot_sync(0xFFFFFFFFu, !have);
        if (!have) {
            const uint64_t cand = next + __popc(want & ((1u << lane) - 1u));
            if (cand < stop) {
                j = (uint32_t)cand;
                x = j;
                have = true;
            }
        }
        next += __popc(want);
        if (__ballot_sync(0xFFFFFFFFu, have) == 0) break;
        if (have) {
            uint32_t A = x >> c, B = x & maskB;
#pragma unroll
            for (int r = 0; r < 10; ++r) {
                // even rounds change A by a function of B, odd rounds change B by a function of A
                const unsigned long long mult = (r & 1) ? 0xCD9E8D57ull : 0xD2511F53ull;
                const uint32_t v = ((r & 1) ? A : B) ^ rk[r];
                const unsigned long long prod = (unsigned long long)v * mult;   // one 32x32->64 multiply
                const uint32_t F = (uint32_t)(prod >> 32) ^ (uint32_t)prod;
                if (r & 1)
                    B = (B ^ F) & maskB;
                else
                    A = (A ^ F) & maskA;
            }
            x = (A << c) | B;
            if (x < M) {          // the walk ends at the first image inside [0, M)
                my_rho[j] = x;
                if (SMEM_HIST)
                    atomicAdd(&sh_hist[x >> s], 1u);
                else
                    atomicAdd(&my_cnt[x >> s], 1ull);
                have = false;
            }
        }
    }
    if (SMEM_HIST) {
        __syncthreads();
        // the chunk's own histogram is kept for the scatter step, which reserves bucket space with it
        uint32_t* mine = cta_hist + ((uint64_t)worker * gridDim.x + blockIdx.x) * buckets;
        for (uint32_t b = threadIdx.x; b < buckets; b += blockDim.x) {
            const uint32_t c = sh_hist[b];
            mine[b] = c;
            if (c) atomicAdd(&my_cnt[b], (unsigned long long)c);
        }
    }
}

// grid = (chunks, workers).  Move every rank of the chunk into its bucket's slice of `sorted`.
// SMEM: with the chunk's histogram from the rank step the CTA reserves one contiguous piece of
// every bucket's slice (a single global atomic per bucket) and hands out places inside it from
// shared memory.  GROUP (needs SMEM): the chunk is first grouped by bucket in shared memory and
// then copied out, so that a warp's stores fall into a few runs instead of 32 separate sectors.
template <bool SMEM, bool GROUP>
__global__ void __launch_bounds__(1024) scatter_kernel(uint32_t k_exp, uint32_t chunk, uint32_t s, uint32_t buckets,
                                                       const uint32_t* __restrict__ rho, uint64_t rho_stride,
                                                       const unsigned long long* __restrict__ pref,
                                                       uint64_t cnt_stride, uint32_t* __restrict__ cursor,
                                                       const uint32_t* __restrict__ cta_hist,
                                                       uint32_t* __restrict__ sorted) {
    extern __shared__ uint32_t sh[];
    __shared__ unsigned long long scan_smem[33];
    uint32_t* sh_place = sh;                  // per bucket: first / next free global place of this CTA's piece
    uint32_t* sh_first = sh + buckets;        // GROUP: first local place of the bucket's run
    uint32_t* sh_next = sh + 2 * buckets;     // GROUP: next free local place
    uint32_t* sh_sorted = sh + 3 * buckets;   // GROUP: the chunk, grouped by bucket
    const uint32_t worker = blockIdx.y;
    const uint32_t* my_rho = rho + (uint64_t)worker * rho_stride;
    uint32_t* my_sorted = sorted + (uint64_t)worker * rho_stride;
    const unsigned long long* my_pref = pref + (uint64_t)worker * cnt_stride;
    uint32_t* my_cur = cursor + (uint64_t)worker * cnt_stride;
    const uint64_t c0 = (uint64_t)blockIdx.x * chunk;
    const uint64_t c1 = (c0 + chunk < k_exp) ? c0 + chunk : k_exp;
    if (SMEM) {
        const uint32_t* mine = cta_hist + ((uint64_t)worker * gridDim.x + blockIdx.x) * buckets;
        if (GROUP) {
            // local run offsets: exclusive scan of the chunk's histogram, consecutive buckets per thread
            const uint32_t per = (buckets + blockDim.x - 1) / blockDim.x;
            const uint32_t b0 = threadIdx.x * per;
            unsigned long long sum = 0;
            for (uint32_t q = 0; q < per; ++q)
                if (b0 + q < buckets) sum += mine[b0 + q];
            unsigned long long total;
            uint32_t run = (uint32_t)block_exclusive_scan64<32>(sum, scan_smem, &total);
            for (uint32_t q = 0; q < per; ++q) {
                const uint32_t b = b0 + q;
                if (b < buckets) {
                    const uint32_t c = mine[b];
                    sh_first[b] = run;
                    sh_next[b] = run;
                    sh_place[b] = c ? (uint32_t)my_pref[b] + atomicAdd(&my_cur[b], c) : 0u;
                    run += c;
                }
            }
        } else {
            for (uint32_t b = threadIdx.x; b < buckets; b += blockDim.x) {
                const uint32_t c = mine[b];
                sh_place[b] = c ? (uint32_t)my_pref[b] + atomicAdd(&my_cur[b], c) : 0u;
            }
        }
        __syncthreads();
    }
    for (uint64_t j0 = c0 + threadIdx.x; j0 < c1; j0 += 4ull * blockDim.x) {
        uint32_t x[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            x[q] = (j < c1) ? my_rho[j] : 0u;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint64_t j = j0 + (uint64_t)q * blockDim.x;
            if (j < c1) {
                const uint32_t b = x[q] >> s;
                if (GROUP) {
                    sh_sorted[atomicAdd(&sh_next[b], 1u)] = x[q];
                } else {
                    const uint32_t pos =
                        SMEM ? atomicAdd(&sh_place[b], 1u) : (uint32_t)my_pref[b] + atomicAdd(&my_cur[b], 1u);
                    if (pos < k_exp) my_sorted[pos] = x[q];
                }
            }
        }
    }
    if (GROUP) {
        __syncthreads();
        const uint32_t len = (c1 > c0) ? (uint32_t)(c1 - c0) : 0u;
        for (uint32_t p = threadIdx.x; p < len; p += blockDim.x) {
            const uint32_t x = sh_sorted[p];
            const uint32_t b = x >> s;
            const uint32_t pos = sh_place[b] + (p - sh_first[b]);
            if (pos < k_exp) my_sorted[pos] = x;
        }
    }
}

// Shared-memory index of bitmap word w: one pad word per 32 keeps a thread's run of
// consecutive words (stride 2, 4 or 8 across lanes) free of bank conflicts.
__device__ __forceinline__ uint32_t sw(uint32_t w) { return w + (w >> 5); }

constexpr uint32_t kDirCache = 2048;
constexpr uint32_t kListCap = 4096;

// grid = (buckets, workers).  Sort the bucket's ranks through a shared bitmap and emit parameter indices.
__global__ void __launch_bounds__(kBucketThreads) bucket_kernel(
    const uint32_t* __restrict__ bitmap, const uint32_t* __restrict__ dir, const uint32_t* __restrict__ bounds,
    uint32_t k_exp, uint32_t s, const uint32_t* __restrict__ sorted, uint64_t rho_stride,
    const unsigned long long* __restrict__ cnt, const unsigned long long* __restrict__ pref,
    const unsigned long long* __restrict__ totals, uint64_t cnt_stride, PtrArray<uint32_t> out, WsHeader* hdr) {
    __shared__ uint32_t bm[2048 + 64];           // up to 2^16 rank bits, padded (see sw)
    __shared__ uint32_t dir_sh[kDirCache + 1];   // directory entries of the bucket's 64-parameter groups (+1)
    __shared__ uint16_t list[kListCap];          // sorted ranks (low s bits) of the current round
    __shared__ uint32_t warp_sums[kBucketThreads / 32];
    const uint32_t worker = blockIdx.y, bucket = blockIdx.x, t = threadIdx.x;
    const uint32_t words = 1u << (s - 5);
    const uint32_t per = words / kBucketThreads;   // 1, 2, 4 or 8 words per thread
    const uint32_t count = (uint32_t)cnt[(uint64_t)worker * cnt_stride + bucket];
    const uint32_t offset = (uint32_t)pref[(uint64_t)worker * cnt_stride + bucket];
    if (bucket == 0 && t == 0 && totals[worker] != k_exp) hdr->status = SLIMDP_ERR_INTERNAL;
    if (count == 0) return;
    for (uint32_t i = t; i < words + (words >> 5); i += kBucketThreads) bm[i] = 0;
    // the bucket's ranks live in directory groups [grp_lo, grp_hi]
    const uint32_t grp_lo = __ldg(bounds + bucket), grp_hi = __ldg(bounds + bucket + 1);
    const uint32_t ngrp = grp_hi - grp_lo + 1;
    const bool cached = ngrp <= kDirCache;
    if (cached)
        for (uint32_t i = t; i <= ngrp; i += kBucketThreads) dir_sh[i] = __ldg(dir + grp_lo + i);
    __syncthreads();
    // groups per rank inside this bucket, for the interpolated first guess of select0
    const uint32_t dir_first = cached ? dir_sh[0] : 0u;
    const float groups_per_rank = cached ? (float)ngrp / (float)(dir_sh[ngrp] - dir_sh[0] + 1u) : 0.0f;
    const uint32_t* my_sorted = sorted + (uint64_t)worker * rho_stride + offset;
    const uint32_t low_mask = (1u << s) - 1u;
    for (uint32_t e = t; e < count; e += kBucketThreads) {
        const uint32_t r = my_sorted[e] & low_mask;
        atomicOr(&bm[sw(r >> 5)], 1u << (r & 31u));
    }
    __syncthreads();
    // place of this thread's first rank in the sorted order: exclusive scan of the popcounts
    uint32_t mine = 0;
    for (uint32_t q = 0; q < per; ++q) mine += __popc(bm[sw(t * per + q)]);
    const uint32_t inc = warp_inclusive_scan(mine);
    if ((t & 31u) == 31u) warp_sums[t >> 5] = inc;
    __syncthreads();
    uint32_t base = inc - mine;
    for (uint32_t wdx = 0; wdx < (t >> 5); ++wdx) base += warp_sums[wdx];
    uint32_t total = 0;
    for (uint32_t wdx = 0; wdx < kBucketThreads / 32; ++wdx) total += warp_sums[wdx];
    if (t == 0 && total != count) hdr->status = SLIMDP_ERR_INTERNAL;   // two ranks collided: pi is not injective
    uint32_t* dst = out.p[worker] + offset;
    const uint32_t first_rank = bucket << s;
    // rounds of up to kListCap ranks: write them to `list` in sorted order, then share them out evenly
    for (uint32_t r0 = 0; r0 < count; r0 += kListCap) {
        if (base < r0 + kListCap && base + mine > r0) {
            uint32_t p = base;
            for (uint32_t q = 0; q < per; ++q) {
                uint32_t word = bm[sw(t * per + q)];
                while (word) {
                    const uint32_t bit = __ffs(word) - 1;
                    word &= word - 1;
                    if (p >= r0 && p < r0 + kListCap) list[p - r0] = (uint16_t)((t * per + q) * 32u + bit);
                    ++p;
                }
            }
        }
        __syncthreads();
        const uint32_t m = (count - r0 < kListCap) ? count - r0 : kListCap;
        uint32_t rel = 0;     // group relative to grp_lo; ranks ascend inside a thread, so it only moves up
        for (uint32_t e = t; e < m; e += kBucketThreads) {
            const uint32_t rank = first_rank + list[e];
            // select0(rank): the 64-parameter group from the directory ...
            uint32_t d0, d1;
            if (cached) {
                uint32_t lo = rel, hi = ngrp - 1;
                // the directory is close to linear inside one bucket: try a small window around the
                // interpolated group first, and search the whole range only if the window misses
                const uint32_t guess = (uint32_t)((float)(rank - dir_first) * groups_per_rank);
                const uint32_t wl = (guess > 8u) ? guess - 8u : 0u;
                const uint32_t win_lo = (wl > lo) ? wl : lo;
                const uint32_t win_hi = (guess + 8u < hi) ? guess + 8u : hi;
                if (win_lo <= win_hi && dir_sh[win_lo] <= rank && dir_sh[win_hi + 1] > rank) {
                    lo = win_lo;
                    hi = win_hi;
                }
                while (lo < hi) {
                    const uint32_t mid = lo + ((hi - lo + 1) >> 1);
                    if (dir_sh[mid] <= rank)
                        lo = mid;
                    else
                        hi = mid - 1;
                }
                rel = lo;
                d0 = dir_sh[rel];
                d1 = dir_sh[rel + 1];
            } else {
                rel = find_block(dir, grp_lo + rel, grp_hi, rank) - grp_lo;
                d0 = __ldg(dir + grp_lo + rel);
                d1 = __ldg(dir + grp_lo + rel + 1);
            }
            const uint32_t grp = grp_lo + rel;
            const uint32_t rem = rank - d0;
            uint32_t idx;
            if (d1 - d0 == kDirStride) {
                idx = grp * kDirStride + rem;   // no core parameter in this group
            } else {
                // ... then the rem-th zero bit of the group's two bitmap words
                const uint2 v = __ldg(reinterpret_cast<const uint2*>(bitmap + (uint64_t)grp * kWordsPerDir));
                const uint32_t z0 = ~v.x, z1 = ~v.y;
                const uint32_t c0 = __popc(z0);
                const bool second = rem >= c0;
                const uint32_t z = second ? z1 : z0;
                const uint32_t r = second ? rem - c0 : rem;
                idx = (r < (uint32_t)__popc(z)) ? grp * kDirStride + (second ? 32u : 0u) + nth_set_bit(z, r)
                                                : 0xFFFFFFFFu;
            }
            if (idx == 0xFFFFFFFFu || offset + r0 + e >= k_exp) {
                hdr->status = SLIMDP_ERR_INTERNAL;   // directory and bitmap disagree
            } else {
                dst[r0 + e] = idx;
            }
        }
        __syncthreads();
    }
}

}  // namespace

uint32_t explore_bucket_shift(uint64_t M) {
    int lg = 0;
    while (lg < 63 && (2ull << lg) <= M) ++lg;   // floor(log2(M)) for M >= 1
    int extra = lg - 22;
    if (extra < 0) extra = 0;
    if (extra > 3) extra = 3;
    return (uint32_t)(13 + extra);
}

// parts: 1 = the steps that need only the sizes (round keys, ranks, bucket grouping),
//        2 = the steps that need the core (bucket bounds, parameter indices), 3 = everything.
slimdp_status launch_explore_parts(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                                   uint32_t first_worker, uint32_t workers, uint32_t round,
                                   const PtrArray<uint32_t>& out, void* ws, int parts, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const ExploreWs L = explore_ws_layout(ws, n, k_exp, workers);
    const uint64_t nd = num_blocks(n) * kDirPerBlock;
    const uint64_t M = n - k_core;
    const uint32_t* bitmap = reinterpret_cast<const uint32_t*>(core_aux);
    const uint32_t* dir =
        reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(core_aux) + slimdp_core_aux_dir_offset(n));
    const uint32_t s = explore_bucket_shift(M);
    const uint64_t buckets = (M + (1ull << s) - 1) >> s;

    const unsigned setup_threads =
        (unsigned)(((buckets + 1) * 32 > 3ull * workers) ? (buckets + 1) * 32 : 3ull * workers);
    explore_setup_kernel<<<(setup_threads + 255) / 256, 256, 0, st>>>(L.hdr, L.round_keys, (uint32_t)seed,
                                                                      (uint32_t)(seed >> 32), first_worker, workers,
                                                                      round, dir, (uint32_t)nd, (uint32_t)M, s,
                                                                      (uint32_t)buckets, L.bounds, parts);
    SLIMDP_LAUNCHED(1);
    if (k_exp == 0) return SLIMDP_OK;
    if (parts & 1) {
    if (cudaMemsetAsync(L.cnt, 0, L.zero_bytes, st) != cudaSuccess) return SLIMDP_ERR_CUDA;

    uint32_t bits = 2;   // the permutation's domain is [0, 2^bits), the smallest that holds M (at least 4)
    while (((uint64_t)1 << bits) < M) ++bits;

    // about two 1024-thread CTAs per SM over all workers; every CTA owns one contiguous chunk of j
    uint64_t chunks = ((uint64_t)sms * 2 + workers - 1) / workers;
    if (chunks * workers > kMaxExploreCtas) chunks = kMaxExploreCtas / workers;
    if (chunks > (k_exp + 1023) / 1024) chunks = (k_exp + 1023) / 1024;
    if (chunks == 0) chunks = 1;
    const uint32_t chunk = (uint32_t)((k_exp + chunks - 1) / chunks);
    const dim3 grid((unsigned)chunks, workers);
    const bool smem = buckets <= kMaxSmemBuckets;
    if (smem) {
        rank_kernel<true><<<grid, 1024, buckets * 4, st>>>((uint32_t)M, (uint32_t)k_exp, chunk, bits, s,
                                                           (uint32_t)buckets, L.round_keys, L.rho, L.rho_stride,
                                                           L.cnt, L.cnt_stride, L.cta_hist);
    } else {
        rank_kernel<false><<<grid, 1024, 0, st>>>((uint32_t)M, (uint32_t)k_exp, chunk, bits, s, (uint32_t)buckets,
                                                  L.round_keys, L.rho, L.rho_stride, L.cnt, L.cnt_stride,
                                                  L.cta_hist);
    }
    SLIMDP_LAUNCHED(1);
    slimdp_status rc =
        launch_block_scan(L.cnt, L.pref, L.tile_sums, L.totals, buckets, workers, L.cnt_stride, L.tile_stride, st);
    if (rc != SLIMDP_OK) return rc;
    const size_t group_smem = (3 * buckets + chunk) * 4;
    if (smem && group_smem <= kGroupSmemMax) {
        if (group_smem > 48 * 1024 &&
            cudaFuncSetAttribute(scatter_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)group_smem) != cudaSuccess)
            return SLIMDP_ERR_CUDA;
        scatter_kernel<true, true><<<grid, 1024, group_smem, st>>>((uint32_t)k_exp, chunk, s, (uint32_t)buckets,
                                                                   L.rho, L.rho_stride, L.pref, L.cnt_stride,
                                                                   L.cursor, L.cta_hist, L.sorted);
    } else if (smem) {
        scatter_kernel<true, false><<<grid, 1024, buckets * 4, st>>>((uint32_t)k_exp, chunk, s, (uint32_t)buckets,
                                                                     L.rho, L.rho_stride, L.pref, L.cnt_stride,
                                                                     L.cursor, L.cta_hist, L.sorted);
    } else {
        scatter_kernel<false, false><<<grid, 1024, 0, st>>>((uint32_t)k_exp, chunk, s, (uint32_t)buckets, L.rho,
                                                     L.rho_stride, L.pref, L.cnt_stride, L.cursor, L.cta_hist,
                                                     L.sorted);
    }
    SLIMDP_LAUNCHED(1);
    }   // parts & 1
    if (!(parts & 2)) return SLIMDP_OK;
    bucket_kernel<<<dim3((unsigned)buckets, workers), kBucketThreads, 0, st>>>(
        bitmap, dir, L.bounds, (uint32_t)k_exp, s, L.sorted, L.rho_stride, L.cnt, L.pref, L.totals, L.cnt_stride,
        out, L.hdr);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

slimdp_status launch_explore(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                             uint32_t first_worker, uint32_t workers, uint32_t round,
                             const PtrArray<uint32_t>& out, void* ws, cudaStream_t st) {
    return launch_explore_parts(core_aux, n, k_core, k_exp, seed, first_worker, workers, round, out, ws, 3, st);
}

// ---- explorer sampling without a caller-supplied workspace ---------------------------------

// Scratch for slimdp_sample_explore_static.  The array lives in every device that loads this
// library, from load to process exit.  Its name is only a handle in host code; the device
// address comes from cudaGetSymbolAddress (once per device, cached below).
constexpr size_t kStaticScratchBytes = (size_t)SLIMDP_STATIC_SCRATCH_MIB << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

slimdp_status launch_explore_static(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                                    uint32_t worker, uint32_t round, uint32_t* exp_idx, int32_t* status_out,
                                    cudaStream_t st) {
    static void* scratch_addr[64];   // per device; every thread that races here stores the same value
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLIMDP_ERR_CUDA;
    if (scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return SLIMDP_ERR_CUDA;
        scratch_addr[dev] = p;
    }
    if (explore_ws_layout(nullptr, n, k_exp, 1).bytes > kStaticScratchBytes) return SLIMDP_ERR_UNSUPPORTED;
    PtrArray<uint32_t> out;
    for (auto& q : out.p) q = nullptr;
    out.p[0] = exp_idx;
    void* ws = scratch_addr[dev];
    // launch_explore clears the counters it needs at zero and resets the status word on every call
    slimdp_status rc = launch_explore(core_aux, n, k_core, k_exp, seed, worker, 1, round, out, ws, st);
    if (rc != SLIMDP_OK) return rc;
    if (status_out != nullptr &&
        cudaMemcpyAsync(status_out, ws, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return SLIMDP_ERR_CUDA;
    return SLIMDP_OK;
}

}  // namespace slimdp
