// slimdp_sample_explore: the exploration operator T_R^k (Section 3.1 item 2,
// Section 3.3 step 2): k_exp distinct parameters drawn uniformly from outside
// the core, anew for every worker and every communication round.
//
// The explorer is { select0(pi(j)) : j < k_exp }, ascending, where pi is the
// keyed permutation of the M non-core ranks and select0(r) the r-th non-core
// parameter.  select0 is monotone, so sorting the ranks sorts the indices, and
// the ranks are uniform on [0, M), so a bucket sort by the ranks' high bits
// is balanced:
//   1. rank: every CTA derives its worker's round keys (three Philox-4x32-10
//      blocks); thread j evaluates pi(j) (10-round alternating Feistel network
//      with cycle walking), stores it and counts it into its bucket (rank >> s);
//      the last CTA of a worker to finish scans that worker's bucket counts;
//   2. scatter: every rank goes to its bucket's slice (order inside a bucket
//      is arbitrary here and is fixed by the next step);
//   3. bucket: one CTA per (bucket, worker) marks its ranks in a 2^s-bit
//      shared-memory bitmap, which sorts them; a block scan of the popcounts
//      gives each rank its output position, and a select0 query (binary
//      search of the per-64 non-core directory inside the bucket's range,
//      seeded by interpolation, then the group's 2 bitmap words, skipped when
//      the group holds no core parameter) turns it into the parameter index.
// No global bitmap, no inter-CTA waiting; the result does not depend on the
// order in which atomics land.
#include <atomic>
#include <type_traits>

#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

namespace {

constexpr int kBucketThreads = 256;
constexpr size_t kGroupSmemMax = 200 * 1024;   // shared memory the scatter step may use to group a chunk
constexpr size_t kGroupSmemLean = 80 * 1024;   // the same when it has to fit beside another kernel's CTA


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

// What identifies a call's random stream, and where the rank step leaves its by-products.
struct RankStream {
    uint32_t seed_lo, seed_hi, first_worker, round;
    WsHeader* hdr;
    uint32_t* ticket;              // per worker, cleared before the launch
    unsigned long long* pref;      // per worker: exclusive prefix sums of the bucket counts
    unsigned long long* totals;    // per worker: their sum
};

// grid = (chunks, workers), 1024 threads.  rho[w][j] = pi(j) for the CTA's chunk of j;
// cnt[w][rho >> s] += 1.  Every CTA derives its worker's round keys itself (three Philox-4x32-10
// blocks).  Lanes whose walk has ended take the next j of their warp's range at once, so a
// long cycle walk in one lane does not idle the other 31.  The last CTA of a worker to finish
// turns that worker's bucket counts into their exclusive prefix sums.
template <bool SMEM_HIST>
__global__ void __launch_bounds__(1024) rank_kernel(uint32_t M, uint32_t k_exp, uint32_t chunk, uint32_t bits,
                                                    uint32_t s, uint32_t buckets, RankStream rs,
                                                    uint32_t* __restrict__ rho, uint64_t rho_stride,
                                                    unsigned long long* __restrict__ cnt, uint64_t cnt_stride,
                                                    uint32_t* __restrict__ cta_hist) {
    extern __shared__ uint32_t sh_hist[];
    __shared__ uint32_t sh_rk[12];
    __shared__ unsigned long long scan_smem[33];
    __shared__ bool last_of_worker;
    const uint32_t worker = blockIdx.y, lane = lane_id();
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) rs.hdr->status = SLIMDP_OK;   // no kernel before this one reports
    if (threadIdx.x < 3) {
        uint32_t out[4];
        philox4x32_10(rs.seed_lo, rs.seed_hi, threadIdx.x, rs.first_worker + worker, rs.round, 0x534C494Du, out);
#pragma unroll
        for (int q = 0; q < 4; ++q) sh_rk[threadIdx.x * 4 + q] = out[q];
    }
    if (SMEM_HIST)
        for (uint32_t b = threadIdx.x; b < buckets; b += blockDim.x) sh_hist[b] = 0;
    __syncthreads();
    uint32_t rk[10];
#pragma unroll
    for (int r = 0; r < 10; ++r) rk[r] = sh_rk[r];
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
    // "last CTA done" per worker: the block barrier orders this CTA's atomics before thread 0's
    // device-wide fence, the fence orders them before the ticket
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        last_of_worker = atomicAdd(&rs.ticket[worker], 1u) == gridDim.x - 1;
        __threadfence();
    }
    __syncthreads();
    if (!last_of_worker) return;
    unsigned long long* my_pref = rs.pref + (uint64_t)worker * cnt_stride;
    unsigned long long carry = 0;
    for (uint32_t b0 = 0; b0 < buckets; b0 += 1024) {
        const uint32_t b = b0 + threadIdx.x;
        const unsigned long long v = (b < buckets) ? __ldcg(my_cnt + b) : 0ull;
        unsigned long long total;
        const unsigned long long ex = block_exclusive_scan64<32>(v, scan_smem, &total);
        if (b < buckets) my_pref[b] = carry + ex;
        carry += total;
    }
    if (threadIdx.x == 0) rs.totals[worker] = carry;
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

constexpr uint32_t kListCap = 4096;

// grid = (buckets, workers).  Sorts one bucket's ranks through a shared bitmap and writes them,
// ascending, to the worker's row of `ranks`: buckets are rank ranges, so the row ends up sorted
// as a whole.  Needs the sizes only, not the core.  WIDE: buckets of 2^17 ranks (s = 17), which
// very long vectors use to keep the number of buckets within what the rank and scatter steps
// count in shared memory.
template <bool WIDE>
__global__ void __launch_bounds__(kBucketThreads) bucket_sort_kernel(
    uint32_t k_exp, uint32_t s, const uint32_t* __restrict__ grouped, uint32_t* __restrict__ ranks,
    uint64_t rho_stride, const unsigned long long* __restrict__ cnt, const unsigned long long* __restrict__ pref,
    const unsigned long long* __restrict__ totals, uint64_t cnt_stride, WsHeader* hdr) {
    using ListEntry = typename std::conditional<WIDE, uint32_t, uint16_t>::type;
    __shared__ uint32_t bm[WIDE ? 4096 + 128 : 2048 + 64];   // up to 2^17 / 2^16 rank bits, padded (see sw)
    __shared__ ListEntry list[kListCap];                     // sorted ranks (low s bits) of the current round
    __shared__ uint32_t warp_sums[kBucketThreads / 32];
    const uint32_t worker = blockIdx.y, bucket = blockIdx.x, t = threadIdx.x;
    const uint32_t words = 1u << (s - 5);
    const uint32_t per = words / kBucketThreads;   // 1 .. 16 words per thread
    const uint32_t count = (uint32_t)cnt[(uint64_t)worker * cnt_stride + bucket];
    const uint32_t offset = (uint32_t)pref[(uint64_t)worker * cnt_stride + bucket];
    if (bucket == 0 && t == 0 && totals[worker] != k_exp) hdr->status = SLIMDP_ERR_INTERNAL;
    if (count == 0) return;
    if ((uint64_t)offset + count > k_exp) {
        if (t == 0) hdr->status = SLIMDP_ERR_INTERNAL;
        return;
    }
    for (uint32_t i = t; i < words + (words >> 5); i += kBucketThreads) bm[i] = 0;
    __syncthreads();
    const uint32_t* src = grouped + (uint64_t)worker * rho_stride + offset;
    const uint32_t low_mask = (1u << s) - 1u;
    for (uint32_t e = t; e < count; e += kBucketThreads) {
        const uint32_t r = src[e] & low_mask;
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
    uint32_t* dst = ranks + (uint64_t)worker * rho_stride + offset;
    const uint32_t first_rank = bucket << s;
    // rounds of up to kListCap ranks: into `list` in sorted order, then out with coalesced stores
    for (uint32_t r0 = 0; r0 < count; r0 += kListCap) {
        if (base < r0 + kListCap && base + mine > r0) {
            uint32_t p = base;
            for (uint32_t q = 0; q < per; ++q) {
                uint32_t word = bm[sw(t * per + q)];
                while (word) {
                    const uint32_t bit = __ffs(word) - 1;
                    word &= word - 1;
                    if (p >= r0 && p < r0 + kListCap) list[p - r0] = (ListEntry)((t * per + q) * 32u + bit);
                    ++p;
                }
            }
        }
        __syncthreads();
        const uint32_t m = (count - r0 < kListCap) ? count - r0 : kListCap;
        for (uint32_t e = t; e < m; e += kBucketThreads) dst[r0 + e] = first_rank + list[e];
        __syncthreads();
    }
}

constexpr uint32_t kSelThreads = 256;
constexpr uint32_t kSelPer = 8;                          // consecutive sorted ranks per thread
constexpr uint32_t kSelTile = kSelThreads * kSelPer;     // per CTA
constexpr uint32_t kDirCache = 6144;                     // directory entries a CTA keeps in shared memory

// cell_group[c] = the 64-parameter group that holds non-core rank c * 4096, c < cells;
// cell_group[cells] = the last group.  A group holds at most 64 ranks, so it contains at most
// one cell boundary, and every boundary below M lies in exactly one group: no search, no races.
__global__ void __launch_bounds__(256) cell_table_kernel(const uint32_t* __restrict__ dir, uint32_t nd,
                                                         uint32_t cells, uint32_t* __restrict__ cell_group) {
    const uint32_t stride = gridDim.x * blockDim.x;
    for (uint32_t d = blockIdx.x * blockDim.x + threadIdx.x; d < nd; d += stride) {
        const uint32_t a = __ldg(dir + d), b = __ldg(dir + d + 1);
        const uint64_t c = ((uint64_t)a + (1u << kCellShift) - 1u) >> kCellShift;   // first boundary at or after a
        if ((c << kCellShift) < b && c < cells) cell_group[c] = d;
        if (d == 0) cell_group[cells] = nd - 1;
    }
}

// grid = (tiles, workers).  idx = select0(core bitmap, rank) for one tile of a worker's sorted
// ranks: the tile's ranks lie in a contiguous run of directory groups, bounded through the cell
// table and kept in shared memory; each thread then walks its consecutive ranks forward
// through that run.  Ascending ranks give ascending indices, so the output is the sorted set.
__global__ void __launch_bounds__(kSelThreads, 5) select0_kernel(const uint32_t* __restrict__ bitmap,
                                                                 const uint32_t* __restrict__ dir, uint32_t nd,
                                                                 const uint32_t* __restrict__ cell_group,
                                                                 uint32_t cells, uint32_t k_exp,
                                                                 const uint32_t* __restrict__ ranks,
                                                                 uint64_t rho_stride, PtrArray<uint32_t> out,
                                                                 WsHeader* hdr, const uint32_t* __restrict__ window,
                                                                 uint32_t rank0) {
    __shared__ uint32_t dir_sh[kDirCache + 1];
    __shared__ uint32_t grp_bounds[2];
    const uint32_t worker = blockIdx.y, t = threadIdx.x;
    // window (a shard's piece of the sorted ranks): positions [window[0], window[1]) of the row, whose ranks
    // count from rank0; without it the whole row
    uint32_t first = 0, count = k_exp;
    if (window != nullptr) {
        first = window[0];
        count = window[1] - first;
    }
    const uint32_t tile0 = blockIdx.x * kSelTile;
    if (tile0 >= count) return;
    const uint32_t m = (count - tile0 < kSelTile) ? count - tile0 : kSelTile;
    const uint32_t* src = ranks + (uint64_t)worker * rho_stride + first + tile0;
    uint32_t* dst = out.p[worker] + tile0;
    if (t < 2) {   // the group of the first cell the tile touches, and of the cell after its last
        const uint32_t cell = ((__ldg(src + (t ? m - 1u : 0u)) - rank0) >> kCellShift) + t;
        grp_bounds[t] = __ldg(cell_group + (cell < cells ? cell : cells));
    }
    // this thread's ranks (the row is 256-byte aligned and tile0, kSelPer are multiples of 4)
    const uint32_t e0 = t * kSelPer;
    uint32_t rank[kSelPer];
    if (window == nullptr && e0 + kSelPer <= m) {
#pragma unroll
        for (uint32_t q = 0; q < kSelPer; q += 4) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + e0 + q));
            rank[q] = v.x;
            rank[q + 1] = v.y;
            rank[q + 2] = v.z;
            rank[q + 3] = v.w;
        }
    } else {
#pragma unroll
        for (uint32_t q = 0; q < kSelPer; ++q) rank[q] = (e0 + q < m) ? __ldg(src + e0 + q) - rank0 : 0u;
    }
    __syncthreads();
    const uint32_t grp_lo = grp_bounds[0], grp_hi = grp_bounds[1];
    if (grp_hi < grp_lo) {
        if (t == 0) hdr->status = SLIMDP_ERR_INTERNAL;   // the ranks are not ascending
        return;
    }
    const uint32_t ngrp = grp_hi - grp_lo + 1;
    const bool cached = ngrp <= kDirCache;
    if (cached)
        for (uint32_t i = t; i <= ngrp; i += kSelThreads) dir_sh[i] = __ldg(dir + grp_lo + i);
    __syncthreads();
    // first every rank's group and its place in the group (shared memory only), then all bitmap
    // words of the thread at once, so that their latencies overlap
    uint32_t grp[kSelPer], rem[kSelPer];
    bool plain[kSelPer];   // no core parameter in the group
    bool bad = false;
    if (cached) {
        // groups per rank inside this tile, for the interpolated first guess
        const uint32_t dir_first = dir_sh[0];
        const float groups_per_rank = (float)ngrp / (float)(dir_sh[ngrp] - dir_first + 1u);
        uint32_t rel = 0;
        if (e0 < m) {
            const uint32_t r = rank[0];
            uint32_t lo = 0, hi = ngrp - 1;
            const uint32_t guess = (uint32_t)((float)(r - dir_first) * groups_per_rank);
            const uint32_t win_lo = (guess > 8u) ? guess - 8u : 0u;
            const uint32_t win_hi = (guess + 8u < hi) ? guess + 8u : hi;
            if (win_lo <= win_hi && dir_sh[win_lo] <= r && dir_sh[win_hi + 1] > r) {
                lo = win_lo;
                hi = win_hi;
            }
            while (lo < hi) {
                const uint32_t mid = lo + ((hi - lo + 1) >> 1);
                if (dir_sh[mid] <= r)
                    lo = mid;
                else
                    hi = mid - 1;
            }
            rel = lo;
        }
#pragma unroll
        for (uint32_t q = 0; q < kSelPer; ++q) {
            const uint32_t r = rank[q];
            if (e0 + q < m)
                while (rel + 1 < ngrp && dir_sh[rel + 1] <= r) ++rel;   // ranks ascend: the group only moves up
            const uint32_t d0 = dir_sh[rel], d1 = dir_sh[rel + 1];
            grp[q] = grp_lo + rel;
            rem[q] = r - d0;
            plain[q] = d1 - d0 == kDirStride;
            bad |= e0 + q < m && !(r >= d0 && r < d1);
        }
    } else {
        // a tile that spans more groups than the cache holds (few ranks over many parameters)
        uint32_t g = grp_lo;
#pragma unroll
        for (uint32_t q = 0; q < kSelPer; ++q) {
            const uint32_t r = rank[q];
            if (e0 + q < m) g = find_block(dir, g, grp_hi, r);
            const uint32_t d0 = __ldg(dir + g), d1 = __ldg(dir + g + 1);
            grp[q] = g;
            rem[q] = r - d0;
            plain[q] = d1 - d0 == kDirStride;
            bad |= e0 + q < m && !(r >= d0 && r < d1);
        }
    }
    uint2 words[kSelPer];
#pragma unroll
    for (uint32_t q = 0; q < kSelPer; ++q)
        words[q] = (e0 + q < m && !plain[q] && !bad)
                       ? __ldg(reinterpret_cast<const uint2*>(bitmap + (uint64_t)grp[q] * kWordsPerDir))
                       : make_uint2(0u, 0u);
    uint32_t idx[kSelPer];
#pragma unroll
    for (uint32_t q = 0; q < kSelPer; ++q) {
        if (plain[q]) {
            idx[q] = grp[q] * kDirStride + rem[q];
        } else {
            const uint32_t z0 = ~words[q].x, z1 = ~words[q].y;
            const uint32_t c0 = __popc(z0);
            const bool second = rem[q] >= c0;
            const uint32_t z = second ? z1 : z0;
            const uint32_t r = second ? rem[q] - c0 : rem[q];
            idx[q] = grp[q] * kDirStride + (second ? 32u : 0u) + nth_set_bit(z, r);
            bad |= e0 + q < m && r >= (uint32_t)__popc(z);
        }
    }
    if (bad) {
        hdr->status = SLIMDP_ERR_INTERNAL;   // directory and bitmap disagree, or the ranks are not sorted
        return;
    }
    if (e0 + kSelPer <= m && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {   // 16-byte stores where the list allows
#pragma unroll
        for (uint32_t q = 0; q < kSelPer; q += 4)
            *reinterpret_cast<uint4*>(dst + e0 + q) = make_uint4(idx[q], idx[q + 1], idx[q + 2], idx[q + 3]);
    } else {
#pragma unroll
        for (uint32_t q = 0; q < kSelPer; ++q)
            if (e0 + q < m) dst[e0 + q] = idx[q];
    }
}

}  // namespace

uint32_t explore_bucket_shift(uint64_t M) {
    int lg = 0;
    while (lg < 63 && (2ull << lg) <= M) ++lg;   // floor(log2(M)) for M >= 1
    int extra = lg - 22;
    if (extra < 0) extra = 0;
    if (extra > 3) extra = 3;
    if (lg >= 28) extra = 4;   // from 2^28 non-core parameters: 2^17 ranks per bucket, at most 8192 buckets up to 2^30
    return (uint32_t)(13 + extra);
}

// parts: 1 = the steps that need only the sizes (round keys, ranks, their sort),
//        2 = the step that needs the core (parameter indices from sorted ranks), 3 = everything.
// lean: part 1 runs beside a kernel that holds most of every SM's shared memory, so its
// kernels keep to small shared-memory footprints (the scatter step does not group its chunk).
slimdp_status launch_explore_parts(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                                   uint32_t first_worker, uint32_t workers, uint32_t round,
                                   const PtrArray<uint32_t>& out, void* ws, int parts, bool lean, cudaStream_t st) {
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

    if (k_exp == 0) {   // nothing to draw; the status word is still this call's
        if ((parts & 1) && cudaMemsetAsync(L.hdr, 0, sizeof(int32_t), st) != cudaSuccess) return SLIMDP_ERR_CUDA;
        return SLIMDP_OK;
    }
    if (parts & 1) {
    if (cudaMemsetAsync(L.cnt, 0, L.zero_bytes, st) != cudaSuccess) return SLIMDP_ERR_CUDA;

    uint32_t bits = 2;   // the permutation's domain is [0, 2^bits), the smallest that holds M (at least 4)
    while (((uint64_t)1 << bits) < M) ++bits;

    // about two 1024-thread CTAs per SM over all workers; every CTA owns one contiguous chunk of j
    uint64_t chunks = ((uint64_t)sms * 2 + workers - 1) / workers;
    if (chunks * workers > kMaxExploreCtas) chunks = kMaxExploreCtas / workers;
    if (chunks > (k_exp + 1023) / 1024) chunks = (k_exp + 1023) / 1024;
    if (chunks == 0) chunks = 1;
    if (lean && buckets <= kMaxSmemBuckets && 3 * buckets * 4 + 4096 < kGroupSmemLean) {
        // more, smaller chunks, so that the scatter step can still group a chunk in the shared memory it gets
        const uint64_t fit = (kGroupSmemLean - 3 * buckets * 4) / 4;
        uint64_t need = (k_exp + fit - 1) / fit;
        if (need * workers > kMaxExploreCtas) need = kMaxExploreCtas / workers;
        if (need > chunks) chunks = need;
    }
    const uint32_t chunk = (uint32_t)((k_exp + chunks - 1) / chunks);
    const dim3 grid((unsigned)chunks, workers);
    const bool smem = buckets <= kMaxSmemBuckets;
    // part 1 may run beside another kernel's CTAs on the same SMs: one shared-memory split for all
    static DeviceOnce attributes;
    if (attributes.needed()) {
        if (!prefer_max_shared(rank_kernel<true>) || !prefer_max_shared(rank_kernel<false>) ||
            !prefer_max_shared(scatter_kernel<true, true>) || !prefer_max_shared(scatter_kernel<true, false>) ||
            !prefer_max_shared(scatter_kernel<false, false>) || !prefer_max_shared(bucket_sort_kernel<false>) ||
            !prefer_max_shared(bucket_sort_kernel<true>) ||
            cudaFuncSetAttribute(scatter_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kGroupSmemMax) != cudaSuccess)
            return SLIMDP_ERR_CUDA;
        attributes.mark();
    }
    const RankStream rs{(uint32_t)seed, (uint32_t)(seed >> 32), first_worker, round, L.hdr, L.ticket, L.pref, L.totals};
    if (smem) {
        rank_kernel<true><<<grid, 1024, buckets * 4, st>>>((uint32_t)M, (uint32_t)k_exp, chunk, bits, s,
                                                           (uint32_t)buckets, rs, L.rho, L.rho_stride, L.cnt,
                                                           L.cnt_stride, L.cta_hist);
    } else {
        rank_kernel<false><<<grid, 1024, 0, st>>>((uint32_t)M, (uint32_t)k_exp, chunk, bits, s, (uint32_t)buckets, rs,
                                                  L.rho, L.rho_stride, L.cnt, L.cnt_stride, L.cta_hist);
    }
    SLIMDP_LAUNCHED(1);
    const size_t group_smem = (3 * buckets + chunk) * 4;
    if (smem && group_smem <= (lean ? kGroupSmemLean : kGroupSmemMax)) {
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
    if (s > 16)
        bucket_sort_kernel<true><<<dim3((unsigned)buckets, workers), kBucketThreads, 0, st>>>(
            (uint32_t)k_exp, s, L.sorted, L.rho, L.rho_stride, L.cnt, L.pref, L.totals, L.cnt_stride, L.hdr);
    else
        bucket_sort_kernel<false><<<dim3((unsigned)buckets, workers), kBucketThreads, 0, st>>>(
            (uint32_t)k_exp, s, L.sorted, L.rho, L.rho_stride, L.cnt, L.pref, L.totals, L.cnt_stride, L.hdr);
    SLIMDP_LAUNCHED(1);
    }   // parts & 1
    if (!(parts & 2)) return SLIMDP_OK;
    const uint32_t cells = (uint32_t)((M + (1u << kCellShift) - 1) >> kCellShift);
    uint64_t tgrid = (nd + 255) / 256;
    if (tgrid > (uint64_t)sms * 8) tgrid = (uint64_t)sms * 8;
    cell_table_kernel<<<(unsigned)tgrid, 256, 0, st>>>(dir, (uint32_t)nd, cells, L.cell_group);
    select0_kernel<<<dim3((unsigned)((k_exp + kSelTile - 1) / kSelTile), workers), kSelThreads, 0, st>>>(
        bitmap, dir, (uint32_t)nd, L.cell_group, cells, (uint32_t)k_exp, L.rho, L.rho_stride, out, L.hdr, nullptr, 0u);
    SLIMDP_LAUNCHED(2);
    return SLIMDP_OK;
}

namespace {

// window[0], window[1]: where the ranks in [rank_lo, rank_hi) sit in the sorted row; *count = how many they
// are, or 0 with the status word set if they do not fit `cap`.
__global__ void rank_window_kernel(const uint32_t* __restrict__ ranks, uint32_t k_exp, uint32_t rank_lo,
                                   unsigned long long rank_hi, unsigned long long cap, uint32_t* window,
                                   uint32_t* count, WsHeader* hdr) {
    uint32_t lo = 0, hi = k_exp;
    while (lo < hi) {   // first position with rank >= rank_lo
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if (ranks[mid] < rank_lo)
            lo = mid + 1;
        else
            hi = mid;
    }
    const uint32_t a = lo;
    hi = k_exp;
    while (lo < hi) {   // first position with rank >= rank_hi
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if ((unsigned long long)ranks[mid] < rank_hi)
            lo = mid + 1;
        else
            hi = mid;
    }
    uint32_t b = lo;
    if ((unsigned long long)(b - a) > cap) {
        hdr->status = SLIMDP_ERR_INTERNAL;   // the caller's list is too short for this shard's share
        b = a;
    }
    window[0] = a;
    window[1] = b;
    *count = b - a;
}

}  // namespace

// One shard's share of a worker's explorer (see slimdp_sample_explore_shard).  The ranks are drawn and
// sorted over ALL shards' non-core parameters (every shard computes the same row); the shard keeps the
// ranks of its own non-core parameters, [noncore_below, noncore_below + n_shard - k_core_shard), and turns
// them into shard-local indices with its own bitmap and directory.
slimdp_status launch_explore_shard(const void* core_aux, uint64_t n_shard, uint64_t k_core_shard,
                                   uint64_t noncore_total, uint64_t noncore_below, uint64_t k_exp, uint64_t seed,
                                   uint32_t worker, uint32_t round, uint32_t* exp_idx, uint64_t cap, uint32_t* count,
                                   void* ws, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const uint64_t n_layout = noncore_total > n_shard ? noncore_total : n_shard;
    const ExploreWs L = explore_ws_layout(ws, n_layout, k_exp, 1);
    uint32_t* window = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(ws) + L.bytes);   // 2 words after the layout
    PtrArray<uint32_t> out;
    for (auto& q : out.p) q = nullptr;
    out.p[0] = exp_idx;
    if (k_exp == 0) {
        if (cudaMemsetAsync(L.hdr, 0, sizeof(int32_t), st) != cudaSuccess ||
            cudaMemsetAsync(count, 0, sizeof(uint32_t), st) != cudaSuccess)
            return SLIMDP_ERR_CUDA;
        return SLIMDP_OK;
    }
    // the sorted ranks of the whole model's explorer: a vector of n_layout parameters with noncore_total of them outside the core
    slimdp_status rc = launch_explore_parts(core_aux, n_layout, n_layout - noncore_total, k_exp, seed, worker, 1, round,
                                            out, ws, 1, false, st);
    if (rc != SLIMDP_OK) return rc;
    const uint64_t m_shard = n_shard - k_core_shard;
    rank_window_kernel<<<1, 1, 0, st>>>(L.rho, (uint32_t)k_exp, (uint32_t)noncore_below, noncore_below + m_shard, cap,
                                        window, count, L.hdr);
    const uint64_t nd = num_blocks(n_shard) * kDirPerBlock;
    const uint32_t* bitmap = reinterpret_cast<const uint32_t*>(core_aux);
    const uint32_t* dir =
        reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(core_aux) + slimdp_core_aux_dir_offset(n_shard));
    const uint32_t cells = (uint32_t)((m_shard + (1u << kCellShift) - 1) >> kCellShift);
    uint64_t tgrid = (nd + 255) / 256;
    if (tgrid > (uint64_t)sms * 8) tgrid = (uint64_t)sms * 8;
    cell_table_kernel<<<(unsigned)tgrid, 256, 0, st>>>(dir, (uint32_t)nd, cells, L.cell_group);
    // the grid covers the most ranks the shard can get; CTAs beyond its share return at once
    const uint64_t most = (k_exp < m_shard ? k_exp : m_shard);
    select0_kernel<<<dim3((unsigned)((most + kSelTile - 1) / kSelTile + 1), 1), kSelThreads, 0, st>>>(
        bitmap, dir, (uint32_t)nd, L.cell_group, cells, (uint32_t)k_exp, L.rho, L.rho_stride, out, L.hdr, window,
        (uint32_t)noncore_below);
    SLIMDP_LAUNCHED(3);
    return SLIMDP_OK;
}

size_t explore_shard_ws_bytes(uint64_t n_shard, uint64_t noncore_total, uint64_t k_exp) {
    const uint64_t n_layout = noncore_total > n_shard ? noncore_total : n_shard;
    return explore_ws_layout(nullptr, n_layout, k_exp, 1).bytes + 256;
}

slimdp_status launch_explore(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                             uint32_t first_worker, uint32_t workers, uint32_t round,
                             const PtrArray<uint32_t>& out, void* ws, cudaStream_t st) {
    return launch_explore_parts(core_aux, n, k_core, k_exp, seed, first_worker, workers, round, out, ws, 3, false,
                                st);
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
    // per device; every thread that gets here first stores the same value.  The address holds for the
    // life of the device's primary context.
    static std::atomic<void*> scratch_addr[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLIMDP_ERR_CUDA;
    void* scratch = scratch_addr[dev].load(std::memory_order_relaxed);
    if (scratch == nullptr) {
        if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || scratch == nullptr)
            return SLIMDP_ERR_CUDA;
        scratch_addr[dev].store(scratch, std::memory_order_relaxed);
    }
    if (explore_ws_layout(nullptr, n, k_exp, 1).bytes > kStaticScratchBytes) return SLIMDP_ERR_UNSUPPORTED;
    PtrArray<uint32_t> out;
    for (auto& q : out.p) q = nullptr;
    out.p[0] = exp_idx;
    void* ws = scratch;
    // launch_explore clears the counters it needs at zero and resets the status word on every call
    slimdp_status rc = launch_explore(core_aux, n, k_core, k_exp, seed, worker, 1, round, out, ws, st);
    if (rc != SLIMDP_OK) return rc;
    if (status_out != nullptr &&
        cudaMemcpyAsync(status_out, ws, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return SLIMDP_ERR_CUDA;
    return SLIMDP_OK;
}

}  // namespace slimdp
