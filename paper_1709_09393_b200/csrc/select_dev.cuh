// Device helpers shared by the kernels of the selection (whole vector, per segment, per shard).
#pragma once

#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

namespace {

constexpr int kFinishThreads = 512;   // two CTAs per SM: one's waits are the other's work
constexpr uint32_t kBarrierSpins = 1u << 24;   // x 64 ns of back-off: about a second


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

// Walks a histogram from its top bin down and finds the bin in which the running count reaches
// `want` (>= 1).  Every thread of the CTA calls it; all get the same answer.  scan_smem: 33 words
// of 64 bits, res: 3 words.  False (nothing written) if the histogram holds fewer than `want`.
template <int THREADS>
__device__ __forceinline__ bool find_rank_bin(const uint32_t* hist, uint32_t nbins, uint32_t want,
                                              unsigned long long* scan_smem, uint32_t* res, uint32_t* bin,
                                              uint32_t* rem) {
    const uint32_t per = (nbins + THREADS - 1) / THREADS;
    const uint32_t first = threadIdx.x * per;   // this thread's bins, counted from the top: first .. first + per - 1
    unsigned long long sum = 0;
    for (uint32_t q = 0; q < per; ++q)
        if (first + q < nbins) sum += __ldcg(hist + (nbins - 1 - (first + q)));
    unsigned long long total;
    unsigned long long above = block_exclusive_scan64<THREADS / 32>(sum, scan_smem, &total);
    if (threadIdx.x == 0) res[0] = 0;
    __syncthreads();
    if (total >= want) {
        for (uint32_t q = 0; q < per; ++q) {
            if (first + q >= nbins) break;
            const uint32_t b = nbins - 1 - (first + q);
            const unsigned long long h = __ldcg(hist + b);
            if (above < want && (unsigned long long)want <= above + h) {
                res[0] = 1;
                res[1] = b;
                res[2] = want - (uint32_t)above;
            }
            above += h;
        }
    }
    __syncthreads();
    const bool found = res[0] != 0;
    *bin = res[1];
    *rem = res[2];
    __syncthreads();
    return found;
}

// Grid barrier of the cooperative launch (all CTAs are resident).  Arrivals are counted in one
// word that only grows: after the e-th barrier it holds e * gridDim.x.  The wait is bounded; if it
// runs out, or another CTA gave up, the abort flag is raised and false is returned to all threads.
__device__ __forceinline__ bool grid_barrier(WsHeader* hdr, uint32_t* epoch) {
    __shared__ uint32_t ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t target = ++(*epoch) * gridDim.x;
        __threadfence();
        atomicAdd(&hdr->barrier, 1u);
        uint32_t good = 1, spins = 0;
        volatile uint32_t* bar = &hdr->barrier;
        volatile uint32_t* ab = &hdr->abort;
        while (*bar < target) {
            if (*ab != 0u || ++spins > kBarrierSpins) {
                *ab = 1u;
                hdr->status = SLIMDP_ERR_INTERNAL;
                good = 0;
                break;
            }
            __nanosleep(64);
        }
        __threadfence();
        ok = good;
    } else {
        ++(*epoch);
    }
    __syncthreads();
    return ok != 0;
}

// Sum of a 64-bit value over the CTA, returned to every thread.  red: one word per warp.
template <int THREADS>
__device__ __forceinline__ unsigned long long cta_sum64(unsigned long long v, unsigned long long* red) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    if ((threadIdx.x & 31u) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long s = 0;
    for (int x = 0; x < THREADS / 32; ++x) s += red[x];
    __syncthreads();
    return s;
}

// ---- last step of a selection: bitmaps to core bitmap, directory and ascending index list ----
//
// G holds the parameters above the threshold, E (may be null: none) those equal to it, of which the
// first hdr->tie_quota in index order belong to the core; cnt holds their counts per 1024-parameter
// block (#greater | #equal << 32).  The finishing kernels end with super_sum_phase (every CTA: the
// counts of each group of kSuperTile blocks) and, after a grid barrier, tile_scan_phase (one CTA:
// the counts below every group).  From then on any warp finds, without waiting for any other, what
// lies below a block (the group's prefix plus at most 63 block counts) and hence every member's
// place in the core: block_selection.  emit_kernel uses it to write the core's bitmap, directory
// and index list; the one-call round's exchange uses it directly and needs no emit.
constexpr uint32_t kSuperTile = 64;    // blocks per group
constexpr int kEmitWarps = 8;

inline uint64_t num_super_tiles(uint64_t nb) { return (nb + kSuperTile - 1) / kSuperTile; }

// Every CTA of the grid: super[s] = sum of cnt over group s (a warp per group).
template <int THREADS>
__device__ __forceinline__ void super_sum_phase(const unsigned long long* cnt, unsigned long long* super,
                                                uint64_t nb) {
    const uint64_t nsuper = (nb + kSuperTile - 1) / kSuperTile;
    const uint32_t lane = lane_id();
    const uint64_t warps = (uint64_t)gridDim.x * (THREADS / 32);
    for (uint64_t s = (uint64_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5); s < nsuper; s += warps) {
        const uint64_t b0 = s * kSuperTile + lane, b1 = b0 + 32;
        unsigned long long v = (b0 < nb ? __ldcg(cnt + b0) : 0ull) + (b1 < nb ? __ldcg(cnt + b1) : 0ull);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
        if (lane == 0) super[s] = v;
    }
}

// One CTA of THREADS threads, after a grid barrier: super[s] <- counts in the groups below s (in
// place); checks the totals against k ((#greater) + min(#equal, r) must be k) and writes the
// directory's last entry.
template <int THREADS>
__device__ __forceinline__ void tile_scan_phase(unsigned long long* super, uint64_t n, uint64_t nb, uint32_t k,
                                                uint32_t ties, WsHeader* hdr, uint32_t* dir,
                                                unsigned long long* scan_smem) {
    const uint64_t nsuper = (nb + kSuperTile - 1) / kSuperTile;
    // every warp owns a stretch of consecutive groups: its sum (independent loads), one scan over the
    // warps' sums, then the stretch again 32 groups at a time, the next 32 asked for ahead
    constexpr uint32_t W = THREADS / 32;
    const uint32_t lane = lane_id(), wid = threadIdx.x >> 5;
    const uint64_t per = ((nsuper + W - 1) / W + 31) / 32 * 32;   // groups per warp, a multiple of 32
    const uint64_t s_lo = min(nsuper, (uint64_t)wid * per), s_hi = min(nsuper, s_lo + per);
    unsigned long long sum = 0;
#pragma unroll 4
    for (uint64_t s = s_lo + lane; s < s_hi; s += 32) sum += __ldcg(super + s);
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
    unsigned long long carry;
    unsigned long long run = block_exclusive_scan64<W>(lane == 0 ? sum : 0ull, scan_smem, &carry);
    run = __shfl_sync(0xFFFFFFFFu, run, 0);   // counts below the warp's stretch
    unsigned long long v = (s_lo + lane < s_hi) ? __ldcg(super + s_lo + lane) : 0ull;
    for (uint64_t s0 = s_lo; s0 < s_hi; s0 += 32) {
        const uint64_t s = s0 + lane;
        const unsigned long long nxt = (s + 32 < s_hi) ? __ldcg(super + s + 32) : 0ull;
        const unsigned long long inc = warp_inclusive_scan64(v);
        if (s < s_hi) super[s] = run + inc - v;
        run += __shfl_sync(0xFFFFFFFFu, inc, 31);
        v = nxt;
    }
    if (threadIdx.x == 0) {
        const uint32_t ng = (uint32_t)carry, ne = (uint32_t)(carry >> 32);
        if (ng + min(ne, ties) != k) hdr->status = SLIMDP_ERR_INTERNAL;
        dir[nb * kDirPerBlock] = (uint32_t)(n - k);
    }
}

// What a warp reads for one 1024-parameter block (lane = bitmap word; blk < nb): the lane's words of
// the two bitmaps and its share of the counts below the block (the group's prefix plus the blocks
// of the group below this one).  Asking and placing are separate so that a warp that walks several
// blocks can ask for the next one before it works on the current one.
struct BlockLoads {
    uint32_t Gw, Ew;
    uint32_t below_g, below_e;   // this lane's share of the group's blocks below the block
    unsigned long long pref;     // counts below the group (every lane holds it)
};

__device__ __forceinline__ BlockLoads block_request(const uint32_t* __restrict__ G, const uint32_t* __restrict__ E,
                                                    const unsigned long long* __restrict__ cnt,
                                                    const unsigned long long* __restrict__ super_pref, uint64_t blk) {
    const uint32_t lane = lane_id();
    BlockLoads L;
    L.Gw = __ldg(G + blk * kWordsPerBlock + lane);
    L.Ew = (E != nullptr) ? __ldg(E + blk * kWordsPerBlock + lane) : 0u;
    const uint64_t super = blk / kSuperTile, first = super * kSuperTile;
    const unsigned long long c0 = (first + lane < blk) ? __ldg(cnt + first + lane) : 0ull;
    const unsigned long long c1 = (first + 32 + lane < blk) ? __ldg(cnt + first + 32 + lane) : 0ull;
    L.pref = __ldg(super_pref + super);
    L.below_g = (uint32_t)c0 + (uint32_t)c1;   // a block counts at most 1024 of either kind
    L.below_e = (uint32_t)(c0 >> 32) + (uint32_t)(c1 >> 32);
    return L;
}

// The block's part of the core (*sel) and the number of core parameters below this lane's word
// (*pos0).  Returns the number of core parameters in the block.
__device__ __forceinline__ uint32_t block_place(const BlockLoads& L, uint32_t ties, uint32_t* sel, uint32_t* pos0) {
    const uint32_t lane = lane_id();
    const uint32_t Gw = L.Gw, Ew = L.Ew;
    const uint32_t pg = __popc(Gw), pe = __popc(Ew);
    // counts in the words below this lane's, both kinds in one word (at most 1024 each)
    uint32_t incl = pg | (pe << 16);
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= (uint32_t)d) incl += up;
    }
    // counts below this lane's word in the whole vector (the core is at most 2^32 - 1 long)
    const uint32_t g_before =
        (uint32_t)L.pref + __reduce_add_sync(0xFFFFFFFFu, L.below_g) + (incl & 0xFFFFu) - pg;
    const uint32_t e_before =
        (uint32_t)(L.pref >> 32) + __reduce_add_sync(0xFFFFFFFFu, L.below_e) + (incl >> 16) - pe;
    // equal keys: admit those whose rank among all equal keys (index order) is below r
    const uint32_t admit = (ties > e_before) ? min(ties - e_before, pe) : 0u;
    uint32_t Ea;
    if (admit == pe)
        Ea = Ew;
    else if (admit == 0)
        Ea = 0;
    else
        Ea = Ew & ((1u << nth_set_bit(Ew, admit)) - 1u);
    *sel = Gw | Ea;
    *pos0 = g_before + min(e_before, ties);
    return __reduce_add_sync(0xFFFFFFFFu, __popc(*sel));
}

__device__ __forceinline__ uint32_t block_selection(const uint32_t* __restrict__ G, const uint32_t* __restrict__ E,
                                                    const unsigned long long* __restrict__ cnt,
                                                    const unsigned long long* __restrict__ super_pref, uint32_t ties,
                                                    uint64_t blk, uint32_t* sel, uint32_t* pos0) {
    const BlockLoads L = block_request(G, E, cnt, super_pref, blk);
    return block_place(L, ties, sel, pos0);
}

// The block's words of the core bitmap and its 16 directory entries.
__device__ __forceinline__ void write_block_aux(uint32_t* __restrict__ bitmap, uint32_t* __restrict__ dir, uint64_t blk,
                                                uint32_t sel, uint32_t pos0) {
    const uint32_t lane = lane_id();
    bitmap[blk * kWordsPerBlock + lane] = sel;
    if ((lane & (kWordsPerDir - 1)) == 0)   // one directory entry per 64 parameters (2 words)
        dir[blk * kDirPerBlock + lane / kWordsPerDir] = (uint32_t)(blk * kBlock) + lane * 32u - pos0;
}

// emit_kernel: half a warp per block, so that one instruction serves two blocks (the kernel is
// bound by the instructions it issues, not by memory).  Lane h of a half holds the block's words 2h
// and 2h + 1, which is one directory group.  Warps walk pairs of blocks in turn, wait for nobody and
// ask for the next pair before they work on the current one.  A block with few members has every
// lane write out its own words' members; otherwise the lanes list their members' offsets in the
// half's piece of shared memory, in index order, and the half writes the list out 16 consecutive
// places at a time.
constexpr uint32_t kEmitDirectMax = 64;   // members per block up to which the lanes write directly

struct HalfLoads {
    uint2 G2, E2;
    uint32_t below;            // this lane's share of the group's blocks below the block: #greater | #equal << 16
    unsigned long long pref;   // counts below the group
};

__device__ __forceinline__ HalfLoads half_request(const uint32_t* __restrict__ G, const uint32_t* __restrict__ E,
                                                  const unsigned long long* __restrict__ cnt,
                                                  const unsigned long long* __restrict__ super_pref, uint64_t blk,
                                                  uint64_t nb, uint32_t hl) {
    HalfLoads L;
    L.G2 = make_uint2(0u, 0u);
    L.E2 = make_uint2(0u, 0u);
    L.below = 0;
    L.pref = 0;
    if (blk >= nb) return L;
    L.G2 = __ldg(reinterpret_cast<const uint2*>(G) + blk * (kWordsPerBlock / 2) + hl);
    if (E != nullptr) L.E2 = __ldg(reinterpret_cast<const uint2*>(E) + blk * (kWordsPerBlock / 2) + hl);
    const uint64_t super = blk / kSuperTile, first = super * kSuperTile;
    unsigned long long c = 0;   // at most 4 blocks of at most 1024 of either kind: no carry between the halves
#pragma unroll
    for (uint32_t q = 0; q < kSuperTile / 16; ++q)
        if (first + 16 * q + hl < blk) c += __ldg(cnt + first + 16 * q + hl);
    L.below = (uint32_t)c | ((uint32_t)(c >> 32) << 16);
    L.pref = __ldg(super_pref + super);
    return L;
}

__global__ void __launch_bounds__(kEmitWarps * 32) emit_kernel(const uint32_t* __restrict__ G,
                                                               const uint32_t* __restrict__ E,
                                                               const unsigned long long* __restrict__ cnt,
                                                               const unsigned long long* __restrict__ super_pref,
                                                               uint64_t nb, uint32_t k, WsHeader* hdr,
                                                               uint32_t* __restrict__ core_idx,
                                                               uint32_t* __restrict__ bitmap,
                                                               uint32_t* __restrict__ dir) {
    static_assert((kSuperTile - 1) * kBlock < 65536u, "the counts of a group's blocks below a block fit 16 bits each");
    __shared__ uint16_t list[kEmitWarps][2][kBlock];
    if (hdr->abort != 0u) return;   // the finishing kernel gave up (the status word says so)
    const uint32_t ties = (E != nullptr) ? hdr->tie_quota : 0u;
    const uint32_t lane = lane_id(), wid = threadIdx.x >> 5;
    const uint32_t half = lane >> 4, hl = lane & 15u;
    const uint64_t pairs = (nb + 1) / 2;
    const uint64_t warps = (uint64_t)gridDim.x * kEmitWarps;
    bool bad = false;
    uint64_t pair = (uint64_t)blockIdx.x * kEmitWarps + wid;
    if (pair >= pairs) return;
    HalfLoads cur = half_request(G, E, cnt, super_pref, 2 * pair + half, nb, hl);
    for (; pair < pairs; pair += warps) {
        const uint64_t blk = 2 * pair + half;
        const bool live = blk < nb;
        HalfLoads nxt = cur;
        if (pair + warps < pairs) nxt = half_request(G, E, cnt, super_pref, 2 * (pair + warps) + half, nb, hl);
        const uint2 G2 = cur.G2, E2 = cur.E2;
        const uint32_t pg = __popc(G2.x) + __popc(G2.y), pe = __popc(E2.x) + __popc(E2.y);
        // counts in the half's lanes below this one, and in the group's blocks below the block
        uint32_t incl = pg | (pe << 16), below = cur.below;
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d, 16);
            if (hl >= (uint32_t)d) incl += up;
        }
#pragma unroll
        for (int d = 8; d >= 1; d >>= 1) below += __shfl_xor_sync(0xFFFFFFFFu, below, d, 16);
        const uint32_t g_before = (uint32_t)cur.pref + (below & 0xFFFFu) + (incl & 0xFFFFu) - pg;
        const uint32_t e_before = (uint32_t)(cur.pref >> 32) + (below >> 16) + (incl >> 16) - pe;
        cur = nxt;
        // equal keys: admit those whose rank among all equal keys (index order) is below r
        const uint32_t admit = (ties > e_before) ? min(ties - e_before, pe) : 0u;
        uint2 sel = G2;
        if (admit == pe) {
            sel.x |= E2.x;
            sel.y |= E2.y;
        } else if (admit != 0) {
            const uint32_t c0 = __popc(E2.x);
            if (admit < c0) {
                sel.x |= E2.x & ((1u << nth_set_bit(E2.x, admit)) - 1u);
            } else {
                sel.x |= E2.x;
                if (admit > c0) sel.y |= E2.y & ((1u << nth_set_bit(E2.y, admit - c0)) - 1u);
            }
        }
        const uint32_t pos0 = g_before + min(e_before, ties);   // core parameters below this lane's words
        uint32_t in_block = __popc(sel.x) + __popc(sel.y);
#pragma unroll
        for (int d = 8; d >= 1; d >>= 1) in_block += __shfl_xor_sync(0xFFFFFFFFu, in_block, d, 16);
        const uint32_t base = __shfl_sync(0xFFFFFFFFu, pos0, 0, 16);   // core parameters below the block
        const uint32_t first = (uint32_t)(blk * kBlock);
        if (live) {
            reinterpret_cast<uint2*>(bitmap)[blk * (kWordsPerBlock / 2) + hl] = sel;
            dir[blk * kDirPerBlock + hl] = first + hl * 64u - pos0;
        }
        const bool staged = live && in_block > kEmitDirectMax;
        if (live && !staged) {
            uint32_t pos = pos0;
            for (uint32_t word = sel.x; word; word &= word - 1, ++pos) {
                if (pos < k)
                    core_idx[pos] = first + hl * 64u + (uint32_t)__ffs(word) - 1u;
                else
                    bad = true;
            }
            for (uint32_t word = sel.y; word; word &= word - 1, ++pos) {
                if (pos < k)
                    core_idx[pos] = first + hl * 64u + 32u + (uint32_t)__ffs(word) - 1u;
                else
                    bad = true;
            }
        }
        if (__any_sync(0xFFFFFFFFu, staged)) {
            uint16_t* mine = list[wid][half];
            if (staged) {
                uint32_t at = pos0 - base;
                for (uint32_t word = sel.x; word; word &= word - 1, ++at)
                    if (at < kBlock) mine[at] = (uint16_t)(hl * 64u + (uint32_t)__ffs(word) - 1u);
                for (uint32_t word = sel.y; word; word &= word - 1, ++at)
                    if (at < kBlock) mine[at] = (uint16_t)(hl * 64u + 32u + (uint32_t)__ffs(word) - 1u);
            }
            __syncwarp();
            if (staged) {
                for (uint32_t e = hl; e < in_block; e += 16) {
                    if (base + e < k)
                        core_idx[base + e] = first + mine[e];
                    else
                        bad = true;
                }
            }
            __syncwarp();   // the lists are free again
        }
    }
    if (bad) hdr->status = SLIMDP_ERR_INTERNAL;
}

inline slimdp_status launch_emit(const uint32_t* G, const uint32_t* E, const unsigned long long* cnt,
                                 const unsigned long long* super_pref, uint64_t n, uint32_t k, WsHeader* hdr,
                                 uint32_t* core_idx, uint32_t* bitmap, uint32_t* dir, cudaStream_t st) {
    const uint64_t nb = num_blocks(n);
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    // one wave: as many CTAs as are resident at once (a second, thinner wave would cost as much again)
    static std::atomic<int> per_sm_cached[64];   // per device; 0 = not asked yet
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SLIMDP_ERR_CUDA;
    int per_sm = (dev >= 0 && dev < 64) ? per_sm_cached[dev].load(std::memory_order_relaxed) : 0;
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, emit_kernel, kEmitWarps * 32, 0) != cudaSuccess ||
            per_sm < 1)
            return SLIMDP_ERR_CUDA;
        if (dev >= 0 && dev < 64) per_sm_cached[dev].store(per_sm, std::memory_order_relaxed);
    }
    uint64_t grid = ((nb + 1) / 2 + kEmitWarps - 1) / kEmitWarps;   // a warp per pair of blocks
    if (grid > (uint64_t)sms * per_sm) grid = (uint64_t)sms * per_sm;
    emit_kernel<<<(unsigned)grid, kEmitWarps * 32, 0, st>>>(G, E, cnt, super_pref, nb, k, hdr, core_idx, bitmap, dir);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace

}  // namespace slimdp
