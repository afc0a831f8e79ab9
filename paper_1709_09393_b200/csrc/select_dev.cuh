// Device helpers shared by the kernels of the selection (whole vector, per segment, per shard).
#pragma once

#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

namespace {

constexpr int kFinishThreads = 512;   // two CTAs per SM: one's waits are the other's work
static_assert(kFinishThreads / 8 == kEmitTile, "a tile is four bitmap words per thread of the finishing kernel");
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

// Last step of a selection, a kernel of its own (one CTA of kFinishThreads threads per kEmitGroup
// tiles): G holds the parameters above the threshold, E (may be null: none) those equal to it, of
// which the first hdr->tie_quota in index order belong to the core; tile_sum their counts per tile
// of kEmitTile blocks.  Writes the core's bitmap, its non-core rank directory and its ascending
// index list, and checks the totals against k.
constexpr uint32_t kEmitGroup = 4;
constexpr uint32_t kEmitOwnLists = 2048;   // members in a warp's 128 words up to which every thread writes its own

__global__ void __launch_bounds__(kFinishThreads, 3) emit_kernel(const uint32_t* __restrict__ G,
                                                                 const uint32_t* __restrict__ E,
                                                                 const unsigned long long* __restrict__ tile_sum,
                                                                 uint64_t n, uint64_t nb, uint32_t k, WsHeader* hdr,
                                                                 uint32_t* __restrict__ core_idx,
                                                                 uint32_t* __restrict__ bitmap,
                                                                 uint32_t* __restrict__ dir) {
    __shared__ unsigned long long scan_smem[33];
    __shared__ unsigned long long red[kFinishThreads / 32];
    if (hdr->abort != 0u) return;   // the finishing kernel gave up (status says so)
    const uint32_t ties = (E != nullptr) ? hdr->tie_quota : 0u;
    const uint32_t t = threadIdx.x, lane = lane_id();
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint64_t ntiles = (nb + kEmitTile - 1) / kEmitTile;
    // this CTA's tiles: blockIdx.x, blockIdx.x + gridDim.x, ... (the core clusters in some layers:
    // neighbouring tiles go to different CTAs, so that the heavy ones are worked on all over the GPU)
    const uint64_t tile_first = blockIdx.x, tile_step = gridDim.x, tile_last = ntiles;
    if (blockIdx.x == 0) {
        unsigned long long all = 0;
        for (uint64_t x = t; x < ntiles; x += kFinishThreads) all += __ldg(tile_sum + x);
        all = cta_sum64<kFinishThreads>(all, red);
        if (t == 0) {
            // whole-vector check: (#greater) + min(#equal, r) must be k
            const uint32_t ng = (uint32_t)all, ne = (uint32_t)(all >> 32);
            if (ng + min(ne, ties) != k) hdr->status = SLIMDP_ERR_INTERNAL;
            dir[nb * kDirPerBlock] = (uint32_t)(n - k);
        }
    }

    // One tile of kEmitTile blocks per step, four consecutive bitmap words per thread; a scan over
    // the tile's words places every member.
    unsigned long long before = 0;   // counts in the tiles below the current one
    uint64_t counted = 0;            // tiles whose counts `before` holds
    const uint32_t w0 = (t & 7u) * 4u;   // first of this thread's four words in its block
    auto load_words = [&](uint64_t tile, uint4* Gw, uint4* Ew) {
        const uint64_t blk = tile * kEmitTile + (t >> 3);
        *Gw = *Ew = make_uint4(0, 0, 0, 0);
        if (tile < tile_last && blk < nb) {
            *Gw = __ldg(reinterpret_cast<const uint4*>(G + blk * kWordsPerBlock + w0));
            if (E != nullptr) *Ew = __ldg(reinterpret_cast<const uint4*>(E + blk * kWordsPerBlock + w0));
        }
    };
    uint4 Gnext, Enext;   // the next tile's words are requested before this tile's are worked on
    load_words(tile_first, &Gnext, &Enext);
    for (uint64_t tile = tile_first; tile < tile_last; tile += tile_step) {
        const uint4 Gw = Gnext, Ew = Enext;
        load_words(tile + tile_step, &Gnext, &Enext);
        unsigned long long v = 0;
        for (uint64_t x = counted + t; x < tile; x += kFinishThreads) v += __ldg(tile_sum + x);
        before += cta_sum64<kFinishThreads>(v, red);
        counted = tile;
        const uint64_t blk = tile * kEmitTile + (t >> 3);
        const bool have = blk < nb;
        const uint32_t gw[4] = {Gw.x, Gw.y, Gw.z, Gw.w}, ew[4] = {Ew.x, Ew.y, Ew.z, Ew.w};
        unsigned long long sum = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) sum += (unsigned long long)__popc(gw[q]) | ((unsigned long long)__popc(ew[q]) << 32);
        unsigned long long total;
        unsigned long long run = before + block_exclusive_scan64<kFinishThreads / 32>(sum, scan_smem, &total);
        uint32_t sel[4], pos0[4], dirv[2] = {0, 0};
        uint32_t members = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t g_before = (uint32_t)run, e_before = (uint32_t)(run >> 32);
            const uint32_t pe = __popc(ew[q]);
            // equal keys: admit those whose rank among all equal keys (index order) is below r
            const uint32_t admit = (ties > e_before) ? min(ties - e_before, pe) : 0u;
            uint32_t Ea;
            if (admit == pe)
                Ea = ew[q];
            else if (admit == 0)
                Ea = 0;
            else
                Ea = ew[q] & ((1u << nth_set_bit(ew[q], admit)) - 1u);
            sel[q] = gw[q] | Ea;
            pos0[q] = g_before + min(e_before, ties);   // core parameters below this word
            members += __popc(sel[q]);
            const uint32_t first = (uint32_t)(blk * kBlock) + (w0 + q) * 32u;
            if ((q & 1) == 0) dirv[q >> 1] = first - pos0[q];   // one directory entry per 64 parameters (2 words)
            run += (unsigned long long)__popc(gw[q]) | ((unsigned long long)pe << 32);
        }
        if (have) {
            *reinterpret_cast<uint4*>(bitmap + blk * kWordsPerBlock + w0) = make_uint4(sel[0], sel[1], sel[2], sel[3]);
            *reinterpret_cast<uint2*>(dir + blk * kDirPerBlock + (w0 >> 1)) = make_uint2(dirv[0], dirv[1]);
        }
        // the index list.  Few members in the warp's 128 words: every thread writes its own; many:
        // the warp writes one word's members at a time (coalesced)
        const uint32_t first0 = (uint32_t)(blk * kBlock) + w0 * 32u;
        const uint32_t warp_members = __reduce_add_sync(0xFFFFFFFFu, members);
        bool bad = false;
        if (warp_members <= kEmitOwnLists) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t pos = pos0[q];
                for (uint32_t word = sel[q]; word; word &= word - 1) {
                    if (pos < k)
                        core_idx[pos] = first0 + q * 32u + (uint32_t)__ffs(word) - 1u;
                    else
                        bad = true;
                    ++pos;
                }
            }
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                for (uint32_t m = __ballot_sync(0xFFFFFFFFu, sel[q] != 0); m; m &= m - 1) {
                    const int src = __ffs(m) - 1;
                    const uint32_t word = __shfl_sync(0xFFFFFFFFu, sel[q], src);
                    const uint32_t base = __shfl_sync(0xFFFFFFFFu, pos0[q], src);
                    const uint32_t first = __shfl_sync(0xFFFFFFFFu, first0, src) + q * 32u;
                    if ((word >> lane) & 1u) {
                        const uint32_t pos = base + __popc(word & lt_mask);
                        if (pos < k)
                            core_idx[pos] = first + lane;
                        else
                            bad = true;
                    }
                }
            }
        }
        if (bad) hdr->status = SLIMDP_ERR_INTERNAL;
        before += total;
        counted = tile + 1;
    }
}

inline slimdp_status launch_emit(const uint32_t* G, const uint32_t* E, const unsigned long long* tile_sum, uint64_t n,
                                 uint32_t k, WsHeader* hdr, uint32_t* core_idx, uint32_t* bitmap, uint32_t* dir,
                                 cudaStream_t st) {
    const uint64_t nb = num_blocks(n);
    const uint64_t ntiles = (nb + kEmitTile - 1) / kEmitTile;
    emit_kernel<<<(unsigned)((ntiles + kEmitGroup - 1) / kEmitGroup), kFinishThreads, 0, st>>>(
        G, E, tile_sum, n, nb, k, hdr, core_idx, bitmap, dir);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace

}  // namespace slimdp
