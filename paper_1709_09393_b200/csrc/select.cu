// slimdp_select_core: exact top-k_core of the scores (Section 3.2: rank by
// significance, keep the top), ties to the smaller index.
//
// Keys are the scores' 32-bit patterns compared as unsigned integers.
//   1. three most-significant-digit-first histogram passes (12 + 10 + 10 bits,
//      shared-memory histograms flushed to global) find the exact k-th largest
//      key T and the number r of keys equal to T that belong to the core;
//   2. one pass classifies every key against T into two bitmaps (greater,
//      equal) and counts both per 1024-parameter block;
//   3. a two-kernel exclusive scan over the block counts;
//   4. one pass over the bitmaps admits the first r equal keys in index order,
//      writes the final core bitmap, the non-core rank directory and the
//      ascending index list (ordered compaction: ballot/popc inside a warp,
//      scanned block offsets across warps; no atomic cursors, no spinning).
#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

namespace {

constexpr int kHistThreads = 512;
constexpr uint32_t kBins0 = 4096;   // pass 0: bits 31..20
constexpr uint32_t kBins12 = 1024;  // pass 1: bits 19..10, pass 2: bits 9..0

__global__ void select_init_kernel(WsHeader* hdr, uint32_t k) {
    hdr->status = SLIMDP_OK;
    hdr->prefix = (k == 0) ? 0xFFFFFFFFu : 0u;   // k = 0: no key is greater than or (with r = 0) admitted at T
    hdr->k_rem = k;
    hdr->ties = 0;
}

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

template <int PASS>
__global__ void __launch_bounds__(kHistThreads) hist_kernel(const uint32_t* __restrict__ keys, uint64_t n,
                                                            const WsHeader* __restrict__ hdr,
                                                            uint32_t* __restrict__ hist) {
    constexpr uint32_t NB = (PASS == 0) ? kBins0 : kBins12;
    __shared__ uint32_t sh[NB];
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
}

// One block of 1024 threads: walk the histogram from the top bin down and
// find the bin holding the k_rem-th largest key.
template <int PASS>
__global__ void __launch_bounds__(1024) find_bin_kernel(WsHeader* hdr, const uint32_t* __restrict__ hist) {
    constexpr uint32_t NB = (PASS == 0) ? kBins0 : kBins12;
    constexpr uint32_t PER = NB / 1024;
    constexpr uint32_t SHIFT = (PASS == 0) ? 20 : (PASS == 1 ? 10 : 0);
    __shared__ unsigned long long smem[33];
    const uint32_t k = hdr->k_rem;
    const uint32_t prefix = hdr->prefix;
    const uint32_t top = NB - 1 - threadIdx.x * PER;   // this thread's highest bin
    uint32_t h[PER];
    unsigned long long sum = 0;
#pragma unroll
    for (uint32_t q = 0; q < PER; ++q) {
        h[q] = hist[top - q];
        sum += h[q];
    }
    unsigned long long total;
    unsigned long long above = block_exclusive_scan64_1024(sum, smem, &total);
    if (total < k) {
        if (threadIdx.x == 0) hdr->status = SLIMDP_ERR_INTERNAL;
        return;
    }
#pragma unroll
    for (uint32_t q = 0; q < PER; ++q) {
        if (above < k && (unsigned long long)k <= above + h[q]) {
            const uint32_t rem = k - (uint32_t)above;
            hdr->prefix = prefix | ((top - q) << SHIFT);
            hdr->k_rem = rem;
            if (PASS == 2) hdr->ties = rem;
        }
        above += h[q];
    }
}

// Warp per 1024-parameter block: two bitmap words per lane and the block's counts.
__global__ void __launch_bounds__(256) classify_kernel(const uint32_t* __restrict__ keys, uint64_t n, uint64_t nb,
                                                       const WsHeader* __restrict__ hdr, uint32_t* __restrict__ G,
                                                       uint32_t* __restrict__ E,
                                                       unsigned long long* __restrict__ cnt) {
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
        dir[nb] = (uint32_t)(n - k_core);
    }
    for (uint64_t blk = warp0; blk < nb; blk += warps) {
        const uint32_t Gw = G[blk * kWordsPerBlock + lane];
        const uint32_t Ew = E[blk * kWordsPerBlock + lane];
        const unsigned long long p = pref[blk];
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
        const uint32_t out_base = sel_before + warp_inclusive_scan(ps) - ps;
        bitmap[blk * kWordsPerBlock + lane] = sel;
        if (lane == 0) dir[blk] = (uint32_t)(blk * kBlock - sel_before);
        const uint32_t any = __ballot_sync(0xFFFFFFFFu, sel != 0);
        for (uint32_t m = any; m; m &= m - 1) {
            const int wd = __ffs(m) - 1;
            const uint32_t word = __shfl_sync(0xFFFFFFFFu, sel, wd);
            const uint32_t base = __shfl_sync(0xFFFFFFFFu, out_base, wd);
            if ((word >> lane) & 1u) {
                const uint32_t pos = base + __popc(word & ((1u << lane) - 1u));
                if (pos < k_core)
                    core_idx[pos] = (uint32_t)(blk * kBlock + wd * 32 + lane);
                else
                    hdr->status = SLIMDP_ERR_INTERNAL;
            }
        }
    }
}

}  // namespace

slimdp_status launch_select(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx, void* core_aux,
                            void* ws, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const SelectWs L = select_ws_layout(ws, n);
    const uint64_t nb = num_blocks(n);
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(scores);
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(core_aux);
    uint32_t* dir = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(core_aux) + slimdp_core_aux_dir_offset(n));

    select_init_kernel<<<1, 1, 0, st>>>(L.hdr, (uint32_t)k_core);
    SLIMDP_LAUNCHED(1);
    if (k_core > 0) {
        if (cudaMemsetAsync(L.hist, 0, 3 * kBins0 * sizeof(uint32_t), st) != cudaSuccess) return SLIMDP_ERR_CUDA;
        const unsigned hgrid = (unsigned)sms * 4;
        hist_kernel<0><<<hgrid, kHistThreads, 0, st>>>(keys, n, L.hdr, L.hist);
        find_bin_kernel<0><<<1, 1024, 0, st>>>(L.hdr, L.hist);
        hist_kernel<1><<<hgrid, kHistThreads, 0, st>>>(keys, n, L.hdr, L.hist + kBins0);
        find_bin_kernel<1><<<1, 1024, 0, st>>>(L.hdr, L.hist + kBins0);
        hist_kernel<2><<<hgrid, kHistThreads, 0, st>>>(keys, n, L.hdr, L.hist + 2 * kBins0);
        find_bin_kernel<2><<<1, 1024, 0, st>>>(L.hdr, L.hist + 2 * kBins0);
        SLIMDP_LAUNCHED(6);
    }
    uint64_t cgrid = (nb + 7) / 8;
    if (cgrid > (uint64_t)sms * 8) cgrid = (uint64_t)sms * 8;
    classify_kernel<<<(unsigned)cgrid, 256, 0, st>>>(keys, n, nb, L.hdr, L.G, L.E, L.cnt);
    SLIMDP_LAUNCHED(1);
    slimdp_status s = launch_block_scan(L.cnt, L.pref, L.tile_sums, L.totals, nb, 1, nb, num_scan_tiles(n), st);
    if (s != SLIMDP_OK) return s;
    emit_kernel<<<(unsigned)cgrid, 256, 0, st>>>(L.G, L.E, L.pref, L.totals, n, nb, (uint32_t)k_core, L.hdr,
                                                 core_idx, bitmap, dir);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
