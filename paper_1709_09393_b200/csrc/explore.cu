// slimdp_sample_explore: the exploration operator T_R^k (Section 3.1 item 2,
// Section 3.3 step 2): k_exp distinct parameters drawn uniformly from outside
// the core, anew for every worker and every communication round.
//
//   1. round keys: three Philox-4x32-10 blocks per worker;
//   2. thread j evaluates the keyed permutation pi(j) of the non-core ranks
//      (10-round Feistel network with cycle walking), turns the rank into a
//      parameter index with a select-zero query on the core bitmap (binary
//      search of the per-1024 rank directory, then a popcount walk over the 32
//      words of the block) and sets that bit in the worker's mark bitmap;
//   3. the mark bitmap is compacted into the ascending index list (per-block
//      popcounts, two-kernel scan, warp-ordered expansion).
#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

namespace {

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

__global__ void explore_setup_kernel(WsHeader* hdr, uint32_t* __restrict__ rk, uint32_t seed_lo, uint32_t seed_hi,
                                     uint32_t first_worker, uint32_t workers, uint32_t round) {
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t == 0) hdr->status = SLIMDP_OK;
    if (t >= workers * 3) return;
    const uint32_t w = t / 3, b = t % 3;
    uint32_t out[4];
    philox4x32_10(seed_lo, seed_hi, b, first_worker + w, round, 0x534C494Du, out);
#pragma unroll
    for (int q = 0; q < 4; ++q) rk[w * 12 + b * 4 + q] = out[q];
}

__global__ void __launch_bounds__(256) mark_kernel(const uint32_t* __restrict__ bitmap,
                                                   const uint32_t* __restrict__ dir, uint32_t nb, uint32_t M,
                                                   uint32_t k_exp, uint32_t h, const uint32_t* __restrict__ rk_all,
                                                   uint32_t* __restrict__ marks, uint64_t mark_stride,
                                                   WsHeader* hdr) {
    const uint32_t worker = blockIdx.y;
    uint32_t rk[10];
#pragma unroll
    for (int r = 0; r < 10; ++r) rk[r] = rk_all[worker * 12 + r];
    const uint32_t mask = (h >= 32) ? 0xFFFFFFFFu : ((1u << h) - 1u);
    uint32_t* my_marks = marks + (uint64_t)worker * mark_stride;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_exp; j += stride) {
        // pi(j): Feistel network, re-applied while the image is outside [0, M)
        uint32_t x = (uint32_t)j;
        do {
            uint32_t L = x >> h, R = x & mask;
#pragma unroll
            for (int r = 0; r < 10; ++r) {
                const uint32_t mult = (r & 1) ? 0xCD9E8D57u : 0xD2511F53u;
                const uint32_t v = R ^ rk[r];
                const uint32_t F = __umulhi(v, mult) ^ (v * mult);
                const uint32_t nr = (L ^ F) & mask;
                L = R;
                R = nr;
            }
            x = (L << h) | R;
        } while (x >= M);
        // select0(x): the x-th (0-based) non-core parameter
        uint32_t lo = 0, hi = nb - 1;
        while (lo < hi) {
            const uint32_t mid = lo + ((hi - lo + 1) >> 1);
            if (__ldg(dir + mid) <= x)
                lo = mid;
            else
                hi = mid - 1;
        }
        uint32_t rem = x - __ldg(dir + lo);
        const uint4* words = reinterpret_cast<const uint4*>(bitmap + (uint64_t)lo * kWordsPerBlock);
        uint32_t found = 0xFFFFFFFFu;
#pragma unroll 1
        for (int q = 0; q < 8 && found == 0xFFFFFFFFu; ++q) {
            const uint4 v = __ldg(words + q);
            const uint32_t z[4] = {~v.x, ~v.y, ~v.z, ~v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t c = __popc(z[e]);
                if (found == 0xFFFFFFFFu) {
                    if (rem < c)
                        found = (uint32_t)(q * 4 + e) * 32u + nth_set_bit(z[e], rem);
                    else
                        rem -= c;
                }
            }
        }
        if (found == 0xFFFFFFFFu) {
            hdr->status = SLIMDP_ERR_INTERNAL;   // directory and bitmap disagree
            continue;
        }
        const uint32_t idx = lo * kBlock + found;
        atomicOr(&my_marks[idx >> 5], 1u << (idx & 31u));
    }
}

__global__ void __launch_bounds__(256) count_marks_kernel(const uint32_t* __restrict__ marks, uint64_t mark_stride,
                                                          uint64_t nb, unsigned long long* __restrict__ cnt,
                                                          uint64_t cnt_stride) {
    const uint32_t worker = blockIdx.y, lane = lane_id();
    const uint32_t* my = marks + (uint64_t)worker * mark_stride;
    const uint64_t warps = (uint64_t)gridDim.x * (blockDim.x >> 5);
    for (uint64_t blk = (uint64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); blk < nb; blk += warps) {
        const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, __popc(my[blk * kWordsPerBlock + lane]));
        if (lane == 0) cnt[(uint64_t)worker * cnt_stride + blk] = c;
    }
}

__global__ void __launch_bounds__(256) expand_marks_kernel(const uint32_t* __restrict__ marks, uint64_t mark_stride,
                                                           uint64_t nb, const unsigned long long* __restrict__ pref,
                                                           const unsigned long long* __restrict__ totals,
                                                           uint64_t cnt_stride, uint32_t k_exp,
                                                           PtrArray<uint32_t> out, WsHeader* hdr) {
    const uint32_t worker = blockIdx.y, lane = lane_id();
    const uint32_t* my = marks + (uint64_t)worker * mark_stride;
    uint32_t* dst = out.p[worker];
    const uint64_t warps = (uint64_t)gridDim.x * (blockDim.x >> 5);
    const uint64_t warp0 = (uint64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (warp0 == 0 && lane == 0 && totals[worker] != k_exp) hdr->status = SLIMDP_ERR_INTERNAL;
    for (uint64_t blk = warp0; blk < nb; blk += warps) {
        const uint32_t sel = my[blk * kWordsPerBlock + lane];
        const uint32_t ps = __popc(sel);
        const uint32_t any = __ballot_sync(0xFFFFFFFFu, sel != 0);
        if (any == 0) continue;
        const uint32_t out_base = (uint32_t)pref[(uint64_t)worker * cnt_stride + blk] + warp_inclusive_scan(ps) - ps;
        for (uint32_t m = any; m; m &= m - 1) {
            const int wd = __ffs(m) - 1;
            const uint32_t word = __shfl_sync(0xFFFFFFFFu, sel, wd);
            const uint32_t base = __shfl_sync(0xFFFFFFFFu, out_base, wd);
            if ((word >> lane) & 1u) {
                const uint32_t pos = base + __popc(word & ((1u << lane) - 1u));
                if (pos < k_exp)
                    dst[pos] = (uint32_t)(blk * kBlock + wd * 32 + lane);
                else
                    hdr->status = SLIMDP_ERR_INTERNAL;
            }
        }
    }
}

}  // namespace

slimdp_status launch_explore(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                             uint32_t first_worker, uint32_t workers, uint32_t round,
                             const PtrArray<uint32_t>& out, void* ws, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const ExploreWs L = explore_ws_layout(ws, n, workers);
    const uint64_t nb = num_blocks(n);
    const uint64_t M = n - k_core;
    const uint32_t* bitmap = reinterpret_cast<const uint32_t*>(core_aux);
    const uint32_t* dir =
        reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(core_aux) + slimdp_core_aux_dir_offset(n));

    explore_setup_kernel<<<1, 256, 0, st>>>(L.hdr, L.round_keys, (uint32_t)seed, (uint32_t)(seed >> 32),
                                            first_worker, workers, round);
    SLIMDP_LAUNCHED(1);
    if (k_exp == 0) return SLIMDP_OK;
    if (cudaMemsetAsync(L.marks, 0, (size_t)workers * L.mark_stride * 4, st) != cudaSuccess) return SLIMDP_ERR_CUDA;

    int b = 1;
    while (((uint64_t)1 << b) < M) ++b;
    const uint32_t h = (uint32_t)((b + 1) / 2);

    uint64_t mgrid = (k_exp + 255) / 256;
    if (mgrid > (uint64_t)sms * 16) mgrid = (uint64_t)sms * 16;
    mark_kernel<<<dim3((unsigned)mgrid, workers), 256, 0, st>>>(bitmap, dir, (uint32_t)nb, (uint32_t)M,
                                                                (uint32_t)k_exp, h, L.round_keys, L.marks,
                                                                L.mark_stride, L.hdr);
    SLIMDP_LAUNCHED(1);
    uint64_t cgrid = (nb + 7) / 8;
    const uint64_t cap = ((uint64_t)sms * 8 + workers - 1) / workers;
    if (cgrid > cap) cgrid = cap;
    if (cgrid == 0) cgrid = 1;
    count_marks_kernel<<<dim3((unsigned)cgrid, workers), 256, 0, st>>>(L.marks, L.mark_stride, nb, L.cnt,
                                                                       L.cnt_stride);
    SLIMDP_LAUNCHED(1);
    slimdp_status s =
        launch_block_scan(L.cnt, L.pref, L.tile_sums, L.totals, nb, workers, L.cnt_stride, L.tile_stride, st);
    if (s != SLIMDP_OK) return s;
    expand_marks_kernel<<<dim3((unsigned)cgrid, workers), 256, 0, st>>>(L.marks, L.mark_stride, nb, L.pref, L.totals,
                                                                        L.cnt_stride, (uint32_t)k_exp, out, L.hdr);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
