// slimdp_select_core_segmented: the ranking of Section 3.2 done layer by layer, the simplest
// "model-specific significance measure" that Section 5 points to.  The vector is cut into
// segments (layers); segment s contributes its seg_k[s] parameters of largest score, ties to the
// smaller index; the core is the union.
//
// One cooperative launch, phases separated by a bounded grid barrier.  Every CTA owns a contiguous
// run of keys and walks the segments that cross it:
//   rounds 0..2  most-significant-digit-first counting of the keys (12 + 10 + 10 bits), one
//                histogram per segment and round; after each round the segments are dealt out to
//                the CTAs, which find each segment's digit of its seg_k[s]-th largest key;
//   rounds 3..5  only if some segment admits a part of its keys equal to its threshold T_s: the same
//                three rounds over the positions (counted from the segment's end, so that "largest"
//                means "smallest index") of the keys equal to T_s; they give the last admitted index;
//   classify     a parameter is in the core iff key > T_s, or key == T_s and its index is admitted:
//                a pure predicate per parameter, so there is no tie bookkeeping afterwards;
//   emit         the selection's common last phase (bitmap, directory, ascending index list).
#include <atomic>

#include "common.cuh"
#include "layout.cuh"
#include "select_dev.cuh"

namespace slimdp {

namespace {

// Digits of the three counting rounds: 12, 10 and 10 bits, most significant first.
__host__ __device__ __forceinline__ uint32_t seg_bins(int r) { return r == 0 ? 4096u : 1024u; }
__host__ __device__ __forceinline__ uint32_t seg_shift(int r) { return r == 0 ? 20u : (r == 1 ? 10u : 0u); }
__host__ __device__ __forceinline__ uint32_t seg_hist_offset(int r) { return r == 0 ? 0u : (r == 1 ? 4096u : 5120u); }
constexpr uint32_t kSegHistWords = 4096u + 1024u + 1024u;   // one segment's histograms of three rounds

// Per segment, in the workspace.
struct SegState {
    uint32_t T;          // key rounds: prefix found so far; then the threshold
    uint32_t rem;        // rank still to resolve; after the key rounds the number of admitted equal keys
    uint32_t ipos;       // index rounds: prefix of the admitted position bound (positions count from the segment's end)
    uint32_t irem;
    uint32_t mode;       // 0: nothing of the segment; 1: key > T or (key == T and position >= ipos); 2: everything
    uint32_t pad[3];
};

static_assert(sizeof(SegState) == 32, "two 16-byte loads");

struct SegArgs {
    const uint32_t* keys;
    uint64_t n, nb;
    uint32_t segments;
    uint32_t k_total;
    const unsigned long long* seg_off;   // [segments + 1]
    const unsigned long long* seg_k;     // [segments]
    SegState* state;                     // [segments]
    uint32_t* hist;                      // [2][segments][kSegHistWords]: key rounds, index rounds
    uint32_t* flags;                     // [0]: some segment needs the index rounds
    WsHeader* hdr;
    uint32_t* G;
    unsigned long long* tile_sum;
    unsigned long long* super_pref;
    uint32_t* core_idx;
    uint32_t* bitmap;
    uint32_t* dir;
};

// A segment's state as other CTAs left it before the last grid barrier (read past this SM's L1).
__device__ __forceinline__ SegState seg_state(const SegState* p) {
    const uint4 lo = __ldcg(reinterpret_cast<const uint4*>(p));
    const uint4 hi = __ldcg(reinterpret_cast<const uint4*>(p) + 1);
    SegState st;
    st.T = lo.x;
    st.rem = lo.y;
    st.ipos = lo.z;
    st.irem = lo.w;
    st.mode = hi.x;
    st.pad[0] = st.pad[1] = st.pad[2] = 0;
    return st;
}

// The segment that holds index i (segments may be empty; i < seg_off[segments]).
__device__ __forceinline__ uint32_t seg_of(const unsigned long long* seg_off, uint32_t segments, uint64_t i) {
    uint32_t lo = 0, hi = segments - 1;   // largest s with seg_off[s] <= i
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo + 1) >> 1);
        if (__ldg(seg_off + mid) <= i)
            lo = mid;
        else
            hi = mid - 1;
    }
    return lo;
}

// Position of parameter i inside its segment, counted from the segment's end and stored so that a
// larger value means a smaller index: the first parameter of a segment has the largest value.
__device__ __forceinline__ uint32_t seg_ipos(uint64_t i, uint64_t seg_begin) {
    return 0xFFFFFFFFu - (uint32_t)(i - seg_begin);
}

// One counting round over this CTA's keys [c0, c1).  INDEX: count positions of keys equal to T_s.
template <bool INDEX>
__device__ __forceinline__ void seg_count_round(const SegArgs& a, int r, uint64_t c0, uint64_t c1, uint32_t* sh) {
    const uint32_t nbins = seg_bins(r), shift = seg_shift(r), hist_off = seg_hist_offset(r);
    uint32_t* hist_base = a.hist + (INDEX ? (size_t)a.segments * kSegHistWords : 0);
    uint64_t pos = c0;
    uint32_t s = (c0 < c1) ? seg_of(a.seg_off, a.segments, c0) : 0;
    while (pos < c1) {
        const uint64_t seg_begin = __ldg(a.seg_off + s), seg_end_all = __ldg(a.seg_off + s + 1);
        const uint64_t end = seg_end_all < c1 ? seg_end_all : c1;
        const SegState st = seg_state(a.state + s);
        const bool counts = st.mode == 1 && (!INDEX || st.irem > 0);
        if (counts && pos < end) {
            for (uint32_t b = threadIdx.x; b < nbins; b += kFinishThreads) sh[b] = 0;
            __syncthreads();
            const uint32_t prefix = INDEX ? st.ipos : st.T;
            for (uint64_t i = pos + threadIdx.x; i < end; i += kFinishThreads) {
                const uint32_t key = __ldcg(a.keys + i);
                uint32_t v = key;
                if (INDEX) {
                    if (key != st.T) continue;
                    v = seg_ipos(i, seg_begin);
                }
                // rounds 1 and 2 count only what agrees with the digits found so far (12, then 22 bits)
                const bool match = (r == 0) || ((v >> (shift + 10)) == (prefix >> (shift + 10)));
                if (match) atomicAdd(&sh[(v >> shift) & (nbins - 1)], 1u);
            }
            __syncthreads();
            uint32_t* hist = hist_base + (size_t)s * kSegHistWords + hist_off;
            for (uint32_t b = threadIdx.x; b < nbins; b += kFinishThreads)
                if (sh[b]) atomicAdd(&hist[b], sh[b]);
            __syncthreads();
        }
        pos = end;
        if (pos == seg_end_all) ++s;
    }
}

// After a round: the segments are dealt out to the CTAs; each finds its segment's digit.
template <bool INDEX>
__device__ __forceinline__ void seg_resolve_round(const SegArgs& a, int r, unsigned long long* scan_smem, uint32_t* res) {
    const uint32_t hist_off = seg_hist_offset(r);
    const uint32_t* hist_base = a.hist + (INDEX ? (size_t)a.segments * kSegHistWords : 0);
    for (uint32_t s = blockIdx.x; s < a.segments; s += gridDim.x) {
        SegState* st = a.state + s;
        const SegState now = seg_state(st);
        const uint32_t mode = now.mode, want = INDEX ? now.irem : now.rem;
        if (mode != 1 || (INDEX && want == 0)) continue;   // CTA-uniform
        const uint32_t* hist = hist_base + (size_t)s * kSegHistWords + hist_off;
        uint32_t bin, rem;
        const bool found = find_rank_bin<kFinishThreads>(hist, seg_bins(r), want, scan_smem, res, &bin, &rem);
        if (threadIdx.x == 0) {
            if (!found) {
                a.hdr->status = SLIMDP_ERR_INTERNAL;
            } else if (INDEX) {
                st->ipos = now.ipos | (bin << seg_shift(r));
                st->irem = rem;
            } else {
                st->T = now.T | (bin << seg_shift(r));
                st->rem = rem;
                if (r == 2) {
                    // hist[bin] keys of the segment equal T; rem of them belong to the core
                    const uint32_t equal = __ldcg(hist + bin);
                    if (rem < equal) {
                        st->irem = rem;          // the index rounds find the rem-th smallest index among them
                        atomicOr(a.flags, 1u);
                    } else {
                        st->irem = 0;            // all of them: every position is admitted
                    }
                    st->ipos = 0;
                }
            }
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kFinishThreads, 2) seg_select_kernel(SegArgs a) {
    __shared__ uint32_t sh[4096];
    __shared__ unsigned long long scan_smem[33];
    __shared__ uint32_t res[3];
    const uint32_t t = threadIdx.x, lane = lane_id(), wid = t >> 5;
    uint32_t epoch = 0;
    // segment states (k = 0: nothing, k = length: everything, else the rounds decide)
    for (uint32_t s = blockIdx.x * kFinishThreads + t; s < a.segments; s += gridDim.x * kFinishThreads) {
        const unsigned long long len = a.seg_off[s + 1] - a.seg_off[s], ks = a.seg_k[s];
        SegState st{};
        st.rem = (uint32_t)ks;
        st.mode = (ks == 0) ? 0u : (ks >= len ? 2u : 1u);
        a.state[s] = st;
    }
    if (!grid_barrier(a.hdr, &epoch)) return;
    // this CTA's run of keys, cut at multiples of 1024
    const uint64_t per = (a.nb + gridDim.x - 1) / gridDim.x;
    const uint64_t b0 = ((uint64_t)blockIdx.x * per < a.nb) ? (uint64_t)blockIdx.x * per : a.nb;
    const uint64_t b1 = (b0 + per < a.nb) ? b0 + per : a.nb;
    const uint64_t c0 = b0 * kBlock, c1 = (b1 * kBlock < a.n) ? b1 * kBlock : a.n;
    for (int r = 0; r < 3; ++r) {
        seg_count_round<false>(a, r, c0, c1, sh);
        if (!grid_barrier(a.hdr, &epoch)) return;
        seg_resolve_round<false>(a, r, scan_smem, res);
        if (!grid_barrier(a.hdr, &epoch)) return;
    }
    if (*reinterpret_cast<volatile uint32_t*>(a.flags) != 0u) {   // the same for every CTA: read after a barrier
        for (int r = 0; r < 3; ++r) {
            seg_count_round<true>(a, r, c0, c1, sh);
            if (!grid_barrier(a.hdr, &epoch)) return;
            seg_resolve_round<true>(a, r, scan_smem, res);
            if (!grid_barrier(a.hdr, &epoch)) return;
        }
    }
    // classify: warp per 1024-parameter block of this CTA's run
    for (uint64_t blk = b0 + wid; blk < b1; blk += kFinishThreads / 32) {
        const uint64_t base = blk * kBlock;
        uint32_t s = seg_of(a.seg_off, a.segments, base + lane < a.n ? base + lane : a.n - 1);
        uint64_t seg_begin = __ldg(a.seg_off + s), seg_end = __ldg(a.seg_off + s + 1);
        SegState st = seg_state(a.state + s);
        uint32_t mine = 0;
        for (int wd = 0; wd < 32; ++wd) {
            const uint64_t i = base + wd * 32 + lane;
            const bool in = i < a.n;
            bool take = false;
            if (in) {
                while (i >= seg_end) {   // on to the segment that holds i (empty segments are passed over)
                    ++s;
                    seg_begin = seg_end;
                    seg_end = __ldg(a.seg_off + s + 1);
                    st = seg_state(a.state + s);
                }
                const uint32_t key = __ldcg(a.keys + i);
                take = st.mode == 2 ||
                       (st.mode == 1 && (key > st.T || (key == st.T && seg_ipos(i, seg_begin) >= st.ipos)));
            }
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, take);
            if (lane == (uint32_t)wd) mine = word;
        }
        a.G[blk * kWordsPerBlock + lane] = mine;
        const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, __popc(mine));
        if (lane == 0 && c) atomicAdd(&a.tile_sum[blk / kEmitTile], (unsigned long long)c);
    }
    if (!grid_barrier(a.hdr, &epoch)) return;
    super_sum_phase<kFinishThreads>(a.tile_sum, a.super_pref, a.nb);
    if (!grid_barrier(a.hdr, &epoch)) return;
    if (blockIdx.x == 0)
        tile_scan_phase<kFinishThreads>(a.super_pref, a.n, a.nb, a.k_total, 0u, a.hdr, a.dir, scan_smem);
}

}  // namespace

namespace {

struct SegWs {
    WsHeader* hdr;
    uint32_t* flags;
    unsigned long long* tile_sum;
    unsigned long long* super_pref;
    uint32_t* hist;
    size_t zero_bytes;   // header, flags, tile counts and histograms, contiguous
    unsigned long long* seg_off;
    unsigned long long* seg_k;
    SegState* state;
    uint32_t* G;
    size_t bytes;
};

SegWs seg_ws_layout(void* ws, uint64_t n, uint32_t segments) {
    const uint64_t nb = num_blocks(n);
    char* p = reinterpret_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char* r = p + off;
        off += align_up(bytes ? bytes : 1, 256);
        return r;
    };
    SegWs L;
    L.hdr = reinterpret_cast<WsHeader*>(take(sizeof(WsHeader)));
    L.flags = reinterpret_cast<uint32_t*>(take(16));
    L.tile_sum = reinterpret_cast<unsigned long long*>(take(((nb + kEmitTile - 1) / kEmitTile) * 8));
    L.hist = reinterpret_cast<uint32_t*>(take((size_t)2 * segments * kSegHistWords * 4));
    L.zero_bytes = off;
    L.super_pref = reinterpret_cast<unsigned long long*>(take(num_super_tiles(nb) * 8));
    L.seg_off = reinterpret_cast<unsigned long long*>(take(((size_t)segments + 1) * 8));
    L.seg_k = reinterpret_cast<unsigned long long*>(take((size_t)segments * 8));
    L.state = reinterpret_cast<SegState*>(take((size_t)segments * sizeof(SegState)));
    L.G = reinterpret_cast<uint32_t*>(take(nb * kWordsPerBlock * 4));
    L.bytes = off;
    return L;
}

}  // namespace

size_t seg_select_ws_bytes(uint64_t n, uint32_t segments) { return seg_ws_layout(nullptr, n, segments).bytes; }

// seg_off / seg_k: HOST arrays, copied into the workspace before the kernel starts.
slimdp_status launch_select_segmented(const float* scores, uint64_t n, const uint64_t* seg_off, const uint64_t* seg_k,
                                      uint32_t segments, uint64_t k_total, uint32_t* core_idx, void* core_aux,
                                      void* ws, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    const SegWs L = seg_ws_layout(ws, n, segments);
    if (cudaMemsetAsync(L.hdr, 0, L.zero_bytes, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
    if (cudaMemcpyAsync(L.seg_off, seg_off, ((size_t)segments + 1) * 8, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(L.seg_k, seg_k, (size_t)segments * 8, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return SLIMDP_ERR_CUDA;
    static std::atomic<int> per_sm_cached[64];   // 0 = not asked yet, < 0 = no cooperative launch here
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLIMDP_ERR_CUDA;
    int f = per_sm_cached[dev].load(std::memory_order_relaxed);
    if (f == 0) {
        int per_sm = 0, coop = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, seg_select_kernel, kFinishThreads, 0) != cudaSuccess)
            return SLIMDP_ERR_CUDA;
        f = (coop && per_sm >= 1) ? (per_sm > 2 ? 2 : per_sm) : -1;
        per_sm_cached[dev].store(f, std::memory_order_relaxed);
    }
    if (f < 0) return SLIMDP_ERR_CUDA;
    uint64_t grid = (n + 16383) / 16384;
    if (grid > (uint64_t)sms * f) grid = (uint64_t)sms * f;
    if (grid < 1) grid = 1;
    SegArgs a{};
    a.keys = reinterpret_cast<const uint32_t*>(scores);
    a.n = n;
    a.nb = num_blocks(n);
    a.segments = segments;
    a.k_total = (uint32_t)k_total;
    a.seg_off = L.seg_off;
    a.seg_k = L.seg_k;
    a.state = L.state;
    a.hist = L.hist;
    a.flags = L.flags;
    a.hdr = L.hdr;
    a.G = L.G;
    a.tile_sum = L.tile_sum;
    a.super_pref = L.super_pref;
    a.core_idx = core_idx;
    a.bitmap = reinterpret_cast<uint32_t*>(core_aux);
    a.dir = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(core_aux) + slimdp_core_aux_dir_offset(n));
    void* args[] = {&a};
    if (cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(seg_select_kernel), dim3((unsigned)grid),
                                    dim3(kFinishThreads), args, 0, st) != cudaSuccess)
        return SLIMDP_ERR_CUDA;
    SLIMDP_LAUNCHED(1);
    return launch_emit(L.G, nullptr, L.tile_sum, L.super_pref, n, (uint32_t)k_total, L.hdr, core_idx, a.bitmap, a.dir, st);
}

}  // namespace slimdp
