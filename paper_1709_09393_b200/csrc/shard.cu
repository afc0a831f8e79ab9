// Selection over a range-sharded model (the parameter-server setting of Section 2.1 with the
// global model cut into contiguous shards, one per GPU).  Score, pack, merge and pull are
// independent per shard; the core is not: Section 3.2 ranks ALL parameters.  The exact global
// threshold is found with the selection's radix rounds cut at their reduction points:
//   per shard   slimdp_select_hist     one digit's histogram of the shard's keys (12 + 10 + 10 bits)
//   all shards  sum of the histograms  (an all-reduce of 4096 64-bit counters)
//   per shard   slimdp_select_resolve  the digit of the wanted rank, from the summed histogram;
//                                      every shard computes the same prefix and remaining rank
//   per shard   slimdp_select_count    keys above / equal to the threshold T in the shard
//   all shards  an all-gather of those two counts: shard g admits
//               min(#equal_g, max(0, r - #equal in shards below g)) of its equal keys, r = k - sum #greater
//   per shard   slimdp_select_emit     the shard's part of the core for (T, its tie quota)
// State that passes from call to call lives in a 16-byte device record (prefix, remaining rank),
// so the chain can be enqueued without a host round trip between the rounds.
#include "common.cuh"

namespace slimdp {

namespace {

struct ShardState {
    uint32_t prefix;      // digits of T found so far (high bits)
    int32_t status;       // SLIMDP_OK, or SLIMDP_ERR_INTERNAL if a summed histogram held fewer keys than the rank
    unsigned long long rem;   // rank still to resolve inside the prefix
};

template <int ROUND>
__device__ __forceinline__ void shard_hist_key(uint32_t key, uint32_t prefix, uint32_t* sh) {
    if (ROUND == 0) {
        atomicAdd(&sh[key >> 20], 1u);
    } else if (ROUND == 1) {
        if ((key >> 20) == (prefix >> 20)) atomicAdd(&sh[(key >> 10) & 1023u], 1u);
    } else {
        if ((key >> 10) == (prefix >> 10)) atomicAdd(&sh[key & 1023u], 1u);
    }
}

// hist[b] += number of the shard's keys whose digit of this round is b (and whose higher digits equal the prefix).
template <int ROUND>
__global__ void __launch_bounds__(512) shard_hist_kernel(const uint32_t* __restrict__ keys, uint64_t n,
                                                         const ShardState* __restrict__ state,
                                                         unsigned long long* __restrict__ hist) {
    constexpr uint32_t NB = (ROUND == 0) ? 4096u : 1024u;
    __shared__ uint32_t sh[NB];
    for (uint32_t b = threadIdx.x; b < NB; b += blockDim.x) sh[b] = 0;
    __syncthreads();
    const uint32_t prefix = (ROUND == 0) ? 0u : state->prefix;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        shard_hist_key<ROUND>(__ldcs(keys + i), prefix, sh);
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < NB; b += blockDim.x)
        if (sh[b]) atomicAdd(&hist[b], (unsigned long long)sh[b]);
}

// One CTA of 1024 threads: walks the summed histogram from its top bin down to the bin in which the
// running count reaches state->rem, and records that digit and the rank left inside it.
__global__ void __launch_bounds__(1024) shard_resolve_kernel(const unsigned long long* __restrict__ hist,
                                                             uint32_t round, ShardState* state) {
    __shared__ unsigned long long smem[33];
    const uint32_t nbins = (round == 0) ? 4096u : 1024u;
    const uint32_t shift = (round == 0) ? 20u : (round == 1 ? 10u : 0u);
    const uint32_t per = nbins / 1024u;   // 4 or 1
    const uint32_t t = threadIdx.x;
    const unsigned long long want = state->rem;
    unsigned long long h[4] = {0, 0, 0, 0}, sum = 0;
    for (uint32_t q = 0; q < per; ++q) {
        h[q] = hist[nbins - 1 - (t * per + q)];
        sum += h[q];
    }
    unsigned long long total;
    unsigned long long above = block_exclusive_scan64<32>(sum, smem, &total);
    if (want == 0) {
        // an empty core (only ever at the first round: a resolved digit leaves a rank of at least 1):
        // no key lies above the largest bit pattern, and no key equal to it is admitted
        if (t == 0) state->prefix = 0xFFFFFFFFu;
        return;
    }
    if (total < want) {
        if (t == 0) state->status = SLIMDP_ERR_INTERNAL;
        return;
    }
    for (uint32_t q = 0; q < per; ++q) {
        if (above < want && want <= above + h[q]) {
            state->prefix = state->prefix | ((nbins - 1 - (t * per + q)) << shift);
            state->rem = want - above;
        }
        above += h[q];
    }
}

// counts[0] += keys above T, counts[1] += keys equal to T, T = state->prefix.
__global__ void __launch_bounds__(512) shard_count_kernel(const uint32_t* __restrict__ keys, uint64_t n,
                                                          const ShardState* __restrict__ state,
                                                          unsigned long long* __restrict__ counts) {
    __shared__ unsigned long long part[2][16];
    const uint32_t T = state->prefix;
    unsigned long long g = 0, e = 0;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const uint32_t key = __ldcs(keys + i);
        g += key > T;
        e += key == T;
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        g += __shfl_xor_sync(0xFFFFFFFFu, g, d);
        e += __shfl_xor_sync(0xFFFFFFFFu, e, d);
    }
    if ((threadIdx.x & 31u) == 0) {
        part[0][threadIdx.x >> 5] = g;
        part[1][threadIdx.x >> 5] = e;
    }
    __syncthreads();
    if (threadIdx.x < 2) {
        unsigned long long s = 0;
        for (int x = 0; x < 16; ++x) s += part[threadIdx.x][x];
        if (s) atomicAdd(&counts[threadIdx.x], s);
    }
}

__global__ void shard_state_init_kernel(ShardState* state, unsigned long long k) {
    state->prefix = 0;
    state->status = SLIMDP_OK;
    state->rem = k;
}

}  // namespace

slimdp_status launch_shard_state_init(void* state, uint64_t k, cudaStream_t st) {
    shard_state_init_kernel<<<1, 1, 0, st>>>(reinterpret_cast<ShardState*>(state), k);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

slimdp_status launch_shard_hist(const float* scores, uint64_t n, uint32_t round, const void* state, uint64_t* hist,
                                cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    if (n == 0) return SLIMDP_OK;
    uint64_t grid = (n + 511) / 512;
    if (grid > (uint64_t)sms * 4) grid = (uint64_t)sms * 4;
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(scores);
    const ShardState* s = reinterpret_cast<const ShardState*>(state);
    unsigned long long* h = reinterpret_cast<unsigned long long*>(hist);
    if (round == 0)
        shard_hist_kernel<0><<<(unsigned)grid, 512, 0, st>>>(keys, n, s, h);
    else if (round == 1)
        shard_hist_kernel<1><<<(unsigned)grid, 512, 0, st>>>(keys, n, s, h);
    else
        shard_hist_kernel<2><<<(unsigned)grid, 512, 0, st>>>(keys, n, s, h);
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

slimdp_status launch_shard_resolve(const uint64_t* hist, uint32_t round, void* state, cudaStream_t st) {
    shard_resolve_kernel<<<1, 1024, 0, st>>>(reinterpret_cast<const unsigned long long*>(hist), round,
                                             reinterpret_cast<ShardState*>(state));
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

slimdp_status launch_shard_count(const float* scores, uint64_t n, const void* state, uint64_t* counts,
                                 cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return SLIMDP_ERR_CUDA;
    if (n == 0) return SLIMDP_OK;
    uint64_t grid = (n + 511) / 512;
    if (grid > (uint64_t)sms * 4) grid = (uint64_t)sms * 4;
    shard_count_kernel<<<(unsigned)grid, 512, 0, st>>>(reinterpret_cast<const uint32_t*>(scores), n,
                                                       reinterpret_cast<const ShardState*>(state),
                                                       reinterpret_cast<unsigned long long*>(counts));
    SLIMDP_LAUNCHED(1);
    return SLIMDP_OK;
}

}  // namespace slimdp
