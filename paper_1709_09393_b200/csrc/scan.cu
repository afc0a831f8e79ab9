// Exclusive prefix sums over per-bitmap-block counters, without inter-CTA waits:
// one kernel reduces tiles of 1024 counters, a second adds the sum of the
// earlier tiles and scans inside each tile.
#include "common.cuh"

namespace slimdp {

namespace {

__global__ void __launch_bounds__(1024) tile_sum_kernel(const unsigned long long* __restrict__ cnt,
                                                        unsigned long long* __restrict__ tile_sums, uint64_t nb,
                                                        uint64_t stride, uint64_t tile_stride) {
    __shared__ unsigned long long smem[33];
    const uint64_t y = blockIdx.y;
    const uint64_t i = (uint64_t)blockIdx.x * kScanTile + threadIdx.x;
    unsigned long long v = (i < nb) ? cnt[y * stride + i] : 0ull;
    unsigned long long total;
    block_exclusive_scan64_1024(v, smem, &total);
    if (threadIdx.x == 0) tile_sums[y * tile_stride + blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) tile_scan_kernel(const unsigned long long* __restrict__ cnt,
                                                         const unsigned long long* __restrict__ tile_sums,
                                                         unsigned long long* __restrict__ pref,
                                                         unsigned long long* __restrict__ totals, uint64_t nb,
                                                         uint64_t stride, uint64_t tile_stride) {
    __shared__ unsigned long long smem[33];
    const uint64_t y = blockIdx.y;
    unsigned long long part = 0;
    for (uint32_t t = threadIdx.x; t < blockIdx.x; t += kScanTile) part += tile_sums[y * tile_stride + t];
    unsigned long long offset;
    block_exclusive_scan64_1024(part, smem, &offset);
    const uint64_t i = (uint64_t)blockIdx.x * kScanTile + threadIdx.x;
    unsigned long long v = (i < nb) ? cnt[y * stride + i] : 0ull;
    unsigned long long total;
    unsigned long long ex = block_exclusive_scan64_1024(v, smem, &total);
    if (i < nb) pref[y * stride + i] = offset + ex;
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) totals[y] = offset + total;
}

}  // namespace

slimdp_status launch_block_scan(const unsigned long long* cnt, unsigned long long* pref,
                                unsigned long long* tile_sums, unsigned long long* totals, uint64_t nb,
                                uint32_t batch, uint64_t stride, uint64_t tile_stride, cudaStream_t st) {
    const uint32_t tiles = (uint32_t)((nb + kScanTile - 1) / kScanTile);
    dim3 grid(tiles, batch);
    if (!prefer_max_shared(tile_sum_kernel) || !prefer_max_shared(tile_scan_kernel)) return SLIMDP_ERR_CUDA;
    tile_sum_kernel<<<grid, 1024, 0, st>>>(cnt, tile_sums, nb, stride, tile_stride);
    tile_scan_kernel<<<grid, 1024, 0, st>>>(cnt, tile_sums, pref, totals, nb, stride, tile_stride);
    SLIMDP_LAUNCHED(2);
    return SLIMDP_OK;
}

}  // namespace slimdp
