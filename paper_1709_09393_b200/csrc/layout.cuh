// Workspace layouts (host-side pointer arithmetic only).
#pragma once

#include "common.cuh"

namespace slimdp {

struct SelectWs {
    WsHeader* hdr;
    uint32_t* hist;                 // 3 x 4096 bins
    uint32_t* G;                    // greater-than-threshold bitmap, nb * 32 words
    uint32_t* E;                    // equal-to-threshold bitmap, nb * 32 words
    unsigned long long* cnt;        // per block: #greater | #equal << 32
    unsigned long long* pref;       // exclusive scan of cnt
    unsigned long long* tile_sums;  // per scan tile
    unsigned long long* totals;     // [1]
    size_t bytes;
};

inline SelectWs select_ws_layout(void* ws, uint64_t n) {
    const uint64_t nb = num_blocks(n), nt = num_scan_tiles(n);
    char* p = reinterpret_cast<char*>(ws);
    size_t off = 0;
    SelectWs L;
    auto take = [&](size_t bytes) {
        char* r = p + off;
        off += align_up(bytes, 256);
        return r;
    };
    L.hdr = reinterpret_cast<WsHeader*>(take(sizeof(WsHeader)));
    L.hist = reinterpret_cast<uint32_t*>(take(3 * 4096 * sizeof(uint32_t)));
    L.G = reinterpret_cast<uint32_t*>(take(nb * kWordsPerBlock * 4));
    L.E = reinterpret_cast<uint32_t*>(take(nb * kWordsPerBlock * 4));
    L.cnt = reinterpret_cast<unsigned long long*>(take(nb * 8));
    L.pref = reinterpret_cast<unsigned long long*>(take(nb * 8));
    L.tile_sums = reinterpret_cast<unsigned long long*>(take(nt * 8));
    L.totals = reinterpret_cast<unsigned long long*>(take(8));
    L.bytes = off;
    return L;
}

struct ExploreWs {
    WsHeader* hdr;
    uint32_t* round_keys;           // 12 words per worker
    uint32_t* marks;                // per worker: nb * 32 words
    unsigned long long* cnt;        // per worker: nb
    unsigned long long* pref;       // per worker: nb
    unsigned long long* tile_sums;  // per worker: nt
    unsigned long long* totals;     // per worker: 1
    uint64_t mark_stride;           // words between workers' bitmaps
    uint64_t cnt_stride;            // entries between workers' counter rows
    uint64_t tile_stride;
    size_t bytes;
};

inline ExploreWs explore_ws_layout(void* ws, uint64_t n, uint32_t workers) {
    const uint64_t nb = num_blocks(n), nt = num_scan_tiles(n);
    char* p = reinterpret_cast<char*>(ws);
    size_t off = 0;
    ExploreWs L;
    auto take = [&](size_t bytes) {
        char* r = p + off;
        off += align_up(bytes, 256);
        return r;
    };
    L.mark_stride = align_up(nb * kWordsPerBlock, 64);
    L.cnt_stride = align_up(nb, 32);
    L.tile_stride = align_up(nt, 32);
    L.hdr = reinterpret_cast<WsHeader*>(take(sizeof(WsHeader)));
    L.round_keys = reinterpret_cast<uint32_t*>(take((size_t)workers * 12 * 4));
    L.marks = reinterpret_cast<uint32_t*>(take((size_t)workers * L.mark_stride * 4));
    L.cnt = reinterpret_cast<unsigned long long*>(take((size_t)workers * L.cnt_stride * 8));
    L.pref = reinterpret_cast<unsigned long long*>(take((size_t)workers * L.cnt_stride * 8));
    L.tile_sums = reinterpret_cast<unsigned long long*>(take((size_t)workers * L.tile_stride * 8));
    L.totals = reinterpret_cast<unsigned long long*>(take((size_t)workers * 8));
    L.bytes = off;
    return L;
}

}  // namespace slimdp
