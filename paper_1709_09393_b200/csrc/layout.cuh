// Workspace layouts (host-side pointer arithmetic only).
#pragma once

#include "common.cuh"

namespace slimdp {

struct SelectWs {
    WsHeader* hdr;
    uint32_t* hist;                 // 6 x 4096 bins: three passes over all keys, three over the candidates
    uint32_t* coarse_hist;          // 256 bins (top 8 key bits of the sampled keys)
    uint32_t* fine_hist;            // 2 x 1024 bins (top 18 key bits inside the two crossing coarse bins)
    uint32_t* coarse_incl;          // 256: samples in coarse bins >= c
    uint32_t* sample;               // 2^18 sampled keys
    uint32_t* G;                    // greater-than-threshold bitmap, nb * 32 words
    uint32_t* E;                    // equal-to-threshold bitmap, nb * 32 words
    unsigned long long* tile_sum;   // per 1024-parameter block: #greater | #equal << 32
    unsigned long long* super_pref; // per group of 64 blocks: their counts, then the counts below the group
    uint32_t* cand_key;             // keys inside the bracket
    uint32_t* cand_idx;             // and their parameter indices
    uint64_t cand_cap;              // entries in each candidate array
    size_t zero_bytes;              // header, histograms and tile counts, contiguous, cleared at the start of every call
    size_t bytes;
};

constexpr uint32_t kEmitTile = 1;     // 1024-parameter blocks per counter of the selection's members (see select_dev.cuh)

inline SelectWs select_ws_layout(void* ws, uint64_t n) {
    const uint64_t nb = num_blocks(n);
    char* p = reinterpret_cast<char*>(ws);
    size_t off = 0;
    SelectWs L;
    auto take = [&](size_t bytes) {
        char* r = p + off;
        off += align_up(bytes, 256);
        return r;
    };
    L.hdr = reinterpret_cast<WsHeader*>(take(sizeof(WsHeader)));
    L.hist = reinterpret_cast<uint32_t*>(take(6 * 4096 * sizeof(uint32_t)));
    L.coarse_hist = reinterpret_cast<uint32_t*>(take(256 * sizeof(uint32_t)));
    L.fine_hist = reinterpret_cast<uint32_t*>(take(2 * 1024 * sizeof(uint32_t)));
    L.tile_sum = reinterpret_cast<unsigned long long*>(take(((nb + kEmitTile - 1) / kEmitTile) * 8));
    L.zero_bytes = off;
    L.super_pref = reinterpret_cast<unsigned long long*>(take((((nb + kEmitTile - 1) / kEmitTile + 63) / 64) * 8));
    L.coarse_incl = reinterpret_cast<uint32_t*>(take(256 * sizeof(uint32_t)));
    L.sample = reinterpret_cast<uint32_t*>(take((size_t)(1u << kSampleBits) * sizeof(uint32_t)));
    L.G = reinterpret_cast<uint32_t*>(take(nb * kWordsPerBlock * 4));
    L.E = reinterpret_cast<uint32_t*>(take(nb * kWordsPerBlock * 4));
    L.cand_cap = (n >= kBracketMinN) ? (n / 16 > 65536 ? n / 16 : 65536) : 0;
    L.cand_key = reinterpret_cast<uint32_t*>(take(L.cand_cap * 4 + 16));
    L.cand_idx = reinterpret_cast<uint32_t*>(take(L.cand_cap * 4 + 16));
    L.bytes = off;
    return L;
}

// Staging area of the one-call round.  While the pass over all parameters has a parameter's K
// update values at hand (the parameter is certainly in the core, or a candidate for it), it sets
// them aside here, so that the exchange streams them instead of gathering them again.  Chunks of
// kStageChunk entries, each chunk K + 1 arrays of kStageChunk words (parameter index, then one array
// per worker); a warp of the pass fills its chunks front to back and takes fresh chunks on demand,
// so fill[c] entries of chunk c are valid and the chunks are in no particular order.
struct StageArea {
    uint32_t* fill;        // per chunk: valid entries (cleared at the start of every call)
    uint32_t* chunks;      // chunk c at chunks + c * (K + 1) * kStageChunk
    uint64_t max_chunks;
    size_t fill_bytes;
    size_t bytes;
};

// Chunks that hold every parameter that may be staged when the bracket holds (fewer than k_core
// certain ones, at most cand_cap candidates) plus, per warp of the pass, the chunk it is filling
// and the one it has in reserve.
inline StageArea stage_layout(void* base, uint64_t n, uint32_t K, uint64_t k_core, uint32_t pass_warps) {
    StageArea A;
    const uint64_t cand_cap = (n >= kBracketMinN) ? (n / 16 > 65536 ? n / 16 : 65536) : 0;
    A.max_chunks = (k_core + cand_cap + kStageChunk - 1) / kStageChunk + 2ull * pass_warps + 1;
    A.fill_bytes = align_up(A.max_chunks * 4, 256);
    A.fill = reinterpret_cast<uint32_t*>(base);
    A.chunks = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(base) + A.fill_bytes);
    A.bytes = A.fill_bytes + A.max_chunks * (size_t)(K + 1) * kStageChunk * 4;
    return A;
}

// What slimdp_round hands the exchange about a filled staging area.
struct ExchangeStage {
    const uint32_t* fill;
    const uint32_t* chunks;
    uint32_t max_chunks;
    WsHeader* select_hdr;
    uint32_t cand_cap;
};

struct ExploreWs {
    WsHeader* hdr;
    uint32_t* rho;                  // per worker: pi(j), j < k_exp; later the same ranks in ascending order
    uint32_t* sorted;               // per worker: the ranks grouped by bucket
    unsigned long long* cnt;        // per worker: ranks per bucket
    uint32_t* cursor;               // per worker: scatter cursors per bucket
    uint32_t* ticket;               // per worker: CTAs of the rank step that have finished
    uint32_t* cta_hist;             // per rank-step CTA: its chunk's ranks per bucket
    uint32_t* cell_group;           // per 4096 non-core ranks: the 64-parameter group that holds the cell's first rank
    unsigned long long* pref;       // per worker: exclusive scan of cnt
    unsigned long long* totals;     // per worker: 1
    uint64_t rho_stride;            // entries between workers' rank rows
    uint64_t cnt_stride;            // entries between workers' bucket rows
    size_t zero_bytes;              // cnt, cursor and ticket, contiguous, cleared before every call
    size_t bytes;
};

constexpr uint32_t kCellShift = 12;          // ranks per cell of the rank -> group table
constexpr uint64_t kMaxSmemBuckets = 8192;   // bucket histograms up to this size live in shared memory (32 KB)
constexpr uint64_t kMaxExploreCtas = 1024;   // rank / scatter CTAs over all workers of one call

// Upper bound on the number of rank buckets for any core size: buckets hold
// 2^13 .. 2^17 ranks, at least 2^16 once there are 2^25 non-core parameters.
inline uint64_t explore_max_buckets(uint64_t n) {
    const uint64_t big = (n + 65535) / 65536;
    return big > 1024 ? big : 1024;
}

inline ExploreWs explore_ws_layout(void* ws, uint64_t n, uint64_t k_exp, uint32_t workers) {
    char* p = reinterpret_cast<char*>(ws);
    size_t off = 0;
    ExploreWs L;
    auto take = [&](size_t bytes) {
        char* r = p + off;
        off += align_up(bytes ? bytes : 1, 256);
        return r;
    };
    L.rho_stride = align_up(k_exp, 64);
    L.cnt_stride = align_up(explore_max_buckets(n), 64);
    L.hdr = reinterpret_cast<WsHeader*>(take(sizeof(WsHeader)));
    L.rho = reinterpret_cast<uint32_t*>(take((size_t)workers * L.rho_stride * 4));
    L.sorted = reinterpret_cast<uint32_t*>(take((size_t)workers * L.rho_stride * 4));
    const size_t zero_begin = off;
    L.cnt = reinterpret_cast<unsigned long long*>(take((size_t)workers * L.cnt_stride * 8));
    L.cursor = reinterpret_cast<uint32_t*>(take((size_t)workers * L.cnt_stride * 4));
    L.ticket = reinterpret_cast<uint32_t*>(take((size_t)workers * 4));
    L.zero_bytes = off - zero_begin;
    L.pref = reinterpret_cast<unsigned long long*>(take((size_t)workers * L.cnt_stride * 8));
    L.totals = reinterpret_cast<unsigned long long*>(take((size_t)workers * 8));
    const uint64_t hist_buckets = explore_max_buckets(n) < kMaxSmemBuckets ? explore_max_buckets(n) : kMaxSmemBuckets;
    L.cta_hist = reinterpret_cast<uint32_t*>(take((size_t)kMaxExploreCtas * hist_buckets * 4));
    L.cell_group = reinterpret_cast<uint32_t*>(take(((n >> kCellShift) + 2) * 4));
    L.bytes = off;
    return L;
}

}  // namespace slimdp
