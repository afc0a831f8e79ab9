// The exported C ABI: argument validation, workspace sizing, and the order
// of kernel launches for each call.  No step of the round runs on the host.
#include <math.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "common.cuh"
#include "layout.cuh"

namespace slimdp {

slimdp_status launch_score(const float* w, const PtrArray<const float>& g, uint32_t K, float c, uint64_t n,
                           float* S, bool vec, cudaStream_t st);
slimdp_status launch_select(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx, void* core_aux,
                            void* ws, cudaStream_t st);
slimdp_status launch_explore(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                             uint32_t first_worker, uint32_t workers, uint32_t round,
                             const PtrArray<uint32_t>& out, void* ws, cudaStream_t st);
slimdp_status launch_gather(const PtrArray<const float>& src, bool same_src, uint32_t workers,
                            const uint32_t* core_idx, uint64_t k_core, const PtrArray<const uint32_t>& exp,
                            uint64_t k_exp, const PtrArray<float>& out, cudaStream_t st);
slimdp_status launch_merge(float* w, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                           const PtrArray<const uint32_t>& exp, uint64_t k_exp, const PtrArray<const float>& val,
                           float eta, cudaStream_t st);

static std::atomic<unsigned long long> g_launches{0};

void count_launches(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

slimdp_status launch_exchange(float* w, uint64_t n, uint32_t K, const PtrArray<const float>& delta,
                              const uint32_t* core_idx, uint64_t k_core, const PtrArray<const uint32_t>& exp,
                              uint64_t k_exp, float eta, const PtrArray<float>& val, const PtrArray<float>& pulled,
                              const uint32_t* ranks, uint64_t rank_stride, const uint32_t* core_bitmap,
                              const uint32_t* core_dir, int32_t* explore_status, cudaStream_t st);
bool exchange_takes_ranks(uint64_t n, uint64_t k_exp);

slimdp_status launch_explore_parts(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                                   uint32_t first_worker, uint32_t workers, uint32_t round,
                                   const PtrArray<uint32_t>& out, void* ws, int parts, bool lean, cudaStream_t st);
bool score_select_fusable(uint64_t n, uint64_t k_core, bool vec);
slimdp_status launch_score_select(const float* w, const PtrArray<const float>& g, uint32_t K, float c, uint64_t n,
                                  float* scores, uint64_t k_core, uint32_t* core_idx, void* core_aux, void* ws,
                                  cudaEvent_t mark_begin, cudaEvent_t mark_end, cudaStream_t gate_stream,
                                  cudaEvent_t gate_fork, cudaEvent_t gate_join, slimdp_status (*after_pass)(void*),
                                  void* after_arg, cudaEvent_t pass_ready, cudaStream_t st);

slimdp_status launch_explore_static(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                                    uint32_t worker, uint32_t round, uint32_t* exp_idx, int32_t* status_out,
                                    cudaStream_t st);

slimdp_status launch_dense_merge_score(float* w, const PtrArray<const float>& g, uint32_t K, float eta, float c,
                                       uint64_t n, float* S, bool vec, cudaStream_t st);
slimdp_status launch_worker_merge(const PtrArray<float>& w_local, uint32_t workers, const uint32_t* core_idx,
                                  uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                                  const PtrArray<const float>& pulled, cudaStream_t st);

slimdp_status launch_signature(const uint32_t* keys, uint64_t count, unsigned long long* sig, cudaStream_t st);

int sm_count() {
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return -1;
        cached[dev] = v;
    }
    return cached[dev];
}

namespace {

constexpr uint64_t kMaxN = 0xFFFFFFFFull;   // indices are uint32_t

bool n_ok(uint64_t n) { return n >= 1 && n <= kMaxN; }
bool k_ok(uint32_t K) { return K >= 1 && K <= SLIMDP_MAX_WORKERS; }

template <typename T>
bool fill(PtrArray<T>& dst, T* const* src, uint32_t count, bool need, size_t align) {
    memset(&dst, 0, sizeof(dst));
    if (src == nullptr) return !need;
    for (uint32_t k = 0; k < count; ++k) {
        if (need && (src[k] == nullptr || (reinterpret_cast<uintptr_t>(src[k]) & (align - 1)) != 0)) return false;
        dst.p[k] = src[k];
    }
    return true;
}

bool sets_ok(uint64_t n, uint64_t k_core, uint64_t k_exp) {
    return n_ok(n) && k_core <= n && k_exp <= n - k_core;
}

}  // namespace
}  // namespace slimdp

using namespace slimdp;

extern "C" {

const char* slimdp_status_string(slimdp_status s) {
    switch (s) {
        case SLIMDP_OK: return "ok";
        case SLIMDP_ERR_INVALID_ARG: return "invalid argument";
        case SLIMDP_ERR_WORKSPACE: return "workspace too small";
        case SLIMDP_ERR_CUDA: return "CUDA error";
        case SLIMDP_ERR_INTERNAL: return "device-side consistency check failed";
        case SLIMDP_ERR_UNSUPPORTED: return "unsupported";
        default: return "unknown status";
    }
}

size_t slimdp_core_aux_dir_offset(uint64_t n) {
    if (!n_ok(n)) return 0;
    return align_up(num_blocks(n) * kWordsPerBlock * 4, 256);
}

size_t slimdp_core_aux_bytes(uint64_t n) {
    if (!n_ok(n)) return 0;
    return slimdp_core_aux_dir_offset(n) + align_up((num_blocks(n) * kDirPerBlock + 1) * 4, 256);
}

size_t slimdp_select_workspace_bytes(uint64_t n) {
    if (!n_ok(n)) return 0;
    return select_ws_layout(nullptr, n).bytes;
}

size_t slimdp_explore_workspace_bytes(uint64_t n, uint64_t k_exp, uint32_t num_workers) {
    if (!n_ok(n) || k_exp > n || !k_ok(num_workers)) return 0;
    return explore_ws_layout(nullptr, n, k_exp, num_workers).bytes;
}

size_t slimdp_workspace_bytes(uint64_t n, uint64_t k_exp, uint32_t K) {
    const size_t a = slimdp_select_workspace_bytes(n), b = slimdp_explore_workspace_bytes(n, k_exp, K);
    if (a == 0 || b == 0) return 0;
    return a > b ? a : b;
}

slimdp_status slimdp_score(const float* w, const float* const* grads, uint32_t K, float c, uint64_t n,
                           float* scores, void* stream) {
    if (!n_ok(n) || !k_ok(K) || !w || !grads || !scores || !isfinite(c)) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(w) || !aligned4(scores)) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> g;
    if (!fill<const float>(g, grads, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    bool vec = aligned16(w) && aligned16(scores);
    for (uint32_t k = 0; k < K; ++k) vec = vec && aligned16(g.p[k]);
    return launch_score(w, g, K, c, n, scores, vec, (cudaStream_t)stream);
}

slimdp_status slimdp_select_core(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx,
                                 void* core_aux, void* ws, size_t ws_bytes, void* stream) {
    if (!n_ok(n) || k_core > n || !scores || !core_aux || !ws) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && !core_idx) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(scores) || !aligned16(core_aux) || !aligned16(ws) || (core_idx && !aligned16(core_idx)))
        return SLIMDP_ERR_INVALID_ARG;
    if (ws_bytes < slimdp_select_workspace_bytes(n)) return SLIMDP_ERR_WORKSPACE;
    return launch_select(scores, n, k_core, core_idx, core_aux, ws, (cudaStream_t)stream);
}

slimdp_status slimdp_sample_explore_batched(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp,
                                            uint64_t seed, uint32_t first_worker, uint32_t num_workers,
                                            uint32_t round, uint32_t* const* exp_idx, void* ws, size_t ws_bytes,
                                            void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(num_workers) || !core_aux || !ws) return SLIMDP_ERR_INVALID_ARG;
    if ((uint64_t)first_worker + num_workers > 0x100000000ull) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned16(core_aux) || !aligned16(ws)) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<uint32_t> out;
    if (!fill<uint32_t>(out, exp_idx, num_workers, k_exp > 0, 16)) return SLIMDP_ERR_INVALID_ARG;
    if (ws_bytes < slimdp_explore_workspace_bytes(n, k_exp, num_workers)) return SLIMDP_ERR_WORKSPACE;
    return launch_explore(core_aux, n, k_core, k_exp, seed, first_worker, num_workers, round, out, ws,
                          (cudaStream_t)stream);
}

slimdp_status slimdp_sample_explore(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp,
                                    uint64_t seed, uint32_t worker, uint32_t round, uint32_t* exp_idx, void* ws,
                                    size_t ws_bytes, void* stream) {
    uint32_t* one[1] = {exp_idx};
    return slimdp_sample_explore_batched(core_aux, n, k_core, k_exp, seed, worker, 1, round, one, ws, ws_bytes,
                                         stream);
}

slimdp_status slimdp_sample_explore_static(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp,
                                           uint64_t seed, uint32_t worker, uint32_t round, uint32_t* exp_idx,
                                           int32_t* status, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !core_aux || !aligned16(core_aux)) return SLIMDP_ERR_INVALID_ARG;
    if (k_exp > 0 && (!exp_idx || !aligned16(exp_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (status && !aligned4(status)) return SLIMDP_ERR_INVALID_ARG;
    if (n > SLIMDP_STATIC_MAX_N || k_exp > SLIMDP_STATIC_MAX_K_EXP) return SLIMDP_ERR_UNSUPPORTED;
    return launch_explore_static(core_aux, n, k_core, k_exp, seed, worker, round, exp_idx, status,
                                 (cudaStream_t)stream);
}

static slimdp_status gather_common(const float* const* srcs, bool same_src, const float* src0, uint32_t K,
                                   uint64_t n, const uint32_t* core_idx, uint64_t k_core,
                                   const uint32_t* const* exp_idx, uint64_t k_exp, float* const* out, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K)) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned16(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> src;
    PtrArray<const uint32_t> exp;
    PtrArray<float> dst;
    if (same_src) {
        if (!src0 || !aligned4(src0)) return SLIMDP_ERR_INVALID_ARG;
        memset(&src, 0, sizeof(src));
        for (uint32_t k = 0; k < K; ++k) src.p[k] = src0;
    } else if (!fill<const float>(src, srcs, K, true, 4)) {
        return SLIMDP_ERR_INVALID_ARG;
    }
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 16)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(dst, out, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp == 0) return SLIMDP_OK;
    return launch_gather(src, same_src, K, core_idx, k_core, exp, k_exp, dst, (cudaStream_t)stream);
}

slimdp_status slimdp_pack_batched(const float* const* deltas, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                  uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                  float* const* val, void* stream) {
    if (!deltas) return SLIMDP_ERR_INVALID_ARG;
    return gather_common(deltas, false, nullptr, K, n, core_idx, k_core, exp_idx, k_exp, val, stream);
}

slimdp_status slimdp_pack(const float* delta, uint64_t n, const uint32_t* core_idx, uint64_t k_core,
                          const uint32_t* exp_idx, uint64_t k_exp, float* val, void* stream) {
    const uint32_t* e[1] = {exp_idx};
    float* o[1] = {val};
    return gather_common(nullptr, true, delta, 1, n, core_idx, k_core, e, k_exp, o, stream);
}

slimdp_status slimdp_pull_batched(const float* w_global, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                  uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                  float* const* out, void* stream) {
    return gather_common(nullptr, true, w_global, K, n, core_idx, k_core, exp_idx, k_exp, out, stream);
}

slimdp_status slimdp_pull(const float* w_global, uint64_t n, const uint32_t* core_idx, uint64_t k_core,
                          const uint32_t* exp_idx, uint64_t k_exp, float* out, void* stream) {
    const uint32_t* e[1] = {exp_idx};
    float* o[1] = {out};
    return gather_common(nullptr, true, w_global, 1, n, core_idx, k_core, e, k_exp, o, stream);
}

slimdp_status slimdp_merge(float* w_global, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                           const uint32_t* const* exp_idx, uint64_t k_exp, const float* const* val, float eta,
                           void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_global || !aligned4(w_global) || !isfinite(eta))
        return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned16(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const uint32_t> exp;
    PtrArray<const float> v;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 16)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const float>(v, val, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp == 0) return SLIMDP_OK;
    return launch_merge(w_global, n, K, core_idx, k_core, exp, k_exp, v, eta, (cudaStream_t)stream);
}

slimdp_status slimdp_exchange(float* w_global, uint64_t n, uint32_t K, const float* const* deltas,
                              const uint32_t* core_idx, uint64_t k_core, const uint32_t* const* exp_idx,
                              uint64_t k_exp, float eta, float* const* val, float* const* pulled, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_global || !aligned4(w_global) || !isfinite(eta))
        return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned16(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> d;
    PtrArray<const uint32_t> exp;
    PtrArray<float> v, o;
    if (!fill<const float>(d, deltas, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 16)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(v, val, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(o, pulled, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp == 0) return SLIMDP_OK;
    return launch_exchange(w_global, n, K, d, core_idx, k_core, exp, k_exp, eta, v, o, nullptr, 0, nullptr, nullptr,
                           nullptr, (cudaStream_t)stream);
}

slimdp_status slimdp_dense_merge_score(float* w_global, const float* const* grads, uint32_t K, float eta, float c,
                                       uint64_t n, float* scores, void* stream) {
    if (!n_ok(n) || !k_ok(K) || !w_global || !grads || !isfinite(c) || !isfinite(eta)) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(w_global) || (scores && !aligned4(scores))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> g;
    if (!fill<const float>(g, grads, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    bool vec = aligned16(w_global) && (!scores || aligned16(scores));
    for (uint32_t k = 0; k < K; ++k) vec = vec && aligned16(g.p[k]);
    return launch_dense_merge_score(w_global, g, K, eta, c, n, scores, vec, (cudaStream_t)stream);
}

slimdp_status slimdp_worker_merge_batched(float* const* w_local, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                          uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                          const float* const* pulled, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_local) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned16(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<float> w;
    PtrArray<const uint32_t> exp;
    PtrArray<const float> v;
    if (!fill<float>(w, w_local, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 16)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const float>(v, pulled, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    return launch_worker_merge(w, K, core_idx, k_core, exp, k_exp, v, (cudaStream_t)stream);
}

slimdp_status slimdp_core_signature(const uint32_t* keys, uint64_t count, uint64_t* signature, void* stream) {
    if (count > kMaxN || !signature || (reinterpret_cast<uintptr_t>(signature) & 7u) != 0) return SLIMDP_ERR_INVALID_ARG;
    if (count > 0 && (!keys || !aligned4(keys))) return SLIMDP_ERR_INVALID_ARG;
    return launch_signature(keys, count, reinterpret_cast<unsigned long long*>(signature), (cudaStream_t)stream);
}

size_t slimdp_wire_bytes(uint64_t k_core, uint64_t k_exp) { return (size_t)(4 * k_core + 8 * k_exp + 8); }

uint64_t slimdp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

slimdp_status slimdp_read_status(const void* ws, void* stream) {
    if (!ws) return SLIMDP_ERR_INVALID_ARG;
    int32_t s = 0;
    if (cudaMemcpyAsync(&s, ws, sizeof(s), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return SLIMDP_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return SLIMDP_ERR_CUDA;
    return (s == SLIMDP_OK) ? SLIMDP_OK : SLIMDP_ERR_INTERNAL;
}

// ---- whole round on device buffers ----------------------------------------
//
// The round's steps form a small graph rather than a chain.  The chain that
// decides the round's time (sampling, the pass over all parameters, the
// threshold, the core, the explorers' indices, the exchange) runs on a stream
// of the highest priority that the library owns, one per device.  The
// explorer's ranks depend on the sizes alone: they are computed and sorted on
// a second stream of the lowest priority, released when the pass starts, in the
// part of each SM that the pass leaves free.  Whenever a kernel of the chain
// becomes ready its CTAs are placed ahead of those of the rank kernels.  The
// caller's stream only forks into the chain at the start of the call and
// waits for it at the end (chain_done), on every path through the call.
// Scoring is folded into the selection's one pass over all parameters, so the
// scores are never written unless the selection has to fall back to its full path.

namespace {
struct SideStream {
    cudaStream_t chain = nullptr, ranks = nullptr, gate = nullptr;
    cudaEvent_t fork = nullptr, pass_ready = nullptr, ranks_done = nullptr, chain_done = nullptr, gate_fork = nullptr,
                gate_join = nullptr;
    bool ready = false;
};
std::mutex g_side_mutex;
thread_local cudaEvent_t t_mark_begin = nullptr, t_mark_end = nullptr;
SideStream g_side[64];

SideStream* side_stream_locked() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    SideStream& s = g_side[dev];
    if (!s.ready) {
        int lo = 0, hi = 0;   // numerically, hi <= lo: hi is the highest priority
        if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithPriority(&s.chain, cudaStreamNonBlocking, hi) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithPriority(&s.gate, cudaStreamNonBlocking, hi) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithPriority(&s.ranks, cudaStreamNonBlocking, lo) != cudaSuccess) return nullptr;
        cudaEvent_t* ev[6] = {&s.fork, &s.pass_ready, &s.ranks_done, &s.chain_done, &s.gate_fork, &s.gate_join};
        for (auto e : ev)
            if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        s.ready = true;
    }
    return &s;
}
}  // namespace

slimdp_status slimdp_round(float* w_global, const float* const* grads, uint32_t K, uint64_t n, float c,
                           uint64_t k_core, uint64_t k_exp, uint64_t seed, uint32_t round, float eta, float* scores,
                           uint32_t* core_idx, void* core_aux, uint32_t* const* exp_idx, float* const* val,
                           float* const* pulled, void* select_ws, size_t select_ws_bytes, void* explore_ws,
                           size_t explore_ws_bytes, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_global || !grads || !scores || !core_aux || !select_ws ||
        !explore_ws || !isfinite(c) || !isfinite(eta))
        return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(w_global) || !aligned4(scores) || !aligned16(core_aux) || !aligned16(select_ws) ||
        !aligned16(explore_ws))
        return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned16(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> g;
    PtrArray<uint32_t> exp_out;
    PtrArray<const uint32_t> exp_in;
    PtrArray<float> v, o;
    if (!fill<const float>(g, grads, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<uint32_t>(exp_out, exp_idx, K, k_exp > 0, 16)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(v, val, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(o, pulled, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    memset(&exp_in, 0, sizeof(exp_in));
    for (uint32_t k = 0; k < K; ++k) exp_in.p[k] = exp_out.p[k];
    if (select_ws_bytes < slimdp_select_workspace_bytes(n)) return SLIMDP_ERR_WORKSPACE;
    if (explore_ws_bytes < slimdp_explore_workspace_bytes(n, k_exp, K)) return SLIMDP_ERR_WORKSPACE;
    {
        const char* a = static_cast<const char*>(select_ws);
        const char* b = static_cast<const char*>(explore_ws);
        if (a < b + explore_ws_bytes && b < a + select_ws_bytes) return SLIMDP_ERR_INVALID_ARG;
    }
    bool vec = aligned16(w_global) && aligned16(scores);
    for (uint32_t k = 0; k < K; ++k) vec = vec && aligned16(g.p[k]);
    const bool fusable = score_select_fusable(n, k_core, vec);

    cudaStream_t st = (cudaStream_t)stream;
    std::lock_guard<std::mutex> lock(g_side_mutex);
    SideStream* side = side_stream_locked();
    if (!side) return SLIMDP_ERR_CUDA;
    cudaStream_t ch = side->chain, rk = side->ranks;

    if (cudaEventRecord(side->fork, st) != cudaSuccess) return SLIMDP_ERR_CUDA;
    if (cudaStreamWaitEvent(ch, side->fork, 0) != cudaSuccess) return SLIMDP_ERR_CUDA;
    // From here on the chain is joined back into `st` whatever happens.
    slimdp_status rc = SLIMDP_OK;
    auto step = [&](slimdp_status s) {
        if (rc == SLIMDP_OK) rc = s;
    };
    auto cuda = [&](cudaError_t e) { step(e == cudaSuccess ? SLIMDP_OK : SLIMDP_ERR_CUDA); };
    cudaEvent_t mark0 = t_mark_begin, mark1 = t_mark_end;
    t_mark_begin = t_mark_end = nullptr;

    // ranks stream: ranks of every worker's explorer, sorted (they need the sizes only).  The stream
    // waits for `after`, an event of the chain: the moment from which the ranks may take SM room.
    struct RankWork {
        const void* core_aux;
        uint64_t n, k_core, k_exp, seed;
        uint32_t K, round;
        const PtrArray<uint32_t>* out;
        void* ws;
        cudaStream_t rk;
        cudaEvent_t after, done;
        bool lean;
    } rank_work{core_aux, n, k_core, k_exp, seed, K, round, &exp_out, explore_ws, rk, side->fork, side->ranks_done,
                false};
    auto enqueue_ranks = [](void* p) -> slimdp_status {
        const RankWork& s = *static_cast<const RankWork*>(p);
        if (cudaStreamWaitEvent(s.rk, s.after, 0) != cudaSuccess) return SLIMDP_ERR_CUDA;
        const slimdp_status r = launch_explore_parts(s.core_aux, s.n, s.k_core, s.k_exp, s.seed, 0, s.K, s.round,
                                                     *s.out, s.ws, 1, s.lean, s.rk);
        if (cudaEventRecord(s.done, s.rk) != cudaSuccess) return SLIMDP_ERR_CUDA;
        return r;
    };
    // chain: the core, scored and selected in one pass where sizes and alignment allow
    if (fusable) {
        rank_work.after = side->pass_ready;   // recorded by the call below just before its pass
        rank_work.lean = true;
        step(launch_score_select(w_global, g, K, c, n, scores, k_core, core_idx, core_aux, select_ws, mark0, mark1,
                                 side->gate, side->gate_fork, side->gate_join, enqueue_ranks, &rank_work,
                                 side->pass_ready, ch));
        // (if the call failed before it reached the hook, ranks_done keeps an earlier record: nothing to wait for)
    } else {
        step(enqueue_ranks(&rank_work));
        if (rc == SLIMDP_OK && mark0) cuda(cudaEventRecord(mark0, ch));
        if (rc == SLIMDP_OK) step(launch_score(w_global, g, K, c, n, scores, vec, ch));
        if (rc == SLIMDP_OK && mark1) cuda(cudaEventRecord(mark1, ch));
        if (rc == SLIMDP_OK) step(launch_select(scores, n, k_core, core_idx, core_aux, select_ws, ch));
    }
    // chain: explorer indices from the sorted ranks and the core, then the exchange; where the
    // exchange's warp ranges line up with the core's directory it computes the indices itself
    cuda(cudaStreamWaitEvent(ch, side->ranks_done, 0));
    if (exchange_takes_ranks(n, k_exp)) {
        const ExploreWs EL = explore_ws_layout(explore_ws, n, k_exp, K);
        if (rc == SLIMDP_OK)
            step(launch_exchange(w_global, n, K, g, core_idx, k_core, exp_in, k_exp, eta, v, o, EL.rho, EL.rho_stride,
                                 reinterpret_cast<const uint32_t*>(core_aux),
                                 reinterpret_cast<const uint32_t*>(static_cast<const char*>(core_aux) +
                                                                   slimdp_core_aux_dir_offset(n)),
                                 &EL.hdr->status, ch));
    } else {
        if (rc == SLIMDP_OK)
            step(launch_explore_parts(core_aux, n, k_core, k_exp, seed, 0, K, round, exp_out, explore_ws, 2, false,
                                      ch));
        if (rc == SLIMDP_OK && k_core + k_exp > 0)
            step(launch_exchange(w_global, n, K, g, core_idx, k_core, exp_in, k_exp, eta, v, o, nullptr, 0, nullptr,
                                 nullptr, nullptr, ch));
    }
    if (cudaEventRecord(side->chain_done, ch) != cudaSuccess || cudaStreamWaitEvent(st, side->chain_done, 0) != cudaSuccess)
        step(SLIMDP_ERR_CUDA);
    return rc;
}

void slimdp_mark_dominant_kernel(void* begin_event, void* end_event) {
    t_mark_begin = (cudaEvent_t)begin_event;
    t_mark_end = (cudaEvent_t)end_event;
}

// ---- whole round on host buffers ------------------------------------------

namespace {
struct Arena {
    float* w;
    float* delta[SLIMDP_MAX_WORKERS];
    float* scores;
    uint32_t* core_idx;
    void* core_aux;
    void* select_ws;
    size_t select_ws_bytes;
    void* explore_ws;
    size_t explore_ws_bytes;
    uint32_t* exp_idx[SLIMDP_MAX_WORKERS];
    float* val[SLIMDP_MAX_WORKERS];
    float* pulled[SLIMDP_MAX_WORKERS];
    size_t bytes;
};

Arena arena_layout(void* base, uint64_t n, uint32_t K, uint64_t k_core, uint64_t k_exp) {
    char* p = reinterpret_cast<char*>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        char* r = p + off;
        off += align_up(bytes ? bytes : 1, 256);
        return r;
    };
    Arena A;
    memset(&A, 0, sizeof(A));
    const uint64_t m = k_core + k_exp;
    A.w = reinterpret_cast<float*>(take(n * 4));
    for (uint32_t k = 0; k < K; ++k) A.delta[k] = reinterpret_cast<float*>(take(n * 4));
    A.scores = reinterpret_cast<float*>(take(n * 4));
    A.core_idx = reinterpret_cast<uint32_t*>(take(k_core * 4));
    A.core_aux = take(slimdp_core_aux_bytes(n));
    A.select_ws_bytes = slimdp_select_workspace_bytes(n);
    A.select_ws = take(A.select_ws_bytes);
    A.explore_ws_bytes = slimdp_explore_workspace_bytes(n, k_exp, K);
    A.explore_ws = take(A.explore_ws_bytes);
    for (uint32_t k = 0; k < K; ++k) A.exp_idx[k] = reinterpret_cast<uint32_t*>(take(k_exp * 4));
    for (uint32_t k = 0; k < K; ++k) A.val[k] = reinterpret_cast<float*>(take(m * 4));
    for (uint32_t k = 0; k < K; ++k) A.pulled[k] = reinterpret_cast<float*>(take(m * 4));
    A.bytes = off;
    return A;
}
}  // namespace

size_t slimdp_round_arena_bytes(uint64_t n, uint32_t K, uint64_t k_core, uint64_t k_exp) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K)) return 0;
    return arena_layout(nullptr, n, K, k_core, k_exp).bytes;
}

slimdp_status slimdp_round_host(float* w_host, const float* const* grads_host, uint32_t K, uint64_t n, float c,
                                uint64_t k_core, uint64_t k_exp, uint64_t seed, uint32_t round, float eta,
                                uint32_t* core_idx_host, uint32_t* const* exp_idx_host, float* const* pulled_host,
                                void* arena, size_t arena_bytes, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_host || !grads_host || !arena || !isfinite(c) || !isfinite(eta))
        return SLIMDP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && !core_idx_host) return SLIMDP_ERR_INVALID_ARG;
    if (k_exp > 0 && !exp_idx_host) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp > 0 && !pulled_host) return SLIMDP_ERR_INVALID_ARG;
    for (uint32_t k = 0; k < K; ++k) {
        if (!grads_host[k]) return SLIMDP_ERR_INVALID_ARG;
        if (k_exp > 0 && !exp_idx_host[k]) return SLIMDP_ERR_INVALID_ARG;
        if (k_core + k_exp > 0 && !pulled_host[k]) return SLIMDP_ERR_INVALID_ARG;
    }
    if (arena_bytes < slimdp_round_arena_bytes(n, K, k_core, k_exp)) return SLIMDP_ERR_WORKSPACE;
    const Arena A = arena_layout(arena, n, K, k_core, k_exp);
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t m = k_core + k_exp;
#define SLIMDP_CUDA(x) \
    if ((x) != cudaSuccess) return SLIMDP_ERR_CUDA
#define SLIMDP_TRY(x)                   \
    do {                                \
        slimdp_status s_ = (x);         \
        if (s_ != SLIMDP_OK) return s_; \
    } while (0)
    SLIMDP_CUDA(cudaMemcpyAsync(A.w, w_host, n * 4, cudaMemcpyHostToDevice, st));
    for (uint32_t k = 0; k < K; ++k)
        SLIMDP_CUDA(cudaMemcpyAsync(A.delta[k], grads_host[k], n * 4, cudaMemcpyHostToDevice, st));
    SLIMDP_TRY(slimdp_round(A.w, A.delta, K, n, c, k_core, k_exp, seed, round, eta, A.scores, A.core_idx, A.core_aux,
                            A.exp_idx, A.val, A.pulled, A.select_ws, A.select_ws_bytes, A.explore_ws,
                            A.explore_ws_bytes, stream));
    SLIMDP_CUDA(cudaMemcpyAsync(w_host, A.w, n * 4, cudaMemcpyDeviceToHost, st));
    if (k_core) SLIMDP_CUDA(cudaMemcpyAsync(core_idx_host, A.core_idx, k_core * 4, cudaMemcpyDeviceToHost, st));
    for (uint32_t k = 0; k < K; ++k) {
        if (k_exp) SLIMDP_CUDA(cudaMemcpyAsync(exp_idx_host[k], A.exp_idx[k], k_exp * 4, cudaMemcpyDeviceToHost, st));
        if (m) SLIMDP_CUDA(cudaMemcpyAsync(pulled_host[k], A.pulled[k], m * 4, cudaMemcpyDeviceToHost, st));
    }
    SLIMDP_TRY(slimdp_read_status(A.select_ws, stream));
    return slimdp_read_status(A.explore_ws, stream);
#undef SLIMDP_CUDA
#undef SLIMDP_TRY
}

}  // extern "C"
