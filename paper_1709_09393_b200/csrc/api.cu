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
                            void* ws, bool emit, cudaStream_t st);
bool round_exchange_applies(uint64_t n, uint64_t k_exp);
slimdp_status launch_round_exchange(float* w, uint64_t n, uint32_t K, const PtrArray<const float>& delta,
                                    uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp, float eta,
                                    const PtrArray<float>& val, const PtrArray<float>& pulled, const uint32_t* ranks,
                                    uint64_t rank_stride, int32_t* explore_status, const uint32_t* G,
                                    const uint32_t* E, const unsigned long long* cnt,
                                    const unsigned long long* super_pref, WsHeader* sel_hdr, uint32_t* core_idx,
                                    uint32_t* core_bitmap, uint32_t* core_dir, cudaStream_t st);
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
                              const uint32_t* core_dir, int32_t* explore_status, const ExchangeStage* stage,
                              cudaStream_t st);
bool exchange_takes_ranks(uint64_t n, uint64_t k_exp);
size_t stage_bytes_for(uint64_t n, uint32_t K, uint64_t k_core);

slimdp_status launch_explore_parts(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                                   uint32_t first_worker, uint32_t workers, uint32_t round,
                                   const PtrArray<uint32_t>& out, void* ws, int parts, bool lean, cudaStream_t st);
bool score_select_fusable(uint64_t n, uint64_t k_core, uint32_t K, bool vec);
slimdp_status launch_score_select(const float* w, const PtrArray<const float>& g, uint32_t K, float c, uint64_t n,
                                  float* scores, uint64_t k_core, uint32_t* core_idx, void* core_aux, void* ws,
                                  cudaEvent_t mark_begin, cudaEvent_t mark_end, slimdp_status (*after_pass)(void*),
                                  void* after_arg, cudaEvent_t pass_ready, void* stage, size_t stage_bytes,
                                  bool* staged, bool emit, cudaStream_t st);

slimdp_status launch_explore_static(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp, uint64_t seed,
                                    uint32_t worker, uint32_t round, uint32_t* exp_idx, int32_t* status_out,
                                    cudaStream_t st);

slimdp_status launch_dense_merge_score(float* w, const PtrArray<const float>& g, uint32_t K, float eta, float c,
                                       uint64_t n, float* S, bool vec, cudaStream_t st);
slimdp_status launch_worker_merge(const PtrArray<float>& w_local, uint32_t workers, const uint32_t* core_idx,
                                  uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                                  const PtrArray<const float>& pulled, cudaStream_t st);

size_t seg_select_ws_bytes(uint64_t n, uint32_t segments);
slimdp_status launch_select_segmented(const float* scores, uint64_t n, const uint64_t* seg_off, const uint64_t* seg_k,
                                      uint32_t segments, uint64_t k_total, uint32_t* core_idx, void* core_aux,
                                      void* ws, cudaStream_t st);
slimdp_status launch_pack_q8(const PtrArray<const float>& delta, uint32_t K, const uint32_t* core_idx,
                             uint64_t k_core, const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                             const PtrArray<int8_t>& codes, const PtrArray<float>& scales, cudaStream_t st);
slimdp_status launch_merge_q8(float* w, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                              const PtrArray<const uint32_t>& exp, uint64_t k_exp,
                              const PtrArray<const int8_t>& codes, const PtrArray<const float>& scales, float eta,
                              cudaStream_t st);
slimdp_status launch_select_given(const float* scores, uint64_t n, uint32_t T, uint32_t ties, uint64_t k_shard,
                                  uint32_t* core_idx, void* core_aux, void* ws, cudaStream_t st);
slimdp_status launch_explore_shard(const void* core_aux, uint64_t n_shard, uint64_t k_core_shard,
                                   uint64_t noncore_total, uint64_t noncore_below, uint64_t k_exp, uint64_t seed,
                                   uint32_t worker, uint32_t round, uint32_t* exp_idx, uint64_t cap, uint32_t* count,
                                   void* ws, cudaStream_t st);
size_t explore_shard_ws_bytes(uint64_t n_shard, uint64_t noncore_total, uint64_t k_exp);
slimdp_status launch_shard_state_init(void* state, uint64_t k, cudaStream_t st);
slimdp_status launch_shard_hist(const float* scores, uint64_t n, uint32_t round, const void* state, uint64_t* hist,
                                cudaStream_t st);
slimdp_status launch_shard_resolve(const uint64_t* hist, uint32_t round, void* state, cudaStream_t st);
slimdp_status launch_shard_count(const float* scores, uint64_t n, const void* state, uint64_t* counts,
                                 cudaStream_t st);
slimdp_status launch_signature(const uint32_t* keys, uint64_t count, unsigned long long* sig, cudaStream_t st);
slimdp_status launch_wire_pack(const uint32_t* core_idx, uint64_t k_core, const uint32_t* exp_idx, uint64_t k_exp,
                               const float* val, const unsigned long long* sig, uint32_t worker, uint32_t round,
                               bool with_keys, void* msg, cudaStream_t st);
slimdp_status launch_wire_unpack(const void* msg, size_t msg_bytes, const unsigned long long* cached_sig,
                                 uint64_t k_core, uint64_t k_exp, uint32_t* core_idx, uint32_t* exp_idx, float* val,
                                 unsigned long long* sig_out, int32_t* status, cudaStream_t st);

int sm_count() {
    static std::atomic<int> cached[64];   // 0 = not asked yet; every thread that asks stores the same value
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    int v = cached[dev].load(std::memory_order_relaxed);
    if (v == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return -1;
        cached[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

namespace {

constexpr uint64_t kMaxN = 0xFFFFFFFFull;   // indices are uint32_t
constexpr uint64_t kFoldedExchangeMaxN = 1ull << 22;   // slimdp_round: up to here the exchange also does the emit's work

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

size_t slimdp_workspace_bytes(uint64_t n, uint32_t K, uint64_t k_core, uint64_t k_exp) {
    if (!sets_ok(n, k_core, k_exp)) return 0;
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
    if (!vec) {
        // all tensors off a 16-byte boundary by the same amount (slices of one allocation): the first
        // one to three parameters go through the scalar kernel, the rest is aligned
        const uintptr_t mis = reinterpret_cast<uintptr_t>(w) & 15u;
        bool same = (reinterpret_cast<uintptr_t>(scores) & 15u) == mis;
        for (uint32_t k = 0; k < K; ++k) same = same && (reinterpret_cast<uintptr_t>(g.p[k]) & 15u) == mis;
        const uint64_t head = (16u - mis) / 4u;
        if (same && n > head) {
            slimdp_status rc = launch_score(w, g, K, c, head, scores, false, (cudaStream_t)stream);
            if (rc != SLIMDP_OK) return rc;
            PtrArray<const float> g2 = g;
            for (uint32_t k = 0; k < K; ++k) g2.p[k] = g.p[k] + head;
            return launch_score(w + head, g2, K, c, n - head, scores + head, true, (cudaStream_t)stream);
        }
    }
    return launch_score(w, g, K, c, n, scores, vec, (cudaStream_t)stream);
}

slimdp_status slimdp_select_core(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx,
                                 void* core_aux, void* ws, size_t ws_bytes, void* stream) {
    if (!n_ok(n) || k_core > n || !scores || !core_aux || !ws) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && !core_idx) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(scores) || !aligned16(core_aux) || !aligned16(ws) || (core_idx && !aligned4(core_idx)))
        return SLIMDP_ERR_INVALID_ARG;
    if (ws_bytes < slimdp_select_workspace_bytes(n)) return SLIMDP_ERR_WORKSPACE;
    return launch_select(scores, n, k_core, core_idx, core_aux, ws, true, (cudaStream_t)stream);
}

slimdp_status slimdp_sample_explore_batched(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp,
                                            uint64_t seed, uint32_t first_worker, uint32_t num_workers,
                                            uint32_t round, uint32_t* const* exp_idx, void* ws, size_t ws_bytes,
                                            void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(num_workers) || !core_aux || !ws) return SLIMDP_ERR_INVALID_ARG;
    if ((uint64_t)first_worker + num_workers > 0x100000000ull) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned16(core_aux) || !aligned16(ws)) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<uint32_t> out;
    if (!fill<uint32_t>(out, exp_idx, num_workers, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
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
    if (k_exp > 0 && (!exp_idx || !aligned4(exp_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (status && !aligned4(status)) return SLIMDP_ERR_INVALID_ARG;
    if (n > SLIMDP_STATIC_MAX_N || k_exp > SLIMDP_STATIC_MAX_K_EXP) return SLIMDP_ERR_UNSUPPORTED;
    return launch_explore_static(core_aux, n, k_core, k_exp, seed, worker, round, exp_idx, status,
                                 (cudaStream_t)stream);
}

static slimdp_status gather_common(const float* const* srcs, bool same_src, const float* src0, uint32_t K,
                                   uint64_t n, const uint32_t* core_idx, uint64_t k_core,
                                   const uint32_t* const* exp_idx, uint64_t k_exp, float* const* out, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K)) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
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
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
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
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const uint32_t> exp;
    PtrArray<const float> v;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const float>(v, val, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp == 0) return SLIMDP_OK;
    return launch_merge(w_global, n, K, core_idx, k_core, exp, k_exp, v, eta, (cudaStream_t)stream);
}

slimdp_status slimdp_exchange(float* w_global, uint64_t n, uint32_t K, const float* const* deltas,
                              const uint32_t* core_idx, uint64_t k_core, const uint32_t* const* exp_idx,
                              uint64_t k_exp, float eta, float* const* val, float* const* pulled, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_global || !aligned4(w_global) || !isfinite(eta))
        return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> d;
    PtrArray<const uint32_t> exp;
    PtrArray<float> v, o;
    if (!fill<const float>(d, deltas, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(v, val, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(o, pulled, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp == 0) return SLIMDP_OK;
    return launch_exchange(w_global, n, K, d, core_idx, k_core, exp, k_exp, eta, v, o, nullptr, 0, nullptr, nullptr,
                           nullptr, nullptr, (cudaStream_t)stream);
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
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<float> w;
    PtrArray<const uint32_t> exp;
    PtrArray<const float> v;
    if (!fill<float>(w, w_local, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const float>(v, pulled, K, k_core + k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    return launch_worker_merge(w, K, core_idx, k_core, exp, k_exp, v, (cudaStream_t)stream);
}

slimdp_status slimdp_core_signature(const uint32_t* keys, uint64_t count, uint64_t* signature, void* stream) {
    if (count > kMaxN || !signature || (reinterpret_cast<uintptr_t>(signature) & 7u) != 0) return SLIMDP_ERR_INVALID_ARG;
    if (count > 0 && (!keys || !aligned4(keys))) return SLIMDP_ERR_INVALID_ARG;
    return launch_signature(keys, count, reinterpret_cast<unsigned long long*>(signature), (cudaStream_t)stream);
}

size_t slimdp_wire_bytes(uint64_t k_core, uint64_t k_exp) { return (size_t)(4 * k_core + 8 * k_exp + 8); }

// ---- per-segment selection --------------------------------------------------

size_t slimdp_select_segmented_workspace_bytes(uint64_t n, uint32_t segments) {
    if (!n_ok(n) || segments < 1 || segments > SLIMDP_MAX_SEGMENTS) return 0;
    return seg_select_ws_bytes(n, segments);
}

slimdp_status slimdp_select_core_segmented(const float* scores, uint64_t n, const uint64_t* seg_off,
                                           const uint64_t* seg_k, uint32_t segments, uint32_t* core_idx,
                                           void* core_aux, void* ws, size_t ws_bytes, void* stream) {
    if (!n_ok(n) || segments < 1 || segments > SLIMDP_MAX_SEGMENTS || !scores || !seg_off || !seg_k || !core_aux ||
        !ws)
        return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(scores) || !aligned16(core_aux) || !aligned16(ws)) return SLIMDP_ERR_INVALID_ARG;
    if (seg_off[0] != 0 || seg_off[segments] != n) return SLIMDP_ERR_INVALID_ARG;
    uint64_t k_total = 0;
    for (uint32_t s = 0; s < segments; ++s) {
        if (seg_off[s + 1] < seg_off[s] || seg_k[s] > seg_off[s + 1] - seg_off[s]) return SLIMDP_ERR_INVALID_ARG;
        k_total += seg_k[s];
    }
    if (k_total > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (ws_bytes < slimdp_select_segmented_workspace_bytes(n, segments)) return SLIMDP_ERR_WORKSPACE;
    return launch_select_segmented(scores, n, seg_off, seg_k, segments, k_total, core_idx, core_aux, ws,
                                   (cudaStream_t)stream);
}

// ---- 8-bit pushed values ---------------------------------------------------

slimdp_status slimdp_pack_q8_batched(const float* const* deltas, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                     uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                     int8_t* const* codes, float* const* scales, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !deltas) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> d;
    PtrArray<const uint32_t> exp;
    PtrArray<int8_t> c;
    PtrArray<float> sc;
    const bool any = k_core + k_exp > 0;
    if (!fill<const float>(d, deltas, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<int8_t>(c, codes, K, any, 1)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<float>(sc, scales, K, any, 4)) return SLIMDP_ERR_INVALID_ARG;
    return launch_pack_q8(d, K, core_idx, k_core, exp, k_exp, c, sc, (cudaStream_t)stream);
}

slimdp_status slimdp_merge_q8(float* w_global, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                              const uint32_t* const* exp_idx, uint64_t k_exp, const int8_t* const* codes,
                              const float* const* scales, float eta, void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_global || !aligned4(w_global) || !isfinite(eta))
        return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const uint32_t> exp;
    PtrArray<const int8_t> c;
    PtrArray<const float> sc;
    const bool any = k_core + k_exp > 0;
    if (!fill<const uint32_t>(exp, exp_idx, K, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const int8_t>(c, codes, K, any, 1)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<const float>(sc, scales, K, any, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!any) return SLIMDP_OK;
    return launch_merge_q8(w_global, n, K, core_idx, k_core, exp, k_exp, c, sc, eta, (cudaStream_t)stream);
}

// ---- selection over a range-sharded model ---------------------------------

size_t slimdp_explore_shard_workspace_bytes(uint64_t n_shard, uint64_t noncore_total, uint64_t k_exp) {
    if (!n_ok(n_shard) || noncore_total > kMaxN || k_exp > noncore_total) return 0;
    return explore_shard_ws_bytes(n_shard, noncore_total, k_exp);
}

slimdp_status slimdp_sample_explore_shard(const void* core_aux, uint64_t n_shard, uint64_t k_core_shard,
                                          uint64_t noncore_total, uint64_t noncore_below, uint64_t k_exp,
                                          uint64_t seed, uint32_t worker, uint32_t round, uint32_t* exp_idx,
                                          uint64_t cap, uint32_t* count, void* ws, size_t ws_bytes, void* stream) {
    if (!n_ok(n_shard) || k_core_shard > n_shard || noncore_total > kMaxN || k_exp > noncore_total || !core_aux ||
        !count || !ws)
        return SLIMDP_ERR_INVALID_ARG;
    if (noncore_below + (n_shard - k_core_shard) > noncore_total) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned16(core_aux) || !aligned16(ws) || !aligned4(count)) return SLIMDP_ERR_INVALID_ARG;
    if (cap > 0 && (!exp_idx || !aligned4(exp_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (ws_bytes < slimdp_explore_shard_workspace_bytes(n_shard, noncore_total, k_exp)) return SLIMDP_ERR_WORKSPACE;
    return launch_explore_shard(core_aux, n_shard, k_core_shard, noncore_total, noncore_below, k_exp, seed, worker,
                                round, exp_idx, cap, count, ws, (cudaStream_t)stream);
}

slimdp_status slimdp_select_shard_begin(uint64_t k_total, void* state, void* stream) {
    if (!state || (reinterpret_cast<uintptr_t>(state) & 7u) != 0) return SLIMDP_ERR_INVALID_ARG;
    return launch_shard_state_init(state, k_total, (cudaStream_t)stream);
}

slimdp_status slimdp_select_hist(const float* scores, uint64_t n_shard, uint32_t round, const void* state,
                                 uint64_t* hist, void* stream) {
    if (n_shard > kMaxN || round > 2 || !state || !hist || (n_shard > 0 && (!scores || !aligned4(scores))))
        return SLIMDP_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(state) | reinterpret_cast<uintptr_t>(hist)) & 7u) != 0)
        return SLIMDP_ERR_INVALID_ARG;
    return launch_shard_hist(scores, n_shard, round, state, hist, (cudaStream_t)stream);
}

slimdp_status slimdp_select_resolve(const uint64_t* hist, uint32_t round, void* state, void* stream) {
    if (round > 2 || !state || !hist) return SLIMDP_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(state) | reinterpret_cast<uintptr_t>(hist)) & 7u) != 0)
        return SLIMDP_ERR_INVALID_ARG;
    return launch_shard_resolve(hist, round, state, (cudaStream_t)stream);
}

slimdp_status slimdp_select_count(const float* scores, uint64_t n_shard, const void* state, uint64_t* counts,
                                  void* stream) {
    if (n_shard > kMaxN || !state || !counts || (n_shard > 0 && (!scores || !aligned4(scores))))
        return SLIMDP_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(state) | reinterpret_cast<uintptr_t>(counts)) & 7u) != 0)
        return SLIMDP_ERR_INVALID_ARG;
    return launch_shard_count(scores, n_shard, state, counts, (cudaStream_t)stream);
}

slimdp_status slimdp_select_emit(const float* scores, uint64_t n_shard, uint32_t threshold_bits, uint64_t tie_quota,
                                 uint64_t k_shard, uint32_t* core_idx, void* core_aux, void* ws, size_t ws_bytes,
                                 void* stream) {
    if (!n_ok(n_shard) || k_shard > n_shard || tie_quota > k_shard || !scores || !core_aux || !ws)
        return SLIMDP_ERR_INVALID_ARG;
    if (k_shard > 0 && !core_idx) return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(scores) || !aligned16(core_aux) || !aligned16(ws) || (core_idx && !aligned4(core_idx)))
        return SLIMDP_ERR_INVALID_ARG;
    if (ws_bytes < slimdp_select_workspace_bytes(n_shard)) return SLIMDP_ERR_WORKSPACE;
    return launch_select_given(scores, n_shard, threshold_bits, (uint32_t)tie_quota, k_shard, core_idx, core_aux, ws,
                               (cudaStream_t)stream);
}

size_t slimdp_wire_message_bytes(uint64_t k_core, uint64_t k_exp, int with_keys) {
    if (k_core > kMaxN || k_exp > kMaxN) return 0;
    return (size_t)(32 + 4 * k_core * (with_keys ? 2 : 1) + 8 * k_exp);
}

slimdp_status slimdp_wire_pack(const uint32_t* core_idx, uint64_t k_core, const uint32_t* exp_idx, uint64_t k_exp,
                               const float* val, const uint64_t* signature, uint32_t worker, uint32_t round,
                               int with_keys, void* msg, void* stream) {
    if (k_core > kMaxN || k_exp > kMaxN || !signature || !msg || !aligned16(msg) ||
        (reinterpret_cast<uintptr_t>(signature) & 7u) != 0)
        return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (k_exp > 0 && (!exp_idx || !aligned4(exp_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp > 0 && (!val || !aligned4(val))) return SLIMDP_ERR_INVALID_ARG;
    return launch_wire_pack(core_idx, k_core, exp_idx, k_exp, val,
                            reinterpret_cast<const unsigned long long*>(signature), worker, round, with_keys != 0, msg,
                            (cudaStream_t)stream);
}

slimdp_status slimdp_wire_unpack(const void* msg, size_t msg_bytes, const uint64_t* cached_signature,
                                 uint64_t k_core, uint64_t k_exp, uint32_t* core_idx, uint32_t* exp_idx, float* val,
                                 uint64_t* signature_out, int32_t* status, void* stream) {
    if (k_core > kMaxN || k_exp > kMaxN || !msg || !aligned16(msg) || !cached_signature || !signature_out || !status)
        return SLIMDP_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(cached_signature) | reinterpret_cast<uintptr_t>(signature_out) |
          reinterpret_cast<uintptr_t>(status)) & 7u) != 0)
        return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (k_exp > 0 && (!exp_idx || !aligned4(exp_idx))) return SLIMDP_ERR_INVALID_ARG;
    if (k_core + k_exp > 0 && (!val || !aligned4(val))) return SLIMDP_ERR_INVALID_ARG;
    // the kernels read the header and the k_core words after it whatever the message turns out to be
    if (msg_bytes < 32 + 4 * k_core) return SLIMDP_ERR_INVALID_ARG;
    return launch_wire_unpack(msg, msg_bytes, reinterpret_cast<const unsigned long long*>(cached_signature), k_core,
                              k_exp, core_idx, exp_idx, val, reinterpret_cast<unsigned long long*>(signature_out),
                              status, (cudaStream_t)stream);
}

slimdp_status slimdp_wire_read_status(const int32_t* status, void* stream) {
    if (!status) return SLIMDP_ERR_INVALID_ARG;
    int32_t s = 0;
    if (cudaMemcpyAsync(&s, status, sizeof(s), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return SLIMDP_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return SLIMDP_ERR_CUDA;
    if (s == 0) return SLIMDP_OK;
    return (s == SLIMDP_WIRE_KEYS_WANTED) ? SLIMDP_WIRE_KEYS_WANTED : SLIMDP_ERR_INVALID_ARG;
}

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
// finishing kernel of the selection, the exchange incl. the explorers'
// indices) runs on the context's stream of the highest priority.  The
// explorer's ranks depend on the sizes alone: they are computed and sorted on
// a second stream of the lowest priority, released when the pass starts, in the
// part of each SM that the pass leaves free.  Whenever a kernel of the chain
// becomes ready its CTAs are placed ahead of those of the rank kernels.  The
// caller's stream only forks into the chain at the start of the call and
// waits for it at the end (chain_done), on every path through the call.
// Scoring is folded into the selection's one pass over all parameters, so the
// scores are never written unless the selection has to fall back to its full path.

}  // extern "C"

struct slimdp_round_ctx {
    std::mutex lock;
    int device = -1;
    cudaStream_t chain = nullptr, ranks = nullptr;
    cudaEvent_t fork = nullptr, pass_ready = nullptr, ranks_done = nullptr, chain_done = nullptr;
};

namespace {
thread_local cudaEvent_t t_mark_begin = nullptr, t_mark_end = nullptr;
std::mutex g_default_mutex;
slimdp_round_ctx* g_default_ctx[64];   // per device, guarded by g_default_mutex

void ctx_release(slimdp_round_ctx* c) {
    cudaEvent_t ev[4] = {c->fork, c->pass_ready, c->ranks_done, c->chain_done};
    for (cudaEvent_t e : ev)
        if (e) cudaEventDestroy(e);
    if (c->chain) cudaStreamDestroy(c->chain);
    if (c->ranks) cudaStreamDestroy(c->ranks);
    delete c;
}

// A context on the current device; nullptr (nothing left behind) if any part of it cannot be created.
slimdp_round_ctx* ctx_make() {
    int dev = 0, lo = 0, hi = 0;   // numerically, hi <= lo: hi is the highest priority
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess)
        return nullptr;
    slimdp_round_ctx* c = new (std::nothrow) slimdp_round_ctx;
    if (!c) return nullptr;
    c->device = dev;
    bool ok = cudaStreamCreateWithPriority(&c->chain, cudaStreamNonBlocking, hi) == cudaSuccess &&
              cudaStreamCreateWithPriority(&c->ranks, cudaStreamNonBlocking, lo) == cudaSuccess;
    cudaEvent_t* ev[4] = {&c->fork, &c->pass_ready, &c->ranks_done, &c->chain_done};
    for (cudaEvent_t* e : ev) ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        ctx_release(c);
        return nullptr;
    }
    return c;
}

slimdp_round_ctx* default_ctx() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_default_mutex);
    if (!g_default_ctx[dev]) g_default_ctx[dev] = ctx_make();
    return g_default_ctx[dev];
}
}  // namespace

extern "C" {

slimdp_status slimdp_round_ctx_create(slimdp_round_ctx** ctx) {
    if (!ctx) return SLIMDP_ERR_INVALID_ARG;
    *ctx = ctx_make();
    return *ctx ? SLIMDP_OK : SLIMDP_ERR_CUDA;
}

slimdp_status slimdp_round_ctx_destroy(slimdp_round_ctx* ctx) {
    if (!ctx) return SLIMDP_ERR_INVALID_ARG;
    ctx_release(ctx);
    return SLIMDP_OK;
}

slimdp_status slimdp_round_release_default_ctx(void) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLIMDP_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_default_mutex);
    if (g_default_ctx[dev]) {
        ctx_release(g_default_ctx[dev]);
        g_default_ctx[dev] = nullptr;
    }
    return SLIMDP_OK;
}

size_t slimdp_round_stage_bytes(uint64_t n, uint32_t K, uint64_t k_core) {
    if (!n_ok(n) || !k_ok(K) || k_core > n) return 0;
    return stage_bytes_for(n, K, k_core);
}

slimdp_status slimdp_round(float* w_global, const float* const* grads, uint32_t K, uint64_t n, float c,
                           uint64_t k_core, uint64_t k_exp, uint64_t seed, uint32_t round, float eta, float* scores,
                           uint32_t* core_idx, void* core_aux, uint32_t* const* exp_idx, float* const* val,
                           float* const* pulled, void* select_ws, size_t select_ws_bytes, void* explore_ws,
                           size_t explore_ws_bytes, void* stage, size_t stage_bytes, slimdp_round_ctx* ctx,
                           void* stream) {
    if (!sets_ok(n, k_core, k_exp) || !k_ok(K) || !w_global || !grads || !scores || !core_aux || !select_ws ||
        !explore_ws || !isfinite(c) || !isfinite(eta))
        return SLIMDP_ERR_INVALID_ARG;
    if (!aligned4(w_global) || !aligned4(scores) || !aligned16(core_aux) || !aligned16(select_ws) ||
        !aligned16(explore_ws))
        return SLIMDP_ERR_INVALID_ARG;
    if (stage && (reinterpret_cast<uintptr_t>(stage) & 255u) != 0) return SLIMDP_ERR_INVALID_ARG;
    if (k_core > 0 && (!core_idx || !aligned4(core_idx))) return SLIMDP_ERR_INVALID_ARG;
    PtrArray<const float> g;
    PtrArray<uint32_t> exp_out;
    PtrArray<const uint32_t> exp_in;
    PtrArray<float> v, o;
    if (!fill<const float>(g, grads, K, true, 4)) return SLIMDP_ERR_INVALID_ARG;
    if (!fill<uint32_t>(exp_out, exp_idx, K, k_exp > 0, 4)) return SLIMDP_ERR_INVALID_ARG;
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
    const bool fusable = score_select_fusable(n, k_core, K, vec);

    cudaStream_t st = (cudaStream_t)stream;
    slimdp_round_ctx* side = ctx ? ctx : default_ctx();
    if (!side) return SLIMDP_ERR_CUDA;
    {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev != side->device) return SLIMDP_ERR_INVALID_ARG;
    }
    std::lock_guard<std::mutex> lock(side->lock);
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
    // chain: the core, scored and selected in one pass where sizes and alignment allow.  Short vectors
    // are bound by the number of dependent launches: there the selection stops after its finishing
    // kernel and the exchange places the core's members itself (one launch less).  On long vectors the
    // separate emit kernel followed by the exchange over the finished index list is as fast or faster
    // (measured: 138 M parameters 1.58 ms either way; 25.6 M parameters with 16 workers 1.10 against 1.18 ms;
    // 7 M parameters with 8 workers 201 against 206 us).
    bool staged = false;
    const bool folded = stage == nullptr && n < kFoldedExchangeMaxN && round_exchange_applies(n, k_exp);
    if (fusable) {
        rank_work.after = side->pass_ready;   // recorded by the call below just before its pass
        rank_work.lean = true;
        step(launch_score_select(w_global, g, K, c, n, scores, k_core, core_idx, core_aux, select_ws, mark0, mark1,
                                 enqueue_ranks, &rank_work, side->pass_ready, stage, stage_bytes, &staged, !folded, ch));
        // (if the call failed before it reached the hook, ranks_done keeps an earlier record: nothing to wait for)
    } else {
        step(enqueue_ranks(&rank_work));
        if (rc == SLIMDP_OK && mark0) cuda(cudaEventRecord(mark0, ch));
        if (rc == SLIMDP_OK) step(launch_score(w_global, g, K, c, n, scores, vec, ch));
        if (rc == SLIMDP_OK && mark1) cuda(cudaEventRecord(mark1, ch));
        if (rc == SLIMDP_OK) step(launch_select(scores, n, k_core, core_idx, core_aux, select_ws, !folded, ch));
    }
    // chain: explorer indices from the sorted ranks and the core, then the exchange; where the
    // exchange's warp ranges line up with the core's directory it computes the indices itself
    cuda(cudaStreamWaitEvent(ch, side->ranks_done, 0));
    const uint32_t* aux_bitmap = reinterpret_cast<const uint32_t*>(core_aux);
    const uint32_t* aux_dir =
        reinterpret_cast<const uint32_t*>(static_cast<const char*>(core_aux) + slimdp_core_aux_dir_offset(n));
    ExchangeStage xs{};
    if (staged) {
        const SelectWs SL = select_ws_layout(select_ws, n);
        const StageArea A = stage_layout(stage, n, K, k_core, (uint32_t)sm_count() * 8u);
        xs = ExchangeStage{A.fill, A.chunks, (uint32_t)A.max_chunks, SL.hdr, (uint32_t)SL.cand_cap};
    }
    const ExchangeStage* xsp = staged ? &xs : nullptr;
    if (folded) {
        const SelectWs SL = select_ws_layout(select_ws, n);
        const ExploreWs EL = explore_ws_layout(explore_ws, n, k_exp, K);
        if (rc == SLIMDP_OK)
            step(launch_round_exchange(w_global, n, K, g, k_core, exp_in, k_exp, eta, v, o, EL.rho, EL.rho_stride,
                                       &EL.hdr->status, SL.G, SL.E, SL.tile_sum, SL.super_pref, SL.hdr, core_idx,
                                       const_cast<uint32_t*>(aux_bitmap), const_cast<uint32_t*>(aux_dir), ch));
    } else if (exchange_takes_ranks(n, k_exp)) {
        const ExploreWs EL = explore_ws_layout(explore_ws, n, k_exp, K);
        if (rc == SLIMDP_OK)
            step(launch_exchange(w_global, n, K, g, core_idx, k_core, exp_in, k_exp, eta, v, o, EL.rho, EL.rho_stride,
                                 aux_bitmap, aux_dir, &EL.hdr->status, xsp, ch));
    } else {
        if (rc == SLIMDP_OK)
            step(launch_explore_parts(core_aux, n, k_core, k_exp, seed, 0, K, round, exp_out, explore_ws, 2, false,
                                      ch));
        if (rc == SLIMDP_OK && k_core + k_exp > 0)
            step(launch_exchange(w_global, n, K, g, core_idx, k_core, exp_in, k_exp, eta, v, o, nullptr, 0,
                                 aux_bitmap, aux_dir, nullptr, xsp, ch));
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
    void* stage;
    size_t stage_bytes;
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
    A.stage_bytes = slimdp_round_stage_bytes(n, K, k_core);
    A.stage = A.stage_bytes ? take(A.stage_bytes) : nullptr;
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
                            A.explore_ws_bytes, A.stage, A.stage_bytes, nullptr, stream));
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
