/* slimdp.h - C ABI of the Slim-DP communication round for NVIDIA B200 (sm_100a).
 *
 * One Slim-DP communication round (Sun et al., "Slim-DP: A Light Communication
 * Data Parallelism for DNN", Algorithm 1 and Section 3.3) touches a flat fp32
 * parameter vector w-bar of n entries and K workers' accumulated updates
 * delta_k of n entries each:
 *
 *   score    S_i = |w_i| + c |g_i|                         (Eq. 1, Section 3.2)
 *   select   core = the k_core parameters of largest S     (Section 3.2; T_S of Section 3.1)
 *   explore  per worker, per round: k_exp random parameters outside the core
 *                                                          (T_R^k, Section 3.1 item 2, Section 3.3 step 2)
 *   pack     T_C(delta_k): the worker's updates on core U explorer
 *                                                          (Section 3.1; extraction, Section 3.5)
 *   merge    w-bar <- w-bar - eta' T_C(delta_k), all k     (Section 3.3 step 3)
 *   pull     T_C(w-bar): merged values on core U explorer  (Section 3.3 step 4)
 *
 * General rules, valid for every entry point unless it says otherwise:
 *   - Every pointer is a DEVICE pointer (memory of the current CUDA device)
 *     unless its comment says HOST.  "HOST array of K device pointers" means a
 *     host-side array whose K entries are device pointers; it is read during
 *     the call and may be freed as soon as the call returns.
 *   - The caller owns every buffer.  The library allocates no device memory,
 *     creates no stream (round contexts excepted, see slimdp_round), and never
 *     synchronises except in slimdp_read_status and slimdp_round_host.  All work is enqueued on `stream` (a cudaStream_t
 *     passed as void*; NULL is the legacy default stream) and is ordered with
 *     other work on that stream.
 *   - Arguments are validated on the host before anything is enqueued.  A
 *     negative return value means nothing (more) was enqueued by that call.
 *   - Indices are 0-based uint32_t, so 1 <= n < 2^32.  fp32 and index buffers
 *     must be 4-byte aligned.  16-byte alignment of all fp32 tensors of a call
 *     selects the vectorised kernels; slimdp_score also takes them when all
 *     tensors are off a 16-byte boundary by the same amount (slices of one
 *     allocation), after one to three leading parameters.  Any alignment is
 *     computed correctly.  core_aux and workspaces must be 16-byte aligned.
 *   - Input and output buffers of one call must not overlap, except where a
 *     buffer is documented as updated in place.
 *   - Results are deterministic: the same inputs give the same bytes on every
 *     call, whatever the launch shape.
 */
#ifndef SLIMDP_H_
#define SLIMDP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t slimdp_status;

enum {
    SLIMDP_OK = 0,
    SLIMDP_ERR_INVALID_ARG = -1, /* null pointer, count out of range, non-finite coefficient, misaligned buffer */
    SLIMDP_ERR_WORKSPACE = -2,   /* workspace / arena smaller than the matching *_bytes query              */
    SLIMDP_ERR_CUDA = -3,        /* a CUDA runtime call or kernel launch failed                             */
    SLIMDP_ERR_INTERNAL = -4,    /* a device-side consistency check failed (reported by slimdp_read_status) */
    SLIMDP_ERR_UNSUPPORTED = -5
};

/* Largest K: the K per-worker device pointers travel by value as kernel arguments. */
#define SLIMDP_MAX_WORKERS 64

/* Parameters per bitmap block (32 words), and per directory entry of core_aux. */
#define SLIMDP_BLOCK 1024
#define SLIMDP_DIR_STRIDE 64

const char* slimdp_status_string(slimdp_status s);

/* ---------------------------------------------------------------- sizes ---
 * core_aux is the device-side description of the core that the explorer
 * sampler reads.  Layout (all uint32_t, little-endian bit order):
 *   bitmap    [nb * 32] words, nb = ceil(n / 1024): bit (i & 31) of word (i >> 5)
 *             is 1 iff parameter i is in the core; bits at i >= n are 0;
 *   directory [nd + 1] words, nd = 16 nb, starting at byte offset slimdp_core_aux_dir_offset(n):
 *             directory[d] = 64 d - (number of core parameters with index < 64 d) for d < nd,
 *             i.e. the number of NON-core parameters below 64 d wherever 64 d <= n;
 *             directory[nd] = n - k_core.
 */
size_t slimdp_core_aux_bytes(uint64_t n);
size_t slimdp_core_aux_dir_offset(uint64_t n);

/* Bytes of scratch that slimdp_select_core needs for n parameters. */
size_t slimdp_select_workspace_bytes(uint64_t n);

/* Bytes of scratch that slimdp_sample_explore (num_workers = 1) or
 * slimdp_sample_explore_batched (num_workers workers in one call) needs to
 * draw k_exp parameters per worker (any k_core). */
size_t slimdp_explore_workspace_bytes(uint64_t n, uint64_t k_exp, uint32_t num_workers);

/* max(select, explore for K workers): one workspace that serves every separate call of a round. */
size_t slimdp_workspace_bytes(uint64_t n, uint32_t K, uint64_t k_core, uint64_t k_exp);

/* ---------------------------------------------------------------- score ---
 * Eq. 1 (Section 3.2).  For every i < n, in fp32:
 *     g      = ((grads[0][i] + grads[1][i]) + ...) + grads[K-1][i]   (left to right)
 *     S[i]   = fma(c, |g|, |w[i]|)                                   (one rounding)
 * and a NaN result is stored as the bit pattern 0x7FC00000.  g is the sum of
 * the updates all K workers pushed densely before a reselection (Section 3.3
 * steps 3 and 6); a caller that already holds an aggregated gradient passes
 * K = 1.  Scores are >= +0, +inf or that NaN, so their bit patterns order them.
 *   w       [n] global model                       (read)
 *   grads   HOST array of K device pointers, each [n] (read), 1 <= K <= SLIMDP_MAX_WORKERS
 *   c       finite, the coefficient of Eq. 1
 *   scores  [n] (written)
 */
slimdp_status slimdp_score(const float* w, const float* const* grads, uint32_t K, float c, uint64_t n,
                           float* scores, void* stream);

/* --------------------------------------------------------------- select ---
 * Core selection T_S (Section 3.1 item 1; the ranking by significance of
 * Section 3.2): the k_core parameters that come first when all n are ordered
 * by (score bit pattern descending as unsigned 32-bit, index ascending).  For scores from slimdp_score this is score
 * descending with ties going to the smaller index and NaN ranking highest.
 *   scores    [n] (read)
 *   k_core    0 <= k_core <= n
 *   core_idx  [k_core] (written): the core, ascending
 *   core_aux  [slimdp_core_aux_bytes(n)] (written): bitmap + directory, see above
 *   ws        [ws_bytes >= slimdp_select_workspace_bytes(n)] scratch, contents undefined after
 * Device-side consistency failures are recorded in the first word of ws; read
 * them with slimdp_read_status(ws, stream).  The last kernel of the selection
 * is a cooperative launch whose CTAs meet at a grid barrier; every wait there
 * is bounded, and a wait that runs out is reported the same way.
 */
slimdp_status slimdp_select_core(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx,
                                 void* core_aux, void* ws, size_t ws_bytes, void* stream);

/* Per-layer selection: the ranking of Section 3.2 done segment by segment, the simplest of the
 * "model-specific" significance measures that Section 5 leaves open.  The vector is cut into
 * `segments` consecutive segments (layers), segment s = [seg_off[s], seg_off[s+1]); segment s
 * contributes its seg_k[s] parameters of largest score, ties to the smaller index; the core is
 * their union.  core_idx (ascending, sum of seg_k entries) and core_aux come out exactly as from
 * slimdp_select_core, so every other call works on the result unchanged.
 *   seg_off  HOST array [segments + 1], seg_off[0] = 0, non-decreasing, seg_off[segments] = n
 *   seg_k    HOST array [segments], seg_k[s] <= length of segment s
 *   (both are copied during the call and may be freed when it returns)
 *   ws       [ws_bytes >= slimdp_select_segmented_workspace_bytes(n, segments)] scratch */
#define SLIMDP_MAX_SEGMENTS 65536
size_t slimdp_select_segmented_workspace_bytes(uint64_t n, uint32_t segments);
slimdp_status slimdp_select_core_segmented(const float* scores, uint64_t n, const uint64_t* seg_off,
                                           const uint64_t* seg_k, uint32_t segments, uint32_t* core_idx,
                                           void* core_aux, void* ws, size_t ws_bytes, void* stream);

/* -------------------------------------------------------------- explore ---
 * Exploration operator T_R^k (Section 3.1 item 2, Section 3.3 step 2): worker
 * `worker` draws, for communication `round`, k_exp distinct parameters
 * uniformly from the M = n - k_core parameters outside the core.  The paper
 * asks only for a random choice; this library fixes the generator so that results can be
 * reproduced bit for bit:
 *   round keys rk[0..11] = three Philox-4x32-10 blocks with key
 *       (seed low word, seed high word) and counters (b, worker, round, 0x534C494D), b = 0, 1, 2;
 *   pi = a 10-round alternating Feistel network on b bits, b the least integer >= 2 with
 *       2^b >= M: x = A * 2^c + B with A of a = floor(b/2) bits and B of c = b - a bits;
 *       even round r: A = (A ^ F(B ^ rk[r])) & (2^a - 1); odd round r: B = (B ^ F(A ^ rk[r])) & (2^c - 1);
 *       F(v) = hi32(p) ^ lo32(p), p = (uint64)v * (r even ? 0xD2511F53 : 0xCD9E8D57);
 *       images >= M are fed through the network again (cycle walking, fewer than 2 passes on average);
 *   explorer = { the pi(j)-th non-core parameter (0-based, ascending) : j < k_exp }.
 *   core_aux  as written by slimdp_select_core for the same n and k_core (read)
 *   k_exp     0 <= k_exp <= n - k_core
 *   exp_idx   [k_exp] (written): the explorer, ascending
 *   ws        [ws_bytes >= slimdp_explore_workspace_bytes(n, k_exp, 1)] scratch
 */
slimdp_status slimdp_sample_explore(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp,
                                    uint64_t seed, uint32_t worker, uint32_t round, uint32_t* exp_idx,
                                    void* ws, size_t ws_bytes, void* stream);

/* The same for workers first_worker .. first_worker + num_workers - 1 in one
 * call; exp_idx is a HOST array of num_workers device pointers, each [k_exp].
 * ws_bytes >= slimdp_explore_workspace_bytes(n, k_exp, num_workers).  Results are
 * identical to num_workers single calls. */
slimdp_status slimdp_sample_explore_batched(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp,
                                            uint64_t seed, uint32_t first_worker, uint32_t num_workers,
                                            uint32_t round, uint32_t* const* exp_idx, void* ws,
                                            size_t ws_bytes, void* stream);

/* The paper has no counterpart of this call; it exists for callers that cannot
 * allocate.  slimdp_sample_explore needs a workspace, and some callers have no
 * way to get one: code that runs after a host application has handed all device
 * memory to its own pool, a plug-in whose host forbids cudaMalloc inside the
 * training loop because it would stall every stream, or a process running
 * under a memory cap that is already spent.  For them this variant draws one
 * worker's explorer with the library's own scratch: a static device array of
 * SLIMDP_STATIC_SCRATCH_MIB MiB that every GPU holding this library keeps from
 * load until the process exits.  It calls no allocator of any kind.
 *   Same arguments and same result (bit for bit) as slimdp_sample_explore,
 *   without ws / ws_bytes.  Limits: n <= SLIMDP_STATIC_MAX_N and
 *   k_exp <= SLIMDP_STATIC_MAX_K_EXP; anything larger returns
 *   SLIMDP_ERR_UNSUPPORTED and enqueues nothing.
 *   status   optional DEVICE int32 (may be NULL): receives, in stream order, the
 *            call's device-side consistency status (SLIMDP_OK or SLIMDP_ERR_INTERNAL).
 * The first call on each device looks up the scratch array's device address
 * (cudaGetSymbolAddress, with that device current); make that first call
 * outside any stream capture.  The address is kept for the life of the device's
 * primary context.  All calls on a device share the one array and
 * each call overwrites what the last one left (it clears what it needs at zero
 * itself), so two calls that may run at the same time on the GPU, e.g. on
 * different streams, race; order them. */
#define SLIMDP_STATIC_SCRATCH_MIB 8
#define SLIMDP_STATIC_MAX_N (1ull << 25)
#define SLIMDP_STATIC_MAX_K_EXP (1ull << 18)
slimdp_status slimdp_sample_explore_static(const void* core_aux, uint64_t n, uint64_t k_core, uint64_t k_exp,
                                           uint64_t seed, uint32_t worker, uint32_t round, uint32_t* exp_idx,
                                           int32_t* status, void* stream);

/* ----------------------------------------------------------------- pack ---
 * Extraction of T_C(delta_k) = T_S(delta_k) U T_R^k(delta_k) (Section 3.1; the
 * extraction cost that Section 3.5 counts):
 *     val[j]          = delta[core_idx[j]]   j < k_core
 *     val[k_core + j] = delta[exp_idx[j]]    j < k_exp
 * The worker's <key, value> buffer (Section 3.5) is the pair
 * (core_idx || exp_idx, val); the core keys are stored once and shared by all
 * workers, which is the key-caching of Section 3.5, so a push carries
 * 4 (k_core + 2 k_exp) bytes.
 *   delta [n] (read), core_idx [k_core], exp_idx [k_exp] (read; entries < n), val [k_core + k_exp] (written)
 */
slimdp_status slimdp_pack(const float* delta, uint64_t n, const uint32_t* core_idx, uint64_t k_core,
                          const uint32_t* exp_idx, uint64_t k_exp, float* val, void* stream);

/* K workers in one call: deltas, exp_idx and val are HOST arrays of K device pointers. */
slimdp_status slimdp_pack_batched(const float* const* deltas, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                  uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                  float* const* val, void* stream);

/* ---------------------------------------------------------------- merge ---
 * Server update (Algorithm 1, Section 3.3 step 3): every worker's push is
 * applied to the global model, workers in ascending order:
 *     for k = 0 .. K-1:  for every pushed (i, v) of worker k:  w[i] = fma(-eta, v, w[i])
 * Explorers of different workers may contain the same parameter; it then
 * receives its updates in ascending k, so the fp32 result is unique.
 * Parameters outside every worker's communication set are not written.
 *   w_global  [n] (updated in place)
 *   exp_idx   HOST array of K device pointers, each [k_exp], ascending, disjoint from core_idx
 *   val       HOST array of K device pointers, each [k_core + k_exp], as written by slimdp_pack
 *   eta       finite, the server step eta'
 */
slimdp_status slimdp_merge(float* w_global, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                           const uint32_t* const* exp_idx, uint64_t k_exp, const float* const* val, float eta,
                           void* stream);

/* ----------------------------------------------------------------- pull ---
 * Pull of T_C(w-bar) (Algorithm 1, Section 3.3 step 4):
 *     out[j] = w_global[core_idx[j]],  out[k_core + j] = w_global[exp_idx[j]].
 */
slimdp_status slimdp_pull(const float* w_global, uint64_t n, const uint32_t* core_idx, uint64_t k_core,
                          const uint32_t* exp_idx, uint64_t k_exp, float* out, void* stream);

/* K workers in one call: exp_idx and out are HOST arrays of K device pointers. */
slimdp_status slimdp_pull_batched(const float* w_global, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                  uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                  float* const* out, void* stream);

/* ------------------------------------------------------------- exchange ---
 * Push, server update and pull of one round for all K workers in one call
 * (Section 3.3 steps 3 and 4; Algorithm 1's Push, Update, Pull).  The results
 * are bit-identical to slimdp_pack_batched, then slimdp_merge, then
 * slimdp_pull_batched on the same arguments; the three steps share one pass
 * over the communication set, so every gathered line is fetched once.
 *   w_global [n] (updated in place), deltas HOST array of K device pointers [n] (read)
 *   val, pulled  HOST arrays of K device pointers, each [k_core + k_exp] (written)
 */
slimdp_status slimdp_exchange(float* w_global, uint64_t n, uint32_t K, const float* const* deltas,
                              const uint32_t* core_idx, uint64_t k_core, const uint32_t* const* exp_idx,
                              uint64_t k_exp, float eta, float* const* val, float* const* pulled, void* stream);

/* ------------------------------------------ the steps either side of the path ---
 * Dense push at a reselection boundary (Algorithm 1: every q-th round the
 * worker pushes its whole update, and the server, after its update, selects a
 * new core; Section 3.3 steps 3 and 6).  One pass applies every worker's
 * WHOLE update to the global model in ascending worker order (this is also
 * Plump-DP's update, Section 2.1) and, if scores is not NULL, scores the
 * UPDATED model with the updates just pushed:
 *     x = w[i];  g = grads[0][i];  x = fma(-eta, grads[0][i], x);
 *     for k = 1..K-1:  g = g + grads[k][i];  x = fma(-eta, grads[k][i], x);
 *     w[i] = x;  scores[i] = fma(c, |g|, |x|)   (NaN stored as 0x7FC00000)
 * Bit-identical to slimdp_merge with everything in the communication set
 * followed by slimdp_score.
 *   w_global [n] (updated in place); grads HOST array of K device pointers [n]; scores [n] or NULL
 */
slimdp_status slimdp_dense_merge_score(float* w_global, const float* const* grads, uint32_t K, float eta, float c,
                                       uint64_t n, float* scores, void* stream);

/* Worker-side Merge (Algorithm 1 "Merge(w_k, w~_k)", Section 3.3 step 5): the
 * values a worker pulled replace its local model's values on its communication
 * set; the rest of the local model is left as local training made it.
 *     w_local[k][core_idx[j]] = pulled[k][j];  w_local[k][exp_idx[k][j]] = pulled[k][k_core + j]
 *   w_local, exp_idx, pulled: HOST arrays of K device pointers ([n], [k_exp], [k_core + k_exp])
 */
slimdp_status slimdp_worker_merge_batched(float* const* w_local, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                          uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                          const float* const* pulled, void* stream);

/* Key caching (Section 3.5): both sides keep the core's keys, so a push carries
 * the core's values and a signature of the keys instead of the keys themselves.
 * slimdp_core_signature writes a 64-bit signature of a key list to device memory:
 *     sig = sum_j mix64(((j << 32) | keys[j]) + 0x9E3779B97F4A7C15)  mod 2^64,
 *     mix64(z): z ^= z >> 30; z *= 0xBF58476D1CE4E5B9; z ^= z >> 27; z *= 0x94D049BB133111EB; z ^= z >> 31
 * (the SplitMix64 output function).  Sender and receiver compare signatures to
 * know that their cached core keys agree; the empty list has signature 0.
 *   keys [count] (read), signature: DEVICE uint64, 8-byte aligned (written)
 * slimdp_wire_bytes: bytes one worker sends per direction and round with key
 * caching: 4 k_core values + 8 k_exp <key, value> pairs + the 8-byte signature,
 * i.e. (2 alpha - beta) n words as in Section 3.5, against 4 n for Plump-DP. */
slimdp_status slimdp_core_signature(const uint32_t* keys, uint64_t count, uint64_t* signature, void* stream);
size_t slimdp_wire_bytes(uint64_t k_core, uint64_t k_exp);

/* ------------------------------------------------ 8-bit pushed values ---
 * Section 2.2 closes by noting that the method combines with quantisation of
 * what is sent.  The paper defines no quantiser; this library fixes a
 * deterministic one so that sender, receiver and a reference agree bit for bit.
 * A worker's packed buffer (core values, then explorer values: k_core + k_exp
 * entries) is cut into buckets of SLIMDP_Q8_BUCKET consecutive entries; a
 * bucket's scale is its largest finite magnitude; a value v becomes the code
 *     rint(v * (127 / scale)) clamped to [-127, 127]   (fp32 division, fp32 product, ties to even),
 * 0 if the scale is 0 or v is a NaN, +-127 if v is an infinity; the receiver
 * reads code * (scale / 127) (fp32 division, fp32 product).  A push then costs
 * k_core + k_exp bytes of codes and one fp32 scale per bucket instead of
 * 4 (k_core + k_exp) bytes of values.
 * slimdp_pack_q8_batched: slimdp_pack_batched with the quantiser folded into its
 *   stores (the fp32 packed buffer is never written).
 *   codes   HOST array of K device pointers, each int8 [k_core + k_exp] (written)
 *   scales  HOST array of K device pointers, each fp32 [ceil((k_core + k_exp) / SLIMDP_Q8_BUCKET)] (written)
 * slimdp_merge_q8: slimdp_merge reading its values through the codes: bit-identical to
 *   slimdp_merge on the decoded values. */
#define SLIMDP_Q8_BUCKET 256
slimdp_status slimdp_pack_q8_batched(const float* const* deltas, uint32_t K, uint64_t n, const uint32_t* core_idx,
                                     uint64_t k_core, const uint32_t* const* exp_idx, uint64_t k_exp,
                                     int8_t* const* codes, float* const* scales, void* stream);
slimdp_status slimdp_merge_q8(float* w_global, uint64_t n, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                              const uint32_t* const* exp_idx, uint64_t k_exp, const int8_t* const* codes,
                              const float* const* scales, float eta, void* stream);

/* ------------------------------------------ selection over a sharded model ---
 * The parameter-server setting of Section 2.1 with the global model cut into
 * contiguous shards, one per GPU.  Scoring, pack, merge and pull work shard by
 * shard on local indices; the core does not, because Section 3.2 ranks all
 * parameters.  These calls are the selection cut at its reduction points, so
 * that the exact global core costs three all-reduces of 4096 counters and one
 * all-gather of two counters per shard:
 *   slimdp_select_shard_begin(k_total, state)         state <- (prefix 0, rank k_total), on every shard
 *   for round = 0, 1, 2 (digits of 12, 10, 10 bits, most significant first):
 *     clear hist; slimdp_select_hist(shard, round, state, hist)   hist[b] += keys of the shard with digit b
 *                                                                 (and the prefix found so far)
 *     sum hist over all shards (all-reduce)
 *     slimdp_select_resolve(hist, round, state)      the digit that holds the wanted rank; the same on every shard
 *   now state holds the threshold T (the k_total-th largest key of the whole model) and r, the
 *   number of keys equal to T that belong to the core
 *   (k_total = 0, the empty core: T = 0xFFFFFFFF and r = 0, so that no key is above T and none is admitted)
 *   clear counts; slimdp_select_count(shard, state, counts)   counts[0] += keys > T, counts[1] += keys == T
 *   all-gather the counts: shard g admits quota_g = min(equal_g, max(0, r - sum of equal_h, h < g))
 *   of its equal keys (ties go to the smaller global index, and shards are index ranges), and its
 *   part of the core has k_g = greater_g + quota_g members
 *   slimdp_select_emit(shard, T, quota_g, k_g, ...)  the shard's core_idx (shard-local indices,
 *   ascending) and core_aux, exactly as slimdp_select_core writes them for a whole vector
 * The concatenation of the shards' lists (local index + shard offset) is bit for bit the core that
 * slimdp_select_core finds on the whole vector.  With one process per GPU the two reductions are
 * NCCL calls on the device buffers `hist` and `counts`; nothing here waits on another GPU.
 *   state   DEVICE record of 16 bytes, 8-byte aligned: uint32 prefix (after round 2: T), int32 status
 *           (SLIMDP_OK, or SLIMDP_ERR_INTERNAL if the summed histogram held fewer keys than the rank),
 *           uint64 remaining rank (after round 2: r)
 *   hist    DEVICE uint64[4096] (rounds 1 and 2 use the first 1024), added to
 *   counts  DEVICE uint64[2], added to
 *   scores  the shard's scores [n_shard] (n_shard may be 0 in hist / count)
 * With the core in place, pack, merge and pull run per shard on shard-local indices as they are.
 * slimdp_sample_explore_shard: one shard's share of a worker's explorer (Section 3.3 step 2 on the
 *   sharded model).  The explorer is drawn over the non-core parameters of ALL shards, numbered in index
 *   order: every shard evaluates the same noncore_total-rank permutation prefix (the generator of
 *   slimdp_sample_explore with M = noncore_total) and keeps the ranks of its own non-core parameters,
 *   [noncore_below, noncore_below + n_shard - k_core_shard), as shard-local indices.  The shards'
 *   lists, each shifted by its shard's offset and concatenated, are bit for bit the explorer that
 *   slimdp_sample_explore draws on the whole vector.  noncore_below and noncore_total come from the
 *   all-gather of the shards' core sizes.
 *   core_aux   the shard's, as written by slimdp_select_emit
 *   exp_idx    [cap] (written: *count entries, ascending); count: DEVICE uint32 (written)
 *   If the shard's share exceeds cap nothing is written, *count = 0 and the workspace's status word
 *   is set (slimdp_read_status).  noncore_total < 2^32.
 *   ws         [ws_bytes >= slimdp_explore_shard_workspace_bytes(n_shard, noncore_total, k_exp)] */
size_t slimdp_explore_shard_workspace_bytes(uint64_t n_shard, uint64_t noncore_total, uint64_t k_exp);
slimdp_status slimdp_sample_explore_shard(const void* core_aux, uint64_t n_shard, uint64_t k_core_shard,
                                          uint64_t noncore_total, uint64_t noncore_below, uint64_t k_exp,
                                          uint64_t seed, uint32_t worker, uint32_t round, uint32_t* exp_idx,
                                          uint64_t cap, uint32_t* count, void* ws, size_t ws_bytes, void* stream);
slimdp_status slimdp_select_shard_begin(uint64_t k_total, void* state, void* stream);
slimdp_status slimdp_select_hist(const float* scores, uint64_t n_shard, uint32_t round, const void* state,
                                 uint64_t* hist, void* stream);
slimdp_status slimdp_select_resolve(const uint64_t* hist, uint32_t round, void* state, void* stream);
slimdp_status slimdp_select_count(const float* scores, uint64_t n_shard, const void* state, uint64_t* counts,
                                  void* stream);
slimdp_status slimdp_select_emit(const float* scores, uint64_t n_shard, uint32_t threshold_bits, uint64_t tie_quota,
                                 uint64_t k_shard, uint32_t* core_idx, void* core_aux, void* ws, size_t ws_bytes,
                                 void* stream);

/* One worker's push as a message (Section 3.5: the core as values plus the
 * signature of its cached keys, the explorer as <key, value> pairs), built and
 * taken apart on the device.  Layout, little-endian, every field 4-byte aligned:
 *      0 u32 magic 0x57504453 ("SDPW")    4 u32 flags (bit 0: the core's keys are included)
 *      8 u64 signature of the sender's core keys (slimdp_core_signature)
 *     16 u32 k_core   20 u32 k_exp   24 u32 worker   28 u32 round
 *     32 [k_core x u32 keys, if flags bit 0]  k_core x f32 values  k_exp x (u32 key, f32 value)
 * i.e. 32 + 4 k_core + 8 k_exp bytes = (2 alpha - beta) n words plus the header
 * while the receiver's cached keys are current, 4 k_core more when the keys
 * travel again.  Values are moved as bits.
 * slimdp_wire_pack:   core_idx [k_core], exp_idx [k_exp], val [k_core + k_exp] as written by
 *   slimdp_pack (read); signature: DEVICE uint64 holding slimdp_core_signature(core_idx) (read);
 *   msg [slimdp_wire_message_bytes(k_core, k_exp, with_keys)], 16-byte aligned (written).
 * slimdp_wire_unpack: the receiver's side.  The verdict is reached on the device and left in
 *   status[0]: 0 = taken apart (exp_idx, val and *signature_out written; core_idx too if the
 *   message carried the keys, after their signature was checked against the header's);
 *   SLIMDP_WIRE_KEYS_WANTED = the sender's keys are not the ones whose signature the receiver has
 *   cached and the message does not carry them: nothing else is written, and the sender's next push
 *   is to be packed with with_keys = 1; -1 = malformed (magic, sizes other than k_core / k_exp /
 *   msg_bytes, unknown flags, keys that do not match the header's signature).
 *   cached_signature: DEVICE uint64 (read); signature_out: DEVICE uint64 (may be the same word);
 *   status: DEVICE scratch of 16 bytes, 8-byte aligned (status[0] is the verdict).
 *   core_idx [k_core], exp_idx [k_exp], val [k_core + k_exp] (written as described).
 * slimdp_wire_read_status synchronises `stream` and returns the verdict as SLIMDP_OK,
 *   SLIMDP_WIRE_KEYS_WANTED or SLIMDP_ERR_INVALID_ARG (malformed). */
#define SLIMDP_WIRE_KEYS_WANTED 1
size_t slimdp_wire_message_bytes(uint64_t k_core, uint64_t k_exp, int with_keys);
slimdp_status slimdp_wire_pack(const uint32_t* core_idx, uint64_t k_core, const uint32_t* exp_idx, uint64_t k_exp,
                               const float* val, const uint64_t* signature, uint32_t worker, uint32_t round,
                               int with_keys, void* msg, void* stream);
slimdp_status slimdp_wire_unpack(const void* msg, size_t msg_bytes, const uint64_t* cached_signature,
                                 uint64_t k_core, uint64_t k_exp, uint32_t* core_idx, uint32_t* exp_idx, float* val,
                                 uint64_t* signature_out, int32_t* status, void* stream);
slimdp_status slimdp_wire_read_status(const int32_t* status, void* stream);

/* --------------------------------------------------------------- status ---
 * Synchronises `stream`, then returns the sticky status word kept in the first
 * 4 bytes of a workspace used by slimdp_select_core / slimdp_sample_explore*:
 * SLIMDP_OK, or SLIMDP_ERR_INTERNAL if a device-side consistency check failed
 * (the outputs of that call are then undefined), or SLIMDP_ERR_CUDA. */
slimdp_status slimdp_read_status(const void* ws, void* stream);

/* Number of kernels this library has launched in this process so far (all
 * devices, all streams).  An accounting aid for benchmarks: read it before and
 * after a timed region.  The paper has no counterpart. */
uint64_t slimdp_launch_count(void);

/* --------------------------------------------------- whole round, device ---
 * One whole round on device buffers (Algorithm 1's communication step; Section
 * 3.3 steps 1 to 4, with the server's Core-Selection(w-bar, delta, beta) taking
 * the model and the updates directly, as Algorithm 1 writes it): the results
 * core_idx, core_aux, exp_idx, val, pulled and the updated w_global are
 * bit-identical to slimdp_score with grads, slimdp_select_core,
 * slimdp_sample_explore_batched for workers 0..K-1 and slimdp_exchange with
 * deltas = grads, called in that order.  What differs is how the device gets
 * there:
 *   - Scoring is folded into the selection's single pass over all parameters
 *     (n >= 2^21, k_core > 0, K <= 20 and 16-byte aligned w_global / grads /
 *     scores; otherwise the calls above run one after the other): each score
 *     is computed as the parameter streams by and classified on the spot, so
 *     the n scores are neither written nor read back.  `scores` is then only
 *     scratch: it holds the scores if the selection had to fall back to its
 *     full path (e.g. millions of equal scores around the threshold) and is
 *     left untouched otherwise.  Callers that want the scores call slimdp_score.
 *   - With a staging area (`stage`, optional) that pass also sets aside the K
 *     update values of every parameter that is certainly in the core or a
 *     candidate for it, while it has them at hand; the exchange then streams
 *     them instead of gathering K + 1 scattered lines per core parameter.
 *     slimdp_round_stage_bytes gives the size (0: staging does not apply to
 *     these sizes, e.g. a core of more than half the parameters); stage = NULL
 *     or a smaller area simply turns staging off.  Results do not depend on it.
 *   - The steps of a round depend on one another as a graph, not a chain: the
 *     explorer's ranks need the sizes only, so they are computed and sorted
 *     beside the pass over all parameters, in the part of every SM that the
 *     pass leaves free (the pass keeps its loads in flight in shared memory,
 *     one CTA per SM, and so needs few registers and threads).  For that the
 *     round runs on two streams of a round context: one of the highest
 *     priority for the chain of kernels that decides the round's time, one of
 *     the lowest for the ranks.  `stream` forks into them at the start of the
 *     call and waits for them at the end, inside the call, so for the caller
 *     the whole round is ordered on `stream` as usual.
 * Round contexts: slimdp_round_ctx_create makes one on the current device (two
 * non-blocking streams, four events; no device memory); the caller owns it,
 * passes it to slimdp_round and destroys it with slimdp_round_ctx_destroy once
 * the rounds that used it have completed.  Calls that share a context are
 * serialised by a lock inside it while they enqueue and run one after the
 * other on its streams; calls with different contexts are independent, on the
 * host and on the device, as long as their buffers are.  ctx = NULL uses a
 * context that the library creates for the device on first use and keeps
 * until slimdp_round_release_default_ctx is called on that device (or the
 * process ends): the one piece of state the library keeps by itself.
 *   w_global [n] (updated in place); grads HOST array of K device pointers [n] (read)
 *   scores [n] scratch (see above); core_idx [k_core], core_aux (written; as slimdp_select_core)
 *   exp_idx HOST array of K device pointers [k_exp] (written)
 *   val, pulled HOST arrays of K device pointers [k_core + k_exp] (written)
 *   select_ws, explore_ws: two workspaces that do NOT overlap (both are in use
 *   at once), of at least slimdp_select_workspace_bytes(n) and
 *   slimdp_explore_workspace_bytes(n, k_exp, K) bytes; each keeps the status
 *   word of its step (slimdp_read_status).
 *   stage [stage_bytes] optional scratch, 256-byte aligned, overlapping nothing else */
typedef struct slimdp_round_ctx slimdp_round_ctx;
slimdp_status slimdp_round_ctx_create(slimdp_round_ctx** ctx);
slimdp_status slimdp_round_ctx_destroy(slimdp_round_ctx* ctx);
slimdp_status slimdp_round_release_default_ctx(void);
size_t slimdp_round_stage_bytes(uint64_t n, uint32_t K, uint64_t k_core);
slimdp_status slimdp_round(float* w_global, const float* const* grads, uint32_t K, uint64_t n, float c,
                           uint64_t k_core, uint64_t k_exp, uint64_t seed, uint32_t round, float eta, float* scores,
                           uint32_t* core_idx, void* core_aux, uint32_t* const* exp_idx, float* const* val,
                           float* const* pulled, void* select_ws, size_t select_ws_bytes, void* explore_ws,
                           size_t explore_ws_bytes, void* stage, size_t stage_bytes, slimdp_round_ctx* ctx,
                           void* stream);

/* Measurement aid (the paper has no counterpart).  The next slimdp_round called
 * from this host thread records `begin_event` just before and `end_event` just
 * after its pass over all parameters (the fused scoring + classification
 * kernel, or slimdp_score's kernel on the unfused path) on the round's stream;
 * the request is used up by that call.  Both are cudaEvent_t handles, passed
 * as void*, created by the caller with timing enabled; NULL cancels. */
void slimdp_mark_dominant_kernel(void* begin_event, void* end_event);

/* ----------------------------------------------------- whole round, host ---
 * One whole round (score, select, K x explore, then the exchange: K x pack,
 * merge, K x pull) on HOST buffers: copies w and the K updates to the device, runs
 * slimdp_round, copies the results back, and synchronises before returning.
 *   w_host       HOST [n]: global model, replaced by the merged model
 *   grads_host   HOST array of K HOST pointers, each [n]
 *   core_idx_host HOST [k_core] (written)
 *   exp_idx_host  HOST array of K HOST pointers, each [k_exp] (written)
 *   pulled_host   HOST array of K HOST pointers, each [k_core + k_exp] (written)
 *   arena         DEVICE scratch of at least slimdp_round_arena_bytes(n, K, k_core, k_exp) bytes, 256-byte aligned
 * Host buffers should be page-locked for full copy bandwidth. */
size_t slimdp_round_arena_bytes(uint64_t n, uint32_t K, uint64_t k_core, uint64_t k_exp);
slimdp_status slimdp_round_host(float* w_host, const float* const* grads_host, uint32_t K, uint64_t n, float c,
                                uint64_t k_core, uint64_t k_exp, uint64_t seed, uint32_t round, float eta,
                                uint32_t* core_idx_host, uint32_t* const* exp_idx_host,
                                float* const* pulled_host, void* arena, size_t arena_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SLIMDP_H_ */
