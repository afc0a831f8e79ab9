// Slim-DP communication round: the plain CPU oracle.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, single-threaded, obviously
// correct statement of what one Slim-DP communication round computes.  It is
// used by the test-suite, by the smoke check and by the benchmark's CPU
// baseline leg, and by nothing else: the CUDA library neither includes, links
// nor calls it, and it shares no code, table or constant generator with the
// CUDA sources.  Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC.
//
// Where the paper gives a plain definition the function below is that
// definition written out:
//   score   Eq. 1 (Section 3.2):  S_i = |w_i| + c |g_i|
//   select  Section 3.2: rank all parameters by S_i, keep the top beta*n (full sort)
//   pack    Section 3.1 / 3.5: T_C(delta_k) = the updates on core U explorer
//   merge   Section 3.3 step 3: w <- w - eta' * T_C(delta_k), every worker, k ascending
//   pull    Section 3.3 step 4: T_C(w) = the merged values on core U explorer
//   dense   Section 2.1: Plump-DP pushes and merges every parameter
//   worker merge  Section 3.3 step 5: pulled values overwrite the local model on T_C
// Readings the paper leaves open (all also listed in the design notes):
//   * g_i is the fp32 sum of the K workers' dense updates, k ascending
//     (Section 3.3 step 6 scores with the updates pushed densely before reselection);
//   * score arithmetic is fp32: left-to-right sum, then one fused multiply-add;
//     a NaN score is stored as 0x7FC00000 and ranks above +inf;
//   * a NaN result of a server update is stored as 0x7FC00000 as well (pack and pull move
//     bits and keep whatever payload they find);
//   * ties in the ranking are broken by ascending parameter index;
//   * the explorer (Section 3.1 item 2, Section 3.3 step 2: a random subset of
//     the parameters outside the core, drawn anew per worker and per
//     communication) is an exact-size uniform subset: the first k_exp images
//     of a keyed pseudo-random permutation of the M = n - k_core non-core
//     ranks (an alternating Feistel network on the smallest power-of-two
//     domain that holds M, with cycle walking).  The paper fixes only "random, outside the core"; the generator
//     (Philox-4x32-10 round keys feeding a cycle-walking Feistel network) is
//     this library's own definition.  It is pinned by the generator's
//     published known answers, by exhaustive bijection checks, by an
//     independent big-integer restatement in the tests, and by a chi-square
//     test of uniform inclusion; the paper prints no sequence to compare with.
//
// Indices are 0-based here (the paper's i in {1..n} is i-1).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

inline uint32_t f32_bits(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    return u;
}
inline float bits_f32(uint32_t u) {
    float x;
    std::memcpy(&x, &u, 4);
    return x;
}

// Philox-4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
// easy as 1, 2, 3", SC'11): ten rounds of two 32x32->64 multiplies, with the
// key bumped by the Weyl constants between rounds.
void philox4x32_10(const uint32_t key_in[2], const uint32_t ctr_in[4], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t k0 = key_in[0], k1 = key_in[1];
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = M0 * c0;
        uint64_t p1 = M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        if (r < 9) { k0 += W0; k1 += W1; }
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

const int FEISTEL_ROUNDS = 10;
const uint32_t STREAM_TAG = 0x534C494Du;

// Twelve round-key words for (seed, worker, round): three Philox blocks with
// key = (seed low word, seed high word), counter = (block, worker, round, tag).
void round_keys(uint64_t seed, uint32_t worker, uint32_t round, uint32_t rk[12]) {
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (uint32_t b = 0; b < 3; ++b) {
        uint32_t ctr[4] = {b, worker, round, STREAM_TAG};
        philox4x32_10(key, ctr, rk + 4 * b);
    }
}

// Width of the Feistel domain for M ranks: b = least integer >= 2 with 2^b >= M.
// The network permutes [0, 2^b): x = A * 2^c + B with A of a = floor(b / 2) bits
// and B of c = b - a bits.
int domain_bits(uint64_t M) {
    int b = 2;
    while (((uint64_t)1 << b) < M) ++b;
    return b;
}

// Round function: both halves of the 64-bit product of v with the round's multiplier, folded.
uint32_t round_function(uint32_t v, int r) {
    const uint64_t mult = (r % 2 == 0) ? 0xD2511F53u : 0xCD9E8D57u;
    const uint64_t p = (uint64_t)v * mult;
    return (uint32_t)(p >> 32) ^ (uint32_t)p;
}

// pi(j) on [0, M): apply the alternating Feistel network to j (even rounds change A by a
// function of B, odd rounds change B by a function of A; each round is invertible, so the
// network is a bijection of [0, 2^b) for any split), and while the image falls outside
// [0, M) apply it again (cycle walking).
uint64_t feistel_perm(uint64_t j, uint64_t M, const uint32_t rk[12]) {
    const int b = domain_bits(M);
    const int a = b / 2, c = b - a;
    const uint32_t maskA = (uint32_t)(((uint64_t)1 << a) - 1);
    const uint32_t maskB = (uint32_t)(((uint64_t)1 << c) - 1);
    uint64_t x = j;
    do {
        uint32_t A = (uint32_t)(x >> c);
        uint32_t B = (uint32_t)(x & maskB);
        for (int r = 0; r < FEISTEL_ROUNDS; ++r) {
            if (r % 2 == 0)
                A = (A ^ round_function(B ^ rk[r], r)) & maskA;
            else
                B = (B ^ round_function(A ^ rk[r], r)) & maskB;
        }
        x = ((uint64_t)A << c) | B;
    } while (x >= M);
    return x;
}

// A merged model value as stored: a NaN result of an update becomes the canonical quiet NaN
// (IEEE 754 leaves the payload that an operation passes on to the implementation; Section 3.3
// step 3 defines the value only), exactly as a NaN score does.
inline float stored_model_value(float x) { return std::isnan(x) ? bits_f32(0x7FC00000u) : x; }

struct Ranked {
    uint32_t key;   // bit pattern of the score
    uint32_t idx;   // parameter index
};

}  // namespace

extern "C" {

void oracle_philox4x32_10(const uint32_t* key, const uint32_t* ctr, uint32_t* out) {
    philox4x32_10(key, ctr, out);
}

void oracle_round_keys(uint64_t seed, uint32_t worker, uint32_t round, uint32_t* rk) {
    round_keys(seed, worker, round, rk);
}

uint64_t oracle_feistel_perm(uint64_t j, uint64_t M, const uint32_t* rk) {
    return feistel_perm(j, M, rk);
}

// Eq. 1.  grads: K pointers to float[n].
void oracle_score(const float* w, const float* const* grads, uint32_t K, float c, uint64_t n, float* scores) {
    for (uint64_t i = 0; i < n; ++i) {
        float g = grads[0][i];
        for (uint32_t k = 1; k < K; ++k) g = g + grads[k][i];
        float s = std::fmaf(c, std::fabs(g), std::fabs(w[i]));
        if (std::isnan(s)) s = bits_f32(0x7FC00000u);
        scores[i] = s;
    }
}

// Section 3.2: sort every parameter by (score descending, index ascending),
// keep the first k_core, report them in ascending index order.  Scores are
// >= +0 or the canonical NaN, so the unsigned bit pattern orders them.
void oracle_select_core(const float* scores, uint64_t n, uint64_t k_core, uint32_t* core_idx) {
    std::vector<Ranked> v(n);
    for (uint64_t i = 0; i < n; ++i) {
        v[i].key = f32_bits(scores[i]);
        v[i].idx = (uint32_t)i;
    }
    std::sort(v.begin(), v.end(), [](const Ranked& a, const Ranked& b) {
        if (a.key != b.key) return a.key > b.key;
        return a.idx < b.idx;
    });
    for (uint64_t j = 0; j < k_core; ++j) core_idx[j] = v[j].idx;
    std::sort(core_idx, core_idx + k_core);
}

// A "model-specific significance measure" (Section 5) in its simplest form: the ranking of
// Section 3.2 done per layer.  The vector is cut into segments [seg_off[s], seg_off[s+1]); segment
// s contributes its seg_k[s] parameters of largest score (ties to the smaller index); the core is
// the union, ascending.
void oracle_select_core_segmented(const float* scores, uint64_t n, const uint64_t* seg_off, const uint64_t* seg_k,
                                  uint32_t segments, uint32_t* core_idx) {
    (void)n;
    uint64_t out = 0;
    for (uint32_t s = 0; s < segments; ++s) {
        const uint64_t b = seg_off[s], e = seg_off[s + 1];
        std::vector<Ranked> v(e - b);
        for (uint64_t i = b; i < e; ++i) {
            v[i - b].key = f32_bits(scores[i]);
            v[i - b].idx = (uint32_t)i;
        }
        std::sort(v.begin(), v.end(), [](const Ranked& x, const Ranked& y) {
            if (x.key != y.key) return x.key > y.key;
            return x.idx < y.idx;
        });
        for (uint64_t j = 0; j < seg_k[s]; ++j) core_idx[out + j] = v[j].idx;
        std::sort(core_idx + out, core_idx + out + seg_k[s]);
        out += seg_k[s];
    }
}

// Section 3.3 step 2: worker `worker`'s explorer for communication `round`.
// core_idx ascending.  noncore = ascending complement; explorer =
// { noncore[pi(j)] : j < k_exp }, ascending.
void oracle_sample_explore(const uint32_t* core_idx, uint64_t n, uint64_t k_core, uint64_t k_exp,
                           uint64_t seed, uint32_t worker, uint32_t round, uint32_t* exp_idx) {
    if (k_exp == 0) return;
    const uint64_t M = n - k_core;
    std::vector<uint32_t> noncore;
    noncore.reserve(M);
    uint64_t c = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (c < k_core && core_idx[c] == i) { ++c; continue; }
        noncore.push_back((uint32_t)i);
    }
    uint32_t rk[12];
    round_keys(seed, worker, round, rk);
    for (uint64_t j = 0; j < k_exp; ++j) exp_idx[j] = noncore[feistel_perm(j, M, rk)];
    std::sort(exp_idx, exp_idx + k_exp);
}

// T_C(delta_k): core values first, explorer values second.
void oracle_pack(const float* delta, const uint32_t* core_idx, uint64_t k_core,
                 const uint32_t* exp_idx, uint64_t k_exp, float* val) {
    for (uint64_t j = 0; j < k_core; ++j) val[j] = delta[core_idx[j]];
    for (uint64_t j = 0; j < k_exp; ++j) val[k_core + j] = delta[exp_idx[j]];
}

// Section 3.3 step 3: every worker's push applied to the global model, k ascending.
void oracle_merge(float* w, uint32_t K, const uint32_t* core_idx, uint64_t k_core,
                  const uint32_t* const* exp_idx, uint64_t k_exp, const float* const* val, float eta) {
    for (uint32_t k = 0; k < K; ++k) {
        for (uint64_t j = 0; j < k_core; ++j) {
            uint32_t i = core_idx[j];
            w[i] = stored_model_value(std::fmaf(-eta, val[k][j], w[i]));
        }
        for (uint64_t j = 0; j < k_exp; ++j) {
            uint32_t i = exp_idx[k][j];
            w[i] = stored_model_value(std::fmaf(-eta, val[k][k_core + j], w[i]));
        }
    }
}

// T_C(w) after the merge.
void oracle_pull(const float* w, const uint32_t* core_idx, uint64_t k_core,
                 const uint32_t* exp_idx, uint64_t k_exp, float* out) {
    for (uint64_t j = 0; j < k_core; ++j) out[j] = w[core_idx[j]];
    for (uint64_t j = 0; j < k_exp; ++j) out[k_core + j] = w[exp_idx[j]];
}

// Worker-side Merge (Algorithm 1; Section 3.3 step 5), read as: the pulled values replace the
// local model's values on the communication set, the rest of the local model is untouched.
void oracle_worker_merge(float* w_local, const uint32_t* core_idx, uint64_t k_core, const uint32_t* exp_idx,
                         uint64_t k_exp, const float* pulled) {
    for (uint64_t j = 0; j < k_core; ++j) w_local[core_idx[j]] = pulled[j];
    for (uint64_t j = 0; j < k_exp; ++j) w_local[exp_idx[j]] = pulled[k_core + j];
}

// Key caching (Section 3.5): signature of a key list, the wrapping sum over positions j of
// mix64(((j << 32) | key_j) + 0x9E3779B97F4A7C15), mix64 = the SplitMix64 output function.
uint64_t oracle_core_signature(const uint32_t* keys, uint64_t count) {
    uint64_t sig = 0;
    for (uint64_t j = 0; j < count; ++j) {
        uint64_t z = ((j << 32) | (uint64_t)keys[j]) + 0x9E3779B97F4A7C15ull;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        z = z ^ (z >> 31);
        sig += z;
    }
    return sig;
}

// ---- one worker's push as a message (Section 3.5: values + a signature of the cached keys for
// the core, <key, value> pairs for the explorer) ------------------------------------------------
// Layout, little-endian, every field 4-byte aligned:
//    0 u32 magic 0x57504453 ("SDPW")      4 u32 flags (bit 0: the core's keys are included)
//    8 u64 signature of the sender's core keys
//   16 u32 k_core   20 u32 k_exp   24 u32 worker   28 u32 round
//   32 [k_core x u32 keys, if flags bit 0]  k_core x f32 values  k_exp x (u32 key, f32 value)
// so a push costs 32 + 4 k_core + 8 k_exp bytes = (2 alpha - beta) n words plus the header when the
// receiver's cached keys are current, and 4 k_core more when they have to be sent again.
uint64_t oracle_wire_message_bytes(uint64_t k_core, uint64_t k_exp, int with_keys) {
    return 32 + 4 * k_core * (with_keys ? 2 : 1) + 8 * k_exp;
}

static void put_u32(uint8_t* p, uint32_t v) {
    for (int b = 0; b < 4; ++b) p[b] = (uint8_t)(v >> (8 * b));
}
static uint32_t get_u32(const uint8_t* p) {
    uint32_t v = 0;
    for (int b = 0; b < 4; ++b) v |= (uint32_t)p[b] << (8 * b);
    return v;
}

void oracle_wire_pack(const uint32_t* core_idx, uint64_t k_core, const uint32_t* exp_idx, uint64_t k_exp,
                      const float* val, uint32_t worker, uint32_t round, int with_keys, uint8_t* msg) {
    const uint64_t sig = oracle_core_signature(core_idx, k_core);
    put_u32(msg + 0, 0x57504453u);
    put_u32(msg + 4, with_keys ? 1u : 0u);
    put_u32(msg + 8, (uint32_t)sig);
    put_u32(msg + 12, (uint32_t)(sig >> 32));
    put_u32(msg + 16, (uint32_t)k_core);
    put_u32(msg + 20, (uint32_t)k_exp);
    put_u32(msg + 24, worker);
    put_u32(msg + 28, round);
    uint8_t* p = msg + 32;
    if (with_keys)
        for (uint64_t j = 0; j < k_core; ++j, p += 4) put_u32(p, core_idx[j]);
    for (uint64_t j = 0; j < k_core; ++j, p += 4) put_u32(p, f32_bits(val[j]));
    for (uint64_t j = 0; j < k_exp; ++j, p += 8) {
        put_u32(p, exp_idx[j]);
        put_u32(p + 4, f32_bits(val[k_core + j]));
    }
}

// The receiver's side.  Returns 0 when the message was taken apart (val, exp_idx and, if the
// message carried the keys, core_idx and *signature_out written), 1 when the sender's keys are not
// the ones the receiver has cached and the message does not carry them ("keys wanted": nothing is
// written; the sender's next push includes the keys), -1 when the message is malformed (magic,
// sizes, or included keys that do not give the signature in the header).
int32_t oracle_wire_unpack(const uint8_t* msg, uint64_t msg_bytes, uint64_t cached_signature, uint64_t k_core,
                           uint64_t k_exp, uint32_t* core_idx, uint32_t* exp_idx, float* val,
                           uint64_t* signature_out) {
    if (msg_bytes < 32 || get_u32(msg) != 0x57504453u) return -1;
    const uint32_t flags = get_u32(msg + 4);
    const uint64_t sig = (uint64_t)get_u32(msg + 8) | ((uint64_t)get_u32(msg + 12) << 32);
    if (flags > 1u || get_u32(msg + 16) != k_core || get_u32(msg + 20) != k_exp) return -1;
    if (msg_bytes != oracle_wire_message_bytes(k_core, k_exp, (int)flags)) return -1;
    const uint8_t* p = msg + 32;
    if (flags & 1u) {
        std::vector<uint32_t> keys(k_core);
        for (uint64_t j = 0; j < k_core; ++j) keys[j] = get_u32(p + 4 * j);
        if (oracle_core_signature(keys.data(), k_core) != sig) return -1;
        for (uint64_t j = 0; j < k_core; ++j) core_idx[j] = keys[j];
        *signature_out = sig;
        p += 4 * k_core;
    } else if (sig != cached_signature) {
        return 1;
    }
    for (uint64_t j = 0; j < k_core; ++j, p += 4) val[j] = bits_f32(get_u32(p));
    for (uint64_t j = 0; j < k_exp; ++j, p += 8) {
        exp_idx[j] = get_u32(p);
        val[k_core + j] = bits_f32(get_u32(p + 4));
    }
    return 0;
}

// ---- 8-bit codes for the pushed values ---------------------------------------------------------
// Section 2.2 ends by noting that the method combines with quantisation of what is sent; the paper
// defines no quantiser, so this library fixes one (deterministic, so that both sides agree bit for
// bit): the packed values are cut into buckets of `bucket` consecutive entries; a bucket's scale is
// the largest finite magnitude in it; a value becomes the signed 8-bit code
//     rint(v * (127 / scale)) clamped to [-127, 127]    (fp32 division, fp32 product, ties to even),
// 0 if the scale is 0 or v is a NaN; an infinity gets +-127.  The receiver reads code * (scale / 127).
void oracle_quantize_q8(const float* val, uint64_t m, uint32_t bucket, int8_t* codes, float* scales) {
    for (uint64_t b0 = 0, b = 0; b0 < m; b0 += bucket, ++b) {
        const uint64_t b1 = (b0 + bucket < m) ? b0 + bucket : m;
        float amax = 0.0f;
        for (uint64_t j = b0; j < b1; ++j) {
            const float a = std::fabs(val[j]);
            if (a <= 3.402823466e+38f && a > amax) amax = a;   // NaNs and infinities do not set the scale
        }
        scales[b] = amax;
        const float inv = (amax > 0.0f) ? 127.0f / amax : 0.0f;
        for (uint64_t j = b0; j < b1; ++j) {
            const float v = val[j];
            float q;
            if (std::isnan(v))
                q = 0.0f;
            else if (std::isinf(v))
                q = (v > 0.0f) ? 127.0f : -127.0f;   // whatever the scale, 0 included
            else
                q = std::rint(v * inv);
            if (q > 127.0f) q = 127.0f;
            if (q < -127.0f) q = -127.0f;
            codes[j] = (int8_t)q;
        }
    }
}

void oracle_dequantize_q8(const int8_t* codes, const float* scales, uint64_t m, uint32_t bucket, float* val) {
    for (uint64_t j = 0; j < m; ++j) {
        const float step = scales[j / bucket] / 127.0f;
        val[j] = (float)codes[j] * step;
    }
}

// Plump-DP (Section 2.1): every worker pushes its whole update.
void oracle_dense_merge(float* w, uint64_t n, uint32_t K, const float* const* grads, float eta) {
    for (uint32_t k = 0; k < K; ++k)
        for (uint64_t i = 0; i < n; ++i) w[i] = stored_model_value(std::fmaf(-eta, grads[k][i], w[i]));
}

}  // extern "C"
