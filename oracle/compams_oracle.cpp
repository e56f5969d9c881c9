// CPU oracle for one COMP-AMS optimizer step.
//
// THIS FILE IS TEST INFRASTRUCTURE. It is a plain, slow, single-purpose restatement of the
// paper's method (Algorithm 2 with the compressors of Definitions 1 and 2 and the AMSGrad update
// of Algorithm 1), written to be checked against the paper by eye. It shares no code with the
// CUDA library, and only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
//
// Arithmetic: all state is fp32 and every fp32 operation below is a separate, correctly rounded
// IEEE operation (build with -ffp-contract=off, no fast-math), because the method is specified on
// fp32 tensors and its compressed outputs (index sets, sign bits) must be reproducible bit for bit.
// Reductions that the paper writes as exact sums (the block L1 norm of Definition 2, the average
// over workers in Algorithm 2) are accumulated wider than fp32 and rounded once.
//
// Random-k (named among the deterministic sparsifiers in Section 2.1, not defined further) is this build's
// reading, stated at randk_block below; its pins: the generator against an independent library
// implementation, the index map being a bijection by brute force, set size, reproducibility and a
// chi-square bound on the inclusion frequencies.
//
// Parity pins (tests/test_oracle_*.py): Top-k against brute force on tiny inputs; the error-feedback
// identity C(x) + e_new = x (proof of Theorem 1); Block-Sign L1 preservation (Section 3.1); the
// q-deviate bounds of Remark 1; the k = d and d_i = 1 identity cases (Assumption 1, q = 0);
// AMSGrad against closed forms at t = 1 and a hand-computed two-step example (Algorithm 1).
// The five full-size workloads themselves have no printed reference values in the paper: for
// them the result is "parity unpinned" beyond these pins.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <new>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { COMPRESSOR_TOPK = 0, COMPRESSOR_BLOCKSIGN = 1, COMPRESSOR_RANDK = 2 };

inline uint32_t float_bits(float x) {
    uint32_t u;
    std::memcpy(&u, &x, sizeof u);
    return u;
}

// Magnitude key: the fp32 bit pattern with the sign bit cleared. For finite values it is
// monotone in |x| when compared as an unsigned integer; +0 and -0 share key 0.
inline uint32_t magnitude_key(float x) { return float_bits(x) & 0x7fffffffu; }

// Number of coordinates Top-k keeps in a block of size d_b for a given ratio:
// floor(ratio * d_b), at least 1 and at most d_b (Section 5.1: "top 1% gradient coordinates").
inline int64_t kept_per_block(double k_ratio, int64_t d_b) {
    int64_t k = (int64_t)std::floor(k_ratio * (double)d_b);
    if (k < 1) k = 1;
    if (k > d_b) k = d_b;
    return k;
}

// Definition 1 (Top-k) on one block x[0..len): marks in keep[] the k coordinates of largest
// magnitude. Among equal magnitudes the lower index wins, which makes the set unique.
// Each coordinate becomes one 64-bit composite (key << 32 | ~index); the k largest composites
// are exactly: larger key first, then smaller index.
void topk_block(const float* x, int64_t len, int64_t k, uint8_t* keep) {
    std::vector<uint64_t> comp((size_t)len);
    for (int64_t j = 0; j < len; ++j)
        comp[(size_t)j] = ((uint64_t)magnitude_key(x[j]) << 32) | (uint64_t)(0xffffffffu - (uint32_t)j);
    if (k < len)
        std::nth_element(comp.begin(), comp.begin() + k, comp.end(), std::greater<uint64_t>());
    std::memset(keep, 0, (size_t)len);
    for (int64_t r = 0; r < k; ++r) {
        uint32_t j = 0xffffffffu - (uint32_t)(comp[(size_t)r] & 0xffffffffu);
        keep[j] = 1;
    }
}

// Definition 2 (Block-Sign) scale of one block: ||x_B||_1 / d_B.
// The L1 norm is summed without rounding: every fp32 magnitude is mant * 2^(E-150) with a 24-bit
// integer mant, so the mantissas are added as integers per exponent E (exact for any realistic
// length), and the 256 per-exponent totals are combined in long double from the smallest up.
// One division in long double, one rounding to fp32.
float blocksign_scale(const float* x, int64_t len) {
    uint64_t bucket[256];
    std::memset(bucket, 0, sizeof bucket);
    for (int64_t j = 0; j < len; ++j) {
        uint32_t key = magnitude_key(x[j]);
        uint32_t e = key >> 23;
        uint32_t frac = key & 0x7fffffu;
        bucket[e] += e ? (uint64_t)(frac | 0x800000u) : (uint64_t)frac;  // e = 0: subnormal, no hidden bit
    }
    long double S = 0.0L;
    for (int e = 0; e < 256; ++e) {
        if (!bucket[e]) continue;
        int exp2 = (e ? e : 1) - 150;
        S += std::ldexp((long double)bucket[e], exp2);
    }
    return (float)(S / (long double)len);
}

// Philox4x64-10, the counter-based generator of Salmon, Moraes, Dror and Shaw ("Parallel random numbers:
// as easy as 1, 2, 3", SC 2011): a 256-bit counter and a 128-bit key give 256 pseudorandom bits. Ten
// rounds; each multiplies two counter words by fixed odd constants, crosses the high and low halves
// with the other two words and the key, and the key advances by Weyl constants between rounds.
void philox4x64_10(const uint64_t ctr[4], const uint64_t key[2], uint64_t out[4]) {
    const uint64_t M0 = 0xD2E7470EE14C6C93ull, M1 = 0xCA5A826395121157ull;
    const uint64_t W0 = 0x9E3779B97F4A7C15ull, W1 = 0xBB67AE8584CAA73Bull;
    uint64_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += W0;
            k1 += W1;
        }
        const unsigned __int128 p0 = (unsigned __int128)M0 * c0, p1 = (unsigned __int128)M1 * c2;
        const uint64_t hi0 = (uint64_t)(p0 >> 64), lo0 = (uint64_t)p0, hi1 = (uint64_t)(p1 >> 64), lo1 = (uint64_t)p1;
        const uint64_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The 32-bit finalizer of MurmurHash3 (Appleby): a bijection of the 32-bit words that mixes every input bit
// into every output bit.
inline uint32_t fmix32(uint32_t h) {
    h ^= h >> 16;
    h *= 0x85ebca6bu;
    h ^= h >> 13;
    h *= 0xc2b2ae35u;
    h ^= h >> 16;
    return h;
}

// The six 32-bit round keys of (seed, step, worker, block): the low and high halves of the first three words
// of one Philox4x64-10 block at counter (0, 0, block, worker) under key (seed, step).
void randk_round_keys(uint64_t seed, uint64_t step, uint64_t worker, uint64_t block, uint32_t keys[6]) {
    const uint64_t ctr[4] = {0, 0, block, worker};
    const uint64_t key[2] = {seed, step};
    uint64_t w[4];
    philox4x64_10(ctr, key, w);
    for (int r = 0; r < 6; ++r) keys[r] = (uint32_t)(r & 1 ? w[r >> 1] >> 32 : w[r >> 1]);
}

// A keyed pseudorandom permutation of {0, ..., m-1}, m < 2^32: a balanced Feistel network of six rounds over the
// smallest even number of bits 2w with 2^(2w) >= m (at least 2), round r mapping (L, R) to
// (R, L xor (fmix32(R xor key_r) mod 2^w)); a result outside [0, m) is fed through the network again until it
// falls inside (cycle walking), which makes the restriction to [0, m) a bijection.
uint64_t randk_permute_keyed(uint64_t m, uint64_t r, const uint32_t keys[6]) {
    int bits = 2;
    while (bits < 32 && ((uint64_t)1 << bits) < m) bits += 2;
    const int w = bits / 2;
    const uint32_t mask = ((uint32_t)1 << w) - 1;
    uint32_t x = (uint32_t)r;
    do {
        uint32_t L = x >> w, R = x & mask;
        for (int round = 0; round < 6; ++round) {
            const uint32_t nR = L ^ (fmix32(R ^ keys[round]) & mask);
            L = R;
            R = nR;
        }
        x = (L << w) | R;
    } while (x >= m);
    return x;
}

uint64_t randk_permute(uint64_t m, uint64_t r, uint64_t seed, uint64_t step, uint64_t worker, uint64_t block) {
    uint32_t keys[6];
    randk_round_keys(seed, step, worker, block, keys);
    return randk_permute_keyed(m, r, keys);
}

// Random-k on one block of `len` coordinates: the kept set is { pi(r) : r = 0 .. k-1 }, pi the permutation
// above for this (seed, step, worker, block): k distinct coordinates, every k-subset (nearly) equally
// likely, the same set whenever the four identifiers are the same. The values play no part.
void randk_block(int64_t len, int64_t k, uint64_t seed, uint64_t step, uint64_t worker, uint64_t block, uint8_t* keep) {
    std::memset(keep, 0, (size_t)len);
    uint32_t keys[6];
    randk_round_keys(seed, step, worker, block, keys);
    for (int64_t r = 0; r < k; ++r) keep[randk_permute_keyed((uint64_t)len, (uint64_t)r, keys)] = 1;
}

struct Oracle {
    int32_t n = 0;
    int64_t d = 0;
    int32_t M = 0;
    std::vector<int64_t> off;  // M + 1 block offsets
    int32_t compressor = 0;
    double k_ratio = 1.0;
    float lr = 0, beta1 = 0, beta2 = 0, eps = 0;
    uint64_t seed = 0;              // Random-k: the seed of the index sets
    uint64_t steps_done = 0;        // iterations so far; the iteration being computed is steps_done + 1
    int64_t K = 0;                  // sum over blocks of kept_per_block (Top-k and Random-k)
    std::vector<int64_t> seg_off;   // M + 1 prefix sums of kept_per_block
    // Algorithm 2 state
    std::vector<float> E;           // [n, d] error accumulators e_{t,i}
    std::vector<float> m, v, vhat;  // [d] server moments
    // Per-step results kept for inspection
    std::vector<float> C;           // [n, d] compressed gradients g~_{t,i}
    std::vector<float> gbar;        // [d] averaged compressed gradient
    std::vector<float> scales;      // [n, M] Block-Sign scales
    std::vector<int32_t> kept_idx;  // [n, K] Top-k kept coordinates, ascending inside each block segment
};

}  // namespace

extern "C" {

int64_t oracle_kept_per_block(double k_ratio, int64_t d_b) { return kept_per_block(k_ratio, d_b); }

void oracle_topk_block(const float* x, int64_t len, int64_t k, uint8_t* keep) { topk_block(x, len, k, keep); }

float oracle_blocksign_scale(const float* x, int64_t len) { return blocksign_scale(x, len); }

void oracle_philox4x64_10(const uint64_t* ctr, const uint64_t* key, uint64_t* out) { philox4x64_10(ctr, key, out); }

uint64_t oracle_randk_permute(uint64_t m, uint64_t r, uint64_t seed, uint64_t step, uint64_t worker, uint64_t block) {
    return randk_permute(m, r, seed, step, worker, block);
}

void oracle_randk_block(int64_t len, int64_t k, uint64_t seed, uint64_t step, uint64_t worker, uint64_t block,
                        uint8_t* keep) {
    randk_block(len, k, seed, step, worker, block, keep);
}

// Algorithm 1 / Algorithm 2 server update on d coordinates given the (averaged) gradient g:
//   m = beta1*m + (1-beta1)*g;  v = beta2*v + (1-beta2)*g^2;  vhat = max(vhat, v);
//   theta = theta - lr * m / sqrt(vhat + eps)          (eps under the root, no bias correction)
void oracle_amsgrad(int64_t d, const float* g, float* m, float* v, float* vhat, float* theta, float lr,
                    float beta1, float beta2, float eps) {
    const float omb1 = 1.0f - beta1;
    const float omb2 = 1.0f - beta2;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        float gj = g[j];
        float mj = (beta1 * m[j]) + (omb1 * gj);
        float vj = (beta2 * v[j]) + (omb2 * (gj * gj));
        float vh = std::fmax(vhat[j], vj);
        float step = (lr * mj) / std::sqrt(vh + eps);
        m[j] = mj;
        v[j] = vj;
        vhat[j] = vh;
        theta[j] = theta[j] - step;
    }
}

void* oracle_create(int32_t n, int64_t d, const int64_t* block_offsets, int32_t num_blocks, int32_t compressor,
                    double k_ratio, float lr, float beta1, float beta2, float eps) {
    if (n < 1 || d < 1 || d >= ((int64_t)1 << 31) || num_blocks < 1 || !block_offsets) return nullptr;
    if (compressor != COMPRESSOR_TOPK && compressor != COMPRESSOR_BLOCKSIGN && compressor != COMPRESSOR_RANDK) return nullptr;
    if (compressor != COMPRESSOR_BLOCKSIGN && !(k_ratio > 0.0 && k_ratio <= 1.0)) return nullptr;
    if (block_offsets[0] != 0 || block_offsets[num_blocks] != d) return nullptr;
    for (int32_t b = 0; b < num_blocks; ++b)
        if (block_offsets[b + 1] <= block_offsets[b]) return nullptr;
    Oracle* o = new (std::nothrow) Oracle();
    if (!o) return nullptr;
    o->n = n;
    o->d = d;
    o->M = num_blocks;
    o->off.assign(block_offsets, block_offsets + num_blocks + 1);
    o->compressor = compressor;
    o->k_ratio = k_ratio;
    o->lr = lr;
    o->beta1 = beta1;
    o->beta2 = beta2;
    o->eps = eps;
    o->seg_off.assign((size_t)num_blocks + 1, 0);
    if (compressor != COMPRESSOR_BLOCKSIGN)
        for (int32_t b = 0; b < num_blocks; ++b)
            o->seg_off[(size_t)b + 1] = o->seg_off[(size_t)b] + kept_per_block(k_ratio, o->off[b + 1] - o->off[b]);
    o->K = o->seg_off[(size_t)num_blocks];
    // Algorithm 2, initialisation: e_{1,i} = 0, m_0 = v_0 = vhat_0 = 0.
    o->E.assign((size_t)n * (size_t)d, 0.0f);
    o->m.assign((size_t)d, 0.0f);
    o->v.assign((size_t)d, 0.0f);
    o->vhat.assign((size_t)d, 0.0f);
    o->C.assign((size_t)n * (size_t)d, 0.0f);
    o->gbar.assign((size_t)d, 0.0f);
    o->scales.assign((size_t)n * (size_t)num_blocks, 0.0f);
    o->kept_idx.assign((size_t)n * (size_t)o->K, 0);
    return o;
}

void oracle_destroy(void* h) { delete (Oracle*)h; }

// Random-k: the seed of the index sets, and the number of iterations done so far (the next oracle_step is
// iteration steps_done + 1; a run resumed from a checkpoint sets it to where the checkpoint was taken).
void oracle_set_seed(void* h, uint64_t seed, uint64_t steps_done) {
    if (!h) return;
    ((Oracle*)h)->seed = seed;
    ((Oracle*)h)->steps_done = steps_done;
}

// Algorithm 2 takes a learning rate eta_t per iteration: the value set here is the eta_t of every
// following oracle_step until it is set again (Section 5.1 divides it by 10 at fixed epochs).
void oracle_set_lr(void* h, float lr) {
    if (h) ((Oracle*)h)->lr = lr;
}

// One iteration t of Algorithm 2 given the workers' stochastic gradients G [n, d] (row i = g_{t,i})
// and the server parameters theta [d], which are updated in place.
int oracle_step(void* h, const float* G, float* theta) {
    Oracle* o = (Oracle*)h;
    if (!o || !G || !theta) return -1;
    const int32_t n = o->n;
    const int64_t d = o->d;
    const int32_t M = o->M;
    const uint64_t t = ++o->steps_done;  // the iteration index, from 1

    // "parallel for worker i in [n]": the workers are independent until the server averages.
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t i = 0; i < n; ++i) {
        const float* g = G + (size_t)i * (size_t)d;
        float* e = o->E.data() + (size_t)i * (size_t)d;
        float* c = o->C.data() + (size_t)i * (size_t)d;
        std::vector<float> x((size_t)d);
        // Error feedback: the corrected gradient x = g_{t,i} + e_{t,i}.
        for (int64_t j = 0; j < d; ++j) x[(size_t)j] = g[j] + e[j];

        // g~_{t,i} = C(x), block by block.
        for (int32_t b = 0; b < M; ++b) {
            const int64_t lo = o->off[(size_t)b], len = o->off[(size_t)b + 1] - lo;
            const float* xb = x.data() + lo;
            if (o->compressor == COMPRESSOR_TOPK || o->compressor == COMPRESSOR_RANDK) {
                const int64_t k = o->seg_off[(size_t)b + 1] - o->seg_off[(size_t)b];
                std::vector<uint8_t> keep((size_t)len);
                if (o->compressor == COMPRESSOR_TOPK)
                    topk_block(xb, len, k, keep.data());
                else
                    randk_block(len, k, o->seed, t, (uint64_t)i, (uint64_t)b, keep.data());
                int32_t* out = o->kept_idx.data() + (size_t)i * (size_t)o->K + o->seg_off[(size_t)b];
                int64_t r = 0;
                for (int64_t j = 0; j < len; ++j) {
                    if (keep[(size_t)j]) {
                        c[lo + j] = xb[j];
                        out[r++] = (int32_t)(lo + j);
                    } else {
                        c[lo + j] = 0.0f;
                    }
                }
            } else {
                const float s = blocksign_scale(xb, len);
                o->scales[(size_t)i * (size_t)M + (size_t)b] = s;
                // sign(x) * s with the IEEE sign bit deciding, so sign(+0) = +1 and sign(-0) = -1:
                // every coordinate carries exactly one bit and ||C(x)_B||_1 = ||x_B||_1.
                for (int64_t j = 0; j < len; ++j) c[lo + j] = std::copysign(s, xb[j]);
            }
        }

        // e_{t+1,i} = e_{t,i} + g_{t,i} - g~_{t,i}, evaluated as (g + e) - g~ with x already rounded.
        // For a kept Top-k coordinate x - x is +0; for a dropped one x - 0 is x.
        for (int64_t j = 0; j < d; ++j) e[j] = x[(size_t)j] - c[j];
    }

    // Server: gbar_t = (1/n) * sum_i g~_{t,i}. The sum over workers is taken in binary64 (exact for
    // these term counts and magnitudes, hence independent of the order), rounded to fp32 once, and
    // divided by n in fp32.
    const float nf = (float)n;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        double acc = 0.0;
        for (int32_t i = 0; i < n; ++i) acc += (double)o->C[(size_t)i * (size_t)d + (size_t)j];
        o->gbar[(size_t)j] = (float)acc / nf;
    }

    // Server: AMSGrad update with gbar_t.
    oracle_amsgrad(d, o->gbar.data(), o->m.data(), o->v.data(), o->vhat.data(), theta, o->lr, o->beta1, o->beta2,
                   o->eps);
    return 0;
}

// Views of the oracle's buffers. which: 0 E [n*d], 1 m, 2 v, 3 vhat, 4 gbar [d], 5 C [n*d],
// 6 scales [n*M], 7 kept_idx [n*K] (int32), 8 seg_off [M+1] (int64).
void* oracle_buffer(void* h, int32_t which, int64_t* count) {
    Oracle* o = (Oracle*)h;
    if (!o) return nullptr;
    switch (which) {
        case 0: *count = (int64_t)o->E.size(); return o->E.data();
        case 1: *count = (int64_t)o->m.size(); return o->m.data();
        case 2: *count = (int64_t)o->v.size(); return o->v.data();
        case 3: *count = (int64_t)o->vhat.size(); return o->vhat.data();
        case 4: *count = (int64_t)o->gbar.size(); return o->gbar.data();
        case 5: *count = (int64_t)o->C.size(); return o->C.data();
        case 6: *count = (int64_t)o->scales.size(); return o->scales.data();
        case 7: *count = (int64_t)o->kept_idx.size(); return o->kept_idx.data();
        case 8: *count = (int64_t)o->seg_off.size(); return o->seg_off.data();
        default: return nullptr;
    }
}

void oracle_set_threads(int32_t t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

int32_t oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
