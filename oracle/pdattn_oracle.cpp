// TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// Plain, slow, fp64 CPU statement of what paged decode attention computes:
//
//     out[s,h,:] = softmax_t( scale * <q[s,h,:], K_s[t,h/G,:]> ) . V_s[t,h/G,:],   t in [0, L_s)
//
// where token t of sequence s lives in physical page block_table[s, t / bs] at slot
// t % bs (the paged KV cache of the rollout engine: Section 2.1 and Section 2.3 describe the
// autoregressive decoding this serves; Appendix A.1.2 gives the cache's per-token footprint
// 2*L*H_kv*d_head*b_dtype/tp that fixes the layout's size).  The split-KV / online-softmax
// method reaches exactly this value up to rounding order, so the oracle is the definition
// written out: a two-pass softmax, no blocking, no rescaling, no splitting.
//
// It shares nothing with the CUDA library: own bf16 helpers, own indexing, no CUDA or torch
// headers.  Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
//
// Pins (tests/test_oracle_pins.py): L = 1 returns V exactly; equal keys / zero scale / zero q
// return the mean of V; page permutation leaves the bits unchanged; dense brute force on tiny
// inputs; L = 2 sigmoid closed form; dominant key; score-shift invariance; convex-hull bound
// and linearity in V; split/merge identity; fp64 library softmax-matmul on an identity table;
// the (sequence, head) pair list against the rows of the full output; the fp8 variants against
// the bf16 path on the decoded values and a dense masked softmax.
//
// Out-of-range block_table entries (id < 0 or id >= num_blocks) inside a sequence's used range
// are not dereferenced: their tokens are left out of the softmax (an explicit mask, not a marker
// value in the scores) and counted in *bad_pages.  Valid inputs are finite; a NaN that reaches a
// live slot all the same propagates to that head's output.

#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);  // exact widening
}

// round-to-nearest-even from double through float's exponent range to bf16
inline uint16_t double_to_bf16_rne(double x) {
    if (std::isnan(x)) return 0x7FC0;
    // Round the double directly to 8 significant bits (avoids double rounding via float).
    if (x == 0.0) return std::signbit(x) ? 0x8000 : 0x0000;
    if (std::isinf(x)) return x > 0 ? 0x7F80 : 0xFF80;
    int e;
    double m = std::frexp(std::fabs(x), &e);      // |x| = m * 2^e, m in [0.5, 1)
    int exp_unb = e - 1;                          // |x| = (2m) * 2^(e-1), 2m in [1,2)
    uint16_t sign = x < 0 ? 0x8000 : 0;
    if (exp_unb < -126) {                         // subnormal in float/bf16 terms
        double scaled = std::ldexp(std::fabs(x), 126 + 7);   // units of 2^-133
        double r = std::nearbyint(scaled);                   // ties-to-even (default mode)
        uint32_t mant = static_cast<uint32_t>(r);
        return static_cast<uint16_t>(sign | mant);           // mant may carry into exponent 1: correct
    }
    double frac = std::ldexp(m, 8);               // in [128, 256): 8 significant bits
    double r = std::nearbyint(frac);
    if (r >= 256.0) { r = 128.0; exp_unb += 1; }
    if (exp_unb > 127) return static_cast<uint16_t>(sign | 0x7F80);
    uint32_t mant = static_cast<uint32_t>(r) - 128u;          // 7 stored bits
    uint32_t expo = static_cast<uint32_t>(exp_unb + 127);
    return static_cast<uint16_t>(sign | (expo << 7) | mant);
}

struct Problem {
    const uint16_t *q, *k, *v;
    const int32_t *block_table, *context_lens;
    int S, Hq, Hkv, d, bs, MB, NB;
    int64_t blk_stride, head_stride, tok_stride;
    double scale;
};

// Scores x_t = scale * <q, k_t> for t in [t0, t1).  live[t - t0] = 0 marks a token whose page id is out
// of range: its score is never computed and it is left out of the softmax.  A NaN that the arithmetic
// itself produces in a live slot stays in x and propagates to the output.
// Returns number of tokens skipped because their page id is out of range.
int64_t scores(const Problem& P, int s, int h, int t0, int t1, std::vector<double>& x, std::vector<char>& live) {
    const int G = P.Hq / P.Hkv;
    const int g = h / G;
    const uint16_t* qrow = P.q + (static_cast<int64_t>(s) * P.Hq + h) * P.d;
    int64_t skipped = 0;
    x.assign(static_cast<size_t>(t1 - t0), 0.0);
    live.assign(static_cast<size_t>(t1 - t0), 1);
    for (int t = t0; t < t1; ++t) {
        int32_t page = P.block_table[static_cast<int64_t>(s) * P.MB + t / P.bs];
        if (page < 0 || page >= P.NB) {
            live[t - t0] = 0;
            ++skipped;
            continue;
        }
        int slot = t % P.bs;
        const uint16_t* krow = P.k + page * P.blk_stride + g * P.head_stride + slot * P.tok_stride;
        double acc = 0.0;
        for (int j = 0; j < P.d; ++j) acc += bf16_to_double(qrow[j]) * bf16_to_double(krow[j]);
        x[t - t0] = P.scale * acc;
    }
    return skipped;
}

// Un-normalised partial over [t0,t1): m = max x, l = sum exp(x-m), acc[j] = sum exp(x-m) v_t[j].
int64_t partial(const Problem& P, int s, int h, int t0, int t1, double* m_out, double* l_out, double* acc) {
    const int G = P.Hq / P.Hkv;
    const int g = h / G;
    std::vector<double> x;
    std::vector<char> live;
    int64_t skipped = scores(P, s, h, t0, t1, x, live);
    // max over the live scores; a NaN among them makes the max (and with it every weight) NaN
    double m = -std::numeric_limits<double>::infinity();
    for (int t = t0; t < t1; ++t) {
        if (!live[t - t0]) continue;
        const double xv = x[t - t0];
        if (std::isnan(xv) || xv > m) m = xv;
        if (std::isnan(m)) break;
    }
    double l = 0.0;
    for (int j = 0; j < P.d; ++j) acc[j] = 0.0;
    for (int t = t0; t < t1; ++t) {
        if (!live[t - t0]) continue;
        double xv = x[t - t0];
        double w = std::exp(xv - m);
        l += w;
        int32_t page = P.block_table[static_cast<int64_t>(s) * P.MB + t / P.bs];
        int slot = t % P.bs;
        const uint16_t* vrow = P.v + page * P.blk_stride + g * P.head_stride + slot * P.tok_stride;
        for (int j = 0; j < P.d; ++j) acc[j] += w * bf16_to_double(vrow[j]);
    }
    *m_out = m;
    *l_out = l;
    return skipped;
}

int64_t one_output(const Problem& P, int s, int h, double* out) {
    int L = P.context_lens[s];
    if (L <= 0) {
        for (int j = 0; j < P.d; ++j) out[j] = 0.0;
        return 0;
    }
    double m, l;
    int64_t skipped = partial(P, s, h, 0, L, &m, &l, out);
    if (l > 0.0 || std::isnan(l)) {
        for (int j = 0; j < P.d; ++j) out[j] /= l;
    } else {
        for (int j = 0; j < P.d; ++j) out[j] = 0.0;   // every token sat in a bad page
    }
    return skipped;
}

}  // namespace

extern "C" {

// Returns 0 on success, -1 on invalid arguments.  All pointers are HOST pointers.
// pairs == NULL: out is [S, Hq, d] doubles.  pairs != NULL: num_pairs (s,h) int32 pairs,
// out is [num_pairs, d] doubles.  bad_pages (optional) receives the number of skipped tokens
// summed over the outputs computed.
int pdattn_oracle_decode(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                         const int32_t* block_table, const int32_t* context_lens,
                         int num_seqs, int num_q_heads, int num_kv_heads, int head_dim, int block_size,
                         int max_blocks_per_seq, int num_blocks,
                         int64_t kv_block_stride, int64_t kv_head_stride, int64_t kv_token_stride,
                         float scale, const int32_t* pairs, int64_t num_pairs,
                         double* out, int num_threads, int64_t* bad_pages) {
    if (num_seqs < 0 || num_q_heads <= 0 || num_kv_heads <= 0 || head_dim <= 0 || block_size <= 0 ||
        num_q_heads % num_kv_heads != 0 || max_blocks_per_seq < 0 || !out)
        return -1;
    Problem P{q, k_cache, v_cache, block_table, context_lens, num_seqs, num_q_heads, num_kv_heads,
              head_dim, block_size, max_blocks_per_seq, num_blocks,
              kv_block_stride, kv_head_stride, kv_token_stride, static_cast<double>(scale)};
    const int64_t total = pairs ? num_pairs : static_cast<int64_t>(num_seqs) * num_q_heads;
    for (int s = 0; s < num_seqs; ++s) {
        int64_t need = (static_cast<int64_t>(context_lens[s]) + block_size - 1) / block_size;
        if (need > max_blocks_per_seq) return -1;
    }
    std::atomic<int64_t> next{0};
    std::atomic<int64_t> skipped{0};
    auto worker = [&]() {
        for (;;) {
            int64_t i = next.fetch_add(1);
            if (i >= total) break;
            int s, h;
            if (pairs) { s = pairs[2 * i]; h = pairs[2 * i + 1]; }
            else { s = static_cast<int>(i / num_q_heads); h = static_cast<int>(i % num_q_heads); }
            skipped += one_output(P, s, h, out + i * head_dim);
        }
    };
    int nt = num_threads > 0 ? num_threads : 1;
    if (nt == 1) {
        worker();
    } else {
        std::vector<std::thread> pool;
        for (int i = 0; i < nt; ++i) pool.emplace_back(worker);
        for (auto& th : pool) th.join();
    }
    if (bad_pages) *bad_pages = skipped.load();
    return 0;
}

// Un-normalised partial of one (s,h) over tokens [t0,t1): natural-log domain max m, sum l, acc[d].
int pdattn_oracle_partial(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                          const int32_t* block_table, const int32_t* context_lens,
                          int num_seqs, int num_q_heads, int num_kv_heads, int head_dim, int block_size,
                          int max_blocks_per_seq, int num_blocks,
                          int64_t kv_block_stride, int64_t kv_head_stride, int64_t kv_token_stride,
                          float scale, int s, int h, int t0, int t1,
                          double* m, double* l, double* acc) {
    if (s < 0 || s >= num_seqs || h < 0 || h >= num_q_heads || t0 < 0 || t1 < t0 || t1 > context_lens[s]) return -1;
    Problem P{q, k_cache, v_cache, block_table, context_lens, num_seqs, num_q_heads, num_kv_heads,
              head_dim, block_size, max_blocks_per_seq, num_blocks,
              kv_block_stride, kv_head_stride, kv_token_stride, static_cast<double>(scale)};
    partial(P, s, h, t0, t1, m, l, acc);
    return 0;
}

// Merge of n partial triples in the order given:
//   M = max_c m_c,  Lsum = sum_c l_c e^(m_c - M),  out = sum_c acc_c e^(m_c - M) / Lsum.
int pdattn_oracle_merge(const double* m, const double* l, const double* acc, int n, int head_dim, double* out) {
    double M = -std::numeric_limits<double>::infinity();
    for (int c = 0; c < n; ++c)
        if (m[c] > M) M = m[c];
    double Lsum = 0.0;
    for (int j = 0; j < head_dim; ++j) out[j] = 0.0;
    for (int c = 0; c < n; ++c) {
        if (!(l[c] > 0.0) && !std::isnan(l[c])) continue;   // an empty partial; a NaN one propagates
        double f = std::exp(m[c] - M);
        Lsum += l[c] * f;
        for (int j = 0; j < head_dim; ++j) out[j] += acc[static_cast<int64_t>(c) * head_dim + j] * f;
    }
    if (Lsum > 0.0 || std::isnan(Lsum))
        for (int j = 0; j < head_dim; ++j) out[j] /= Lsum;
    return 0;
}

uint16_t pdattn_oracle_bf16_rne(double x) { return double_to_bf16_rne(x); }
double pdattn_oracle_bf16_to_double(uint16_t b) { return bf16_to_double(b); }

// ---- fp8 KV cache (the per-token footprint b_kv of Appendix A.1.2 carries the cache dtype's byte size) ----
// K and V are stored as e4m3 codes with one fp32 scale per KV head: real value = scale[g] * e4m3(code).
// e4m3 (the finite-only 8-bit format): 1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits; no infinities;
// S.1111.111 is NaN; exponent field 0 holds the subnormals m/8 * 2^-6.
// Layouts: k8 [num_blocks, num_kv_heads, block_size, head_dim], v8 [num_blocks, num_kv_heads, head_dim, block_size]
// (V is kept transposed inside a page), both dense.
double pdattn_oracle_e4m3_to_double(uint8_t b) {
    const int sign = b >> 7, e = (b >> 3) & 15, m = b & 7;
    if (e == 15 && m == 7) return std::numeric_limits<double>::quiet_NaN();
    const double v = e == 0 ? std::ldexp(static_cast<double>(m), -9) : std::ldexp(static_cast<double>(8 + m), e - 10);
    return sign ? -v : v;
}

int pdattn_oracle_decode_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                             const float* v_scale, const int32_t* block_table, const int32_t* context_lens,
                             int num_seqs, int num_q_heads, int num_kv_heads, int head_dim, int block_size,
                             int max_blocks_per_seq, int num_blocks, float scale, double* out, int num_threads,
                             int64_t* bad_pages) {
    if (num_seqs < 0 || num_q_heads <= 0 || num_kv_heads <= 0 || head_dim <= 0 || block_size <= 0 ||
        num_q_heads % num_kv_heads != 0 || max_blocks_per_seq < 0 || !out || !k_scale || !v_scale)
        return -1;
    const int G = num_q_heads / num_kv_heads, d = head_dim, bs = block_size;
    for (int s = 0; s < num_seqs; ++s)
        if ((static_cast<int64_t>(context_lens[s]) + bs - 1) / bs > max_blocks_per_seq) return -1;
    const int64_t total = static_cast<int64_t>(num_seqs) * num_q_heads;
    std::atomic<int64_t> next{0}, skipped{0};
    auto worker = [&]() {
        std::vector<double> x;
        std::vector<char> live;
        for (;;) {
            const int64_t i = next.fetch_add(1);
            if (i >= total) break;
            const int s = static_cast<int>(i / num_q_heads), h = static_cast<int>(i % num_q_heads), g = h / G;
            const int L = context_lens[s];
            double* o = out + i * d;
            for (int j = 0; j < d; ++j) o[j] = 0.0;
            if (L <= 0) continue;
            const uint16_t* qrow = q + i * d;
            x.assign(static_cast<size_t>(L), 0.0);
            live.assign(static_cast<size_t>(L), 1);
            double xmax = -std::numeric_limits<double>::infinity();
            for (int t = 0; t < L; ++t) {
                const int32_t page = block_table[static_cast<int64_t>(s) * max_blocks_per_seq + t / bs];
                if (page < 0 || page >= num_blocks) {     // not dereferenced, left out of the softmax, counted
                    live[t] = 0;
                    ++skipped;
                    continue;
                }
                const uint8_t* krow = k8 + ((static_cast<int64_t>(page) * num_kv_heads + g) * bs + t % bs) * d;
                double acc = 0.0;
                for (int j = 0; j < d; ++j)
                    acc += bf16_to_double(qrow[j]) * (static_cast<double>(k_scale[g]) * pdattn_oracle_e4m3_to_double(krow[j]));
                x[t] = static_cast<double>(scale) * acc;
                if (std::isnan(x[t]) || x[t] > xmax) xmax = x[t];   // a NaN score of a live slot propagates
            }
            double Z = 0.0;
            for (int t = 0; t < L; ++t) {
                if (!live[t]) continue;
                const double w = std::exp(x[t] - xmax);
                Z += w;
                const int32_t page = block_table[static_cast<int64_t>(s) * max_blocks_per_seq + t / bs];
                const uint8_t* vblk = v8 + (static_cast<int64_t>(page) * num_kv_heads + g) * d * bs;
                for (int j = 0; j < d; ++j)
                    o[j] += w * (static_cast<double>(v_scale[g]) * pdattn_oracle_e4m3_to_double(vblk[j * bs + t % bs]));
            }
            for (int j = 0; j < d; ++j) o[j] = (Z > 0.0 || std::isnan(Z)) ? o[j] / Z : 0.0;
        }
    };
    const int nt = num_threads > 0 ? num_threads : 1;
    if (nt == 1) {
        worker();
    } else {
        std::vector<std::thread> pool;
        for (int i = 0; i < nt; ++i) pool.emplace_back(worker);
        for (auto& th : pool) th.join();
    }
    if (bad_pages) *bad_pages = skipped.load();
    return 0;
}

}  // extern "C"
