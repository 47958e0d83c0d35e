// CPU oracle for the lightning-indexer hot path: TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, FP64 restatement of what the path computes, written from the
// paper's definitions. It shares no code with the CUDA library and must never
// be called from the product path; only tests, the smoke check and the
// benchmark's cpu_baseline / reference legs may load it.
//
// What it follows:
//   * score  I[t,s] = sum_h w[t,h] * ReLU(q[t,h] . k[s]) for every preceding
//     token s <= t  (Sec. 2.1 "DeepSeek Sparse Attention": a multi-head
//     ReLU-gated dot product against the keys of all preceding tokens; the
//     closed formula is the one the benchmark spec fixes);
//   * T_t = Top-k(I_t)  (Sec. 3 "Notation");
//   * decode: the same for one new query against a whole cached context
//     (Sec. 4.2 "Decode": a per-token indexer pass over the full context).
// The Full/Shared layer schedule (Sec. 3 "Overview", Figure 2(b)) is host
// logic and lives in oracle/schedule.py.
//
// Readings where the paper is silent: the token itself counts as "preceding"
// (mask s <= t); rows with fewer than k candidates select all of them and pad
// with -1; ties go to the lowest index; indices are emitted in ascending order.
//
// Pins (tests/test_oracle_*.py): hand-computed tiny case, non-negative inputs
// reducing to a BLAS matrix product, rank-1 closed form, one-hot inputs,
// all-negative gate, sliding-window / sink top-k closed forms, duplicate-key
// tie-break, exhaustive number-format round trips against the format
// definitions; the quantiser against a library conversion and closed forms.
// No function here is "parity unpinned".

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// BF16 is the upper half of an IEEE-754 binary32 (1 sign, 8 exponent, 7 mantissa bits).
inline double bf16_to_f64(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return static_cast<double>(f);
}

// E4M3 "FN": 1 sign, 4 exponent bits (bias 7), 3 mantissa bits, subnormals at
// exponent field 0 (step 2^-9), largest finite 448 (0x7E), S.1111.111 is NaN,
// no infinities.
inline double e4m3_to_f64(uint8_t c) {
    int sign = (c >> 7) & 1;
    int e = (c >> 3) & 0xF;
    int m = c & 0x7;
    double v;
    if (e == 0xF && m == 0x7) {
        v = std::numeric_limits<double>::quiet_NaN();
    } else if (e == 0) {
        v = std::ldexp(static_cast<double>(m), -9);           // m/8 * 2^-6
    } else {
        v = std::ldexp(1.0 + static_cast<double>(m) / 8.0, e - 7);
    }
    return sign ? -v : v;
}

// float -> bf16, round to nearest even (finite inputs; NaN kept quiet).
inline uint16_t f32_to_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return static_cast<uint16_t>((u >> 16) | 0x40);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

// float -> e4m3fn, round to nearest even, saturating to +-448. Done by
// searching the 127 non-negative finite codes: obviously correct, slow.
inline uint8_t f32_to_e4m3(float f) {
    if (std::isnan(f)) return 0x7F;
    uint8_t sign = std::signbit(f) ? 0x80 : 0x00;
    double a = std::fabs(static_cast<double>(f));
    if (a >= 448.0) return sign | 0x7E;
    int best = 0;
    double best_err = std::numeric_limits<double>::infinity();
    for (int c = 0; c <= 0x7E; ++c) {
        double err = std::fabs(e4m3_to_f64(static_cast<uint8_t>(c)) - a);
        if (err < best_err || (err == best_err && (c & 1) == 0)) {   // tie -> even mantissa
            best_err = err;
            best = c;
        }
    }
    return sign | static_cast<uint8_t>(best);
}

struct Decoded {
    int dtype;             // 0 = bf16, 1 = e4m3 with per-token fp32 scales
    const void* ptr;
    const float* scale;    // per row (token) or nullptr
    int64_t row_elems;     // elements per token row (H*d for q, d for k)
    double at(int64_t token, int64_t i) const {
        double v;
        if (dtype == 0) {
            v = bf16_to_f64(static_cast<const uint16_t*>(ptr)[token * row_elems + i]);
        } else {
            v = e4m3_to_f64(static_cast<const uint8_t*>(ptr)[token * row_elems + i]);
            v *= static_cast<double>(scale[token]);
        }
        return v;
    }
};

// One score row: I[s] for s in [0, n_keys) for the query at `qrow` (row of the q
// array), heads H, head dim d. Definition order: for each key, for each head,
// the full dot product, the gate, the weighted add.
void score_row(const Decoded& q, const Decoded& k, const float* w_row, int64_t qrow, int64_t k_row0,
               int64_t n_keys, int H, int d, double* out) {
    std::vector<double> qd(static_cast<size_t>(H) * d);
    for (int h = 0; h < H; ++h)
        for (int i = 0; i < d; ++i) qd[static_cast<size_t>(h) * d + i] = q.at(qrow, static_cast<int64_t>(h) * d + i);
    std::vector<double> kd(d);
    for (int64_t s = 0; s < n_keys; ++s) {
        for (int i = 0; i < d; ++i) kd[i] = k.at(k_row0 + s, i);
        double I = 0.0;
        for (int h = 0; h < H; ++h) {
            double x = 0.0;
            for (int i = 0; i < d; ++i) x += qd[static_cast<size_t>(h) * d + i] * kd[i];
            if (x > 0.0) I += static_cast<double>(w_row[h]) * x;
        }
        out[s] = I;
    }
}

// Top-k of scores[0..n): the min(k, n) largest, ties to the lowest index,
// emitted in ascending index order, padded with -1 up to k entries.
void topk_row(const double* scores, int64_t n, int k, int32_t* out) {
    std::vector<int32_t> order(static_cast<size_t>(n));
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
        if (scores[a] != scores[b]) return scores[a] > scores[b];
        return a < b;
    });
    int64_t kk = std::min<int64_t>(k, n);
    std::vector<int32_t> sel(order.begin(), order.begin() + kk);
    std::sort(sel.begin(), sel.end());
    for (int64_t j = 0; j < k; ++j) out[j] = j < kk ? sel[static_cast<size_t>(j)] : -1;
}

}  // namespace

extern "C" {

int orc_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

double orc_bf16_to_f64(uint16_t h) { return bf16_to_f64(h); }
double orc_e4m3_to_f64(uint8_t c) { return e4m3_to_f64(c); }
uint16_t orc_f32_to_bf16(float f) { return f32_to_bf16(f); }
uint8_t orc_f32_to_e4m3(float f) { return f32_to_e4m3(f); }

int orc_topk(const double* scores, int64_t n, int k, int32_t* out) {
    if (n < 0 || k < 1) return 1;
    topk_row(scores, n, k, out);
    return 0;
}

// Prefill rows. q holds q_len rows that are positions q_begin .. q_begin+q_len-1;
// k holds L_k >= q_begin+q_len rows. `rows` lists local row indices into q (NULL:
// all q_len rows). For listed row r with position t = q_begin + r:
//   scores_out[j*ld + s] = I[t,s] for s <= t, -inf for t < s < L_k   (if non-NULL)
//   topk_out[j*k_top ..] = Top-k over s in [0, t]                     (if non-NULL)
int orc_prefill(const void* q, const void* k, const float* w, const float* q_scale, const float* k_scale,
                int64_t q_begin, int64_t q_len, int64_t L_k, int H, int d, int k_top, int dtype,
                const int64_t* rows, int64_t n_rows, double* scores_out, int64_t ld, int32_t* topk_out) {
    if (q_begin < 0 || q_len < 0 || L_k < q_begin + q_len || H < 1 || d < 1 || k_top < 1) return 1;
    if (dtype != 0 && dtype != 1) return 1;
    if (dtype == 1 && (!q_scale || !k_scale)) return 1;
    if (scores_out && ld < L_k) return 1;
    int64_t n = rows ? n_rows : q_len;
    Decoded qd{dtype, q, q_scale, static_cast<int64_t>(H) * d};
    Decoded kd{dtype, k, k_scale, d};
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t j = 0; j < n; ++j) {
        int64_t r = rows ? rows[j] : j;
        if (r < 0 || r >= q_len) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        int64_t t = q_begin + r;
        std::vector<double> row(static_cast<size_t>(t + 1));
        score_row(qd, kd, w + r * H, r, 0, t + 1, H, d, row.data());
        if (scores_out) {
            double* o = scores_out + j * ld;
            for (int64_t s = 0; s <= t; ++s) o[s] = row[static_cast<size_t>(s)];
            for (int64_t s = t + 1; s < L_k; ++s) o[s] = -std::numeric_limits<double>::infinity();
        }
        if (topk_out) topk_row(row.data(), t + 1, k_top, topk_out + j * k_top);
    }
    return bad;
}

// Decode step. Sequence b: query q_step[b], keys are rows k_offsets[b] ..
// k_offsets[b]+lens[b]-1 of the cache (lens counts the current token); every
// cached position is visible.
//   scores_out[b*ld + s] = I[b,s] for s < lens[b], -inf up to ld  (if non-NULL)
//   topk_out[b*k_top ..] = Top-k over s in [0, lens[b])           (if non-NULL)
int orc_decode(const void* q_step, const void* k_cache, const float* w, const float* q_scale,
               const float* k_scale, const int64_t* k_offsets, const int32_t* lens, int B, int H, int d,
               int k_top, int dtype, double* scores_out, int64_t ld, int32_t* topk_out) {
    if (B < 0 || H < 1 || d < 1 || k_top < 1) return 1;
    if (dtype != 0 && dtype != 1) return 1;
    if (dtype == 1 && (!q_scale || !k_scale)) return 1;
    Decoded qd{dtype, q_step, q_scale, static_cast<int64_t>(H) * d};
    Decoded kd{dtype, k_cache, k_scale, d};
    for (int b = 0; b < B; ++b) {
        int64_t n = lens[b];
        if (n < 0 || (scores_out && ld < n)) return 1;
        std::vector<double> row(static_cast<size_t>(n));
        // rows of one sequence are split across threads; each key is independent
        int nthreads = orc_threads();
        int64_t chunk = (n + nthreads - 1) / std::max(nthreads, 1);
#pragma omp parallel for schedule(static, 1)
        for (int c = 0; c < nthreads; ++c) {
            int64_t s0 = c * chunk, s1 = std::min<int64_t>(n, s0 + chunk);
            if (s0 < s1) score_row(qd, kd, w + static_cast<int64_t>(b) * H, b, k_offsets[b] + s0, s1 - s0, H, d, row.data() + s0);
        }
        if (scores_out) {
            double* o = scores_out + static_cast<int64_t>(b) * ld;
            for (int64_t s = 0; s < n; ++s) o[s] = row[static_cast<size_t>(s)];
            for (int64_t s = n; s < ld; ++s) o[s] = -std::numeric_limits<double>::infinity();
        }
        if (topk_out) topk_row(row.data(), n, k_top, topk_out + static_cast<int64_t>(b) * k_top);
    }
    return 0;
}

// Per-token FP8 quantiser, the step in front of the indexer (Sec. 2.1: the indexer runs in FP8
// arithmetic). Reading taken: one fp32 scale per token, scale = max(amax, 1e-12) / 448 and
// code = e4m3(x / scale) with round-to-nearest-even and saturation. The code is an integer decided by
// floating point, so the decision is taken in the precision the kernel uses: IEEE binary32 for amax,
// the two divisions and the rounding input. x: [n_tokens, row_elems] bf16 codes.
int orc_quantize_e4m3(const uint16_t* x, int64_t n_tokens, int64_t row_elems, uint8_t* codes, float* scale) {
    if (n_tokens < 0 || row_elems < 1) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_tokens; ++r) {
        float amax = 0.0f;
        for (int64_t i = 0; i < row_elems; ++i) {
            float v = static_cast<float>(bf16_to_f64(x[r * row_elems + i]));
            amax = std::fmax(amax, std::fabs(v));
        }
        const float sc = std::fmax(amax, 1e-12f) / 448.0f;
        scale[r] = sc;
        for (int64_t i = 0; i < row_elems; ++i) {
            float v = static_cast<float>(bf16_to_f64(x[r * row_elems + i]));
            codes[r * row_elems + i] = f32_to_e4m3(v / sc);
        }
    }
    return 0;
}

}  // extern "C"
