// lsgd_oracle.cpp — TEST INFRASTRUCTURE, not part of the product.
//
// A plain, slow, single-threaded CPU statement of what the hot path of one
// biased-local-SGD round computes, in double precision, written directly from
// the definitions.  It exists so that the CUDA library can be checked element
// by element against something obviously correct.  Only tests, the smoke check
// and the benchmark's CPU-baseline leg may call it; the CUDA library neither
// links nor includes anything from this directory, and nothing here includes
// anything of the library's.  No blocking, no fusion, no reordering beyond what
// each definition states.
//
// Pins (checked by the CPU test-suite against facts that do not come from this
// file): closed forms ln C / softplus / C = 1, shift and permutation invariance,
// a library log-sum-exp, brute-force selection, one-hot / uniform / (32,1)-step
// weights.  Ordering of NaN, +-0 and all-ignored samples is a convention of this
// library, not of the paper: parity unpinned for those cases (convention only).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;  // bf16 is the top half of an fp32
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

inline double logit_at(const void* logits, int dtype, int64_t pos) {
    if (dtype == 0) return static_cast<double>(static_cast<const float*>(logits)[pos]);
    return bf16_to_double(static_cast<const uint16_t*>(logits)[pos]);
}

// Order used by the selector (Section 4.2: the highest-loss samples; ties by
// lower index).  Values are compared after canonicalisation: -0 == +0, every NaN
// is one value that ranks above +inf.
inline bool is_nan(float v) { return v != v; }
inline bool ranks_before(float a, float b) {  // true if a is strictly "higher loss" than b
    if (is_nan(a)) return !is_nan(b);
    if (is_nan(b)) return false;
    return a > b;  // -0.0 > +0.0 is false and vice versa: they tie
}

}  // namespace

extern "C" {

// Per-sample loss record (Algorithm 1, "record all individual loss"): softmax
// cross-entropy with natural log per token, mean over the tokens that are not
// ignored.
//   token:   l = (m - x_y) + log(sum_j exp(x_j - m)),  m = max_j x_j
//   sample:  L_n = (sum over unmasked t, ascending, of l[n,t]) / count,  0 if count == 0
// A label outside [0, C) that is not ignore_index gives NaN and is counted.
// loss_out [N] double; token_out [N*T] double or NULL (NaN-free: ignored tokens get 0).
int oracle_score(const void* logits, int dtype, const int64_t* labels, int64_t N, int64_t T, int64_t C,
                 int64_t ignore_index, double* loss_out, double* token_out, int64_t* bad_labels) {
    int64_t bad = 0;
    for (int64_t n = 0; n < N; ++n) {
        double sum = 0.0;
        int64_t cnt = 0;
        for (int64_t t = 0; t < T; ++t) {
            const int64_t row = n * T + t;
            const int64_t y = labels[row];
            double l = 0.0;
            if (y == ignore_index) {
                if (token_out) token_out[row] = 0.0;
                continue;
            }
            if (y < 0 || y >= C) {
                l = std::numeric_limits<double>::quiet_NaN();
                ++bad;
            } else {
                double m = logit_at(logits, dtype, row * C);
                for (int64_t j = 1; j < C; ++j) m = std::max(m, logit_at(logits, dtype, row * C + j));
                double s = 0.0;
                for (int64_t j = 0; j < C; ++j) s += std::exp(logit_at(logits, dtype, row * C + j) - m);
                l = (m - logit_at(logits, dtype, row * C + y)) + std::log(s);
            }
            if (token_out) token_out[row] = l;
            sum += l;
            ++cnt;
        }
        loss_out[n] = cnt ? sum / static_cast<double>(cnt) : 0.0;
    }
    if (bad_labels) *bad_labels = bad;
    return 0;
}

// Deterministic loss-based top-k (Section 4.2): the first k of a stable sort of
// 0..N-1 by "higher loss first"; stability gives "then lower index".
//   order 0: that prefix as is (loss descending);  order 1: the same set, index ascending.
// vals_out (may be NULL) receives losses[idx] unchanged.
int oracle_topk(const float* losses, int64_t N, int64_t k, int order, int32_t* idx_out, float* vals_out) {
    if (k < 0 || k > N) return 1;
    std::vector<int32_t> perm(static_cast<size_t>(N));
    std::iota(perm.begin(), perm.end(), 0);
    std::stable_sort(perm.begin(), perm.end(),
                     [&](int32_t a, int32_t b) { return ranks_before(losses[a], losses[b]); });
    perm.resize(static_cast<size_t>(k));
    if (order == 1) std::sort(perm.begin(), perm.end());
    for (int64_t j = 0; j < k; ++j) {
        idx_out[j] = perm[static_cast<size_t>(j)];
        if (vals_out) vals_out[j] = losses[perm[static_cast<size_t>(j)]];
    }
    return 0;
}

// Biased model aggregation, Eq. 3:  out[j] = sum_i w_i x_i[j], ascending i, in
// double; out_f32 is its single rounding to fp32.  abs_out (may be NULL) is
// sum_i |w_i x_i[j]|, the scale against which a relative error is meaningful
// when terms cancel.
int oracle_aggregate(const float* const* replicas, const float* w, int32_t P, int64_t D, double* out,
                     float* out_f32, double* abs_out) {
    for (int64_t j = 0; j < D; ++j) {
        double acc = 0.0, mag = 0.0;
        for (int32_t i = 0; i < P; ++i) {
            const double term = static_cast<double>(w[i]) * static_cast<double>(replicas[i][j]);
            acc += term;
            mag += std::fabs(term);
        }
        if (out) out[j] = acc;
        if (out_f32) out_f32[j] = static_cast<float>(acc);
        if (abs_out) abs_out[j] = mag;
    }
    return 0;
}

// Eq. 3's weights from local step counts: w_i = tau_i / sum_j tau_j, in double,
// rounded once to fp32.
int oracle_weights_from_steps(const int32_t* tau, int32_t P, float* w_out) {
    double total = 0.0;
    for (int32_t i = 0; i < P; ++i) total += static_cast<double>(tau[i]);
    if (!(total > 0.0)) return 1;
    for (int32_t i = 0; i < P; ++i) w_out[i] = static_cast<float>(static_cast<double>(tau[i]) / total);
    return 0;
}

}  // extern "C"
