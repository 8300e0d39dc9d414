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
// weights; for the per-epoch data allocation, the generator's published known
// answers, the paper's own (32, 8, 1, 2) setting for the sizes, and the
// statistics that "uniformly without replacement" fixes (valid subsets, every
// subset equally likely, uniform and independent priorities); for the round
// aggregation, the pinned Eq. 3 routine, float64 numpy, its fixed points and a
// library's bf16 rounding.  Ordering of NaN,
// +-0 and all-ignored samples is a convention of this library, not of the
// paper: parity unpinned for those cases (convention only).  The same holds for
// which random stream feeds a draw (counter layout, 30-bit priorities, ties by
// lower index): the paper asks only for a random draw; the distribution is pinned, the
// particular bits are this library's convention.
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

// Per-sample loss record (Algorithm 1, the step that stores every processed sample's loss): softmax
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

// ---------------------------------------------------------------------------
// Per-epoch data allocation (Section 4.2; Algorithm 1, the four steps before the
// training loop).
// ---------------------------------------------------------------------------
namespace {

// Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random
// numbers: as easy as 1, 2, 3", SC'11): a 128-bit counter and a 64-bit key give
// four 32-bit words.  One round multiplies words 0 and 2 of the counter by two
// fixed odd constants, swaps the product halves into place and mixes the key in;
// the key is advanced by two Weyl constants between rounds.
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c[4] = {ctr_in[0], ctr_in[1], ctr_in[2], ctr_in[3]};
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = M0 * c[0], p1 = M1 * c[2];
        const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
        const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
        const uint32_t n0 = hi1 ^ c[1] ^ k0, n1 = lo1, n2 = hi0 ^ c[3] ^ k1, n3 = lo0;
        c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
        k0 += W0;
        k1 += W1;
    }
    for (int i = 0; i < 4; ++i) out[i] = c[i];
}

// Random priority of sample i in draw `stream` under `seed`: 30 bits.  Samples
// 4j .. 4j+3 share one Philox block: counter (j, 0, stream_lo, stream_hi), key
// (seed_lo, seed_hi); sample i takes word i mod 4, top 30 bits.
uint32_t priority_of(int64_t i, uint64_t seed, uint64_t stream) {
    const uint32_t ctr[4] = {static_cast<uint32_t>(i >> 2), 0u, static_cast<uint32_t>(stream),
                             static_cast<uint32_t>(stream >> 32)};
    const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
    uint32_t w[4];
    philox4x32_10(ctr, key, w);
    return w[i & 3] >> 2;
}

}  // namespace

extern "C" {

int oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
    return 0;
}

// Section 4.2: of N samples per epoch the fast workers get
//   N_F = tau_F P_F / (tau_F P_F + tau_S P_S) * N   (rounded down),
// the slow workers the rest, N_S = N - N_F (so that one epoch covers N samples),
// and k = lambda * N_F (rounded down) of the fast workers' samples are the
// highest-loss ones.  lambda arrives as the double nearest to a decimal fraction,
// which may lie just below it (0.29 * 100 is 28.999999999999996 in double), so a
// product within 2^-51 (relative) of an integer counts as that integer.
int oracle_allocation_sizes(int64_t N, int32_t tau_f, int32_t p_f, int32_t tau_s, int32_t p_s, double lambda,
                            int64_t* n_fast, int64_t* n_slow, int64_t* k_high) {
    if (N < 0 || tau_f < 0 || p_f < 0 || tau_s < 0 || p_s < 0 || !(lambda >= 0.0 && lambda <= 1.0)) return 1;
    const __int128 a = static_cast<__int128>(tau_f) * p_f, b = static_cast<__int128>(tau_s) * p_s;
    if (a + b == 0) return 1;
    const int64_t nf = static_cast<int64_t>(a * N / (a + b));
    *n_fast = nf;
    *n_slow = N - nf;
    const double prod = lambda * static_cast<double>(nf), near = std::round(prod);
    int64_t k = std::fabs(prod - near) <= near * 0x1p-51 ? static_cast<int64_t>(near)
                                                         : static_cast<int64_t>(std::floor(prod));
    *k_high = std::min(std::max<int64_t>(k, 0), nf);
    return 0;
}

// The even split of a list of n entries over P workers: worker p gets the
// contiguous range [floor(p n / P), floor((p+1) n / P)), so shares differ by at
// most one entry and together cover the list once.
int oracle_worker_share(int64_t n, int32_t P, int32_t p, int64_t* begin, int64_t* end) {
    if (n < 0 || P < 1 || p < 0 || p >= P) return 1;
    *begin = static_cast<int64_t>(static_cast<__int128>(n) * p / P);
    *end = static_cast<int64_t>(static_cast<__int128>(n) * (p + 1) / P);
    return 0;
}

// Uniform sampling without replacement (Section 4.2: the fast group's fill from
// the samples that were not selected, and the slow group's draw from all N
// samples): every sample gets an independent random priority; the draw is
// the m candidates with the highest priority (ties: lower index), listed in that
// order.  Candidates are the indices 0..N-1 that are not in exclude_idx.
// Independent, identically distributed priorities make every m-subset of the
// candidates equally likely and the listed order a uniform random order.
int oracle_draw_uniform(int64_t N, int64_t m, uint64_t seed, uint64_t stream, const int32_t* exclude_idx,
                        int64_t n_exclude, int32_t* out_idx) {
    std::vector<char> excluded(static_cast<size_t>(N), 0);
    for (int64_t j = 0; j < n_exclude; ++j)
        if (exclude_idx[j] >= 0 && exclude_idx[j] < N) excluded[static_cast<size_t>(exclude_idx[j])] = 1;
    std::vector<int32_t> cand;
    for (int64_t i = 0; i < N; ++i)
        if (!excluded[static_cast<size_t>(i)]) cand.push_back(static_cast<int32_t>(i));
    if (m < 0 || m > static_cast<int64_t>(cand.size())) return 1;
    std::vector<uint32_t> pri(static_cast<size_t>(N));
    for (int64_t i = 0; i < N; ++i) pri[static_cast<size_t>(i)] = priority_of(i, seed, stream);
    std::stable_sort(cand.begin(), cand.end(), [&](int32_t a, int32_t b) { return pri[a] > pri[b]; });
    for (int64_t j = 0; j < m; ++j) out_idx[j] = cand[static_cast<size_t>(j)];
    return 0;
}

// The priorities themselves (for the tests' statistics).
int oracle_priorities(int64_t N, uint64_t seed, uint64_t stream, uint32_t* out) {
    for (int64_t i = 0; i < N; ++i) out[i] = priority_of(i, seed, stream);
    return 0;
}

// Data allocation for the fast workers (Section 4.2; Algorithm 1, the selection
// step and the random fill that follows it): the k highest-loss samples in loss-descending order,
// followed by n_fill samples drawn uniformly without replacement from the other
// N - k.
int oracle_fast_allocation(const float* losses, int64_t N, int64_t k, int64_t n_fill, uint64_t seed, uint64_t stream,
                           int32_t* out_idx) {
    if (k < 0 || n_fill < 0 || k + n_fill > N) return 1;
    if (oracle_topk(losses, N, k, 0, out_idx, nullptr) != 0) return 1;
    return oracle_draw_uniform(N, n_fill, seed, stream, out_idx, k, out_idx + k);
}

}  // extern "C"

// ---------------------------------------------------------------------------
// One round's aggregation as the training loop uses it (Section 2, the local-SGD
// update rule; Eq. 3; Algorithm 1: every worker continues from x_{t+1}).
// ---------------------------------------------------------------------------
namespace {

inline double replica_at(const void* rep, int dtype, int64_t j) {
    if (dtype == 0) return static_cast<double>(static_cast<const float*>(rep)[j]);
    return bf16_to_double(static_cast<const uint16_t*>(rep)[j]);
}

// fp32 -> bf16, round to nearest, ties to even (bf16 = the upper 16 bits of an fp32).
inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, sizeof u);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return static_cast<uint16_t>((u >> 16) | 0x0040u);  // NaN stays NaN
    const uint32_t lower = u & 0xFFFFu, keep = u >> 16;
    uint32_t r = keep;
    if (lower > 0x8000u || (lower == 0x8000u && (keep & 1u))) r = keep + 1u;
    return static_cast<uint16_t>(r);
}

}  // namespace

extern "C" {

// x_{t+1}[j] from the P replicas (fp32, or bf16 widened exactly), in double, ascending i:
//   base == NULL:  sum_i w_i x_i[j]                          (Eq. 3)
//   base != NULL:  base[j] + sum_i w_i (x_i[j] - base[j])    (the same update written around x_t = base, as in
//                  Section 2's rule x_{t+1} = x_t - eta * (averaged local progress); equal to Eq. 3 when sum w = 1)
// out (double), out_f32 (its rounding), out_bf16 (out_f32 rounded once more to bf16: what a bf16 replica holds after
// the broadcast), abs_out (the error scale: sum_i |w_i x_i|, or sum_i |w_i (x_i - base)| in the delta form).  Any of
// the four may be NULL.
int oracle_aggregate_round(const void* const* replicas, int dtype, const float* w, int32_t P, int64_t D,
                           const float* base, double* out, float* out_f32, uint16_t* out_bf16, double* abs_out) {
    for (int64_t j = 0; j < D; ++j) {
        const double b = base ? static_cast<double>(base[j]) : 0.0;
        double acc = 0.0, mag = 0.0;
        for (int32_t i = 0; i < P; ++i) {
            const double term = static_cast<double>(w[i]) * (replica_at(replicas[i], dtype, j) - b);
            acc += term;
            mag += std::fabs(term);
        }
        const double r = b + acc;
        if (out) out[j] = r;
        if (out_f32) out_f32[j] = static_cast<float>(r);
        if (out_bf16) out_bf16[j] = f32_to_bf16_rne(static_cast<float>(r));
        if (abs_out) abs_out[j] = mag;
    }
    return 0;
}

}  // extern "C"
