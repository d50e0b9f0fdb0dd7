// KeyDiff eviction step -- CPU oracle.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// A plain, slow, fp64 restatement of the per-KV-head eviction step of KeyDiff
// (block-wise prefill: append a block of B new keys/values to a cache bounded by
// a budget N, then evict back down to N).  Only the test-suite, the smoke check
// and the benchmark's CPU-baseline leg may call this file.  It shares no code,
// header, table or constant with the CUDA path and is never a fallback for it.
//
// What each function follows:
//   * scores       -- App. B.1 ("FLOP count of KeyDiff"): the two expressions
//                     mu(K^) = (1/n) sum_i k_i/||k_i||  and
//                     s_i = mu.k_i / max(||mu||*||k_i||, eps),
//                     i.e. Eq. (efficient-keydiff) of Sec. 3.2 written out.
//   * selection    -- Eq. (efficient-keydiff): S = topk(-CosSim(mu, k_i), N);
//                     topk as defined below Eq. (attn_based_eviction_policy):
//                     "indices of the N largest values".
//   * gather       -- Eq. (keydiff): K' = gather(K,S), V' = gather(V,S).
//   * when to evict-- Sec. 2.3 / Eq. (eviction_policy): only if the updated
//                     cache is larger than N; Eq. (block_processing) for the
//                     concatenation order (cache rows first, block rows after).
//   * pairwise     -- Eq. (keydiff) literally: CosSim(K) 1, O(n^2); used only as
//                     a cross-check of the anchor form (App. C derivation).
//
// Readings where the paper is silent (the same list is kept in the design notes):
//   - anchor is the mean of the NORMALISED keys (the equation's form);
//   - eps = 1e-8 by default, applied to the product ||mu||*||k_i|| as printed;
//   - a key's normalisation uses k_i / max(||k_i||, eps) so a zero key adds the
//     zero vector to the anchor and scores 0;
//   - the stored "eviction score" is e_i = -s_i (with -0 mapped to +0); the N
//     LARGEST e are kept;
//   - ties: total order (e descending, token index ascending) -- among equal
//     scores the older token is kept;
//   - kept rows are written in original token order (ascending index).
//
// Two variants of the method are restated as well (the *_ex entry points):
//   * raw-mean anchor (anchor_mode 1) -- Sec. 3.2, the sentence after Eq. (efficient-keydiff) and
//     the caption of the method figure: the anchor is the mean of the keys themselves,
//     mu(K) = (1/n) sum_i k_i; the score formula is unchanged.
//   * sliding window (recent_window w) -- Sec. 3.2, "KeyDiff with sliding window": part of the
//     budget is reserved for the most recent tokens and KeyDiff manages the rest.  Reading (the
//     paper gives no formula): the last w of the n tokens are always kept, the N - w tokens with
//     the largest eviction score are kept among the first n - w, and the anchor is still formed
//     from all n keys.
//
//   * unordered slot reuse (the *_slots entry point) -- Eq. (keydiff) gathers the kept rows but fixes
//     no order for them (attention does not depend on the order of the cached pairs).  Reading: kept
//     cache rows stay in their slots; the kept block rows, in block order, fill the freed slots (those
//     of evicted cache rows and, while the cache is not full, the empty ones) in ascending slot
//     order; a side array holds each slot's token position.  Candidates are numbered cache slots
//     first, block rows after; equal scores keep the lower candidate number.  The sliding window is
//     then defined on positions: tokens among the last w of the sequence are always kept.
//
// Every function is pinned by tests that do not call back into this file:
// hand-worked examples, closed forms, the pairwise identity evaluated in numpy,
// brute force over all subsets, and structural invariants.  No function here is
// "parity unpinned".
//
// Arithmetic: IEEE double throughout, plain left-to-right loops, no blocking,
// no SIMD intrinsics, no reordering beyond what the formulas state.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <thread>
#include <vector>

namespace {

// bf16 is the upper half of an IEEE binary32, so widening is exact.
inline double bf16_bits_to_double(uint16_t bits) {
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// App. B.1, both expressions.  K is n x d row-major doubles.
// Outputs (any may be null): r[n] key norms, mu[d] anchor, *m anchor norm,
// s[n] cosine similarities of each key to the anchor.
// anchor_mode 0: mu = mean of k_i/||k_i|| (the equation); 1: mu = mean of k_i (Sec. 3.2, text).
void scores_f64(const double* K, int64_t n, int64_t d, double eps,
                double* r_out, double* mu_out, double* m_out, double* s_out, int anchor_mode = 0) {
    std::vector<double> r(n), mu(d, 0.0);
    // ||k_i|| = sqrt(k_i . k_i)
    for (int64_t i = 0; i < n; ++i) {
        double ss = 0.0;
        for (int64_t c = 0; c < d; ++c) ss += K[i * d + c] * K[i * d + c];
        r[i] = std::sqrt(ss);
    }
    // mu = (1/n) sum_i k_i / ||k_i||   (guarded divisor, see header)
    for (int64_t i = 0; i < n; ++i) {
        const double div = anchor_mode == 1 ? 1.0 : std::max(r[i], eps);   // raw mean: mu = (1/n) sum_i k_i
        for (int64_t c = 0; c < d; ++c) mu[c] += K[i * d + c] / div;
    }
    for (int64_t c = 0; c < d; ++c) mu[c] /= static_cast<double>(n);
    // ||mu||
    double mm = 0.0;
    for (int64_t c = 0; c < d; ++c) mm += mu[c] * mu[c];
    const double m = std::sqrt(mm);
    // s_i = mu . k_i / max(||mu|| * ||k_i||, eps)
    for (int64_t i = 0; i < n; ++i) {
        double dot = 0.0;
        for (int64_t c = 0; c < d; ++c) dot += mu[c] * K[i * d + c];
        const double s = dot / std::max(m * r[i], eps);
        if (s_out) s_out[i] = s;
    }
    if (r_out) std::copy(r.begin(), r.end(), r_out);
    if (mu_out) std::copy(mu.begin(), mu.end(), mu_out);
    if (m_out) *m_out = m;
}

// e_i = -s_i, with -0 canonicalised to +0.
inline double eviction_score(double s) {
    const double e = -s;
    return e == 0.0 ? 0.0 : e;
}

// topk(e, N) under the total order (e desc, index asc); result sorted ascending
// by index (original token order).  Returns the number kept = min(N, n).
int64_t select_topn(const double* e, int64_t n, int64_t N, int64_t* S_out,
                    double* tau_out) {
    const int64_t keep = std::min(N, n);
    std::vector<int64_t> order(n);
    std::iota(order.begin(), order.end(), int64_t{0});
    // stable sort by e descending: equal scores stay in ascending index order
    std::stable_sort(order.begin(), order.end(),
                     [e](int64_t a, int64_t b) { return e[a] > e[b]; });
    if (tau_out) *tau_out = keep > 0 ? e[order[keep - 1]] : 0.0;
    std::vector<int64_t> S(order.begin(), order.begin() + keep);
    std::sort(S.begin(), S.end());
    std::copy(S.begin(), S.end(), S_out);
    return keep;
}

// Sliding window: the last w of the n tokens are kept unconditionally; among the first n - w the
// N - w with the largest e are kept (same order and tie rule).  Requires 0 <= w <= N.  tau = score of
// the last token kept by the score rule (0 if none is).
int64_t select_topn_window(const double* e, int64_t n, int64_t N, int64_t w, int64_t* S_out, double* tau_out) {
    if (n <= N) return select_topn(e, n, N, S_out, tau_out);
    const int64_t head = n - w;                       // tokens the score rule decides on
    std::vector<int64_t> S(N);
    double tau = 0.0;
    const int64_t kept_head = head > 0 ? select_topn(e, head, N - w, S.data(), &tau) : 0;   // == N - w
    for (int64_t j = 0; j < w; ++j) S[kept_head + j] = head + j;                            // the window, in order
    std::copy(S.begin(), S.begin() + kept_head + w, S_out);
    if (tau_out) *tau_out = tau;
    return kept_head + w;
}

struct HeadArgs {
    const uint16_t* k_cache; const uint16_t* v_cache; int64_t len;
    const uint16_t* new_k;   const uint16_t* new_v;   int64_t B;
    int64_t N; int64_t d; double eps;
    uint16_t* k_out; uint16_t* v_out; int64_t* len_out;
    double* e_out; int64_t* S_out; double* tau_out; double* m_out;
    int anchor_mode = 0; int64_t window = 0;
};

// One unit (one KV head of one layer of one sequence), Eq. (eviction_policy)
// with pi_N = KeyDiff.
void evict_head(const HeadArgs& a) {
    const int64_t n = a.len + a.B, d = a.d;
    // logical concatenation [K_cache || k_block] along the token axis
    auto k_row = [&](int64_t i) { return i < a.len ? a.k_cache + i * d : a.new_k + (i - a.len) * d; };
    auto v_row = [&](int64_t i) { return i < a.len ? a.v_cache + i * d : a.new_v + (i - a.len) * d; };
    std::vector<int64_t> S(std::min(a.N, n));
    double tau = 0.0, m = 0.0;
    if (n <= a.N) {
        // budget not exceeded: nothing is evicted, nothing is scored
        std::iota(S.begin(), S.end(), int64_t{0});
    } else {
        std::vector<double> K(static_cast<size_t>(n) * d), s(n), e(n);
        for (int64_t i = 0; i < n; ++i)
            for (int64_t c = 0; c < d; ++c) K[i * d + c] = bf16_bits_to_double(k_row(i)[c]);
        scores_f64(K.data(), n, d, a.eps, nullptr, nullptr, &m, s.data(), a.anchor_mode);
        for (int64_t i = 0; i < n; ++i) e[i] = eviction_score(s[i]);
        select_topn_window(e.data(), n, a.N, a.window, S.data(), &tau);
        if (a.e_out) std::copy(e.begin(), e.end(), a.e_out);
    }
    // gather(K,S), gather(V,S): bit-exact row copies in token order
    for (size_t j = 0; j < S.size(); ++j) {
        std::memcpy(a.k_out + j * d, k_row(S[j]), d * sizeof(uint16_t));
        std::memcpy(a.v_out + j * d, v_row(S[j]), d * sizeof(uint16_t));
    }
    if (a.len_out) *a.len_out = static_cast<int64_t>(S.size());
    if (a.S_out) std::copy(S.begin(), S.end(), a.S_out);
    if (a.tau_out) *a.tau_out = tau;
    if (a.m_out) *a.m_out = m;
}

// One unit with unordered slot reuse.  pos_in[len]: token position held by each valid slot;
// the block rows are tokens next_pos .. next_pos + B - 1.  Outputs: the whole new cache
// (k_out/v_out, N rows, the first min(N, len + B) slots valid), pos_out[N], src_out[N] = candidate
// number (slot for a cache row, len + j for block row j) of what each valid slot now holds.
struct SlotArgs {
    const int64_t* pos_in; int64_t next_pos; int64_t* pos_out; int64_t* src_out;
};
void evict_head_slots(const HeadArgs& a, const SlotArgs& sa) {
    const int64_t n = a.len + a.B, d = a.d, N = a.N;
    auto k_row = [&](int64_t i) { return i < a.len ? a.k_cache + i * d : a.new_k + (i - a.len) * d; };
    auto v_row = [&](int64_t i) { return i < a.len ? a.v_cache + i * d : a.new_v + (i - a.len) * d; };
    auto pos_of = [&](int64_t i) { return i < a.len ? sa.pos_in[i] : sa.next_pos + (i - a.len); };
    // the cache as it stands
    for (int64_t i = 0; i < a.len; ++i) {
        std::memcpy(a.k_out + i * d, k_row(i), d * sizeof(uint16_t));
        std::memcpy(a.v_out + i * d, v_row(i), d * sizeof(uint16_t));
        sa.pos_out[i] = sa.pos_in[i];
        sa.src_out[i] = i;
    }
    std::vector<char> keep(n, 1);
    double tau = 0.0, m = 0.0;
    if (n > N) {
        std::vector<double> K(static_cast<size_t>(n) * d), s(n), e(n);
        for (int64_t i = 0; i < n; ++i)
            for (int64_t c = 0; c < d; ++c) K[i * d + c] = bf16_bits_to_double(k_row(i)[c]);
        scores_f64(K.data(), n, d, a.eps, nullptr, nullptr, &m, s.data(), a.anchor_mode);
        for (int64_t i = 0; i < n; ++i) e[i] = eviction_score(s[i]);
        if (a.e_out) std::copy(e.begin(), e.end(), a.e_out);
        // the window: tokens among the last `window` positions of the sequence are kept whatever they score
        const int64_t first_recent = sa.next_pos + a.B - a.window;
        std::vector<int64_t> rest;            // candidates the score rule decides on, in candidate order
        for (int64_t i = 0; i < n; ++i) if (pos_of(i) < first_recent) rest.push_back(i);
        const int64_t in_window = n - static_cast<int64_t>(rest.size());
        const int64_t quota = N - in_window;  // places left for them
        std::vector<double> er(rest.size());
        for (size_t j = 0; j < rest.size(); ++j) er[j] = e[rest[j]];
        std::vector<int64_t> S(std::max<int64_t>(quota, 0));
        const int64_t kept_rest = (quota > 0 && !rest.empty()) ? select_topn(er.data(), er.size(), quota, S.data(), &tau) : 0;
        for (int64_t i : rest) keep[i] = 0;
        for (int64_t j = 0; j < kept_rest; ++j) keep[rest[S[j]]] = 1;
    }
    // freed slots in ascending order take the kept block rows in block order
    int64_t slot = 0;
    auto next_free = [&]() {
        while (slot < a.len && keep[slot]) ++slot;   // slots >= len are empty
        return slot++;
    };
    for (int64_t j = 0; j < a.B; ++j) {
        const int64_t i = a.len + j;
        if (!keep[i]) continue;
        const int64_t t = next_free();
        std::memcpy(a.k_out + t * d, k_row(i), d * sizeof(uint16_t));
        std::memcpy(a.v_out + t * d, v_row(i), d * sizeof(uint16_t));
        sa.pos_out[t] = pos_of(i);
        sa.src_out[t] = i;
    }
    if (a.len_out) *a.len_out = std::min(N, n);
    if (a.tau_out) *a.tau_out = tau;
    if (a.m_out) *a.m_out = m;
}

}  // namespace

extern "C" {

// Scores of n keys (row-major doubles).  s = cosine to the anchor (NOT negated).
void kd_oracle_scores(const double* K, int64_t n, int64_t d, double eps,
                      double* r, double* mu, double* m, double* s) {
    scores_f64(K, n, d, eps, r, mu, m, s);
}

// The same with the anchor variant chosen: 0 = mean of normalised keys, 1 = mean of raw keys.
void kd_oracle_scores_ex(const double* K, int64_t n, int64_t d, double eps, int32_t anchor_mode,
                         double* r, double* mu, double* m, double* s) {
    scores_f64(K, n, d, eps, r, mu, m, s, anchor_mode);
}

// Kept indices (ascending) with a window of w always-kept most recent tokens; returns the count.
int64_t kd_oracle_select_window(const double* e, int64_t n, int64_t N, int64_t w, int64_t* S, double* tau) {
    return select_topn_window(e, n, N, w, S, tau);
}

// e[i] = eviction score of cosine s[i].
void kd_oracle_eviction_scores(const double* s, int64_t n, double* e) {
    for (int64_t i = 0; i < n; ++i) e[i] = eviction_score(s[i]);
}

// Indices (ascending) of the min(N,n) kept tokens; returns that count.
int64_t kd_oracle_select(const double* e, int64_t n, int64_t N, int64_t* S, double* tau) {
    return select_topn(e, n, N, S, tau);
}

// Eq. (keydiff) literally: rowsum[i] = sum_j k_i.k_j / (||k_i|| ||k_j||).
void kd_oracle_pairwise_rowsum(const double* K, int64_t n, int64_t d, double* rowsum) {
    std::vector<double> r(n);
    for (int64_t i = 0; i < n; ++i) {
        double ss = 0.0;
        for (int64_t c = 0; c < d; ++c) ss += K[i * d + c] * K[i * d + c];
        r[i] = std::sqrt(ss);
    }
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            double dot = 0.0;
            for (int64_t c = 0; c < d; ++c) dot += K[i * d + c] * K[j * d + c];
            acc += dot / (r[i] * r[j]);
        }
        rowsum[i] = acc;
    }
}

// One unit on bf16 bit patterns.  k_cache/v_cache hold `len` valid rows of d
// elements, new_k/new_v hold B rows.  k_out/v_out receive min(N, len+B) rows.
// e_out (len+B doubles, written only when an eviction happens), S_out
// (min(N,len+B) indices), tau_out, m_out may be null.
void kd_oracle_evict_head_bf16(const uint16_t* k_cache, const uint16_t* v_cache, int64_t len,
                               const uint16_t* new_k, const uint16_t* new_v, int64_t B,
                               int64_t N, int64_t d, double eps,
                               uint16_t* k_out, uint16_t* v_out, int64_t* len_out,
                               double* e_out, int64_t* S_out, double* tau_out, double* m_out) {
    evict_head(HeadArgs{k_cache, v_cache, len, new_k, new_v, B, N, d, eps,
                        k_out, v_out, len_out, e_out, S_out, tau_out, m_out});
}

// U independent units.  Layouts: caches [U][N][d] (rows [0,len) valid), blocks
// [U][B][d], outputs k_out/v_out [U][N][d], e_out [U][len+B], S_out [U][N],
// tau_out/m_out [U].  Units are spread over n_threads std::threads (each unit is
// still computed by the single-threaded routine above).  Returns the number of
// threads actually used.
int32_t kd_oracle_evict_units_bf16(const uint16_t* k_cache, const uint16_t* v_cache, int64_t len,
                                   const uint16_t* new_k, const uint16_t* new_v, int64_t B,
                                   int64_t N, int64_t d, double eps, int64_t U,
                                   uint16_t* k_out, uint16_t* v_out,
                                   double* e_out, int64_t* S_out, double* tau_out, double* m_out,
                                   int32_t n_threads) {
    const int64_t n = len + B;
    auto run_unit = [&](int64_t u) {
        evict_head(HeadArgs{k_cache + u * N * d, v_cache + u * N * d, len,
                            new_k + u * B * d, new_v + u * B * d, B, N, d, eps,
                            k_out + u * N * d, v_out + u * N * d, nullptr,
                            e_out ? e_out + u * n : nullptr,
                            S_out ? S_out + u * N : nullptr,
                            tau_out ? tau_out + u : nullptr,
                            m_out ? m_out + u : nullptr});
    };
    int32_t T = std::max<int32_t>(1, std::min<int64_t>(n_threads, U));
    if (T == 1) {
        for (int64_t u = 0; u < U; ++u) run_unit(u);
        return 1;
    }
    std::vector<std::thread> pool;
    for (int32_t t = 0; t < T; ++t)
        pool.emplace_back([&, t] { for (int64_t u = t; u < U; u += T) run_unit(u); });
    for (auto& th : pool) th.join();
    return T;
}

// The same with the anchor variant and the sliding window chosen (single-threaded per call; the
// Python wrapper spreads units over threads by calling it on slices).
void kd_oracle_evict_units_bf16_ex(const uint16_t* k_cache, const uint16_t* v_cache, int64_t len,
                                   const uint16_t* new_k, const uint16_t* new_v, int64_t B,
                                   int64_t N, int64_t d, double eps, int64_t U, int32_t anchor_mode, int64_t window,
                                   uint16_t* k_out, uint16_t* v_out,
                                   double* e_out, int64_t* S_out, double* tau_out, double* m_out) {
    const int64_t n = len + B;
    for (int64_t u = 0; u < U; ++u) {
        HeadArgs a{k_cache + u * N * d, v_cache + u * N * d, len, new_k + u * B * d, new_v + u * B * d, B, N, d, eps,
                   k_out + u * N * d, v_out + u * N * d, nullptr,
                   e_out ? e_out + u * n : nullptr, S_out ? S_out + u * N : nullptr,
                   tau_out ? tau_out + u : nullptr, m_out ? m_out + u : nullptr};
        a.anchor_mode = anchor_mode;
        a.window = window;
        evict_head(a);
    }
}

// U units with unordered slot reuse (single-threaded per call).  pos_in/pos_out/src_out: [U][N];
// e_out [U][len+B] (written only when an eviction happens); the other layouts as above.
void kd_oracle_evict_units_bf16_slots(const uint16_t* k_cache, const uint16_t* v_cache, const int64_t* pos_in,
                                      int64_t len, int64_t next_pos,
                                      const uint16_t* new_k, const uint16_t* new_v, int64_t B,
                                      int64_t N, int64_t d, double eps, int64_t U, int32_t anchor_mode, int64_t window,
                                      uint16_t* k_out, uint16_t* v_out, int64_t* pos_out, int64_t* src_out,
                                      double* e_out, double* tau_out, double* m_out) {
    const int64_t n = len + B;
    for (int64_t u = 0; u < U; ++u) {
        HeadArgs a{k_cache + u * N * d, v_cache + u * N * d, len, new_k + u * B * d, new_v + u * B * d, B, N, d, eps,
                   k_out + u * N * d, v_out + u * N * d, nullptr,
                   e_out ? e_out + u * n : nullptr, nullptr,
                   tau_out ? tau_out + u : nullptr, m_out ? m_out + u : nullptr};
        a.anchor_mode = anchor_mode;
        a.window = window;
        evict_head_slots(a, SlotArgs{pos_in + u * N, next_pos, pos_out + u * N, src_out + u * N});
    }
}

}  // extern "C"
