// CPU ORACLE for the SkipKV eviction / decode hot path.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, step-by-step restatement of what the path computes, written from the
// paper's definitions (Section 4.1 "Skipping KV Storage with Sentence-level Scoring",
// Section 4.2 "Skipping KV Generation with Adaptive Steering", Algorithm 1).  It shares no
// code with the CUDA library and must never be reached from the product path; only the
// tests, the smoke check and the benchmark's cpu-baseline leg may build or call it.
//
// All floating-point accumulation is in double; bf16 inputs are widened exactly; each
// output is rounded once (fp32 scores, bf16 attention output).  No blocking, fusion or
// reordering beyond what each definition states.  OpenMP is used only across independent
// (sequence, KV head) slabs in the *_batch entry points.
//
// Readings of the paper taken here (the paper is silent or ambiguous on each):
//  * sentence embeddings are mean-pooled KEY rows of the (layer, KV head) slab;
//  * a sentence's score is Eq. "I_final" applied to sentence means (lambda is constant
//    over a sentence), and whole sentences are kept or evicted;
//  * the token importance is mean over the window rows of the max over the query heads
//    of a group of the softmax attention weights (no second softmax);
//  * redundancy R: row softmax of the cosine Gram matrix with the diagonal excluded,
//    then column mean with divisor S;
//  * lambda_i = max_{j>i} G_ij when that exceeds tau (strictly later sentences only).
// Parity of these readings with the authors' code is unpinned; each function below is
// pinned against closed forms / brute force in tests/test_oracle_pins.py.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return static_cast<double>(f);
}

inline float bits_to_float(uint32_t u) {
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

// double -> bf16, round to nearest even, decided in double (no double rounding).
inline uint16_t double_to_bf16(double x) {
    if (std::isnan(x)) return 0x7fc0;
    float f = static_cast<float>(x);
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if (std::isinf(f)) return static_cast<uint16_t>(u >> 16);
    uint32_t lo = u & 0xffff0000u;            // toward zero in magnitude
    uint32_t hi = lo + 0x10000u;              // next bf16 away from zero
    double dlo = std::fabs(static_cast<double>(bits_to_float(lo)));
    double dhi = std::fabs(static_cast<double>(bits_to_float(hi)));
    double ax = std::fabs(x);
    double elo = ax - dlo, ehi = dhi - ax;
    uint32_t pick;
    if (elo < ehi) pick = lo;
    else if (ehi < elo) pick = hi;
    else pick = ((lo >> 16) & 1u) ? hi : lo;  // tie: even mantissa
    return static_cast<uint16_t>(pick >> 16);
}

inline uint16_t float_to_bf16(float f) { return double_to_bf16(static_cast<double>(f)); }

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------------------
// O1  Token importance (Section 4.1, "Token Importance Score": A^i = softmax(Q^i K^{g(i)T}/sqrt(d)),
//     I^{h_k} from the max over the group's heads, normalised over the window).
//     K: [N][d] bf16 rows of one (sequence, KV head) slab; Q: [n][alpha][d] bf16, the n
//     query heads of that KV head's group.  tok_imp[t] = (1/alpha) sum_w max_q A^q[w][t].
// ---------------------------------------------------------------------------------------
void oracle_token_importance(const uint16_t* K, const uint16_t* Q, int N, int n, int alpha, int d,
                             double* tok_imp) {
    for (int t = 0; t < N; ++t) tok_imp[t] = 0.0;
    if (N == 0) return;
    const double scale = 1.0 / std::sqrt(static_cast<double>(d));
    std::vector<double> A(static_cast<size_t>(n) * N);
    for (int w = 0; w < alpha; ++w) {
        for (int q = 0; q < n; ++q) {
            const uint16_t* qrow = Q + (static_cast<size_t>(q) * alpha + w) * d;
            double* a = A.data() + static_cast<size_t>(q) * N;
            double mx = -std::numeric_limits<double>::infinity();
            for (int t = 0; t < N; ++t) {
                const uint16_t* krow = K + static_cast<size_t>(t) * d;
                double s = 0.0;
                for (int c = 0; c < d; ++c) s += bf16_to_double(qrow[c]) * bf16_to_double(krow[c]);
                s *= scale;
                a[t] = s;
                mx = std::max(mx, s);
            }
            double z = 0.0;
            for (int t = 0; t < N; ++t) { a[t] = std::exp(a[t] - mx); z += a[t]; }
            for (int t = 0; t < N; ++t) a[t] /= z;
        }
        for (int t = 0; t < N; ++t) {
            double m = A[t];
            for (int q = 1; q < n; ++q) m = std::max(m, A[static_cast<size_t>(q) * N + t]);
            tok_imp[t] += m;
        }
    }
    for (int t = 0; t < N; ++t) tok_imp[t] /= static_cast<double>(alpha);
}

// ---------------------------------------------------------------------------------------
// O2  Sentence pooling (Section 4.1, "Sentence Similarity Score": v_i = mean of the rows
//     of sentence i; normalisation as in the redundancy equation, x / (||x||_2 + eps)).
//     imp[i] = mean of tok_imp over the sentence; vbar: [S][d].
// ---------------------------------------------------------------------------------------
void oracle_pool(const uint16_t* K, int d, const int32_t* sent_off, int S, const double* tok_imp,
                 double eps, double* imp, double* vbar) {
    for (int i = 0; i < S; ++i) {
        const int b = sent_off[i], e = sent_off[i + 1];
        const double len = static_cast<double>(e - b);
        double si = 0.0;
        for (int t = b; t < e; ++t) si += tok_imp[t];
        imp[i] = (e > b) ? si / len : 0.0;
        double* v = vbar + static_cast<size_t>(i) * d;
        for (int c = 0; c < d; ++c) v[c] = 0.0;
        for (int t = b; t < e; ++t)
            for (int c = 0; c < d; ++c) v[c] += bf16_to_double(K[static_cast<size_t>(t) * d + c]);
        double nrm = 0.0;
        for (int c = 0; c < d; ++c) { v[c] = (e > b) ? v[c] / len : 0.0; nrm += v[c] * v[c]; }
        nrm = std::sqrt(nrm) + eps;
        for (int c = 0; c < d; ++c) v[c] /= nrm;
    }
}

// ---------------------------------------------------------------------------------------
// O3  Gram terms (pairwise sentence similarity, Eq. "PSS"; redundant set P; token
//     redundancy equation R = mean(softmax(Kbar Kbar^T)) taken at sentence granularity).
//     G_ij = vbar_i . vbar_j
//     P_jk = exp(G_jk) / sum_{k' != j} exp(G_jk')  (k != j),  P_jj = 0
//     red_i = (1/S) sum_j P_ji
//     lam_i = max_{j>i} G_ij  if that is > tau, else 0
//     G_out (nullable): [S][S].
// ---------------------------------------------------------------------------------------
void oracle_gram_terms(const double* vbar, int S, int d, double tau, double* G_out, double* red,
                       double* lam) {
    std::vector<double> G(static_cast<size_t>(S) * S);
    for (int i = 0; i < S; ++i)
        for (int j = 0; j < S; ++j) {
            double s = 0.0;
            for (int c = 0; c < d; ++c)
                s += vbar[static_cast<size_t>(i) * d + c] * vbar[static_cast<size_t>(j) * d + c];
            G[static_cast<size_t>(i) * S + j] = s;
        }
    if (G_out) std::copy(G.begin(), G.end(), G_out);
    for (int i = 0; i < S; ++i) red[i] = 0.0;
    for (int j = 0; j < S; ++j) {
        const double* g = G.data() + static_cast<size_t>(j) * S;
        double mx = -std::numeric_limits<double>::infinity();
        for (int k = 0; k < S; ++k) if (k != j) mx = std::max(mx, g[k]);
        double z = 0.0;
        for (int k = 0; k < S; ++k) if (k != j) z += std::exp(g[k] - mx);
        for (int k = 0; k < S; ++k) if (k != j) red[k] += std::exp(g[k] - mx) / z;
    }
    for (int i = 0; i < S; ++i) red[i] /= static_cast<double>(S);
    for (int i = 0; i < S; ++i) {
        double m = -std::numeric_limits<double>::infinity();
        for (int j = i + 1; j < S; ++j) m = std::max(m, G[static_cast<size_t>(i) * S + j]);
        lam[i] = (m > tau) ? m : 0.0;
    }
}

// ---------------------------------------------------------------------------------------
// O4  Final score (Eq. "I_final"): sigma*imp - (1-sigma)*red - lam, rounded once to fp32.
// ---------------------------------------------------------------------------------------
void oracle_final_score(const double* imp, const double* red, const double* lam, int S, double sigma,
                        float* score) {
    for (int i = 0; i < S; ++i)
        score[i] = static_cast<float>(sigma * imp[i] - (1.0 - sigma) * red[i] - lam[i]);
}

// ---------------------------------------------------------------------------------------
// O5  Selection under the budget (Section 4.1: evict in increasing order of final score
//     until the cache meets budget B).  Whole sentences.  If the slab already fits, keep
//     all.  Otherwise sentences that intersect the last protect_tail tokens rank first (in
//     index order); the rest rank by (score descending, index ascending); walk the ranking
//     summing lengths and keep the longest prefix whose total is <= budget (stop at the
//     first sentence that does not fit).  Returns n_kept; kept_idx ascending; new_len.
// ---------------------------------------------------------------------------------------
int oracle_select(const float* score, const int32_t* sent_off, int S, int budget, int protect_tail,
                  uint8_t* keep, int32_t* kept_idx, int32_t* new_len) {
    const int total = (S > 0) ? sent_off[S] : 0;
    for (int i = 0; i < S; ++i) keep[i] = 0;
    if (total <= budget) {
        for (int i = 0; i < S; ++i) { keep[i] = 1; kept_idx[i] = i; }
        *new_len = total;
        return S;
    }
    std::vector<int> order(S);
    std::vector<uint8_t> forced(S, 0);
    for (int i = 0; i < S; ++i) {
        order[i] = i;
        forced[i] = (protect_tail > 0 && sent_off[i + 1] > total - protect_tail && sent_off[i + 1] > sent_off[i]) ? 1 : 0;
    }
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        if (forced[a] != forced[b]) return forced[a] > forced[b];
        if (forced[a]) return a < b;
        if (score[a] != score[b]) return score[a] > score[b];
        return a < b;
    });
    long long cum = 0;
    for (int r = 0; r < S; ++r) {
        const int i = order[r];
        const int len = sent_off[i + 1] - sent_off[i];
        if (cum + len > budget) break;
        cum += len;
        keep[i] = 1;
    }
    int nk = 0;
    for (int i = 0; i < S; ++i) if (keep[i]) kept_idx[nk++] = i;
    *new_len = static_cast<int32_t>(cum);
    return nk;
}

// ---------------------------------------------------------------------------------------
// O6  Compaction (Section 4.1, "Updating Cache Ranges After Eviction", Eq. "after").
//     Survivor list p_1 < ... < p_B' = token indices of kept sentences in order.
//     K_out[k] = K[p_k] (same for V).  New ranges: b_i <- min{k : p_k >= b_i},
//     e_i <- max{k : p_k <= e_i} (inclusive ends), evaluated literally; a sentence with no
//     survivor is dropped.  new_sent_off is the CSR (exclusive-end) form of those ranges.
//     Returns the number of surviving sentences, or -1 if the literal remap is not the
//     contiguous prefix-sum form (cannot happen for whole-sentence eviction).
// ---------------------------------------------------------------------------------------
int oracle_compact(const uint16_t* K, const uint16_t* V, int d, const uint8_t* keep,
                   const int32_t* sent_off, const int32_t* sent_id, int S, uint16_t* K_out,
                   uint16_t* V_out, int32_t* index_map, int32_t* new_sent_off, int32_t* new_sent_id,
                   int32_t* new_len) {
    std::vector<int> p;
    for (int i = 0; i < S; ++i)
        if (keep[i])
            for (int t = sent_off[i]; t < sent_off[i + 1]; ++t) p.push_back(t);
    const int B = static_cast<int>(p.size());
    for (int k = 0; k < B; ++k) {
        index_map[k] = p[k];
        std::memcpy(K_out + static_cast<size_t>(k) * d, K + static_cast<size_t>(p[k]) * d, sizeof(uint16_t) * d);
        std::memcpy(V_out + static_cast<size_t>(k) * d, V + static_cast<size_t>(p[k]) * d, sizeof(uint16_t) * d);
    }
    int ns = 0;
    int expect_b = 0;
    new_sent_off[0] = 0;
    for (int i = 0; i < S; ++i) {
        const int b = sent_off[i], e = sent_off[i + 1] - 1;  // inclusive end
        if (e < b) continue;                                 // empty range
        int nb = -1, ne = -1;
        for (int k = 0; k < B; ++k) if (p[k] >= b) { nb = k; break; }
        for (int k = B - 1; k >= 0; --k) if (p[k] <= e) { ne = k; break; }
        if (nb < 0 || ne < 0 || nb > ne) continue;           // no survivor: range discarded
        if (nb != expect_b) return -1;
        new_sent_id[ns] = sent_id[i];
        new_sent_off[ns + 1] = ne + 1;
        expect_b = ne + 1;
        ++ns;
    }
    if (expect_b != B) return -1;
    *new_len = B;
    return ns;
}

// ---------------------------------------------------------------------------------------
// O7  Decode attention for one KV head's group (the attention equation of Section 4.1 with
//     a single query per head): out[q] = sum_t softmax_t(q.K[t]/sqrt(d)) V[t], bf16 out.
//     len == 0 gives zeros.
// ---------------------------------------------------------------------------------------
void oracle_decode_attn(const uint16_t* q, const uint16_t* K, const uint16_t* V, int len, int n, int d,
                        uint16_t* out, double* out_f64) {
    const double scale = 1.0 / std::sqrt(static_cast<double>(d));
    std::vector<double> s(std::max(len, 1)), acc(d);
    for (int j = 0; j < n; ++j) {
        std::fill(acc.begin(), acc.end(), 0.0);
        if (len > 0) {
            double mx = -std::numeric_limits<double>::infinity();
            for (int t = 0; t < len; ++t) {
                double x = 0.0;
                for (int c = 0; c < d; ++c)
                    x += bf16_to_double(q[static_cast<size_t>(j) * d + c]) * bf16_to_double(K[static_cast<size_t>(t) * d + c]);
                s[t] = x * scale;
                mx = std::max(mx, s[t]);
            }
            double z = 0.0;
            for (int t = 0; t < len; ++t) { s[t] = std::exp(s[t] - mx); z += s[t]; }
            for (int t = 0; t < len; ++t) {
                const double p = s[t] / z;
                for (int c = 0; c < d; ++c) acc[c] += p * bf16_to_double(V[static_cast<size_t>(t) * d + c]);
            }
        }
        for (int c = 0; c < d; ++c) {
            out[static_cast<size_t>(j) * d + c] = double_to_bf16(acc[c]);
            if (out_f64) out_f64[static_cast<size_t>(j) * d + c] = acc[c];
        }
    }
}

// ---------------------------------------------------------------------------------------
// O8  Steering add (Section 4.2: H <- H + alpha_t * v at delimiter tokens).  One fp32 fused
//     multiply-add per element, rounded to bf16; rows with flag == 0 are untouched.
// ---------------------------------------------------------------------------------------
void oracle_steer(int batch, int d_model, uint16_t* hidden, const uint16_t* v, const float* alpha,
                  const uint8_t* flag) {
    for (int b = 0; b < batch; ++b) {
        if (!flag[b]) continue;
        for (int c = 0; c < d_model; ++c) {
            uint16_t* h = hidden + static_cast<size_t>(b) * d_model + c;
            const float hf = static_cast<float>(bf16_to_double(*h));
            const float vf = static_cast<float>(bf16_to_double(v[c]));
            *h = float_to_bf16(std::fmaf(alpha[b], vf, hf));
        }
    }
}

// ---------------------------------------------------------------------------------------
// Batch drivers over the ragged slab layout (sequence b owns rows [slab_off[b]*Hk,
// (slab_off[b]+cap[b])*Hk); head h owns cap[b] consecutive rows).  One OpenMP task per
// (sequence, KV head) slab; nothing else is parallel.
// ---------------------------------------------------------------------------------------
void oracle_score_batch(int batch, int Hq, int Hk, int d, int alpha, int max_sent,
                        const int64_t* slab_off, const int32_t* cap, const uint16_t* K,
                        const uint16_t* q_win, const int32_t* kv_len, const int32_t* sent_off,
                        const int32_t* n_sent, double sigma, double tau, double eps,
                        double* tok_imp /*nullable, same row indexing as K */, double* sent_imp,
                        double* sent_red, double* sent_lam, float* sent_score) {
    const int n = Hq / Hk;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < batch * Hk; ++bh) {
        const int b = bh / Hk, h = bh % Hk;
        const size_t row0 = static_cast<size_t>(slab_off[b]) * Hk + static_cast<size_t>(h) * cap[b];
        const int N = kv_len[bh];
        const int S = n_sent[bh];
        const uint16_t* Ks = K + row0 * d;
        const uint16_t* Qs = q_win + (static_cast<size_t>(b) * Hq + static_cast<size_t>(h) * n) * alpha * d;
        const int32_t* so = sent_off + static_cast<size_t>(bh) * (max_sent + 1);
        std::vector<double> ti(std::max(N, 1)), vbar(static_cast<size_t>(std::max(S, 1)) * d);
        oracle_token_importance(Ks, Qs, N, n, alpha, d, ti.data());
        if (tok_imp) std::copy(ti.begin(), ti.begin() + N, tok_imp + row0);
        double* imp = sent_imp + static_cast<size_t>(bh) * max_sent;
        double* red = sent_red + static_cast<size_t>(bh) * max_sent;
        double* lam = sent_lam + static_cast<size_t>(bh) * max_sent;
        oracle_pool(Ks, d, so, S, ti.data(), eps, imp, vbar.data());
        oracle_gram_terms(vbar.data(), S, d, tau, nullptr, red, lam);
        oracle_final_score(imp, red, lam, S, sigma, sent_score + static_cast<size_t>(bh) * max_sent);
    }
}

void oracle_select_batch(int n_slabs, int max_sent, const float* sent_score, const int32_t* sent_off,
                         const int32_t* n_sent, int budget, int protect_tail, uint8_t* keep,
                         int32_t* kept_idx, int32_t* n_kept, int32_t* new_len) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < n_slabs; ++bh)
        n_kept[bh] = oracle_select(sent_score + static_cast<size_t>(bh) * max_sent,
                                   sent_off + static_cast<size_t>(bh) * (max_sent + 1), n_sent[bh], budget,
                                   protect_tail, keep + static_cast<size_t>(bh) * max_sent,
                                   kept_idx + static_cast<size_t>(bh) * max_sent, new_len + bh);
}

// In-place on copies held by the caller: K and V are overwritten slab by slab (through a
// temporary), tables updated.  index_map: [same row indexing as K], nullable.  Returns 0,
// or -1 if any slab's literal range remap disagreed with the prefix-sum form.
int oracle_compact_batch(int batch, int Hk, int d, int max_sent, const int64_t* slab_off,
                         const int32_t* cap, uint16_t* K, uint16_t* V, const uint8_t* keep,
                         int32_t* sent_off, int32_t* sent_id, int32_t* n_sent, int32_t* kv_len,
                         int32_t* index_map) {
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < batch * Hk; ++bh) {
        const int b = bh / Hk, h = bh % Hk;
        const size_t row0 = static_cast<size_t>(slab_off[b]) * Hk + static_cast<size_t>(h) * cap[b];
        const int S = n_sent[bh];
        int32_t* so = sent_off + static_cast<size_t>(bh) * (max_sent + 1);
        int32_t* sid = sent_id + static_cast<size_t>(bh) * max_sent;
        const int N = kv_len[bh];
        std::vector<uint16_t> Ko(static_cast<size_t>(std::max(N, 1)) * d), Vo(static_cast<size_t>(std::max(N, 1)) * d);
        std::vector<int32_t> im(std::max(N, 1)), nso(S + 1), nsid(std::max(S, 1));
        int32_t nl = 0;
        const int ns = oracle_compact(K + row0 * d, V + row0 * d, d, keep + static_cast<size_t>(bh) * max_sent, so,
                                      sid, S, Ko.data(), Vo.data(), im.data(), nso.data(), nsid.data(), &nl);
        if (ns < 0) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        std::memcpy(K + row0 * d, Ko.data(), sizeof(uint16_t) * static_cast<size_t>(nl) * d);
        std::memcpy(V + row0 * d, Vo.data(), sizeof(uint16_t) * static_cast<size_t>(nl) * d);
        if (index_map) std::copy(im.begin(), im.begin() + nl, index_map + row0);
        for (int i = 0; i <= ns; ++i) so[i] = nso[i];
        for (int i = ns + 1; i <= max_sent; ++i) so[i] = nl;
        for (int i = 0; i < ns; ++i) sid[i] = nsid[i];
        for (int i = ns; i < max_sent; ++i) sid[i] = -1;
        n_sent[bh] = ns;
        kv_len[bh] = nl;
    }
    return bad ? -1 : 0;
}

void oracle_decode_attn_batch(int batch, int Hq, int Hk, int d, const int64_t* slab_off,
                              const int32_t* cap, const uint16_t* q, const uint16_t* K,
                              const uint16_t* V, const int32_t* kv_len, uint16_t* out, double* out_f64) {
    const int n = Hq / Hk;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < batch * Hk; ++bh) {
        const int b = bh / Hk, h = bh % Hk;
        const size_t row0 = static_cast<size_t>(slab_off[b]) * Hk + static_cast<size_t>(h) * cap[b];
        const size_t o = (static_cast<size_t>(b) * Hq + static_cast<size_t>(h) * n) * d;
        oracle_decode_attn(q + o, K + row0 * d, V + row0 * d, kv_len[bh], n, d, out + o,
                           out_f64 ? out_f64 + o : nullptr);
    }
}

int oracle_max_threads(void);
}  // extern "C"

#ifdef _OPENMP
#include <omp.h>
extern "C" int oracle_max_threads(void) { return omp_get_max_threads(); }
extern "C" void oracle_set_threads(int n) { omp_set_num_threads(n); }
#else
extern "C" int oracle_max_threads(void) { return 1; }
extern "C" void oracle_set_threads(int) {}
#endif
