// CPU oracle for the S3-Attention streaming-scan hot path.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain statement of what the path computes, written from the paper's
// definitions.  It is used by the tests, by the smoke check and by the benchmark's CPU-baseline
// leg, and by nothing else: the product (the CUDA library) never includes, links or calls it and
// shares no source with it.  All floating-point arithmetic is fp64 unless a comment says that the
// method fixes fp32 (the final fused span score).  OpenMP only splits independent tokens/queries
// between threads; the arithmetic of one output never depends on the thread count.
//
// Parity pins (tests/test_oracle_*.py): numpy fp64 matmul, brute-force full sort, closed forms
// (identity SAE, x = b_dec, one-hot x, IDF(0) = 1, IDF(e-1) = 1/2), the index-size formula with the
// paper's printed 256 MiB instance, index inversion, a hand-computed co-activation example, and
// planted-mistake checks.  Nothing here is "parity unpinned".
//
// Readings of points the paper leaves open are listed where they are applied.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <utility>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// Sec. 3.3, Eq. 1 (before the ReLU): pre[t,f] = sum_i W_enc[i,f] * (x[t,i] - b_dec[i]) + b_enc[f].
// W_enc is stored [d_in, d_sae] row-major; feature f is column f.  The sum runs over i = 0..d_in-1
// in index order, in fp64, starting from 0; b_enc is added last.  Inputs are fp32 arrays (bf16 inputs
// are passed widened, which is exact).
void s3o_preact(const float* x, const float* W, const float* b_enc, const float* b_dec,
                int64_t T, int d_in, int d_sae, double* pre /*[T,d_sae]*/)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        double* out = pre + t * (int64_t)d_sae;
        for (int f = 0; f < d_sae; ++f) out[f] = 0.0;
        for (int i = 0; i < d_in; ++i) {
            const double xc = (double)x[t * (int64_t)d_in + i] - (double)b_dec[i];
            const float* wrow = W + (int64_t)i * d_sae;
            for (int f = 0; f < d_sae; ++f) out[f] += (double)wrow[f] * xc;
        }
        for (int f = 0; f < d_sae; ++f) out[f] += (double)b_enc[f];
    }
}

// Sec. 3.3, Eq. 1 (ReLU) and Eq. 2 (TopK), Sec. 3.4 Eq. 3 (Indices).
// Reading: only strictly positive activations can be selected, so a token yields min(k, #positive)
// features; equal activations are ordered by lower feature id.  Each output row is sorted by
// (activation descending, id ascending) and padded with id -1 / value 0.  The activation is
// reported rounded to fp32.
void s3o_topk(const double* pre, int64_t T, int d_sae, int k, int32_t* ids /*[T,k]*/, float* vals /*[T,k]*/)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const double* z = pre + t * (int64_t)d_sae;
        std::vector<std::pair<double, int32_t>> cand;
        for (int f = 0; f < d_sae; ++f)
            if (z[f] > 0.0) cand.emplace_back(z[f], f);
        std::sort(cand.begin(), cand.end(), [](const std::pair<double, int32_t>& a, const std::pair<double, int32_t>& b) {
            if (a.first != b.first) return a.first > b.first;
            return a.second < b.second;
        });
        for (int j = 0; j < k; ++j) {
            if (j < (int)cand.size()) {
                ids[t * k + j] = cand[j].second;
                vals[t * k + j] = (float)cand[j].first;
            } else {
                ids[t * k + j] = -1;
                vals[t * k + j] = 0.0f;
            }
        }
    }
}

// Sec. 3.4, Eq. 4 for one chunk: I[f] <- I[f] U {t} for every f in F_t, written as a CSR.
// Pairs (f, pos_base + t) are collected in token order and stably sorted by f, so each list is in
// ascending absolute position.  ids < 0 are padding and are skipped.  row_ptr has d_sae+1 entries.
// pval (optional, may be null together with vals) carries the activation next to each position.
void s3o_postings(const int32_t* ids, const float* vals, int64_t T, int k, int d_sae, int64_t pos_base,
                  uint32_t* row_ptr, int32_t* pos, float* pval)
{
    struct Pair { int32_t f; int32_t p; float v; };
    std::vector<Pair> pairs;
    for (int64_t t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            const int32_t f = ids[t * k + j];
            if (f >= 0) pairs.push_back({f, (int32_t)(pos_base + t), vals ? vals[t * k + j] : 0.0f});
        }
    std::stable_sort(pairs.begin(), pairs.end(), [](const Pair& a, const Pair& b) { return a.f < b.f; });
    for (int f = 0; f <= d_sae; ++f) row_ptr[f] = 0;
    for (const Pair& p : pairs) row_ptr[p.f + 1] += 1;
    for (int f = 0; f < d_sae; ++f) row_ptr[f + 1] += row_ptr[f];
    for (size_t i = 0; i < pairs.size(); ++i) {
        pos[i] = pairs[i].p;
        if (pval) pval[i] = pairs[i].v;
    }
}

// Sec. 3.4: the host index of one layer is, per feature, the concatenation of the chunk lists in
// arrival order (chunks arrive in ascending position, so lists stay ascending).
void s3o_index_merge(int n_chunks, const uint32_t* const* row_ptrs, const int32_t* const* poss, int d_sae,
                     uint64_t* row_ptr /*[d_sae+1]*/, int32_t* pos)
{
    row_ptr[0] = 0;
    for (int f = 0; f < d_sae; ++f) {
        uint64_t n = 0;
        for (int c = 0; c < n_chunks; ++c) n += row_ptrs[c][f + 1] - row_ptrs[c][f];
        row_ptr[f + 1] = row_ptr[f] + n;
    }
    for (int f = 0; f < d_sae; ++f) {
        uint64_t o = row_ptr[f];
        for (int c = 0; c < n_chunks; ++c)
            for (uint32_t i = row_ptrs[c][f]; i < row_ptrs[c][f + 1]; ++i) pos[o++] = poss[c][i];
    }
}

// Appendix IDF definition: IDF(f) = 1 / (log(1 + freq(f)) + 1), natural logarithm (reading).
double s3o_idf(double freq) { return 1.0 / (std::log(1.0 + freq) + 1.0); }

// Span scoring straight from the tokens' feature sets (no posting lists are consulted).
//
// ctx_ids [n_layers, L, k]   the context tokens' feature ids per layer (-1 = padding)
// q_ids   [n_layers, Q, nq, kq], q_vals same shape: the query tokens' features and activations
// Span j covers positions [j*stride, j*stride + width); n_spans = (L - width)/stride + 1 (0 if L < width).
//
// Query aggregation (reading of Eq. 5 for a query of several tokens):
//   cQ(f) = number of the query's tokens whose feature set contains f,
//   aQ(f) = sum of those tokens' activations of f (token order, fp64).
// mode 0 (co-activation count): coact[q,j] = sum_l sum_f min(cQ_l(f), cS_l(f,j)),
//   cS_l(f,j) = number of positions in span j whose layer-l feature set contains f.
// mode 1 (Eq. 6 summed over the span): w[q,j] = sum_l sum_f aQ_l(f) * IDF_l(f) * cS_l(f,j), features
//   in ascending id, layers in ascending order, fp64; freq_l(f) = number of context positions with f
//   active in layer l; features with freq > stop_freq are skipped when stop_freq > 0 (the paper's
//   hard stop-feature threshold).
void s3o_score_spans(const int32_t* ctx_ids, int64_t L, int k, int d_sae, int n_layers,
                     const int32_t* q_ids, const float* q_vals, int Q, int nq, int kq,
                     int width, int stride, int mode, int64_t stop_freq,
                     int64_t* coact /*[Q,n_spans] or null*/, double* wscore /*[Q,n_spans] or null*/)
{
    const int64_t n_spans = (L >= width) ? (L - width) / stride + 1 : 0;
    if (n_spans == 0) return;
    // document frequency per layer and feature
    std::vector<std::vector<int64_t>> freq(n_layers, std::vector<int64_t>(d_sae, 0));
    for (int l = 0; l < n_layers; ++l)
        for (int64_t t = 0; t < L; ++t)
            for (int j = 0; j < k; ++j) {
                const int32_t f = ctx_ids[((int64_t)l * L + t) * k + j];
                if (f >= 0) freq[l][f] += 1;
            }
#pragma omp parallel for schedule(dynamic, 1)
    for (int q = 0; q < Q; ++q) {
        std::vector<int64_t> acc_i(n_spans, 0);
        std::vector<double> acc_w(n_spans, 0.0);
        std::vector<int32_t> cQ(d_sae), cS(d_sae);
        std::vector<double> aQ(d_sae);
        for (int l = 0; l < n_layers; ++l) {
            std::fill(cQ.begin(), cQ.end(), 0);
            std::fill(aQ.begin(), aQ.end(), 0.0);
            for (int u = 0; u < nq; ++u)
                for (int j = 0; j < kq; ++j) {
                    const int64_t o = (((int64_t)l * Q + q) * nq + u) * kq + j;
                    const int32_t f = q_ids[o];
                    if (f >= 0) { cQ[f] += 1; aQ[f] += (double)q_vals[o]; }
                }
            for (int64_t s = 0; s < n_spans; ++s) {
                std::fill(cS.begin(), cS.end(), 0);
                for (int64_t t = s * stride; t < s * stride + width; ++t)
                    for (int j = 0; j < k; ++j) {
                        const int32_t f = ctx_ids[((int64_t)l * L + t) * k + j];
                        if (f >= 0) cS[f] += 1;
                    }
                if (mode == 0) {
                    int64_t sum = 0;
                    for (int f = 0; f < d_sae; ++f) sum += std::min(cQ[f], cS[f]);
                    acc_i[s] += sum;
                } else {
                    double sum = 0.0;
                    for (int f = 0; f < d_sae; ++f) {
                        if (cQ[f] == 0 || cS[f] == 0) continue;
                        if (stop_freq > 0 && freq[l][f] > stop_freq) continue;
                        sum += aQ[f] * s3o_idf((double)freq[l][f]) * (double)cS[f];
                    }
                    acc_w[s] += sum;
                }
            }
        }
        for (int64_t s = 0; s < n_spans; ++s) {
            if (coact) coact[q * n_spans + s] = acc_i[s];
            if (wscore) wscore[q * n_spans + s] = acc_w[s];
        }
    }
}

// Score fusion and span selection (benchmark definition; the paper's own fusion is a set union).
// score[q,j] = fl32( fl32(alpha * base) + fl32(beta * bm25[q,j]) ), base = (float)coact or (float)wscore;
// every operation is a single fp32 rounding (no fused multiply-add; compile with -ffp-contract=off).
// bm25 == null means no lexical term: score = fl32(alpha * base).
// The s best spans are taken from a full sort by (score descending, span index ascending); when
// n_spans < s the tail is padded with index -1 / score 0.
void s3o_fuse_select(const int64_t* coact, const double* wscore, const float* bm25, float alpha, float beta,
                     int Q, int64_t n_spans, int s, int32_t* top_idx /*[Q,s]*/, float* top_score /*[Q,s]*/,
                     float* all_scores /*[Q,n_spans] or null*/)
{
#pragma omp parallel for schedule(static)
    for (int q = 0; q < Q; ++q) {
        std::vector<std::pair<float, int32_t>> sc(n_spans);
        for (int64_t j = 0; j < n_spans; ++j) {
            const float base = coact ? (float)coact[q * n_spans + j] : (float)wscore[q * n_spans + j];
            volatile float a = alpha * base;
            float v = a;
            if (bm25) {
                volatile float b = beta * bm25[q * n_spans + j];
                volatile float sum = a + b;
                v = sum;
            }
            sc[j] = {v, (int32_t)j};
            if (all_scores) all_scores[q * n_spans + j] = v;
        }
        std::sort(sc.begin(), sc.end(), [](const std::pair<float, int32_t>& a, const std::pair<float, int32_t>& b) {
            if (a.first != b.first) return a.first > b.first;
            return a.second < b.second;
        });
        for (int j = 0; j < s; ++j) {
            if (j < n_spans) { top_idx[q * s + j] = sc[j].second; top_score[q * s + j] = sc[j].first; }
            else { top_idx[q * s + j] = -1; top_score[q * s + j] = 0.0f; }
        }
    }
}

// Sec. 3.5, "Semantic Density Estimation" and "Adaptive Granularity" (Eq. 6; Alg. 1, Phase 2: S <- accumulate,
// S' <- Conv1D(S), Idx <- NMS_Select(S', top_k)), straight from the tokens' feature sets.
//
//   S[t]  = sum_l sum_{f in F_t^(l)} w_l(f),   w_l(f) = aQ_l(f) * IDF_l(f) for the query's features (else 0)
//   S'[t] = sum_{d=0}^{K-1} S[t - floor(K/2) + d]          (positions outside [0, L) count as 0)
//   centres: repeat n_centers times: the alive position with the largest S' (ties: lowest position); stop
//            when nothing alive has S' > 0; positions within nms_radius of a centre are no longer alive.
// Readings (the paper leaves these open): the query's tokens are aggregated as in s3o_score_spans, with
// aQ_l(f) summed in fp32 in query-token order; the smoothing kernel is a box of K unit taps centred on t;
// suppression is by distance to the chosen centres. So that the peak positions (an argmax) do not depend
// on summation order, every weight is taken in fixed point, w = rint(aQ * IDF * 2^24) / 2^24, and S, S' are
// then exact integer sums; this is the precision the selection is made in.
// Features with freq > stop_freq are skipped when stop_freq > 0.
void s3o_position_density(const int32_t* ctx_ids, int64_t L, int k, int d_sae, int n_layers,
                          const int32_t* q_ids, const float* q_vals, int Q, int nq, int kq,
                          int conv_kernel, int nms_radius, int n_centers, int64_t stop_freq,
                          double* S /*[Q,L] or null*/, double* D /*[Q,L] or null*/,
                          int32_t* centers /*[Q,n_centers]*/, float* center_density /*[Q,n_centers]*/)
{
    std::vector<std::vector<int64_t>> freq(n_layers, std::vector<int64_t>(d_sae, 0));
    for (int l = 0; l < n_layers; ++l)
        for (int64_t t = 0; t < L; ++t)
            for (int j = 0; j < k; ++j) {
                const int32_t f = ctx_ids[((int64_t)l * L + t) * k + j];
                if (f >= 0) freq[l][f] += 1;
            }
    const double scale = 16777216.0;   // 2^24
#pragma omp parallel for schedule(dynamic, 1)
    for (int q = 0; q < Q; ++q) {
        std::vector<int64_t> s_fix(L, 0), d_fix(L, 0);
        std::vector<int64_t> w(d_sae);
        std::vector<float> aQ(d_sae);
        std::vector<char> inq(d_sae);
        for (int l = 0; l < n_layers; ++l) {
            std::fill(aQ.begin(), aQ.end(), 0.0f);
            std::fill(inq.begin(), inq.end(), 0);
            for (int u = 0; u < nq; ++u)
                for (int j = 0; j < kq; ++j) {
                    const int64_t o = (((int64_t)l * Q + q) * nq + u) * kq + j;
                    const int32_t f = q_ids[o];
                    if (f >= 0) { volatile float sum = aQ[f] + q_vals[o]; aQ[f] = sum; inq[f] = 1; }
                }
            for (int f = 0; f < d_sae; ++f) {
                w[f] = 0;
                if (!inq[f]) continue;
                if (stop_freq > 0 && freq[l][f] > stop_freq) continue;
                w[f] = (int64_t)std::llrint((double)aQ[f] * s3o_idf((double)freq[l][f]) * scale);
            }
            for (int64_t t = 0; t < L; ++t)
                for (int j = 0; j < k; ++j) {
                    const int32_t f = ctx_ids[((int64_t)l * L + t) * k + j];
                    if (f >= 0) s_fix[t] += w[f];
                }
        }
        const int64_t half = conv_kernel / 2;
        for (int64_t t = 0; t < L; ++t) {
            int64_t sum = 0;
            for (int64_t d = 0; d < conv_kernel; ++d) {
                const int64_t u = t - half + d;
                if (u >= 0 && u < L) sum += s_fix[u];
            }
            d_fix[t] = sum;
        }
        for (int64_t t = 0; t < L; ++t) {
            if (S) S[q * L + t] = (double)s_fix[t] / scale;
            if (D) D[q * L + t] = (double)d_fix[t] / scale;
        }
        std::vector<char> alive(L, 1);
        for (int i = 0; i < n_centers; ++i) {
            int64_t best = -1;
            for (int64_t t = 0; t < L; ++t)
                if (alive[t] && d_fix[t] > 0 && (best < 0 || d_fix[t] > d_fix[best])) best = t;
            if (best < 0) { centers[q * n_centers + i] = -1; center_density[q * n_centers + i] = 0.0f; continue; }
            centers[q * n_centers + i] = (int32_t)best;
            center_density[q * n_centers + i] = (float)((double)d_fix[best] / scale);
            for (int64_t t = std::max<int64_t>(0, best - nms_radius); t <= std::min<int64_t>(L - 1, best + nms_radius); ++t) alive[t] = 0;
        }
    }
}

// Sec. 3.3, the reconstruction stated after Eq. 2: x_hat = z_hat W_dec + b_dec, with z_hat the Top-k code given as
// (id, value) pairs per token (id < 0 = padding). W_dec is [d_sae, d_in] row-major: row f is feature f's direction.
// fp64; the k terms are added in the order given, b_dec last. sqerr[t] (nullable) = sum_i (x[t,i] - x_hat[t,i])^2,
// the per-token reconstruction error whose batch mean is the quantity an SAE is trained to reduce.
void s3o_decode(const int32_t* ids, const float* vals, int64_t T, int k, const float* W_dec, const float* b_dec,
                int d_in, int d_sae, const float* x /*[T,d_in] or null*/, double* x_hat /*[T,d_in]*/, double* sqerr /*[T] or null*/)
{
    (void)d_sae;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        double* out = x_hat + t * (int64_t)d_in;
        for (int i = 0; i < d_in; ++i) out[i] = 0.0;
        for (int j = 0; j < k; ++j) {
            const int32_t f = ids[t * k + j];
            if (f < 0) continue;
            const double z = (double)vals[t * k + j];
            const float* row = W_dec + (int64_t)f * d_in;
            for (int i = 0; i < d_in; ++i) out[i] += z * (double)row[i];
        }
        for (int i = 0; i < d_in; ++i) out[i] += (double)b_dec[i];
        if (sqerr && x) {
            double e = 0.0;
            for (int i = 0; i < d_in; ++i) {
                const double d = (double)x[t * (int64_t)d_in + i] - out[i];
                e += d * d;
            }
            sqerr[t] = e;
        }
    }
}

int s3o_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}

}  // extern "C"
