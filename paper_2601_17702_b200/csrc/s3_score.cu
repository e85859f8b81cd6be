// Query-time span scoring (Sec. 3.5, Eq. 5-6; appendix IDF definition) fused with score fusion and
// top-s selection. One thread block per query:
//   a. aggregate the query tokens' Top-k into unique features with cQ (token count) and aQ (summed
//      activation): block bitonic sort of (id, entry) keys, then run detection;
//   b. fetch the unique features' list bounds in one parallel sweep, cut all lists into 32-posting
//      pieces and deal the pieces out evenly over the warps (a long list is simply many pieces, so
//      skewed list lengths do not unbalance the block). Every posting works out by itself which
//      spans it still adds to (see posting_range), for any width/stride. Min-count mode records the
//      range as +1/-1 in a difference array that one prefix sum turns into min(cQ, cS) totals;
//      weighted mode adds aQ*IDF to each span of the range in fp64;
//   c. fuse with the lexical score vector and pick the s best spans (score desc, index asc).
#include "s3_kernels.cuh"
#include "s3_query.cuh"

namespace s3 {

namespace {

struct CompactLayers {
    s3_compact_view v[S3_MAX_SCORE_LAYERS];
};
constexpr int CBATCH = 8;        // compact index: blocks of 32 postings a warp decodes side by side

struct ScoreArgs {
    const int32_t* q_ids;
    const float* q_vals;
    const float* bm25;
    int64_t ld_bm25;
    int32_t* top_idx;
    float* top_score;
    float* all_scores;
    int n_layers, d_sae, Q, nk /* nq*k */, npad, n_spans, width, stride, mode, s;
    float alpha, beta;
    int64_t stop_freq;
    int stride_shift;   // log2(stride) when the stride is a power of two, else -1
    unsigned long long stride_magic;   // ceil(2^64 / stride) (stride >= 2)
};

__device__ __forceinline__ uint32_t orderable(float v)
{
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// floor(p / stride) for 0 <= p < 2^31: a shift when the stride is a power of two (POW2), else the high word
// of p * ceil(2^64 / stride), which is exact for every 32-bit p.
template <bool POW2>
__device__ __forceinline__ int div_stride(int p, const ScoreArgs& a)
{
    if (POW2) return p >> a.stride_shift;
    return static_cast<int>(__umul64hi(static_cast<unsigned long long>(p), a.stride_magic));
}

// Spans that posting i of a list (position p, ascending positions) still adds to. The posting lies in
// spans lo(p)..hi(p), lo(p) = p >= width ? floor((p-width)/stride)+1 : 0, hi(p) = floor(p/stride).
// In min-count mode span j already holds cQ earlier postings of the feature exactly when posting i-cQ
// lies in it, i.e. when j <= hi(p_{i-cQ}); so the posting adds one to spans max(lo(p), hi(p_{i-cQ})+1)
// .. hi(p) only, and the totals come out as min(cQ, cS(f, j)). p_prev < 0 means "no such posting".
template <bool POW2>
__device__ __forceinline__ void posting_range(const ScoreArgs& a, int p, int p_prev, int& j_lo, int& j_hi)
{
    j_hi = div_stride<POW2>(p, a);
    j_lo = p >= a.width ? div_stride<POW2>(p - a.width, a) + 1 : 0;
    if (p_prev >= 0) {
        const int j_prev = div_stride<POW2>(p_prev, a) + 1;
        j_lo = j_prev > j_lo ? j_prev : j_lo;
    }
    j_hi = j_hi < a.n_spans - 1 ? j_hi : a.n_spans - 1;
}

// Compact index: the positions of a block of cnt postings in three steps, so that a warp can have the loads of
// several blocks in flight: header, the payload words of the lane's value, then value -> gap -> 32-lane prefix sum.
struct PieceHead {
    int first;
    unsigned long long desc;     // (payload word offset << 6) | width
    uint32_t cnt;                // postings in the block; 0 = no block
};
__device__ __forceinline__ PieceHead block_head(const s3_compact_view& v, uint32_t blk, uint32_t cnt)
{
    PieceHead h;
    h.first = __ldg(v.d_blk_first + blk);
    h.desc = __ldg(reinterpret_cast<const unsigned long long*>(v.d_blk_desc) + blk);
    h.cnt = cnt;
    return h;
}
__device__ __forceinline__ void block_value_words(const s3_compact_view& v, const PieceHead& h, int lane, uint32_t& lo, uint32_t& hi)
{
    lo = 0; hi = 0;
    const uint32_t width = static_cast<uint32_t>(h.desc & 63u);
    if (lane >= 1 && lane < static_cast<int>(h.cnt) && width) {
        const uint32_t* w = v.d_payload + (h.desc >> 6) + (((lane - 1) * width) >> 5);
        lo = __ldg(w);
        hi = __ldg(w + 1);                    // the payload's closing word keeps this in bounds
    }
}
__device__ __forceinline__ int block_positions(const PieceHead& h, int lane, uint32_t lo, uint32_t hi)
{
    const uint32_t width = static_cast<uint32_t>(h.desc & 63u);
    const uint32_t v = __funnelshift_r(lo, hi, ((lane - 1) * width) & 31) & ((1u << width) - 1u);
    int d = lane == 0 ? h.first : (lane < static_cast<int>(h.cnt) ? static_cast<int>(v) + 1 : 0);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, d, o);
        if (lane >= o) d += y;
    }
    return lane < static_cast<int>(h.cnt) ? d : -1;
}
// A full block decoded on the spot (three dependent steps; the rare path of the scorer).
__device__ __noinline__ int block_positions_now(const s3_compact_view& v, uint32_t blk, int lane)
{
    const PieceHead h = block_head(v, blk, 32u);
    uint32_t lo, hi;
    block_value_words(v, h, lane, lo, hi);
    return block_positions(h, lane, lo, hi);
}

template <bool POW2, bool COMPACT>
__global__ void __launch_bounds__(ST)
score_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ CompactLayers clayers,
             const __grid_constant__ ScoreArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    const bool weighted = a.mode == S3_SCORE_WEIGHTED;
    const ScoreSmem SL = score_smem(a.nk, a.npad, a.n_spans, weighted);
    int* acc_i = reinterpret_cast<int*>(score_smem_raw + SL.acc_off);          // min-count: difference array [n_spans+1]
    double* acc_d = reinterpret_cast<double*>(score_smem_raw + SL.acc_off);    // weighted: fp64 per span
    uint32_t* sel = reinterpret_cast<uint32_t*>(score_smem_raw + SL.acc_off);  // phase c: orderable fused scores
    unsigned long long* ulo = reinterpret_cast<unsigned long long*>(score_smem_raw + SL.ulo_off);
    uint32_t* keys = reinterpret_cast<uint32_t*>(score_smem_raw + SL.keys_off);
    uint32_t* ulen = keys;                                                      // keys are dead once aQ is summed
    int32_t* ufeat = reinterpret_cast<int32_t*>(score_smem_raw + SL.ufeat_off);
    int32_t* ustart = reinterpret_cast<int32_t*>(score_smem_raw + SL.ustart_off);
    float* uaq = reinterpret_cast<float*>(score_smem_raw + SL.uaq_off);
    uint16_t* owner = reinterpret_cast<uint16_t*>(score_smem_raw + SL.owner_off);
    uint32_t* cstart = reinterpret_cast<uint32_t*>(score_smem_raw + SL.cstart_off);   // same storage as ufeat: a thread
                                                                                        // reads ufeat[u], then writes cstart[u]
    __shared__ uint32_t ws[SW + 1];
    __shared__ unsigned long long red[SW];
    __shared__ int n_unique_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = blockIdx.x;

    if (weighted) { for (int j = tid; j < a.n_spans + 1; j += ST) acc_d[j] = 0.0; }
    else          { for (int j = tid; j < a.n_spans + 2; j += ST) acc_i[j] = 0; }
    __syncthreads();

    for (int l = 0; l < a.n_layers; ++l) {
        const int32_t* qi = a.q_ids + ((size_t)l * a.Q + q) * a.nk;
        const float* qv = a.q_vals + ((size_t)l * a.Q + q) * a.nk;
        const int U = aggregate_query(qi, qv, a.nk, a.npad, a.d_sae, weighted, keys, ufeat, ustart, uaq, ws, &n_unique_s);
        // b. list bounds of every unique feature (independent loads), then the pieces' prefix sum
        const int32_t* __restrict__ pos = layers.v[l].d_pos;
        const uint32_t piece_total = cut_lists(layers.v[l].d_row_ptr, U, weighted ? a.stop_freq : 0, ufeat, ulo, ulen, cstart, ws,
                                               COMPACT ? clayers.v[l].d_blk_ptr : nullptr);

        // The pieces are walked a window at a time; inside a window every warp takes an equal share. BATCH
        // pieces per round: first all their loads are issued, then their updates, so that a warp has BATCH
        // independent memory round trips in flight instead of one.
        for (uint32_t win0 = 0; win0 < piece_total; win0 += WIN) {
            const uint32_t win1 = piece_total - win0 < WIN ? piece_total : win0 + WIN;
            tabulate_owners(cstart, U, win0, win1, owner);
            const uint32_t n_win = win1 - win0;
            const uint32_t c_begin = win0 + static_cast<uint32_t>(static_cast<uint64_t>(n_win) * warp / SW);
            const uint32_t c_end = win0 + static_cast<uint32_t>(static_cast<uint64_t>(n_win) * (warp + 1) / SW);
            if constexpr (COMPACT) {
                // A piece is one block of the compact index. The headers of the next CBATCH blocks are fetched while
                // the payload words of the current ones are in flight, so a batch waits for one memory round trip.
                // In min-count mode posting i also needs the position of posting i - cQ of its list: the 32 lanes'
                // targets lie in at most two blocks, x = floor((32 j - cQ)/32) and x + 1. Block j itself is at hand; an
                // earlier block j - d is piece b - d of this warp (its pieces are consecutive) and is taken from the
                // batch or from the last two blocks of the previous batch; only when it lies further back (the start
                // of the warp's share, cQ > 64) is it decoded on the spot.
                const s3_compact_view& cv = clayers.v[l];
                auto fetch_head = [&](uint32_t c) {
                    PieceHead h;
                    h.first = 0; h.desc = 0; h.cnt = 0;
                    if (c < c_end) {
                        const int u = owner[c - win0];
                        const uint32_t j = c - cstart[u];
                        const uint32_t left = ulen[u] - 32u * j;
                        h = block_head(cv, static_cast<uint32_t>(ulo[u]) + j, left < 32u ? left : 32u);
                    }
                    return h;
                };
                PieceHead hn[CBATCH];
#pragma unroll
                for (int b = 0; b < CBATCH; ++b) hn[b] = fetch_head(c_begin + b);
                int carry1 = -1, carry2 = -1;                              // positions of pieces c0 - 1 and c0 - 2
                for (uint32_t c0 = c_begin; c0 < c_end; c0 += CBATCH) {
                    PieceHead hc[CBATCH];
                    uint32_t lo[CBATCH], hi[CBATCH];
                    int hist[CBATCH + 2];
#pragma unroll
                    for (int b = 0; b < CBATCH; ++b) {
                        hc[b] = hn[b];
                        block_value_words(cv, hc[b], lane, lo[b], hi[b]);
                    }
#pragma unroll
                    for (int b = 0; b < CBATCH; ++b) hn[b] = fetch_head(c0 + CBATCH + b);
                    hist[0] = carry2; hist[1] = carry1;
                    const int avail = c0 - c_begin < 2u ? static_cast<int>(c0 - c_begin) : 2;
#pragma unroll
                    for (int b = 0; b < CBATCH; ++b) {
                        hist[b + 2] = -1;
                        if (hc[b].cnt == 0) continue;                      // uniform over the warp
                        const int p = block_positions(hc[b], lane, lo[b], hi[b]);
                        hist[b + 2] = p;
                        const int u = owner[c0 + b - win0];
                        int p_prev = -1;
                        if (!weighted) {
                            const int j = static_cast<int>(c0 + b - cstart[u]);
                            const int cq = ustart[u + 1] - ustart[u];
                            const int x = (32 * j - cq) >> 5;              // floor, may be negative
                            int pr[3] = {p, -1, -1};
#pragma unroll
                            for (int r = 1; r <= 2; ++r) {
                                const int xb = x + r - 1;
                                if (xb >= 0 && xb < j) {
                                    const int d = j - xb;
                                    if (d <= b + avail) {
#pragma unroll
                                        for (int e = 1; e <= b + 2; ++e)
                                            if (d == e) pr[r] = hist[b + 2 - e];
                                    } else {
                                        pr[r] = block_positions_now(cv, static_cast<uint32_t>(ulo[u]) + xb, lane);
                                    }
                                }
                            }
                            const int src = (lane - cq) & 31;
                            const int v0 = __shfl_sync(0xffffffffu, pr[0], src);
                            const int v1 = __shfl_sync(0xffffffffu, pr[1], src);
                            const int v2 = __shfl_sync(0xffffffffu, pr[2], src);
                            const int t = 32 * j + lane - cq;              // list index of the earlier posting
                            if (t >= 0) {
                                const int tb = t >> 5;
                                p_prev = tb == j ? v0 : (tb == x ? v1 : v2);
                            }
                        }
                        if (p < 0) continue;
                        int j_lo, j_hi;
                        posting_range<POW2>(a, p, p_prev, j_lo, j_hi);
                        if (weighted) {
                            const double w = static_cast<double>(uaq[u]) * (1.0 / (log(1.0 + static_cast<double>(ulen[u])) + 1.0));
                            for (int jj = j_lo; jj <= j_hi; ++jj) atomicAdd(&acc_d[jj], w);
                        } else if (j_lo <= j_hi) {
                            atomicAdd(&acc_i[j_lo], 1);
                            atomicAdd(&acc_i[j_hi + 1], -1);
                        }
                    }
                    carry2 = hist[CBATCH]; carry1 = hist[CBATCH + 1];
                }
            } else
            for (uint32_t c0 = c_begin; c0 < c_end; c0 += BATCH) {
                int p[BATCH], p_prev[BATCH], ub[BATCH];
#pragma unroll
                for (int b = 0; b < BATCH; ++b) {
                    const uint32_t c = c0 + b;
                    p[b] = -1; p_prev[b] = -1; ub[b] = 0;
                    if (c < c_end) {
                        const int u = owner[c - win0];
                        ub[b] = u;
                        const int32_t* __restrict__ list = pos + ulo[u];
                        const uint32_t i = (c - cstart[u]) * PIECE + lane;
                        if (i < ulen[u]) {
                            p[b] = __ldg(list + i);
                            if (!weighted) {
                                const uint32_t cq = static_cast<uint32_t>(ustart[u + 1] - ustart[u]);
                                if (i >= cq) p_prev[b] = __ldg(list + i - cq);
                            }
                        }
                    }
                }
#pragma unroll
                for (int b = 0; b < BATCH; ++b) {
                    if (p[b] < 0) continue;
                    int j_lo, j_hi;
                    posting_range<POW2>(a, p[b], p_prev[b], j_lo, j_hi);
                    if (weighted) {
                        const double w = static_cast<double>(uaq[ub[b]]) *
                                         (1.0 / (log(1.0 + static_cast<double>(ulen[ub[b]])) + 1.0));
                        for (int j = j_lo; j <= j_hi; ++j) atomicAdd(&acc_d[j], w);
                    } else if (j_lo <= j_hi) {
                        atomicAdd(&acc_i[j_lo], 1);
                        atomicAdd(&acc_i[j_hi + 1], -1);
                    }
                }
            }
            __syncthreads();
        }
    }

    // min-count mode: difference array -> per-span totals (inclusive prefix sum, in place)
    if (!weighted) {
        uint32_t carry = 0;
        for (int j0 = 0; j0 < a.n_spans; j0 += ST) {
            const int j = j0 + tid;
            const uint32_t v = j < a.n_spans ? static_cast<uint32_t>(acc_i[j]) : 0u;
            uint32_t total;
            const uint32_t ex = block_exclusive_scan(v, ws, total) + carry;
            if (j < a.n_spans) acc_i[j] = static_cast<int>(ex + v);
            carry += total;
        }
        __syncthreads();
    }

    // c. fusion (one fp32 rounding per operation); the orderable score replaces the accumulator in place.
    // A pass reads its accumulators before any thread of the pass writes (the 4-byte results of weighted
    // mode land on 8-byte accumulators of the same or an earlier pass only).
    for (int j0 = 0; j0 < a.n_spans; j0 += ST) {
        const int j = j0 + tid;
        float v = 0.0f;
        if (j < a.n_spans) {
            const float base = weighted ? __double2float_rn(acc_d[j]) : __int2float_rn(acc_i[j]);
            v = __fmul_rn(a.alpha, base);
            if (a.bm25) v = __fadd_rn(v, __fmul_rn(a.beta, a.bm25[(size_t)q * a.ld_bm25 + j]));
            if (a.all_scores) a.all_scores[(size_t)q * a.n_spans + j] = v;
        }
        __syncthreads();
        if (j < a.n_spans) sel[j] = orderable(v);
    }
    __syncthreads();
    for (int r = 0; r < a.s; ++r) {
        unsigned long long best = 0ull;
        for (int j = tid; j < a.n_spans; j += ST) {
            const uint32_t o = sel[j];
            const unsigned long long key = o ? ((static_cast<unsigned long long>(o) << 32) | static_cast<uint32_t>(~static_cast<uint32_t>(j))) : 0ull;
            best = key > best ? key : best;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (lane == 0) red[warp] = best;
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < SW; ++w) best = red[w] > best ? red[w] : best;
            int idx = -1;
            float sc = 0.0f;
            if (best != 0ull) {
                idx = static_cast<int>(~static_cast<uint32_t>(best));
                const uint32_t o = static_cast<uint32_t>(best >> 32);
                sc = __uint_as_float((o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o);
                sel[idx] = 0u;                       // taken (0 is not the image of any non-NaN score)
            }
            a.top_idx[(size_t)q * a.s + r] = idx;
            a.top_score[(size_t)q * a.s + r] = sc;
        }
        __syncthreads();
    }
}

}  // namespace

namespace {

s3_status launch_score_impl(const ScoreLayers& layers, const CompactLayers* clayers, int n_layers, int d_sae, const int32_t* d_q_ids,
                            const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                            const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                            float* d_all_scores, cudaStream_t stream)
{
    static int max_smem_dev[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    int max_smem = dev < 64 ? max_smem_dev[dev] : 0;
    if (max_smem == 0) {
        S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        S3_CUDA_TRY(cudaFuncSetAttribute(score_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        S3_CUDA_TRY(cudaFuncSetAttribute(score_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        S3_CUDA_TRY(cudaFuncSetAttribute(score_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        S3_CUDA_TRY(cudaFuncSetAttribute(score_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        if (dev < 64) max_smem_dev[dev] = max_smem;
    }
    ScoreArgs a;
    a.q_ids = d_q_ids; a.q_vals = d_q_vals; a.bm25 = d_bm25; a.ld_bm25 = ld_bm25;
    a.top_idx = d_top_idx; a.top_score = d_top_score; a.all_scores = d_all_scores;
    a.n_layers = n_layers; a.d_sae = d_sae; a.Q = Q; a.nk = nq * k;
    int npad = 32;
    while (npad < a.nk) npad <<= 1;
    a.npad = npad; a.n_spans = n_spans; a.width = p->width; a.stride = p->stride; a.mode = p->mode; a.s = p->s;
    a.alpha = p->alpha; a.beta = p->beta; a.stop_freq = p->stop_freq;
    a.stride_shift = (p->stride & (p->stride - 1)) == 0 ? __builtin_ctz(static_cast<unsigned>(p->stride)) : -1;
    a.stride_magic = p->stride >= 2 ? ~0ull / static_cast<unsigned long long>(p->stride) + 1ull : 0ull;
    const size_t smem = score_smem(a.nk, npad, n_spans, p->mode == S3_SCORE_WEIGHTED).total;
    S3_REQUIRE(smem + 2048 <= static_cast<size_t>(max_smem), S3_ERR_UNSUPPORTED,
               "n_spans = %d with nq*k = %d needs %zu bytes of shared memory per query, %d available", n_spans, a.nk, smem,
               max_smem - 2048);
    if (clayers) {
        if (a.stride_shift >= 0) score_kernel<true, true><<<Q, ST, smem, stream>>>(layers, *clayers, a);
        else score_kernel<false, true><<<Q, ST, smem, stream>>>(layers, *clayers, a);
    } else {
        CompactLayers none = {};
        if (a.stride_shift >= 0) score_kernel<true, false><<<Q, ST, smem, stream>>>(layers, none, a);
        else score_kernel<false, false><<<Q, ST, smem, stream>>>(layers, none, a);
    }
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace

s3_status launch_score(const s3_csr_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
                       const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                       const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                       float* d_all_scores, cudaStream_t stream)
{
    ScoreLayers layers = {};
    for (int l = 0; l < n_layers; ++l) layers.v[l] = h_layers[l];
    return launch_score_impl(layers, nullptr, n_layers, d_sae, d_q_ids, d_q_vals, Q, nq, k, n_spans, p, d_bm25, ld_bm25,
                             d_top_idx, d_top_score, d_all_scores, stream);
}

s3_status launch_score_compact(const s3_compact_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
                               const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                               const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                               float* d_all_scores, cudaStream_t stream)
{
    ScoreLayers layers = {};
    CompactLayers cl = {};
    for (int l = 0; l < n_layers; ++l) {
        cl.v[l] = h_layers[l];
        layers.v[l].d_row_ptr = h_layers[l].d_row_ptr;
        layers.v[l].d_pos = nullptr;
    }
    return launch_score_impl(layers, &cl, n_layers, d_sae, d_q_ids, d_q_vals, Q, nq, k, n_spans, p, d_bm25, ld_bm25,
                             d_top_idx, d_top_score, d_all_scores, stream);
}

}  // namespace s3
