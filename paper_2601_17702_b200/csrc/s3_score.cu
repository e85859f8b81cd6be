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
#include "s3_common.cuh"

namespace s3 {

namespace {

constexpr int ST = 512;          // threads per block
constexpr int SW = ST / 32;      // warps
constexpr int PIECE = 32;        // postings per work item
constexpr int BATCH = 8;         // work items a warp keeps in flight

struct ScoreLayers {
    s3_csr_view v[S3_MAX_SCORE_LAYERS];
};

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
};

// Shared-memory carve-up, identical on host and device.
struct ScoreSmem {
    uint32_t acc_off, keys_off, ufeat_off, ustart_off, uaq_off, ulo_off, cstart_off, total;
};
__host__ __device__ inline ScoreSmem score_smem(int nk, int npad, int n_spans, bool weighted)
{
    ScoreSmem L;
    uint32_t o = 0;
    L.acc_off = o;    o += (static_cast<uint32_t>(n_spans) + 2) * (weighted ? 8u : 4u);  o = (o + 15u) & ~15u;
    L.ulo_off = o;    o += static_cast<uint32_t>(nk) * 8u;
    L.keys_off = o;   o += static_cast<uint32_t>(npad) * 4u;
    L.ufeat_off = o;  L.cstart_off = o;  o += (static_cast<uint32_t>(nk) + 1u) * 4u;   // cstart[u] replaces ufeat[u]
    L.ustart_off = o; o += (static_cast<uint32_t>(nk) + 1u) * 4u;
    L.uaq_off = o;    o += weighted ? static_cast<uint32_t>(nk) * 4u : 0u;
    L.total = o + 16u;
    return L;
}

__device__ __forceinline__ uint32_t orderable(float v)
{
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* ws, uint32_t& total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) ws[warp] = inc;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (int w = 0; w < SW; ++w) { const uint32_t t = ws[w]; ws[w] = run; run += t; }
        ws[SW] = run;
    }
    __syncthreads();
    const uint32_t res = ws[warp] + inc - v;
    total = ws[SW];
    __syncthreads();
    return res;
}

// floor(p / stride) for p >= 0 (shift when the stride is a power of two).
__device__ __forceinline__ int div_stride(int p, const ScoreArgs& a)
{
    return a.stride_shift >= 0 ? (p >> a.stride_shift) : (p / a.stride);
}

// Spans that posting i of a list (position p, ascending positions) still adds to. The posting lies in
// spans lo(p)..hi(p), lo(p) = p >= width ? floor((p-width)/stride)+1 : 0, hi(p) = floor(p/stride).
// In min-count mode span j already holds cQ earlier postings of the feature exactly when posting i-cQ
// lies in it, i.e. when j <= hi(p_{i-cQ}); so the posting adds one to spans max(lo(p), hi(p_{i-cQ})+1)
// .. hi(p) only, and the totals come out as min(cQ, cS(f, j)). p_prev < 0 means "no such posting".
__device__ __forceinline__ void posting_range(const ScoreArgs& a, int p, int p_prev, int& j_lo, int& j_hi)
{
    j_hi = div_stride(p, a);
    j_lo = p >= a.width ? div_stride(p - a.width, a) + 1 : 0;
    if (p_prev >= 0) {
        const int j_prev = div_stride(p_prev, a) + 1;
        j_lo = j_prev > j_lo ? j_prev : j_lo;
    }
    j_hi = j_hi < a.n_spans - 1 ? j_hi : a.n_spans - 1;
}

__global__ void __launch_bounds__(ST)
score_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ ScoreArgs a)
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
        // a. sort (id, entry) keys ascending; invalid ids sort last
        for (int i = tid; i < a.npad; i += ST) {
            uint32_t key = 0xFFFFFFFFu;
            if (i < a.nk) {
                const int32_t f = qi[i];
                if (f >= 0 && f < a.d_sae) key = (static_cast<uint32_t>(f) << 12) | static_cast<uint32_t>(i);
            }
            keys[i] = key;
        }
        __syncthreads();
        for (int size = 2; size <= a.npad; size <<= 1) {
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                for (int i = tid; i < (a.npad >> 1); i += ST) {
                    const int pos = 2 * i - (i & (stride - 1));   // stride is a power of two
                    const bool asc = (pos & size) == 0;
                    const uint32_t x = keys[pos], y = keys[pos + stride];
                    if ((x > y) == asc) { keys[pos] = y; keys[pos + stride] = x; }
                }
                __syncthreads();
            }
        }
        // run detection -> unique features
        uint32_t carry = 0;
        for (int i0 = 0; i0 < a.nk; i0 += ST) {
            const int i = i0 + tid;
            uint32_t head = 0;
            if (i < a.nk && keys[i] != 0xFFFFFFFFu)
                head = (i == 0) || ((keys[i] >> 12) != (keys[i - 1] >> 12));
            uint32_t total;
            const uint32_t u = block_exclusive_scan(head, ws, total) + carry;
            if (head) { ufeat[u] = static_cast<int32_t>(keys[i] >> 12); ustart[u] = i; }
            carry += total;
        }
        if (tid == 0) {
            int lo = 0, hi = a.nk;   // first invalid key (keys sorted, invalid last)
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (keys[mid] == 0xFFFFFFFFu) hi = mid; else lo = mid + 1; }
            ustart[carry] = lo;
            n_unique_s = static_cast<int>(carry);
        }
        __syncthreads();
        const int U = n_unique_s;
        for (int u = tid; weighted && u < U; u += ST) {   // aQ: activations summed in query-token order (fp32)
            float s = 0.0f;
            for (int i = ustart[u]; i < ustart[u + 1]; ++i) s = __fadd_rn(s, qv[keys[i] & 0xFFFu]);
            uaq[u] = s;
        }
        __syncthreads();

        // b. list bounds of every unique feature (independent loads), then the pieces' prefix sum
        const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
        const int32_t* __restrict__ pos = layers.v[l].d_pos;
        uint32_t piece_carry = 0;
        for (int u0 = 0; u0 < U; u0 += ST) {
            const int u = u0 + tid;
            uint32_t n_pieces = 0;
            if (u < U) {
                const int f = ufeat[u];
                const uint64_t lo = __ldg(row_ptr + f), hi = __ldg(row_ptr + f + 1);
                uint64_t len = hi - lo;
                if (len > 0x7FFFFFFFull) len = 0x7FFFFFFFull;          // positions are int32: a list cannot be longer
                if (weighted && a.stop_freq > 0 && static_cast<int64_t>(len) > a.stop_freq) len = 0;   // stop feature
                ulo[u] = lo;
                ulen[u] = static_cast<uint32_t>(len);
                n_pieces = static_cast<uint32_t>((len + PIECE - 1) / PIECE);
            }
            uint32_t total;
            const uint32_t ex = block_exclusive_scan(n_pieces, ws, total) + piece_carry;
            if (u < U) cstart[u] = ex;
            piece_carry += total;
        }
        if (tid == 0) cstart[U] = piece_carry;
        __syncthreads();

        // each warp takes an equal share of consecutive pieces and walks them with a running feature cursor
        const uint32_t n_pieces_total = piece_carry;
        const uint32_t c_begin = static_cast<uint32_t>(static_cast<uint64_t>(n_pieces_total) * warp / SW);
        const uint32_t c_end = static_cast<uint32_t>(static_cast<uint64_t>(n_pieces_total) * (warp + 1) / SW);
        if (c_begin < c_end) {
            int lo_u = 0, hi_u = U;              // last u with cstart[u] <= c_begin
            while (hi_u - lo_u > 1) { const int mid = (lo_u + hi_u) >> 1; if (cstart[mid] <= c_begin) lo_u = mid; else hi_u = mid; }
            int u = lo_u;
            // BATCH pieces per round: first all their loads are issued, then their updates, so that a warp
            // has BATCH independent memory round trips in flight instead of one.
            for (uint32_t c0 = c_begin; c0 < c_end; c0 += BATCH) {
                int p[BATCH], p_prev[BATCH], ub[BATCH];
#pragma unroll
                for (int b = 0; b < BATCH; ++b) {
                    const uint32_t c = c0 + b;
                    p[b] = -1; p_prev[b] = -1; ub[b] = 0;
                    if (c < c_end) {
                        while (cstart[u + 1] <= c) ++u;
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
                    posting_range(a, p[b], p_prev[b], j_lo, j_hi);
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
        }
        __syncthreads();
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

s3_status launch_score(const s3_csr_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
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
        S3_CUDA_TRY(cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        if (dev < 64) max_smem_dev[dev] = max_smem;
    }
    ScoreLayers layers;
    for (int l = 0; l < n_layers; ++l) layers.v[l] = h_layers[l];
    ScoreArgs a;
    a.q_ids = d_q_ids; a.q_vals = d_q_vals; a.bm25 = d_bm25; a.ld_bm25 = ld_bm25;
    a.top_idx = d_top_idx; a.top_score = d_top_score; a.all_scores = d_all_scores;
    a.n_layers = n_layers; a.d_sae = d_sae; a.Q = Q; a.nk = nq * k;
    int npad = 32;
    while (npad < a.nk) npad <<= 1;
    a.npad = npad; a.n_spans = n_spans; a.width = p->width; a.stride = p->stride; a.mode = p->mode; a.s = p->s;
    a.alpha = p->alpha; a.beta = p->beta; a.stop_freq = p->stop_freq;
    a.stride_shift = (p->stride & (p->stride - 1)) == 0 ? __builtin_ctz(static_cast<unsigned>(p->stride)) : -1;
    const size_t smem = score_smem(a.nk, npad, n_spans, p->mode == S3_SCORE_WEIGHTED).total;
    S3_REQUIRE(smem + 2048 <= static_cast<size_t>(max_smem), S3_ERR_UNSUPPORTED,
               "n_spans = %d with nq*k = %d needs %zu bytes of shared memory per query, %d available", n_spans, a.nk, smem,
               max_smem - 2048);
    score_kernel<<<Q, ST, smem, stream>>>(layers, a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
