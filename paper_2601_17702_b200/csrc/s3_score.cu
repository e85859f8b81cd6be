// Query-time span scoring (Sec. 3.5, Eq. 5-6; appendix IDF definition) fused with score fusion and
// top-s selection. One thread block per query:
//   a. aggregate the query tokens' Top-k into unique features with cQ (token count) and aQ (summed
//      activation): block bitonic sort of (id, entry) keys, then run detection;
//   b. one warp per unique feature walks that feature's posting list (coalesced 128-byte loads),
//      turns positions into span indices, run-length-counts cS(f, span) with warp votes and adds
//      min(cQ, cS) (or aQ*IDF*cS) to the query's per-span accumulators in shared memory;
//      overlapping spans (stride < width) are handled as ceil(width/stride) interleaved tilings;
//   c. fuse with the lexical score vector and pick the s best spans (score desc, index asc).
#include "s3_common.cuh"

namespace s3 {

namespace {

constexpr int ST = 256;          // threads per block
constexpr int SW = ST / 32;      // warps

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
};

__device__ __forceinline__ uint32_t orderable(float v)
{
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint32_t block_exclusive_scan256(uint32_t v, uint32_t* ws, uint32_t& total)
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

__global__ void __launch_bounds__(ST)
score_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ ScoreArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem[];
    // layout: acc[n_spans] (8 B each) | keys[npad] u32 | ufeat[nk] | ustart[nk+1] | uaq[nk]
    unsigned long long* acc = reinterpret_cast<unsigned long long*>(score_smem);
    uint32_t* keys = reinterpret_cast<uint32_t*>(acc + a.n_spans);
    int32_t* ufeat = reinterpret_cast<int32_t*>(keys + a.npad);
    int32_t* ustart = ufeat + a.nk;
    float* uaq = reinterpret_cast<float*>(ustart + a.nk + 1);
    __shared__ uint32_t ws[SW + 1];
    __shared__ unsigned long long red[SW];
    __shared__ int n_unique_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = blockIdx.x;
    const bool weighted = a.mode == S3_SCORE_WEIGHTED;
    int* acc_i = reinterpret_cast<int*>(acc);          // min-count mode: int32 per span (first 4 bytes of each slot unused layout: dense int array)
    double* acc_d = reinterpret_cast<double*>(acc);    // weighted mode: fp64 per span

    for (int j = tid; j < a.n_spans; j += ST) acc[j] = 0ull;   // zero bits = 0 (int) = +0.0 (double)
    __syncthreads();

    const int n_phase = (a.width + a.stride - 1) / a.stride;
    const int period = n_phase * a.stride;

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
                    const int pos = ((i / stride) * (stride << 1)) + (i % stride);
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
            const uint32_t u = block_exclusive_scan256(head, ws, total) + carry;
            if (head) { ufeat[u] = static_cast<int32_t>(keys[i] >> 12); ustart[u] = i; }
            carry += total;
        }
        if (tid == 0) {
            int n_valid = 0;   // first invalid key (keys sorted, invalid last): binary search
            int lo = 0, hi = a.nk;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (keys[mid] == 0xFFFFFFFFu) hi = mid; else lo = mid + 1; }
            n_valid = lo;
            ustart[carry] = n_valid;
            n_unique_s = static_cast<int>(carry);
        }
        __syncthreads();
        const int U = n_unique_s;
        for (int u = tid; u < U; u += ST) {   // aQ: activations summed in query-token order (fp32)
            float s = 0.0f;
            for (int i = ustart[u]; i < ustart[u + 1]; ++i) s = __fadd_rn(s, qv[keys[i] & 0xFFFu]);
            uaq[u] = s;
        }
        __syncthreads();

        // b. posting walk, one warp per unique feature
        const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
        const int32_t* __restrict__ pos = layers.v[l].d_pos;
        for (int u = warp; u < U; u += SW) {
            const int f = ufeat[u];
            const int cq = ustart[u + 1] - ustart[u];
            const uint64_t lo = row_ptr[f], hi = row_ptr[f + 1];
            const int64_t len = static_cast<int64_t>(hi - lo);
            double w = 0.0;
            if (weighted) {
                if (a.stop_freq > 0 && len > a.stop_freq) continue;
                w = static_cast<double>(uaq[u]) * (1.0 / (log(1.0 + static_cast<double>(len)) + 1.0));
            }
            const int32_t* list = pos + lo;
            for (int r = 0; r < n_phase; ++r) {
                const int off = r * a.stride;
                int carry_key = -1, carry_cnt = 0;
                for (int64_t i0 = 0; i0 < len; i0 += 32) {
                    const int64_t i = i0 + lane;
                    int key = -1;
                    if (i < len) {
                        const int p = list[i] - off;
                        if (p >= 0) {
                            const int t = p / period;
                            const int j = r + t * n_phase;
                            if (p - t * period < a.width && j < a.n_spans) key = j;
                        }
                    }
                    const int prev = __shfl_up_sync(0xffffffffu, key, 1);
                    const bool head = (lane == 0) || (key != prev);
                    const uint32_t heads = __ballot_sync(0xffffffffu, head);
                    int cnt = 0;
                    if (head) {
                        const uint32_t above = (lane == 31) ? 0u : (heads >> (lane + 1)) << (lane + 1);
                        const int end = above ? (__ffs(above) - 1) : 32;
                        cnt = end - lane;
                    }
                    if (lane == 0) {
                        if (key == carry_key) cnt += carry_cnt;
                        else if (carry_key >= 0) {
                            if (weighted) atomicAdd(&acc_d[carry_key], w * carry_cnt);
                            else atomicAdd(&acc_i[carry_key], min(cq, carry_cnt));
                        }
                    }
                    const int last_head = 31 - __clz(heads);
                    if (head && lane != last_head && key >= 0) {
                        if (weighted) atomicAdd(&acc_d[key], w * cnt);
                        else atomicAdd(&acc_i[key], min(cq, cnt));
                    }
                    carry_key = __shfl_sync(0xffffffffu, key, last_head);
                    carry_cnt = __shfl_sync(0xffffffffu, cnt, last_head);
                }
                if (lane == 0 && carry_key >= 0) {
                    if (weighted) atomicAdd(&acc_d[carry_key], w * carry_cnt);
                    else atomicAdd(&acc_i[carry_key], min(cq, carry_cnt));
                }
            }
        }
        __syncthreads();
    }

    // c. fusion (one fp32 rounding per operation) and selection keys
    // min-count accumulators are a dense int array over the first 4*n_spans bytes; read them all
    // before the 8-byte selection keys overwrite the buffer.
    float fused[64];  // n_spans <= 16384 = 64 * ST
    const int per = (a.n_spans + ST - 1) / ST;
    for (int e = 0; e < per; ++e) {
        const int j = e * ST + tid;
        float v = 0.0f;
        if (j < a.n_spans) {
            const float base = weighted ? __double2float_rn(acc_d[j]) : __int2float_rn(acc_i[j]);
            v = __fmul_rn(a.alpha, base);
            if (a.bm25) v = __fadd_rn(v, __fmul_rn(a.beta, a.bm25[(size_t)q * a.ld_bm25 + j]));
            if (a.all_scores) a.all_scores[(size_t)q * a.n_spans + j] = v;
        }
        fused[e] = v;
    }
    __syncthreads();
    for (int e = 0; e < per; ++e) {
        const int j = e * ST + tid;
        if (j < a.n_spans)
            acc[j] = (static_cast<unsigned long long>(orderable(fused[e])) << 32) | static_cast<uint32_t>(~static_cast<uint32_t>(j));
    }
    __syncthreads();
    for (int r = 0; r < a.s; ++r) {
        unsigned long long best = 0ull;
        for (int j = tid; j < a.n_spans; j += ST) best = acc[j] > best ? acc[j] : best;
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
                acc[idx] = 0ull;
            }
            a.top_idx[(size_t)q * a.s + r] = idx;
            a.top_score[(size_t)q * a.s + r] = sc;
        }
        __syncthreads();
    }
}

}  // namespace

size_t score_smem_bytes(int nk, int npad, int n_spans)
{
    return (size_t)n_spans * 8 + (size_t)npad * 4 + (size_t)nk * 4 + (size_t)(nk + 1) * 4 + (size_t)nk * 4 + 16;
}

s3_status launch_score(const s3_csr_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
                       const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                       const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                       float* d_all_scores, cudaStream_t stream)
{
    static bool attr_set[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 64 && !attr_set[dev]) {
        S3_CUDA_TRY(cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        attr_set[dev] = true;
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
    const size_t smem = score_smem_bytes(a.nk, npad, n_spans);
    score_kernel<<<Q, ST, smem, stream>>>(layers, a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
