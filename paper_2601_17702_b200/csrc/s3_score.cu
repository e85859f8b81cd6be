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
constexpr int WIN = 8192;        // pieces whose owning feature is tabulated at a time

struct ScoreLayers {
    s3_csr_view v[S3_MAX_SCORE_LAYERS];
};
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

// Shared-memory carve-up, identical on host and device.
struct ScoreSmem {
    uint32_t acc_off, keys_off, ufeat_off, ustart_off, uaq_off, ulo_off, cstart_off, owner_off, total;
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
    o = (o + 3u) & ~3u;
    L.owner_off = o;  o += WIN * 2u;                                   // owning feature of each piece of the window
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

// Phase a, shared by the scoring kernels: the query's nk (id, value) entries -> unique features. Sorts
// (id, entry) keys ascending (invalid ids last), detects runs: ufeat[u] = id, ustart[u]..ustart[u+1] = its
// entries in keys[] (so cQ = ustart[u+1] - ustart[u]), and, if wanted, uaq[u] = the entries' activations summed
// in query-token order in fp32. Returns the number of unique features. Called by the whole block.
__device__ __forceinline__ int aggregate_query(const int32_t* qi, const float* qv, int nk, int npad, int d_sae, bool want_aq,
                                               uint32_t* keys, int32_t* ufeat, int32_t* ustart, float* uaq, uint32_t* ws,
                                               int* n_unique_s)
{
    const int tid = threadIdx.x;
    for (int i = tid; i < npad; i += ST) {
        uint32_t key = 0xFFFFFFFFu;
        if (i < nk) {
            const int32_t f = qi[i];
            if (f >= 0 && f < d_sae) key = (static_cast<uint32_t>(f) << 12) | static_cast<uint32_t>(i);
        }
        keys[i] = key;
    }
    __syncthreads();
    for (int size = 2; size <= npad; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = tid; i < (npad >> 1); i += ST) {
                const int pos = 2 * i - (i & (stride - 1));   // stride is a power of two
                const bool asc = (pos & size) == 0;
                const uint32_t x = keys[pos], y = keys[pos + stride];
                if ((x > y) == asc) { keys[pos] = y; keys[pos + stride] = x; }
            }
            __syncthreads();
        }
    }
    uint32_t carry = 0;
    for (int i0 = 0; i0 < nk; i0 += ST) {
        const int i = i0 + tid;
        uint32_t head = 0;
        if (i < nk && keys[i] != 0xFFFFFFFFu)
            head = (i == 0) || ((keys[i] >> 12) != (keys[i - 1] >> 12));
        uint32_t total;
        const uint32_t u = block_exclusive_scan(head, ws, total) + carry;
        if (head) { ufeat[u] = static_cast<int32_t>(keys[i] >> 12); ustart[u] = i; }
        carry += total;
    }
    if (tid == 0) {
        int lo = 0, hi = nk;   // first invalid key (keys sorted, invalid last)
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (keys[mid] == 0xFFFFFFFFu) hi = mid; else lo = mid + 1; }
        ustart[carry] = lo;
        *n_unique_s = static_cast<int>(carry);
    }
    __syncthreads();
    const int U = *n_unique_s;
    for (int u = tid; want_aq && u < U; u += ST) {   // aQ: activations summed in query-token order (fp32)
        float s = 0.0f;
        for (int i = ustart[u]; i < ustart[u + 1]; ++i) s = __fadd_rn(s, qv[keys[i] & 0xFFFu]);
        uaq[u] = s;
    }
    __syncthreads();
    return U;
}

// Phase b head, shared by the scoring kernels: list bounds of the U unique features (ulo, ulen; a list longer
// than stop_freq > 0 counts as empty) and the exclusive prefix cstart[0..U] of their 32-posting pieces. ulen
// may share storage with keys, cstart with ufeat (a thread reads ufeat[u] before it writes cstart[u]).
// Returns the number of pieces. Called by the whole block.
__device__ __forceinline__ uint32_t cut_lists(const uint64_t* __restrict__ row_ptr, int U, int64_t stop_freq,
                                              const int32_t* ufeat, unsigned long long* ulo, uint32_t* ulen,
                                              uint32_t* cstart, uint32_t* ws, const uint32_t* __restrict__ blk_ptr = nullptr)
{
    const int tid = threadIdx.x;
    uint32_t piece_carry = 0;
    for (int u0 = 0; u0 < U; u0 += ST) {
        const int u = u0 + tid;
        uint32_t n_pieces = 0;
        if (u < U) {
            const int f = ufeat[u];
            const uint64_t lo = __ldg(row_ptr + f), hi = __ldg(row_ptr + f + 1);
            uint64_t len = hi - lo;
            if (len > 0x7FFFFFFFull) len = 0x7FFFFFFFull;          // positions are int32: a list cannot be longer
            if (stop_freq > 0 && static_cast<int64_t>(len) > stop_freq) len = 0;   // stop feature
            ulo[u] = blk_ptr ? static_cast<unsigned long long>(__ldg(blk_ptr + f)) : lo;   // compact index: first block
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
    return piece_carry;
}

// Owning feature of each piece win0 .. win1-1 (binary search in the pieces' prefix, one piece per thread and
// step), so that the walk below needs no running cursor and its loads are independent of each other.
__device__ __forceinline__ void tabulate_owners(const uint32_t* cstart, int U, uint32_t win0, uint32_t win1, uint16_t* owner)
{
    for (uint32_t c = win0 + threadIdx.x; c < win1; c += ST) {
        int lo = 0, hi = U;                  // last u with cstart[u] <= c (pieces of empty lists share a start)
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cstart[mid] <= c) lo = mid; else hi = mid; }
        owner[c - win0] = static_cast<uint16_t>(lo);
    }
    __syncthreads();
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

// ---- per-position relevance, smoothed density, peak selection (Sec. 3.5 Eq. 6, "Adaptive Granularity") --------
// Weights are taken in fixed point (2^-24) so that S, the density and therefore the peaks are exact integer results
// whatever order the postings are visited in. Four kernels:
//   features   : per (query, layer) the unique query features and their weights w_l(f) (0 for stop features);
//   skip       : per (layer, feature, position tile) the index of the list's first posting inside the tile (binary
//                search; the lists are ascending), so that a block can gather one tile's part of every list;
//   accumulate : per (position tile, query) S[t] += w_l(f) over the tile's postings of every query feature, in 64-bit
//                shared-memory accumulators (one atomic per posting stays on the SM), written out once;
//   peaks      : per query the density D[t] = sum of S over the K positions starting at t - K/2 (a tile of S plus its
//                halo is prefix-summed in shared memory, D[t] is the difference of two prefix values) and greedy
//                non-maximum suppression over D with per-segment maxima in shared memory: a round reduces the segment
//                maxima, takes the best position (ties: lowest), clears D within the radius and redoes only the touched
//                segments.
constexpr int MIN_SEG_SHIFT = 8;      // a segment of the maxima table holds 2^seg_shift >= 256 positions,
constexpr int MAX_SEGS = 2048;       // the smallest power of two that covers L with MAX_SEGS segments
constexpr int CONV_TILE = 2048;      // positions smoothed per pass through shared memory
constexpr int MAX_CONV_KERNEL = 1024;
constexpr int POS_TILE = 8192;       // positions accumulated per block (64 KB of 64-bit sums)
constexpr int FCHUNK = 1024;         // query features handled per pass of the accumulate kernel
constexpr int AWIN = 4096;           // pieces whose owning feature is tabulated at a time there
constexpr int APIECE = 16;           // postings per piece there: a tile holds a fraction of a list, so half a warp per piece

struct DensityArgs {
    const int32_t* q_ids;
    const float* q_vals;
    long long* s_fix;        // [Q][L]
    long long* d_fix;        // [Q][L]
    int32_t* feat_cnt;       // [n_layers][Q]
    int32_t* feat_id;        // [n_layers][Q][nk]
    long long* feat_w;       // [n_layers][Q][nk]
    uint32_t* skip;          // [n_layers][d_sae][n_tiles + 1]
    int32_t* centers;        // [Q][n_centers]
    float* center_density;   // [Q][n_centers]
    float* s_out;            // [Q][L] or null
    float* d_out;            // [Q][L] or null
    long long L;
    int n_layers, d_sae, Q, nk, npad, conv_kernel, nms_radius, n_centers, seg_shift, n_tiles;
    int64_t stop_freq;
};

__device__ __forceinline__ bool better(long long v, long long p, long long bv, long long bp)
{
    return v > bv || (v == bv && v > 0 && p < bp);
}

// Maximum (value, lowest position) of d[lo..hi) over the calling warp.
__device__ __forceinline__ void warp_segment_max(const long long* d, long long lo, long long hi, int lane, long long& bv, long long& bp)
{
    bv = 0; bp = -1;
    for (long long t = lo + lane; t < hi; t += 32) {
        const long long v = d[t];
        if (better(v, t, bv, bp)) { bv = v; bp = t; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long ov = __shfl_xor_sync(0xffffffffu, bv, o), op = __shfl_xor_sync(0xffffffffu, bp, o);
        if (better(ov, op, bv, bp)) { bv = ov; bp = op; }
    }
}

__global__ void __launch_bounds__(ST)
density_features_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ DensityArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    const ScoreSmem SL = score_smem(a.nk, a.npad, 0, true);
    uint32_t* keys = reinterpret_cast<uint32_t*>(score_smem_raw + SL.keys_off);
    int32_t* ufeat = reinterpret_cast<int32_t*>(score_smem_raw + SL.ufeat_off);
    int32_t* ustart = reinterpret_cast<int32_t*>(score_smem_raw + SL.ustart_off);
    float* uaq = reinterpret_cast<float*>(score_smem_raw + SL.uaq_off);
    __shared__ uint32_t ws[SW + 1];
    __shared__ int n_unique_s;
    const int q = blockIdx.x, l = blockIdx.y;
    const size_t slot = (size_t)l * a.Q + q;
    const int U = aggregate_query(a.q_ids + slot * a.nk, a.q_vals + slot * a.nk, a.nk, a.npad, a.d_sae, true, keys, ufeat, ustart,
                                  uaq, ws, &n_unique_s);
    const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
    for (int u = threadIdx.x; u < U; u += ST) {
        const int f = ufeat[u];
        uint64_t len = __ldg(row_ptr + f + 1) - __ldg(row_ptr + f);
        if (len > 0x7FFFFFFFull) len = 0x7FFFFFFFull;
        long long w = 0;                                   // w = rint(aQ * IDF(freq) * 2^24), IDF = 1 / (ln(1 + freq) + 1)
        if (len > 0 && !(a.stop_freq > 0 && static_cast<int64_t>(len) > a.stop_freq))
            w = __double2ll_rn(static_cast<double>(uaq[u]) * (1.0 / (log(1.0 + static_cast<double>(len)) + 1.0)) * 16777216.0);
        a.feat_id[slot * a.nk + u] = f;
        a.feat_w[slot * a.nk + u] = w;
    }
    if (threadIdx.x == 0) a.feat_cnt[slot] = U;
}

// skip[l][f][p] = number of postings of feature f (layer l) at positions below p * POS_TILE, p = 0 .. n_tiles.
__global__ void __launch_bounds__(ST)
density_skip_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ DensityArgs a)
{
    const int l = blockIdx.y;
    const long long per_layer = (long long)a.d_sae * (a.n_tiles + 1);
    const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
    const int32_t* __restrict__ pos = layers.v[l].d_pos;
    for (long long i = (long long)blockIdx.x * ST + threadIdx.x; i < per_layer; i += (long long)gridDim.x * ST) {
        const int f = static_cast<int>(i / (a.n_tiles + 1)), p = static_cast<int>(i % (a.n_tiles + 1));
        const uint64_t base = __ldg(row_ptr + f);
        uint64_t len = __ldg(row_ptr + f + 1) - base;
        if (len > 0x7FFFFFFFull) len = 0x7FFFFFFFull;
        const long long bound = (long long)p * POS_TILE;
        uint32_t lo = 0, hi = static_cast<uint32_t>(len);     // first index with pos >= bound
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (__ldg(pos + base + mid) < bound) lo = mid + 1; else hi = mid;
        }
        a.skip[(size_t)l * per_layer + i] = lo;
    }
}

__global__ void __launch_bounds__(ST)
density_accumulate_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ DensityArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    unsigned long long* acc = reinterpret_cast<unsigned long long*>(score_smem_raw);          // [POS_TILE]
    unsigned long long* ulo = acc + POS_TILE;                                                  // [FCHUNK] first posting (absolute)
    long long* uw = reinterpret_cast<long long*>(ulo + FCHUNK);                                // [FCHUNK]
    uint32_t* ulen = reinterpret_cast<uint32_t*>(uw + FCHUNK);                                 // [FCHUNK]
    uint32_t* cstart = ulen + FCHUNK;                                                          // [FCHUNK + 1]
    uint16_t* owner = reinterpret_cast<uint16_t*>(cstart + FCHUNK + 4);                        // [AWIN]
    __shared__ uint32_t ws[SW + 1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, q = blockIdx.y;
    const long long t0 = (long long)tile * POS_TILE;
    const int n_here = static_cast<int>(a.L - t0 < POS_TILE ? a.L - t0 : POS_TILE);
    for (int i = tid; i < POS_TILE; i += ST) acc[i] = 0ull;
    __syncthreads();
    for (int l = 0; l < a.n_layers; ++l) {
        const size_t slot = (size_t)l * a.Q + q;
        const int U = a.feat_cnt[slot];
        const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
        const int32_t* __restrict__ pos = layers.v[l].d_pos;
        const uint32_t* __restrict__ skip = a.skip + (size_t)l * a.d_sae * (a.n_tiles + 1);
        for (int u0 = 0; u0 < U; u0 += FCHUNK) {
            const int n_u = U - u0 < FCHUNK ? U - u0 : FCHUNK;
            // the tile's part of every list of the chunk and the exclusive prefix of its 32-posting pieces
            uint32_t carry = 0;
            for (int i0 = 0; i0 < n_u; i0 += ST) {
                const int i = i0 + tid;
                uint32_t n_pieces = 0;
                if (i < n_u) {
                    const int f = a.feat_id[slot * a.nk + u0 + i];
                    const long long w = a.feat_w[slot * a.nk + u0 + i];
                    const uint32_t* sk = skip + (size_t)f * (a.n_tiles + 1) + tile;
                    const uint32_t first = __ldg(sk), last = __ldg(sk + 1);
                    const uint32_t len = w != 0 ? last - first : 0u;
                    ulo[i] = __ldg(row_ptr + f) + first;
                    ulen[i] = len;
                    uw[i] = w;
                    n_pieces = (len + APIECE - 1) / APIECE;
                }
                uint32_t total;
                const uint32_t ex = block_exclusive_scan(n_pieces, ws, total) + carry;
                if (i < n_u) cstart[i] = ex;
                carry += total;
            }
            if (tid == 0) cstart[n_u] = carry;
            __syncthreads();
            const uint32_t piece_total = carry;
            for (uint32_t win0 = 0; win0 < piece_total; win0 += AWIN) {
                const uint32_t win1 = piece_total - win0 < AWIN ? piece_total : win0 + AWIN;
                for (uint32_t c = win0 + tid; c < win1; c += ST) {
                    int lo = 0, hi = n_u;              // last i with cstart[i] <= c
                    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cstart[mid] <= c) lo = mid; else hi = mid; }
                    owner[c - win0] = static_cast<uint16_t>(lo);
                }
                __syncthreads();
                const uint32_t n_win = win1 - win0;
                const uint32_t c_begin = win0 + static_cast<uint32_t>(static_cast<uint64_t>(n_win) * warp / SW);
                const uint32_t c_end = win0 + static_cast<uint32_t>(static_cast<uint64_t>(n_win) * (warp + 1) / SW);
                for (uint32_t c0 = c_begin; c0 < c_end; c0 += 2 * BATCH) {
                    int p[BATCH], ub[BATCH];
#pragma unroll
                    for (int b = 0; b < BATCH; ++b) {
                        const uint32_t c = c0 + 2 * b + (lane >> 4);          // each half of the warp takes a piece
                        p[b] = -1; ub[b] = 0;
                        if (c < c_end) {
                            const int i = owner[c - win0];
                            ub[b] = i;
                            const uint32_t j = (c - cstart[i]) * APIECE + (lane & 15);
                            if (j < ulen[i]) p[b] = __ldg(pos + ulo[i] + j);
                        }
                    }
#pragma unroll
                    for (int b = 0; b < BATCH; ++b) {
                        const long long rel = p[b] - t0;
                        if (p[b] >= 0 && rel >= 0 && rel < n_here) atomicAdd(&acc[rel], static_cast<unsigned long long>(uw[ub[b]]));
                    }
                }
                __syncthreads();
            }
        }
    }
    long long* S = a.s_fix + (size_t)q * a.L + t0;
    for (int i = tid; i < n_here; i += ST) S[i] = static_cast<long long>(acc[i]);
}

__global__ void __launch_bounds__(ST)
density_peaks_kernel(const __grid_constant__ DensityArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    long long* seg_val = reinterpret_cast<long long*>(score_smem_raw);                             // [MAX_SEGS]
    long long* seg_pos = seg_val + MAX_SEGS;
    long long* tile = seg_pos + MAX_SEGS;                                                         // [CONV_TILE + MAX_CONV_KERNEL]
    __shared__ long long red_v[SW], red_p[SW], pick_s, scan_tot[SW + 1];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = blockIdx.x;
    const long long L = a.L;
    long long* S = a.s_fix + (size_t)q * L;
    long long* D = a.d_fix + (size_t)q * L;

    // density: K taps starting at t - K/2. Per tile of CONV_TILE positions: S[t0 - K/2 .. t0 + CONV_TILE + K - K/2) goes
    // to shared memory, is replaced by its inclusive prefix sum P (each thread scans a run of consecutive entries, the
    // runs' totals are scanned across the block), and D[t0 + i] = P[i + K - 1] - P[i - 1].
    const long long half = a.conv_kernel / 2;
    const int n_tile = CONV_TILE + a.conv_kernel - 1;                     // entries staged per tile
    const int run = (n_tile + ST - 1) / ST;
    for (long long t0 = 0; t0 < L; t0 += CONV_TILE) {
        for (int i = tid; i < n_tile; i += ST) {
            const long long t = t0 - half + i;
            tile[i] = (t >= 0 && t < L) ? S[t] : 0;
        }
        __syncthreads();
        const int i_lo = tid * run, i_hi = i_lo + run < n_tile ? i_lo + run : n_tile;
        long long sum = 0;
        for (int i = i_lo; i < i_hi; ++i) { sum += tile[i]; tile[i] = sum; }
        long long inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        if (lane == 31) scan_tot[warp] = inc;
        __syncthreads();
        if (tid == 0) {
            long long acc = 0;
            for (int w = 0; w < SW; ++w) { const long long v = scan_tot[w]; scan_tot[w] = acc; acc += v; }
        }
        __syncthreads();
        const long long base = scan_tot[warp] + inc - sum;
        for (int i = i_lo; i < i_hi; ++i) tile[i] += base;
        __syncthreads();
        for (int i = tid; i < CONV_TILE; i += ST) {
            const long long t = t0 + i;
            if (t >= L) break;
            const long long d = tile[i + a.conv_kernel - 1] - (i > 0 ? tile[i - 1] : 0);
            D[t] = d;
            if (a.d_out) a.d_out[(size_t)q * L + t] = static_cast<float>(static_cast<double>(d) * (1.0 / 16777216.0));
            if (a.s_out) a.s_out[(size_t)q * L + t] = static_cast<float>(static_cast<double>(S[t]) * (1.0 / 16777216.0));
        }
        __syncthreads();
    }

    // segment maxima
    const int seg = 1 << a.seg_shift;
    const int n_segs = static_cast<int>((L + seg - 1) >> a.seg_shift);
    for (int sg = warp; sg < n_segs; sg += SW) {
        long long bv, bp;
        const long long lo = (long long)sg << a.seg_shift, hi = lo + seg < L ? lo + seg : L;
        warp_segment_max(D, lo, hi, lane, bv, bp);
        if (lane == 0) { seg_val[sg] = bv; seg_pos[sg] = bp; }
    }
    __syncthreads();

    for (int r = 0; r < a.n_centers; ++r) {
        long long bv = 0, bp = -1;
        for (int sg = tid; sg < n_segs; sg += ST)
            if (better(seg_val[sg], seg_pos[sg], bv, bp)) { bv = seg_val[sg]; bp = seg_pos[sg]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const long long ov = __shfl_xor_sync(0xffffffffu, bv, o), op = __shfl_xor_sync(0xffffffffu, bp, o);
            if (better(ov, op, bv, bp)) { bv = ov; bp = op; }
        }
        if (lane == 0) { red_v[warp] = bv; red_p[warp] = bp; }
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < SW; ++w)
                if (better(red_v[w], red_p[w], bv, bp)) { bv = red_v[w]; bp = red_p[w]; }
            a.centers[(size_t)q * a.n_centers + r] = bv > 0 ? static_cast<int32_t>(bp) : -1;
            a.center_density[(size_t)q * a.n_centers + r] = bv > 0 ? static_cast<float>(static_cast<double>(bv) * (1.0 / 16777216.0)) : 0.0f;
            pick_s = bv > 0 ? bp : -1;
        }
        __syncthreads();
        const long long c = pick_s;
        if (c < 0) continue;               // nothing left above zero: the remaining rounds pad (uniform for the block)
        const long long k_lo = c - a.nms_radius < 0 ? 0 : c - a.nms_radius;
        const long long k_hi = c + a.nms_radius >= L ? L - 1 : c + a.nms_radius;
        for (long long t = k_lo + tid; t <= k_hi; t += ST) D[t] = 0;
        __syncthreads();
        const int sg_lo = static_cast<int>(k_lo >> a.seg_shift), sg_hi = static_cast<int>(k_hi >> a.seg_shift);
        for (int sg = sg_lo + warp; sg <= sg_hi; sg += SW) {
            long long sv, sp;
            const long long lo = (long long)sg << a.seg_shift, hi = lo + seg < L ? lo + seg : L;
            warp_segment_max(D, lo, hi, lane, sv, sp);
            if (lane == 0) { seg_val[sg] = sv; seg_pos[sg] = sp; }
        }
        __syncthreads();
    }
}

}  // namespace

namespace {

// ---- head aggregation (Sec. 3.3: the SAE reads one head's projection; Sec. 3.4: "Top-k sparsity per token after head
// aggregation") -----------------------------------------------------------------------------------------------------
// One block per token (grid-stride). The token's H*k (id, value) pairs go through the same sort / run detection as a
// query's entries; a feature's activations are added in head order (fp32); the unique features with a positive sum
// become 64-bit keys (sum bits, ~id) that a bitonic sort orders by (sum descending, id ascending).
struct HeadAggArgs {
    const int32_t* ids;      // [T, H*k]
    const float* vals;
    int32_t* out_ids;        // [T, k_out]
    float* out_vals;
    int T, nk, npad, d_sae, k_out;
};

__global__ void __launch_bounds__(ST) head_aggregate_kernel(const __grid_constant__ HeadAggArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    const ScoreSmem SL = score_smem(a.nk, a.npad, 0, true);
    unsigned long long* sel = reinterpret_cast<unsigned long long*>(score_smem_raw + ((SL.total + 15u) & ~15u));   // [npad]
    uint32_t* keys = reinterpret_cast<uint32_t*>(score_smem_raw + SL.keys_off);
    int32_t* ufeat = reinterpret_cast<int32_t*>(score_smem_raw + SL.ufeat_off);
    int32_t* ustart = reinterpret_cast<int32_t*>(score_smem_raw + SL.ustart_off);
    float* uaq = reinterpret_cast<float*>(score_smem_raw + SL.uaq_off);
    __shared__ uint32_t ws[SW + 1];
    __shared__ int n_unique_s;
    const int tid = threadIdx.x;
    for (int t = blockIdx.x; t < a.T; t += gridDim.x) {
        __syncthreads();
        const int U = aggregate_query(a.ids + (size_t)t * a.nk, a.vals + (size_t)t * a.nk, a.nk, a.npad, a.d_sae, true, keys, ufeat,
                                      ustart, uaq, ws, &n_unique_s);
        int upad = 32;
        while (upad < U) upad <<= 1;
        for (int u = tid; u < upad; u += ST) {
            unsigned long long key = 0ull;
            if (u < U && uaq[u] > 0.0f) key = make_key(__float_as_uint(uaq[u]), static_cast<uint32_t>(ufeat[u]));
            sel[u] = key;
        }
        __syncthreads();
        for (int size = 2; size <= upad; size <<= 1) {
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                for (int i = tid; i < (upad >> 1); i += ST) {
                    const int pos = 2 * i - (i & (stride - 1));
                    const bool desc = (pos & size) == 0;
                    const unsigned long long x = sel[pos], y = sel[pos + stride];
                    if ((x < y) == desc) { sel[pos] = y; sel[pos + stride] = x; }
                }
                __syncthreads();
            }
        }
        for (int j = tid; j < a.k_out; j += ST) {
            const unsigned long long key = j < upad ? sel[j] : 0ull;
            a.out_ids[(size_t)t * a.k_out + j] = key ? static_cast<int32_t>(~static_cast<uint32_t>(key)) : -1;
            a.out_vals[(size_t)t * a.k_out + j] = key ? __uint_as_float(static_cast<uint32_t>(key >> 32)) : 0.0f;
        }
    }
}

}  // namespace

s3_status launch_head_aggregate(const int32_t* d_ids, const float* d_vals, int T, int H, int k, int d_sae, int k_out,
                                int32_t* d_out_ids, float* d_out_vals, cudaStream_t stream)
{
    HeadAggArgs a;
    a.ids = d_ids; a.vals = d_vals; a.out_ids = d_out_ids; a.out_vals = d_out_vals;
    a.T = T; a.nk = H * k; a.d_sae = d_sae; a.k_out = k_out;
    int npad = 32;
    while (npad < a.nk) npad <<= 1;
    a.npad = npad;
    const size_t smem = ((score_smem(a.nk, npad, 0, true).total + 15u) & ~15u) + static_cast<size_t>(npad) * 8;
    static bool attr_set[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 64 && !attr_set[dev]) {
        int max_smem = 0;
        S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        S3_CUDA_TRY(cudaFuncSetAttribute(head_aggregate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        attr_set[dev] = true;
    }
    const int max_grid = device_sm_count() * 8;
    head_aggregate_kernel<<<T < max_grid ? T : max_grid, ST, smem, stream>>>(a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

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

namespace s3 {

namespace {

struct DensityScratch {
    size_t s_fix, d_fix, feat_cnt, feat_id, feat_w, skip, total;
};
DensityScratch density_scratch(int Q, int64_t L, int n_layers, int d_sae, int nk)
{
    const size_t q = static_cast<size_t>(Q), l = static_cast<size_t>(L), nl = static_cast<size_t>(n_layers);
    const size_t n_tiles = (l + POS_TILE - 1) / POS_TILE;
    DensityScratch d;
    size_t o = 0;
    d.s_fix = o;    o += round_up(q * l * 8, 256);
    d.d_fix = o;    o += round_up(q * l * 8, 256);
    d.feat_w = o;   o += round_up(nl * q * nk * 8, 256);
    d.feat_id = o;  o += round_up(nl * q * nk * 4, 256);
    d.feat_cnt = o; o += round_up(nl * q * 4, 256);
    d.skip = o;     o += round_up(nl * static_cast<size_t>(d_sae) * (n_tiles + 1) * 4, 256);
    d.total = o;
    return d;
}

}  // namespace

size_t density_workspace_bytes(int Q, int64_t L, int n_layers, int d_sae, int nq, int k)
{
    return density_scratch(Q, L, n_layers, d_sae, nq * k).total;
}

s3_status launch_density(const s3_csr_view* h_layers, int n_layers, int d_sae, int64_t L, const int32_t* d_q_ids,
                         const float* d_q_vals, int Q, int nq, int k, int conv_kernel, int nms_radius, int n_centers,
                         int64_t stop_freq, int32_t* d_centers, float* d_center_density, float* d_s_out, float* d_d_out,
                         void* d_scratch, cudaStream_t stream)
{
    static int max_smem_dev[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    int max_smem = dev < 64 ? max_smem_dev[dev] : 0;
    if (max_smem == 0) {
        S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        S3_CUDA_TRY(cudaFuncSetAttribute(density_features_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        S3_CUDA_TRY(cudaFuncSetAttribute(density_accumulate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        S3_CUDA_TRY(cudaFuncSetAttribute(density_peaks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        if (dev < 64) max_smem_dev[dev] = max_smem;
    }
    int seg_shift = MIN_SEG_SHIFT;
    while (((L + (1ll << seg_shift) - 1) >> seg_shift) > MAX_SEGS) ++seg_shift;
    S3_REQUIRE(conv_kernel <= MAX_CONV_KERNEL, S3_ERR_UNSUPPORTED, "conv_kernel = %d exceeds %d", conv_kernel, MAX_CONV_KERNEL);
    ScoreLayers layers;
    for (int l = 0; l < n_layers; ++l) layers.v[l] = h_layers[l];
    const DensityScratch sc = density_scratch(Q, L, n_layers, d_sae, nq * k);
    unsigned char* base = static_cast<unsigned char*>(d_scratch);
    DensityArgs a;
    a.q_ids = d_q_ids; a.q_vals = d_q_vals;
    a.s_fix = reinterpret_cast<long long*>(base + sc.s_fix);
    a.d_fix = reinterpret_cast<long long*>(base + sc.d_fix);
    a.feat_cnt = reinterpret_cast<int32_t*>(base + sc.feat_cnt);
    a.feat_id = reinterpret_cast<int32_t*>(base + sc.feat_id);
    a.feat_w = reinterpret_cast<long long*>(base + sc.feat_w);
    a.skip = reinterpret_cast<uint32_t*>(base + sc.skip);
    a.centers = d_centers; a.center_density = d_center_density; a.s_out = d_s_out; a.d_out = d_d_out;
    a.L = L; a.n_layers = n_layers; a.d_sae = d_sae; a.Q = Q; a.nk = nq * k;
    int npad = 32;
    while (npad < a.nk) npad <<= 1;
    a.npad = npad; a.conv_kernel = conv_kernel; a.nms_radius = nms_radius; a.n_centers = n_centers; a.stop_freq = stop_freq;
    a.seg_shift = seg_shift;
    a.n_tiles = static_cast<int>((L + POS_TILE - 1) / POS_TILE);

    const size_t smem_feat = score_smem(a.nk, npad, 0, true).total;
    S3_REQUIRE(smem_feat + 2048 <= static_cast<size_t>(max_smem), S3_ERR_UNSUPPORTED, "nq*k = %d needs %zu bytes of shared memory", a.nk,
               smem_feat);
    density_features_kernel<<<dim3(Q, n_layers), ST, smem_feat, stream>>>(layers, a);
    if (a.n_tiles > 0) {
        const long long per_layer = (long long)d_sae * (a.n_tiles + 1);
        const long long want = (per_layer + ST - 1) / ST;
        const int cap = device_sm_count() * 16;
        density_skip_kernel<<<dim3(static_cast<unsigned>(want < cap ? want : cap), n_layers), ST, 0, stream>>>(layers, a);
        const size_t smem_acc = static_cast<size_t>(POS_TILE) * 8 + FCHUNK * (8 + 8 + 4) + (FCHUNK + 4) * 4 + AWIN * 2;
        density_accumulate_kernel<<<dim3(a.n_tiles, Q), ST, smem_acc, stream>>>(layers, a);
    }
    const size_t smem_peaks = 2 * MAX_SEGS * 8 + static_cast<size_t>(CONV_TILE + MAX_CONV_KERNEL) * 8;
    density_peaks_kernel<<<Q, ST, smem_peaks, stream>>>(a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
