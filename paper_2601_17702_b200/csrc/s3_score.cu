// Query-time span scoring (Sec. 3.5, Eq. 5-6; appendix IDF definition) fused with score fusion and
// top-s selection. A query is handled by one thread block or, when there are fewer queries than the GPU
// has room for, by several blocks that each take a share of its posting lists:
//   a. aggregate the query tokens' Top-k into unique features with cQ (token count) and aQ (summed
//      activation): block bitonic sort of (id, entry) keys, then run detection;
//   b. fetch the unique features' list bounds in one parallel sweep and cut all lists into 32-posting
//      pieces (a long list is simply many pieces, so skewed list lengths do not unbalance anything). The
//      block tabulates one 16-byte descriptor per piece of its share (where the piece starts, how many
//      postings it has, cQ, the feature) and its warps walk the pieces, one broadcast descriptor load per
//      piece. Every posting works out by itself which spans it still adds to (see posting_range), for any
//      width/stride, and records the range as +w / -w in a difference array in shared memory that one
//      prefix sum turns into per-span totals: w = 1 in min-count mode (totals are min(cQ, cS) sums), and in
//      weighted mode w = aQ*IDF as a fixed-point integer whose unit is chosen per query from the largest
//      weight, so that the sums are exact integers and do not depend on the order of the additions;
//   c. fuse with the lexical score vector and pick the s best spans (score desc, index asc). With several
//      blocks per query each adds its difference array to the query's array in the workspace; the block
//      that arrives last (a ticket counter, nobody waits) finishes the query.
#include "s3_kernels.cuh"
#include "s3_query.cuh"

namespace s3 {

namespace {

struct CompactLayers {
    s3_compact_view v[S3_MAX_SCORE_LAYERS];
};
constexpr int CBATCH = 8;        // compact index: blocks of 32 postings a warp decodes side by side
constexpr int WINP = 1024;       // pieces whose descriptors are tabulated at a time
constexpr int MAX_SPLIT = 148;   // blocks per query at most

// One 32-posting piece of a posting list.
struct PieceDesc {
    unsigned long long start;    // raw CSR: index of the piece's first posting in pos; compact: its block index
    uint32_t first_i;            // list index of the piece's first posting
    uint32_t meta;               // postings in the piece (6 bits) | cQ << 6 (13 bits) | unique-feature index << 19
};
__device__ __forceinline__ uint32_t piece_count(uint32_t meta) { return meta & 63u; }
__device__ __forceinline__ uint32_t piece_cq(uint32_t meta) { return (meta >> 6) & 0x1FFFu; }
__device__ __forceinline__ uint32_t piece_owner(uint32_t meta) { return meta >> 19; }

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
    int n_split;                       // blocks per query
    unsigned long long* acc_g;         // [Q][n_spans + 2] sum of the blocks' difference arrays (n_split > 1), zeroed by the launcher
    uint32_t* tickets;                 // [Q] blocks of the query that have added theirs, zeroed by the launcher
};

// Shared-memory carve-up, identical on host and device.
struct ScoreLayout {
    uint32_t acc_off, ulo_off, keys_off, ufeat_off, ustart_off, uaq_off, uw_off, table_off, total;
};
__host__ __device__ inline ScoreLayout score_layout(int nk, int npad, int n_spans, bool weighted)
{
    ScoreLayout L;
    uint32_t o = 0;
    L.acc_off = o;    o += (static_cast<uint32_t>(n_spans) + 2) * (weighted ? 8u : 4u);  o = (o + 15u) & ~15u;
    L.ulo_off = o;    o += static_cast<uint32_t>(nk) * 8u;
    L.uw_off = o;     o += weighted ? static_cast<uint32_t>(nk) * 8u : 0u;
    L.table_off = o;  o += WINP * 16u;
    L.keys_off = o;   o += static_cast<uint32_t>(npad) * 4u;
    L.ufeat_off = o;  o += (static_cast<uint32_t>(nk) + 1u) * 4u;                      // cstart[u] replaces ufeat[u]
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

// Adds w to the difference array at j_lo and takes it away again after j_hi.
template <bool WEIGHTED>
__device__ __forceinline__ void add_range(int* acc_i, unsigned long long* acc_w, int j_lo, int j_hi, unsigned long long w)
{
    if (j_lo > j_hi) return;
    if (WEIGHTED) {
        atomicAdd(&acc_w[j_lo], w);
        atomicAdd(&acc_w[j_hi + 1], 0ull - w);
    } else {
        atomicAdd(&acc_i[j_lo], 1);
        atomicAdd(&acc_i[j_hi + 1], -1);
    }
}

__device__ __forceinline__ double block_max_double(double v, double* red /*[SW]*/)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double m = red[0];
    for (int w = 1; w < SW; ++w) m = fmax(m, red[w]);
    return m;
}

template <bool POW2, bool COMPACT, bool WEIGHTED>
__global__ void __launch_bounds__(ST)
score_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ CompactLayers clayers,
             const __grid_constant__ ScoreArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    const ScoreLayout SL = score_layout(a.nk, a.npad, a.n_spans, WEIGHTED);
    int* acc_i = reinterpret_cast<int*>(score_smem_raw + SL.acc_off);                              // min-count: difference array [n_spans+2]
    unsigned long long* acc_w = reinterpret_cast<unsigned long long*>(score_smem_raw + SL.acc_off);  // weighted: fixed-point, same shape
    uint32_t* sel = reinterpret_cast<uint32_t*>(score_smem_raw + SL.acc_off);                       // phase c: orderable fused scores
    unsigned long long* ulo = reinterpret_cast<unsigned long long*>(score_smem_raw + SL.ulo_off);
    long long* uw = reinterpret_cast<long long*>(score_smem_raw + SL.uw_off);                       // weighted: fixed-point aQ*IDF
    PieceDesc* table = reinterpret_cast<PieceDesc*>(score_smem_raw + SL.table_off);
    uint32_t* keys = reinterpret_cast<uint32_t*>(score_smem_raw + SL.keys_off);
    uint32_t* ulen = keys;                                                      // keys are dead once aQ is summed
    int32_t* ufeat = reinterpret_cast<int32_t*>(score_smem_raw + SL.ufeat_off);
    int32_t* ustart = reinterpret_cast<int32_t*>(score_smem_raw + SL.ustart_off);
    float* uaq = reinterpret_cast<float*>(score_smem_raw + SL.uaq_off);
    uint32_t* cstart = reinterpret_cast<uint32_t*>(score_smem_raw + SL.ufeat_off);   // same storage as ufeat: a thread
                                                                                       // reads ufeat[u], then writes cstart[u]
    __shared__ uint32_t ws[SW + 1];
    __shared__ unsigned long long red[SW];
    __shared__ int n_unique_s;
    __shared__ uint32_t ticket_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = blockIdx.x / a.n_split, part = blockIdx.x - q * a.n_split;

    if (WEIGHTED) { for (int j = tid; j < a.n_spans + 2; j += ST) acc_w[j] = 0ull; }
    else          { for (int j = tid; j < a.n_spans + 2; j += ST) acc_i[j] = 0; }
    __syncthreads();

    // Weighted mode: the unit of the fixed-point weights. A first pass over the layers finds the query's largest
    // weight and its number of postings; unit = 2^(exponent of the largest weight + 1 - bits) with bits chosen so
    // that the sum of all contributions stays below 2^62.
    int wexp = 0;                 // weights are stored as llrint(ldexp(w, wexp))
    if (WEIGHTED) {
        double wmax = 0.0;
        unsigned long long n_post = 0;
        for (int l = 0; l < a.n_layers; ++l) {
            const int32_t* qi = a.q_ids + ((size_t)l * a.Q + q) * a.nk;
            const float* qv = a.q_vals + ((size_t)l * a.Q + q) * a.nk;
            const int U = aggregate_query(qi, qv, a.nk, a.npad, a.d_sae, true, keys, ufeat, ustart, uaq, ws, &n_unique_s);
            const uint32_t pieces = cut_lists(layers.v[l].d_row_ptr, U, a.stop_freq, ufeat, ulo, ulen, cstart, ws,
                                              COMPACT ? clayers.v[l].d_blk_ptr : nullptr);
            n_post += static_cast<unsigned long long>(pieces) * PIECE;
            double m = 0.0;
            for (int u = tid; u < U; u += ST)
                if (ulen[u]) m = fmax(m, static_cast<double>(uaq[u]) * (1.0 / (log(1.0 + static_cast<double>(ulen[u])) + 1.0)));
            wmax = fmax(wmax, block_max_double(m, reinterpret_cast<double*>(red)));
            __syncthreads();
        }
        int bits = 61;
        while (bits > 20 && (n_post >> (61 - bits)) != 0ull) --bits;          // n_post < 2^(61 - bits + 1)
        wexp = wmax > 0.0 ? bits - 1 - ilogb(wmax) : 0;
    }

    for (int l = 0; l < a.n_layers; ++l) {
        const int32_t* qi = a.q_ids + ((size_t)l * a.Q + q) * a.nk;
        const float* qv = a.q_vals + ((size_t)l * a.Q + q) * a.nk;
        const int U = aggregate_query(qi, qv, a.nk, a.npad, a.d_sae, WEIGHTED, keys, ufeat, ustart, uaq, ws, &n_unique_s);
        // b. list bounds of every unique feature (independent loads), then the pieces' prefix sum
        const int32_t* __restrict__ pos = layers.v[l].d_pos;
        const uint32_t piece_total = cut_lists(layers.v[l].d_row_ptr, U, WEIGHTED ? a.stop_freq : 0, ufeat, ulo, ulen, cstart, ws,
                                               COMPACT ? clayers.v[l].d_blk_ptr : nullptr);
        if (WEIGHTED) {
            for (int u = tid; u < U; u += ST) {
                const double w = static_cast<double>(uaq[u]) * (1.0 / (log(1.0 + static_cast<double>(ulen[u])) + 1.0));
                uw[u] = ulen[u] ? __double2ll_rn(ldexp(w, wexp)) : 0ll;
            }
            __syncthreads();
        }
        // this block's share of the layer's pieces
        const uint32_t share0 = static_cast<uint32_t>(static_cast<uint64_t>(piece_total) * part / a.n_split);
        const uint32_t share1 = static_cast<uint32_t>(static_cast<uint64_t>(piece_total) * (part + 1) / a.n_split);

        // The share is walked a window at a time; inside a window every warp takes an equal run of consecutive
        // pieces. BATCH pieces per round: first all their loads are issued, then their updates, so that a warp has
        // BATCH independent memory round trips in flight instead of one.
        for (uint32_t win0 = share0; win0 < share1; win0 += WINP) {
            const uint32_t win1 = share1 - win0 < WINP ? share1 : win0 + WINP;
            // descriptors: owner by binary search in the pieces' prefix (last u with cstart[u] <= c; pieces of
            // empty lists share a start), one piece per thread and step
            for (uint32_t c = win0 + tid; c < win1; c += ST) {
                int lo = 0, hi = U;
                while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cstart[mid] <= c) lo = mid; else hi = mid; }
                const uint32_t j = c - cstart[lo];
                const uint32_t left = ulen[lo] - PIECE * j;
                PieceDesc d;
                d.start = ulo[lo] + (COMPACT ? j : PIECE * j);
                d.first_i = PIECE * j;
                d.meta = (left < PIECE ? left : PIECE) | (static_cast<uint32_t>(ustart[lo + 1] - ustart[lo]) << 6) |
                         (static_cast<uint32_t>(lo) << 19);
                table[c - win0] = d;
            }
            __syncthreads();
            const uint32_t n_win = win1 - win0;
            const uint32_t c_begin = static_cast<uint32_t>(static_cast<uint64_t>(n_win) * warp / SW);
            const uint32_t c_end = static_cast<uint32_t>(static_cast<uint64_t>(n_win) * (warp + 1) / SW);
            if constexpr (COMPACT) {
                // A piece is one block of the compact index. The headers of the next CBATCH blocks are fetched while
                // the payload words of the current ones are in flight, so a batch waits for one memory round trip.
                // In min-count mode posting i also needs the position of posting i - cQ of its list: the 32 lanes'
                // targets lie in at most two blocks, x = floor((32 j - cQ)/32) and x + 1. Block j itself is at hand; an
                // earlier block j - d is piece b - d of this warp (its pieces are consecutive) and is taken from the
                // batch or from the last two blocks of the previous batch; only when it lies further back (the start
                // of the warp's run, cQ > 64) is it decoded on the spot.
                const s3_compact_view& cv = clayers.v[l];
                auto fetch_head = [&](uint32_t c) {
                    PieceHead h;
                    h.first = 0; h.desc = 0; h.cnt = 0;
                    if (c < c_end) {
                        const PieceDesc d = table[c];
                        h = block_head(cv, static_cast<uint32_t>(d.start), piece_count(d.meta));
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
                        const PieceDesc d = table[c0 + b];
                        int p_prev = -1;
                        if (!WEIGHTED) {
                            const int j = static_cast<int>(d.first_i >> 5);
                            const int cq = static_cast<int>(piece_cq(d.meta));
                            const int x = (32 * j - cq) >> 5;              // floor, may be negative
                            int pr[3] = {p, -1, -1};
#pragma unroll
                            for (int r = 1; r <= 2; ++r) {
                                const int xb = x + r - 1;
                                if (xb >= 0 && xb < j) {
                                    const int dd = j - xb;
                                    if (dd <= b + avail) {
#pragma unroll
                                        for (int e = 1; e <= b + 2; ++e)
                                            if (dd == e) pr[r] = hist[b + 2 - e];
                                    } else {
                                        pr[r] = block_positions_now(cv, static_cast<uint32_t>(d.start) - dd, lane);
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
                        add_range<WEIGHTED>(acc_i, acc_w, j_lo, j_hi, WEIGHTED ? static_cast<unsigned long long>(uw[piece_owner(d.meta)]) : 1ull);
                    }
                    carry2 = hist[CBATCH]; carry1 = hist[CBATCH + 1];
                }
            } else
            for (uint32_t c0 = c_begin; c0 < c_end; c0 += BATCH) {
                int p[BATCH], p_prev[BATCH];
                uint32_t own[BATCH];
#pragma unroll
                for (int b = 0; b < BATCH; ++b) {
                    p[b] = -1; p_prev[b] = -1; own[b] = 0;
                    if (c0 + b < c_end) {
                        const uint4 raw = *reinterpret_cast<const uint4*>(&table[c0 + b]);       // one broadcast load per piece
                        const unsigned long long start = (static_cast<unsigned long long>(raw.y) << 32) | raw.x;
                        own[b] = piece_owner(raw.w);
                        if (static_cast<uint32_t>(lane) < piece_count(raw.w)) {
                            const int32_t* __restrict__ src = pos + start + lane;
                            p[b] = __ldg(src);
                            if (!WEIGHTED) {
                                const uint32_t cq = piece_cq(raw.w);
                                if (raw.z + lane >= cq) p_prev[b] = __ldg(src - cq);
                            }
                        }
                    }
                }
#pragma unroll
                for (int b = 0; b < BATCH; ++b) {
                    if (p[b] < 0) continue;
                    int j_lo, j_hi;
                    posting_range<POW2>(a, p[b], p_prev[b], j_lo, j_hi);
                    add_range<WEIGHTED>(acc_i, acc_w, j_lo, j_hi, WEIGHTED ? static_cast<unsigned long long>(uw[own[b]]) : 1ull);
                }
            }
            __syncthreads();
        }
    }

    // Several blocks per query: add this block's difference array to the query's in the workspace; the block that
    // takes the last ticket reads the sum back and finishes the query.
    if (a.n_split > 1) {
        unsigned long long* g = a.acc_g + static_cast<size_t>(q) * (a.n_spans + 2);
        for (int j = tid; j < a.n_spans + 2; j += ST) {
            if (WEIGHTED) { if (acc_w[j]) atomicAdd(&g[j], acc_w[j]); }
            else if (acc_i[j]) atomicAdd(reinterpret_cast<int*>(&g[j]), acc_i[j]);
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) ticket_s = atomicAdd(&a.tickets[q], 1u);
        __syncthreads();
        if (ticket_s != static_cast<uint32_t>(a.n_split - 1)) return;
        __threadfence();
        for (int j = tid; j < a.n_spans + 2; j += ST) {
            const unsigned long long v = __ldcg(&g[j]);
            if (WEIGHTED) acc_w[j] = v; else acc_i[j] = static_cast<int>(static_cast<uint32_t>(v));
        }
        __syncthreads();
    }

    // difference array -> per-span totals (inclusive prefix sum, in place)
    if (WEIGHTED) {
        unsigned long long carry = 0;
        for (int j0 = 0; j0 < a.n_spans; j0 += ST) {
            const int j = j0 + tid;
            unsigned long long inc = j < a.n_spans ? acc_w[j] : 0ull;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            __syncthreads();
            if (lane == 31) red[warp] = inc;
            __syncthreads();
            unsigned long long before = carry;
            for (int w = 0; w < warp; ++w) before += red[w];
            if (j < a.n_spans) acc_w[j] = before + inc;
            for (int w = 0; w < SW; ++w) carry += red[w];
        }
        __syncthreads();
    } else {
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
            const float base = WEIGHTED ? __double2float_rn(ldexp(static_cast<double>(static_cast<long long>(acc_w[j])), -wexp))
                                        : __int2float_rn(acc_i[j]);
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

// No span fits into the context: every query gets s times "no span".
__global__ void score_empty_kernel(int32_t* top_idx, float* top_score, size_t n)
{
    const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) { top_idx[i] = -1; top_score[i] = 0.0f; }
}

template <bool POW2, bool COMPACT, bool WEIGHTED>
s3_status launch_variant(const ScoreLayers& layers, const CompactLayers& cl, const ScoreArgs& a, size_t smem, int max_smem, int dev,
                         cudaStream_t stream)
{
    static bool attr_set[64] = {};
    if (dev >= 64 || !attr_set[dev]) {
        S3_CUDA_TRY(cudaFuncSetAttribute(score_kernel<POW2, COMPACT, WEIGHTED>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        if (dev < 64) attr_set[dev] = true;
    }
    score_kernel<POW2, COMPACT, WEIGHTED><<<a.Q * a.n_split, ST, smem, stream>>>(layers, cl, a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace

size_t score_workspace_bytes(int Q, int n_spans)
{
    if (Q <= 0 || n_spans <= 0) return 0;
    return round_up(static_cast<size_t>(Q) * 4, 256) + static_cast<size_t>(Q) * (n_spans + 2) * 8;
}

namespace {

s3_status launch_score_impl(const ScoreLayers& layers, const CompactLayers* clayers, int n_layers, int d_sae, const int32_t* d_q_ids,
                            const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                            const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                            float* d_all_scores, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    if (n_spans == 0) {
        const size_t n = static_cast<size_t>(Q) * p->s;
        score_empty_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(d_top_idx, d_top_score, n);
        S3_CUDA_TRY(cudaGetLastError());
        return S3_OK;
    }
    static int max_smem_dev[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    int max_smem = dev < 64 ? max_smem_dev[dev] : 0;
    if (max_smem == 0) {
        S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
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
    const bool weighted = p->mode == S3_SCORE_WEIGHTED;
    const size_t smem = score_layout(a.nk, npad, n_spans, weighted).total;
    S3_REQUIRE(smem + 2048 <= static_cast<size_t>(max_smem), S3_ERR_UNSUPPORTED,
               "n_spans = %d with nq*k = %d needs %zu bytes of shared memory per query, %d available", n_spans, a.nk, smem,
               max_smem - 2048);
    // Few queries: cut each over several blocks (about two blocks per SM in all) when the workspace has room for the
    // queries' shared difference arrays; otherwise one block per query.
    a.n_split = 1;
    a.acc_g = nullptr; a.tickets = nullptr;
    const int want = 2 * device_sm_count() / Q;
    if (want > 1 && ws_bytes >= 256 + score_workspace_bytes(Q, n_spans)) {
        a.n_split = want > MAX_SPLIT ? MAX_SPLIT : want;
        a.tickets = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(d_ws) + 256);
        a.acc_g = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(d_ws) + 256 + round_up(static_cast<size_t>(Q) * 4, 256));
        // the shared sums and tickets start from zero (a small range: this path is taken for few queries only)
        S3_CUDA_TRY(cudaMemsetAsync(a.tickets, 0, score_workspace_bytes(Q, n_spans), stream));
    }
    CompactLayers none = {};
    const CompactLayers& cl = clayers ? *clayers : none;
    const bool pow2 = a.stride_shift >= 0, compact = clayers != nullptr;
#define S3_SCORE_CASE(P, C, W) \
    if (pow2 == P && compact == C && weighted == W) return launch_variant<P, C, W>(layers, cl, a, smem, max_smem, dev, stream);
    S3_SCORE_CASE(true, false, false) S3_SCORE_CASE(false, false, false) S3_SCORE_CASE(true, true, false) S3_SCORE_CASE(false, true, false)
    S3_SCORE_CASE(true, false, true) S3_SCORE_CASE(false, false, true) S3_SCORE_CASE(true, true, true) S3_SCORE_CASE(false, true, true)
#undef S3_SCORE_CASE
    return S3_OK;
}

}  // namespace

s3_status launch_score(const s3_csr_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
                       const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                       const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                       float* d_all_scores, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    ScoreLayers layers = {};
    for (int l = 0; l < n_layers; ++l) layers.v[l] = h_layers[l];
    return launch_score_impl(layers, nullptr, n_layers, d_sae, d_q_ids, d_q_vals, Q, nq, k, n_spans, p, d_bm25, ld_bm25,
                             d_top_idx, d_top_score, d_all_scores, d_ws, ws_bytes, stream);
}

s3_status launch_score_compact(const s3_compact_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
                               const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                               const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                               float* d_all_scores, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    ScoreLayers layers = {};
    CompactLayers cl = {};
    for (int l = 0; l < n_layers; ++l) {
        cl.v[l] = h_layers[l];
        layers.v[l].d_row_ptr = h_layers[l].d_row_ptr;
        layers.v[l].d_pos = nullptr;
    }
    return launch_score_impl(layers, &cl, n_layers, d_sae, d_q_ids, d_q_vals, Q, nq, k, n_spans, p, d_bm25, ld_bm25,
                             d_top_idx, d_top_score, d_all_scores, d_ws, ws_bytes, stream);
}

}  // namespace s3
