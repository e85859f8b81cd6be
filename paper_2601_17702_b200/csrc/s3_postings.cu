// Per-chunk CSR posting lists (Sec. 3.4, Eq. 4: I[f] <- I[f] U {t} for every f in F_t).
//
// The chunk's (feature, token) pairs arrive in token order and leave grouped by feature with the tokens of
// each feature ascending: a counting sort by feature that must keep the input order. Two launches over all
// chunk-layers ("items") of a batch, all integer, no block waits for another:
//
//   1. partition  block = one run of consecutive tokens (<= 8192 pairs). The features are cut into buckets
//                 of 2^fbits consecutive ids (about 4096 pairs per bucket and item); the block counts its
//                 pairs per bucket in shared memory, scans the counts, regroups the run by bucket in shared
//                 memory and writes it back over the run's own range of an intermediate array as 32-bit
//                 entries (feature within bucket << tbits | token), plus one directory row
//                 dir[run][bucket] = offset of the bucket inside the run.
//   2. bucket     block = one bucket of one item. It collects the bucket's segment of every run, counts the
//                 entries per (feature, token window) with shared-memory atomics that also hand each entry
//                 its arrival rank inside that small group, scans the counters in (feature, window) order,
//                 and places every token at group offset + rank. A list is then ascending except inside
//                 groups that hold more than one entry; those few are sorted in place (the tokens of one
//                 feature are distinct, so the order is unique). The block finally writes its features'
//                 row_ptr and its contiguous part of pos (and pval) with coalesced stores.
//
// The bucket's first output offset is the sum of its directory column, so nothing is scanned across blocks.
// Whatever the scheduling, every list comes out ascending and the result is bit-identical from run to run.
// A bucket that holds more than 8192 entries (skewed dictionaries) is sorted in several sweeps over ranges
// of its features; a single list longer than that is produced from a token bitmap.
#include "s3_common.cuh"
#include "s3_kernels.cuh"

namespace s3 {

namespace {

constexpr int NT = 512;                  // threads per block, both kernels
constexpr int NW = NT / 32;
constexpr int PER = 16;                  // pairs per thread in the partition kernel
constexpr int RUN_PAIRS = NT * PER;      // pairs per run at most
constexpr int B_MAX = 4 * NT;            // buckets per item at most (four per thread in the scan)
constexpr int FB_MAX = 12;               // at most 4096 features per bucket
constexpr int CAP = 8192;                // entries sorted at once in shared memory
constexpr int TBL_BITS = 12;             // (feature, window) counters of one sort
constexpr int TBL = 1 << TBL_BITS;
constexpr int MAX_RUNS = 4 * NT;         // runs whose segment table fits in shared memory
constexpr int BM_WORDS = 2 * CAP;        // bitmap words of the single-list path (e_stage + sorted)
constexpr int TARGET_BUCKET = 4096;      // planned mean entries per bucket

struct ItemPlan {
    unsigned long long interm_off, idx_off, dir_off;   // byte offsets in the workspace
    int n_runs, tok_per_run, n_buckets;
    uint32_t magic_k;                                   // floor(2^32 / k) + 1 (k >= 2): p / k = umulhi(p, magic) for p < 8192
    unsigned char tbits, fbits, wbits, has_val;         // token bits, feature-in-bucket bits, log2(windows)
    int blk1_start, blk2_start;
};

struct PostingsPlan {
    s3_postings_item items[S3_MAX_POSTINGS_ITEMS];
    ItemPlan ip[S3_MAX_POSTINGS_ITEMS];
    int n_items, n_blk1, n_blk2;
    unsigned char* ws;
    uint32_t* status;
};

__device__ __forceinline__ int find_item1(const PostingsPlan& pl, int blk)
{
    int it = 0;
    while (it + 1 < pl.n_items && blk >= pl.ip[it + 1].blk1_start) ++it;
    return it;
}
__device__ __forceinline__ int find_item2(const PostingsPlan& pl, int blk)
{
    int it = 0;
    while (it + 1 < pl.n_items && blk >= pl.ip[it + 1].blk2_start) ++it;
    return it;
}

// Exclusive prefix of one value per thread over the block; *total = the block's sum. Two barriers.
__device__ __forceinline__ uint32_t block_scan_excl(uint32_t v, uint32_t* warp_sums /*[NW]*/, uint32_t* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += u;
    }
    __syncthreads();                                   // the previous use of warp_sums is over
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    const uint32_t w = lane < NW ? warp_sums[lane] : 0u;
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < NW; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += u;
    }
    *total = __shfl_sync(0xffffffffu, winc, NW - 1);
    return __shfl_sync(0xffffffffu, winc - w, warp) + inc - v;
}

// ---- 1. runs regrouped by bucket ----------------------------------------------------------------------
template <bool VALS>
__global__ void __launch_bounds__(NT, 2)
postings_partition_kernel(const __grid_constant__ PostingsPlan pl)
{
    extern __shared__ uint32_t sm[];
    uint32_t* hist = sm;                       // [B_MAX]
    uint32_t* stage = hist + B_MAX;            // [RUN_PAIRS]
    uint32_t* stage_idx = stage + RUN_PAIRS;   // [RUN_PAIRS] (VALS)
    __shared__ uint32_t warp_sums[NW];

    const int item = find_item1(pl, blockIdx.x);
    const s3_postings_item& it = pl.items[item];
    const ItemPlan& ip = pl.ip[item];
    const int run = blockIdx.x - ip.blk1_start;
    const int tid = threadIdx.x;
    const int B = ip.n_buckets, k = it.k, d_sae = it.d_sae;
    const int t_lo = run * ip.tok_per_run;
    const int t_hi = min(it.T, t_lo + ip.tok_per_run);
    const uint32_t n_pairs = (uint32_t)(t_hi - t_lo) * (uint32_t)k;
    const size_t pair_base = (size_t)t_lo * k;
    const int32_t* __restrict__ src = it.d_ids + pair_base;
    const uint32_t fbits = ip.fbits, tbits = ip.tbits, fmask = (1u << fbits) - 1u, magic = ip.magic_k;
    const bool vals = VALS && ip.has_val;

    for (int b = tid; b < B; b += NT) hist[b] = 0;
    __syncthreads();

    // all loads first, so that the run's sixteen memory round trips per thread overlap
    int32_t fid[PER];
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const uint32_t p = tid + j * NT;
        fid[j] = p < n_pairs ? __ldcs(src + p) : -1;
    }
    uint32_t e[PER], ba[PER];                  // entry; bucket << 16 | arrival rank inside the bucket
    bool bad = false;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const uint32_t p = tid + j * NT;
        const int32_t f = fid[j];
        ba[j] = 0xFFFFFFFFu;
        e[j] = 0;
        if (f >= d_sae) bad = true;
        else if (f >= 0) {
            const uint32_t b = (uint32_t)f >> fbits;
            const uint32_t t = (uint32_t)t_lo + (k == 1 ? p : __umulhi(p, magic));
            e[j] = (((uint32_t)f & fmask) << tbits) | t;
            ba[j] = (b << 16) | atomicAdd(&hist[b], 1u);
        }
    }
    if (bad) dev_set_error(pl.status, DEV_BAD_FEATURE_ID);
    __syncthreads();

    // exclusive scan of the bucket counts, four per thread; the directory row goes out on the way
    uint32_t c[4], tsum = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        c[q] = 4 * tid + q < B ? hist[4 * tid + q] : 0u;
        tsum += c[q];
    }
    uint32_t total;
    uint32_t run_off = block_scan_excl(tsum, warp_sums, &total);
    uint16_t* dir = reinterpret_cast<uint16_t*>(pl.ws + ip.dir_off) + (size_t)run * (B + 1);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (4 * tid + q < B) {
            hist[4 * tid + q] = run_off;
            dir[4 * tid + q] = (uint16_t)run_off;
        }
        run_off += c[q];
    }
    if (tid == 0) dir[B] = (uint16_t)total;
    __syncthreads();

#pragma unroll
    for (int j = 0; j < PER; ++j) {
        if (ba[j] != 0xFFFFFFFFu) {
            const uint32_t slot = hist[ba[j] >> 16] + (ba[j] & 0xFFFFu);
            stage[slot] = e[j];
            if (vals) stage_idx[slot] = (uint32_t)pair_base + tid + j * NT;
        }
    }
    __syncthreads();

    uint32_t* dst = reinterpret_cast<uint32_t*>(pl.ws + ip.interm_off) + pair_base;
    for (uint32_t i = tid; i < total; i += NT) dst[i] = stage[i];
    if (vals) {
        uint32_t* dst_idx = reinterpret_cast<uint32_t*>(pl.ws + ip.idx_off) + pair_base;
        for (uint32_t i = tid; i < total; i += NT) dst_idx[i] = stage_idx[i];
    }
}

// ---- 2. one bucket sorted by (feature, token) and written out -----------------------------------------------
struct BucketCtx {
    // shared memory
    uint32_t* tbl;          // [TBL/2] words, two 16-bit (feature, window) counters each
    uint32_t* e_stage;      // [CAP] entries in arrival order
    uint32_t* sorted;       // [CAP] tokens in output order
    uint16_t* a_stage;      // [CAP] rank of the entry inside its (feature, window) group
    uint16_t* seg;          // [3 * MAX_RUNS] start, length, stage offset of every run's segment; later the conflict list
    uint32_t* idx_stage;    // [CAP] pair index of the entry (values only)
    uint32_t* sorted_idx;   // [CAP]
    uint32_t* warp_sums;    // [NW]
    uint32_t* counters;     // [2]: staged entries, conflict groups
    // the item
    const uint32_t* interm;
    const uint32_t* idx;
    const uint16_t* dir;
    const s3_postings_item* it;
    uint32_t* status;
    int n_runs, B, b, run_stride;
    uint32_t tbits, fbits, wbits, wshift, tmask;
};

// Sorts the entries of the bucket whose feature (relative to the bucket) lies in [f_lo, f_hi) and writes them to
// pos[out_base ...). FILTER = false: the whole bucket, segments and staging offsets taken from the shared-memory
// table. The caller guarantees at most CAP entries in the range.
template <bool VALS, bool FILTER>
__device__ void sort_range(const BucketCtx& c, uint32_t f_lo, uint32_t f_hi, uint32_t n_known, uint32_t out_base, bool write_row_ptr)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool vals = VALS && c.it->d_vals != nullptr;
    const uint32_t idx0 = f_lo << c.wbits;
    {
        uint4* t4 = reinterpret_cast<uint4*>(c.tbl);
        for (int i = tid; i < TBL / 8; i += NT) t4[i] = make_uint4(0, 0, 0, 0);
        if (tid < 2) c.counters[tid] = 0;
    }
    __syncthreads();

    // phase A: stage the entries, count them per (feature, window), keep each one's arrival rank in its group
    for (int r = warp; r < c.n_runs; r += NW) {
        uint32_t s, len, so = 0;
        if (FILTER) {
            const uint16_t* d = c.dir + (size_t)r * (c.B + 1) + c.b;
            s = __ldg(d);
            len = __ldg(d + 1) - s;
        } else {
            s = c.seg[r];
            len = c.seg[MAX_RUNS + r];
            so = c.seg[2 * MAX_RUNS + r];
        }
        const uint32_t* src = c.interm + (size_t)r * c.run_stride + s;
        for (uint32_t j0 = 0; j0 < len; j0 += 32) {
            const uint32_t j = j0 + lane;
            const bool valid = j < len;
            const uint32_t e = valid ? __ldcg(src + j) : 0u;
            bool keep = valid;
            uint32_t i = so + j;
            if (FILTER) {
                const uint32_t f = e >> c.tbits;
                keep = valid && f >= f_lo && f < f_hi;
                const uint32_t m = __ballot_sync(0xffffffffu, keep);
                if (m == 0) continue;
                uint32_t base = 0;
                if (lane == 0) base = atomicAdd(&c.counters[0], (uint32_t)__popc(m));
                base = __shfl_sync(0xffffffffu, base, 0);
                i = base + __popc(m & ((1u << lane) - 1u));
            }
            if (keep) {
                const uint32_t g = (e >> c.wshift) - idx0;
                const uint32_t sh = (g & 1u) << 4;
                const uint32_t old = atomicAdd(&c.tbl[g >> 1], 1u << sh);
                c.e_stage[i] = e;
                c.a_stage[i] = (uint16_t)(old >> sh);
                if (vals) c.idx_stage[i] = __ldcg(c.idx + (size_t)r * c.run_stride + s + j);
            }
        }
    }
    __syncthreads();
    const uint32_t n = FILTER ? c.counters[0] : n_known;
    __syncthreads();
    if (tid == 0) c.counters[0] = 0;            // from here on: the number of large groups

    // exclusive scan of the counters in (feature, window) order: TBL / 2 / NT words (two counters each) per thread
    {
        constexpr int WPT = TBL / 2 / NT;
        static_assert(WPT == 4, "one uint4 of counters per thread");
        uint4* t4 = reinterpret_cast<uint4*>(c.tbl) + tid;
        const uint4 v0 = t4[0];
        uint32_t w[WPT] = {v0.x, v0.y, v0.z, v0.w};
        uint32_t run = 0;
#pragma unroll
        for (int q = 0; q < WPT; ++q) {
            const uint32_t lo = w[q] & 0xFFFFu, hi = w[q] >> 16;
            w[q] = run | ((run + lo) << 16);
            run += lo + hi;
        }
        uint32_t total;
        const uint32_t base = block_scan_excl(run, c.warp_sums, &total) * 0x00010001u;
#pragma unroll
        for (int q = 0; q < WPT; ++q) w[q] += base;
        t4[0] = make_uint4(w[0], w[1], w[2], w[3]);
    }
    __syncthreads();

    // phase B: every token to its group's offset + its rank; groups with a second entry are noted
    const uint16_t* tbl16 = reinterpret_cast<const uint16_t*>(c.tbl);
    uint16_t* conf = c.seg;
    for (uint32_t i = tid; i < n; i += NT) {
        const uint32_t e = c.e_stage[i], a = c.a_stage[i];
        const uint32_t g = (e >> c.wshift) - idx0;
        const uint32_t slot = tbl16[g] + a;
        c.sorted[slot] = e & c.tmask;
        if (vals) c.sorted_idx[slot] = c.idx_stage[i];
        if (a == 1) conf[atomicAdd(&c.counters[1], 1u)] = (uint16_t)g;
    }
    __syncthreads();

    // groups of two or more entries (a repeated token breaks the input contract). Up to eight entries: insertion sort
    // by the group's thread. Larger groups (a feature present in many tokens of one window) go to a second list that
    // the warps take one group at a time: every entry counts the group's smaller tokens, which is its rank.
    const uint32_t n_conf = c.counters[1];
    uint16_t* big = c.a_stage;                  // ranks are dead after phase B
    uint32_t* tmp = c.e_stage;                  // so are the staged entries
    for (uint32_t ci = tid; ci < n_conf; ci += NT) {
        const uint32_t g = conf[ci];
        const uint32_t s = tbl16[g], e_ = g + 1 < (uint32_t)TBL ? tbl16[g + 1] : n;
        if (e_ - s > 8u) { big[atomicAdd(&c.counters[0], 1u)] = (uint16_t)g; continue; }
        for (uint32_t x = s + 1; x < e_; ++x) {
            const uint32_t v = c.sorted[x];
            const uint32_t vi = vals ? c.sorted_idx[x] : 0u;
            uint32_t y = x;
            while (y > s && c.sorted[y - 1] >= v) {
                if (c.sorted[y - 1] == v) { dev_set_error(c.status, DEV_DUPLICATE_ID); break; }
                c.sorted[y] = c.sorted[y - 1];
                if (vals) c.sorted_idx[y] = c.sorted_idx[y - 1];
                --y;
            }
            c.sorted[y] = v;
            if (vals) c.sorted_idx[y] = vi;
        }
    }
    __syncthreads();
    const uint32_t n_big = c.counters[0];
    for (uint32_t bi = warp; bi < n_big; bi += NW) {
        const uint32_t g = big[bi];
        const uint32_t s = tbl16[g], e_ = g + 1 < (uint32_t)TBL ? tbl16[g + 1] : n, cnt = e_ - s;
        for (uint32_t i = lane; i < cnt; i += 32) {
            const uint32_t v = c.sorted[s + i];
            uint32_t rank = 0;
            for (uint32_t j = 0; j < cnt; ++j) {
                const uint32_t u = c.sorted[s + j];
                rank += (u < v || (u == v && j < i)) ? 1u : 0u;
                if (u == v && j != i) dev_set_error(c.status, DEV_DUPLICATE_ID);
            }
            tmp[s + rank] = v;
            if (vals) c.idx_stage[s + rank] = c.sorted_idx[s + i];
        }
        __syncwarp();
        for (uint32_t i = lane; i < cnt; i += 32) {
            c.sorted[s + i] = tmp[s + i];
            if (vals) c.sorted_idx[s + i] = c.idx_stage[s + i];
        }
    }
    __syncthreads();

    const s3_postings_item& it = *c.it;
    const int32_t pos_base = (int32_t)it.pos_base;
    for (uint32_t i = tid; i < n; i += NT) {
        __stcs(it.d_pos + out_base + i, pos_base + (int32_t)c.sorted[i]);
        if (vals) it.d_pval[out_base + i] = __ldg(it.d_vals + c.sorted_idx[i]);
    }
    if (write_row_ptr) {
        for (uint32_t f = f_lo + tid; f < f_hi; f += NT) {
            const uint32_t fg = ((uint32_t)c.b << c.fbits) + f;
            if (fg < (uint32_t)it.d_sae) it.d_row_ptr[fg] = out_base + tbl16[(f - f_lo) << c.wbits];
        }
    }
    __syncthreads();
}

// One list longer than CAP: its tokens are distinct, so a bitmap over the tokens, read back in order, is the
// sorted list. Sweeps of BM_WORDS * 32 tokens.
template <bool VALS>
__device__ void bitmap_list(const BucketCtx& c, uint32_t f_rel, uint32_t out_base)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const s3_postings_item& it = *c.it;
    const bool vals = VALS && it.d_vals != nullptr;
    uint32_t* bm = c.e_stage;                               // e_stage and sorted are contiguous
    const int32_t f_glob = (int32_t)(((uint32_t)c.b << c.fbits) + f_rel);
    constexpr uint32_t SWEEP = (uint32_t)BM_WORDS * 32u;
    constexpr int WPT = BM_WORDS / NT;                      // words per thread, consecutive
    uint32_t out = out_base;
    for (uint32_t t0 = 0; t0 < (uint32_t)it.T; t0 += SWEEP) {
        for (int i = tid; i < BM_WORDS; i += NT) bm[i] = 0;
        __syncthreads();
        for (int r = warp; r < c.n_runs; r += NW) {
            const uint16_t* d = c.dir + (size_t)r * (c.B + 1) + c.b;
            const uint32_t s = __ldg(d), len = __ldg(d + 1) - s;
            const uint32_t* src = c.interm + (size_t)r * c.run_stride + s;
            for (uint32_t j = lane; j < len; j += 32) {
                const uint32_t e = __ldcg(src + j);
                const uint32_t t = (e & c.tmask) - t0;
                if ((e >> c.tbits) == f_rel && t < SWEEP) {
                    const uint32_t bit = 1u << (t & 31u);
                    if (atomicOr(&bm[t >> 5], bit) & bit) dev_set_error(c.status, DEV_DUPLICATE_ID);
                }
            }
        }
        __syncthreads();
        uint32_t cnt = 0;
        for (int q = 0; q < WPT; ++q) cnt += __popc(bm[tid * WPT + q]);
        uint32_t total;
        uint32_t off = out + block_scan_excl(cnt, c.warp_sums, &total);
        for (int q = 0; q < WPT; ++q) {
            uint32_t bits = bm[tid * WPT + q];
            while (bits) {
                const uint32_t bit = __ffs(bits) - 1;
                bits &= bits - 1;
                const uint32_t t = t0 + (uint32_t)(tid * WPT + q) * 32u + bit;
                it.d_pos[off] = (int32_t)it.pos_base + (int32_t)t;
                if (vals) {
                    const int32_t* row = it.d_ids + (size_t)t * it.k;
                    float v = 0.f;
                    for (int j = 0; j < it.k; ++j)
                        if (__ldg(row + j) == f_glob) { v = __ldg(it.d_vals + (size_t)t * it.k + j); break; }
                    it.d_pval[off] = v;
                }
                ++off;
            }
        }
        out += total;
        __syncthreads();
    }
}

template <bool VALS>
__global__ void __launch_bounds__(NT, VALS ? 1 : 2)
postings_bucket_kernel(const __grid_constant__ PostingsPlan pl)
{
    extern __shared__ uint32_t sm[];
    __shared__ uint32_t warp_sums[NW];
    __shared__ uint32_t counters[2];
    const int item = find_item2(pl, blockIdx.x);
    const s3_postings_item& it = pl.items[item];
    const ItemPlan& ip = pl.ip[item];
    const int tid = threadIdx.x;

    BucketCtx c;
    c.tbl = sm;
    c.e_stage = c.tbl + TBL / 2;
    c.sorted = c.e_stage + CAP;
    c.a_stage = reinterpret_cast<uint16_t*>(c.sorted + CAP);
    c.seg = c.a_stage + CAP;
    c.idx_stage = reinterpret_cast<uint32_t*>(c.seg + 3 * MAX_RUNS);
    c.sorted_idx = c.idx_stage + CAP;
    c.warp_sums = warp_sums;
    c.counters = counters;
    c.interm = reinterpret_cast<const uint32_t*>(pl.ws + ip.interm_off);
    c.idx = reinterpret_cast<const uint32_t*>(pl.ws + ip.idx_off);
    c.dir = reinterpret_cast<const uint16_t*>(pl.ws + ip.dir_off);
    c.it = &it;
    c.status = pl.status;
    c.n_runs = ip.n_runs;
    c.B = ip.n_buckets;
    c.b = blockIdx.x - ip.blk2_start;
    c.run_stride = ip.tok_per_run * it.k;
    c.tbits = ip.tbits;
    c.fbits = ip.fbits;
    c.wbits = ip.wbits;
    c.wshift = c.tbits - c.wbits;
    c.tmask = (1u << c.tbits) - 1u;

    // the bucket's segment in every run: first output offset = sum of the starts, size = sum of the lengths
    uint32_t bucket_base = 0, n_total = 0;
    const bool table_fits = c.n_runs <= MAX_RUNS;
    if (c.n_runs <= 128) {
        // the usual chunk: one warp, four runs per lane, shuffles only
        if (tid < 32) {
            uint32_t s4[4], l4[4], sum_s = 0, sum_l = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = 4 * tid + q;
                s4[q] = l4[q] = 0;
                if (r < c.n_runs) {
                    const uint16_t* d = c.dir + (size_t)r * (c.B + 1) + c.b;
                    s4[q] = __ldg(d);
                    l4[q] = __ldg(d + 1) - s4[q];
                }
                sum_s += s4[q];
                sum_l += l4[q];
            }
            uint32_t inc = sum_l;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
                if (tid >= o) inc += u;
                sum_s += __shfl_xor_sync(0xffffffffu, sum_s, o);
            }
            uint32_t off = inc - sum_l;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = 4 * tid + q;
                if (r < c.n_runs) {
                    c.seg[r] = (uint16_t)s4[q];
                    c.seg[MAX_RUNS + r] = (uint16_t)l4[q];
                    c.seg[2 * MAX_RUNS + r] = (uint16_t)off;
                }
                off += l4[q];
            }
            if (tid == 31) { counters[0] = sum_s; counters[1] = inc; }
        }
        __syncthreads();
        bucket_base = counters[0];
        n_total = counters[1];
        __syncthreads();
    } else
    for (int r0 = 0; r0 < c.n_runs; r0 += MAX_RUNS) {
        uint32_t s4[4], l4[4], sum_s = 0, sum_l = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int r = r0 + 4 * tid + q;
            s4[q] = l4[q] = 0;
            if (r < c.n_runs) {
                const uint16_t* d = c.dir + (size_t)r * (c.B + 1) + c.b;
                s4[q] = __ldg(d);
                l4[q] = __ldg(d + 1) - s4[q];
            }
            sum_s += s4[q];
            sum_l += l4[q];
        }
        uint32_t tot_l, tot_s;
        uint32_t off = n_total + block_scan_excl(sum_l, warp_sums, &tot_l);
        block_scan_excl(sum_s, warp_sums, &tot_s);
        if (table_fits) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = 4 * tid + q;
                if (r < c.n_runs) {
                    c.seg[r] = (uint16_t)s4[q];
                    c.seg[MAX_RUNS + r] = (uint16_t)l4[q];
                    c.seg[2 * MAX_RUNS + r] = (uint16_t)off;
                }
                off += l4[q];
            }
        }
        bucket_base += tot_s;
        n_total += tot_l;
    }
    __syncthreads();

    const uint32_t F = 1u << c.fbits;
    const uint32_t f_glob0 = (uint32_t)c.b << c.fbits;
    const uint32_t nf = min(F, (uint32_t)it.d_sae - f_glob0);
    if (c.b == c.B - 1 && tid == 0) it.d_row_ptr[it.d_sae] = bucket_base + n_total;

    if (table_fits && n_total <= (uint32_t)CAP) {
        sort_range<VALS, false>(c, 0, nf, n_total, bucket_base, true);
        return;
    }

    // large bucket: list lengths by global atomics into the bucket's own row_ptr entries, scanned in place
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t* rp = it.d_row_ptr + f_glob0;
    for (uint32_t f = tid; f < nf; f += NT) rp[f] = 0;
    __syncthreads();
    for (int r = warp; r < c.n_runs; r += NW) {
        const uint16_t* d = c.dir + (size_t)r * (c.B + 1) + c.b;
        const uint32_t s = __ldg(d), len = __ldg(d + 1) - s;
        const uint32_t* src = c.interm + (size_t)r * c.run_stride + s;
        for (uint32_t j = lane; j < len; j += 32) atomicAdd(&rp[__ldcg(src + j) >> c.tbits], 1u);
    }
    __syncthreads();
    uint32_t carry = bucket_base;
    for (uint32_t f0 = 0; f0 < nf; f0 += NT) {
        const uint32_t f = f0 + tid;
        const uint32_t v = f < nf ? __ldcg(rp + f) : 0u;
        uint32_t total;
        const uint32_t ex = block_scan_excl(v, warp_sums, &total);
        if (f < nf) rp[f] = carry + ex;
        carry += total;
    }
    __syncthreads();
    const uint32_t end_all = bucket_base + n_total;
    uint32_t f_lo = 0;
    while (f_lo < nf) {
        const uint32_t start = __ldcg(rp + f_lo);
        // the largest f_hi in (f_lo, nf] whose lists [f_lo, f_hi) hold at most CAP entries
        uint32_t lo = f_lo, hi = nf;                       // end(lo) - start <= CAP holds for lo = f_lo
        while (lo < hi) {
            const uint32_t mid = (lo + hi + 1) >> 1;
            const uint32_t end_mid = mid < nf ? __ldcg(rp + mid) : end_all;
            if (end_mid - start <= (uint32_t)CAP) lo = mid; else hi = mid - 1;
        }
        if (lo == f_lo) {
            bitmap_list<VALS>(c, f_lo, start);
            f_lo += 1;
        } else {
            const uint32_t end_hi = lo < nf ? __ldcg(rp + lo) : end_all;
            if (end_hi > start) sort_range<VALS, true>(c, f_lo, lo, 0, start, false);
            f_lo = lo;
        }
    }
}

int ceil_log2(uint64_t v)
{
    int b = 0;
    while ((1ull << b) < v) ++b;
    return b;
}

// Geometry of one item. Returns false when no bucket width fits (dictionary too wide for the token count).
bool plan_item(int T, int k, int d_sae, ItemPlan* ip, size_t* interm_bytes, size_t* dir_bytes)
{
    const uint64_t P = (uint64_t)T * k > 0 ? (uint64_t)T * k : 1;
    const int tbits = T > 1 ? ceil_log2((uint64_t)T) : 1;
    int fb = 0;
    while (fb < FB_MAX && ((P << (fb + 1)) / (uint64_t)d_sae) <= (uint64_t)TARGET_BUCKET) ++fb;
    const int fb_hi = FB_MAX < 32 - tbits ? FB_MAX : 32 - tbits;
    const int fb_lo = ceil_log2(((uint64_t)d_sae + B_MAX - 1) / B_MAX);
    if (fb_lo > fb_hi) return false;
    fb = fb < fb_lo ? fb_lo : (fb > fb_hi ? fb_hi : fb);
    ip->tbits = (unsigned char)tbits;
    ip->fbits = (unsigned char)fb;
    const int wb = TBL_BITS - fb < tbits ? TBL_BITS - fb : tbits;
    ip->wbits = (unsigned char)wb;
    ip->n_buckets = (int)(((uint64_t)d_sae + (1ull << fb) - 1) >> fb);
    ip->tok_per_run = RUN_PAIRS / k > 0 ? RUN_PAIRS / k : 1;
    ip->n_runs = T > 0 ? (T + ip->tok_per_run - 1) / ip->tok_per_run : 0;
    ip->magic_k = k >= 2 ? (uint32_t)((1ull << 32) / (uint64_t)k) + 1u : 0u;
    *interm_bytes = round_up((size_t)T * k * 4, 256);
    *dir_bytes = round_up((size_t)ip->n_runs * (ip->n_buckets + 1) * 2, 256);
    return true;
}

}  // namespace

size_t postings_workspace_bytes(int T, int k, int d_sae)
{
    if (T < 0 || k < 1 || d_sae < 1) return 0;
    ItemPlan ip;
    size_t interm = 0, dir = 0;
    if (!plan_item(T, k, d_sae, &ip, &interm, &dir)) return 0;
    return 2 * interm + dir;          // entries, pair indices (items with values), directory
}

s3_status launch_postings(const s3_postings_item* h_items, int n_items, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    constexpr size_t smem1 = (size_t)(B_MAX + RUN_PAIRS) * 4, smem1v = smem1 + (size_t)RUN_PAIRS * 4;
    constexpr size_t smem2 = (size_t)TBL * 2 + (size_t)CAP * (4 + 4 + 2) + (size_t)3 * MAX_RUNS * 2, smem2v = smem2 + (size_t)CAP * 8;
    static bool attr_set[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 64 && !attr_set[dev]) {
        S3_CUDA_TRY(cudaFuncSetAttribute(postings_partition_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1));
        S3_CUDA_TRY(cudaFuncSetAttribute(postings_partition_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1v));
        S3_CUDA_TRY(cudaFuncSetAttribute(postings_bucket_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2));
        S3_CUDA_TRY(cudaFuncSetAttribute(postings_bucket_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2v));
        attr_set[dev] = true;
    }
    PostingsPlan pl;
    pl.n_items = n_items;
    pl.ws = static_cast<unsigned char*>(d_ws);
    pl.status = static_cast<uint32_t*>(d_ws);
    size_t off = 256;
    int blk1 = 0, blk2 = 0;
    bool any_vals = false;
    for (int i = 0; i < n_items; ++i) {
        pl.items[i] = h_items[i];
        ItemPlan& ip = pl.ip[i];
        size_t interm = 0, dir = 0;
        S3_REQUIRE(plan_item(h_items[i].T, h_items[i].k, h_items[i].d_sae, &ip, &interm, &dir), S3_ERR_UNSUPPORTED,
                   "item %d: d_sae = %d is too wide for T = %d tokens (token bits + bucket bits exceed 32)", i, h_items[i].d_sae,
                   h_items[i].T);
        ip.has_val = h_items[i].d_vals != nullptr;
        any_vals |= ip.has_val != 0;
        ip.interm_off = off;
        off += interm;
        ip.idx_off = off;
        if (ip.has_val) off += interm;
        ip.dir_off = off;
        off += dir;
        ip.blk1_start = blk1;
        ip.blk2_start = blk2;
        blk1 += ip.n_runs;
        blk2 += ip.n_buckets;
    }
    pl.n_blk1 = blk1;
    pl.n_blk2 = blk2;
    S3_REQUIRE(off <= ws_bytes, S3_ERR_CAPACITY, "postings workspace holds %zu bytes, %zu needed", ws_bytes, off);
    if (blk1 > 0) {
        if (any_vals) postings_partition_kernel<true><<<blk1, NT, smem1v, stream>>>(pl);
        else postings_partition_kernel<false><<<blk1, NT, smem1, stream>>>(pl);
        S3_CUDA_TRY(cudaGetLastError());
    }
    if (blk2 > 0) {
        if (any_vals) postings_bucket_kernel<true><<<blk2, NT, smem2v, stream>>>(pl);
        else postings_bucket_kernel<false><<<blk2, NT, smem2, stream>>>(pl);
        S3_CUDA_TRY(cudaGetLastError());
    }
    return S3_OK;
}

}  // namespace s3
