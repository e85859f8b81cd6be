// Final selection of the Top-k (Sec. 3.3, Eq. 2): merges the unordered partial candidate lists that
// the encode kernels leave per (token, column slice) into each token's k best, ordered by
// (value descending, id ascending), and unpacks them into ids / values.
#include "s3_topk.cuh"

namespace s3 {

namespace {

constexpr int kMergeWarps = kMergeRowsPerBlock;

// One warp per token: bitonic sort (descending) of the token's n_slices*k keys, padded with zeros to
// a power of two, in the warp's private shared-memory segment.
__global__ void __launch_bounds__(kMergeWarps * 32)
topk_merge_kernel(const uint64_t* __restrict__ part, int T, int n, int npad, int k,
                  int32_t* __restrict__ ids, float* __restrict__ vals)
{
    extern __shared__ uint64_t merge_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * kMergeWarps + warp;
    if (t >= T) return;
    uint64_t* buf = merge_smem + (size_t)warp * npad;
    const uint64_t* src = part + (size_t)t * n;
    for (int i = lane; i < npad; i += 32) buf[i] = (i < n) ? src[i] : 0ull;
    __syncwarp();
    for (int size = 2; size <= npad; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = lane; i < (npad >> 1); i += 32) {
                const int pos = ((i / stride) * (stride << 1)) + (i % stride);
                const bool desc = (pos & size) == 0;
                const uint64_t a = buf[pos], b = buf[pos + stride];
                if ((a < b) == desc) { buf[pos] = b; buf[pos + stride] = a; }
            }
            __syncwarp();
        }
    }
    for (int j = lane; j < k; j += 32) {
        const uint64_t key = buf[j];
        ids[(size_t)t * k + j] = key ? static_cast<int32_t>(~static_cast<uint32_t>(key)) : -1;
        vals[(size_t)t * k + j] = key ? __uint_as_float(static_cast<uint32_t>(key >> 32)) : 0.0f;
    }
}

// Exact Top-k of one row from the candidate lists of its slices. One warp per row:
//   1. survivors = candidates above the best bound published for the row (at least k values exceed it,
//      so nothing at or below it can be among the k best), gathered into the warp's shared-memory buffer;
//   2. when they do not fit (many short lists, each with its own k survivors, at a large k), the bound is raised
//      first from the lists themselves: a 64-bucket histogram of the float bits above the bound gives the
//      highest bucket edge that k candidates still reach, with finer buckets when the k-th value's bucket alone
//      is too full (a radix selection, one pass over the lists per step), and the gather is repeated;
//   3. bitonic sort of the survivors (a couple of hundred keys at most in the usual case);
//   4. rows that still do not fit after kRefineSteps (long runs of equal values) fall back to k rounds of
//      "largest key below the previous one" over the lists in global memory.
constexpr int kCandBuf = 512;    // survivor slots per warp (1024 halves the warps an SM holds: key SAE encode + merge 0.269 -> 0.260 ms at 512)
constexpr int kRefineSteps = 8;

// Calls f(key, valid) for all candidates of the row, 128 at a time (four per lane), every lane of the warp taking
// part in every call. Up to 32 lists at a time (more in rounds): the lists' lengths are prefix-summed over the
// lanes, and the entries of all those lists form one flat range, so the loads of different lists are in flight
// together instead of one list after the other. f returns false to stop the walk.
template <typename F>
__device__ __forceinline__ void walk_lists(const uint64_t* __restrict__ cand, const uint32_t* __restrict__ counts, int t, int n_slices,
                                           uint32_t cap, uint32_t* start, int lane, F f)
{
    bool go = true;
    for (int s0 = 0; s0 < n_slices && go; s0 += 32) {
        const int ns = n_slices - s0 < 32 ? n_slices - s0 : 32;
        const uint32_t my_cnt = lane < ns ? counts[(size_t)t * n_slices + s0 + lane] : 0u;
        uint32_t inc = my_cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        const uint32_t total = __shfl_sync(0xffffffffu, inc, 31);
        __syncwarp();
        start[lane] = inc - my_cnt;                            // first flat index of list s0 + lane
        __syncwarp();
        const uint64_t* lists = cand + ((size_t)t * n_slices + s0) * cap;
        for (uint32_t i0 = 0; i0 < total && go; i0 += 128) {
            uint64_t key[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t i = i0 + q * 32 + lane;
                key[q] = 0ull;
                if (i < total) {
                    int lo = 0, hi = 32;                       // last list whose start is <= i (empty lists share a start)
#pragma unroll
                    for (int step = 0; step < 5; ++step) {
                        const int mid = (lo + hi) >> 1;
                        if (start[mid] <= i) lo = mid; else hi = mid;
                    }
                    key[q] = lists[(size_t)lo * cap + (i - start[lo])];
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (go) go = f(key[q]);
        }
    }
}

// Highest of 64 buckets that at least k counted values reach (0 when only bucket 0 does). Lane l holds buckets 2l, 2l+1.
__device__ __forceinline__ int highest_bucket_with_k(const uint32_t* hist, int k, int lane)
{
    const uint32_t h0 = hist[2 * lane], h1 = hist[2 * lane + 1];
    uint32_t suf = h0 + h1;                                  // buckets >= 2l, after the scan
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += up;
    }
    int best = (suf - h0 >= static_cast<uint32_t>(k)) ? 2 * lane + 1 : ((suf >= static_cast<uint32_t>(k)) ? 2 * lane : 0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const int other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    return best;
}

// Ten blocks per SM (48 registers): the kernel waits on its list loads, so resident warps count (heads, k = 32: 1.156 -> 1.131 ms
// for encode + merge; 72 registers allowed seven blocks).
__global__ void __launch_bounds__(kMergeWarps * 32, 10)
candidate_merge_kernel(const __grid_constant__ MergeGroup g)
{
    __shared__ uint64_t cand_buf[kMergeWarps][kCandBuf];
    __shared__ uint32_t cand_hist[kMergeWarps][64];
    __shared__ uint32_t cand_start[kMergeWarps][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * kMergeWarps + warp;
    int item = g.n_items - 1;
    while (item > 0 && g.item[item].row_start > row) --item;
    const MergeItem& mi = g.item[item];
    const int t = row - mi.row_start;
    if (t >= mi.T) return;
    const uint64_t* __restrict__ cand = mi.cand;
    const uint32_t* __restrict__ counts = mi.counts;
    const uint32_t* __restrict__ hint = mi.hint;
    int32_t* __restrict__ ids = mi.ids;
    float* __restrict__ vals = mi.vals;
    const int n_slices = mi.n_slices, k = mi.k;
    const uint32_t cap = mi.cap;
    uint64_t* buf = cand_buf[warp];
    uint32_t* hist = cand_hist[warp];
    uint32_t* start = cand_start[warp];
    float tau = __uint_as_float(hint[t]);
    uint32_t n = 0;            // survivors so far (warp-uniform)
    bool overflow = false;
    int shift = 19;            // bucket = float bits >> shift: 16 buckets per octave at first
    for (int round = 0;; ++round) {
        n = 0;
        overflow = false;
        walk_lists(cand, counts, t, n_slices, cap, start, lane, [&](uint64_t key) {
            const bool keep = __uint_as_float(static_cast<uint32_t>(key >> 32)) > tau;   // key 0: value 0, never kept
            const uint32_t m = __ballot_sync(0xffffffffu, keep);
            if (n + __popc(m) > kCandBuf) { overflow = true; return false; }
            if (keep) buf[n + __popc(m & ((1u << lane) - 1u))] = key;
            n += __popc(m);
            return true;
        });
        if (!overflow || round == kRefineSteps) break;
        // too many candidates above the bound: raise it to the highest bucket edge that k of them reach
        hist[lane] = 0; hist[lane + 32] = 0;
        __syncwarp();
        const uint32_t base = __float_as_uint(tau) >> shift;
        walk_lists(cand, counts, t, n_slices, cap, start, lane, [&](uint64_t key) {
            const uint32_t vb = static_cast<uint32_t>(key >> 32);
            if (__uint_as_float(vb) > tau) {
                const uint32_t idx = (vb >> shift) - base;
                atomicAdd(&hist[idx > 63u ? 63u : idx], 1u);
            }
            return true;
        });
        __syncwarp();
        const int best = highest_bucket_with_k(hist, k, lane);
        const uint32_t edge = ((base + static_cast<uint32_t>(best)) << shift) - 1u;      // value >= edge of bucket `best`
        if (best > 0 && edge > __float_as_uint(tau)) tau = __uint_as_float(edge);
        else if (shift >= 6) shift -= 6;                   // the k-th value's bucket alone is too full: finer buckets
        else { round = kRefineSteps - 1; }                  // single float values left: equal keys, the fallback handles them
        __syncwarp();
    }
    if (!overflow && n > 2u * static_cast<uint32_t>(k)) {
        // Many more survivors than k: tighten the bound once more before sorting. A 64-bucket histogram over the
        // float bits above the bound's bucket (16 buckets per octave) shows the highest bucket edge that k
        // survivors still reach; what lies below it is dropped.
        hist[lane] = 0; hist[lane + 32] = 0;
        __syncwarp();
        const int base = static_cast<int>(__float_as_uint(tau) >> 19);
        for (uint32_t i = lane; i < n; i += 32) {
            int idx = static_cast<int>(static_cast<uint32_t>(buf[i] >> 32) >> 19) - base;
            idx = idx < 0 ? 0 : (idx > 63 ? 63 : idx);
            atomicAdd(&hist[idx], 1u);
        }
        __syncwarp();
        const int best = highest_bucket_with_k(hist, k, lane);
        if (best > 0) {
            const float tau2 = __uint_as_float((static_cast<uint32_t>(base + best) << 19) - 1u);   // value >= edge
            uint32_t w = 0;
            for (uint32_t i0 = 0; i0 < n; i0 += 32) {
                const uint32_t i = i0 + lane;
                const uint64_t key = i < n ? buf[i] : 0ull;
                const bool keep = i < n && __uint_as_float(static_cast<uint32_t>(key >> 32)) > tau2;
                const uint32_t m = __ballot_sync(0xffffffffu, keep);
                if (keep) buf[w + __popc(m & ((1u << lane) - 1u))] = key;      // w <= i0: never an unread slot
                w += __popc(m);
            }
            __syncwarp();
            n = w;
        }
    }
    if (!overflow) {
        uint32_t npad = 32;
        while (npad < n) npad <<= 1;
        for (uint32_t i = n + lane; i < npad; i += 32) buf[i] = 0ull;
        __syncwarp();
        for (uint32_t size = 2; size <= npad; size <<= 1) {
            for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
                for (uint32_t i = lane; i < (npad >> 1); i += 32) {
                    const uint32_t pos = 2 * i - (i & (stride - 1));
                    const bool desc = (pos & size) == 0;
                    const uint64_t a = buf[pos], b = buf[pos + stride];
                    if ((a < b) == desc) { buf[pos] = b; buf[pos + stride] = a; }
                }
                __syncwarp();
            }
        }
        for (int j = lane; j < k; j += 32) {
            const uint64_t key = static_cast<uint32_t>(j) < n ? buf[j] : 0ull;
            ids[(size_t)t * k + j] = key ? static_cast<int32_t>(~static_cast<uint32_t>(key)) : -1;
            vals[(size_t)t * k + j] = key ? __uint_as_float(static_cast<uint32_t>(key >> 32)) : 0.0f;
        }
        return;
    }
    // fallback: selection by repeated maximum (keys are distinct, so "below the previous" removes exactly one)
    uint64_t prev = ~0ull;
    for (int j = 0; j < k; ++j) {
        uint64_t best = 0ull;
        for (int s = 0; s < n_slices; ++s) {
            const uint32_t cnt = counts[(size_t)t * n_slices + s];
            const uint64_t* list = cand + ((size_t)t * n_slices + s) * cap;
            for (uint32_t i = lane; i < cnt; i += 32) {
                const uint64_t key = list[i];
                if (key < prev && key > best) best = key;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const uint64_t other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (lane == 0) {
            ids[(size_t)t * k + j] = best ? static_cast<int32_t>(~static_cast<uint32_t>(best)) : -1;
            vals[(size_t)t * k + j] = best ? __uint_as_float(static_cast<uint32_t>(best >> 32)) : 0.0f;
        }
        prev = best ? best : 0ull;      // nothing left: every later round finds nothing either
    }
}

}  // namespace

void launch_topk_merge(const uint64_t* d_part, int T, int n_slices, int k, int32_t* d_ids, float* d_vals,
                       cudaStream_t stream)
{
    if (T <= 0) return;
    const int n = n_slices * k;
    int npad = 32;
    while (npad < n) npad <<= 1;
    const size_t smem = (size_t)kMergeWarps * npad * sizeof(uint64_t);
    const int grid = (T + kMergeWarps - 1) / kMergeWarps;
    topk_merge_kernel<<<grid, kMergeWarps * 32, smem, stream>>>(d_part, T, n, npad, k, d_ids, d_vals);
}

void launch_candidate_merge_group(const MergeGroup& g, int total_rows, cudaStream_t stream)
{
    if (total_rows <= 0) return;
    candidate_merge_kernel<<<total_rows / kMergeWarps, kMergeWarps * 32, 0, stream>>>(g);
}

void launch_candidate_merge(const uint64_t* d_cand, const uint32_t* d_counts, const uint32_t* d_hint, int T, int n_slices,
                            uint32_t cap, int k, int32_t* d_ids, float* d_vals, cudaStream_t stream)
{
    if (T <= 0) return;
    MergeGroup g;
    g.n_items = 1;
    g.item[0] = MergeItem{d_cand, d_counts, d_hint, d_ids, d_vals, T, n_slices, k, cap, 0};
    launch_candidate_merge_group(g, (T + kMergeWarps - 1) / kMergeWarps * kMergeWarps, stream);
}

}  // namespace s3
