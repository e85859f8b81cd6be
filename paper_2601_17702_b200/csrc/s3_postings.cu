// Per-chunk CSR posting lists (Sec. 3.4, Eq. 4: I[f] <- I[f] U {t} for every f in F_t).
//
// One thread block builds one chunk-layer in a single launch, with the per-feature counters /
// write cursors held in shared memory (4 bytes per feature):
//   1. histogram of the ids (shared-memory atomics)           -> list lengths
//   2. exclusive block scan                                   -> row_ptr (global) and cursors (shared)
//   3. ordered scatter, sub-tile by sub-tile in token order   -> pos (and pval)
// Step 3 keeps every list in ascending position: a sub-tile is a run of consecutive tokens; inside
// it each pair takes a ticket from its feature's cursor (the top 8 bits of the cursor word count the
// sub-tile's tickets, the low 24 bits keep the run start), and pairs that share a feature within
// the sub-tile then re-rank themselves by position before the final write. Features are distinct
// within a token, so a feature gets at most one ticket per token and at most 255 per sub-tile.
#include "s3_common.cuh"

namespace s3 {

namespace {

constexpr int PT = 1024;   // threads per block
constexpr int PER = 4;     // pairs per thread per sub-tile
constexpr uint32_t LOW24 = 0x00FFFFFFu;

struct PostingsBatch {
    s3_postings_item items[S3_MAX_POSTINGS_ITEMS];
};

__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* warp_sums, uint32_t& total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = warp_sums[lane];
        uint32_t winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        warp_sums[lane] = winc - w;          // exclusive prefix of the warp sums
        if (lane == 31) warp_sums[32] = winc;  // block total
    }
    __syncthreads();
    const uint32_t res = warp_sums[warp] + inc - v;
    total = warp_sums[32];
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(PT)
postings_kernel(const __grid_constant__ PostingsBatch batch, uint32_t* __restrict__ status)
{
    extern __shared__ uint32_t cursor[];     // [d_sae]
    __shared__ uint32_t warp_sums[33];

    const s3_postings_item it = batch.items[blockIdx.x];
    const int tid = threadIdx.x;
    const int d_sae = it.d_sae, k = it.k;
    const int64_t n_pairs = (int64_t)it.T * k;
    const int32_t* __restrict__ ids = it.d_ids;

    for (int f = tid; f < d_sae; f += PT) cursor[f] = 0;
    __syncthreads();

    // 1. histogram
    for (int64_t p = tid; p < n_pairs; p += PT) {
        const int32_t f = ids[p];
        if (f >= 0) {
            if (f < d_sae) atomicAdd(&cursor[f], 1u);
            else dev_set_error(status, DEV_BAD_FEATURE_ID);
        }
    }
    __syncthreads();

    // 2. exclusive scan -> row_ptr, cursors
    uint32_t carry = 0;
    for (int f0 = 0; f0 < d_sae; f0 += PT) {
        const int f = f0 + tid;
        const uint32_t v = (f < d_sae) ? cursor[f] : 0u;
        uint32_t total;
        const uint32_t ex = block_exclusive_scan(v, warp_sums, total) + carry;
        if (f < d_sae) { cursor[f] = ex; it.d_row_ptr[f] = ex; }
        carry += total;
    }
    if (tid == 0) it.d_row_ptr[d_sae] = carry;
    __syncthreads();

    // 3. ordered scatter
    int ts = (PT * PER) / k;
    ts = ts < 1 ? 1 : (ts > 255 ? 255 : ts);
    const int64_t sub_pairs = (int64_t)ts * k;
    const int64_t cap = n_pairs;
    const bool has_val = it.d_vals != nullptr && it.d_pval != nullptr;
    for (int64_t base = 0; base < n_pairs; base += sub_pairs) {
        const int64_t lim = (n_pairs - base < sub_pairs) ? (n_pairs - base) : sub_pairs;
        int32_t f[PER];
        uint32_t a[PER], cm[PER];
        int32_t mypos[PER];
        float myval[PER];
        bool any_multi = false;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int64_t q = tid + (int64_t)j * PT;
            f[j] = -1;
            if (q < lim) {
                const int64_t p = base + q;
                const int32_t fj = ids[p];
                if (fj >= 0 && fj < d_sae) {
                    f[j] = fj;
                    mypos[j] = (int32_t)(it.pos_base + p / k);
                    if (has_val) myval[j] = it.d_vals[p];
                    a[j] = atomicAdd(&cursor[fj], 1u << 24) >> 24;
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (f[j] >= 0) {
                cm[j] = cursor[f[j]];
                const uint32_t m = cm[j] >> 24, c = cm[j] & LOW24;
                if (m == 1) {
                    if (c < cap) { it.d_pos[c] = mypos[j]; if (has_val) it.d_pval[c] = myval[j]; }
                } else {
                    any_multi = true;
                    if ((int64_t)c + a[j] < cap) it.d_pos[c + a[j]] = mypos[j];   // provisional slot
                }
            }
        }
        const int multi = __syncthreads_or(any_multi ? 1 : 0);
        if (multi) {
            uint32_t rank[PER];
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                rank[j] = 0;
                if (f[j] >= 0 && (cm[j] >> 24) > 1) {
                    const uint32_t m = cm[j] >> 24, c = cm[j] & LOW24;
                    for (uint32_t e = 0; e < m; ++e)
                        if ((int64_t)c + e < cap && __ldcg(&it.d_pos[c + e]) < mypos[j]) ++rank[j];
                }
            }
            __syncthreads();
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                if (f[j] >= 0 && (cm[j] >> 24) > 1) {
                    const uint32_t c = cm[j] & LOW24;
                    if ((int64_t)c + rank[j] < cap) {
                        it.d_pos[c + rank[j]] = mypos[j];
                        if (has_val) it.d_pval[c + rank[j]] = myval[j];
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < PER; ++j)
            if (f[j] >= 0 && a[j] == 0) cursor[f[j]] = (cm[j] & LOW24) + (cm[j] >> 24);
        __syncthreads();
    }
}

}  // namespace

s3_status launch_postings(const s3_postings_item* h_items, int n_items, uint32_t* d_status, cudaStream_t stream)
{
    static bool attr_set[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 64 && !attr_set[dev]) {
        S3_CUDA_TRY(cudaFuncSetAttribute(postings_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 49152 * 4));
        attr_set[dev] = true;
    }
    PostingsBatch batch;
    int max_d = 0;
    for (int i = 0; i < n_items; ++i) {
        batch.items[i] = h_items[i];
        if (h_items[i].d_sae > max_d) max_d = h_items[i].d_sae;
    }
    postings_kernel<<<n_items, PT, (size_t)max_d * sizeof(uint32_t), stream>>>(batch, d_status);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
