// Per-row running Top-k (Sec. 3.3, Eq. 2) kept as a min-heap of 64-bit candidate keys in shared memory.
//
// One thread owns one row. The heap of row r lives at heap[slot * ROWS + r], so the 32 lanes of a
// warp always hit 32 different banks whatever slot each lane touches. The root (slot 0) is the
// worst retained candidate; a new candidate enters only if its key is larger than the root's.
// A heap initialised with zeros ("no candidate") needs no fill phase: zeros are simply the first
// entries to be replaced, and whatever zeros remain at the end are the row's padding.
#pragma once

#include "s3_common.cuh"

namespace s3 {

template <int ROWS>
__device__ __forceinline__ void heap_init(uint64_t* heap, int row, int k)
{
    for (int s = 0; s < k; ++s) heap[s * ROWS + row] = 0ull;
}

// Replaces the root by `key` (caller guarantees key > root) and restores the heap. Returns the new root.
template <int ROWS>
__device__ __forceinline__ uint64_t heap_replace_root(uint64_t* heap, int row, int k, uint64_t key)
{
    int i = 0;
    while (true) {
        int c = 2 * i + 1;
        if (c >= k) break;
        uint64_t kc = heap[c * ROWS + row];
        if (c + 1 < k) {
            const uint64_t k2 = heap[(c + 1) * ROWS + row];
            if (k2 < kc) { kc = k2; c = c + 1; }
        }
        if (kc >= key) break;
        heap[i * ROWS + row] = kc;
        i = c;
    }
    heap[i * ROWS + row] = key;
    return heap[row];
}

// Layout of the partial lists exchanged between the encode kernels and the merge kernel:
// part[(t * n_slices + slice) * k + j], j = 0..k-1, unordered, 0 = empty.
void launch_topk_merge(const uint64_t* d_part, int T, int n_slices, int k, int32_t* d_ids, float* d_vals,
                       cudaStream_t stream);

// Candidate lists of the tensor-core encode: cand[(t * n_slices + slice) * cap + i], i < counts[t * n_slices + slice],
// unordered keys; hint[t] = float bits of a bound that at least k values of row t exceed.
// The same for the candidate lists of several encoder calls in one launch; row_start = first row of the item in the
// launch's flattened row range (a multiple of kMergeRowsPerBlock).
constexpr int kMergeRowsPerBlock = 4;
struct MergeItem {
    const uint64_t* cand;
    const uint32_t* counts;
    const uint32_t* hint;
    int32_t* ids;
    float* vals;
    int T, n_slices, k;
    uint32_t cap;
    int row_start;
};
struct MergeGroup {
    MergeItem item[S3_MAX_ENCODE_ITEMS];
    int n_items;
};
void launch_candidate_merge_group(const MergeGroup& g, int total_rows, cudaStream_t stream);

void launch_candidate_merge(const uint64_t* d_cand, const uint32_t* d_counts, const uint32_t* d_hint, int T, int n_slices,
                            uint32_t cap, int k, int32_t* d_ids, float* d_vals, cudaStream_t stream);

}  // namespace s3
