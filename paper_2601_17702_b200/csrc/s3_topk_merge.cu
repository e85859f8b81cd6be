// Final selection of the Top-k (Sec. 3.3, Eq. 2): merges the unordered partial candidate lists that
// the encode kernels leave per (token, column slice) into each token's k best, ordered by
// (value descending, id ascending), and unpacks them into ids / values.
#include "s3_topk.cuh"

namespace s3 {

namespace {

constexpr int kMergeWarps = 4;

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

}  // namespace s3
