// Head aggregation of per-head Top-k codes (Sec. 3.3, Sec. 3.4).
#include "s3_kernels.cuh"
#include "s3_query.cuh"

namespace s3 {

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

// The same result with one warp per token, for tokens of at most kWarpTokenPairs (id, value) pairs: the block-wide kernel
// above spends most of its time in block barriers on 256 pairs (8 heads x k = 32: 0.23 ms for 8192 tokens).
// keys = (id << 12 | index) sorted ascending puts a feature's entries next to each other in head order; the first entry
// of a run adds the run's activations in that order (fp32) and leaves the key (sum bits, ~id), every other slot 0; a
// second sort (descending) brings the k_out largest sums, ties to the lower id, to the front.
constexpr int kWarpTokenPairs = 512;       // at 1024 entries a warp's two sorts take as long as the block's (0.64 against 0.60 ms)
constexpr int kAggWarps = 4;

__global__ void __launch_bounds__(kAggWarps * 32) head_aggregate_warp_kernel(const __grid_constant__ HeadAggArgs a)
{
    extern __shared__ __align__(16) unsigned char agg_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned long long* sel = reinterpret_cast<unsigned long long*>(agg_smem) + static_cast<size_t>(warp) * a.npad;
    uint32_t* keys = reinterpret_cast<uint32_t*>(agg_smem + static_cast<size_t>(kAggWarps) * a.npad * 8) + static_cast<size_t>(warp) * a.npad;
    const int npad = a.npad, nk = a.nk;
    for (int t = blockIdx.x * kAggWarps + warp; t < a.T; t += gridDim.x * kAggWarps) {
        const int32_t* qi = a.ids + static_cast<size_t>(t) * nk;
        const float* qv = a.vals + static_cast<size_t>(t) * nk;
        for (int i = lane; i < npad; i += 32) {
            uint32_t key = 0xFFFFFFFFu;
            if (i < nk) {
                const int32_t f = qi[i];
                if (f >= 0 && f < a.d_sae) key = (static_cast<uint32_t>(f) << 12) | static_cast<uint32_t>(i);
            }
            keys[i] = key;
        }
        __syncwarp();
        for (int size = 2; size <= npad; size <<= 1)
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                for (int i = lane; i < (npad >> 1); i += 32) {
                    const int pos = 2 * i - (i & (stride - 1));
                    const bool asc = (pos & size) == 0;
                    const uint32_t x = keys[pos], y = keys[pos + stride];
                    if ((x > y) == asc) { keys[pos] = y; keys[pos + stride] = x; }
                }
                __syncwarp();
            }
        for (int i = lane; i < npad; i += 32) {
            unsigned long long key = 0ull;
            const uint32_t ki = keys[i];
            if (ki != 0xFFFFFFFFu && (i == 0 || (keys[i - 1] >> 12) != (ki >> 12))) {
                float sum = 0.0f;
                for (int j = i; j < npad && keys[j] != 0xFFFFFFFFu && (keys[j] >> 12) == (ki >> 12); ++j)
                    sum = __fadd_rn(sum, qv[keys[j] & 0xFFFu]);
                if (sum > 0.0f) key = make_key(__float_as_uint(sum), ki >> 12);
            }
            sel[i] = key;
        }
        __syncwarp();
        for (int size = 2; size <= npad; size <<= 1)
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                for (int i = lane; i < (npad >> 1); i += 32) {
                    const int pos = 2 * i - (i & (stride - 1));
                    const bool desc = (pos & size) == 0;
                    const unsigned long long x = sel[pos], y = sel[pos + stride];
                    if ((x < y) == desc) { sel[pos] = y; sel[pos + stride] = x; }
                }
                __syncwarp();
            }
        for (int j = lane; j < a.k_out; j += 32) {
            const unsigned long long key = j < npad ? sel[j] : 0ull;
            a.out_ids[static_cast<size_t>(t) * a.k_out + j] = key ? static_cast<int32_t>(~static_cast<uint32_t>(key)) : -1;
            a.out_vals[static_cast<size_t>(t) * a.k_out + j] = key ? __uint_as_float(static_cast<uint32_t>(key >> 32)) : 0.0f;
        }
        __syncwarp();
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
    if (a.nk <= kWarpTokenPairs) {
        const size_t wsmem = static_cast<size_t>(kAggWarps) * npad * 12;
        static bool wattr_set[64] = {};
        int wdev = 0;
        S3_CUDA_TRY(cudaGetDevice(&wdev));
        if (wdev < 64 && !wattr_set[wdev]) {
            S3_CUDA_TRY(cudaFuncSetAttribute(head_aggregate_warp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kAggWarps * kWarpTokenPairs * 12));
            wattr_set[wdev] = true;
        }
        const int blocks = (T + kAggWarps - 1) / kAggWarps, cap = device_sm_count() * 16;
        head_aggregate_warp_kernel<<<blocks < cap ? blocks : cap, kAggWarps * 32, wsmem, stream>>>(a);
        S3_CUDA_TRY(cudaGetLastError());
        return S3_OK;
    }
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

}  // namespace s3
