// Compact inverted index (Sec. 3.4, memory analysis: contiguous integer arrays with delta encoding and optional
// stop-feature pruning). One layer's merged CSR becomes, per feature, blocks of 32 postings: the block's first
// position, and the gaps (minus one) to the following positions bit-packed at the block's own width. A block is
// what one warp of the span scorer gathers at a time, so decoding is a 32-lane prefix sum.
//
//   plan    : kept list length (stop features keep nothing) and block count per feature;
//   scans   : prefix sums of both (one thread block each; the build runs once per context);
//   measure : one warp per block: first position, width = bit length of the largest gap-1, payload words;
//   scan    : prefix sum of the payload words;
//   pack    : one warp per block: values OR-ed into a shared-memory image of the block, copied out; descriptor
//             = (word offset << 6) | width. A zero word closes the payload so a two-word read never leaves it.
#include "s3_common.cuh"
#include "s3_kernels.cuh"

namespace s3 {

namespace {

constexpr int CT = 256;          // threads per block of the per-feature and per-block kernels
constexpr int SCAN_T = 1024;     // threads of the single-block scans

struct CompactArgs {
    const uint64_t* row_ptr;
    const int32_t* pos;
    uint64_t* out_row_ptr;
    uint32_t* blk_ptr;
    int32_t* blk_first;
    uint64_t* blk_desc;
    uint32_t* payload;
    uint64_t* word_off;      // scratch [cap_blocks + 1]
    uint64_t* sizes;         // [4]: kept postings, blocks, payload words (with the closing word), needed capacity flag
    uint32_t* status;
    uint64_t cap_blocks, cap_words;
    int64_t stop_freq;
    int d_sae;
};

__global__ void __launch_bounds__(CT) compact_plan_kernel(const __grid_constant__ CompactArgs a)
{
    const int f = blockIdx.x * CT + threadIdx.x;
    if (f > a.d_sae) return;
    uint64_t len = 0;
    if (f < a.d_sae) {
        len = a.row_ptr[f + 1] - a.row_ptr[f];
        if (a.stop_freq > 0 && len > static_cast<uint64_t>(a.stop_freq)) len = 0;
    }
    a.out_row_ptr[f] = len;
    a.blk_ptr[f] = static_cast<uint32_t>((len + 31) / 32);
}

// Exclusive prefix sum of v[0..n) in place by one thread block. The arrays here carry one extra slot whose input
// is 0, so the total lands in v[n-1].
template <typename T>
__device__ void block_scan_in_place(T* v, uint64_t n)
{
    __shared__ T warp_tot[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    T carry = 0;
    for (uint64_t i0 = 0; i0 < n; i0 += SCAN_T) {
        const uint64_t i = i0 + tid;
        const T x = i < n ? v[i] : T(0);
        T inc = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const T y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const T t = warp_tot[lane];
            T ti = t;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const T y = __shfl_up_sync(0xffffffffu, ti, o);
                if (lane >= o) ti += y;
            }
            warp_tot[lane] = ti - t;
            if (lane == 31) warp_tot[32] = ti;
        }
        __syncthreads();
        if (i < n) v[i] = carry + warp_tot[warp] + inc - x;
        carry += warp_tot[32];
        __syncthreads();
    }
}

// block 0: kept lengths -> out_row_ptr; block 1: block counts -> blk_ptr (both d_sae + 1 entries)
__global__ void __launch_bounds__(SCAN_T) compact_scan_features_kernel(const __grid_constant__ CompactArgs a)
{
    if (blockIdx.x == 0) block_scan_in_place<uint64_t>(a.out_row_ptr, static_cast<uint64_t>(a.d_sae) + 1);
    else block_scan_in_place<uint32_t>(a.blk_ptr, static_cast<uint64_t>(a.d_sae) + 1);
}

// Feature that owns block b: the last f with blk_ptr[f] <= b (features without blocks share a start).
__device__ __forceinline__ int owner_of_block(const uint32_t* blk_ptr, int d_sae, uint32_t b)
{
    int lo = 0, hi = d_sae;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (blk_ptr[mid] <= b) lo = mid; else hi = mid;
    }
    return lo;
}

// The 32 postings of block b: lane's position (or -1 past the block's end) and the block's posting count.
__device__ __forceinline__ int load_block(const CompactArgs& a, uint32_t b, int lane, uint32_t& cnt)
{
    const int f = owner_of_block(a.blk_ptr, a.d_sae, b);
    const uint64_t kept = a.out_row_ptr[f + 1] - a.out_row_ptr[f];
    const uint64_t j = b - a.blk_ptr[f];
    const uint64_t left = kept - 32 * j;
    cnt = left < 32 ? static_cast<uint32_t>(left) : 32u;
    return lane < static_cast<int>(cnt) ? a.pos[a.row_ptr[f] + 32 * j + lane] : -1;
}

__global__ void __launch_bounds__(CT) compact_measure_kernel(const __grid_constant__ CompactArgs a)
{
    const uint32_t n_blocks = a.blk_ptr[a.d_sae];
    const int lane = threadIdx.x & 31;
    const uint32_t warp0 = (blockIdx.x * CT + threadIdx.x) >> 5, n_warps = gridDim.x * (CT / 32);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.sizes[0] = a.out_row_ptr[a.d_sae];
        a.sizes[1] = n_blocks;
        if (n_blocks <= a.cap_blocks) a.word_off[n_blocks] = 0;
        else dev_set_error(a.status, DEV_COMPACT_CAPACITY);
    }
    if (n_blocks > a.cap_blocks) return;
    for (uint32_t b = warp0; b < n_blocks; b += n_warps) {
        uint32_t cnt;
        const int p = load_block(a, b, lane, cnt);
        const int prev = __shfl_up_sync(0xffffffffu, p, 1);
        uint32_t g = (lane >= 1 && lane < static_cast<int>(cnt)) ? static_cast<uint32_t>(p - prev - 1) : 0u;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) g |= __shfl_xor_sync(0xffffffffu, g, o);   // OR has the same bit length as max
        const uint32_t width = 32 - __clz(g);
        if (lane == 0) {
            a.blk_first[b] = p;
            a.blk_desc[b] = width;
            a.word_off[b] = (static_cast<uint64_t>(cnt - 1) * width + 31) / 32;
        }
    }
}

__global__ void __launch_bounds__(SCAN_T) compact_scan_words_kernel(const __grid_constant__ CompactArgs a)
{
    const uint32_t n_blocks = a.blk_ptr[a.d_sae];
    if (n_blocks > a.cap_blocks) return;
    block_scan_in_place<uint64_t>(a.word_off, static_cast<uint64_t>(n_blocks) + 1);
    if (threadIdx.x == 0) {
        const uint64_t words = a.word_off[n_blocks] + 1;      // with the closing word
        a.sizes[2] = words;
        a.sizes[3] = 0;
        if (words > a.cap_words) dev_set_error(a.status, DEV_COMPACT_CAPACITY);
        else a.payload[words - 1] = 0;
    }
}

__global__ void __launch_bounds__(CT) compact_pack_kernel(const __grid_constant__ CompactArgs a)
{
    __shared__ uint32_t image[CT / 32][32];
    const uint32_t n_blocks = a.blk_ptr[a.d_sae];
    if (n_blocks > a.cap_blocks || a.word_off[n_blocks] + 1 > a.cap_words) return;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t warp0 = (blockIdx.x * CT + threadIdx.x) >> 5, n_warps = gridDim.x * (CT / 32);
    for (uint32_t b = warp0; b < n_blocks; b += n_warps) {
        uint32_t cnt;
        const int p = load_block(a, b, lane, cnt);
        const int prev = __shfl_up_sync(0xffffffffu, p, 1);
        const uint32_t width = static_cast<uint32_t>(a.blk_desc[b]);
        const uint64_t off = a.word_off[b];
        const uint32_t n_words = static_cast<uint32_t>(a.word_off[b + 1] - off);
        image[w][lane] = 0;
        __syncwarp();
        if (lane >= 1 && lane < static_cast<int>(cnt) && width) {
            const uint64_t g = static_cast<uint32_t>(p - prev - 1);
            const uint32_t bit = (lane - 1) * width;
            const uint64_t shifted = g << (bit & 31);
            atomicOr(&image[w][bit >> 5], static_cast<uint32_t>(shifted));
            if (shifted >> 32) atomicOr(&image[w][(bit >> 5) + 1], static_cast<uint32_t>(shifted >> 32));
        }
        __syncwarp();
        if (lane < static_cast<int>(n_words)) a.payload[off + lane] = image[w][lane];
        __syncwarp();
        if (lane == 0) a.blk_desc[b] = (off << 6) | width;
    }
}

// The inverse of the build: every block's positions written back as a plain position array (one warp per block:
// gaps unpacked, 32-lane prefix sum), so that a consumer of the raw CSR can be fed from the compact form.
struct ExpandArgs {
    s3_compact_view v;
    int32_t* pos;
    uint64_t cap_postings;
    uint32_t* status;
    int d_sae;
};

__global__ void __launch_bounds__(CT) compact_expand_kernel(const __grid_constant__ ExpandArgs a)
{
    const uint32_t n_blocks = a.v.d_blk_ptr[a.d_sae];
    if (a.v.d_row_ptr[a.d_sae] > a.cap_postings) {
        if (blockIdx.x == 0 && threadIdx.x == 0) dev_set_error(a.status, DEV_COMPACT_CAPACITY);
        return;
    }
    const int lane = threadIdx.x & 31;
    const uint32_t warp0 = (blockIdx.x * CT + threadIdx.x) >> 5, n_warps = gridDim.x * (CT / 32);
    for (uint32_t b = warp0; b < n_blocks; b += n_warps) {
        const int f = owner_of_block(a.v.d_blk_ptr, a.d_sae, b);
        const uint64_t base = a.v.d_row_ptr[f], kept = a.v.d_row_ptr[f + 1] - base;
        const uint64_t j = b - a.v.d_blk_ptr[f];
        const uint64_t left = kept - 32 * j;
        const int cnt = left < 32 ? static_cast<int>(left) : 32;
        const uint64_t desc = a.v.d_blk_desc[b];
        const uint32_t width = static_cast<uint32_t>(desc & 63u);
        uint32_t val = 0;
        if (lane >= 1 && lane < cnt && width) {
            const uint32_t bit = (lane - 1) * width;
            const uint32_t* w = a.v.d_payload + (desc >> 6) + (bit >> 5);
            val = __funnelshift_r(w[0], w[1], bit & 31) & ((1u << width) - 1u);     // the closing word keeps w[1] in bounds
        }
        int d = lane == 0 ? a.v.d_blk_first[b] : (lane < cnt ? static_cast<int>(val) + 1 : 0);
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, d, o);
            if (lane >= o) d += y;
        }
        if (lane < cnt) a.pos[base + 32 * j + lane] = d;
    }
}

}  // namespace

void compact_bound(uint64_t n_postings, int d_sae, uint64_t* max_blocks, uint64_t* max_words)
{
    const uint64_t lists = n_postings < static_cast<uint64_t>(d_sae) ? n_postings : static_cast<uint64_t>(d_sae);
    *max_blocks = n_postings / 32 + lists;       // a list of n postings has at most n/32 + 1 blocks
    *max_words = n_postings + 1;                 // c - 1 values of at most 31 bits fit c - 1 words; one closing word
}

size_t compact_workspace_bytes(uint64_t n_postings, int d_sae)
{
    uint64_t b, w;
    compact_bound(n_postings, d_sae, &b, &w);
    return static_cast<size_t>(b + 1) * 8;
}

s3_status launch_compact_build(const uint64_t* d_row_ptr, const int32_t* d_pos, int d_sae, int64_t stop_freq,
                               uint64_t* d_out_row_ptr, uint32_t* d_blk_ptr, int32_t* d_blk_first, uint64_t* d_blk_desc,
                               uint64_t cap_blocks, uint32_t* d_payload, uint64_t cap_words, uint64_t* d_sizes,
                               uint32_t* d_status, void* d_scratch, cudaStream_t stream)
{
    CompactArgs a;
    a.row_ptr = d_row_ptr; a.pos = d_pos; a.out_row_ptr = d_out_row_ptr; a.blk_ptr = d_blk_ptr;
    a.blk_first = d_blk_first; a.blk_desc = d_blk_desc; a.payload = d_payload;
    a.word_off = static_cast<uint64_t*>(d_scratch); a.sizes = d_sizes; a.status = d_status;
    a.cap_blocks = cap_blocks; a.cap_words = cap_words; a.stop_freq = stop_freq; a.d_sae = d_sae;
    const int grid = device_sm_count() * 8;
    compact_plan_kernel<<<(d_sae + 1 + CT - 1) / CT, CT, 0, stream>>>(a);
    compact_scan_features_kernel<<<2, SCAN_T, 0, stream>>>(a);
    compact_measure_kernel<<<grid, CT, 0, stream>>>(a);
    compact_scan_words_kernel<<<1, SCAN_T, 0, stream>>>(a);
    compact_pack_kernel<<<grid, CT, 0, stream>>>(a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

s3_status launch_compact_expand(const s3_compact_view& v, int d_sae, int32_t* d_pos, uint64_t cap_postings, uint32_t* d_status,
                                cudaStream_t stream)
{
    ExpandArgs a;
    a.v = v; a.pos = d_pos; a.cap_postings = cap_postings; a.status = d_status; a.d_sae = d_sae;
    compact_expand_kernel<<<device_sm_count() * 8, CT, 0, stream>>>(a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
