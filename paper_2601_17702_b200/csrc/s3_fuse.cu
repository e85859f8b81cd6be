// Hybrid fusion of index sets (Sec. 3.6, Eq. 7): M_final = M_S3 U M_BM25 U M_Bias per query, as ascending unique
// positions. One block per query marks the members in a bitmap of L bits (global scratch): the windows around
// the selected density peaks, the supplied lexical positions, the first `lead` and last `tail` positions; a
// block scan over the words' population counts then gives every word its place in the output.
#include "s3_common.cuh"
#include "s3_kernels.cuh"

namespace s3 {

namespace {

constexpr int FT = 256;   // threads per block

struct FuseArgs {
    const int32_t* centers;   // [Q, n_centers], -1 = none
    const int32_t* lexical;   // [Q, n_lex] or null; < 0 = padding, >= L ignored
    uint32_t* bitmap;         // [Q, n_words]
    int32_t* out_idx;         // [Q, cap]
    int32_t* out_count;       // [Q]
    long long L, n_words;
    int n_centers, n_lex, span_width, lead, tail, cap;
};

__device__ __forceinline__ void mark(uint32_t* bm, long long t, long long L)
{
    if (t >= 0 && t < L) atomicOr(&bm[t >> 5], 1u << (t & 31));
}

__global__ void __launch_bounds__(FT)
fuse_sets_kernel(const __grid_constant__ FuseArgs a)
{
    __shared__ uint32_t warp_sums[FT / 32 + 1];
    const int q = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* bm = a.bitmap + (size_t)q * a.n_words;
    for (long long w = tid; w < a.n_words; w += FT) bm[w] = 0;
    __syncthreads();

    const long long n_win = (long long)a.n_centers * a.span_width;
    for (long long i = tid; i < n_win; i += FT) {
        const int c = a.centers[(size_t)q * a.n_centers + i / a.span_width];
        if (c >= 0) mark(bm, (long long)c - a.span_width / 2 + i % a.span_width, a.L);
    }
    if (a.lexical)
        for (int j = tid; j < a.n_lex; j += FT) mark(bm, a.lexical[(size_t)q * a.n_lex + j], a.L);
    for (long long t = tid; t < a.lead; t += FT) mark(bm, t, a.L);
    for (long long t = tid; t < a.tail; t += FT) mark(bm, a.L - 1 - t, a.L);
    __syncthreads();

    uint32_t carry = 0;
    for (long long w0 = 0; w0 < a.n_words; w0 += FT) {
        const long long w = w0 + tid;
        uint32_t bits = w < a.n_words ? bm[w] : 0u;
        const uint32_t v = __popc(bits);
        uint32_t inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += u;
        }
        if (lane == 31) warp_sums[warp] = inc;
        __syncthreads();
        if (tid == 0) {
            uint32_t run = 0;
            for (int i = 0; i < FT / 32; ++i) { const uint32_t t = warp_sums[i]; warp_sums[i] = run; run += t; }
            warp_sums[FT / 32] = run;
        }
        __syncthreads();
        uint32_t at = carry + warp_sums[warp] + inc - v;
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            if (at < static_cast<uint32_t>(a.cap)) a.out_idx[(size_t)q * a.cap + at] = static_cast<int32_t>(w * 32 + b);
            ++at;
        }
        carry += warp_sums[FT / 32];
        __syncthreads();
    }
    for (long long i = (long long)carry + tid; i < a.cap; i += FT) a.out_idx[(size_t)q * a.cap + i] = -1;
    if (tid == 0) a.out_count[q] = static_cast<int32_t>(carry);
}

}  // namespace

size_t fuse_workspace_bytes(int Q, int64_t L) { return static_cast<size_t>(Q) * static_cast<size_t>((L + 31) / 32) * 4; }

s3_status launch_fuse_sets(const int32_t* d_centers, int Q, int n_centers, int span_width, const int32_t* d_lexical, int n_lex,
                           int lead, int tail, int64_t L, int32_t* d_out_idx, int cap, int32_t* d_out_count, void* d_scratch,
                           cudaStream_t stream)
{
    FuseArgs a;
    a.centers = d_centers; a.lexical = d_lexical; a.bitmap = static_cast<uint32_t*>(d_scratch);
    a.out_idx = d_out_idx; a.out_count = d_out_count;
    a.L = L; a.n_words = (L + 31) / 32;
    a.n_centers = n_centers; a.n_lex = n_lex; a.span_width = span_width; a.lead = lead; a.tail = tail; a.cap = cap;
    fuse_sets_kernel<<<Q, FT, 0, stream>>>(a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
