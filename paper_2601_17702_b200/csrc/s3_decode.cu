// SAE decode (Sec. 3.3, the reconstruction stated after Eq. 2): x_hat = z_hat W_dec + b_dec for the Top-k code of
// every token, and optionally the token's squared reconstruction error against x. A token needs k rows of W_dec
// (k * d_in elements, mostly L2 hits: a dictionary row is shared by every token that activates it) and writes d_in
// values: gather-bound, no contraction worth a tensor core at k <= 64.
//
// One block per token (grid-stride). The token's (id, value) pairs sit in shared memory; a thread owns VEC
// consecutive columns per pass and adds the k scaled rows in the order given with fp32 FMAs, b_dec last.
#include <cuda_bf16.h>

#include "s3_common.cuh"
#include "s3_kernels.cuh"

namespace s3 {

namespace {

constexpr int DT = 128;      // threads per block
constexpr int UNROLL = 4;    // dictionary rows in flight per thread

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void load(const __nv_bfloat16* p, float* out)
    {
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p));
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); out[2 * i] = f.x; out[2 * i + 1] = f.y; }
    }
};
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ static void load(const float* p, float* out)
    {
        const float4 raw = __ldg(reinterpret_cast<const float4*>(p));
        out[0] = raw.x; out[1] = raw.y; out[2] = raw.z; out[3] = raw.w;
    }
};

struct DecodeArgs {
    const void* W_dec;
    const float* b_dec;
    const int32_t* ids;
    const float* vals;
    const void* x;
    float* x_hat;
    float* sqerr;
    long long ld_xhat, ldx;
    int T, k, d_in, d_sae;
};

template <typename T>
__global__ void __launch_bounds__(DT) sae_decode_kernel(const __grid_constant__ DecodeArgs a)
{
    constexpr int N = Vec<T>::N;
    __shared__ int32_t s_id[S3_MAX_K];
    __shared__ float s_val[S3_MAX_K];
    __shared__ float s_red[DT / 32];
    const T* __restrict__ W = static_cast<const T*>(a.W_dec);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int t = blockIdx.x; t < a.T; t += gridDim.x) {
        __syncthreads();                                      // the previous token's pairs are no longer read
        if (tid < a.k) {
            int32_t f = a.ids[(size_t)t * a.k + tid];
            if (f >= a.d_sae) f = -1;                          // never read outside the dictionary
            s_id[tid] = f;
            s_val[tid] = a.vals[(size_t)t * a.k + tid];
        }
        __syncthreads();
        float err = 0.0f;
        for (int c0 = tid * N; c0 < a.d_in; c0 += DT * N) {
            float acc[N];
#pragma unroll
            for (int i = 0; i < N; ++i) acc[i] = 0.0f;
            for (int j0 = 0; j0 < a.k; j0 += UNROLL) {
                float w[UNROLL][N];
                float z[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int j = j0 + u;
                    const int32_t f = j < a.k ? s_id[j] : -1;
                    z[u] = f >= 0 ? s_val[j] : 0.0f;
                    if (f >= 0) Vec<T>::load(W + (size_t)f * a.d_in + c0, w[u]);
                    else {
#pragma unroll
                        for (int i = 0; i < N; ++i) w[u][i] = 0.0f;
                    }
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u)
#pragma unroll
                    for (int i = 0; i < N; ++i) acc[i] = __fmaf_rn(z[u], w[u][i], acc[i]);
            }
#pragma unroll
            for (int i = 0; i < N; ++i) acc[i] = __fadd_rn(acc[i], __ldg(a.b_dec + c0 + i));
            if (a.x_hat) {
                float* out = a.x_hat + (size_t)t * a.ld_xhat + c0;
#pragma unroll
                for (int i = 0; i < N; i += 4) *reinterpret_cast<float4*>(out + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
            }
            if (a.sqerr) {
                float xv[N];
                Vec<T>::load(static_cast<const T*>(a.x) + (size_t)t * a.ldx + c0, xv);
#pragma unroll
                for (int i = 0; i < N; ++i) { const float d = xv[i] - acc[i]; err = __fmaf_rn(d, d, err); }
            }
        }
        if (a.sqerr) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) err += __shfl_xor_sync(0xffffffffu, err, o);
            if (lane == 0) s_red[warp] = err;
            __syncthreads();
            if (tid == 0) {
                float e = 0.0f;
                for (int w = 0; w < DT / 32; ++w) e += s_red[w];
                a.sqerr[t] = e;
            }
        }
    }
}

}  // namespace

s3_status launch_decode(const void* d_W_dec, const float* d_b_dec, int d_in, int d_sae, s3_dtype dtype, const int32_t* d_ids,
                        const float* d_vals, int T, int k, float* d_xhat, int64_t ld_xhat, const void* d_x, int64_t ldx,
                        float* d_sqerr, cudaStream_t stream)
{
    DecodeArgs a;
    a.W_dec = d_W_dec; a.b_dec = d_b_dec; a.ids = d_ids; a.vals = d_vals; a.x = d_x; a.x_hat = d_xhat; a.sqerr = d_sqerr;
    a.ld_xhat = ld_xhat; a.ldx = ldx; a.T = T; a.k = k; a.d_in = d_in; a.d_sae = d_sae;
    const int max_grid = device_sm_count() * 16;
    const int grid = T < max_grid ? T : max_grid;
    if (dtype == S3_BF16) sae_decode_kernel<__nv_bfloat16><<<grid, DT, 0, stream>>>(a);
    else sae_decode_kernel<float><<<grid, DT, 0, stream>>>(a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
