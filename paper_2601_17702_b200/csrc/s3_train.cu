// One training step of a Top-k SAE on fp32 parameters: gradients of the batch-mean squared reconstruction error
// (Sec. 3.3: x_hat = z_hat W_dec + b_dec) through the Top-k code with the active set fixed, and the Adam update the paper
// trains with (appendix, training configuration). The forward pass is the library's own encode; this file starts from its
// (id, value) pairs.
//
// backward: one block per token (grid-stride). With g = (2/T)(x_hat - x) in shared memory:
//     gz[j]        = W_dec[f_j, :] . g                                   (a warp per selected feature)
//     gW_dec[f_j]  += z_j * g                  gb_enc[f_j] += gz[j]
//     gW_enc[:,f_j]+= gz[j] * (x - b_dec)      gb_dec      += g - sum_j gz[j] W_enc[:, f_j]
//   accumulated with fp32 atomics (the sums over tokens have no fixed order; the tests allow for that). The per-token
//   squared errors go to scratch and are summed by one block in a fixed order.
// adam: elementwise, bias corrections passed in.
#include <cuda_bf16.h>

#include "s3_common.cuh"
#include "s3_kernels.cuh"

namespace s3 {

namespace {

constexpr int TT = 128;      // threads per block

struct BackwardArgs {
    const float* W_enc;      // [d_in, d_sae]
    const float* W_dec;      // [d_sae, d_in]
    const float* b_enc;      // read only when vals is null
    const float* b_dec;
    const float* x;
    const int32_t* ids;
    const float* vals;       // null: z is recomputed in fp32 from the parameters
    float* gW_enc;
    float* gb_enc;
    float* gW_dec;
    float* gb_dec;
    float* sqerr;            // [T] scratch
    long long ldx;
    int T, k, d_in, d_sae;
};

__global__ void __launch_bounds__(TT) sae_backward_kernel(const __grid_constant__ BackwardArgs a)
{
    extern __shared__ float g_s[];                       // [d_in] gradient w.r.t. x_hat, then [d_in] centred input
    float* xc_s = g_s + a.d_in;
    __shared__ int32_t s_id[S3_MAX_K];
    __shared__ float s_z[S3_MAX_K], s_gz[S3_MAX_K];
    __shared__ float s_red[TT / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float scale = 2.0f / static_cast<float>(a.T);
    for (int t = blockIdx.x; t < a.T; t += gridDim.x) {
        __syncthreads();
        if (tid < a.k) {
            int32_t f = a.ids[(size_t)t * a.k + tid];
            if (f >= a.d_sae) f = -1;
            s_id[tid] = f;
            s_z[tid] = (f >= 0 && a.vals) ? a.vals[(size_t)t * a.k + tid] : 0.0f;
        }
        if (a.vals == nullptr) {
            // z[j] = W_enc[:, f_j] . (x - b_dec) + b_enc[f_j] in fp32 (the ids may come from a bf16 forward pass)
            for (int c = tid; c < a.d_in; c += TT) xc_s[c] = a.x[(size_t)t * a.ldx + c] - __ldg(a.b_dec + c);
            __syncthreads();
            for (int j = warp; j < a.k; j += TT / 32) {
                const int32_t f = s_id[j];
                float dot = 0.0f;
                if (f >= 0)
                    for (int c = lane; c < a.d_in; c += 32) dot = __fmaf_rn(__ldg(a.W_enc + (size_t)c * a.d_sae + f), xc_s[c], dot);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                if (lane == 0) s_z[j] = f >= 0 ? dot + __ldg(a.b_enc + f) : 0.0f;
            }
        }
        __syncthreads();
        float err = 0.0f;
        for (int c = tid; c < a.d_in; c += TT) {
            float acc = 0.0f;
            for (int j = 0; j < a.k; ++j) {
                const int32_t f = s_id[j];
                if (f >= 0) acc = __fmaf_rn(s_z[j], __ldg(a.W_dec + (size_t)f * a.d_in + c), acc);
            }
            const float bd = __ldg(a.b_dec + c), xv = a.x[(size_t)t * a.ldx + c];
            const float r = (acc + bd) - xv;
            err = __fmaf_rn(r, r, err);
            g_s[c] = scale * r;
            xc_s[c] = xv - bd;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) err += __shfl_xor_sync(0xffffffffu, err, o);
        if (lane == 0) s_red[warp] = err;
        __syncthreads();
        if (tid == 0) {
            float e = 0.0f;
            for (int w = 0; w < TT / 32; ++w) e += s_red[w];
            a.sqerr[t] = e;
        }
        // gz[j] = W_dec[f_j, :] . g, a warp per selected feature
        for (int j = warp; j < a.k; j += TT / 32) {
            const int32_t f = s_id[j];
            float dot = 0.0f;
            if (f >= 0)
                for (int c = lane; c < a.d_in; c += 32) dot = __fmaf_rn(__ldg(a.W_dec + (size_t)f * a.d_in + c), g_s[c], dot);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            if (lane == 0) s_gz[j] = f >= 0 ? dot : 0.0f;
        }
        __syncthreads();
        for (int c = tid; c < a.d_in; c += TT) {
            const float g = g_s[c], xc = xc_s[c];
            float through_encoder = 0.0f;
            for (int j = 0; j < a.k; ++j) {
                const int32_t f = s_id[j];
                if (f < 0) continue;
                atomicAdd(a.gW_dec + (size_t)f * a.d_in + c, s_z[j] * g);
                atomicAdd(a.gW_enc + (size_t)c * a.d_sae + f, s_gz[j] * xc);
                through_encoder = __fmaf_rn(s_gz[j], __ldg(a.W_enc + (size_t)c * a.d_sae + f), through_encoder);
            }
            atomicAdd(a.gb_dec + c, g - through_encoder);
        }
        if (tid < a.k && s_id[tid] >= 0) atomicAdd(a.gb_enc + s_id[tid], s_gz[tid]);
    }
}

// loss = (1/T) * sum of the per-token squared errors, added in a fixed order by one block
__global__ void __launch_bounds__(1024) sae_loss_kernel(const float* sqerr, int T, float* loss)
{
    __shared__ double part[1024];
    double s = 0.0;
    for (int t = threadIdx.x; t < T; t += 1024) s += static_cast<double>(sqerr[t]);
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = static_cast<float>(part[0] / static_cast<double>(T));
}

__global__ void __launch_bounds__(256) adam_kernel(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v,
                                                   const float* __restrict__ g, size_t n, float lr, float beta1, float beta2,
                                                   float eps, float corr1, float corr2)
{
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (size_t)gridDim.x * 256) {
        const float gi = g[i];
        const float mi = __fmaf_rn(beta1, m[i], (1.0f - beta1) * gi);
        const float vi = __fmaf_rn(beta2, v[i], (1.0f - beta2) * gi * gi);
        m[i] = mi;
        v[i] = vi;
        p[i] -= lr * (mi * corr1) / (sqrtf(vi * corr2) + eps);
    }
}

__global__ void __launch_bounds__(256) cast_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t n)
{
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (size_t)gridDim.x * 256) dst[i] = __float2bfloat16_rn(src[i]);
}

}  // namespace

s3_status launch_cast_bf16(const float* d_src, void* d_dst, size_t n, cudaStream_t stream)
{
    const size_t want = (n + 255) / 256;
    const size_t cap = static_cast<size_t>(device_sm_count()) * 16;
    cast_bf16_kernel<<<static_cast<unsigned>(want < cap ? want : cap), 256, 0, stream>>>(d_src, static_cast<__nv_bfloat16*>(d_dst), n);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

s3_status launch_sae_backward(const float* d_W_enc, const float* d_b_enc, const float* d_W_dec, const float* d_b_dec, const float* d_x, int64_t ldx,
                              const int32_t* d_ids, const float* d_vals, int T, int k, int d_in, int d_sae, float* d_gW_enc,
                              float* d_gb_enc, float* d_gW_dec, float* d_gb_dec, float* d_loss, float* d_sqerr, cudaStream_t stream)
{
    const size_t n_w = static_cast<size_t>(d_in) * d_sae;
    S3_CUDA_TRY(cudaMemsetAsync(d_gW_enc, 0, n_w * 4, stream));
    S3_CUDA_TRY(cudaMemsetAsync(d_gW_dec, 0, n_w * 4, stream));
    S3_CUDA_TRY(cudaMemsetAsync(d_gb_enc, 0, static_cast<size_t>(d_sae) * 4, stream));
    S3_CUDA_TRY(cudaMemsetAsync(d_gb_dec, 0, static_cast<size_t>(d_in) * 4, stream));
    BackwardArgs a;
    a.W_enc = d_W_enc; a.b_enc = d_b_enc; a.W_dec = d_W_dec; a.b_dec = d_b_dec; a.x = d_x; a.ids = d_ids; a.vals = d_vals;
    a.gW_enc = d_gW_enc; a.gb_enc = d_gb_enc; a.gW_dec = d_gW_dec; a.gb_dec = d_gb_dec; a.sqerr = d_sqerr;
    a.ldx = ldx; a.T = T; a.k = k; a.d_in = d_in; a.d_sae = d_sae;
    const int max_grid = device_sm_count() * 16;
    sae_backward_kernel<<<T < max_grid ? T : max_grid, TT, static_cast<size_t>(d_in) * 8, stream>>>(a);
    sae_loss_kernel<<<1, 1024, 0, stream>>>(d_sqerr, T, d_loss);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

s3_status launch_adam(float* d_p, float* d_m, float* d_v, const float* d_g, size_t n, float lr, float beta1, float beta2, float eps,
                      float corr1, float corr2, cudaStream_t stream)
{
    const size_t want = (n + 255) / 256;
    const size_t cap = static_cast<size_t>(device_sm_count()) * 16;
    adam_kernel<<<static_cast<unsigned>(want < cap ? want : cap), 256, 0, stream>>>(d_p, d_m, d_v, d_g, n, lr, beta1, beta2, eps, corr1,
                                                                                  corr2);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
