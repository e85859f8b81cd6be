// fp32 SAE encode + ReLU + running Top-k (Sec. 3.3, Eq. 1-2) on the FP32 pipes.
//
// Used for fp32 inputs, where the result must agree with the definition to ~1e-6: every
// pre-activation is an fp32 FMA chain over i = 0..d_in-1 of W_enc[i,f] * (x[t,i] - b_dec[i]),
// then + b_enc[f]. A thread block owns 128 tokens and one slice of the feature columns; it walks the
// slice in 128-column tiles (register-tiled 8x8 outer products from shared memory), drops each
// finished tile into shared memory and lets one thread per token fold it into that token's heap.
// The pre-activation tile never leaves the SM.
#include "s3_topk.cuh"

namespace s3 {

namespace {

constexpr int BM = 128, BN = 128, BK = 16, THREADS = 256, CT_LD = BN + 1;

__global__ void __launch_bounds__(THREADS)
encode_simt_kernel(const float* __restrict__ x, int64_t ldx, const float* __restrict__ W,
                   const float* __restrict__ b_enc, const float* __restrict__ b_dec,
                   int T, int d_in, int d_sae, int k, int n_slices, int n_col_tiles,
                   uint64_t* __restrict__ part)
{
    extern __shared__ __align__(16) unsigned char simt_smem[];
    float* As = reinterpret_cast<float*>(simt_smem);            // [BK][BM]
    float* Bs = As + BK * BM;                                   // [BK][BN]
    float* Ct = Bs + BK * BN;                                   // [BM][CT_LD]
    uint64_t* heap = reinterpret_cast<uint64_t*>(Ct + BM * CT_LD + 1);  // [k][BM], 8-byte aligned below
    heap = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(heap) + 7) & ~uintptr_t(7));

    const int tid = threadIdx.x;
    const int n_mtiles = (T + BM - 1) / BM;
    const int slice = blockIdx.x / n_mtiles, mt = blockIdx.x % n_mtiles;
    const int row0 = mt * BM;
    const int tile_lo = (int)((int64_t)slice * n_col_tiles / n_slices);
    const int tile_hi = (int)((int64_t)(slice + 1) * n_col_tiles / n_slices);
    const int ty = tid >> 4, tx = tid & 15;

    if (tid < BM) heap_init<BM>(heap, tid, k);
    __syncthreads();

    for (int nt = tile_lo; nt < tile_hi; ++nt) {
        const int n0 = nt * BN;
        float acc[8][8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

        for (int k0 = 0; k0 < d_in; k0 += BK) {
            {   // A tile: 128 rows x 16, thread -> (row, 8 consecutive i)
                const int r = tid >> 1, kk0 = (tid & 1) * 8;
                const int t = row0 + r;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int i = k0 + kk0 + q;
                    float v = 0.0f;
                    if (t < T && i < d_in) v = x[(int64_t)t * ldx + i] - b_dec[i];
                    As[(kk0 + q) * BM + r] = v;
                }
            }
            {   // B tile: 16 x 128 columns, thread -> (i, 8 consecutive columns)
                const int kk = tid >> 4, c0 = (tid & 15) * 8;
                const int i = k0 + kk;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int c = n0 + c0 + q;
                    Bs[kk * BN + c0 + q] = (i < d_in && c < d_sae) ? W[(int64_t)i * d_sae + c] : 0.0f;
                }
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < BK; ++kk) {
                float a[8], b[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) a[i] = As[kk * BM + ty * 8 + i];
#pragma unroll
                for (int j = 0; j < 8; ++j) b[j] = Bs[kk * BN + tx * 8 + j];
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(b[j], a[i], acc[i][j]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = n0 + tx * 8 + j;
            const float be = (c < d_sae) ? b_enc[c] : 0.0f;
#pragma unroll
            for (int i = 0; i < 8; ++i) Ct[(ty * 8 + i) * CT_LD + tx * 8 + j] = acc[i][j] + be;
        }
        __syncthreads();
        if (tid < BM) {
            uint64_t root = heap[tid];
            const int ncols = min(BN, d_sae - n0);
            for (int c = 0; c < ncols; ++c) {
                const float v = Ct[tid * CT_LD + c];
                const uint64_t key = make_key(__float_as_uint(v), (uint32_t)(n0 + c));
                if (v > 0.0f && key > root) root = heap_replace_root<BM>(heap, tid, k, key);
            }
        }
        __syncthreads();
    }
    if (tid < BM && row0 + tid < T) {
        uint64_t* dst = part + ((size_t)(row0 + tid) * n_slices + slice) * k;
        for (int j = 0; j < k; ++j) dst[j] = heap[j * BM + tid];
    }
}

}  // namespace

size_t encode_simt_smem_bytes(int k)
{
    return (size_t)(BK * BM + BK * BN + BM * CT_LD + 4) * sizeof(float) + (size_t)k * BM * sizeof(uint64_t) + 16;
}

int encode_simt_col_tiles(int d_sae) { return (d_sae + BN - 1) / BN; }
int encode_simt_row_tiles(int T) { return (T + BM - 1) / BM; }

s3_status launch_encode_simt(const float* d_x, int64_t ldx, const float* d_W, const float* d_b_enc,
                             const float* d_b_dec, int T, int d_in, int d_sae, int k, int n_slices,
                             uint64_t* d_part, cudaStream_t stream)
{
    const size_t smem = encode_simt_smem_bytes(k);
    static bool attr_set[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 64 && !attr_set[dev]) {
        int max_smem = 0;
        S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        S3_CUDA_TRY(cudaFuncSetAttribute(encode_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
        attr_set[dev] = true;
    }
    S3_REQUIRE(smem <= 227u * 1024u, S3_ERR_UNSUPPORTED, "k = %d needs %zu bytes of shared memory per block", k, smem);
    const int grid = n_slices * encode_simt_row_tiles(T);
    encode_simt_kernel<<<grid, THREADS, smem, stream>>>(d_x, ldx, d_W, d_b_enc, d_b_dec, T, d_in, d_sae, k, n_slices,
                                                       encode_simt_col_tiles(d_sae), d_part);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
