// s3_sae_encode_topk_static: the SAE encode + Top-k for callers that cannot hand the library any
// scratch memory of their own.
//
// Some hosts of this library run in places where allocating device memory is off the table: a
// serving loop whose memory pool was sized and frozen at start-up, a plugin that is handed only its
// input and output buffers by the framework around it, or code running while another component
// holds the allocator. The regular entry point wants a caller-allocated workspace for the partial
// Top-k lists that the column slices of the encode exchange with the merge kernel. This variant
// keeps that workspace in a fixed array that is part of the library image itself, so the call
// allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine.
//
// The price: the array has a fixed size (S3_STATIC_SCRATCH_BYTES, held by every GPU that loads the
// library until the process exits), larger requests are refused, and all calls on one device share
// the one array.
#include <mutex>

#include "s3_common.cuh"

namespace {

// The scratch itself. In host code this name is only a handle for the runtime's symbol look-up and
// must never be passed to a kernel; the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[S3_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the current device, looked up once per device.
s3_status static_scratch_address(void** out)
{
    using namespace s3;
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    S3_REQUIRE(dev >= 0 && dev < kMaxDevices, S3_ERR_UNSUPPORTED, "device ordinal %d is beyond the %d supported", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        S3_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        S3_REQUIRE(p != nullptr, S3_ERR_CUDA, "cudaGetSymbolAddress returned a null address for the built-in scratch array");
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return S3_OK;
}

}  // namespace

extern "C" s3_status s3_sae_encode_topk_static(const s3_sae* sae, const void* d_x, int64_t ldx, int T, int k,
                                               int32_t* d_ids, float* d_vals, uint32_t* d_status_out, void* stream)
{
    using namespace s3;
    S3_REQUIRE(sae != nullptr, S3_ERR_INVALID_ARG, "sae is null");
    S3_REQUIRE(T >= 0, S3_ERR_INVALID_ARG, "T = %d is negative", T);
    S3_REQUIRE(k >= 1 && k <= S3_MAX_K, S3_ERR_INVALID_ARG, "k = %d out of range [1, %d]", k, S3_MAX_K);
    const size_t need = s3_sae_encode_workspace_bytes(sae, T, k);
    S3_REQUIRE(need != 0 && need <= static_cast<size_t>(S3_STATIC_SCRATCH_BYTES), S3_ERR_CAPACITY,
               "T = %d tokens at k = %d need %zu bytes of scratch but the built-in array holds %zu; split the call into smaller "
               "token ranges or use s3_sae_encode_topk with a workspace of your own",
               T, k, need, static_cast<size_t>(S3_STATIC_SCRATCH_BYTES));
    void* scratch = nullptr;
    const s3_status st = static_scratch_address(&scratch);
    if (st != S3_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left. The partial lists are fully rewritten for the
    // T tokens of this call; only the status block has to start from zero.
    S3_CUDA_TRY(cudaMemsetAsync(scratch, 0, S3_WS_HEADER_BYTES, cs));
    const s3_status rc = s3_sae_encode_topk(sae, d_x, ldx, T, k, d_ids, d_vals, scratch, S3_STATIC_SCRATCH_BYTES, stream);
    if (rc != S3_OK) return rc;
    if (d_status_out)
        S3_CUDA_TRY(cudaMemcpyAsync(d_status_out, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice, cs));
    return S3_OK;
}
