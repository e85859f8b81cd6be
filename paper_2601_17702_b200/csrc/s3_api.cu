// C ABI of the s3scan library: argument checks, handles and dispatch. All compute is in the kernels.
#include <stdarg.h>
#include <string.h>

#include <new>

#include "s3_kernels.cuh"
#include "s3_topk.cuh"

namespace s3 {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

s3_status fail(s3_status code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int device_sm_count()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    if (dev < 64 && cached[dev]) return cached[dev];
    int n = 1;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 1;
    if (dev < 64) cached[dev] = n;
    return n;
}

int device_cc_major()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return 0;
    return major;
}

}  // namespace s3

using namespace s3;

struct s3_sae {
    const void* d_W;
    const float* d_b_enc;
    const float* d_b_dec;
    int d_in, d_sae;
    s3_dtype dtype;
    int n_slices_override, max_ctas;
    EncodeTcState tc;
};

namespace {

constexpr int kMaxSlices = 16;

int col_tiles(const s3_sae* sae) { return sae->dtype == S3_BF16 ? encode_tc_col_tiles(sae->d_sae) : encode_simt_col_tiles(sae->d_sae); }
int row_tiles(const s3_sae* sae, int T) { return sae->dtype == S3_BF16 ? encode_tc_row_tiles(T) : encode_simt_row_tiles(T); }

// Uniform column slices per row block: the caller's override (s3_sae_set_schedule), clamped to what the kernel takes; for
// the fp32 kernel without an override, enough (row block, slice) thread blocks to cover the SMs. The bf16 launch
// schedules itself when there is no override.
int pick_slices(const s3_sae* sae, int T)
{
    const int nct = col_tiles(sae);
    const int cap = nct < kMaxSlices ? nct : kMaxSlices;
    const int lo = sae->dtype == S3_BF16 ? encode_tc_min_slices(sae->d_sae) : 1;
    if (sae->n_slices_override > 0) {
        const int s = sae->n_slices_override < cap ? sae->n_slices_override : cap;
        return s < lo ? lo : s;
    }
    const int nrt = row_tiles(sae, T);
    int n_sm = device_sm_count();
    if (sae->max_ctas > 0 && sae->max_ctas < n_sm) n_sm = sae->max_ctas;
    const int s = (n_sm + nrt - 1) / nrt;
    return s < lo ? lo : (s > cap ? cap : s);
}

}  // namespace

extern "C" {

const char* s3_last_error(void) { return g_err; }
int s3_version(void) { return 100; }

s3_status s3_workspace_status(const void* d_ws, void* stream, uint32_t* code_out)
{
    S3_REQUIRE(d_ws != nullptr, S3_ERR_INVALID_ARG, "d_ws is null");
    uint32_t code = 0;
    S3_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    S3_CUDA_TRY(cudaMemcpy(&code, d_ws, sizeof(code), cudaMemcpyDeviceToHost));
    if (code_out) *code_out = code;
    if (code == DEV_OK) return S3_OK;
    if (code == DEV_BAD_FEATURE_ID) return fail(S3_ERR_INVALID_ARG, "a feature id >= d_sae was met on the device (code %u)", code);
    if (code == DEV_DUPLICATE_ID) return fail(S3_ERR_INVALID_ARG, "a token carried the same feature id twice (code %u)", code);
    if (code == DEV_COMPACT_CAPACITY) return fail(S3_ERR_CAPACITY, "compact index: block or payload buffer too small (code %u)", code);
    return fail(S3_ERR_TIMEOUT, "a bounded device-side wait ran out (code %u)", code);
}

// ---------------------------------------------------------------------------------------------- SAE
size_t s3_sae_prepared_bytes(int d_in, int d_sae, s3_dtype dtype)
{
    if (d_in < 1 || d_sae < 1) return 0;
    return dtype == S3_BF16 ? encode_tc_prepared_bytes(d_in, d_sae) : 256;
}

s3_status s3_sae_create(s3_sae** out, const void* d_W_enc, const float* d_b_enc, const float* d_b_dec, int d_in,
                        int d_sae, s3_dtype dtype, void* d_prepared, size_t prepared_bytes, void* stream)
{
    S3_REQUIRE(out != nullptr, S3_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    S3_REQUIRE(d_W_enc && d_b_enc && d_b_dec, S3_ERR_INVALID_ARG, "null weight pointer");
    S3_REQUIRE(aligned16(d_W_enc) && aligned16(d_b_enc) && aligned16(d_b_dec), S3_ERR_INVALID_ARG,
               "weight pointers must be 16-byte aligned");
    S3_REQUIRE(dtype == S3_BF16 || dtype == S3_F32, S3_ERR_INVALID_ARG, "unknown dtype %d", (int)dtype);
    S3_REQUIRE(d_in >= 1 && d_sae >= 1, S3_ERR_INVALID_ARG, "d_in = %d, d_sae = %d out of range", d_in, d_sae);
    S3_REQUIRE(d_sae <= 262144, S3_ERR_UNSUPPORTED, "d_sae = %d exceeds 262144", d_sae);
    if (dtype == S3_BF16) {
        S3_REQUIRE(d_in % 8 == 0 && d_sae % 8 == 0, S3_ERR_UNSUPPORTED,
                   "bf16 encode needs d_in and d_sae to be multiples of 8 (got %d, %d)", d_in, d_sae);
        S3_REQUIRE(d_prepared != nullptr && aligned16(d_prepared), S3_ERR_INVALID_ARG, "d_prepared is null or misaligned");
        S3_REQUIRE(prepared_bytes >= encode_tc_prepared_bytes(d_in, d_sae), S3_ERR_CAPACITY,
                   "d_prepared holds %zu bytes, %zu needed", prepared_bytes, encode_tc_prepared_bytes(d_in, d_sae));
    }
    int n_dev = 0;
    S3_CUDA_TRY(cudaGetDeviceCount(&n_dev));
    S3_REQUIRE(device_cc_major() == 10, S3_ERR_UNSUPPORTED, "this library runs on sm_100 devices only (found compute capability %d.x)",
               device_cc_major());
    s3_sae* sae = new (std::nothrow) s3_sae();
    S3_REQUIRE(sae != nullptr, S3_ERR_NOMEM, "out of host memory");
    sae->d_W = d_W_enc; sae->d_b_enc = d_b_enc; sae->d_b_dec = d_b_dec;
    sae->d_in = d_in; sae->d_sae = d_sae; sae->dtype = dtype;
    sae->n_slices_override = 0; sae->max_ctas = 0;
    if (dtype == S3_BF16) {
        const s3_status st = encode_tc_prepare(&sae->tc, d_W_enc, d_b_enc, d_b_dec, d_in, d_sae, d_prepared,
                                               static_cast<cudaStream_t>(stream));
        if (st != S3_OK) { delete sae; return st; }
    }
    *out = sae;
    return S3_OK;
}

s3_status s3_sae_destroy(s3_sae* sae)
{
    delete sae;
    return S3_OK;
}

s3_status s3_sae_set_schedule(s3_sae* sae, int n_slices, int max_ctas)
{
    S3_REQUIRE(sae != nullptr, S3_ERR_INVALID_ARG, "sae is null");
    S3_REQUIRE(n_slices >= 0 && n_slices <= kMaxSlices && max_ctas >= 0, S3_ERR_INVALID_ARG,
               "n_slices must be in [0, %d] and max_ctas >= 0", kMaxSlices);
    sae->n_slices_override = n_slices;
    sae->max_ctas = max_ctas;
    return S3_OK;
}

size_t s3_sae_encode_workspace_bytes(const s3_sae* sae, int T_max, int k)
{
    if (!sae || T_max < 0 || k < 1 || k > S3_MAX_K) return 0;
    const int nct = col_tiles(sae);
    const int smax = nct < kMaxSlices ? nct : kMaxSlices;
    if (sae->dtype == S3_BF16) return S3_WS_HEADER_BYTES + 192 + encode_tc_workspace_bytes(T_max, smax, k);
    return S3_WS_HEADER_BYTES + (size_t)T_max * smax * k * sizeof(uint64_t);
}

s3_status s3_sae_encode_topk(const s3_sae* sae, const void* d_x, int64_t ldx, int T, int k, int32_t* d_ids, float* d_vals,
                             void* d_ws, size_t ws_bytes, void* stream)
{
    S3_REQUIRE(sae != nullptr, S3_ERR_INVALID_ARG, "sae is null");
    S3_REQUIRE(T >= 0, S3_ERR_INVALID_ARG, "T = %d is negative", T);
    S3_REQUIRE(k >= 1 && k <= sae->d_sae, S3_ERR_INVALID_ARG, "k = %d out of range [1, d_sae = %d]", k, sae->d_sae);
    S3_REQUIRE(k <= S3_MAX_K, S3_ERR_UNSUPPORTED, "k = %d exceeds the supported maximum %d", k, S3_MAX_K);
    if (T == 0) return S3_OK;
    S3_REQUIRE(d_x && d_ids && d_vals && d_ws, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(aligned16(d_x) && aligned16(d_ws) && (reinterpret_cast<uintptr_t>(d_ids) & 3) == 0 &&
                   (reinterpret_cast<uintptr_t>(d_vals) & 3) == 0,
               S3_ERR_INVALID_ARG, "misaligned device pointer");
    S3_REQUIRE(ldx >= sae->d_in, S3_ERR_INVALID_ARG, "ldx = %lld is smaller than d_in = %d", (long long)ldx, sae->d_in);
    if (sae->dtype == S3_BF16) S3_REQUIRE(ldx % 8 == 0, S3_ERR_INVALID_ARG, "ldx = %lld must be a multiple of 8 for bf16", (long long)ldx);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t* status = static_cast<uint32_t*>(d_ws);
    if (sae->dtype == S3_BF16) {
        // column slices: the caller's override, else the launch's own schedule
        const int forced = sae->n_slices_override > 0 ? pick_slices(sae, T) : 0;
        const EncodeTcItem it = {&sae->tc, d_x, ldx, T, sae->d_in, sae->d_sae, k, forced, d_ids, d_vals};
        const size_t need = S3_WS_HEADER_BYTES + 192 + encode_tc_group_workspace_need(&it, 1, sae->max_ctas);
        S3_REQUIRE(ws_bytes >= need, S3_ERR_CAPACITY, "workspace holds %zu bytes, %zu needed", ws_bytes, need);
        return launch_encode_tc(&sae->tc, d_x, ldx, T, sae->d_in, sae->d_sae, k, forced, sae->max_ctas,
                                static_cast<unsigned char*>(d_ws) + 256, status, d_ids, d_vals, st);
    }
    const int n_slices = pick_slices(sae, T);
    const size_t need = S3_WS_HEADER_BYTES + (size_t)T * n_slices * k * sizeof(uint64_t);
    S3_REQUIRE(ws_bytes >= need, S3_ERR_CAPACITY, "workspace holds %zu bytes, %zu needed", ws_bytes, need);
    uint64_t* part = reinterpret_cast<uint64_t*>(static_cast<unsigned char*>(d_ws) + S3_WS_HEADER_BYTES);
    const s3_status rc = launch_encode_simt(static_cast<const float*>(d_x), ldx, static_cast<const float*>(sae->d_W), sae->d_b_enc,
                                            sae->d_b_dec, T, sae->d_in, sae->d_sae, k, n_slices, part, st);
    if (rc != S3_OK) return rc;
    launch_topk_merge(part, T, n_slices, k, d_ids, d_vals, st);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

static s3_status check_encode_item(const s3_encode_item& it, int idx)
{
    S3_REQUIRE(it.sae != nullptr, S3_ERR_INVALID_ARG, "item %d: sae is null", idx);
    S3_REQUIRE(it.sae->dtype == S3_BF16, S3_ERR_UNSUPPORTED, "item %d: the grouped launch takes bf16 encoders only", idx);
    S3_REQUIRE(it.T >= 0, S3_ERR_INVALID_ARG, "item %d: T = %d is negative", idx, it.T);
    S3_REQUIRE(it.k >= 1 && it.k <= it.sae->d_sae, S3_ERR_INVALID_ARG, "item %d: k = %d out of range [1, d_sae = %d]", idx, it.k,
               it.sae->d_sae);
    S3_REQUIRE(it.k <= S3_MAX_K, S3_ERR_UNSUPPORTED, "item %d: k = %d exceeds the supported maximum %d", idx, it.k, S3_MAX_K);
    if (it.T == 0) return S3_OK;
    S3_REQUIRE(it.d_x && it.d_ids && it.d_vals, S3_ERR_INVALID_ARG, "item %d: null device pointer", idx);
    S3_REQUIRE(aligned16(it.d_x) && (reinterpret_cast<uintptr_t>(it.d_ids) & 3) == 0 && (reinterpret_cast<uintptr_t>(it.d_vals) & 3) == 0,
               S3_ERR_INVALID_ARG, "item %d: misaligned device pointer", idx);
    S3_REQUIRE(it.ldx >= it.sae->d_in && it.ldx % 8 == 0, S3_ERR_INVALID_ARG, "item %d: ldx = %lld must be a multiple of 8 and >= d_in",
               idx, (long long)it.ldx);
    return S3_OK;
}

size_t s3_sae_encode_grouped_workspace_bytes(const s3_encode_item* h_items, int n_items)
{
    if (!h_items || n_items < 0) return 0;
    size_t n = 256;
    for (int i = 0; i < n_items; ++i) {
        const s3_encode_item& it = h_items[i];
        if (!it.sae || it.sae->dtype != S3_BF16 || it.T <= 0 || it.k < 1) continue;
        // a caller's slice override counts as given; otherwise the bound that holds whatever schedule the launch picks
        n += it.sae->n_slices_override > 0 ? encode_tc_workspace_bytes(it.T, pick_slices(it.sae, it.T), it.k)
                                           : encode_tc_workspace_bound(it.T, it.k);
    }
    return n;
}

int s3_sae_encode_ctas(const s3_sae* sae, int T)
{
    if (!sae || T <= 0) return 0;
    if (sae->dtype != S3_BF16) return device_sm_count();
    const EncodeTcItem it = {&sae->tc, nullptr, 0, T, sae->d_in, sae->d_sae, 1, sae->n_slices_override > 0 ? pick_slices(sae, T) : 0,
                             nullptr, nullptr};
    return encode_tc_group_ctas(&it, 1, sae->max_ctas);
}

int s3_encode_schedule_describe(const int32_t* T, const int32_t* d_in, const int32_t* d_sae, const int32_t* k, int n_items,
                                int n_pairs, int32_t* h_units, int max_units, int32_t* h_slots)
{
    if (!T || !d_in || !d_sae || !k || !h_slots || n_items < 1 || n_items > S3_MAX_ENCODE_ITEMS || n_pairs < 1 || max_units < 0 ||
        (max_units > 0 && !h_units))
        return -2;
    EncodeTcItem items[S3_MAX_ENCODE_ITEMS];
    for (int i = 0; i < n_items; ++i) {
        if (T[i] < 1 || d_in[i] < 1 || d_sae[i] < 1 || k[i] < 1) return -2;
        items[i] = EncodeTcItem{nullptr, nullptr, 0, T[i], d_in[i], d_sae[i], k[i], 0, nullptr, nullptr};
    }
    return encode_tc_describe_schedule(items, n_items, n_pairs, h_units, max_units, h_slots);
}

s3_status s3_sae_encode_topk_grouped(const s3_encode_item* h_items, int n_items, int max_ctas_arg, void* d_ws, size_t ws_bytes,
                                     void* stream)
{
    S3_REQUIRE(max_ctas_arg >= 0, S3_ERR_INVALID_ARG, "max_ctas is negative");
    S3_REQUIRE(n_items >= 0, S3_ERR_INVALID_ARG, "n_items is negative");
    if (n_items == 0) return S3_OK;
    S3_REQUIRE(h_items != nullptr, S3_ERR_INVALID_ARG, "h_items is null");
    S3_REQUIRE(n_items <= S3_MAX_ENCODE_ITEMS, S3_ERR_UNSUPPORTED, "n_items = %d exceeds %d", n_items, S3_MAX_ENCODE_ITEMS);
    S3_REQUIRE(d_ws != nullptr && aligned16(d_ws), S3_ERR_INVALID_ARG, "d_ws is null or misaligned");
    EncodeTcItem items[S3_MAX_ENCODE_ITEMS];
    int n = 0, max_ctas = max_ctas_arg;
    for (int i = 0; i < n_items; ++i) {
        const s3_status st = check_encode_item(h_items[i], i);
        if (st != S3_OK) return st;
        const s3_encode_item& it = h_items[i];
        if (it.T == 0) continue;
        items[n++] = EncodeTcItem{&it.sae->tc, it.d_x, it.ldx, it.T, it.sae->d_in, it.sae->d_sae, it.k,
                                  it.sae->n_slices_override > 0 ? pick_slices(it.sae, it.T) : 0, it.d_ids, it.d_vals};
        if (it.sae->max_ctas > 0 && (max_ctas == 0 || it.sae->max_ctas < max_ctas)) max_ctas = it.sae->max_ctas;
    }
    if (n == 0) return S3_OK;
    const size_t need = 256 + encode_tc_group_workspace_need(items, n, max_ctas);
    S3_REQUIRE(ws_bytes >= need, S3_ERR_CAPACITY, "workspace holds %zu bytes, %zu needed", ws_bytes, need);
    return launch_encode_tc_group(items, n, max_ctas, static_cast<unsigned char*>(d_ws) + 256, static_cast<uint32_t*>(d_ws),
                                  static_cast<cudaStream_t>(stream));
}

size_t s3_sae_project_encode_workspace_bytes(const s3_sae* sae, int T_max, int n_heads, int k)
{
    if (!sae || T_max < 0 || n_heads < 1 || k < 1 || sae->dtype != S3_BF16) return 0;
    return 256 + encode_proj_tc_workspace_bytes(T_max, n_heads, k);
}

s3_status s3_sae_project_encode_topk(const s3_sae* proj, const s3_sae* sae, const void* d_h, int64_t ldh, int T, int n_heads, int k,
                                     int32_t* d_ids, float* d_vals, void* d_ws, size_t ws_bytes, void* stream)
{
    S3_REQUIRE(proj != nullptr && sae != nullptr, S3_ERR_INVALID_ARG, "null handle");
    S3_REQUIRE(proj->dtype == S3_BF16 && sae->dtype == S3_BF16, S3_ERR_UNSUPPORTED, "bf16 projection and encoder only");
    S3_REQUIRE(sae->d_in == 128, S3_ERR_UNSUPPORTED, "the per-head encoder must read d_head = 128 values, not %d", sae->d_in);
    S3_REQUIRE(n_heads >= 1 && proj->d_sae == n_heads * 128, S3_ERR_INVALID_ARG, "the projection yields %d columns, %d heads of 128 expected",
               proj->d_sae, n_heads);
    S3_REQUIRE(T >= 0, S3_ERR_INVALID_ARG, "T = %d is negative", T);
    S3_REQUIRE(k >= 1 && k <= sae->d_sae, S3_ERR_INVALID_ARG, "k = %d out of range [1, d_sae = %d]", k, sae->d_sae);
    S3_REQUIRE(k <= S3_MAX_K, S3_ERR_UNSUPPORTED, "k = %d exceeds the supported maximum %d", k, S3_MAX_K);
    S3_REQUIRE(static_cast<int64_t>(T) * n_heads <= INT32_MAX, S3_ERR_UNSUPPORTED, "T * n_heads exceeds 2^31");
    if (T == 0) return S3_OK;
    S3_REQUIRE(d_h && d_ids && d_vals && d_ws, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(aligned16(d_h) && aligned16(d_ws), S3_ERR_INVALID_ARG, "misaligned device pointer");
    S3_REQUIRE(ldh >= proj->d_in && ldh % 8 == 0, S3_ERR_INVALID_ARG, "ldh = %lld must be a multiple of 8 and >= d_model", (long long)ldh);
    const size_t need = s3_sae_project_encode_workspace_bytes(sae, T, n_heads, k);
    S3_REQUIRE(ws_bytes >= need, S3_ERR_CAPACITY, "workspace holds %zu bytes, %zu needed", ws_bytes, need);
    return launch_encode_proj_tc(&proj->tc, &sae->tc, d_h, ldh, T, proj->d_in, n_heads, sae->d_sae, k, sae->max_ctas,
                                 static_cast<unsigned char*>(d_ws) + 256, static_cast<uint32_t*>(d_ws), d_ids, d_vals,
                                 static_cast<cudaStream_t>(stream));
}

s3_status s3_sae_preact(const s3_sae* sae, const void* d_x, int64_t ldx, int T, void* d_out, int64_t ld_out, s3_dtype out_dtype,
                        void* d_ws, size_t ws_bytes, void* stream)
{
    S3_REQUIRE(sae != nullptr, S3_ERR_INVALID_ARG, "sae is null");
    S3_REQUIRE(sae->dtype == S3_BF16, S3_ERR_UNSUPPORTED, "dense pre-activations are built for bf16 encoders only");
    S3_REQUIRE(out_dtype == S3_BF16 || out_dtype == S3_F32, S3_ERR_INVALID_ARG, "unknown output dtype %d", (int)out_dtype);
    S3_REQUIRE(T >= 0, S3_ERR_INVALID_ARG, "T = %d is negative", T);
    if (T == 0) return S3_OK;
    S3_REQUIRE(d_x && d_out && d_ws, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(ws_bytes >= S3_WS_HEADER_BYTES, S3_ERR_CAPACITY, "workspace smaller than %d bytes", S3_WS_HEADER_BYTES);
    S3_REQUIRE(aligned16(d_x) && aligned16(d_out), S3_ERR_INVALID_ARG, "misaligned device pointer");
    S3_REQUIRE(ldx >= sae->d_in && ldx % 8 == 0, S3_ERR_INVALID_ARG, "ldx = %lld must be a multiple of 8 and >= d_in", (long long)ldx);
    const int vec = out_dtype == S3_BF16 ? 8 : 4;
    S3_REQUIRE(ld_out >= sae->d_sae && ld_out % vec == 0, S3_ERR_INVALID_ARG, "ld_out = %lld must be a multiple of %d and >= d_sae",
               (long long)ld_out, vec);
    return launch_preact_tc(&sae->tc, d_x, ldx, T, sae->d_in, sae->d_sae, sae->n_slices_override > 0 ? pick_slices(sae, T) : 0, sae->max_ctas,
                            static_cast<uint32_t*>(d_ws), d_out, ld_out, out_dtype == S3_BF16, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- postings
size_t s3_postings_workspace_bytes(int T_max, int k, int d_sae)
{
    return 256 + postings_workspace_bytes(T_max, k, d_sae);
}

static s3_status check_item(const s3_postings_item& it, int idx)
{
    S3_REQUIRE(it.T >= 0 && it.k >= 1 && it.d_sae >= 1, S3_ERR_INVALID_ARG, "item %d: T = %d, k = %d, d_sae = %d out of range", idx, it.T,
               it.k, it.d_sae);
    S3_REQUIRE(it.d_sae <= (1 << 20), S3_ERR_UNSUPPORTED, "item %d: d_sae = %d exceeds 2^20", idx, it.d_sae);
    S3_REQUIRE(it.k <= 4096, S3_ERR_UNSUPPORTED, "item %d: k = %d exceeds 4096", idx, it.k);
    S3_REQUIRE((int64_t)it.T * it.k <= (1ll << 27), S3_ERR_UNSUPPORTED, "item %d: T*k = %lld exceeds 2^27", idx,
               (long long)it.T * it.k);
    S3_REQUIRE(it.d_row_ptr != nullptr, S3_ERR_INVALID_ARG, "item %d: d_row_ptr is null", idx);
    S3_REQUIRE(it.T == 0 || (it.d_ids && it.d_pos), S3_ERR_INVALID_ARG, "item %d: null device pointer", idx);
    S3_REQUIRE((it.d_vals == nullptr) == (it.d_pval == nullptr), S3_ERR_INVALID_ARG,
               "item %d: d_vals and d_pval must be both null or both non-null", idx);
    S3_REQUIRE(it.pos_base >= 0, S3_ERR_INVALID_ARG, "item %d: pos_base is negative", idx);
    S3_REQUIRE(it.pos_base + it.T <= INT32_MAX, S3_ERR_CAPACITY, "item %d: positions beyond int32 (pos_base %lld + T %d)", idx,
               (long long)it.pos_base, it.T);
    return S3_OK;
}

s3_status s3_postings_build_batched(const s3_postings_item* h_items, int n_items, void* d_ws, size_t ws_bytes, void* stream)
{
    S3_REQUIRE(n_items >= 0, S3_ERR_INVALID_ARG, "n_items is negative");
    if (n_items == 0) return S3_OK;
    S3_REQUIRE(h_items != nullptr, S3_ERR_INVALID_ARG, "h_items is null");
    S3_REQUIRE(n_items <= S3_MAX_POSTINGS_ITEMS, S3_ERR_UNSUPPORTED, "n_items = %d exceeds %d", n_items, S3_MAX_POSTINGS_ITEMS);
    S3_REQUIRE(d_ws != nullptr && ws_bytes >= S3_WS_HEADER_BYTES, S3_ERR_CAPACITY, "workspace missing or smaller than %d bytes",
               S3_WS_HEADER_BYTES);
    for (int i = 0; i < n_items; ++i) {
        const s3_status st = check_item(h_items[i], i);
        if (st != S3_OK) return st;
    }
    return launch_postings(h_items, n_items, d_ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

s3_status s3_postings_build(const int32_t* d_ids, const float* d_vals, int T, int k, int d_sae, int64_t pos_base,
                            uint32_t* d_row_ptr, int32_t* d_pos, float* d_pval, void* d_ws, size_t ws_bytes, void* stream)
{
    s3_postings_item it;
    it.d_ids = d_ids; it.d_vals = d_vals; it.T = T; it.k = k; it.d_sae = d_sae; it.reserved = 0;
    it.pos_base = pos_base; it.d_row_ptr = d_row_ptr; it.d_pos = d_pos; it.d_pval = d_pval;
    return s3_postings_build_batched(&it, 1, d_ws, ws_bytes, stream);
}

// ---------------------------------------------------------------------------------------------- scoring
size_t s3_score_workspace_bytes(int Q, int nq, int k, int n_layers, int n_spans, int s)
{
    (void)nq; (void)k; (void)n_layers; (void)s;
    return 256 + score_workspace_bytes(Q, n_spans);
}

}  // extern "C"

namespace {

// Argument checks shared by the two scoring entry points; *n_spans_out receives the span count.
s3_status check_score_args(const void* h_layers, int n_layers, int d_sae, int64_t L, const int32_t* d_q_ids, const float* d_q_vals,
                           int Q, int nq, int k, const s3_score_params* p, const float* d_bm25, int64_t ld_bm25,
                           const int32_t* d_top_idx, const float* d_top_score, const void* d_ws, size_t ws_bytes, int64_t* n_spans_out)
{
    S3_REQUIRE(h_layers && p, S3_ERR_INVALID_ARG, "null argument");
    S3_REQUIRE(n_layers >= 1 && n_layers <= S3_MAX_SCORE_LAYERS, S3_ERR_UNSUPPORTED, "n_layers = %d out of [1, %d]", n_layers,
               S3_MAX_SCORE_LAYERS);
    S3_REQUIRE(d_sae >= 1 && d_sae <= (1 << 20), S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    S3_REQUIRE(L >= 0 && L <= INT32_MAX, S3_ERR_INVALID_ARG, "L out of range");
    S3_REQUIRE(Q >= 0 && nq >= 1 && k >= 1, S3_ERR_INVALID_ARG, "Q = %d, nq = %d, k = %d out of range", Q, nq, k);
    S3_REQUIRE((int64_t)nq * k <= 4096, S3_ERR_UNSUPPORTED, "nq*k = %lld exceeds 4096", (long long)nq * k);
    S3_REQUIRE(p->width >= 1 && p->stride >= 1, S3_ERR_INVALID_ARG, "width = %d, stride = %d must be >= 1", p->width, p->stride);
    S3_REQUIRE(p->mode == S3_SCORE_MINCOUNT || p->mode == S3_SCORE_WEIGHTED, S3_ERR_INVALID_ARG, "unknown mode %d", p->mode);
    S3_REQUIRE(p->s >= 1 && p->s <= 64, S3_ERR_UNSUPPORTED, "s = %d out of [1, 64]", p->s);
    const int64_t n_spans = (L >= p->width) ? (L - p->width) / p->stride + 1 : 0;
    S3_REQUIRE(n_spans <= 16384, S3_ERR_UNSUPPORTED, "n_spans = %lld exceeds 16384", (long long)n_spans);
    *n_spans_out = n_spans;
    if (Q == 0) return S3_OK;
    S3_REQUIRE(d_q_ids && d_q_vals && d_top_idx && d_top_score, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(d_ws != nullptr && ws_bytes >= S3_WS_HEADER_BYTES, S3_ERR_CAPACITY, "workspace missing or smaller than %d bytes",
               S3_WS_HEADER_BYTES);
    S3_REQUIRE(d_bm25 == nullptr || ld_bm25 >= n_spans, S3_ERR_INVALID_ARG, "ld_bm25 smaller than n_spans");
    return S3_OK;
}

}  // namespace

extern "C" {

s3_status s3_coactivation_score_topspans(const s3_csr_view* h_layers, int n_layers, int d_sae, int64_t L,
                                         const int32_t* d_q_ids, const float* d_q_vals, int Q, int nq, int k,
                                         const s3_score_params* p, const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx,
                                         float* d_top_score, float* d_all_scores, void* d_ws, size_t ws_bytes, void* stream)
{
    int64_t n_spans = 0;
    const s3_status st = check_score_args(h_layers, n_layers, d_sae, L, d_q_ids, d_q_vals, Q, nq, k, p, d_bm25, ld_bm25, d_top_idx,
                                          d_top_score, d_ws, ws_bytes, &n_spans);
    if (st != S3_OK || Q == 0) return st;
    for (int l = 0; l < n_layers; ++l)
        S3_REQUIRE(h_layers[l].d_row_ptr && (h_layers[l].d_pos || n_spans == 0), S3_ERR_INVALID_ARG, "layer %d: null CSR pointer", l);
    return launch_score(h_layers, n_layers, d_sae, d_q_ids, d_q_vals, Q, nq, k, (int)n_spans, p, d_bm25, ld_bm25, d_top_idx,
                        d_top_score, d_all_scores, d_ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

s3_status s3_coactivation_score_topspans_compact(const s3_compact_view* h_layers, int n_layers, int d_sae, int64_t L,
                                                 const int32_t* d_q_ids, const float* d_q_vals, int Q, int nq, int k,
                                                 const s3_score_params* p, const float* d_bm25, int64_t ld_bm25,
                                                 int32_t* d_top_idx, float* d_top_score, float* d_all_scores, void* d_ws,
                                                 size_t ws_bytes, void* stream)
{
    int64_t n_spans = 0;
    const s3_status st = check_score_args(h_layers, n_layers, d_sae, L, d_q_ids, d_q_vals, Q, nq, k, p, d_bm25, ld_bm25, d_top_idx,
                                          d_top_score, d_ws, ws_bytes, &n_spans);
    if (st != S3_OK || Q == 0) return st;
    for (int l = 0; l < n_layers; ++l)
        S3_REQUIRE(h_layers[l].d_row_ptr && h_layers[l].d_blk_ptr && h_layers[l].d_blk_first && h_layers[l].d_blk_desc &&
                       h_layers[l].d_payload,
                   S3_ERR_INVALID_ARG, "layer %d: null pointer in the compact view", l);
    return launch_score_compact(h_layers, n_layers, d_sae, d_q_ids, d_q_vals, Q, nq, k, (int)n_spans, p, d_bm25, ld_bm25,
                                d_top_idx, d_top_score, d_all_scores, d_ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- compact index
s3_status s3_compact_bound(uint64_t n_postings, int d_sae, uint64_t* max_blocks, uint64_t* max_words)
{
    S3_REQUIRE(max_blocks && max_words, S3_ERR_INVALID_ARG, "null output pointer");
    S3_REQUIRE(d_sae >= 1 && d_sae <= (1 << 20), S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    S3_REQUIRE(n_postings <= (1ull << 36), S3_ERR_UNSUPPORTED, "more than 2^36 postings in one layer");
    compact_bound(n_postings, d_sae, max_blocks, max_words);
    return S3_OK;
}

size_t s3_compact_workspace_bytes(uint64_t n_postings, int d_sae)
{
    if (d_sae < 1 || d_sae > (1 << 20) || n_postings > (1ull << 36)) return 0;
    return 256 + compact_workspace_bytes(n_postings, d_sae);
}

s3_status s3_compact_build(const uint64_t* d_row_ptr, const int32_t* d_pos, uint64_t n_postings, int d_sae, int64_t stop_freq,
                           uint64_t* d_out_row_ptr, uint32_t* d_blk_ptr, int32_t* d_blk_first, uint64_t* d_blk_desc,
                           uint64_t cap_blocks, uint32_t* d_payload, uint64_t cap_words, uint64_t* d_sizes, void* d_ws,
                           size_t ws_bytes, void* stream)
{
    S3_REQUIRE(d_sae >= 1 && d_sae <= (1 << 20), S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    S3_REQUIRE(n_postings <= (1ull << 36), S3_ERR_UNSUPPORTED, "more than 2^36 postings in one layer");
    S3_REQUIRE(stop_freq >= 0, S3_ERR_INVALID_ARG, "stop_freq must not be negative");
    S3_REQUIRE(d_row_ptr && (d_pos || n_postings == 0) && d_out_row_ptr && d_blk_ptr && d_sizes, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE((d_blk_first && d_blk_desc) || cap_blocks == 0, S3_ERR_INVALID_ARG, "null block arrays");
    S3_REQUIRE(d_payload != nullptr && cap_words >= 1, S3_ERR_CAPACITY, "the payload needs at least its closing word");
    uint64_t need_blocks, need_words;
    compact_bound(n_postings, d_sae, &need_blocks, &need_words);
    const uint64_t scratch_blocks = cap_blocks < need_blocks ? cap_blocks : need_blocks;
    S3_REQUIRE(d_ws != nullptr && ws_bytes >= 256 + (scratch_blocks + 1) * 8, S3_ERR_CAPACITY, "workspace holds %zu bytes, %zu needed",
               ws_bytes, static_cast<size_t>(256 + (scratch_blocks + 1) * 8));
    return launch_compact_build(d_row_ptr, d_pos, d_sae, stop_freq, d_out_row_ptr, d_blk_ptr, d_blk_first, d_blk_desc, scratch_blocks,
                                d_payload, cap_words, d_sizes, static_cast<uint32_t*>(d_ws),
                                static_cast<unsigned char*>(d_ws) + 256, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- density
size_t s3_density_workspace_bytes(int Q, int64_t L, int n_layers, int d_sae, int nq, int k)
{
    if (Q < 0 || L < 0 || n_layers < 1 || d_sae < 1 || nq < 1 || k < 1) return 0;
    return 256 + density_workspace_bytes(Q, L, n_layers, d_sae, nq, k);
}

s3_status s3_position_density_topcenters(const s3_csr_view* h_layers, int n_layers, int d_sae, int64_t L,
                                         const int32_t* d_q_ids, const float* d_q_vals, int Q, int nq, int k,
                                         const s3_density_params* p, int32_t* d_centers, float* d_center_density, float* d_S,
                                         float* d_density, void* d_ws, size_t ws_bytes, void* stream)
{
    S3_REQUIRE(h_layers && p, S3_ERR_INVALID_ARG, "null argument");
    S3_REQUIRE(n_layers >= 1 && n_layers <= S3_MAX_SCORE_LAYERS, S3_ERR_UNSUPPORTED, "n_layers = %d out of [1, %d]", n_layers,
               S3_MAX_SCORE_LAYERS);
    S3_REQUIRE(d_sae >= 1 && d_sae <= (1 << 20), S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    S3_REQUIRE(L >= 0, S3_ERR_INVALID_ARG, "L is negative");
    S3_REQUIRE(L <= 4194304, S3_ERR_UNSUPPORTED, "L = %lld exceeds 4194304", (long long)L);
    S3_REQUIRE(Q >= 0 && nq >= 1 && k >= 1, S3_ERR_INVALID_ARG, "Q = %d, nq = %d, k = %d out of range", Q, nq, k);
    S3_REQUIRE((int64_t)nq * k <= 4096, S3_ERR_UNSUPPORTED, "nq*k = %lld exceeds 4096", (long long)nq * k);
    S3_REQUIRE(p->conv_kernel >= 1 && p->nms_radius >= 0 && p->n_centers >= 1, S3_ERR_INVALID_ARG,
               "conv_kernel = %d, nms_radius = %d, n_centers = %d out of range", p->conv_kernel, p->nms_radius, p->n_centers);
    S3_REQUIRE(p->conv_kernel <= 1024 && p->n_centers <= 1024, S3_ERR_UNSUPPORTED, "conv_kernel and n_centers may not exceed 1024");
    if (Q == 0) return S3_OK;
    S3_REQUIRE(d_q_ids && d_q_vals && d_centers && d_center_density, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(d_ws != nullptr && ws_bytes >= s3_density_workspace_bytes(Q, L, n_layers, d_sae, nq, k), S3_ERR_CAPACITY,
               "workspace holds %zu bytes, %zu needed", ws_bytes, s3_density_workspace_bytes(Q, L, n_layers, d_sae, nq, k));
    for (int l = 0; l < n_layers; ++l)
        S3_REQUIRE(h_layers[l].d_row_ptr && h_layers[l].d_pos, S3_ERR_INVALID_ARG, "layer %d: null CSR pointer", l);
    return launch_density(h_layers, n_layers, d_sae, L, d_q_ids, d_q_vals, Q, nq, k, p->conv_kernel, p->nms_radius, p->n_centers,
                          p->stop_freq, d_centers, d_center_density, d_S, d_density, static_cast<unsigned char*>(d_ws) + 256,
                          static_cast<cudaStream_t>(stream));
}

s3_status s3_compact_expand(const s3_compact_view* h_view, int d_sae, int32_t* d_pos, uint64_t cap_postings, void* d_ws,
                            size_t ws_bytes, void* stream)
{
    S3_REQUIRE(h_view != nullptr, S3_ERR_INVALID_ARG, "h_view is null");
    S3_REQUIRE(d_sae >= 1 && d_sae <= (1 << 20), S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    S3_REQUIRE(h_view->d_row_ptr && h_view->d_blk_ptr && h_view->d_payload, S3_ERR_INVALID_ARG, "null pointer in the compact view");
    S3_REQUIRE(d_pos != nullptr || cap_postings == 0, S3_ERR_INVALID_ARG, "d_pos is null");
    S3_REQUIRE(d_ws != nullptr && ws_bytes >= S3_WS_HEADER_BYTES, S3_ERR_CAPACITY, "workspace missing or smaller than %d bytes",
               S3_WS_HEADER_BYTES);
    return launch_compact_expand(*h_view, d_sae, d_pos, cap_postings, static_cast<uint32_t*>(d_ws), static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- head aggregation
s3_status s3_head_aggregate_topk(const int32_t* d_ids, const float* d_vals, int T, int H, int k, int d_sae, int k_out,
                                 int32_t* d_out_ids, float* d_out_vals, void* stream)
{
    S3_REQUIRE(T >= 0 && H >= 1 && k >= 1 && k_out >= 1, S3_ERR_INVALID_ARG, "T = %d, H = %d, k = %d, k_out = %d out of range", T, H, k,
               k_out);
    S3_REQUIRE((int64_t)H * k <= 4096, S3_ERR_UNSUPPORTED, "H*k = %lld exceeds 4096", (long long)H * k);
    S3_REQUIRE(k_out <= 4096, S3_ERR_UNSUPPORTED, "k_out = %d exceeds 4096", k_out);
    S3_REQUIRE(d_sae >= 1 && d_sae <= (1 << 20), S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    if (T == 0) return S3_OK;
    S3_REQUIRE(d_ids && d_vals && d_out_ids && d_out_vals, S3_ERR_INVALID_ARG, "null device pointer");
    return launch_head_aggregate(d_ids, d_vals, T, H, k, d_sae, k_out, d_out_ids, d_out_vals, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- SAE decode
s3_status s3_sae_decode(const void* d_W_dec, const float* d_b_dec, int d_in, int d_sae, s3_dtype dtype, const int32_t* d_ids,
                        const float* d_vals, int T, int k, float* d_xhat, int64_t ld_xhat, const void* d_x, int64_t ldx,
                        float* d_sqerr, void* stream)
{
    S3_REQUIRE(dtype == S3_BF16 || dtype == S3_F32, S3_ERR_INVALID_ARG, "unknown dtype %d", (int)dtype);
    const int vec = dtype == S3_BF16 ? 8 : 4;
    S3_REQUIRE(d_in >= 1 && d_sae >= 1 && d_in % vec == 0, S3_ERR_INVALID_ARG, "d_in = %d must be a positive multiple of %d", d_in, vec);
    S3_REQUIRE(k >= 1 && k <= S3_MAX_K, S3_ERR_UNSUPPORTED, "k = %d out of [1, %d]", k, S3_MAX_K);
    S3_REQUIRE(T >= 0, S3_ERR_INVALID_ARG, "T is negative");
    if (T == 0) return S3_OK;
    S3_REQUIRE(d_W_dec && d_b_dec && d_ids && d_vals, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(d_xhat || d_sqerr, S3_ERR_INVALID_ARG, "neither x_hat nor sqerr is wanted");
    S3_REQUIRE(aligned16(d_W_dec) && aligned16(d_b_dec), S3_ERR_INVALID_ARG, "W_dec and b_dec must be 16-byte aligned");
    if (d_xhat) S3_REQUIRE(aligned16(d_xhat) && ld_xhat >= d_in && ld_xhat % 4 == 0, S3_ERR_INVALID_ARG,
                           "x_hat must be 16-byte aligned with a row pitch that is a multiple of 4 and >= d_in");
    if (d_sqerr) S3_REQUIRE(d_x && aligned16(d_x) && ldx >= d_in && ldx % vec == 0, S3_ERR_INVALID_ARG,
                            "sqerr needs x, 16-byte aligned with a row pitch that is a multiple of %d and >= d_in", vec);
    return launch_decode(d_W_dec, d_b_dec, d_in, d_sae, dtype, d_ids, d_vals, T, k, d_xhat, ld_xhat, d_x, ldx, d_sqerr,
                         static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- SAE training step
size_t s3_sae_backward_workspace_bytes(int T)
{
    if (T < 0) return 0;
    return 256 + round_up(static_cast<size_t>(T) * 4, 256);
}

s3_status s3_sae_backward(const float* d_W_enc, const float* d_b_enc, const float* d_W_dec, const float* d_b_dec, const float* d_x, int64_t ldx,
                          const int32_t* d_ids, const float* d_vals, int T, int k, int d_in, int d_sae, float* d_gW_enc,
                          float* d_gb_enc, float* d_gW_dec, float* d_gb_dec, float* d_loss, void* d_ws, size_t ws_bytes, void* stream)
{
    S3_REQUIRE(T >= 1 && d_in >= 1 && d_sae >= 1, S3_ERR_INVALID_ARG, "T = %d, d_in = %d, d_sae = %d out of range", T, d_in, d_sae);
    S3_REQUIRE(k >= 1 && k <= S3_MAX_K, S3_ERR_UNSUPPORTED, "k = %d out of [1, %d]", k, S3_MAX_K);
    S3_REQUIRE(d_in <= 4096, S3_ERR_UNSUPPORTED, "d_in = %d exceeds 4096", d_in);
    S3_REQUIRE(ldx >= d_in, S3_ERR_INVALID_ARG, "ldx = %lld is smaller than d_in = %d", (long long)ldx, d_in);
    S3_REQUIRE(d_W_enc && d_W_dec && d_b_dec && d_x && d_ids && d_gW_enc && d_gb_enc && d_gW_dec && d_gb_dec && d_loss,
               S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(d_vals != nullptr || d_b_enc != nullptr, S3_ERR_INVALID_ARG, "without d_vals the code is recomputed and needs d_b_enc");
    S3_REQUIRE(d_ws != nullptr && ws_bytes >= s3_sae_backward_workspace_bytes(T), S3_ERR_CAPACITY, "workspace holds %zu bytes, %zu needed",
               ws_bytes, s3_sae_backward_workspace_bytes(T));
    return launch_sae_backward(d_W_enc, d_b_enc, d_W_dec, d_b_dec, d_x, ldx, d_ids, d_vals, T, k, d_in, d_sae, d_gW_enc, d_gb_enc, d_gW_dec,
                               d_gb_dec, d_loss, reinterpret_cast<float*>(static_cast<unsigned char*>(d_ws) + 256),
                               static_cast<cudaStream_t>(stream));
}

s3_status s3_cast_f32_to_bf16(const float* d_src, void* d_dst, size_t n, void* stream)
{
    if (n == 0) return S3_OK;
    S3_REQUIRE(d_src && d_dst, S3_ERR_INVALID_ARG, "null device pointer");
    return launch_cast_bf16(d_src, d_dst, n, static_cast<cudaStream_t>(stream));
}

s3_status s3_adam_update(float* d_param, float* d_m, float* d_v, const float* d_grad, size_t n, const s3_adam_params* p, void* stream)
{
    S3_REQUIRE(p != nullptr, S3_ERR_INVALID_ARG, "params is null");
    S3_REQUIRE(p->step >= 1, S3_ERR_INVALID_ARG, "step = %d must count from 1", p->step);
    S3_REQUIRE(p->beta1 >= 0.0f && p->beta1 < 1.0f && p->beta2 >= 0.0f && p->beta2 < 1.0f && p->eps >= 0.0f, S3_ERR_INVALID_ARG,
               "beta1 = %g, beta2 = %g must lie in [0, 1) and eps = %g must not be negative", p->beta1, p->beta2, p->eps);
    if (n == 0) return S3_OK;
    S3_REQUIRE(d_param && d_m && d_v && d_grad, S3_ERR_INVALID_ARG, "null device pointer");
    const double c1 = 1.0 / (1.0 - pow(static_cast<double>(p->beta1), p->step));
    const double c2 = 1.0 / (1.0 - pow(static_cast<double>(p->beta2), p->step));
    return launch_adam(d_param, d_m, d_v, d_grad, n, p->lr, p->beta1, p->beta2, p->eps, static_cast<float>(c1), static_cast<float>(c2),
                       static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- index-set fusion
size_t s3_fuse_workspace_bytes(int Q, int64_t L)
{
    if (Q < 0 || L < 0) return 0;
    return 256 + fuse_workspace_bytes(Q, L);
}

s3_status s3_fuse_index_sets(const int32_t* d_centers, int Q, int n_centers, int span_width, const int32_t* d_lexical, int n_lex,
                             int lead, int tail, int64_t L, int32_t* d_out_idx, int cap, int32_t* d_out_count, void* d_ws,
                             size_t ws_bytes, void* stream)
{
    S3_REQUIRE(Q >= 0 && n_centers >= 0 && n_lex >= 0, S3_ERR_INVALID_ARG, "Q = %d, n_centers = %d, n_lex = %d out of range", Q,
               n_centers, n_lex);
    S3_REQUIRE(span_width >= 0 && lead >= 0 && tail >= 0 && cap >= 0, S3_ERR_INVALID_ARG,
               "span_width = %d, lead = %d, tail = %d, cap = %d must not be negative", span_width, lead, tail, cap);
    S3_REQUIRE(L >= 0 && L <= INT32_MAX, S3_ERR_INVALID_ARG, "L out of range");
    if (Q == 0) return S3_OK;
    S3_REQUIRE(d_out_count != nullptr && (cap == 0 || d_out_idx != nullptr), S3_ERR_INVALID_ARG, "null output pointer");
    S3_REQUIRE(n_centers == 0 || d_centers != nullptr, S3_ERR_INVALID_ARG, "d_centers is null");
    S3_REQUIRE(d_ws != nullptr && ws_bytes >= s3_fuse_workspace_bytes(Q, L), S3_ERR_CAPACITY, "workspace holds %zu bytes, %zu needed",
               ws_bytes, s3_fuse_workspace_bytes(Q, L));
    return launch_fuse_sets(d_centers, Q, n_centers, span_width, d_lexical, d_lexical ? n_lex : 0, lead, tail, L, d_out_idx, cap,
                            d_out_count, static_cast<unsigned char*>(d_ws) + 256, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
