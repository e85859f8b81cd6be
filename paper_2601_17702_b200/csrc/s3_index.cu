// Host-resident inverted index (Sec. 3.4): each appended chunk-layer CSR is copied device->pinned host
// on the index's own stream, ordered after the producer by an event, so the scan loop never blocks
// the host and device memory stays bounded by the chunk size. The index keeps, per layer, the list of
// chunk segments in arrival order; the merged per-layer CSR is produced on demand.
#include <algorithm>
#include <new>
#include <vector>

#include "s3_common.cuh"

namespace {

struct Slab {
    unsigned char* base;
    size_t size, used;
};

struct Segment {
    int T, k;
    int64_t pos_base;
    uint32_t* row_ptr;   // [d_sae+1] pinned
    int32_t* pos;        // [T*k] pinned
    float* pval;         // nullable
    int64_t nnz;         // -1 until validated by sync
};

}  // namespace

struct s3_index {
    int n_layers = 0, d_sae = 0;
    int device = 0;
    size_t slab_bytes = 0;
    std::vector<Slab> slabs;
    std::vector<std::vector<Segment>> layers;
    std::vector<int64_t> next_pos;           // per layer: first position a new chunk may start at
    std::vector<cudaEvent_t> produced, reusable;   // per layer
    cudaEvent_t all_copied = nullptr;
    cudaStream_t copy_stream = nullptr;
    bool dirty = false;                      // copies enqueued since the last sync
};

namespace {

using namespace s3;

s3_status arena_alloc(s3_index* ix, size_t bytes, void** out)
{
    bytes = round_up(bytes, 256);
    if (ix->slabs.empty() || ix->slabs.back().size - ix->slabs.back().used < bytes) {
        const size_t want = std::max(bytes, ix->slab_bytes);
        void* p = nullptr;
        const cudaError_t e = cudaHostAlloc(&p, want, cudaHostAllocDefault);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return fail(e == cudaErrorMemoryAllocation ? S3_ERR_NOMEM : S3_ERR_CUDA,
                        "pinned allocation of %zu bytes failed: %s", want, cudaGetErrorString(e));
        }
        ix->slabs.push_back({static_cast<unsigned char*>(p), want, 0});
    }
    Slab& s = ix->slabs.back();
    *out = s.base + s.used;
    s.used += bytes;
    return S3_OK;
}

s3_status validate_new_segments(s3_index* ix)
{
    for (auto& segs : ix->layers)
        for (Segment& g : segs) {
            if (g.nnz >= 0) continue;
            const uint32_t* rp = g.row_ptr;
            S3_REQUIRE(rp[0] == 0, S3_ERR_STATE, "segment row_ptr[0] = %u, expected 0", rp[0]);
            for (int f = 0; f < ix->d_sae; ++f)
                S3_REQUIRE(rp[f + 1] >= rp[f], S3_ERR_STATE, "segment row_ptr not monotone at feature %d", f);
            S3_REQUIRE(static_cast<int64_t>(rp[ix->d_sae]) <= static_cast<int64_t>(g.T) * g.k, S3_ERR_CAPACITY,
                       "segment holds %u postings but only T*k = %lld were copied", rp[ix->d_sae],
                       static_cast<long long>(g.T) * g.k);
            g.nnz = rp[ix->d_sae];
        }
    return S3_OK;
}

}  // namespace

extern "C" {

s3_status s3_index_create(s3_index** out, int n_layers, int d_sae, size_t pinned_slab_bytes)
{
    using namespace s3;
    S3_REQUIRE(out != nullptr, S3_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    S3_REQUIRE(n_layers >= 1 && n_layers <= 4096, S3_ERR_INVALID_ARG, "n_layers = %d out of range", n_layers);
    S3_REQUIRE(d_sae >= 1, S3_ERR_INVALID_ARG, "d_sae = %d out of range", d_sae);
    s3_index* ix = new (std::nothrow) s3_index();
    S3_REQUIRE(ix != nullptr, S3_ERR_NOMEM, "out of host memory");
    ix->n_layers = n_layers;
    ix->d_sae = d_sae;
    ix->slab_bytes = pinned_slab_bytes ? pinned_slab_bytes : (size_t(64) << 20);
    ix->layers.resize(n_layers);
    ix->next_pos.assign(n_layers, 0);
    cudaError_t e = cudaGetDevice(&ix->device);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ix->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ix->all_copied, cudaEventDisableTiming);
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
        cudaEvent_t a = nullptr, b = nullptr;
        e = cudaEventCreateWithFlags(&a, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b, cudaEventDisableTiming);
        if (a) ix->produced.push_back(a);
        if (b) ix->reusable.push_back(b);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        s3_index_destroy(ix);
        return fail(S3_ERR_CUDA, "index stream/event creation failed: %s", cudaGetErrorString(e));
    }
    *out = ix;
    return S3_OK;
}

s3_status s3_index_reserve(s3_index* ix, size_t bytes)
{
    using namespace s3;
    S3_REQUIRE(ix != nullptr, S3_ERR_INVALID_ARG, "index is null");
    size_t free_bytes = ix->slabs.empty() ? 0 : ix->slabs.back().size - ix->slabs.back().used;
    if (free_bytes >= bytes) return S3_OK;
    void* p = nullptr;
    const size_t want = round_up(bytes, 4096);
    const cudaError_t e = cudaHostAlloc(&p, want, cudaHostAllocDefault);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return fail(e == cudaErrorMemoryAllocation ? S3_ERR_NOMEM : S3_ERR_CUDA,
                    "pinned reservation of %zu bytes failed: %s", want, cudaGetErrorString(e));
    }
    ix->slabs.push_back({static_cast<unsigned char*>(p), want, 0});
    return S3_OK;
}

s3_status s3_index_append(s3_index* ix, int layer, const uint32_t* d_row_ptr, const int32_t* d_pos,
                          const float* d_pval, int T, int k, int64_t pos_base, void* producer_stream,
                          void** reuse_event_out)
{
    using namespace s3;
    S3_REQUIRE(ix != nullptr, S3_ERR_INVALID_ARG, "index is null");
    S3_REQUIRE(layer >= 0 && layer < ix->n_layers, S3_ERR_INVALID_ARG, "layer %d out of range", layer);
    S3_REQUIRE(d_row_ptr != nullptr && d_pos != nullptr, S3_ERR_INVALID_ARG, "null device pointer");
    S3_REQUIRE(T >= 0 && k >= 1, S3_ERR_INVALID_ARG, "T = %d, k = %d out of range", T, k);
    S3_REQUIRE(pos_base >= 0, S3_ERR_INVALID_ARG, "pos_base is negative");
    S3_REQUIRE(pos_base + T <= INT32_MAX, S3_ERR_CAPACITY, "positions beyond int32 (pos_base %lld + T %d)",
               static_cast<long long>(pos_base), T);
    S3_REQUIRE(pos_base >= ix->next_pos[layer], S3_ERR_STATE,
               "chunk at position %lld arrives after positions up to %lld were indexed for layer %d",
               static_cast<long long>(pos_base), static_cast<long long>(ix->next_pos[layer]), layer);
    const size_t n = static_cast<size_t>(T) * k;
    Segment g{T, k, pos_base, nullptr, nullptr, nullptr, -1};
    void* p = nullptr;
    s3_status st = arena_alloc(ix, (size_t)(ix->d_sae + 1) * sizeof(uint32_t), &p);
    if (st != S3_OK) return st;
    g.row_ptr = static_cast<uint32_t*>(p);
    st = arena_alloc(ix, std::max<size_t>(n, 1) * sizeof(int32_t), &p);
    if (st != S3_OK) return st;
    g.pos = static_cast<int32_t*>(p);
    if (d_pval) {
        st = arena_alloc(ix, std::max<size_t>(n, 1) * sizeof(float), &p);
        if (st != S3_OK) return st;
        g.pval = static_cast<float*>(p);
    }
    cudaStream_t prod = static_cast<cudaStream_t>(producer_stream);
    S3_CUDA_TRY(cudaEventRecord(ix->produced[layer], prod));
    S3_CUDA_TRY(cudaStreamWaitEvent(ix->copy_stream, ix->produced[layer], 0));
    S3_CUDA_TRY(cudaMemcpyAsync(g.row_ptr, d_row_ptr, (size_t)(ix->d_sae + 1) * sizeof(uint32_t),
                                cudaMemcpyDeviceToHost, ix->copy_stream));
    if (n) {
        S3_CUDA_TRY(cudaMemcpyAsync(g.pos, d_pos, n * sizeof(int32_t), cudaMemcpyDeviceToHost, ix->copy_stream));
        if (d_pval)
            S3_CUDA_TRY(cudaMemcpyAsync(g.pval, d_pval, n * sizeof(float), cudaMemcpyDeviceToHost, ix->copy_stream));
    }
    S3_CUDA_TRY(cudaEventRecord(ix->reusable[layer], ix->copy_stream));
    if (reuse_event_out) *reuse_event_out = ix->reusable[layer];
    ix->layers[layer].push_back(g);
    ix->next_pos[layer] = pos_base + T;
    ix->dirty = true;
    return S3_OK;
}

s3_status s3_index_stream_wait(s3_index* ix, void* stream)
{
    using namespace s3;
    S3_REQUIRE(ix != nullptr, S3_ERR_INVALID_ARG, "index is null");
    S3_CUDA_TRY(cudaEventRecord(ix->all_copied, ix->copy_stream));
    S3_CUDA_TRY(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), ix->all_copied, 0));
    return S3_OK;
}

s3_status s3_index_sync(s3_index* ix)
{
    using namespace s3;
    S3_REQUIRE(ix != nullptr, S3_ERR_INVALID_ARG, "index is null");
    if (ix->dirty) {
        S3_CUDA_TRY(cudaStreamSynchronize(ix->copy_stream));
        ix->dirty = false;
    }
    return validate_new_segments(ix);
}

s3_status s3_index_layer_postings(s3_index* ix, int layer, uint64_t* n_out)
{
    using namespace s3;
    S3_REQUIRE(ix != nullptr && n_out != nullptr, S3_ERR_INVALID_ARG, "null argument");
    S3_REQUIRE(layer >= 0 && layer < ix->n_layers, S3_ERR_INVALID_ARG, "layer %d out of range", layer);
    const s3_status st = s3_index_sync(ix);
    if (st != S3_OK) return st;
    uint64_t n = 0;
    for (const Segment& g : ix->layers[layer]) n += static_cast<uint64_t>(g.nnz);
    *n_out = n;
    return S3_OK;
}

s3_status s3_index_export_csr(s3_index* ix, int layer, uint64_t* h_row_ptr, int32_t* h_pos, float* h_pval)
{
    using namespace s3;
    S3_REQUIRE(ix != nullptr && h_row_ptr != nullptr, S3_ERR_INVALID_ARG, "null argument");
    S3_REQUIRE(layer >= 0 && layer < ix->n_layers, S3_ERR_INVALID_ARG, "layer %d out of range", layer);
    const s3_status st = s3_index_sync(ix);
    if (st != S3_OK) return st;
    const std::vector<Segment>& segs = ix->layers[layer];
    const int D = ix->d_sae;
    // list length of feature f = sum of the segments' lengths; prefix sum gives the merged offsets
    h_row_ptr[0] = 0;
    for (int f = 0; f < D; ++f) {
        uint64_t len = 0;
        for (const Segment& g : segs) len += g.row_ptr[f + 1] - g.row_ptr[f];
        h_row_ptr[f + 1] = h_row_ptr[f] + len;
    }
    if (h_row_ptr[D] == 0) return S3_OK;
    S3_REQUIRE(h_pos != nullptr, S3_ERR_INVALID_ARG, "h_pos is null");
    if (h_pval)
        for (const Segment& g : segs)
            S3_REQUIRE(g.pval != nullptr || g.nnz == 0, S3_ERR_STATE, "values requested but a chunk was appended without them");
    // segment-major copy keeps each source read sequential; a running per-feature cursor places it
    std::vector<uint64_t> cursor(h_row_ptr, h_row_ptr + D);
    for (const Segment& g : segs) {
        for (int f = 0; f < D; ++f) {
            const uint32_t b = g.row_ptr[f], e = g.row_ptr[f + 1];
            if (e == b) continue;
            std::copy(g.pos + b, g.pos + e, h_pos + cursor[f]);
            if (h_pval) std::copy(g.pval + b, g.pval + e, h_pval + cursor[f]);
            cursor[f] += e - b;
        }
    }
    return S3_OK;
}

s3_status s3_index_stats(s3_index* ix, s3_index_stats_t* out)
{
    using namespace s3;
    S3_REQUIRE(ix != nullptr && out != nullptr, S3_ERR_INVALID_ARG, "null argument");
    const s3_status st = s3_index_sync(ix);
    if (st != S3_OK) return st;
    s3_index_stats_t s{};
    for (const Slab& b : ix->slabs) { s.host_bytes += (int64_t)b.used; s.host_bytes_reserved += (int64_t)b.size; }
    std::vector<uint64_t> len(ix->d_sae);
    for (int l = 0; l < ix->n_layers; ++l) {
        std::fill(len.begin(), len.end(), 0);
        for (const Segment& g : ix->layers[l]) {
            s.n_chunks += 1;
            s.n_postings += g.nnz;
            for (int f = 0; f < ix->d_sae; ++f) len[f] += g.row_ptr[f + 1] - g.row_ptr[f];
        }
        for (int f = 0; f < ix->d_sae; ++f) s.max_list_len = std::max<int64_t>(s.max_list_len, (int64_t)len[f]);
        s.n_positions = std::max(s.n_positions, ix->next_pos[l]);
    }
    *out = s;
    return S3_OK;
}

s3_status s3_index_destroy(s3_index* ix)
{
    if (!ix) return S3_OK;
    if (ix->copy_stream) (void)cudaStreamSynchronize(ix->copy_stream);
    for (cudaEvent_t e : ix->produced) (void)cudaEventDestroy(e);
    for (cudaEvent_t e : ix->reusable) (void)cudaEventDestroy(e);
    if (ix->all_copied) (void)cudaEventDestroy(ix->all_copied);
    if (ix->copy_stream) (void)cudaStreamDestroy(ix->copy_stream);
    for (Slab& b : ix->slabs) (void)cudaFreeHost(b.base);
    (void)cudaGetLastError();
    delete ix;
    return S3_OK;
}

}  // extern "C"
