// Device helpers shared by the kernels that read a query's Top-k codes and walk posting lists (span scoring, position
// density, head aggregation): block size, the shared-memory carve-up, the block scan, the aggregation of (id, value)
// entries into unique features, the cut of posting lists into 32-posting pieces and the piece -> feature table.
// Everything lives in an unnamed namespace: each translation unit that includes this file gets its own copy.
#pragma once

#include "s3_common.cuh"

namespace s3 {

namespace {

constexpr int ST = 512;          // threads per block
constexpr int SW = ST / 32;      // warps
constexpr int PIECE = 32;        // postings per work item
constexpr int BATCH = 8;         // work items a warp keeps in flight
constexpr int WIN = 8192;        // pieces whose owning feature is tabulated at a time

struct ScoreLayers {
    s3_csr_view v[S3_MAX_SCORE_LAYERS];
};

// Shared-memory carve-up, identical on host and device.
struct ScoreSmem {
    uint32_t acc_off, keys_off, ufeat_off, ustart_off, uaq_off, ulo_off, cstart_off, owner_off, total;
};
__host__ __device__ inline ScoreSmem score_smem(int nk, int npad, int n_spans, bool weighted)
{
    ScoreSmem L;
    uint32_t o = 0;
    L.acc_off = o;    o += (static_cast<uint32_t>(n_spans) + 2) * (weighted ? 8u : 4u);  o = (o + 15u) & ~15u;
    L.ulo_off = o;    o += static_cast<uint32_t>(nk) * 8u;
    L.keys_off = o;   o += static_cast<uint32_t>(npad) * 4u;
    L.ufeat_off = o;  L.cstart_off = o;  o += (static_cast<uint32_t>(nk) + 1u) * 4u;   // cstart[u] replaces ufeat[u]
    L.ustart_off = o; o += (static_cast<uint32_t>(nk) + 1u) * 4u;
    L.uaq_off = o;    o += weighted ? static_cast<uint32_t>(nk) * 4u : 0u;
    o = (o + 3u) & ~3u;
    L.owner_off = o;  o += WIN * 2u;                                   // owning feature of each piece of the window
    L.total = o + 16u;
    return L;
}

__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* ws, uint32_t& total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) ws[warp] = inc;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (int w = 0; w < SW; ++w) { const uint32_t t = ws[w]; ws[w] = run; run += t; }
        ws[SW] = run;
    }
    __syncthreads();
    const uint32_t res = ws[warp] + inc - v;
    total = ws[SW];
    __syncthreads();
    return res;
}

// Phase a, shared by the scoring kernels: the query's nk (id, value) entries -> unique features. Sorts
// (id, entry) keys ascending (invalid ids last), detects runs: ufeat[u] = id, ustart[u]..ustart[u+1] = its
// entries in keys[] (so cQ = ustart[u+1] - ustart[u]), and, if wanted, uaq[u] = the entries' activations summed
// in query-token order in fp32. Returns the number of unique features. Called by the whole block.
__device__ __forceinline__ int aggregate_query(const int32_t* qi, const float* qv, int nk, int npad, int d_sae, bool want_aq,
                                               uint32_t* keys, int32_t* ufeat, int32_t* ustart, float* uaq, uint32_t* ws,
                                               int* n_unique_s)
{
    const int tid = threadIdx.x;
    for (int i = tid; i < npad; i += ST) {
        uint32_t key = 0xFFFFFFFFu;
        if (i < nk) {
            const int32_t f = qi[i];
            if (f >= 0 && f < d_sae) key = (static_cast<uint32_t>(f) << 12) | static_cast<uint32_t>(i);
        }
        keys[i] = key;
    }
    __syncthreads();
    for (int size = 2; size <= npad; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = tid; i < (npad >> 1); i += ST) {
                const int pos = 2 * i - (i & (stride - 1));   // stride is a power of two
                const bool asc = (pos & size) == 0;
                const uint32_t x = keys[pos], y = keys[pos + stride];
                if ((x > y) == asc) { keys[pos] = y; keys[pos + stride] = x; }
            }
            __syncthreads();
        }
    }
    uint32_t carry = 0;
    for (int i0 = 0; i0 < nk; i0 += ST) {
        const int i = i0 + tid;
        uint32_t head = 0;
        if (i < nk && keys[i] != 0xFFFFFFFFu)
            head = (i == 0) || ((keys[i] >> 12) != (keys[i - 1] >> 12));
        uint32_t total;
        const uint32_t u = block_exclusive_scan(head, ws, total) + carry;
        if (head) { ufeat[u] = static_cast<int32_t>(keys[i] >> 12); ustart[u] = i; }
        carry += total;
    }
    if (tid == 0) {
        int lo = 0, hi = nk;   // first invalid key (keys sorted, invalid last)
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (keys[mid] == 0xFFFFFFFFu) hi = mid; else lo = mid + 1; }
        ustart[carry] = lo;
        *n_unique_s = static_cast<int>(carry);
    }
    __syncthreads();
    const int U = *n_unique_s;
    for (int u = tid; want_aq && u < U; u += ST) {   // aQ: activations summed in query-token order (fp32)
        float s = 0.0f;
        for (int i = ustart[u]; i < ustart[u + 1]; ++i) s = __fadd_rn(s, qv[keys[i] & 0xFFFu]);
        uaq[u] = s;
    }
    __syncthreads();
    return U;
}

// Phase b head, shared by the scoring kernels: list bounds of the U unique features (ulo, ulen; a list longer
// than stop_freq > 0 counts as empty) and the exclusive prefix cstart[0..U] of their 32-posting pieces. ulen
// may share storage with keys, cstart with ufeat (a thread reads ufeat[u] before it writes cstart[u]).
// Returns the number of pieces. Called by the whole block.
__device__ __forceinline__ uint32_t cut_lists(const uint64_t* __restrict__ row_ptr, int U, int64_t stop_freq,
                                              const int32_t* ufeat, unsigned long long* ulo, uint32_t* ulen,
                                              uint32_t* cstart, uint32_t* ws, const uint32_t* __restrict__ blk_ptr = nullptr)
{
    const int tid = threadIdx.x;
    uint32_t piece_carry = 0;
    for (int u0 = 0; u0 < U; u0 += ST) {
        const int u = u0 + tid;
        uint32_t n_pieces = 0;
        if (u < U) {
            const int f = ufeat[u];
            const uint64_t lo = __ldg(row_ptr + f), hi = __ldg(row_ptr + f + 1);
            uint64_t len = hi - lo;
            if (len > 0x7FFFFFFFull) len = 0x7FFFFFFFull;          // positions are int32: a list cannot be longer
            if (stop_freq > 0 && static_cast<int64_t>(len) > stop_freq) len = 0;   // stop feature
            ulo[u] = blk_ptr ? static_cast<unsigned long long>(__ldg(blk_ptr + f)) : lo;   // compact index: first block
            ulen[u] = static_cast<uint32_t>(len);
            n_pieces = static_cast<uint32_t>((len + PIECE - 1) / PIECE);
        }
        uint32_t total;
        const uint32_t ex = block_exclusive_scan(n_pieces, ws, total) + piece_carry;
        if (u < U) cstart[u] = ex;
        piece_carry += total;
    }
    if (tid == 0) cstart[U] = piece_carry;
    __syncthreads();
    return piece_carry;
}

// Owning feature of each piece win0 .. win1-1 (binary search in the pieces' prefix, one piece per thread and
// step), so that the walk below needs no running cursor and its loads are independent of each other.
__device__ __forceinline__ void tabulate_owners(const uint32_t* cstart, int U, uint32_t win0, uint32_t win1, uint16_t* owner)
{
    for (uint32_t c = win0 + threadIdx.x; c < win1; c += ST) {
        int lo = 0, hi = U;                  // last u with cstart[u] <= c (pieces of empty lists share a start)
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cstart[mid] <= c) lo = mid; else hi = mid; }
        owner[c - win0] = static_cast<uint16_t>(lo);
    }
    __syncthreads();
}

}  // namespace

}  // namespace s3
