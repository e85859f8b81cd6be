// Per-position relevance, smoothed density and peak selection (Sec. 3.5 Eq. 6, "Adaptive Granularity"; Alg. 1 Phase 2):
// the paper's own retrieval tail, beside the fixed-width span scorer of s3_score.cu.
#include "s3_kernels.cuh"
#include "s3_query.cuh"

namespace s3 {

namespace {

// ---- per-position relevance, smoothed density, peak selection (Sec. 3.5 Eq. 6, "Adaptive Granularity") --------
// Weights are taken in fixed point (2^-24) so that S, the density and therefore the peaks are exact integer results
// whatever order the postings are visited in. Four kernels:
//   features   : per (query, layer) the unique query features and their weights w_l(f) (0 for stop features);
//   skip       : per (layer, feature, position tile) the index of the list's first posting inside the tile (binary
//                search; the lists are ascending), so that a block can gather one tile's part of every list;
//   accumulate : per (position tile, query) S[t] += w_l(f) over the tile's postings of every query feature, in 64-bit
//                shared-memory accumulators (one atomic per posting stays on the SM), written out once;
//   peaks      : per query the density D[t] = sum of S over the K positions starting at t - K/2 (a tile of S plus its
//                halo is prefix-summed in shared memory, D[t] is the difference of two prefix values) and greedy
//                non-maximum suppression over D with per-segment maxima in shared memory: a round reduces the segment
//                maxima, takes the best position (ties: lowest), clears D within the radius and redoes only the touched
//                segments.
constexpr int MIN_SEG_SHIFT = 8;      // a segment of the maxima table holds 2^seg_shift >= 256 positions,
constexpr int MAX_SEGS = 2048;       // the smallest power of two that covers L with MAX_SEGS segments
constexpr int CONV_TILE = 2048;      // positions smoothed per pass through shared memory
constexpr int MAX_CONV_KERNEL = 1024;
constexpr int POS_TILE = 8192;       // positions accumulated per block (64 KB of 64-bit sums)
constexpr int FCHUNK = 1024;         // query features handled per pass of the accumulate kernel
constexpr int AWIN = 4096;           // pieces whose owning feature is tabulated at a time there
constexpr int APIECE = 16;           // postings per piece there: a tile holds a fraction of a list, so half a warp per piece

struct DensityArgs {
    const int32_t* q_ids;
    const float* q_vals;
    long long* s_fix;        // [Q][L]
    long long* d_fix;        // [Q][L]
    int32_t* feat_cnt;       // [n_layers][Q]
    int32_t* feat_id;        // [n_layers][Q][nk]
    long long* feat_w;       // [n_layers][Q][nk]
    uint32_t* skip;          // [n_layers][d_sae][n_tiles + 1]
    int32_t* centers;        // [Q][n_centers]
    float* center_density;   // [Q][n_centers]
    float* s_out;            // [Q][L] or null
    float* d_out;            // [Q][L] or null
    long long L;
    int n_layers, d_sae, Q, nk, npad, conv_kernel, nms_radius, n_centers, seg_shift, n_tiles;
    int64_t stop_freq;
};

__device__ __forceinline__ bool better(long long v, long long p, long long bv, long long bp)
{
    return v > bv || (v == bv && v > 0 && p < bp);
}

// Maximum (value, lowest position) of d[lo..hi) over the calling warp.
__device__ __forceinline__ void warp_segment_max(const long long* d, long long lo, long long hi, int lane, long long& bv, long long& bp)
{
    bv = 0; bp = -1;
    for (long long t = lo + lane; t < hi; t += 32) {
        const long long v = d[t];
        if (better(v, t, bv, bp)) { bv = v; bp = t; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long ov = __shfl_xor_sync(0xffffffffu, bv, o), op = __shfl_xor_sync(0xffffffffu, bp, o);
        if (better(ov, op, bv, bp)) { bv = ov; bp = op; }
    }
}

__global__ void __launch_bounds__(ST)
density_features_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ DensityArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    const ScoreSmem SL = score_smem(a.nk, a.npad, 0, true);
    uint32_t* keys = reinterpret_cast<uint32_t*>(score_smem_raw + SL.keys_off);
    int32_t* ufeat = reinterpret_cast<int32_t*>(score_smem_raw + SL.ufeat_off);
    int32_t* ustart = reinterpret_cast<int32_t*>(score_smem_raw + SL.ustart_off);
    float* uaq = reinterpret_cast<float*>(score_smem_raw + SL.uaq_off);
    __shared__ uint32_t ws[SW + 1];
    __shared__ int n_unique_s;
    const int q = blockIdx.x, l = blockIdx.y;
    const size_t slot = (size_t)l * a.Q + q;
    const int U = aggregate_query(a.q_ids + slot * a.nk, a.q_vals + slot * a.nk, a.nk, a.npad, a.d_sae, true, keys, ufeat, ustart,
                                  uaq, ws, &n_unique_s);
    const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
    for (int u = threadIdx.x; u < U; u += ST) {
        const int f = ufeat[u];
        uint64_t len = __ldg(row_ptr + f + 1) - __ldg(row_ptr + f);
        if (len > 0x7FFFFFFFull) len = 0x7FFFFFFFull;
        long long w = 0;                                   // w = rint(aQ * IDF(freq) * 2^24), IDF = 1 / (ln(1 + freq) + 1)
        if (len > 0 && !(a.stop_freq > 0 && static_cast<int64_t>(len) > a.stop_freq))
            w = __double2ll_rn(static_cast<double>(uaq[u]) * (1.0 / (log(1.0 + static_cast<double>(len)) + 1.0)) * 16777216.0);
        a.feat_id[slot * a.nk + u] = f;
        a.feat_w[slot * a.nk + u] = w;
    }
    if (threadIdx.x == 0) a.feat_cnt[slot] = U;
}

// skip[l][f][p] = number of postings of feature f (layer l) at positions below p * POS_TILE, p = 0 .. n_tiles.
__global__ void __launch_bounds__(ST)
density_skip_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ DensityArgs a)
{
    const int l = blockIdx.y;
    const long long per_layer = (long long)a.d_sae * (a.n_tiles + 1);
    const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
    const int32_t* __restrict__ pos = layers.v[l].d_pos;
    for (long long i = (long long)blockIdx.x * ST + threadIdx.x; i < per_layer; i += (long long)gridDim.x * ST) {
        const int f = static_cast<int>(i / (a.n_tiles + 1)), p = static_cast<int>(i % (a.n_tiles + 1));
        const uint64_t base = __ldg(row_ptr + f);
        uint64_t len = __ldg(row_ptr + f + 1) - base;
        if (len > 0x7FFFFFFFull) len = 0x7FFFFFFFull;
        const long long bound = (long long)p * POS_TILE;
        uint32_t lo = 0, hi = static_cast<uint32_t>(len);     // first index with pos >= bound
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (__ldg(pos + base + mid) < bound) lo = mid + 1; else hi = mid;
        }
        a.skip[(size_t)l * per_layer + i] = lo;
    }
}

__global__ void __launch_bounds__(ST)
density_accumulate_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ DensityArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    unsigned long long* acc = reinterpret_cast<unsigned long long*>(score_smem_raw);          // [POS_TILE]
    unsigned long long* ulo = acc + POS_TILE;                                                  // [FCHUNK] first posting (absolute)
    long long* uw = reinterpret_cast<long long*>(ulo + FCHUNK);                                // [FCHUNK]
    uint32_t* ulen = reinterpret_cast<uint32_t*>(uw + FCHUNK);                                 // [FCHUNK]
    uint32_t* cstart = ulen + FCHUNK;                                                          // [FCHUNK + 1]
    uint16_t* owner = reinterpret_cast<uint16_t*>(cstart + FCHUNK + 4);                        // [AWIN]
    __shared__ uint32_t ws[SW + 1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, q = blockIdx.y;
    const long long t0 = (long long)tile * POS_TILE;
    const int n_here = static_cast<int>(a.L - t0 < POS_TILE ? a.L - t0 : POS_TILE);
    for (int i = tid; i < POS_TILE; i += ST) acc[i] = 0ull;
    __syncthreads();
    for (int l = 0; l < a.n_layers; ++l) {
        const size_t slot = (size_t)l * a.Q + q;
        const int U = a.feat_cnt[slot];
        const uint64_t* __restrict__ row_ptr = layers.v[l].d_row_ptr;
        const int32_t* __restrict__ pos = layers.v[l].d_pos;
        const uint32_t* __restrict__ skip = a.skip + (size_t)l * a.d_sae * (a.n_tiles + 1);
        for (int u0 = 0; u0 < U; u0 += FCHUNK) {
            const int n_u = U - u0 < FCHUNK ? U - u0 : FCHUNK;
            // the tile's part of every list of the chunk and the exclusive prefix of its 32-posting pieces
            uint32_t carry = 0;
            for (int i0 = 0; i0 < n_u; i0 += ST) {
                const int i = i0 + tid;
                uint32_t n_pieces = 0;
                if (i < n_u) {
                    const int f = a.feat_id[slot * a.nk + u0 + i];
                    const long long w = a.feat_w[slot * a.nk + u0 + i];
                    const uint32_t* sk = skip + (size_t)f * (a.n_tiles + 1) + tile;
                    const uint32_t first = __ldg(sk), last = __ldg(sk + 1);
                    const uint32_t len = w != 0 ? last - first : 0u;
                    ulo[i] = __ldg(row_ptr + f) + first;
                    ulen[i] = len;
                    uw[i] = w;
                    n_pieces = (len + APIECE - 1) / APIECE;
                }
                uint32_t total;
                const uint32_t ex = block_exclusive_scan(n_pieces, ws, total) + carry;
                if (i < n_u) cstart[i] = ex;
                carry += total;
            }
            if (tid == 0) cstart[n_u] = carry;
            __syncthreads();
            const uint32_t piece_total = carry;
            for (uint32_t win0 = 0; win0 < piece_total; win0 += AWIN) {
                const uint32_t win1 = piece_total - win0 < AWIN ? piece_total : win0 + AWIN;
                for (uint32_t c = win0 + tid; c < win1; c += ST) {
                    int lo = 0, hi = n_u;              // last i with cstart[i] <= c
                    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cstart[mid] <= c) lo = mid; else hi = mid; }
                    owner[c - win0] = static_cast<uint16_t>(lo);
                }
                __syncthreads();
                const uint32_t n_win = win1 - win0;
                const uint32_t c_begin = win0 + static_cast<uint32_t>(static_cast<uint64_t>(n_win) * warp / SW);
                const uint32_t c_end = win0 + static_cast<uint32_t>(static_cast<uint64_t>(n_win) * (warp + 1) / SW);
                for (uint32_t c0 = c_begin; c0 < c_end; c0 += 2 * BATCH) {
                    int p[BATCH], ub[BATCH];
#pragma unroll
                    for (int b = 0; b < BATCH; ++b) {
                        const uint32_t c = c0 + 2 * b + (lane >> 4);          // each half of the warp takes a piece
                        p[b] = -1; ub[b] = 0;
                        if (c < c_end) {
                            const int i = owner[c - win0];
                            ub[b] = i;
                            const uint32_t j = (c - cstart[i]) * APIECE + (lane & 15);
                            if (j < ulen[i]) p[b] = __ldg(pos + ulo[i] + j);
                        }
                    }
#pragma unroll
                    for (int b = 0; b < BATCH; ++b) {
                        const long long rel = p[b] - t0;
                        if (p[b] >= 0 && rel >= 0 && rel < n_here) atomicAdd(&acc[rel], static_cast<unsigned long long>(uw[ub[b]]));
                    }
                }
                __syncthreads();
            }
        }
    }
    long long* S = a.s_fix + (size_t)q * a.L + t0;
    for (int i = tid; i < n_here; i += ST) S[i] = static_cast<long long>(acc[i]);
}

__global__ void __launch_bounds__(ST)
density_peaks_kernel(const __grid_constant__ DensityArgs a)
{
    extern __shared__ __align__(16) unsigned char score_smem_raw[];
    long long* seg_val = reinterpret_cast<long long*>(score_smem_raw);                             // [MAX_SEGS]
    long long* seg_pos = seg_val + MAX_SEGS;
    long long* tile = seg_pos + MAX_SEGS;                                                         // [CONV_TILE + MAX_CONV_KERNEL]
    __shared__ long long red_v[SW], red_p[SW], pick_s, scan_tot[SW + 1];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = blockIdx.x;
    const long long L = a.L;
    long long* S = a.s_fix + (size_t)q * L;
    long long* D = a.d_fix + (size_t)q * L;

    // density: K taps starting at t - K/2. Per tile of CONV_TILE positions: S[t0 - K/2 .. t0 + CONV_TILE + K - K/2) goes
    // to shared memory, is replaced by its inclusive prefix sum P (each thread scans a run of consecutive entries, the
    // runs' totals are scanned across the block), and D[t0 + i] = P[i + K - 1] - P[i - 1].
    const long long half = a.conv_kernel / 2;
    const int n_tile = CONV_TILE + a.conv_kernel - 1;                     // entries staged per tile
    const int run = (n_tile + ST - 1) / ST;
    for (long long t0 = 0; t0 < L; t0 += CONV_TILE) {
        for (int i = tid; i < n_tile; i += ST) {
            const long long t = t0 - half + i;
            tile[i] = (t >= 0 && t < L) ? S[t] : 0;
        }
        __syncthreads();
        const int i_lo = tid * run, i_hi = i_lo + run < n_tile ? i_lo + run : n_tile;
        long long sum = 0;
        for (int i = i_lo; i < i_hi; ++i) { sum += tile[i]; tile[i] = sum; }
        long long inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        if (lane == 31) scan_tot[warp] = inc;
        __syncthreads();
        if (tid == 0) {
            long long acc = 0;
            for (int w = 0; w < SW; ++w) { const long long v = scan_tot[w]; scan_tot[w] = acc; acc += v; }
        }
        __syncthreads();
        const long long base = scan_tot[warp] + inc - sum;
        for (int i = i_lo; i < i_hi; ++i) tile[i] += base;
        __syncthreads();
        for (int i = tid; i < CONV_TILE; i += ST) {
            const long long t = t0 + i;
            if (t >= L) break;
            const long long d = tile[i + a.conv_kernel - 1] - (i > 0 ? tile[i - 1] : 0);
            D[t] = d;
            if (a.d_out) a.d_out[(size_t)q * L + t] = static_cast<float>(static_cast<double>(d) * (1.0 / 16777216.0));
            if (a.s_out) a.s_out[(size_t)q * L + t] = static_cast<float>(static_cast<double>(S[t]) * (1.0 / 16777216.0));
        }
        __syncthreads();
    }

    // segment maxima
    const int seg = 1 << a.seg_shift;
    const int n_segs = static_cast<int>((L + seg - 1) >> a.seg_shift);
    for (int sg = warp; sg < n_segs; sg += SW) {
        long long bv, bp;
        const long long lo = (long long)sg << a.seg_shift, hi = lo + seg < L ? lo + seg : L;
        warp_segment_max(D, lo, hi, lane, bv, bp);
        if (lane == 0) { seg_val[sg] = bv; seg_pos[sg] = bp; }
    }
    __syncthreads();

    for (int r = 0; r < a.n_centers; ++r) {
        long long bv = 0, bp = -1;
        for (int sg = tid; sg < n_segs; sg += ST)
            if (better(seg_val[sg], seg_pos[sg], bv, bp)) { bv = seg_val[sg]; bp = seg_pos[sg]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const long long ov = __shfl_xor_sync(0xffffffffu, bv, o), op = __shfl_xor_sync(0xffffffffu, bp, o);
            if (better(ov, op, bv, bp)) { bv = ov; bp = op; }
        }
        if (lane == 0) { red_v[warp] = bv; red_p[warp] = bp; }
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < SW; ++w)
                if (better(red_v[w], red_p[w], bv, bp)) { bv = red_v[w]; bp = red_p[w]; }
            a.centers[(size_t)q * a.n_centers + r] = bv > 0 ? static_cast<int32_t>(bp) : -1;
            a.center_density[(size_t)q * a.n_centers + r] = bv > 0 ? static_cast<float>(static_cast<double>(bv) * (1.0 / 16777216.0)) : 0.0f;
            pick_s = bv > 0 ? bp : -1;
        }
        __syncthreads();
        const long long c = pick_s;
        if (c < 0) continue;               // nothing left above zero: the remaining rounds pad (uniform for the block)
        const long long k_lo = c - a.nms_radius < 0 ? 0 : c - a.nms_radius;
        const long long k_hi = c + a.nms_radius >= L ? L - 1 : c + a.nms_radius;
        for (long long t = k_lo + tid; t <= k_hi; t += ST) D[t] = 0;
        __syncthreads();
        const int sg_lo = static_cast<int>(k_lo >> a.seg_shift), sg_hi = static_cast<int>(k_hi >> a.seg_shift);
        for (int sg = sg_lo + warp; sg <= sg_hi; sg += SW) {
            long long sv, sp;
            const long long lo = (long long)sg << a.seg_shift, hi = lo + seg < L ? lo + seg : L;
            warp_segment_max(D, lo, hi, lane, sv, sp);
            if (lane == 0) { seg_val[sg] = sv; seg_pos[sg] = sp; }
        }
        __syncthreads();
    }
}

}  // namespace

namespace {

struct DensityScratch {
    size_t s_fix, d_fix, feat_cnt, feat_id, feat_w, skip, total;
};
DensityScratch density_scratch(int Q, int64_t L, int n_layers, int d_sae, int nk)
{
    const size_t q = static_cast<size_t>(Q), l = static_cast<size_t>(L), nl = static_cast<size_t>(n_layers);
    const size_t n_tiles = (l + POS_TILE - 1) / POS_TILE;
    DensityScratch d;
    size_t o = 0;
    d.s_fix = o;    o += round_up(q * l * 8, 256);
    d.d_fix = o;    o += round_up(q * l * 8, 256);
    d.feat_w = o;   o += round_up(nl * q * nk * 8, 256);
    d.feat_id = o;  o += round_up(nl * q * nk * 4, 256);
    d.feat_cnt = o; o += round_up(nl * q * 4, 256);
    d.skip = o;     o += round_up(nl * static_cast<size_t>(d_sae) * (n_tiles + 1) * 4, 256);
    d.total = o;
    return d;
}

}  // namespace

size_t density_workspace_bytes(int Q, int64_t L, int n_layers, int d_sae, int nq, int k)
{
    return density_scratch(Q, L, n_layers, d_sae, nq * k).total;
}

s3_status launch_density(const s3_csr_view* h_layers, int n_layers, int d_sae, int64_t L, const int32_t* d_q_ids,
                         const float* d_q_vals, int Q, int nq, int k, int conv_kernel, int nms_radius, int n_centers,
                         int64_t stop_freq, int32_t* d_centers, float* d_center_density, float* d_s_out, float* d_d_out,
                         void* d_scratch, cudaStream_t stream)
{
    static int max_smem_dev[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    int max_smem = dev < 64 ? max_smem_dev[dev] : 0;
    if (max_smem == 0) {
        S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        S3_CUDA_TRY(cudaFuncSetAttribute(density_features_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        S3_CUDA_TRY(cudaFuncSetAttribute(density_accumulate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        S3_CUDA_TRY(cudaFuncSetAttribute(density_peaks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem - 1024));
        if (dev < 64) max_smem_dev[dev] = max_smem;
    }
    int seg_shift = MIN_SEG_SHIFT;
    while (((L + (1ll << seg_shift) - 1) >> seg_shift) > MAX_SEGS) ++seg_shift;
    S3_REQUIRE(conv_kernel <= MAX_CONV_KERNEL, S3_ERR_UNSUPPORTED, "conv_kernel = %d exceeds %d", conv_kernel, MAX_CONV_KERNEL);
    ScoreLayers layers;
    for (int l = 0; l < n_layers; ++l) layers.v[l] = h_layers[l];
    const DensityScratch sc = density_scratch(Q, L, n_layers, d_sae, nq * k);
    unsigned char* base = static_cast<unsigned char*>(d_scratch);
    DensityArgs a;
    a.q_ids = d_q_ids; a.q_vals = d_q_vals;
    a.s_fix = reinterpret_cast<long long*>(base + sc.s_fix);
    a.d_fix = reinterpret_cast<long long*>(base + sc.d_fix);
    a.feat_cnt = reinterpret_cast<int32_t*>(base + sc.feat_cnt);
    a.feat_id = reinterpret_cast<int32_t*>(base + sc.feat_id);
    a.feat_w = reinterpret_cast<long long*>(base + sc.feat_w);
    a.skip = reinterpret_cast<uint32_t*>(base + sc.skip);
    a.centers = d_centers; a.center_density = d_center_density; a.s_out = d_s_out; a.d_out = d_d_out;
    a.L = L; a.n_layers = n_layers; a.d_sae = d_sae; a.Q = Q; a.nk = nq * k;
    int npad = 32;
    while (npad < a.nk) npad <<= 1;
    a.npad = npad; a.conv_kernel = conv_kernel; a.nms_radius = nms_radius; a.n_centers = n_centers; a.stop_freq = stop_freq;
    a.seg_shift = seg_shift;
    a.n_tiles = static_cast<int>((L + POS_TILE - 1) / POS_TILE);

    const size_t smem_feat = score_smem(a.nk, npad, 0, true).total;
    S3_REQUIRE(smem_feat + 2048 <= static_cast<size_t>(max_smem), S3_ERR_UNSUPPORTED, "nq*k = %d needs %zu bytes of shared memory", a.nk,
               smem_feat);
    density_features_kernel<<<dim3(Q, n_layers), ST, smem_feat, stream>>>(layers, a);
    if (a.n_tiles > 0) {
        const long long per_layer = (long long)d_sae * (a.n_tiles + 1);
        const long long want = (per_layer + ST - 1) / ST;
        const int cap = device_sm_count() * 16;
        density_skip_kernel<<<dim3(static_cast<unsigned>(want < cap ? want : cap), n_layers), ST, 0, stream>>>(layers, a);
        const size_t smem_acc = static_cast<size_t>(POS_TILE) * 8 + FCHUNK * (8 + 8 + 4) + (FCHUNK + 4) * 4 + AWIN * 2;
        density_accumulate_kernel<<<dim3(a.n_tiles, Q), ST, smem_acc, stream>>>(layers, a);
    }
    const size_t smem_peaks = 2 * MAX_SEGS * 8 + static_cast<size_t>(CONV_TILE + MAX_CONV_KERNEL) * 8;
    density_peaks_kernel<<<Q, ST, smem_peaks, stream>>>(a);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace s3
