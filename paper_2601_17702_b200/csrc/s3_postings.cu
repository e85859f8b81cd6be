// Per-chunk CSR posting lists (Sec. 3.4, Eq. 4: I[f] <- I[f] U {t} for every f in F_t).
//
// A chunk-layer ("item") is cut into runs of consecutive tokens, one thread block per run, so that a
// launch over a handful of items still fills the GPU. Four small kernels, all integer, no inter-block
// waiting:
//   1. count    block (item, run): histogram of the run's ids in shared memory -> table[run][f]
//   2. colscan  thread per feature: exclusive prefix of table[.][f] down the runs (in place) and the
//               feature's total (its list length) -> row_ptr[f]
//   3. rowscan  block per item: in-place exclusive scan of row_ptr[0..d_sae), total -> row_ptr[d_sae]
//   4. scatter  block (item, run): cursor[f] = row_ptr[f] + table[run][f] in shared memory, then the
//               run's tokens in order, 64 at a time: every pair takes a ticket from its feature's
//               counter; a feature hit once in the 64 tokens writes straight to cursor[f]; a feature
//               hit several times records the hitting tokens in a 64-bit mask (small hash table), and
//               each of its pairs ranks itself by counting the mask bits below its own token.
// Every list therefore comes out in ascending position whatever the block scheduling, and the result
// is bit-identical from run to run. Features are handled in ranges of 32768 per pass (one pass for
// the usual dictionary sizes).
#include "s3_common.cuh"
#include "s3_kernels.cuh"

namespace s3 {

namespace {

constexpr int PT = 1024;            // threads per block
constexpr int PER = 4;              // pairs per thread per sub-tile
constexpr int SUB_PAIRS = PT * PER; // pairs per sub-tile
constexpr int SUB_TOK = 64;         // tokens per sub-tile at most (one mask bit each)
constexpr int RANGE = 32768;        // features per pass
constexpr int HASH = 4096;          // mask slots (at most SUB_PAIRS/2 features can be hit twice)
constexpr int MAX_BLOCKS_TOTAL = 1024;

struct PostingsPlan {
    s3_postings_item items[S3_MAX_POSTINGS_ITEMS];
    unsigned long long table_off[S3_MAX_POSTINGS_ITEMS];   // byte offset of the item's table in the workspace
    int blk_start[S3_MAX_POSTINGS_ITEMS + 1];              // first block of each item in the flattened grid
    int tok_per_blk[S3_MAX_POSTINGS_ITEMS];
    int wide[S3_MAX_POSTINGS_ITEMS];                       // table entries are 32-bit (else 16-bit)
    int n_items;
    unsigned char* ws;
    uint32_t* status;
};

__device__ __forceinline__ int find_item(const PostingsPlan& pl, int blk)
{
    int it = 0;
    while (it + 1 < pl.n_items && blk >= pl.blk_start[it + 1]) ++it;
    return it;
}

__device__ __forceinline__ uint32_t table_get(const unsigned char* tab, bool wide, size_t idx)
{
    return wide ? reinterpret_cast<const uint32_t*>(tab)[idx] : reinterpret_cast<const uint16_t*>(tab)[idx];
}
__device__ __forceinline__ void table_put(unsigned char* tab, bool wide, size_t idx, uint32_t v)
{
    if (wide) reinterpret_cast<uint32_t*>(tab)[idx] = v;
    else reinterpret_cast<uint16_t*>(tab)[idx] = static_cast<uint16_t>(v);
}

// ---- 1. per-run histograms -------------------------------------------------------------------------
__global__ void __launch_bounds__(PT)
postings_count_kernel(const __grid_constant__ PostingsPlan pl)
{
    extern __shared__ uint32_t hist[];       // [min(d_sae, RANGE)]
    const int item = find_item(pl, blockIdx.x);
    const s3_postings_item& it = pl.items[item];
    const int run = blockIdx.x - pl.blk_start[item];
    const int tid = threadIdx.x;
    const int d_sae = it.d_sae, k = it.k;
    const int t_lo = run * pl.tok_per_blk[item];
    const int t_hi = min(it.T, t_lo + pl.tok_per_blk[item]);
    const int64_t p_lo = (int64_t)t_lo * k, p_hi = (int64_t)t_hi * k;
    const int32_t* __restrict__ ids = it.d_ids;
    unsigned char* tab = pl.ws + pl.table_off[item];
    const bool wide = pl.wide[item] != 0;

    for (int f0 = 0; f0 < d_sae; f0 += RANGE) {
        const int nf = min(RANGE, d_sae - f0);
        for (int f = tid; f < nf; f += PT) hist[f] = 0;
        __syncthreads();
        for (int64_t p = p_lo + tid; p < p_hi; p += 4 * PT) {
            int32_t f[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) f[j] = (p + (int64_t)j * PT < p_hi) ? __ldg(ids + p + (int64_t)j * PT) : -1;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (f[j] < 0) continue;
                if (f[j] >= d_sae) { if (f0 == 0) dev_set_error(pl.status, DEV_BAD_FEATURE_ID); }
                else if (f[j] >= f0 && f[j] < f0 + nf) atomicAdd(&hist[f[j] - f0], 1u);
            }
        }
        __syncthreads();
        for (int f = tid; f < nf; f += PT) table_put(tab, wide, (size_t)run * d_sae + f0 + f, hist[f]);
        __syncthreads();
    }
}

// ---- 2. per-feature prefix over the runs ---------------------------------------------------------------
// Thread per feature. The runs are taken eight at a time: eight independent loads, a prefix in
// registers, eight stores, so that the memory round trips of a column overlap.
template <typename E>
__device__ __forceinline__ uint32_t colscan_column(E* col, size_t pitch, int n_runs)
{
    uint32_t run_sum = 0;
    for (int r0 = 0; r0 < n_runs; r0 += 8) {
        uint32_t c[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) c[j] = (r0 + j < n_runs) ? static_cast<uint32_t>(col[(size_t)(r0 + j) * pitch]) : 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (r0 + j < n_runs) col[(size_t)(r0 + j) * pitch] = static_cast<E>(run_sum);
            run_sum += c[j];
        }
    }
    return run_sum;
}

__global__ void __launch_bounds__(256)
postings_colscan_kernel(const __grid_constant__ PostingsPlan pl)
{
    const int item = blockIdx.y;
    const s3_postings_item& it = pl.items[item];
    const int f = blockIdx.x * 256 + threadIdx.x;
    if (f >= it.d_sae) return;
    const int n_runs = pl.blk_start[item + 1] - pl.blk_start[item];
    unsigned char* tab = pl.ws + pl.table_off[item];
    const uint32_t total = pl.wide[item] ? colscan_column(reinterpret_cast<uint32_t*>(tab) + f, it.d_sae, n_runs)
                                         : colscan_column(reinterpret_cast<uint16_t*>(tab) + f, it.d_sae, n_runs);
    it.d_row_ptr[f] = total;             // list length for now; the row scan turns it into the offset
}

// ---- 3. row_ptr = exclusive scan of the list lengths, in place ------------------------------------------------
// One block per item walks the array in tiles of 1024 consecutive entries (coalesced): warp scans, a scan of
// the 32 warp sums, and a running carry from tile to tile.
__global__ void __launch_bounds__(PT)
postings_rowscan_kernel(const __grid_constant__ PostingsPlan pl)
{
    __shared__ uint32_t warp_sums[2][33];
    const s3_postings_item& it = pl.items[blockIdx.x];
    uint32_t* rp = it.d_row_ptr;
    const int n = it.d_sae;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t carry = 0;
    int buf = 0;
    uint32_t v_next = threadIdx.x < n ? rp[threadIdx.x] : 0u;
    for (int i0 = 0; i0 < n; i0 += PT, buf ^= 1) {
        const int i = i0 + threadIdx.x;
        const uint32_t v = v_next;
        v_next = (i + PT < n) ? rp[i + PT] : 0u;            // next tile's load overlaps this tile's scan
        uint32_t inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += u;
        }
        if (lane == 31) warp_sums[buf][warp] = inc;
        __syncthreads();
        uint32_t w = warp_sums[buf][lane];                   // every warp scans the 32 warp sums itself
        uint32_t winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += u;
        }
        const uint32_t before_warp = __shfl_sync(0xffffffffu, winc - w, warp);
        const uint32_t tile_total = __shfl_sync(0xffffffffu, winc, 31);
        if (i < n) rp[i] = carry + before_warp + inc - v;
        carry += tile_total;
    }
    if (threadIdx.x == 0) rp[n] = carry;
}

// ---- 4. ordered scatter ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t hash_feature(uint32_t f) { return (f * 2654435761u) >> 20; }   // 12 bits

__global__ void __launch_bounds__(PT)
postings_scatter_kernel(const __grid_constant__ PostingsPlan pl)
{
    extern __shared__ uint32_t smem_u32[];
    // cursor[nf] | tick[nf/4 + 1] (one byte per feature) | hkey[HASH] | hbits[2*HASH]
    const int item = find_item(pl, blockIdx.x);
    const s3_postings_item& it = pl.items[item];
    const int run = blockIdx.x - pl.blk_start[item];
    const int tid = threadIdx.x;
    const int d_sae = it.d_sae, k = it.k;
    const int nf_max = min(RANGE, d_sae);
    uint32_t* cursor = smem_u32;
    uint32_t* tick = cursor + nf_max;
    uint32_t* hkey = tick + (nf_max + 3) / 4 + 1;
    uint32_t* hbits = hkey + HASH;

    const int t_lo = run * pl.tok_per_blk[item];
    const int t_hi = min(it.T, t_lo + pl.tok_per_blk[item]);
    const int32_t* __restrict__ ids = it.d_ids;
    const unsigned char* tab = pl.ws + pl.table_off[item];
    const bool wide = pl.wide[item] != 0;
    const bool has_val = it.d_vals != nullptr && it.d_pval != nullptr;
    int sub_tok = SUB_PAIRS / k;
    sub_tok = sub_tok < 1 ? 1 : (sub_tok > SUB_TOK ? SUB_TOK : sub_tok);

    for (int i = tid; i < HASH; i += PT) { hkey[i] = 0; hbits[2 * i] = 0; hbits[2 * i + 1] = 0; }

    for (int f0 = 0; f0 < d_sae; f0 += RANGE) {
        const int nf = min(RANGE, d_sae - f0);
        for (int f = tid; f < nf; f += PT)
            cursor[f] = it.d_row_ptr[f0 + f] + table_get(tab, wide, (size_t)run * d_sae + f0 + f);
        for (int f = tid; f < (nf + 3) / 4 + 1; f += PT) tick[f] = 0;
        __syncthreads();

        for (int ts = t_lo; ts < t_hi; ts += sub_tok) {
            const int n_tok = min(sub_tok, t_hi - ts);
            const int n_pairs = n_tok * k;
            const int64_t p0 = (int64_t)ts * k;
            int lf[PER];          // feature relative to f0, -1 = nothing to do
            uint32_t tk[PER];     // ticket within the sub-tile
            int tau[PER];         // token offset within the sub-tile
            // tickets
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                const int q = tid + j * PT;
                lf[j] = -1;
                if (q < n_pairs) {
                    const int32_t f = __ldg(ids + p0 + q);
                    if (f >= f0 && f < f0 + nf) {
                        lf[j] = f - f0;
                        tau[j] = q / k;
                        const int sh = 8 * (lf[j] & 3);
                        tk[j] = (atomicAdd(&tick[lf[j] >> 2], 1u << sh) >> sh) & 0xFFu;
                    }
                }
            }
            __syncthreads();
            // single hits write now; multiple hits publish their token in the feature's mask
            uint32_t m[PER], slot[PER];
            bool any_multi = false;
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                if (lf[j] < 0) continue;
                m[j] = (tick[lf[j] >> 2] >> (8 * (lf[j] & 3))) & 0xFFu;
                if (m[j] == 1) {
                    const uint32_t c = cursor[lf[j]];
                    it.d_pos[c] = (int32_t)(it.pos_base + ts + tau[j]);
                    if (has_val) it.d_pval[c] = it.d_vals[p0 + tid + j * PT];
                } else {
                    any_multi = true;
                    uint32_t h = hash_feature((uint32_t)lf[j]);
                    const uint32_t want = (uint32_t)lf[j] + 1u;
                    for (int probe = 0; probe < HASH; ++probe) {      // the table cannot fill up: <= HASH/2 keys
                        const uint32_t old = atomicCAS(&hkey[h], 0u, want);
                        if (old == 0u || old == want) break;
                        h = (h + 1) & (HASH - 1);
                    }
                    slot[j] = h;
                    atomicOr(&hbits[2 * h + (tau[j] >> 5)], 1u << (tau[j] & 31));
                }
            }
            const int multi = __syncthreads_or(any_multi ? 1 : 0);
            if (multi) {
#pragma unroll
                for (int j = 0; j < PER; ++j) {
                    if (lf[j] < 0 || m[j] == 1) continue;
                    const uint32_t b0 = hbits[2 * slot[j]], b1 = hbits[2 * slot[j] + 1];
                    const uint32_t rank = tau[j] < 32 ? __popc(b0 & ((1u << tau[j]) - 1u))
                                                      : __popc(b0) + __popc(b1 & ((1u << (tau[j] - 32)) - 1u));
                    const uint32_t c = cursor[lf[j]] + rank;
                    it.d_pos[c] = (int32_t)(it.pos_base + ts + tau[j]);
                    if (has_val) it.d_pval[c] = it.d_vals[p0 + tid + j * PT];
                }
                __syncthreads();
            }
            // the first ticket holder of each feature advances the cursor and clears the counters
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                if (lf[j] < 0) continue;
                if (tk[j] == 0) {
                    cursor[lf[j]] += m[j];
                    atomicSub(&tick[lf[j] >> 2], m[j] << (8 * (lf[j] & 3)));
                }
                if (m[j] != 1) { hkey[slot[j]] = 0; hbits[2 * slot[j]] = 0; hbits[2 * slot[j] + 1] = 0; }
            }
            __syncthreads();
        }
    }
}

size_t table_bytes(int T, int d_sae, int n_runs)
{
    const size_t entry = T > 65535 ? 4 : 2;
    return round_up((size_t)n_runs * d_sae * entry, 256);
}

int runs_for(int T, int tok_per_blk) { return T > 0 ? (T + tok_per_blk - 1) / tok_per_blk : 0; }

}  // namespace

// Tokens per block such that the launch has about two blocks per SM over all items, at least one
// 64-token sub-tile each, and no more than MAX_BLOCKS_TOTAL blocks in all.
static int plan_tokens_per_block(const s3_postings_item* items, int n_items, int target_blocks)
{
    int64_t total = 0;
    for (int i = 0; i < n_items; ++i) total += items[i].T;
    int64_t tpb = (total + target_blocks - 1) / (target_blocks > 0 ? target_blocks : 1);
    if (tpb < SUB_TOK) tpb = SUB_TOK;
    tpb = (tpb + SUB_TOK - 1) / SUB_TOK * SUB_TOK;
    while (true) {
        int64_t blocks = 0;
        for (int i = 0; i < n_items; ++i) blocks += runs_for(items[i].T, (int)tpb);
        if (blocks <= MAX_BLOCKS_TOTAL) break;
        tpb *= 2;
    }
    return (int)tpb;
}

size_t postings_workspace_bytes(int T, int k, int d_sae)
{
    (void)k;
    if (T <= 0 || d_sae <= 0) return 0;
    // the plan of a batch never uses fewer than SUB_TOK tokens per block, nor more than MAX_BLOCKS_TOTAL blocks
    int runs = runs_for(T, SUB_TOK);
    if (runs > MAX_BLOCKS_TOTAL) runs = MAX_BLOCKS_TOTAL;
    return table_bytes(T, d_sae, runs);
}

s3_status launch_postings(const s3_postings_item* h_items, int n_items, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    static bool attr_set[64] = {};
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 64 && !attr_set[dev]) {
        S3_CUDA_TRY(cudaFuncSetAttribute(postings_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, RANGE * 4));
        S3_CUDA_TRY(cudaFuncSetAttribute(postings_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         RANGE * 4 + RANGE + 16 + HASH * 12));
        attr_set[dev] = true;
    }
    PostingsPlan pl;
    pl.n_items = n_items;
    pl.ws = static_cast<unsigned char*>(d_ws);
    pl.status = static_cast<uint32_t*>(d_ws);
    const int tpb = plan_tokens_per_block(h_items, n_items, 2 * device_sm_count());
    size_t off = S3_WS_HEADER_BYTES;
    int blocks = 0, max_d = 0, max_tiles = 0;
    for (int i = 0; i < n_items; ++i) {
        pl.items[i] = h_items[i];
        pl.tok_per_blk[i] = tpb;
        pl.blk_start[i] = blocks;
        const int runs = runs_for(h_items[i].T, tpb);
        blocks += runs;
        pl.wide[i] = h_items[i].T > 65535 ? 1 : 0;
        off = round_up(off, 256);
        pl.table_off[i] = off;
        off += table_bytes(h_items[i].T, h_items[i].d_sae, runs);
        if (h_items[i].d_sae > max_d) max_d = h_items[i].d_sae;
        const int tiles = (h_items[i].d_sae + 255) / 256;
        if (tiles > max_tiles) max_tiles = tiles;
    }
    pl.blk_start[n_items] = blocks;
    S3_REQUIRE(off <= ws_bytes, S3_ERR_CAPACITY, "postings workspace holds %zu bytes, %zu needed", ws_bytes, off);
    const int nf = max_d < RANGE ? max_d : RANGE;
    if (blocks > 0) {
        postings_count_kernel<<<blocks, PT, (size_t)nf * 4, stream>>>(pl);
        S3_CUDA_TRY(cudaGetLastError());
    }
    postings_colscan_kernel<<<dim3(max_tiles, n_items), 256, 0, stream>>>(pl);
    S3_CUDA_TRY(cudaGetLastError());
    postings_rowscan_kernel<<<n_items, PT, 0, stream>>>(pl);
    S3_CUDA_TRY(cudaGetLastError());
    if (blocks > 0) {
        const size_t smem = (size_t)nf * 4 + ((size_t)(nf + 3) / 4 + 1) * 4 + (size_t)HASH * 12;
        postings_scatter_kernel<<<blocks, PT, smem, stream>>>(pl);
        S3_CUDA_TRY(cudaGetLastError());
    }
    return S3_OK;
}

}  // namespace s3
