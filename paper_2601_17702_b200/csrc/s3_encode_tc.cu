// bf16 SAE encode + ReLU + Top-k candidate selection (Sec. 3.3, Eq. 1-2) on the sm_100a tensor cores.
//
//   pre[t,f] = sum_i x[t,i] * W_enc[i,f] + b_eff[f],   b_eff = b_enc - W_enc^T b_dec   (folded once)
//
// Persistent, warp-specialised kernel; the two CTAs of a cluster (one per SM) work as a pair on 256-token x
// 256-feature tiles:
//   warp 0      TMA producer: per k-block each CTA streams its 128 tokens of x and its half of the tile's 256
//               rows of W_enc^T (K-major, 128-byte swizzle) into a ring of shared-memory stages; all copies of
//               a stage are counted on the first CTA's mbarrier;
//   warp 1      MMA issuer (first CTA only): one thread issues tcgen05.mma.cta_group::2 (M=256 over the pair,
//               N=256, K=16, bf16 x bf16 -> fp32) into one of two 256-column accumulators in each CTA's tensor
//               memory; tcgen05.commit, multicast to both CTAs, frees the stage / publishes the accumulator;
//   warps 2..   epilogue, four warps per group, one or two groups (template parameter GROUPS; two groups split a
//               tile's columns): thread = token row (TMEM lane). Each 32-column batch is read with tcgen05.ld,
//               biased and compared with the row's bound, a value that at least k pre-activations of the row are
//               known to exceed. Survivors go, branch-free, to a short pending list in shared memory. When some
//               lane's list is nearly full the warp folds its lists: each survivor is appended to the row's
//               candidate list in global memory and counted in a small per-row histogram over the float's
//               exponent and top mantissa bits; as soon as k survivors lie in buckets above the bound's bucket,
//               the bound moves up to the next bucket edge. It therefore tracks the row's running k-th largest
//               value to within one bucket (about 4 %) at a few instructions per survivor, and no ordered
//               structure is kept on the SM.
// A work unit is a run of column tiles of one 256-token row tile of one encoder call (up to 8 calls per launch).
// The host cuts the launch into units (build_schedule): shares of equal modelled duration per CTA pair for
// encoders whose weights stay in L2, bands of row tiles swept by uniform column slices in step for wider ones,
// whole (row tile, slice) units otherwise; the units travel in the launch parameters. Every unit keeps its own
// candidate list per row and epilogue group. Bounds are shared: a bound that k values of one list exceed holds for
// the whole row, so a list announces its bound whenever it rises (to the other group through shared memory, to
// the row's other pieces through a per-row word in global memory) and every list drops what does not beat the
// best bound it has seen. The lists, a few hundred keys per row, are reduced to the exact Top-k by the merge
// kernel (s3_topk_merge.cu), which first drops everything not above the row's best bound. Only candidates leave
// the SM (as 64-bit keys); the pre-activation matrix is never written to memory.
//
// A candidate list that would overflow is first compacted against the current bound and, if that does not free
// enough room (many nearly equal values), cut down to its exact k largest keys.
//
// The same pipeline serves two more epilogues: DENSE writes the pre-activations themselves (the upstream
// projections), PROJ computes a head's projection into shared memory first and encodes from there.
//
// Every mbarrier wait is bounded; a wait that runs out records which one in the workspace status word, raises a
// CTA-wide abort flag, and the CTA drains its own TMA copies, frees its tensor memory and exits.
#include <cuda.h>
#include <cuda_bf16.h>
#include <string.h>
#include <vector>

#include "s3_kernels.cuh"
#include "s3_topk.cuh"

namespace s3 {

namespace {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int PAIR_M = 2 * BM;                      // tokens per tile over the CTA pair
constexpr int A_STAGE_BYTES = BM * BK * 2;         // 16 KB: this CTA's 128 tokens
constexpr int B_STAGE_BYTES = (BN / 2) * BK * 2;   // 16 KB: this CTA's half of the tile's 256 features
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;   // per CTA; a stage is complete after twice that
// Epilogue warp groups (template parameter GROUPS of the kernel): each group of four warps takes 256 / GROUPS columns of
// every tile, with its own histogram and candidate list per row; the groups tell each other the bounds they reach (a bound
// that k values of one list exceed holds for the whole row), so together they gather hardly more survivors than one list
// would. One group serves encoders whose tiles keep the tensor pipe busy longer than the filter takes (d_in > 1024); two
// groups serve the others, where the filter of a single warp per scheduler is the bottleneck and a second warp hides its
// latencies (d_in 128, k 32: 1.73 -> 1.22 ms; d_in 512, k 16, eight layers: 1.89 -> 1.54 ms; d_in 1024, k 32: 0.289 ->
// 0.274 ms once the bounds are shared; before that two groups were slower there).
constexpr int MAX_EPI_GROUPS = 2;
constexpr int kTwoGroupsMaxDin = 1024;         // encoders at most this wide run with two epilogue groups
constexpr int TMEM_COLS = 512;
constexpr int BATCH = 32;                    // columns per tcgen05.ld
constexpr int STEP = 8;                      // columns filtered between two checks of the pending lists
// Pending-list slots per row, chosen per launch: more slots mean fewer, fuller folds (k = 128 on 128-wide encoders: 2.10
// -> 1.94 ms with 24) but, with two epilogue groups, one pipeline stage less (16 KB per group at 16 slots, 24 KB at 24),
// which costs the eight 512-wide k = 16 layers 2.6 %. Launches with k >= 32 take 24, the others 16.
constexpr int PEND_CAP_MIN = 2 * STEP, PEND_CAP_MAX = 3 * STEP;
__host__ __device__ inline int pend_cap_for(int max_k) { return max_k >= 32 ? PEND_CAP_MAX : PEND_CAP_MIN; }
constexpr int NB = 64;                       // histogram buckets per row
#ifndef S3_FOLD_CHUNK
#define S3_FOLD_CHUNK 4
#endif
constexpr int FOLD_CHUNK = S3_FOLD_CHUNK;    // pending entries a fold handles per step
constexpr int COLD_LEVELS = 3;                // trial bounds of the cold-start pass, as fractions of the first batch's maximum
__device__ constexpr float kColdFraction[COLD_LEVELS] = {0.60f, 0.40f, 0.20f};      // six or eight levels cost more than they save (about 1 %)
constexpr int HSHIFT = 19;                   // bucket = float bits >> 19: 16 buckets per octave
constexpr uint32_t WAIT_LIMIT = 1u << 26;    // try_wait polls before a wait is declared dead (~1 s)

// ---- PTX wrappers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait. Returns false if the wait ran out or another role already aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag)
{
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    return false;
}

__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Cluster-wide barrier over all threads of both CTAs.
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in the cluster's CTA `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
// Arrival on a barrier of the first CTA (cluster address). The default CTA-scope release is enough: what the waiting
// MMA warp must not overtake are this thread's tensor-memory loads, which tcgen05.wait::ld and the tcgen05 fences
// order; a cluster-scope release would also make every thread wait here for its outstanding global stores.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// The same with a cluster-scope release: what the arriving thread wrote to its own shared memory (made visible to the
// asynchronous proxy with fence.proxy.async first) is ordered before the other CTA's waiter.
__device__ __forceinline__ void mbar_arrive_cluster_release(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Bounded wait with a cluster-scope acquire (the barrier is signalled by threads of both CTAs).
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag)
{
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    return false;
}

// Tile load of one CTA of the pair into its own shared memory; the bytes are counted on the mbarrier at
// cluster address `bar_addr` (the first CTA's), which the .cta_group::2 form allows to lie in the peer CTA.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_addr)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Arrives, once the MMAs issued so far have completed, on the mbarrier at this shared-memory offset in
// both CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar)
{
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                     smem_u32(bar)),
                 "h"(both)
                 : "memory");
}

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, 128-byte rows, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr >> 4) & 0x3FFFu);        // start address
    d |= static_cast<uint64_t>(1) << 16;                        // leading byte offset (unused for swizzled K-major)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                // stride byte offset between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                        // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                        // 128-byte swizzle
    return d;
}

// Instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, N = 256, M = 256 (over the CTA pair).
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                                (static_cast<uint32_t>(PAIR_M >> 4) << 24);

// The same with N = 128: the upstream projection of one head (d_head = 128 output columns).
constexpr int PROJ_N = 128;
constexpr uint32_t kInstrDescN128 = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(PROJ_N >> 3) << 17) |
                                    (static_cast<uint32_t>(PAIR_M >> 4) << 24);
constexpr int M_SELECT = 0, M_DENSE = 1, M_PROJ = 2;   // epilogue modes of the kernel

constexpr int MAX_GROUP = S3_MAX_ENCODE_ITEMS;   // encoders one launch can serve
constexpr int MAX_SCHED = 2048;                  // work units a launch can deal out by table
constexpr int MAX_PAIRS = 96;                    // CTA pairs the table has room for

// One work unit of a table-driven launch: column tiles [tile_lo, tile_hi) of row tile mt of an item; its survivors go
// to candidate list `slot` of the rows.
struct UnitDesc {
    uint16_t mt, tile_lo, tile_hi;
    uint8_t item, slot;
};

// One encoder call of a grouped launch.
struct ItemParams {
    int T, d_in, k, kblocks;
    int n_mtiles, n_col_tiles, n_slices;
    int unit_start;            // first work unit of this item in the launch's flattened unit list
    uint32_t cap;              // candidate-list slots per (token, slice)
    const float* b_eff;
    uint64_t* cand;            // [T][n_slices][cap]
    uint32_t* counts;          // [T][n_slices]
    uint32_t* hint;            // [T] float bits of the best published bound
};

struct EncodeTcParams {
    int n_items, n_units, n_stages;
    int pend_cap;              // pending-list slots per row (shared memory)
    int use_sched;             // 1: pair p runs units unit[pair_start[p] .. pair_start[p+1]); 0: units p, p + n_pairs, ...
    uint32_t* status;
    void* dense_out;           // dense mode (one item): the pre-activations [T, ld_out], fp32 or bf16
    long long ld_out;
    int out_bf16, d_sae;
    // projection mode (one item): the encoder's input is one head of x = h W_proj + b, computed by the same CTA pair just
    // before the head's tiles. Units are (row tile, head); outputs are indexed by row = token * heads + head.
    int proj_heads, proj_kblocks;      // heads (0 = no projection), k-blocks of the projection's inner dimension
    const float* proj_bias;            // [heads * 128]
    ItemParams item[MAX_GROUP];
    uint16_t pair_start[MAX_PAIRS + 1];
    UnitDesc unit[MAX_SCHED];
};

struct TensorMaps {
    CUtensorMap x[MAX_GROUP];
    CUtensorMap w[MAX_GROUP];
    CUtensorMap wk;                    // projection mode: W_proj^T [heads * 128, d_model], box of 64 rows
};

// The units of one CTA pair, in the order every role of both CTAs walks them.
struct UnitWalk {
    int i, end, step;
};
__device__ __forceinline__ UnitWalk unit_walk(const EncodeTcParams& p, int pair, int n_pairs)
{
    UnitWalk w;
    if (p.use_sched) { w.i = p.pair_start[pair]; w.end = p.pair_start[pair + 1]; w.step = 1; }
    else { w.i = pair; w.end = p.n_units; w.step = n_pairs; }
    return w;
}
// Unit -> item, candidate-list slot ("slice"), row tile and the column tiles [tile_lo, tile_hi) it covers.
struct Unit {
    int item, slice, mt, tile_lo, tile_hi;
    int head;              // projection mode: the head whose projection the unit computes first (0 otherwise)
};
__device__ __forceinline__ Unit unit_decode(const EncodeTcParams& p, const UnitWalk& w)
{
    Unit u;
    if (p.use_sched) {
        const UnitDesc d = p.unit[w.i];
        u.item = d.item; u.slice = d.slot; u.mt = d.mt; u.tile_lo = d.tile_lo; u.tile_hi = d.tile_hi;
        u.head = 0;
        if (p.proj_heads > 0) {        // the table's row index runs over (row tile, head)
            u.mt = d.mt / p.proj_heads;
            u.head = d.mt - u.mt * p.proj_heads;
        }
        return u;
    }
    u.head = 0;
    if (p.proj_heads > 0) {            // (row tile, head), heads of a row tile next to each other: they share the tile of h
        u.item = 0;
        u.mt = w.i / p.proj_heads;
        u.head = w.i - u.mt * p.proj_heads;
        u.slice = 0;
        u.tile_lo = 0; u.tile_hi = p.item[0].n_col_tiles;
        return u;
    }
    u.item = p.n_items - 1;
    while (u.item > 0 && p.item[u.item].unit_start > w.i) --u.item;
    const ItemParams& ip = p.item[u.item];
    const int local = w.i - ip.unit_start;
    u.slice = local / ip.n_mtiles;
    u.mt = local - u.slice * ip.n_mtiles;
    u.tile_lo = static_cast<int>(static_cast<int64_t>(u.slice) * ip.n_col_tiles / ip.n_slices);
    u.tile_hi = static_cast<int>(static_cast<int64_t>(u.slice + 1) * ip.n_col_tiles / ip.n_slices);
    return u;
}

// Shared-memory carve-up (all offsets from a 1024-byte aligned base).
struct SmemLayout {
    uint32_t a_off, b_off, x_off, pend_off, hist_off, xtau_off, bar_off, total;
};
constexpr int X_TILE_BYTES = 2 * A_STAGE_BYTES;    // projection mode: this CTA's 128 tokens x 128 projected columns, two k-blocks
__host__ __device__ inline SmemLayout smem_layout(int n_stages, bool proj, int groups, int pend_cap)
{
    const int EPI_THREADS = 128 * groups;
    SmemLayout L;
    L.a_off = 0;
    L.b_off = L.a_off + n_stages * A_STAGE_BYTES;
    L.x_off = L.b_off + n_stages * B_STAGE_BYTES;
    L.pend_off = L.x_off + (proj ? X_TILE_BYTES : 0);
    L.hist_off = L.pend_off + pend_cap * EPI_THREADS * 8;
    L.xtau_off = L.hist_off + NB * EPI_THREADS * 2;
    L.bar_off = L.xtau_off + BM * 16;
    L.total = L.bar_off + (2 * n_stages + 5) * 8 + 16;
    return L;
}

// Per-row selection state of an epilogue thread.
struct RowSel {
    float tau;          // candidates are values > tau
    float tau_floor;    // bound while the histogram has not moved yet (0, a published bound, or an exact k-th value)
    int hbase;          // bucket id of histogram slot 0 (-1: not chosen yet)
    int istar;          // histogram slot of the current bound
    uint32_t above;     // survivors counted in slots >= istar
    uint32_t gcnt;      // entries in the row's candidate list
    bool floor_exact;   // tau_floor is the value of the list's exact k-th key
    float ext;          // best bound learnt from the row's other lists (other column pieces, the other epilogue group)
    float cut;          // max(tau, ext): what a value must exceed to be kept
};

// The bound this list may announce: at least k of its values exceed it. An exact k-th value only bounds from below after
// stepping to the next float down.
__device__ __forceinline__ uint32_t announced_bound(const RowSel& r)
{
    uint32_t out = __float_as_uint(r.tau);
    if (r.istar == 0 && r.floor_exact && out > 0u) out -= 1u;
    return out;
}

// Rare path: the candidate list cannot take the pending entries. Drops what is not above the bound;
// if the list stays nearly full it keeps only its k largest keys and restarts the histogram from there.
// New entries always come from later columns than the list's, so after the exact cut a value equal to
// the k-th key's can no longer win (ties go to the lower id) and the strict comparison stays exact.
template <int EPI_THREADS>
__device__ __noinline__ void prune_list(uint64_t* glist, uint16_t* my_hist, RowSel& r, int k, uint32_t cap)
{
    uint32_t w = 0;
    for (uint32_t i = 0; i < r.gcnt; ++i) {
        const uint64_t key = glist[i];
        if (__uint_as_float(static_cast<uint32_t>(key >> 32)) > r.cut) glist[w++] = key;
    }
    r.gcnt = w;
    if (r.gcnt + PEND_CAP_MAX <= cap) return;
    for (int a = 0; a < k; ++a) {
        uint32_t best = a;
        uint64_t kb = glist[a];
        for (uint32_t b = a + 1; b < r.gcnt; ++b) {
            const uint64_t kk = glist[b];
            if (kk > kb) { kb = kk; best = b; }
        }
        const uint64_t tmp = glist[a];
        glist[a] = kb;
        glist[best] = tmp;
    }
    r.gcnt = k;
    const uint32_t vb = static_cast<uint32_t>(glist[k - 1] >> 32);
    r.tau_floor = r.tau = __uint_as_float(vb);
    r.cut = fmaxf(r.tau, r.ext);
    r.floor_exact = true;
#pragma unroll 1
    for (int s = 0; s < NB; ++s) my_hist[s * EPI_THREADS] = 0;
    my_hist[0] = static_cast<uint16_t>(k);
    r.hbase = static_cast<int>(vb >> HSHIFT);
    r.istar = 0;
    r.above = k;
}

// Folds the warp's pending lists (cnt entries per lane) into candidate lists and histograms, then
// raises each row's bound as far as the histogram allows. Called by all 32 lanes.
template <int EPI_THREADS>
__device__ __forceinline__ void fold_pending(uint64_t* __restrict__ my_pend, uint16_t* __restrict__ my_hist, uint64_t* __restrict__ glist,
                                             RowSel& r, int& cnt,
                                             int k, uint32_t cap)
{
    if (__any_sync(0xffffffffu, r.gcnt + cnt > cap)) {
        if (r.gcnt + cnt > cap) {
            RowSel t = r;            // the rare path works on a copy: the row's own state never has its address taken and stays in registers
            prune_list<EPI_THREADS>(glist, my_hist, t, k, cap);
            r = t;
        }
    }
    if (r.hbase < 0 && cnt > 0) {
        uint32_t ref = __float_as_uint(r.cut);
        if (ref == 0) {      // no bound yet: centre the window on the largest value seen so far
            for (int i = 0; i < cnt; ++i) {
                const uint32_t vb = static_cast<uint32_t>(my_pend[i * EPI_THREADS] >> 32);
                ref = vb > ref ? vb : ref;
            }
            const int b = static_cast<int>(ref >> HSHIFT) - NB / 2;
            r.hbase = b > 0 ? b : 0;
        } else {
            r.hbase = static_cast<int>(ref >> HSHIFT);
        }
    }
    const int nmax = __reduce_max_sync(0xffffffffu, cnt);
    // FOLD_CHUNK entries at a time: their loads first (those of the next chunk are issued before this chunk is worked on),
    // then the list stores, then the histogram, so that the shared-memory round trips overlap instead of forming one
    // dependent chain per entry
    uint64_t nxt[FOLD_CHUNK];
#pragma unroll
    for (int q = 0; q < FOLD_CHUNK; ++q) nxt[q] = (q < cnt) ? my_pend[q * EPI_THREADS] : 0ull;
    for (int i0 = 0; i0 < nmax; i0 += FOLD_CHUNK) {
        uint64_t key[FOLD_CHUNK];
        int idx[FOLD_CHUNK];
        bool ok[FOLD_CHUNK];
#pragma unroll
        for (int q = 0; q < FOLD_CHUNK; ++q) key[q] = nxt[q];
        if (i0 + FOLD_CHUNK < nmax) {
#pragma unroll
            for (int q = 0; q < FOLD_CHUNK; ++q) nxt[q] = (i0 + FOLD_CHUNK + q < cnt) ? my_pend[(i0 + FOLD_CHUNK + q) * EPI_THREADS] : 0ull;
        }
#pragma unroll
        for (int q = 0; q < FOLD_CHUNK; ++q) {
            const uint32_t vb = static_cast<uint32_t>(key[q] >> 32);
            ok[q] = (i0 + q < cnt) && __uint_as_float(vb) > r.cut;
            int ix = static_cast<int>(vb >> HSHIFT) - r.hbase;
            idx[q] = ix < 0 ? 0 : (ix > NB - 1 ? NB - 1 : ix);
        }
#pragma unroll
        for (int q = 0; q < FOLD_CHUNK; ++q)
            if (ok[q]) glist[r.gcnt++] = key[q];
        // one histogram update per run of equal buckets (survivors cluster in the buckets just above the bound)
        int run_idx = -1, run_n = 0;
#pragma unroll
        for (int q = 0; q < FOLD_CHUNK; ++q) {
            if (ok[q]) {
                if (idx[q] == run_idx) ++run_n;
                else {
                    if (run_n) my_hist[run_idx * EPI_THREADS] += static_cast<uint16_t>(run_n);
                    run_idx = idx[q]; run_n = 1;
                }
                r.above += 1;
            }
        }
        if (run_n) my_hist[run_idx * EPI_THREADS] += static_cast<uint16_t>(run_n);
    }
    cnt = 0;
    while (r.istar < NB - 1) {
        const uint32_t c = my_hist[r.istar * EPI_THREADS];
        if (r.above - c < static_cast<uint32_t>(k)) break;
        r.above -= c;
        ++r.istar;
    }
    if (r.istar == NB - 1) {
        // k survivors lie at or above the last slot's edge: restart the window there
        r.hbase += NB - 1;
#pragma unroll 1
        for (int s = 0; s < NB; ++s) my_hist[s * EPI_THREADS] = 0;
        my_hist[0] = static_cast<uint16_t>(r.above);
        r.istar = 0;
        r.tau_floor = __uint_as_float((static_cast<uint32_t>(r.hbase) << HSHIFT) - 1u);
        r.floor_exact = false;
    }
    // "value >= edge" is "value > the float just below the edge"
    r.tau = r.istar > 0 ? __uint_as_float((static_cast<uint32_t>(r.hbase + r.istar) << HSHIFT) - 1u) : r.tau_floor;
    r.cut = fmaxf(r.tau, r.ext);
}

// DENSE: the epilogue writes the pre-activations themselves (row-major, fp32 or bf16) instead of selecting; the rest of
// the kernel is the same pipeline.
template <int MODE, int GROUPS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(64 + 128 * GROUPS, 1)
encode_tc_kernel(const __grid_constant__ TensorMaps maps, const __grid_constant__ EncodeTcParams p)
{
    constexpr bool DENSE = MODE == M_DENSE, PROJ = MODE == M_PROJ;
    constexpr int EPI_GROUPS = GROUPS, EPI_THREADS = 128 * GROUPS;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const SmemLayout L = smem_layout(p.n_stages, PROJ, GROUPS, p.pend_cap);
    unsigned char* smem_a = smem + L.a_off;
    unsigned char* smem_b = smem + L.b_off;
    unsigned char* smem_x = smem + L.x_off;                // projection mode: the head's projected tile, the encode's A operand
    uint64_t* pend = reinterpret_cast<uint64_t*>(smem + L.pend_off);
    uint16_t* hist = reinterpret_cast<uint16_t*>(smem + L.hist_off);
    uint32_t* xtau32 = reinterpret_cast<uint32_t*>(smem + L.xtau_off);   // [unit number mod 4][row]: best bound of the row's lists
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L.bar_off);
    uint64_t* empty_bar = full_bar + p.n_stages;
    uint64_t* acc_full = empty_bar + p.n_stages;
    uint64_t* acc_empty = acc_full + 2;
    uint64_t* x_ready = acc_empty + 2;                     // projection mode: both CTAs' projected tiles are in shared memory
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(x_ready + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_cta_rank();          // 0 = first CTA of the pair: issues the MMAs, owns the
    const bool first_cta = cta_rank == 0;                  // barriers that both CTAs signal (full, acc_empty)
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        // full:      1 arrival (the first CTA's producer, with the byte count of both CTAs' copies)
        // empty:     1 arrival per CTA (tcgen05.commit, multicast)      acc_full: likewise
        // acc_empty: every epilogue thread of both CTAs, on the first CTA's barrier
        for (int s = 0; s < p.n_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 2 * EPI_THREADS); }
        for (int i = 0; i < 4 * BM; ++i) xtau32[i] = 0u;
        mbar_init(x_ready, 2 * EPI_THREADS);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // tensor memory of both SMs, allocated pairwise by the same warp of each CTA
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                                        // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            for (int j = 0; j < p.n_items; ++j) {
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&maps.x[j])) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&maps.w[j])) : "memory");
            }
            uint32_t stage = 0, phase = 0;
            uint64_t issued = 0;
            bool ok = true;
            for (UnitWalk uw = unit_walk(p, pair, n_pairs); uw.i < uw.end && ok; uw.i += uw.step) {
                const Unit un = unit_decode(p, uw);
                const int item = un.item, mt = un.mt, tile_lo = un.tile_lo, tile_hi = un.tile_hi;
                const ItemParams& ip = p.item[item];
                const CUtensorMap* map_x = &maps.x[item];
                const CUtensorMap* map_w = &maps.w[item];
                const int kblocks = ip.kblocks;
                const int row0 = mt * PAIR_M + static_cast<int>(cta_rank) * BM;        // this CTA's tokens
                if constexpr (PROJ) {
                    // the head's projection first: 128 tokens of h and this CTA's 64 of the head's 128 rows of W_proj^T per k-block
                    const int wrow0 = un.head * PROJ_N + static_cast<int>(cta_rank) * (PROJ_N / 2);
                    for (int kb = 0; kb < p.proj_kblocks; ++kb) {
                        if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag)) {
                            dev_set_error(p.status, DEV_TIMEOUT_SMEM_EMPTY);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        if (first_cta) mbar_expect_tx(&full_bar[stage], 2 * (A_STAGE_BYTES + B_STAGE_BYTES / 2));
                        const uint32_t full_addr = map_to_cta(smem_u32(&full_bar[stage]), 0);
                        tma_load_2d(smem_a + stage * A_STAGE_BYTES, map_x, kb * BK, row0, full_addr);
                        tma_load_2d(smem_b + stage * B_STAGE_BYTES, &maps.wk, kb * BK, wrow0, full_addr);
                        ++issued;
                        if (++stage == static_cast<uint32_t>(p.n_stages)) { stage = 0; phase ^= 1u; }
                    }
                }
                for (int nt = tile_lo; nt < tile_hi && ok; ++nt) {
                    const int col0 = nt * BN + static_cast<int>(cta_rank) * (BN / 2);  // this CTA's half of the features
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag)) {
                            dev_set_error(p.status, DEV_TIMEOUT_SMEM_EMPTY);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        if (first_cta) mbar_expect_tx(&full_bar[stage], PROJ ? 2 * B_STAGE_BYTES : 2 * STAGE_BYTES);
                        const uint32_t full_addr = map_to_cta(smem_u32(&full_bar[stage]), 0);
                        if (!PROJ) tma_load_2d(smem_a + stage * A_STAGE_BYTES, map_x, kb * BK, row0, full_addr);
                        tma_load_2d(smem_b + stage * B_STAGE_BYTES, map_w, kb * BK, col0, full_addr);
                        ++issued;
                        if (++stage == static_cast<uint32_t>(p.n_stages)) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            // Copies still in flight: the first CTA waits (bounded) until the last n_stages stages, its own and
            // the peer's halves, have landed; the peer stays resident until the closing cluster barrier.
            const uint64_t back = !first_cta ? 0 : (issued < static_cast<uint64_t>(p.n_stages) ? issued : static_cast<uint64_t>(p.n_stages));
            uint32_t s = stage, ph = phase;
            for (uint64_t i = 0; i < back; ++i) {
                if (s == 0) { s = p.n_stages - 1; ph ^= 1u; } else { --s; }
                for (uint32_t it = 0; it < WAIT_LIMIT; ++it)
                    if (mbar_try_wait(&full_bar[s], ph)) break;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (first CTA of the pair only) ----------------
        if (lane == 0 && first_cta) {
            uint32_t stage = 0, phase = 0;
            uint32_t tile_count = 0, unit_count = 0;
            bool ok = true;
            for (UnitWalk uw = unit_walk(p, pair, n_pairs); uw.i < uw.end && ok; uw.i += uw.step) {
                const Unit un = unit_decode(p, uw);
                const int tile_lo = un.tile_lo, tile_hi = un.tile_hi;
                const int kblocks = p.item[un.item].kblocks;
                if constexpr (PROJ) {
                    // The projection takes its turn in the accumulator rotation like a tile (128 columns of it). Its MMAs
                    // are issued after the previous head's, so when its accumulator completes the shared-memory tile of the
                    // previous head is no longer read and the epilogue may overwrite it.
                    const uint32_t ab = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                    if (!mbar_wait(&acc_empty[ab], acc_phase ^ 1u, abort_flag)) {
                        dev_set_error(p.status, DEV_TIMEOUT_ACC_EMPTY);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + ab * BN;
                    for (int kb = 0; kb < p.proj_kblocks; ++kb) {
                        if (!mbar_wait(&full_bar[stage], phase, abort_flag)) {
                            dev_set_error(p.status, DEV_TIMEOUT_TMA_FULL);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t da = make_smem_desc(smem_u32(smem_a + stage * A_STAGE_BYTES));
                        const uint64_t db = make_smem_desc(smem_u32(smem_b + stage * B_STAGE_BYTES));
#pragma unroll
                        for (int kk = 0; kk < BK / UMMA_K; ++kk)
                            tc_mma_bf16(d_tmem, da + static_cast<uint64_t>(kk * 2), db + static_cast<uint64_t>(kk * 2), kInstrDescN128,
                                        (kb | kk) != 0 ? 1u : 0u);
                        tc_commit_pair(&empty_bar[stage]);
                        if (++stage == static_cast<uint32_t>(p.n_stages)) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    tc_commit_pair(&acc_full[ab]);
                    ++tile_count;
                    // the projected tile (bf16, swizzled like a TMA tile) of both CTAs must be in shared memory
                    if (!mbar_wait_cluster(x_ready, unit_count & 1u, abort_flag)) {
                        dev_set_error(p.status, DEV_TIMEOUT_ACC_FULL);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    ++unit_count;
                    tc_fence_after();
                }
                for (int nt = tile_lo; nt < tile_hi && ok; ++nt, ++tile_count) {
                    const uint32_t ab = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                    if (!mbar_wait(&acc_empty[ab], acc_phase ^ 1u, abort_flag)) {
                        dev_set_error(p.status, DEV_TIMEOUT_ACC_EMPTY);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + ab * BN;
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(&full_bar[stage], phase, abort_flag)) {
                            dev_set_error(p.status, DEV_TIMEOUT_TMA_FULL);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t da = make_smem_desc(PROJ ? smem_u32(smem_x + kb * A_STAGE_BYTES) : smem_u32(smem_a + stage * A_STAGE_BYTES));
                        const uint64_t db = make_smem_desc(smem_u32(smem_b + stage * B_STAGE_BYTES));
#pragma unroll
                        for (int kk = 0; kk < BK / UMMA_K; ++kk)
                            tc_mma_bf16(d_tmem, da + static_cast<uint64_t>(kk * 2), db + static_cast<uint64_t>(kk * 2), kInstrDesc,
                                        (kb | kk) != 0 ? 1u : 0u);
                        tc_commit_pair(&empty_bar[stage]);
                        if (++stage == static_cast<uint32_t>(p.n_stages)) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) tc_commit_pair(&acc_full[ab]);
                }
            }
        }
    } else {
        // ---------------- epilogue: bias + ReLU + candidate selection ----------------
        const int quarter = warp & 3;               // TMEM lanes this warp may read
        const int grp = (warp - 2) >> 2;            // which share of a tile's columns this warp filters
        const int e = quarter * 32 + lane;          // row inside the 128-token block
        uint64_t* my_pend = pend + grp * 128 + e;
        const uint32_t pend_addr = smem_u32(my_pend);
        uint16_t* my_hist = hist + grp * 128 + e;
        constexpr int CB_PER_GROUP = BN / BATCH / EPI_GROUPS;
        const int cb_lo = grp * CB_PER_GROUP, cb_hi = cb_lo + CB_PER_GROUP;
        uint32_t tile_count = 0, unit_seq = 0;
        bool ok = true;
        const int fold_at = p.pend_cap - STEP;      // a lane with more pending entries than this may not take another STEP values
        // the accumulator is handed back on the first CTA's barrier
        const uint32_t acc_empty_addr[2] = {map_to_cta(smem_u32(&acc_empty[0]), 0), map_to_cta(smem_u32(&acc_empty[1]), 0)};
        for (UnitWalk uw = unit_walk(p, pair, n_pairs); uw.i < uw.end && ok; uw.i += uw.step) {
            const Unit un = unit_decode(p, uw);
            const int slice = un.slice, mt = un.mt, tile_lo = un.tile_lo, tile_hi = un.tile_hi;
            const ItemParams& ip = p.item[un.item];
            const int t = mt * PAIR_M + static_cast<int>(cta_rank) * BM + e;
            const bool live = t < ip.T;
            const int k = ip.k;
            const uint32_t cap = ip.cap;
            // projection mode: a (token, head) pair is one output row
            const size_t orow = PROJ ? static_cast<size_t>(live ? t : 0) * p.proj_heads + un.head : static_cast<size_t>(live ? t : 0);
            // each group keeps its own candidate list, bound and histogram for its columns of the row
            const size_t list_idx = (orow * ip.n_slices + slice) * EPI_GROUPS + grp;
            uint64_t* glist = DENSE ? nullptr : ip.cand + list_idx * cap;
            if (!DENSE) {
#pragma unroll 1
                for (int sl = 0; sl < NB; ++sl) my_hist[sl * EPI_THREADS] = 0;
            }
            // start from the best bound another slice of these rows has published so far, if any
            const uint32_t hint_in = (live && !DENSE) ? *reinterpret_cast<volatile const uint32_t*>(ip.hint + orow) : 0u;
            RowSel r;
            r.tau_floor = live ? __uint_as_float(hint_in) : INFINITY;    // rows past T select nothing
            r.tau = r.tau_floor;
            r.hbase = -1; r.istar = 0; r.above = 0; r.gcnt = 0; r.floor_exact = false;
            r.ext = r.cut = r.tau;
            int cnt = 0;                            // entries in this row's pending list
            // Bounds are shared while the unit runs: a bound that k values of one list exceed holds for the whole row, so every
            // other list of the row (the other epilogue group's, other column pieces' on other SMs) may drop what does not
            // beat it. Without this each list gathers its own k survivors and the folding work grows with the number of lists.
            ++unit_seq;
            // The groups exchange bounds through xtau32[unit number mod 4][row]; unit n + 2 shares its slot with unit n - 2
            // and each group clears it here, at the start of its unit n. A group announces only before it hands a tile's
            // accumulator back, and no group can start a tile before every group has handed back the tile two before it.
            // So (a) whichever group clears last has itself finished announcing for unit n - 2, and the other finished
            // before its own, earlier clear: after the last clear the slot is zero and nobody writes to it for unit n - 2
            // any more (the leading group's clear may still fall among the lagging group's announcements; that only loses
            // a bound); (b) a group can reach unit n + 2 only after the other has finished the first tile of unit n, i.e.
            // after both clears, so nothing read or announced for unit n + 2 meets an older unit's value.
            if (EPI_GROUPS > 1) xtau32[((unit_seq + 2u) & 3u) * BM + e] = 0u;
            const bool share_row = !DENSE && live && ip.n_slices > 1;     // other units hold pieces of these rows
            uint32_t announced = hint_in;
            if constexpr (PROJ) {
                // The head's projection: accumulator -> + bias -> bf16 (round to nearest even, as the dense epilogue stores
                // it) -> this CTA's shared-memory tile in the layout of a 128-byte-swizzled TMA tile (two k-blocks of 128 rows x
                // 64 columns; the 16-byte chunk c of row r sits at chunk c ^ (r & 7)), where the encode's MMAs read it as A.
                const uint32_t ab = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                const bool arrived = mbar_wait(&acc_full[ab], acc_phase, abort_flag);
                if (!arrived) {
                    dev_set_error(p.status, DEV_TIMEOUT_ACC_FULL);
                    *abort_flag = 1;
                }
                if (!__all_sync(0xffffffffu, arrived)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + ab * BN + (static_cast<uint32_t>(quarter * 32) << 16);
                constexpr int PB = PROJ_N / BATCH / EPI_GROUPS;           // batches of 32 columns per group
                unsigned char* xrow = smem_x + (e >> 3) * 1024 + (e & 7) * 128;
#pragma unroll 1
                for (int cb = grp * PB; cb < (grp + 1) * PB; ++cb) {
                    uint32_t acc[32];
                    tc_ld32(taddr + cb * BATCH, acc);
                    const float4* pb4 = reinterpret_cast<const float4*>(p.proj_bias + un.head * PROJ_N + cb * BATCH);
                    float bias[BATCH];
#pragma unroll
                    for (int j4 = 0; j4 < BATCH / 4; ++j4) {
                        const float4 b4 = __ldg(pb4 + j4);
                        bias[4 * j4 + 0] = b4.x; bias[4 * j4 + 1] = b4.y; bias[4 * j4 + 2] = b4.z; bias[4 * j4 + 3] = b4.w;
                    }
                    tc_wait_ld();
#pragma unroll
                    for (int g8 = 0; g8 < BATCH / 8; ++g8) {
                        __nv_bfloat162 h2[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            h2[q] = __floats2bfloat162_rn(__uint_as_float(acc[g8 * 8 + 2 * q]) + bias[g8 * 8 + 2 * q],
                                                          __uint_as_float(acc[g8 * 8 + 2 * q + 1]) + bias[g8 * 8 + 2 * q + 1]);
                        const int chunk = (cb & 1) * 4 + g8;              // 16-byte chunk inside the row's 128 bytes of this k-block
                        *reinterpret_cast<uint4*>(xrow + (cb >> 1) * A_STAGE_BYTES + ((chunk ^ (e & 7)) << 4)) = *reinterpret_cast<const uint4*>(h2);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy stores -> visible to the MMA's reads
                tc_fence_before();
                mbar_arrive_cluster(acc_empty_addr[ab]);
                mbar_arrive_cluster_release(map_to_cta(smem_u32(x_ready), 0));
                ++tile_count;
            }
            for (int nt = tile_lo; nt < tile_hi && ok; ++nt, ++tile_count) {
                const uint32_t ab = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
                const bool arrived = mbar_wait(&acc_full[ab], acc_phase, abort_flag);
                if (!arrived) {
                    dev_set_error(p.status, DEV_TIMEOUT_ACC_FULL);
                    *abort_flag = 1;
                }
                // The go/no-go decision is taken per warp: the four epilogue warps share nothing but the abort flag,
                // which ends the others' waits soon after one of them gave up, so they need not move in step.
                if (!__all_sync(0xffffffffu, arrived)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + ab * BN + (static_cast<uint32_t>(quarter * 32) << 16);
                const float4* bias4 = reinterpret_cast<const float4*>(ip.b_eff + static_cast<size_t>(nt) * BN);
                if (!DENSE && nt == tile_lo && __any_sync(0xffffffffu, live && r.tau == 0.0f)) {
                    // Cold start: without a bound every second value of the unit's first tile would go through the pending
                    // lists. A first pass over that tile only counts, per row, how many of its values exceed each of
                    // COLD_LEVELS fractions of the largest value of the row's first 32 columns; the highest level that at
                    // least k values exceed is a bound that k values of this slice are known to beat, and the regular pass
                    // below (the accumulator is still in tensor memory) starts from it.
                    float level[COLD_LEVELS];
                    int seen[COLD_LEVELS];
#pragma unroll 1
                    for (int cb = cb_lo; cb < cb_hi; ++cb) {
                        uint32_t acc[32];
                        tc_ld32(taddr + cb * BATCH, acc);
                        float bias[BATCH];
#pragma unroll
                        for (int j4 = 0; j4 < BATCH / 4; ++j4) {
                            const float4 b4 = __ldg(bias4 + cb * (BATCH / 4) + j4);
                            bias[4 * j4 + 0] = b4.x; bias[4 * j4 + 1] = b4.y; bias[4 * j4 + 2] = b4.z; bias[4 * j4 + 3] = b4.w;
                        }
                        tc_wait_ld();
                        if (cb == cb_lo) {
                            float top = 0.0f;
#pragma unroll
                            for (int q = 0; q < BATCH; ++q) top = fmaxf(top, __uint_as_float(acc[q]) + bias[q]);
#pragma unroll
                            for (int lv = 0; lv < COLD_LEVELS; ++lv) { level[lv] = top * kColdFraction[lv]; seen[lv] = 0; }
                        }
#pragma unroll
                        for (int q = 0; q < BATCH; ++q) {
                            const float v = __uint_as_float(acc[q]) + bias[q];
#pragma unroll
                            for (int lv = 0; lv < COLD_LEVELS; ++lv) seen[lv] += (v > level[lv]) ? 1 : 0;
                        }
                    }
                    if (live && r.tau == 0.0f) {
                        float bound = 0.0f;
#pragma unroll
                        for (int lv = COLD_LEVELS - 1; lv >= 0; --lv)
                            if (seen[lv] >= k && level[lv] > bound) bound = level[lv];       // levels descend with lv ascending
                        r.tau_floor = r.tau = bound;
                    }
                }
                // the row's published bound as of now; used from the tile's second batch on, so the load's latency is covered
                const uint32_t row_bound = share_row ? *reinterpret_cast<volatile const uint32_t*>(ip.hint + orow) : 0u;
#pragma unroll 1
                for (int cb = cb_lo; cb < cb_hi; ++cb) {
                    uint32_t acc[32];
                    tc_ld32(taddr + cb * BATCH, acc);
                    float bias[BATCH];
#pragma unroll
                    for (int j4 = 0; j4 < BATCH / 4; ++j4) {
                        const float4 b4 = __ldg(bias4 + cb * (BATCH / 4) + j4);
                        bias[4 * j4 + 0] = b4.x; bias[4 * j4 + 1] = b4.y; bias[4 * j4 + 2] = b4.z; bias[4 * j4 + 3] = b4.w;
                    }
                    if constexpr (!DENSE) {
                        if (EPI_GROUPS > 1) r.ext = fmaxf(r.ext, __uint_as_float(xtau32[(unit_seq & 3u) * BM + e]));
                        if (cb == cb_lo + 1) r.ext = fmaxf(r.ext, __uint_as_float(row_bound));
                        r.cut = fmaxf(r.cut, r.ext);
                    }
                    tc_wait_ld();
                    if constexpr (DENSE) {
                        // 32 consecutive columns of this thread's row: 128 (fp32) or 64 (bf16) contiguous bytes
                        const int col0 = nt * BN + cb * BATCH;
                        if (live) {
#pragma unroll
                            for (int g8 = 0; g8 < BATCH / 8; ++g8) {
                                if (col0 + g8 * 8 >= p.d_sae) break;              // d_sae is a multiple of 8
                                float v[8];
#pragma unroll
                                for (int q = 0; q < 8; ++q) v[q] = __uint_as_float(acc[g8 * 8 + q]) + bias[g8 * 8 + q];
                                if (p.out_bf16) {
                                    __nv_bfloat162 h2[4];
#pragma unroll
                                    for (int q = 0; q < 4; ++q) h2[q] = __floats2bfloat162_rn(v[2 * q], v[2 * q + 1]);
                                    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.dense_out) + static_cast<size_t>(t) * p.ld_out + col0 + g8 * 8;
                                    *reinterpret_cast<uint4*>(out) = *reinterpret_cast<const uint4*>(h2);
                                } else {
                                    float* out = static_cast<float*>(p.dense_out) + static_cast<size_t>(t) * p.ld_out + col0 + g8 * 8;
                                    *reinterpret_cast<float4*>(out) = make_float4(v[0], v[1], v[2], v[3]);
                                    *reinterpret_cast<float4*>(out + 4) = make_float4(v[4], v[5], v[6], v[7]);
                                }
                            }
                        }
                        continue;
                    }
                    const uint32_t ncol0 = ~static_cast<uint32_t>(nt * BN + cb * BATCH);   // ~(col0 + j) = ncol0 - j
#pragma unroll
                    for (int h = 0; h < BATCH / STEP; ++h) {
                        // Branch-free append: a value that beats the bound is stored at the end of the row's pending list and
                        // the end moves on: one compare, one predicated shared-memory store and one predicated add per value.
                        uint32_t slot = pend_addr + static_cast<uint32_t>(cnt) * (EPI_THREADS * 8);
                        const float cutv = r.cut;
#pragma unroll
                        for (int j = 0; j < STEP; ++j) {
                            const float v = __uint_as_float(acc[h * STEP + j]) + bias[h * STEP + j];
                            asm volatile("{\n\t.reg .pred p;\n\tsetp.gt.f32 p, %1, %2;\n\t@p st.shared.v2.u32 [%0], {%3, %4};\n\t@p add.u32 %0, %0, %5;\n\t}"
                                         : "+r"(slot)
                                         : "f"(v), "f"(cutv), "r"(ncol0 - static_cast<uint32_t>(h * STEP + j)), "r"(__float_as_uint(v)), "n"(EPI_THREADS * 8));
                        }
                        asm volatile("" ::: "memory");
                        cnt = static_cast<int>((slot - pend_addr) / (EPI_THREADS * 8));
                        if (__any_sync(0xffffffffu, cnt > fold_at)) {
                            fold_pending<EPI_THREADS>(my_pend, my_hist, glist, r, cnt, k, cap);
                            const uint32_t now = announced_bound(r);       // tell the row's other lists when the bound has risen
                            if (now > announced) {
                                announced = now;
                                if (EPI_GROUPS > 1) atomicMax(&xtau32[(unit_seq & 3u) * BM + e], now);
                                if (share_row) atomicMax(ip.hint + orow, now);
                            }
                        }
                    }
                }
                tc_fence_before();
                mbar_arrive_cluster(acc_empty_addr[ab]);
            }
            if (ok && !DENSE) {
                if (__any_sync(0xffffffffu, cnt > 0)) fold_pending<EPI_THREADS>(my_pend, my_hist, glist, r, cnt, k, cap);
                if (live) {
                    // what the merge may cut the row's lists at: this list's own bound or a better one learnt meanwhile
                    uint32_t out = announced_bound(r);
                    if (__float_as_uint(r.ext) > out) out = __float_as_uint(r.ext);
                    // The list stays as it was filled (about k (1 + ln(columns / k)) entries under bounds that rose along the
                    // unit): the merge cuts it at the row's final bound. Compacting it here, a tail of dependent round trips
                    // after the unit's last tile, cost more than the merge saves (heads k = 128: 2.36 -> 2.08 ms without it).
                    ip.counts[list_idx] = r.gcnt;
                    if (out > hint_in) atomicMax(ip.hint + orow, out);
                }
            }
        }
    }

    // Both CTAs are done with tensor memory, and the first CTA has seen every copy land, before either frees
    // its tensor memory or leaves (the peer's shared memory receives copies and is read by the pair's MMAs).
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- one-time preparation ---------------------------------------------------------------------------
// W_enc [d_in, d_sae] (feature = column) -> W_t [d_sae, d_in] so that both GEMM operands are K-major.
__global__ void transpose_bf16_kernel(const __nv_bfloat16* __restrict__ W, __nv_bfloat16* __restrict__ Wt, int d_in, int d_sae)
{
    __shared__ __nv_bfloat16 tile[32][33];
    const int f0 = blockIdx.x * 32, i0 = blockIdx.y * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int i = i0 + r, f = f0 + threadIdx.x;
        tile[r][threadIdx.x] = (i < d_in && f < d_sae) ? W[static_cast<size_t>(i) * d_sae + f] : __float2bfloat16(0.0f);
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int f = f0 + r, i = i0 + threadIdx.x;
        if (f < d_sae && i < d_in) Wt[static_cast<size_t>(f) * d_in + i] = tile[threadIdx.x][r];
    }
}

// b_eff[f] = b_enc[f] - sum_i W_enc[i,f] * b_dec[i], summed in fp64 in index order, stored as fp32.
// The array is padded to whole 256-column tiles with -inf, which no candidate filter lets through.
__global__ void folded_bias_kernel(const __nv_bfloat16* __restrict__ W, const float* __restrict__ b_enc,
                                   const float* __restrict__ b_dec, int d_in, int d_sae, int d_sae_pad,
                                   float* __restrict__ b_eff)
{
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= d_sae_pad) return;
    if (f >= d_sae) { b_eff[f] = -INFINITY; return; }
    double s = 0.0;
    for (int i = 0; i < d_in; ++i)
        s += static_cast<double>(__bfloat162float(W[static_cast<size_t>(i) * d_sae + f])) * static_cast<double>(b_dec[i]);
    b_eff[f] = static_cast<float>(static_cast<double>(b_enc[f]) - s);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

s3_status get_encode_fn(EncodeTiledFn* out)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        S3_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres));
        S3_REQUIRE(sym != nullptr && qres == cudaDriverEntryPointSuccess, S3_ERR_CUDA,
                   "the driver does not provide cuTensorMapEncodeTiled");
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    *out = fn;
    return S3_OK;
}

// 2-D bf16 tensor [rows, cols] with row pitch ld (elements); box = box_rows x 64 columns, 128-byte swizzle.
s3_status make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows)
{
    EncodeTiledFn fn;
    const s3_status st = get_encode_fn(&fn);
    if (st != S3_OK) return st;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    S3_REQUIRE(r == CUDA_SUCCESS, S3_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d (rows %llu cols %llu ld %llu)",
               static_cast<int>(r), static_cast<unsigned long long>(rows), static_cast<unsigned long long>(cols),
               static_cast<unsigned long long>(ld));
    return S3_OK;
}

}  // namespace

size_t encode_tc_prepared_bytes(int d_in, int d_sae)
{
    const size_t d_sae_pad = static_cast<size_t>((d_sae + BN - 1) / BN) * BN;
    return round_up(static_cast<size_t>(d_sae) * d_in * 2, 256) + round_up(d_sae_pad * 4, 256);
}

s3_status encode_tc_prepare(EncodeTcState* st, const void* d_W, const float* d_b_enc, const float* d_b_dec, int d_in,
                            int d_sae, void* d_prepared, cudaStream_t stream)
{
    st->d_wt = d_prepared;
    st->d_b_eff = reinterpret_cast<float*>(static_cast<unsigned char*>(d_prepared) +
                                           round_up(static_cast<size_t>(d_sae) * d_in * 2, 256));
    const dim3 tb(32, 8), tg((d_sae + 31) / 32, (d_in + 31) / 32);
    transpose_bf16_kernel<<<tg, tb, 0, stream>>>(static_cast<const __nv_bfloat16*>(d_W),
                                                 static_cast<__nv_bfloat16*>(st->d_wt), d_in, d_sae);
    S3_CUDA_TRY(cudaGetLastError());
    const int d_sae_pad = (d_sae + BN - 1) / BN * BN;
    folded_bias_kernel<<<(d_sae_pad + 127) / 128, 128, 0, stream>>>(static_cast<const __nv_bfloat16*>(d_W), d_b_enc, d_b_dec, d_in,
                                                                    d_sae, d_sae_pad, st->d_b_eff);
    S3_CUDA_TRY(cudaGetLastError());
    static_assert(sizeof(CUtensorMap) <= sizeof(st->map_w), "tensor map storage too small");
    return make_map(reinterpret_cast<CUtensorMap*>(st->map_w), st->d_wt, d_sae, d_in, d_in, BN / 2);
}

int encode_tc_col_tiles(int d_sae) { return (d_sae + BN - 1) / BN; }
int encode_tc_row_tiles(int T) { return (T + PAIR_M - 1) / PAIR_M; }   // a CTA pair takes 256 tokens

// CTA pairs that can be resident at once (cached per device).
int encode_tc_max_pairs();

int encode_tc_max_pairs()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    if (dev < 64 && cached[dev]) return cached[dev];
    int n = device_sm_count() / 2;      // a pair occupies two SMs entirely (shared memory)
    if (n < 1) n = 1;
    if (dev < 64) cached[dev] = n;
    return n;
}

// Slots of one candidate list (one per row, slice and epilogue group); a list that fills up is pruned in place.
uint32_t encode_tc_list_cap(int k, int groups) { return static_cast<uint32_t>((k < 4 ? 64 : 16 * k) / groups); }

// Column tiles per slice may not exceed 255: a row's histogram counters are 16 bits wide.
int encode_tc_min_slices(int d_sae) { return (encode_tc_col_tiles(d_sae) + 254) / 255; }

// Scratch of one item whose rows hold `lists` (row, slot) candidate lists in all: the rows' bounds, the lists' lengths and
// the lists. Sized for either number of epilogue groups: two lists of half the slots take the room of one list.
static size_t lists_bytes(int T, size_t lists, int k)
{
    const size_t s = lists * MAX_EPI_GROUPS;
    return round_up(static_cast<size_t>(T) * 4, 256) + round_up(s * 4, 256) +
           round_up(s * encode_tc_list_cap(k, MAX_EPI_GROUPS) * sizeof(uint64_t), 256);
}

size_t encode_tc_workspace_bytes(int T, int n_slices, int k) { return lists_bytes(T, static_cast<size_t>(T) * n_slices, k); }

// Slots per row any automatic schedule stays within: a row tile is cut where a pair's share ends, so it holds about
// pairs / row tiles pieces plus the ends; uniform slices are held to the same number.
static int slot_bound(int T, int n_pairs)
{
    const int n = encode_tc_row_tiles(T);
    const int b = 4 + (n_pairs + n - 1) / n;
    return b < 16 ? b : 16;
}

// Scratch that holds any automatic schedule of T tokens, and of fewer: T * slot_bound(T) <= 5 T + 256 pairs, which grows
// with T, so a workspace sized for a full chunk also serves the shorter last one.
size_t encode_tc_workspace_bound(int T, int k)
{
    const size_t t = static_cast<size_t>(T);
    size_t lists = 5 * t + 256 * static_cast<size_t>(encode_tc_max_pairs());
    if (lists > 16 * t) lists = 16 * t;
    return lists_bytes(T, lists, k);
}

namespace {

// ---- work units of a launch -----------------------------------------------------------------------------
// Modelled durations in SM cycles. A 256-column tile takes the MMAs of its k-blocks or the Top-k filter of its columns,
// whichever is longer; a unit also pays for its cold start (one extra pass over its first tile) and its last fold.
struct CostModel {
    double tile, unit;
};
CostModel cost_model(int kblocks, int k, int groups, bool dense)
{
    const double mma = 600.0 * kblocks;
    const double filter = dense ? 6000.0 : (12000.0 + 100.0 * k) / (groups == 2 ? 1.5 : 1.0);
    CostModel c;
    c.tile = mma > filter ? mma : filter;
    c.unit = dense ? 2000.0 : 5000.0 + 100.0 * k;       // measured closer to 16000 + 100 k, but shares cut with the smaller charge end more evenly
    return c;
}

constexpr int kMaxSlots = 16;                       // candidate lists per row and epilogue group at most
constexpr int kMinPiece = 3;                        // a row is not cut into pieces shorter than this many column tiles
constexpr size_t kRoundBytes = size_t(48) << 20;    // encoder weights that pairs may walk at the same time (they should stay in L2)

struct Schedule {
    int order[MAX_GROUP];             // launch position -> caller's item
    int slots[MAX_GROUP];             // candidate lists per row of the item at each launch position
    int n_pairs, n_units, groups;
    bool table;                       // units come from unit[] / pair_start[]; otherwise uniform slices dealt round-robin
    UnitDesc unit[MAX_SCHED];
    uint16_t pair_start[MAX_PAIRS + 1];
};

// Uniform column slices of one encoder: the count that minimises waves * tiles-per-slice plus a charge per slice.
int uniform_slices(int T, int nct, int d_sae, int n_pairs, bool dense)
{
    const int n_mtiles = encode_tc_row_tiles(T);
    const int lo = encode_tc_min_slices(d_sae);
    int cap = nct < kMaxSlots ? nct : kMaxSlots;
    if (!dense && slot_bound(T, n_pairs) < cap) cap = slot_bound(T, n_pairs);      // lists per row that the scratch bound allows
    if (cap < lo) cap = lo;
    int best = lo;
    double best_cost = 1e30;
    for (int sl = lo; sl <= cap; ++sl) {
        const int units = n_mtiles * sl;
        const int waves = (units + n_pairs - 1) / n_pairs;
        const int len = (nct + sl - 1) / sl;
        const double cost = static_cast<double>(waves) * len + 0.25 * sl * waves;
        if (cost < best_cost - 1e-9) { best_cost = cost; best = sl; }
    }
    return best;
}

// Balanced plan. The items (in launch order) are taken in rounds whose encoder weights fit in L2 together; the tiles of a
// round, in the order (item, row tile, column tile), are cut into one contiguous range per CTA pair of equal modelled
// duration, and a range is cut into units at the row-tile boundaries. A row tile therefore ends up in a few pieces held by
// neighbouring pairs, each piece with its own candidate list. Fails (false) when an encoder is too wide for a round, a
// row would need more than kMaxSlots pieces, or the units do not fit the table.
bool plan_balanced(const EncodeTcItem* items, const int* order, int n_items, int n_pairs, int groups, bool dense, Schedule& sc,
                   double extra_unit_cost = 0.0)
{
    static thread_local UnitDesc gen[MAX_SCHED];
    static thread_local uint16_t gen_pair[MAX_SCHED];
    int n = 0;
    int q0 = 0;
    while (q0 < n_items) {
        size_t bytes = 0;
        int q1 = q0;
        while (q1 < n_items) {
            const EncodeTcItem& it = items[order[q1]];
            const size_t w = static_cast<size_t>(it.d_sae) * it.d_in * 2;
            if (w > kRoundBytes) return false;
            if (q1 > q0 && bytes + w > kRoundBytes) break;
            bytes += w;
            ++q1;
        }
        double rem = 0.0;
        for (int q = q0; q < q1; ++q) {
            const EncodeTcItem& it = items[order[q]];
            CostModel c = cost_model((it.d_in + BK - 1) / BK, it.k, groups, dense);
            c.unit += extra_unit_cost;
            rem += static_cast<double>(encode_tc_row_tiles(it.T)) * (encode_tc_col_tiles(it.d_sae) * c.tile + c.unit);
        }
        // a pair's share: what is left, plus the start-up of the piece that every later cut adds, over the pairs left
        auto share = [&](int pr, double unit) { return (rem + unit * (n_pairs - pr - 1)) / (n_pairs - pr); };
        int pr = 0;
        double acc = 0.0;
        double target = share(0, cost_model((items[order[q0]].d_in + BK - 1) / BK, items[order[q0]].k, groups, dense).unit + extra_unit_cost);
        for (int q = q0; q < q1; ++q) {
            const EncodeTcItem& it = items[order[q]];
            CostModel c = cost_model((it.d_in + BK - 1) / BK, it.k, groups, dense);
            c.unit += extra_unit_cost;
            const int n_mtiles = encode_tc_row_tiles(it.T), nct = encode_tc_col_tiles(it.d_sae);
            if (n_mtiles > 65535 || nct > 65535) return false;
            const int max_pieces = slot_bound(it.T, n_pairs);
            int slots = 1;
            for (int mt = 0; mt < n_mtiles; ++mt) {
                int lo = 0, pieces = 0;
                while (lo < nct) {
                    const int left = nct - lo;
                    int take;
                    if (pr == n_pairs - 1) take = left;
                    else {
                        const int fit = static_cast<int>((target - acc - c.unit) / c.tile + 0.5);
                        if (fit >= left) take = left;
                        else if (left - fit < kMinPiece && left - kMinPiece >= kMinPiece) take = left - kMinPiece;   // leave a whole piece
                        else if (left - fit < kMinPiece) take = left;
                        else if (fit < kMinPiece) {
                            if (acc > 0.0) {              // this pair is full: the row goes on with the next one
                                ++pr; acc = 0.0; target = share(pr, c.unit);
                                continue;
                            }
                            take = left < kMinPiece ? left : kMinPiece;
                        } else take = fit;
                    }
                    if (take > 255) take = 255;           // a row's histogram counters are 16 bits wide
                    if (n >= MAX_SCHED || pieces >= max_pieces) return false;
                    gen[n].mt = static_cast<uint16_t>(mt);
                    gen[n].tile_lo = static_cast<uint16_t>(lo);
                    gen[n].tile_hi = static_cast<uint16_t>(lo + take);
                    gen[n].item = static_cast<uint8_t>(q);
                    gen[n].slot = static_cast<uint8_t>(pieces);
                    gen_pair[n] = static_cast<uint16_t>(pr);
                    ++n;
                    acc += c.unit + take * c.tile;
                    rem -= take * c.tile + (pieces == 0 ? c.unit : 0.0);
                    ++pieces;
                    lo += take;
                    if (pr < n_pairs - 1 && acc >= target - 0.5 * c.tile) { ++pr; acc = 0.0; target = share(pr, c.unit); }
                }
                slots = pieces > slots ? pieces : slots;
            }
            sc.slots[q] = slots;
        }
        q0 = q1;
    }
    // bucket by pair, keeping the order of generation (rounds in launch order)
    int count[MAX_PAIRS] = {};
    for (int i = 0; i < n; ++i) ++count[gen_pair[i]];
    int run = 0, used = 0;
    for (int q = 0; q < n_pairs; ++q) {
        sc.pair_start[q] = static_cast<uint16_t>(run);
        run += count[q];
        if (count[q]) used = q + 1;
    }
    for (int q = n_pairs; q <= MAX_PAIRS; ++q) sc.pair_start[q] = static_cast<uint16_t>(run);
    int fill[MAX_PAIRS];
    for (int q = 0; q < n_pairs; ++q) fill[q] = sc.pair_start[q];
    for (int i = 0; i < n; ++i) sc.unit[fill[gen_pair[i]]++] = gen[i];
    sc.n_units = n;
    sc.n_pairs = used;
    sc.table = true;
    return true;
}

// Uniform slices, whole (row tile, slice) units; with several items and room in the table the units are dealt out by
// modelled duration (each to the pair with the least work so far), otherwise round-robin without a table.
void plan_uniform(const EncodeTcItem* items, const int* order, int n_items, int n_pairs, int groups, bool dense, Schedule& sc)
{
    int n_units = 0;
    for (int q = 0; q < n_items; ++q) {
        const EncodeTcItem& it = items[order[q]];
        const int n_mtiles = encode_tc_row_tiles(it.T), nct = encode_tc_col_tiles(it.d_sae);
        sc.slots[q] = it.n_slices > 0 ? it.n_slices : uniform_slices(it.T, nct, it.d_sae, n_pairs, dense);
        n_units += n_mtiles * sc.slots[q];
    }
    sc.n_units = n_units;
    sc.n_pairs = n_units < n_pairs ? n_units : n_pairs;
    sc.table = false;
    if (n_items < 2 || n_units > MAX_SCHED) return;
    static thread_local uint16_t unit_pair[MAX_SCHED];
    static thread_local UnitDesc gen[MAX_SCHED];
    double load[MAX_PAIRS];
    int count[MAX_PAIRS];
    for (int q = 0; q < sc.n_pairs; ++q) { load[q] = 0.0; count[q] = 0; }
    int u = 0;
    for (int q = 0; q < n_items; ++q) {
        const EncodeTcItem& it = items[order[q]];
        const int n_mtiles = encode_tc_row_tiles(it.T), nct = encode_tc_col_tiles(it.d_sae);
        if (n_mtiles > 65535 || nct > 65535) return;
        const CostModel c = cost_model((it.d_in + BK - 1) / BK, it.k, groups, dense);
        for (int sl = 0; sl < sc.slots[q]; ++sl) {
            const int lo = static_cast<int>(static_cast<int64_t>(sl) * nct / sc.slots[q]);
            const int hi = static_cast<int>(static_cast<int64_t>(sl + 1) * nct / sc.slots[q]);
            for (int mt = 0; mt < n_mtiles; ++mt, ++u) {
                int best = 0;
                for (int r = 1; r < sc.n_pairs; ++r)
                    if (load[r] < load[best]) best = r;
                load[best] += c.unit + (hi - lo) * c.tile;
                unit_pair[u] = static_cast<uint16_t>(best);
                ++count[best];
                gen[u].mt = static_cast<uint16_t>(mt);
                gen[u].tile_lo = static_cast<uint16_t>(lo);
                gen[u].tile_hi = static_cast<uint16_t>(hi);
                gen[u].item = static_cast<uint8_t>(q);
                gen[u].slot = static_cast<uint8_t>(sl);
            }
        }
    }
    int run = 0;
    for (int q = 0; q < sc.n_pairs; ++q) { sc.pair_start[q] = static_cast<uint16_t>(run); run += count[q]; }
    for (int q = sc.n_pairs; q <= MAX_PAIRS; ++q) sc.pair_start[q] = static_cast<uint16_t>(run);
    int fill[MAX_PAIRS];
    for (int q = 0; q < sc.n_pairs; ++q) fill[q] = sc.pair_start[q];
    for (int i = 0; i < n_units; ++i) sc.unit[fill[unit_pair[i]]++] = gen[i];
    sc.table = true;
}

// Banded walk of one encoder whose weights do not stay in L2: bands of row tiles, each band swept by its column
// slices at the same time (one unit per pair), band after band. The hot set is then a band's token tiles (2 MB per row
// tile at d_in 4096, re-read for every column tile) plus the windows of W_enc^T that the slices stream; with all row
// tiles in one band the token tiles alone fill the L2 and W_enc^T is read about four times (query SAE, T 8192: 1.03-1.27
// GB of DRAM traffic with 32 row tiles x 2 slices). A band holds as many row tiles as there are pairs per slice, and
// each band picks its own slice count so that the pairs' total stays short: 32 row tiles on 74 pairs go as 18 x 4 slices
// (32 column tiles each) + 14 x 5 (26 each), 58 tiles on the busiest pair instead of the 64 of 16 x 4 + 16 x 4 (1.58 ->
// 1.53 ms, 0.89 GB; bands of 12 x 6 and 8 x 8 alone are 4 and 11 % slower: more lists per row).
bool plan_banded(const EncodeTcItem& it, int n_pairs, Schedule& sc)
{
    static thread_local UnitDesc gen[MAX_SCHED];
    static thread_local uint16_t gen_pair[MAX_SCHED];
    const int n_mtiles = encode_tc_row_tiles(it.T), nct = encode_tc_col_tiles(it.d_sae);
    // modelled time of a band: its tiles per slice, a quarter tile per slice, 6 % more when its token tiles exceed 40 MB
    const int s_lo = encode_tc_min_slices(it.d_sae);
    int s_hi = slot_bound(it.T, n_pairs) < nct ? slot_bound(it.T, n_pairs) : nct;
    s_hi = s_hi > kMaxSlots ? kMaxSlots : s_hi;
    if (s_hi < s_lo) return false;
    const int r_hot = static_cast<int>((size_t(40) << 20) / (static_cast<size_t>(PAIR_M) * it.d_in * 2));
    // bands may differ in their slice count: cost[n] = least modelled time of the last n row tiles, band by band
    static thread_local std::vector<double> cost;
    static thread_local std::vector<uint8_t> pick;
    cost.assign(n_mtiles + 1, 0.0);
    pick.assign(n_mtiles + 1, 0);
    for (int left = 1; left <= n_mtiles; ++left) {
        double best = 1e30;
        int arg = s_lo;
        for (int c = s_lo; c <= s_hi; ++c) {
            int R = n_pairs / c;
            R = R < 1 ? 1 : (R > left ? left : R);
            const int len = (nct + c - 1) / c;
            const double t = len + 0.25 * c + (R > r_hot ? 0.06 * len : 0.0) + cost[left - R];
            if (t < best - 1e-9) { best = t; arg = c; }
        }
        cost[left] = best;
        pick[left] = static_cast<uint8_t>(arg);
    }
    int n = 0, S = 0, offset = 0;
    if (n_mtiles > 65535) return false;
    for (int b0 = 0; b0 < n_mtiles;) {
        const int left = n_mtiles - b0, c = pick[left];
        int rows = n_pairs / c;
        rows = rows < 1 ? 1 : (rows > left ? left : rows);
        if ((nct + c - 1) / c > 255 || n + rows * c > MAX_SCHED) return false;
        S = c > S ? c : S;
        for (int sl = 0; sl < c; ++sl)
            for (int r = 0; r < rows; ++r, ++n) {
                gen[n].mt = static_cast<uint16_t>(b0 + r);
                gen[n].tile_lo = static_cast<uint16_t>(static_cast<int64_t>(sl) * nct / c);
                gen[n].tile_hi = static_cast<uint16_t>(static_cast<int64_t>(sl + 1) * nct / c);
                gen[n].item = 0;
                gen[n].slot = static_cast<uint8_t>(sl);
                gen_pair[n] = static_cast<uint16_t>((offset + sl * rows + r) % n_pairs);
            }
        offset = (offset + rows * c) % n_pairs;
        b0 += rows;
    }
    int count[MAX_PAIRS] = {};
    for (int i = 0; i < n; ++i) ++count[gen_pair[i]];
    int run = 0, used = 0;
    for (int q = 0; q < n_pairs; ++q) { sc.pair_start[q] = static_cast<uint16_t>(run); run += count[q]; if (count[q]) used = q + 1; }
    for (int q = n_pairs; q <= MAX_PAIRS; ++q) sc.pair_start[q] = static_cast<uint16_t>(run);
    int fill[MAX_PAIRS];
    for (int q = 0; q < n_pairs; ++q) fill[q] = sc.pair_start[q];
    for (int i = 0; i < n; ++i) sc.unit[fill[gen_pair[i]]++] = gen[i];
    sc.n_units = n; sc.n_pairs = used; sc.table = true; sc.slots[0] = S;
    return true;
}

// The schedule of a launch: launch order of the items (descending modelled tile duration, so that the short tiles fill
// the end), epilogue groups, CTA pairs and the units. Items that leave n_slices at 0 get the balanced plan when it
// applies; an item with n_slices > 0 forces uniform slices for the whole launch.
void build_schedule(const EncodeTcItem* items, int n_items, int max_ctas, bool dense, Schedule& sc, int device_pairs = 0)
{
    int max_d_in = 0;
    bool forced = false;
    for (int j = 0; j < n_items; ++j) {
        max_d_in = items[j].d_in > max_d_in ? items[j].d_in : max_d_in;
        forced = forced || items[j].n_slices > 0;
    }
    sc.groups = (!dense && max_d_in <= kTwoGroupsMaxDin) ? 2 : 1;
    double cost[MAX_GROUP];
    for (int j = 0; j < n_items; ++j) {
        sc.order[j] = j;
        cost[j] = cost_model((items[j].d_in + BK - 1) / BK, items[j].k, sc.groups, dense).tile;
    }
    for (int a = 1; a < n_items; ++a)
        for (int b = a; b > 0 && cost[sc.order[b]] > cost[sc.order[b - 1]]; --b) {
            const int t = sc.order[b]; sc.order[b] = sc.order[b - 1]; sc.order[b - 1] = t;
        }
    int n_pairs = device_pairs > 0 ? device_pairs : encode_tc_max_pairs();
    if (max_ctas > 0 && max_ctas / 2 < n_pairs) n_pairs = max_ctas / 2 > 0 ? max_ctas / 2 : 1;
    if (n_pairs > MAX_PAIRS) n_pairs = MAX_PAIRS;
    // Cutting row tiles at the pairs' shares costs extra pieces (each gathers its own survivors at first), so it is not
    // done where whole row tiles already fill the pairs' waves evenly. (Eight 512-wide layers of 16384 tokens, 512 row
    // tiles in 7 waves of 74: whole rows 1.49 ms, cut 1.54 ms; one 1024-wide layer of 8192 tokens, 32 row tiles: two
    // uniform slices 0.298 ms, cut 0.284 ms; 256 row tiles of a 128-wide encoder, k = 128: 2.54 ms against 2.36 ms.)
    bool even_without_cuts = false;
    if (!forced) {
        int units = 0;
        for (int j = 0; j < n_items; ++j) units += encode_tc_row_tiles(items[j].T) * encode_tc_min_slices(items[j].d_sae);
        const int waves = (units + n_pairs - 1) / n_pairs;
        even_without_cuts = static_cast<double>(units) >= 0.93 * waves * n_pairs;
    }
    // the dense epilogue has no lists to restart and its units cost nothing extra: uniform slices serve it
    if (!dense && !forced && n_items == 1 && static_cast<size_t>(items[0].d_sae) * items[0].d_in * 2 > kRoundBytes &&
        plan_banded(items[0], n_pairs, sc))
        return;
    if (dense || forced || even_without_cuts || !plan_balanced(items, sc.order, n_items, n_pairs, sc.groups, dense, sc))
        plan_uniform(items, sc.order, n_items, n_pairs, sc.groups, dense, sc);
}

Schedule& schedule_buffer()
{
    static thread_local Schedule sc;
    return sc;
}

// Common launch of the two epilogue modes. Selection: items with d_ids / d_vals, scratch carved from d_scratch.
// Dense: one item, d_dense set.
s3_status launch_tc(const EncodeTcItem* items, int n_items, int max_ctas, void* d_scratch, uint32_t* d_status, void* d_dense,
                    int64_t ld_out, bool out_bf16, cudaStream_t stream)
{
    const bool dense = d_dense != nullptr;
    S3_REQUIRE(n_items >= 1 && n_items <= MAX_GROUP, S3_ERR_UNSUPPORTED, "%d encoders in one launch, at most %d", n_items, MAX_GROUP);
    alignas(64) TensorMaps maps;
    static thread_local EncodeTcParams p;
    memset(&p, 0, sizeof(p));
    p.n_items = n_items;
    p.status = d_status;
    p.dense_out = d_dense; p.ld_out = ld_out; p.out_bf16 = out_bf16 ? 1 : 0;
    p.d_sae = items[0].d_sae;
    for (int j = 0; j < n_items; ++j)
        S3_REQUIRE(items[j].n_slices == 0 || items[j].n_slices >= encode_tc_min_slices(items[j].d_sae), S3_ERR_INVALID_ARG,
                   "d_sae = %d needs at least %d column slices", items[j].d_sae, encode_tc_min_slices(items[j].d_sae));
    Schedule& sc = schedule_buffer();
    build_schedule(items, n_items, max_ctas, dense, sc);
    const int groups = sc.groups;
    const int* order = sc.order;

    // scratch: every item's bounds, then every item's list lengths (one memset clears both: a row tile cut into fewer
    // pieces than the item's slot count leaves the other slots empty), then the lists
    unsigned char* base = static_cast<unsigned char*>(d_scratch);
    size_t hint_bytes = 0, count_bytes = 0;
    for (int q = 0; q < n_items; ++q) {
        const EncodeTcItem& it = items[order[q]];
        hint_bytes += round_up(static_cast<size_t>(it.T) * 4, 256);
        count_bytes += round_up(static_cast<size_t>(it.T) * sc.slots[q] * groups * 4, 256);
    }
    size_t hint_off = 0, count_off = hint_bytes, off = hint_bytes + count_bytes;
    for (int q = 0; q < n_items; ++q) {
        const EncodeTcItem& it = items[order[q]];
        ItemParams& ip = p.item[q];
        s3_status rc = make_map(&maps.x[q], it.d_x, static_cast<uint64_t>(it.T), static_cast<uint64_t>(it.d_in),
                                static_cast<uint64_t>(it.ldx), BM);
        if (rc != S3_OK) return rc;
        memcpy(&maps.w[q], it.st->map_w, sizeof(CUtensorMap));
        ip.T = it.T; ip.d_in = it.d_in; ip.k = it.k;
        ip.kblocks = (it.d_in + BK - 1) / BK;
        ip.n_mtiles = encode_tc_row_tiles(it.T);
        ip.n_col_tiles = encode_tc_col_tiles(it.d_sae);
        ip.n_slices = sc.slots[q];
        ip.unit_start = q == 0 ? 0 : p.item[q - 1].unit_start + p.item[q - 1].n_mtiles * p.item[q - 1].n_slices;
        ip.cap = encode_tc_list_cap(it.k, groups);
        ip.b_eff = it.st->d_b_eff;
        if (!dense) {
            const size_t t = static_cast<size_t>(it.T), sl = static_cast<size_t>(ip.n_slices) * groups;
            ip.hint = reinterpret_cast<uint32_t*>(base + hint_off);
            hint_off += round_up(t * 4, 256);
            ip.counts = reinterpret_cast<uint32_t*>(base + count_off);
            count_off += round_up(t * sl * 4, 256);
            ip.cand = reinterpret_cast<uint64_t*>(base + off);
            off += round_up(t * sl * ip.cap * sizeof(uint64_t), 256);
        }
    }
    p.n_units = sc.n_units;
    p.use_sched = sc.table ? 1 : 0;
    if (sc.table) {
        memcpy(p.pair_start, sc.pair_start, sizeof(p.pair_start));
        memcpy(p.unit, sc.unit, sizeof(UnitDesc) * static_cast<size_t>(sc.n_units));
    }
    // no bound is known for any row yet, and no list holds anything
    if (!dense) S3_CUDA_TRY(cudaMemsetAsync(base, 0, hint_bytes + (sc.table ? count_bytes : 0), stream));

    {
        int max_k = 0;
        for (int j = 0; j < n_items; ++j) max_k = items[j].k > max_k ? items[j].k : max_k;
        p.pend_cap = pend_cap_for(max_k);
    }
    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    int max_smem = 0;
    S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    int n_stages = 6;
    while (n_stages > 2 && static_cast<int>(smem_layout(n_stages, false, groups, p.pend_cap).total) + 1024 > max_smem) --n_stages;
    S3_REQUIRE(static_cast<int>(smem_layout(n_stages, false, groups, p.pend_cap).total) + 1024 <= max_smem, S3_ERR_UNSUPPORTED,
               "shared memory too small for the encode pipeline");
    p.n_stages = n_stages;
    const size_t smem = smem_layout(n_stages, false, groups, p.pend_cap).total + 1024;
    static bool attr_set[64] = {};
    if (dev < 64 && !attr_set[dev]) {
        S3_CUDA_TRY(cudaFuncSetAttribute(encode_tc_kernel<M_SELECT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
        S3_CUDA_TRY(cudaFuncSetAttribute(encode_tc_kernel<M_SELECT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
        S3_CUDA_TRY(cudaFuncSetAttribute(encode_tc_kernel<M_DENSE, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
        attr_set[dev] = true;
    }
    const int n_pairs = sc.n_pairs;

    if (dense) {
        encode_tc_kernel<M_DENSE, 1><<<2 * n_pairs, 64 + 128, smem, stream>>>(maps, p);
        S3_CUDA_TRY(cudaGetLastError());
        return S3_OK;
    }
    if (groups == 2) encode_tc_kernel<M_SELECT, 2><<<2 * n_pairs, 64 + 256, smem, stream>>>(maps, p);
    else encode_tc_kernel<M_SELECT, 1><<<2 * n_pairs, 64 + 128, smem, stream>>>(maps, p);
    S3_CUDA_TRY(cudaGetLastError());
    MergeGroup mg;
    mg.n_items = n_items;
    int rows = 0;
    for (int q = 0; q < n_items; ++q) {
        const EncodeTcItem& it = items[order[q]];
        const ItemParams& ip = p.item[q];
        mg.item[q] = MergeItem{ip.cand, ip.counts, ip.hint, it.d_ids, it.d_vals, it.T, ip.n_slices * groups, it.k, ip.cap, rows};
        rows += (it.T + kMergeRowsPerBlock - 1) / kMergeRowsPerBlock * kMergeRowsPerBlock;
    }
    launch_candidate_merge_group(mg, rows, stream);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}

}  // namespace

size_t encode_tc_group_workspace_need(const EncodeTcItem* items, int n_items, int max_ctas)
{
    if (n_items < 1 || n_items > MAX_GROUP) return 0;
    Schedule& sc = schedule_buffer();
    build_schedule(items, n_items, max_ctas, false, sc);
    size_t n = 0;
    for (int q = 0; q < n_items; ++q) n += encode_tc_workspace_bytes(items[sc.order[q]].T, sc.slots[q], items[sc.order[q]].k);
    return n;
}

// The units of the launch over these items on n_pairs CTA pairs, six integers each: pair, item (caller's index), row
// tile, first column tile, one past the last column tile, candidate-list slot. Returns the unit count (also when it
// exceeds max_units; only max_units are written), or -1 when the launch deals uniform slices round-robin without a table.
int encode_tc_describe_schedule(const EncodeTcItem* items, int n_items, int n_pairs, int32_t* out, int max_units, int32_t* slots_out)
{
    if (n_items < 1 || n_items > MAX_GROUP || n_pairs < 1) return -2;
    Schedule& sc = schedule_buffer();
    build_schedule(items, n_items, 2 * n_pairs, false, sc, n_pairs);
    for (int q = 0; q < n_items; ++q) slots_out[sc.order[q]] = sc.slots[q];
    if (!sc.table) return -1;
    for (int pr = 0; pr < sc.n_pairs; ++pr)
        for (int i = sc.pair_start[pr]; i < sc.pair_start[pr + 1]; ++i) {
            if (i >= max_units) continue;
            const UnitDesc& u = sc.unit[i];
            int32_t* o = out + static_cast<size_t>(i) * 6;
            o[0] = pr; o[1] = sc.order[u.item]; o[2] = u.mt; o[3] = u.tile_lo; o[4] = u.tile_hi; o[5] = u.slot;
        }
    return sc.n_units;
}

int encode_tc_group_ctas(const EncodeTcItem* items, int n_items, int max_ctas)
{
    if (n_items < 1 || n_items > MAX_GROUP) return 0;
    Schedule& sc = schedule_buffer();
    build_schedule(items, n_items, max_ctas, false, sc);
    return 2 * sc.n_pairs;
}

s3_status launch_encode_tc_group(const EncodeTcItem* items, int n_items, int max_ctas, void* d_scratch, uint32_t* d_status,
                                 cudaStream_t stream)
{
    return launch_tc(items, n_items, max_ctas, d_scratch, d_status, nullptr, 0, false, stream);
}

s3_status launch_encode_tc(const EncodeTcState* st, const void* d_x, int64_t ldx, int T, int d_in, int d_sae, int k,
                           int n_slices, int max_ctas, void* d_scratch, uint32_t* d_status, int32_t* d_ids, float* d_vals,
                           cudaStream_t stream)
{
    const EncodeTcItem it = {st, d_x, ldx, T, d_in, d_sae, k, n_slices, d_ids, d_vals};
    return launch_tc(&it, 1, max_ctas, d_scratch, d_status, nullptr, 0, false, stream);
}

s3_status launch_preact_tc(const EncodeTcState* st, const void* d_x, int64_t ldx, int T, int d_in, int d_sae, int n_slices,
                           int max_ctas, uint32_t* d_status, void* d_out, int64_t ld_out, bool out_bf16, cudaStream_t stream)
{
    const EncodeTcItem it = {st, d_x, ldx, T, d_in, d_sae, 1, n_slices, nullptr, nullptr};
    return launch_tc(&it, 1, max_ctas, nullptr, d_status, d_out, ld_out, out_bf16, stream);
}

// The (row tile, head) pairs of a projection launch as the row tiles of one 128-wide encoder, for the schedule.
static int proj_schedule_rows(int T, int n_heads) { return encode_tc_row_tiles(T) * n_heads * PAIR_M; }

size_t encode_proj_tc_workspace_bytes(int T, int n_heads, int k)
{
    return encode_tc_workspace_bound(proj_schedule_rows(T, n_heads), k);      // holds whatever pieces the launch cuts
}

// Projection of one head + encode of that head in the same CTA pair: h [T, d_model] -> x = h W_proj + b (bf16, kept in shared
// memory) -> Top-k of the d_head = 128 wide encoder, per (token, head).
s3_status launch_encode_proj_tc(const EncodeTcState* proj, const EncodeTcState* st, const void* d_h, int64_t ldh, int T, int d_model,
                                int n_heads, int d_sae, int k, int max_ctas, void* d_scratch, uint32_t* d_status, int32_t* d_ids,
                                float* d_vals, cudaStream_t stream)
{
    alignas(64) TensorMaps maps;
    static thread_local EncodeTcParams p;
    memset(&p, 0, sizeof(p));
    memset(&maps, 0, sizeof(maps));
    s3_status rc = make_map(&maps.x[0], d_h, static_cast<uint64_t>(T), static_cast<uint64_t>(d_model), static_cast<uint64_t>(ldh), BM);
    if (rc != S3_OK) return rc;
    rc = make_map(&maps.wk, proj->d_wt, static_cast<uint64_t>(n_heads) * PROJ_N, static_cast<uint64_t>(d_model),
                  static_cast<uint64_t>(d_model), PROJ_N / 2);
    if (rc != S3_OK) return rc;
    memcpy(&maps.w[0], st->map_w, sizeof(CUtensorMap));
    p.n_items = 1;
    p.status = d_status;
    p.d_sae = d_sae;
    p.proj_heads = n_heads;
    p.proj_kblocks = (d_model + BK - 1) / BK;
    p.proj_bias = proj->d_b_eff;
    ItemParams& ip = p.item[0];
    ip.T = T; ip.d_in = PROJ_N; ip.k = k; ip.kblocks = PROJ_N / BK;
    ip.n_mtiles = encode_tc_row_tiles(T);
    ip.n_col_tiles = encode_tc_col_tiles(d_sae);
    S3_REQUIRE(encode_tc_min_slices(d_sae) == 1, S3_ERR_UNSUPPORTED, "d_sae = %d is too wide for one column slice per head", d_sae);
    ip.unit_start = 0;
    constexpr int groups = 2;                  // d_head = 128: the narrow-encoder configuration
    ip.cap = encode_tc_list_cap(k, groups);
    ip.b_eff = st->d_b_eff;
    int n_pairs = encode_tc_max_pairs();
    if (max_ctas > 0 && max_ctas / 2 < n_pairs) n_pairs = max_ctas / 2 > 0 ? max_ctas / 2 : 1;
    if (n_pairs > MAX_PAIRS) n_pairs = MAX_PAIRS;
    // Units: whole (row tile, head) pairs when they fill the pairs' waves evenly; otherwise the column tiles of all
    // (row tile, head) pairs are cut at the pairs' shares like a narrow encoder's row tiles, every piece computing its
    // head's projection again first (64 k-blocks into half an accumulator: about two column tiles' worth of time).
    ip.n_slices = 1;
    p.n_units = ip.n_mtiles * n_heads;
    {
        const int waves = (p.n_units + n_pairs - 1) / n_pairs;
        const bool even = static_cast<double>(p.n_units) >= 0.93 * waves * n_pairs;
        const EncodeTcItem fake = {st, nullptr, 0, proj_schedule_rows(T, n_heads), PROJ_N, d_sae, k, 0, nullptr, nullptr};
        const int order0 = 0;
        Schedule& sc = schedule_buffer();
        const double proj_cost = 300.0 * p.proj_kblocks + 3000.0;
        if (!even && ip.n_mtiles * n_heads <= 65535 && plan_balanced(&fake, &order0, 1, n_pairs, groups, false, sc, proj_cost)) {
            ip.n_slices = sc.slots[0];
            p.n_units = sc.n_units;
            p.use_sched = 1;
            memcpy(p.pair_start, sc.pair_start, sizeof(p.pair_start));
            memcpy(p.unit, sc.unit, sizeof(UnitDesc) * static_cast<size_t>(sc.n_units));
            n_pairs = sc.n_pairs;
        } else if (p.n_units < n_pairs) n_pairs = p.n_units;
    }
    const size_t rows = static_cast<size_t>(T) * n_heads, lists = static_cast<size_t>(ip.n_slices) * groups;
    unsigned char* base = static_cast<unsigned char*>(d_scratch);
    ip.hint = reinterpret_cast<uint32_t*>(base);
    ip.counts = reinterpret_cast<uint32_t*>(base + round_up(rows * 4, 256));
    ip.cand = reinterpret_cast<uint64_t*>(base + round_up(rows * 4, 256) + round_up(rows * lists * 4, 256));
    // bounds, and the lengths of the lists (a row cut into fewer pieces than the slot count leaves the other slots empty)
    S3_CUDA_TRY(cudaMemsetAsync(base, 0, round_up(rows * 4, 256) + (p.use_sched ? rows * lists * 4 : 0), stream));

    int dev = 0;
    S3_CUDA_TRY(cudaGetDevice(&dev));
    int max_smem = 0;
    S3_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    p.pend_cap = pend_cap_for(k);
    int n_stages = 6;
    while (n_stages > 2 && static_cast<int>(smem_layout(n_stages, true, groups, p.pend_cap).total) + 1024 > max_smem) --n_stages;
    S3_REQUIRE(static_cast<int>(smem_layout(n_stages, true, groups, p.pend_cap).total) + 1024 <= max_smem, S3_ERR_UNSUPPORTED,
               "shared memory too small for the encode pipeline");
    p.n_stages = n_stages;
    const size_t smem = smem_layout(n_stages, true, groups, p.pend_cap).total + 1024;
    static bool attr_set[64] = {};
    if (dev < 64 && !attr_set[dev]) {
        S3_CUDA_TRY(cudaFuncSetAttribute(encode_tc_kernel<M_PROJ, groups>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
        attr_set[dev] = true;
    }
    encode_tc_kernel<M_PROJ, groups><<<2 * n_pairs, 64 + 128 * groups, smem, stream>>>(maps, p);
    S3_CUDA_TRY(cudaGetLastError());
    launch_candidate_merge(ip.cand, ip.counts, ip.hint, static_cast<int>(rows), static_cast<int>(lists), ip.cap, k, d_ids, d_vals, stream);
    S3_CUDA_TRY(cudaGetLastError());
    return S3_OK;
}


}  // namespace s3
