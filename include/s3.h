/*
 * s3scan -- C ABI of the B200 (sm_100a) streaming-scan hot path of S^3-Attention.
 *
 *   scan      : SAE encode + ReLU + Top-k  ->  per-chunk CSR postings  ->  async append to a host index
 *   retrieval : query feature aggregation  ->  span co-activation scores  ->  score fusion + top-s spans
 *
 * Conventions
 *   - Every function returns s3_status (0 = S3_OK, negative = error). No exception crosses the ABI.
 *     s3_last_error() gives a thread-local message for the last failing call on this thread.
 *   - Pointer names say where the memory lives: d_* = device, h_* = host. The CALLER owns every
 *     device buffer; the library never allocates or frees device memory. Sizes of caller-provided
 *     scratch come from the *_bytes() queries.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). All device work
 *     is enqueued on it and returns asynchronously; only s3_index_sync, s3_index_export_csr,
 *     s3_index_stats and s3_workspace_status wait for the device.
 *   - A workspace (`d_ws`) starts with a 64-byte status block. Zero it once before first use.
 *     A kernel whose bounded wait runs out writes a non-zero code there (sticky) and returns early;
 *     s3_workspace_status reads it. Calls that share one workspace must not overlap on the device.
 *   - Device pointers must be 16-byte aligned unless stated otherwise.
 *   - sm_100a only. There is no CPU path: without a CUDA device the compute entry points fail with
 *     S3_ERR_CUDA.
 */
#ifndef S3_H_
#define S3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t s3_status;
enum {
    S3_OK = 0,
    S3_ERR_INVALID_ARG = -1,  /* null / misaligned pointer, size out of range                      */
    S3_ERR_UNSUPPORTED = -2,  /* valid request outside the implemented limits (stated per call)    */
    S3_ERR_CUDA = -3,         /* a CUDA runtime/driver call failed (message has the CUDA error)    */
    S3_ERR_NOMEM = -4,        /* host (pinned) allocation failed                                   */
    S3_ERR_CAPACITY = -5,     /* a caller-provided buffer or an int32 position range is too small  */
    S3_ERR_TIMEOUT = -6,      /* a bounded device-side wait ran out (see s3_workspace_status)      */
    S3_ERR_STATE = -7         /* call not allowed in the object's current state                    */
};

typedef enum { S3_BF16 = 0, S3_F32 = 1 } s3_dtype;

#define S3_MAX_K 128           /* largest Top-k per token                                           */
#define S3_MAX_POSTINGS_ITEMS 32
#define S3_MAX_ENCODE_ITEMS 8    /* encoder calls one grouped launch can serve                        */
#define S3_MAX_SCORE_LAYERS 16
#define S3_WS_HEADER_BYTES 64

const char* s3_last_error(void);
int s3_version(void);

/* Reads the status block of a workspace after waiting for `stream`.
 * Returns S3_OK, or S3_ERR_TIMEOUT if a kernel gave up on a bounded wait; *code_out (nullable, host)
 * receives the raw code (which wait ran out). */
s3_status s3_workspace_status(const void* d_ws, void* stream, uint32_t* code_out);

/* ------------------------------------------------------------------------------------------------
 * SAE encode + ReLU + Top-k            (paper Sec. 3.3 Eq. 1-2; Sec. 3.4 Eq. 3; Sec. 3.5 Eq. 5)
 *
 *   pre[t,f] = sum_i W_enc[i,f] * (x[t,i] - b_dec[i]) + b_enc[f]
 *   per token: the min(k, #{f : pre[t,f] > 0}) largest strictly positive pre[t,.]; ids and values,
 *   ordered by (value descending, id ascending); the row is padded with id -1 / value 0.
 *   The [T, d_sae] pre-activation is never written to device memory.
 *
 * W_enc is [d_in, d_sae] row-major (feature f = column f), dtype bf16 or fp32; b_enc [d_sae] and
 * b_dec [d_in] are fp32. x is [T, d_in] row-major with row pitch ldx (elements), same dtype as W_enc.
 *
 * S3_BF16: products of bf16 inputs accumulated in fp32 on the tensor cores; b_dec is folded into an
 *          effective bias b_eff[f] = b_enc[f] - sum_i W_enc[i,f] b_dec[i] (fp64 sum, stored fp32).
 *          Requires d_in % 8 == 0, ldx % 8 == 0, d_sae % 8 == 0.
 * S3_F32 : fp32 FMA accumulation of W_enc[i,f] * (x[t,i] - b_dec[i]) in index order, no folding.
 * Limits : 1 <= k <= min(S3_MAX_K, d_sae); d_sae <= 65536 * 4; anything else -> S3_ERR_UNSUPPORTED /
 *          S3_ERR_INVALID_ARG. T == 0 is a no-op.
 *
 * s3_sae_create runs a one-time preparation on `stream` (bf16: a K-major copy of W_enc and b_eff)
 * into the caller's `d_prepared` buffer of s3_sae_prepared_bytes() bytes, which must stay alive and
 * untouched, like W_enc/b_enc/b_dec themselves, for the life of the handle. The handle is host
 * memory only.
 * ---------------------------------------------------------------------------------------------- */
typedef struct s3_sae s3_sae;

size_t s3_sae_prepared_bytes(int d_in, int d_sae, s3_dtype dtype);
s3_status s3_sae_create(s3_sae** out, const void* d_W_enc, const float* d_b_enc, const float* d_b_dec,
                        int d_in, int d_sae, s3_dtype dtype, void* d_prepared, size_t prepared_bytes,
                        void* stream);
s3_status s3_sae_destroy(s3_sae* sae);
/* Scratch for the per-slice Top-k candidate lists of up to T_max tokens (includes the status block). */
size_t s3_sae_encode_workspace_bytes(const s3_sae* sae, int T_max, int k);
s3_status s3_sae_encode_topk(const s3_sae* sae, const void* d_x, int64_t ldx, int T, int k,
                             int32_t* d_ids /*[T,k]*/, float* d_vals /*[T,k]*/,
                             void* d_ws, size_t ws_bytes, void* stream);
/* The same GEMM with a dense epilogue: d_out [T, ld_out] (fp32 or bf16, rounded to nearest even) receives the
 * pre-activations pre[t,f] of Eq. 1 before the ReLU, nothing is selected. With zero biases this is a plain projection
 * x W (e.g. the key projection K = W_K h, paper appendix on chunk-independent prefill, whose output feeds
 * s3_sae_encode_topk on the same stream while it is still in the L2 cache); it also serves to inspect an encoder.
 * bf16 encoders only (S3_ERR_UNSUPPORTED otherwise). ld_out must be a multiple of 8 (bf16) or 4 (fp32) and >= d_sae;
 * d_out 16-byte aligned. Workspace: the 64-byte status block only. */
s3_status s3_sae_preact(const s3_sae* sae, const void* d_x, int64_t ldx, int T, void* d_out, int64_t ld_out,
                        s3_dtype out_dtype, void* d_ws, size_t ws_bytes, void* stream);
/* Tuning knob: number of uniform column slices each row block of the encode is split into (0 = the launch cuts its own
 * work units, see s3_encode_schedule_describe) and the largest number of thread blocks a launch may use (0 = all SMs).
 * Results do not depend on either. */
s3_status s3_sae_set_schedule(s3_sae* sae, int n_slices, int max_ctas);

/* ------------------------------------------------------------------------------------------------
 * Grouped SAE encode + Top-k            (paper Alg. 1 Phase 1: inside each chunk the scan loops over the
 *                                        target layers, `for l in TargetLayers: feats <- E_l.encode(K_l)`;
 *                                        Sec. 3.3 / 3.4: one SAE per target layer)
 *
 * Up to S3_MAX_ENCODE_ITEMS independent encoder calls (the layers' key SAEs of one chunk, key and query SAEs
 * together, ...) as ONE persistent launch followed by one selection launch: the work units of all items are
 * cut and dealt out over the SMs by their modelled duration, so the SMs stay busy across items of unequal size and
 * the launch ends evenly. Each item has its own encoder, input, T, k and outputs; the results are those of
 * s3_sae_encode_topk item by item (bit-identical: the selection is exact, whatever the schedule).
 * bf16 encoders only (S3_ERR_UNSUPPORTED otherwise); an item with T == 0 is skipped. `h_items` is a HOST
 * array. max_ctas > 0 limits the launch to that many thread blocks (an even number is used), for launches that
 * share the GPU with another stream's kernel. Workspace: s3_sae_encode_grouped_workspace_bytes(h_items, n_items) (status block + room for every item's
 * candidate lists under any schedule; it grows with T, so the size for a full chunk also serves a shorter last one).
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    const s3_sae* sae;
    const void* d_x;     /* [T, d_in] with row pitch ldx */
    int64_t ldx;
    int32_t T, k;
    int32_t* d_ids;      /* [T,k] */
    float* d_vals;       /* [T,k] */
} s3_encode_item;

size_t s3_sae_encode_grouped_workspace_bytes(const s3_encode_item* h_items, int n_items);
s3_status s3_sae_encode_topk_grouped(const s3_encode_item* h_items, int n_items, int max_ctas /*0 = all SMs*/,
                                     void* d_ws, size_t ws_bytes, void* stream);
/* Thread blocks (one per SM) that s3_sae_encode_topk will occupy for T tokens: a launch over few work units leaves SMs
 * free, on which a grouped launch limited with max_ctas can run at the same time from another stream. */
int s3_sae_encode_ctas(const s3_sae* sae, int T);
/* The work units a launch over n_items bf16 encoder calls (HOST arrays T, d_in, d_sae, k) is cut into on n_pairs pairs of
 * thread blocks; host arithmetic only, no device is touched. A unit is a run of 256-column tiles of one 256-token row
 * tile of one item, and its survivors go to one of the row's candidate lists ("slot"). Encoders whose weights stay in L2
 * are cut into one contiguous share of equal modelled duration per pair (pieces of at least three column tiles, a row
 * tile spread over neighbouring pairs); wider encoders walk bands of row tiles with uniform column slices in step, so that the pairs of a
 * slice read the same weight tiles at the same time and a band's token tiles stay in L2. Writes six integers per unit to h_units (pair, item, row tile, first column
 * tile, one past the last, slot), at most max_units units, and every item's slots per row to h_slots [n_items].
 * Returns the number of units, -1 when the launch deals uniform slices round-robin without a unit table (only h_slots is
 * written), -2 on invalid arguments. The selection result never depends on the schedule (Eq. 3 is exact). */
int s3_encode_schedule_describe(const int32_t* T, const int32_t* d_in, const int32_t* d_sae, const int32_t* k, int n_items,
                                int n_pairs, int32_t* h_units, int max_units, int32_t* h_slots);

/* ------------------------------------------------------------------------------------------------
 * Upstream projection fused with the per-head encode
 *            (paper appendix on chunk-independent prefill: the keys of a chunk are K = W_K h; Sec. 3.3: the SAE
 *             reads one head's projection, x in R^d_head, with one encoder and one feature-ID space for all heads)
 *
 * `proj` is a bf16 handle (s3_sae_create) over W_proj [d_model, n_heads * 128] with bias b_enc and b_dec = 0, i.e.
 * x = h W_proj + b; `sae` is the bf16 encoder of one head (d_in = 128). For every token t and head j:
 *     x[t,j,:] = bf16(h[t,:] W_proj[:, 128 j : 128 (j+1)] + b)         (fp32 accumulation, round to nearest even)
 *     ids / vals [t,j,:] = the Top-k code of x[t,j,:] as s3_sae_encode_topk defines it.
 * A CTA pair computes the head's 256 x 128 tile of x, keeps it in shared memory as the encode GEMM's token operand and
 * runs the encoder's column tiles on it, so x reaches neither HBM nor L2. The result equals, bit for bit,
 * s3_sae_preact (bf16 output) followed by s3_sae_encode_topk on the [T * n_heads, 128] view, and feeds
 * s3_head_aggregate_topk. h is [T, d_model] bf16 with row pitch ldh (multiple of 8).
 * Limits: d_head = 128 exactly; k <= S3_MAX_K; d_sae <= 65280. Workspace:
 * s3_sae_project_encode_workspace_bytes(sae, T, n_heads, k).
 * ---------------------------------------------------------------------------------------------- */
size_t s3_sae_project_encode_workspace_bytes(const s3_sae* sae, int T_max, int n_heads, int k);
s3_status s3_sae_project_encode_topk(const s3_sae* proj, const s3_sae* sae, const void* d_h, int64_t ldh, int T, int n_heads,
                                     int k, int32_t* d_ids /*[T,n_heads,k]*/, float* d_vals /*[T,n_heads,k]*/,
                                     void* d_ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * SAE encode + ReLU + Top-k without any caller-provided scratch
 *
 * (The paper has no counterpart of this call: it exists for the way some programs have to use this
 *  library, not for the method.)
 *
 * Same result as s3_sae_encode_topk, for callers that cannot allocate device memory: a serving
 * process whose memory pool is sized once and then frozen, a plugin that only ever sees the input
 * and output buffers its host framework passes in, code that runs while something else owns the
 * allocator. The partial Top-k lists that s3_sae_encode_topk keeps in the caller's `d_ws` live
 * here in an array of S3_STATIC_SCRATCH_BYTES bytes built into the library image. Each GPU that
 * loads the library carries that array until the process exits. The call itself allocates and
 * frees nothing, on the host side of CUDA or through any library.
 *
 *   - Size limit: the call is refused with S3_ERR_CAPACITY when
 *     s3_sae_encode_workspace_bytes(sae, T, k) > S3_STATIC_SCRATCH_BYTES (for bf16 encoders with 16 or
 *     more column tiles that is about T*k <= 8100, e.g. 250 tokens at k = 32). Split longer inputs by
 *     token range.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and remembers it. Make that first call before starting any stream capture.
 *   - One array per device, shared by every call and keeping the previous call's contents. The
 *     call clears the 64-byte status block at its start and rewrites the lists it uses, so stale
 *     contents never reach a result. Two calls whose device work overlaps (different streams or
 *     threads, same device) race on the array: order them on one stream or with events.
 *   - d_status_out (device, 4 bytes, nullable) receives the status word of this call on `stream`
 *     after the kernels: 0, or the code of a bounded wait that ran out (as s3_workspace_status).
 * Inputs, outputs, alignment rules, dtype rules and asynchrony are those of s3_sae_encode_topk.
 * ---------------------------------------------------------------------------------------------- */
#define S3_STATIC_SCRATCH_BYTES (16u << 20)
s3_status s3_sae_encode_topk_static(const s3_sae* sae, const void* d_x, int64_t ldx, int T, int k,
                                    int32_t* d_ids /*[T,k]*/, float* d_vals /*[T,k]*/,
                                    uint32_t* d_status_out /*nullable*/, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Postings build                                       (paper Sec. 3.4 Eq. 4: I[f] <- I[f] U {t})
 *
 * Groups the (feature, position) pairs of one chunk of one layer into a CSR:
 *   row_ptr[f] = number of pairs with id < f  (row_ptr has d_sae + 1 entries, uint32)
 *   pos[row_ptr[f] .. row_ptr[f+1]) = ascending absolute positions pos_base + t with f in F_t
 * ids [T,k] int32; entries < 0 are padding and are skipped; ids within a token must be distinct (a repeated id
 * keeps both of its pairs and is reported through the workspace status as S3_ERR_INVALID_ARG, as is an
 * id >= d_sae, whose pair is dropped).
 * d_vals / d_pval (both null or both non-null) carry each pair's activation next to its position.
 * d_pos (and d_pval) must hold T*k entries. The result is bit-exact and run-to-run identical.
 * Limits: d_sae <= 2^20, k <= 4096, T*k <= 2^27, pos_base + T <= 2^31 - 1 (S3_ERR_CAPACITY: positions are
 *         int32); ceil(log2 T) + ceil(log2(d_sae / 2048)) <= 32 (S3_ERR_UNSUPPORTED; only dictionaries beyond
 *         65536 features meet it, at more than 2^23 tokens per item). T == 0 writes zeros to row_ptr.
 * Workspace: the status block, the item's pairs regrouped by feature range (4 bytes per pair, 8 with values)
 * and a small directory; s3_postings_workspace_bytes(T, k, d_sae) bounds it for one item, and a batch needs
 * the sum of its items' values. The batched form processes up to S3_MAX_POSTINGS_ITEMS independent
 * chunk-layers in two launches; `items` is a HOST array. Batches that follow one another on a stream should
 * share one workspace: the regrouped pairs are then rewritten in place and stay in the L2 cache.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    const int32_t* d_ids;
    const float* d_vals; /* nullable */
    int32_t T, k, d_sae, reserved;
    int64_t pos_base;
    uint32_t* d_row_ptr; /* [d_sae+1] */
    int32_t* d_pos;      /* [T*k]     */
    float* d_pval;       /* nullable  */
} s3_postings_item;

size_t s3_postings_workspace_bytes(int T_max, int k, int d_sae);
s3_status s3_postings_build(const int32_t* d_ids, const float* d_vals, int T, int k, int d_sae,
                            int64_t pos_base, uint32_t* d_row_ptr, int32_t* d_pos, float* d_pval,
                            void* d_ws, size_t ws_bytes, void* stream);
s3_status s3_postings_build_batched(const s3_postings_item* h_items, int n_items,
                                    void* d_ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Host-resident inverted index                         (paper Sec. 3.4: the index lives on the CPU and
 *                                                        device memory is bounded by the chunk size)
 *
 * s3_index_append enqueues, without blocking the host: an event on `producer_stream`, then on the
 * index's own copy stream device->pinned-host copies of row_ptr (d_sae+1 words) and of T*k
 * positions (and values if d_pval != NULL). Chunks of one layer must arrive in ascending,
 * non-overlapping position order (else S3_ERR_STATE). The device buffers may be overwritten once
 * the copy is done: pass the stream that will overwrite them to s3_index_stream_wait (device-side
 * wait, host does not block), or use *reuse_event_out (a cudaEvent_t owned by the index, valid
 * until the next append of the same layer).
 * Pinned memory grows in slabs of `pinned_slab_bytes`; growing calls the pinned allocator, which
 * may synchronise the device, so reserve up front (s3_index_reserve) for an uninterrupted scan.
 * ---------------------------------------------------------------------------------------------- */
typedef struct s3_index s3_index;
typedef struct {
    int64_t n_chunks;        /* appended chunk-layers                       */
    int64_t n_postings;      /* sum of row_ptr[d_sae] over synced segments  */
    int64_t host_bytes;      /* pinned bytes in use                         */
    int64_t host_bytes_reserved;
    int64_t max_list_len;    /* longest merged posting list over all layers */
    int64_t n_positions;     /* largest position + 1 seen                   */
} s3_index_stats_t;

s3_status s3_index_create(s3_index** out, int n_layers, int d_sae, size_t pinned_slab_bytes);
s3_status s3_index_reserve(s3_index* index, size_t bytes);
s3_status s3_index_append(s3_index* index, int layer, const uint32_t* d_row_ptr, const int32_t* d_pos,
                          const float* d_pval, int T, int k, int64_t pos_base, void* producer_stream,
                          void** reuse_event_out /*nullable*/);
s3_status s3_index_stream_wait(s3_index* index, void* stream);
/* Waits for every copy; checks that each segment's row_ptr is monotone and ends at <= T*k. */
s3_status s3_index_sync(s3_index* index);
s3_status s3_index_stats(s3_index* index, s3_index_stats_t* out);
s3_status s3_index_layer_postings(s3_index* index, int layer, uint64_t* n_out);
/* Merges the layer's chunk segments into one CSR on the host: per feature the chunk lists
 * concatenated in arrival order (ascending positions). h_row_ptr [d_sae+1] uint64; h_pos (and
 * h_pval, nullable) must hold s3_index_layer_postings() entries. */
s3_status s3_index_export_csr(s3_index* index, int layer, uint64_t* h_row_ptr, int32_t* h_pos, float* h_pval);
s3_status s3_index_destroy(s3_index* index);

/* ------------------------------------------------------------------------------------------------
 * Co-activation span scoring + fusion + top-s
 *            (paper Sec. 3.5 Eq. 5-6 and the appendix IDF definition; fixed-width spans, min-count
 *             score and score fusion follow the benchmark definition, see below)
 *
 * Spans: span j covers positions [j*stride, j*stride + width); n_spans = (L - width)/stride + 1
 * (0 if L < width); positions after the last full span are ignored.
 * Per query q and layer l, from the query tokens' Top-k (q_ids/q_vals [n_layers, Q, nq, k], ids < 0
 * skipped):  cQ(f) = number of query tokens whose set contains f,  aQ(f) = sum of their activations
 * (fp32, token order).
 *   mode S3_SCORE_MINCOUNT : base[q,j] = sum_l sum_f min(cQ_l(f), cS_l(f,j))          (integer, exact)
 *   mode S3_SCORE_WEIGHTED : base[q,j] = sum_l sum_f aQ_l(f) * IDF_l(f) * cS_l(f,j)   (Eq. 6 summed over
 *        the span; IDF(f) = 1/(ln(1+freq(f))+1), freq = the feature's posting-list length in layer l;
 *        features with freq > stop_freq are skipped when stop_freq > 0). The weights aQ*IDF (fp64) are
 *        rounded to a fixed-point grid of at least 40 bits below the query's largest weight and summed as
 *        integers, so the result does not depend on the order of the additions: it is identical from run
 *        to run, and within 1e-5 (relative) of the fp64 sum whenever a span's weights lie within a factor
 *        2^20 of the query's largest.
 * with cS_l(f,j) = number of postings of f inside span j.
 * Fusion: score = fl32(fl32(alpha*base) + fl32(beta*bm25[q,j])) (bm25 nullable: score = fl32(alpha*base)).
 * Output: the s best spans per query by (score descending, span index ascending); padded with
 * index -1 / score 0 when n_spans < s. d_all_scores (nullable) receives every fused score.
 *
 * `h_layers` is a HOST array of n_layers views whose pointers are DEVICE pointers to one merged CSR
 * per layer (row_ptr uint64 [d_sae+1], pos int32 ascending per feature).
 * Limits: n_layers <= S3_MAX_SCORE_LAYERS; nq*k <= 4096; n_spans <= 16384; s <= 64;
 *         width, stride >= 1. Per query the kernel keeps 4 (min-count) or 8 (weighted) bytes per span and
 *         about 28 bytes per query entry in shared memory; a combination beyond the SM's capacity
 *         (only weighted mode near both maxima) returns S3_ERR_UNSUPPORTED. n_spans == 0 (L < width) writes
 *         index -1 / score 0 for every query and reads no posting.
 * Workspace: the status block is enough (then one thread block works on each query). With
 *         s3_score_workspace_bytes(Q, ...) bytes a batch of few queries is cut over several blocks per query
 *         (a single query runs on up to 148 of them); the blocks add their partial sums in the workspace,
 *         which the call clears first. Results are the same either way.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    const uint64_t* d_row_ptr;
    const int32_t* d_pos;
} s3_csr_view;

enum { S3_SCORE_MINCOUNT = 0, S3_SCORE_WEIGHTED = 1 };

typedef struct {
    int32_t width, stride, mode, s;
    float alpha, beta;
    int64_t stop_freq; /* 0 = off */
} s3_score_params;

size_t s3_score_workspace_bytes(int Q, int nq, int k, int n_layers, int n_spans, int s);
s3_status s3_coactivation_score_topspans(const s3_csr_view* h_layers, int n_layers, int d_sae, int64_t L,
                                         const int32_t* d_q_ids, const float* d_q_vals, int Q, int nq, int k,
                                         const s3_score_params* params, const float* d_bm25, int64_t ld_bm25,
                                         int32_t* d_top_idx /*[Q,s]*/, float* d_top_score /*[Q,s]*/,
                                         float* d_all_scores /*[Q,n_spans] nullable*/,
                                         void* d_ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Per-position relevance, semantic density and peak selection
 *            (paper Sec. 3.5 Eq. 6 "Semantic Density Estimation" and "Adaptive Granularity";
 *             Alg. 1 Phase 2: S <- accumulate, S' <- Conv1D(S), Idx <- NMS_Select(S', top_k))
 *
 * Per query q, with the query aggregation of s3_coactivation_score_topspans (aQ_l(f) = the query tokens'
 * activations of f summed in fp32 in token order; IDF_l(f) = 1/(ln(1+freq_l(f))+1), freq = posting-list
 * length; lists longer than stop_freq > 0 are skipped):
 *   S[t]  = sum_l sum_{f in query} [t in I_l[f]] * w_l(f),     w_l(f) = rint(aQ_l(f) * IDF_l(f) * 2^24) / 2^24
 *   S'[t] = sum_{d=0}^{K-1} S[t - floor(K/2) + d]               (box of K = conv_kernel unit taps centred on t,
 *                                                                 positions outside [0, L) count as 0)
 *   centres: n_centers rounds of "alive position with the largest S' (ties: lowest position)"; a round finds
 *            nothing once no alive position has S' > 0 (centre -1, density 0); positions within nms_radius
 *            of a chosen centre are no longer alive.
 * The fixed-point weights make S and S' exact integer sums, so the peaks do not depend on the order in
 * which postings are visited and are bit-identical to the CPU definition. The shape of the smoothing
 * kernel, the suppression rule and the multi-token aggregation are readings of points the paper leaves open.
 *
 * h_layers as for s3_coactivation_score_topspans. Outputs: d_centers [Q, n_centers] int32, d_center_density
 * [Q, n_centers] fp32 (S' at the centre); d_S / d_density (nullable) [Q, L] fp32 copies of S and S'.
 * Limits: n_layers <= S3_MAX_SCORE_LAYERS; nq*k <= 4096; 1 <= conv_kernel <= 1024; nms_radius >= 0;
 *         1 <= n_centers <= 1024; L <= 4194304.
 * Workspace: s3_density_workspace_bytes(Q, L, n_layers, d_sae, nq, k): two 64-bit words per query and
 *         position, the queries' unique features and weights (12 bytes per query entry and layer), one 32-bit
 *         offset per layer, feature and tile of 8192 positions, plus the status block.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t conv_kernel, nms_radius, n_centers, reserved;
    int64_t stop_freq; /* 0 = off */
} s3_density_params;

size_t s3_density_workspace_bytes(int Q, int64_t L, int n_layers, int d_sae, int nq, int k);
s3_status s3_position_density_topcenters(const s3_csr_view* h_layers, int n_layers, int d_sae, int64_t L,
                                         const int32_t* d_q_ids, const float* d_q_vals, int Q, int nq, int k,
                                         const s3_density_params* params, int32_t* d_centers /*[Q,n_centers]*/,
                                         float* d_center_density /*[Q,n_centers]*/, float* d_S /*[Q,L] nullable*/,
                                         float* d_density /*[Q,L] nullable*/, void* d_ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Head aggregation + Top-k       (paper Sec. 3.3: the SAE reads one head's projection, x in R^d_head, with one
 *                                 feature-ID space for all of them; Sec. 3.4 defines k as the per-token sparsity
 *                                 once the heads are aggregated. The rule itself is not given; this is the reading.)
 *
 * d_ids / d_vals [T, H, k] hold, per token, the Top-k codes of its H heads (e.g. s3_sae_encode_topk on the
 * [T*H, d_head] view of the projections). Per token: a(f) = sum of f's activations over the heads whose code
 * holds it (fp32, heads in ascending order; id < 0 or >= d_sae skipped); output the k_out features with the
 * largest a(f) > 0 by (a descending, id ascending), padded with id -1 / value 0. The result has the layout
 * of an encode result and feeds s3_postings_build.
 * Limits: H*k <= 4096; k_out <= 4096; d_sae <= 2^20. No workspace. T == 0 is a no-op.
 * ---------------------------------------------------------------------------------------------- */
s3_status s3_head_aggregate_topk(const int32_t* d_ids, const float* d_vals, int T, int H, int k, int d_sae, int k_out,
                                 int32_t* d_out_ids /*[T,k_out]*/, float* d_out_vals /*[T,k_out]*/, void* stream);

/* ------------------------------------------------------------------------------------------------
 * SAE decode                     (paper Sec. 3.3, the reconstruction stated after Eq. 2:
 *                                 x_hat = z_hat W_dec + b_dec)
 *
 * z_hat is the Top-k code as returned by s3_sae_encode_topk: d_ids / d_vals [T, k], id < 0 (padding) or
 * id >= d_sae contributing nothing. W_dec is [d_sae, d_in] row-major (row f = direction of feature f), bf16
 * or fp32; b_dec fp32 [d_in]. Per token the k scaled rows are added in the order given with fp32 FMAs
 * starting from 0, b_dec last.
 *   d_xhat  (nullable) fp32 [T, ld_xhat]  : the reconstruction;
 *   d_sqerr (nullable) fp32 [T]           : sum_i (x[t,i] - x_hat[t,i])^2 against d_x [T, ldx] (same dtype as
 *                                           W_dec), the per-token reconstruction error (fp32, fixed order).
 * At least one of the two is required. Limits: 1 <= k <= S3_MAX_K; d_in a multiple of 8 (bf16) or 4 (fp32);
 * pitches multiples of 4 (x_hat) and of 8 / 4 (x). No workspace. T == 0 is a no-op.
 * ---------------------------------------------------------------------------------------------- */
s3_status s3_sae_decode(const void* d_W_dec, const float* d_b_dec, int d_in, int d_sae, s3_dtype dtype,
                        const int32_t* d_ids, const float* d_vals, int T, int k,
                        float* d_xhat, int64_t ld_xhat, const void* d_x, int64_t ldx, float* d_sqerr, void* stream);

/* ------------------------------------------------------------------------------------------------
 * SAE training step on fp32 parameters      (paper appendix, training configuration: Top-K SAEs trained with
 *                                             Adam, learning rate 1e-3, batches of 4096 tokens; Sec. 3.3 for the
 *                                             model. The loss is not printed; reading below.)
 *
 * s3_sae_backward: with z_hat the Top-k code of the batch (d_ids / d_vals [T, k] from s3_sae_encode_topk on the
 * same parameters; id < 0 = padding) and x_hat = z_hat W_dec + b_dec,
 *     loss = (1/T) sum_t ||x_hat_t - x_t||^2,
 * and its gradients through the code with the active set held fixed (z[t,j] = W_enc[:,f].(x_t - b_dec) + b_enc[f]
 * for the selected f):  gW_enc [d_in, d_sae], gb_enc [d_sae], gW_dec [d_sae, d_in], gb_dec [d_in], all fp32 and
 * overwritten. The sums over tokens are fp32 atomics (no fixed order); the loss is added in a fixed order.
 * d_vals may be NULL: z is then recomputed in fp32 from W_enc, b_enc, b_dec and x for the given ids, which is the
 * form to use when the ids come from a bf16 forward pass over a bf16 copy of the parameters (s3_cast_f32_to_bf16,
 * s3_sae_create with S3_BF16): the tensor cores pick the active set, the gradient is taken in fp32.
 * All arrays fp32, x with row pitch ldx. Limits: 1 <= k <= S3_MAX_K, d_in <= 4096, T >= 1.
 * Workspace: s3_sae_backward_workspace_bytes(T).
 *
 * s3_adam_update: one Adam step on n parameters, in place (Kingma & Ba):
 *     m = beta1 m + (1-beta1) g;  v = beta2 v + (1-beta2) g^2;
 *     p -= lr * (m / (1-beta1^step)) / (sqrt(v / (1-beta2^step)) + eps),        step counted from 1.
 * A training step is: encode -> backward -> one update per parameter tensor (-> s3_sae_create again for bf16 use).
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    float lr, beta1, beta2, eps;
    int32_t step, reserved;
} s3_adam_params;

size_t s3_sae_backward_workspace_bytes(int T);
s3_status s3_sae_backward(const float* d_W_enc, const float* d_b_enc /*nullable with d_vals*/, const float* d_W_dec,
                          const float* d_b_dec, const float* d_x, int64_t ldx,
                          const int32_t* d_ids, const float* d_vals, int T, int k, int d_in, int d_sae,
                          float* d_gW_enc, float* d_gb_enc, float* d_gW_dec, float* d_gb_dec, float* d_loss,
                          void* d_ws, size_t ws_bytes, void* stream);
s3_status s3_cast_f32_to_bf16(const float* d_src, void* d_dst, size_t n, void* stream);   /* round to nearest even */
s3_status s3_adam_update(float* d_param, float* d_m, float* d_v, const float* d_grad, size_t n,
                         const s3_adam_params* params, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Compact inverted index        (paper Sec. 3.4, memory analysis: contiguous integer arrays with delta
 *                                encoding and optional stop-feature pruning; the appendix's hard frequency
 *                                threshold for stop features. The layout is this library's.)
 *
 * One layer's merged CSR (row_ptr uint64 [d_sae+1], pos int32 strictly ascending per feature) becomes
 *   row_ptr   uint64 [d_sae+1] : prefix sum of the KEPT list lengths; a feature whose list is longer than
 *                                stop_freq > 0 keeps no postings (it then counts as absent in every
 *                                scoring mode, and the kept features' freq, hence IDF, is unchanged);
 *   blk_ptr   uint32 [d_sae+1] : prefix sum of the lists' block counts, a list of n postings having
 *                                ceil(n/32) blocks of 32 postings (the last one shorter);
 *   blk_first int32  [n_blocks]: first position of the block;
 *   blk_desc  uint64 [n_blocks]: (word offset of the block's payload << 6) | width, width = bit length of
 *                                the largest (gap - 1) between consecutive positions inside the block;
 *   payload   uint32 [n_words] : per block of c postings its c-1 values (gap - 1), `width` bits each, back
 *                                to back from bit 0 of the block's first word, least significant bit first,
 *                                in ceil((c-1)*width/32) words; one zero word closes the array.
 * A full block takes 12 bytes plus ceil(31*width/32) words instead of 128 bytes.
 *
 * s3_compact_bound gives capacities that always suffice (blocks <= n/32 + min(n, d_sae), words <= n + 1).
 * s3_compact_build runs five small kernels on `stream`; d_sizes (device, 4 x uint64) receives
 * {kept postings, n_blocks, n_words, 0}. If a capacity is too small nothing beyond it is written, the
 * workspace status is set (s3_workspace_status returns S3_ERR_CAPACITY) and d_sizes holds what is needed
 * as far as it was computed. Workspace: s3_compact_workspace_bytes(n_postings, d_sae).
 *
 * s3_coactivation_score_topspans_compact is s3_coactivation_score_topspans reading this form: a warp
 * decodes a block with one prefix sum; results are identical to scoring the pruned CSR.
 *
 * s3_compact_save / s3_compact_file_info / s3_compact_load move HOST copies of the arrays to and from a
 * file (checksummed per layer; load verifies the checksum and that every offset stays inside its array,
 * and refuses the file otherwise with S3_ERR_INVALID_ARG). In s3_compact_load the caller provides
 * buffers with capacities in n_blocks / n_words (from s3_compact_file_info); the actual sizes are written
 * back. I/O failures return S3_ERR_STATE.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    const uint64_t* d_row_ptr;
    const uint32_t* d_blk_ptr;
    const int32_t* d_blk_first;
    const uint64_t* d_blk_desc;
    const uint32_t* d_payload;
} s3_compact_view;

typedef struct {
    uint64_t* h_row_ptr;
    uint32_t* h_blk_ptr;
    int32_t* h_blk_first;
    uint64_t* h_blk_desc;
    uint32_t* h_payload;
    uint64_t n_blocks, n_words;
} s3_compact_host_layer;

s3_status s3_compact_bound(uint64_t n_postings, int d_sae, uint64_t* max_blocks, uint64_t* max_words);
size_t s3_compact_workspace_bytes(uint64_t n_postings, int d_sae);
s3_status s3_compact_build(const uint64_t* d_row_ptr, const int32_t* d_pos, uint64_t n_postings, int d_sae,
                           int64_t stop_freq, uint64_t* d_out_row_ptr, uint32_t* d_blk_ptr, int32_t* d_blk_first,
                           uint64_t* d_blk_desc, uint64_t cap_blocks, uint32_t* d_payload, uint64_t cap_words,
                           uint64_t* d_sizes /*[4]*/, void* d_ws, size_t ws_bytes, void* stream);
s3_status s3_coactivation_score_topspans_compact(const s3_compact_view* h_layers, int n_layers, int d_sae, int64_t L,
                                                 const int32_t* d_q_ids, const float* d_q_vals, int Q, int nq, int k,
                                                 const s3_score_params* params, const float* d_bm25, int64_t ld_bm25,
                                                 int32_t* d_top_idx, float* d_top_score, float* d_all_scores,
                                                 void* d_ws, size_t ws_bytes, void* stream);
/* Writes the kept postings back as a plain position array (d_pos, cap_postings entries; the CSR's row_ptr is the
 * view's own d_row_ptr): the inverse of s3_compact_build on the pruned index. A d_pos that is too small sets the
 * workspace status (S3_ERR_CAPACITY from s3_workspace_status) and writes nothing. *h_view holds device pointers. */
s3_status s3_compact_expand(const s3_compact_view* h_view, int d_sae, int32_t* d_pos, uint64_t cap_postings,
                            void* d_ws, size_t ws_bytes, void* stream);
s3_status s3_compact_save(const char* path, int n_layers, int d_sae, const s3_compact_host_layer* h_layers);
s3_status s3_compact_file_info(const char* path, int* n_layers, int* d_sae, uint64_t* h_n_blocks, uint64_t* h_n_words,
                               int cap_layers);
s3_status s3_compact_load(const char* path, int n_layers, int d_sae, s3_compact_host_layer* h_layers);

/* ------------------------------------------------------------------------------------------------
 * Hybrid fusion of index sets                  (paper Sec. 3.6 Eq. 7: M_final = M_S3 U M_BM25 U M_Bias;
 *                                               Alg. 1 Phase 3: Idx_Final <- Idx_S3 U Idx_Lexical U LeadTail)
 *
 * Per query q, the ascending, duplicate-free positions in [0, L) of
 *   M_S3   : the window [c - span_width/2, c - span_width/2 + span_width) around every centre c >= 0 of
 *            d_centers [Q, n_centers] (as returned by s3_position_density_topcenters; the paper's rule for
 *            variable-length spans is not given, a fixed window centred on the peak stands in),
 *   M_BM25 : the supplied lexical positions d_lexical [Q, n_lex] (nullable; entries < 0 are padding,
 *            entries >= L are ignored),
 *   M_Bias : the first `lead` and the last `tail` positions.
 * d_out_idx [Q, cap] int32 receives the positions (-1 after the last one), d_out_count [Q] the size of the
 * set; when it exceeds cap only the cap lowest positions are written. The caller gathers tokens with them.
 * Workspace: s3_fuse_workspace_bytes(Q, L) (one bit per query and position, plus the status block).
 * ---------------------------------------------------------------------------------------------- */
size_t s3_fuse_workspace_bytes(int Q, int64_t L);
s3_status s3_fuse_index_sets(const int32_t* d_centers, int Q, int n_centers, int span_width,
                             const int32_t* d_lexical /*nullable*/, int n_lex, int lead, int tail, int64_t L,
                             int32_t* d_out_idx /*[Q,cap]*/, int cap, int32_t* d_out_count /*[Q]*/,
                             void* d_ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* S3_H_ */
