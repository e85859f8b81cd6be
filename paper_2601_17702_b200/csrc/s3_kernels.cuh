// Host-side interface between the C ABI (s3_api.cu) and the kernel files: launchers, size queries and host state, one group
// per .cu file.
#pragma once

#include "s3_common.cuh"

namespace s3 {

struct EncodeTcState {
    void* d_wt = nullptr;        // W_enc^T [d_sae, d_in] bf16 inside the caller's prepared buffer
    float* d_b_eff = nullptr;    // folded bias [d_sae]
    alignas(64) unsigned char map_w[128];   // TMA descriptor of W_enc^T
};

size_t encode_tc_prepared_bytes(int d_in, int d_sae);
s3_status encode_tc_prepare(EncodeTcState* st, const void* d_W, const float* d_b_enc, const float* d_b_dec, int d_in,
                            int d_sae, void* d_prepared, cudaStream_t stream);
int encode_tc_col_tiles(int d_sae);
int encode_tc_row_tiles(int T);
int encode_tc_min_slices(int d_sae);
int encode_tc_max_pairs();         // CTA pairs (work units in flight) of the bf16 encode on this device
size_t encode_tc_workspace_bytes(int T, int n_slices, int k);     // scratch after the status block
size_t encode_tc_workspace_bound(int T, int k);    // holds any automatic schedule of T tokens or fewer
// Encode kernel + candidate merge: writes ids / vals [T,k].
s3_status launch_encode_tc(const EncodeTcState* st, const void* d_x, int64_t ldx, int T, int d_in, int d_sae, int k,
                           int n_slices, int max_ctas, void* d_scratch, uint32_t* d_status, int32_t* d_ids, float* d_vals,
                           cudaStream_t stream);

// Several encoder calls in one persistent launch (each with its own encoder, input, k and outputs); scratch as the sum of
// encode_tc_workspace_bytes over the items.
struct EncodeTcItem {
    const EncodeTcState* st;
    const void* d_x;
    int64_t ldx;
    int T, d_in, d_sae, k, n_slices;      // n_slices: uniform column slices per row tile; 0 = scheduled by the launch
    int32_t* d_ids;
    float* d_vals;
};
// Exact scratch bytes and thread blocks of the launch these items would get (only T, d_in, d_sae, k, n_slices are read).
size_t encode_tc_group_workspace_need(const EncodeTcItem* items, int n_items, int max_ctas);
int encode_tc_group_ctas(const EncodeTcItem* items, int n_items, int max_ctas);
int encode_tc_describe_schedule(const EncodeTcItem* items, int n_items, int n_pairs, int32_t* out, int max_units, int32_t* slots_out);
s3_status launch_encode_tc_group(const EncodeTcItem* items, int n_items, int max_ctas, void* d_scratch, uint32_t* d_status,
                                 cudaStream_t stream);

// Projection of a head and its encode in one launch (the projected tile never leaves the SM): proj maps d_model -> n_heads * 128,
// st is the 128-wide encoder shared by the heads; ids / vals [T, n_heads, k].
size_t encode_proj_tc_workspace_bytes(int T, int n_heads, int k);
s3_status launch_encode_proj_tc(const EncodeTcState* proj, const EncodeTcState* st, const void* d_h, int64_t ldh, int T, int d_model,
                                int n_heads, int d_sae, int k, int max_ctas, void* d_scratch, uint32_t* d_status, int32_t* d_ids,
                                float* d_vals, cudaStream_t stream);

// The same GEMM with a dense epilogue: pre-activations [T, ld_out] as fp32 or bf16.
s3_status launch_preact_tc(const EncodeTcState* st, const void* d_x, int64_t ldx, int T, int d_in, int d_sae, int n_slices,
                           int max_ctas, uint32_t* d_status, void* d_out, int64_t ld_out, bool out_bf16, cudaStream_t stream);

size_t encode_simt_smem_bytes(int k);
int encode_simt_col_tiles(int d_sae);
int encode_simt_row_tiles(int T);
s3_status launch_encode_simt(const float* d_x, int64_t ldx, const float* d_W, const float* d_b_enc,
                             const float* d_b_dec, int T, int d_in, int d_sae, int k, int n_slices,
                             uint64_t* d_part, cudaStream_t stream);

size_t postings_workspace_bytes(int T, int k, int d_sae);   // table bytes of one item (multiple of 256)
s3_status launch_postings(const s3_postings_item* h_items, int n_items, void* d_ws, size_t ws_bytes, cudaStream_t stream);

size_t score_workspace_bytes(int Q, int n_spans);   // after the 256-byte head of the workspace: tickets + shared difference arrays
s3_status launch_score(const s3_csr_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
                       const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                       const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                       float* d_all_scores, void* d_ws, size_t ws_bytes, cudaStream_t stream);

s3_status launch_score_compact(const s3_compact_view* h_layers, int n_layers, int d_sae, const int32_t* d_q_ids,
                               const float* d_q_vals, int Q, int nq, int k, int n_spans, const s3_score_params* p,
                               const float* d_bm25, int64_t ld_bm25, int32_t* d_top_idx, float* d_top_score,
                               float* d_all_scores, void* d_ws, size_t ws_bytes, cudaStream_t stream);
void compact_bound(uint64_t n_postings, int d_sae, uint64_t* max_blocks, uint64_t* max_words);
size_t compact_workspace_bytes(uint64_t n_postings, int d_sae);
s3_status launch_compact_build(const uint64_t* d_row_ptr, const int32_t* d_pos, int d_sae, int64_t stop_freq,
                               uint64_t* d_out_row_ptr, uint32_t* d_blk_ptr, int32_t* d_blk_first, uint64_t* d_blk_desc,
                               uint64_t cap_blocks, uint32_t* d_payload, uint64_t cap_words, uint64_t* d_sizes,
                               uint32_t* d_status, void* d_scratch, cudaStream_t stream);
s3_status launch_decode(const void* d_W_dec, const float* d_b_dec, int d_in, int d_sae, s3_dtype dtype, const int32_t* d_ids,
                        const float* d_vals, int T, int k, float* d_xhat, int64_t ld_xhat, const void* d_x, int64_t ldx,
                        float* d_sqerr, cudaStream_t stream);
s3_status launch_head_aggregate(const int32_t* d_ids, const float* d_vals, int T, int H, int k, int d_sae, int k_out,
                                int32_t* d_out_ids, float* d_out_vals, cudaStream_t stream);
s3_status launch_compact_expand(const s3_compact_view& v, int d_sae, int32_t* d_pos, uint64_t cap_postings, uint32_t* d_status,
                                cudaStream_t stream);
s3_status launch_cast_bf16(const float* d_src, void* d_dst, size_t n, cudaStream_t stream);
s3_status launch_sae_backward(const float* d_W_enc, const float* d_b_enc, const float* d_W_dec, const float* d_b_dec, const float* d_x, int64_t ldx,
                              const int32_t* d_ids, const float* d_vals, int T, int k, int d_in, int d_sae, float* d_gW_enc,
                              float* d_gb_enc, float* d_gW_dec, float* d_gb_dec, float* d_loss, float* d_sqerr, cudaStream_t stream);
s3_status launch_adam(float* d_p, float* d_m, float* d_v, const float* d_g, size_t n, float lr, float beta1, float beta2, float eps,
                      float corr1, float corr2, cudaStream_t stream);
size_t fuse_workspace_bytes(int Q, int64_t L);
s3_status launch_fuse_sets(const int32_t* d_centers, int Q, int n_centers, int span_width, const int32_t* d_lexical, int n_lex,
                           int lead, int tail, int64_t L, int32_t* d_out_idx, int cap, int32_t* d_out_count, void* d_scratch,
                           cudaStream_t stream);
size_t density_workspace_bytes(int Q, int64_t L, int n_layers, int d_sae, int nq, int k);
s3_status launch_density(const s3_csr_view* h_layers, int n_layers, int d_sae, int64_t L, const int32_t* d_q_ids,
                         const float* d_q_vals, int Q, int nq, int k, int conv_kernel, int nms_radius, int n_centers,
                         int64_t stop_freq, int32_t* d_centers, float* d_center_density, float* d_s_out, float* d_d_out,
                         void* d_scratch, cudaStream_t stream);

}  // namespace s3
