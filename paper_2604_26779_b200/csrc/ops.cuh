// Launchers of the library's kernels (internal interface between the translation units).
#pragma once

#include "common.cuh"

namespace spec {

// sampling.cu
// row r at logits + r*row_stride; its (max, sum exp) at stats + 2*r*stats_stride; probs (nullable) [rows][V]
spec_status launch_softmax_rows(int rows, int V, const float* logits, size_t row_stride, float temperature, float* stats,
                                size_t stats_stride, float* probs, cudaStream_t st);
// q rows are q_width wide; with t2d (target id -> row of q, or -1) the draft distribution lives on a subset of the vocabulary
spec_status launch_reject_sample(bool from_logits, int B, int k, int V, const float* p, const float* p_stats,
                                 const float* q, const float* q_stats, int q_width, const int32_t* t2d,
                                 const int32_t* draft, int draft_stride,
                                 float temperature, uint64_t seed, const uint32_t* step_dev, uint32_t step,
                                 int32_t* out_tokens, int32_t* n_emitted, int32_t* status, float* out_logp, cudaStream_t st);
// one token per row from logits and their statistics: uniform Philox(seed; *step_dev, row, slot, stream_tag)
spec_status launch_sample_logits(int rows, int V, const float* logits, size_t row_stride, const float* stats,
                                 size_t stats_stride, float temperature, uint64_t seed, const uint32_t* step_dev,
                                 uint32_t slot, uint32_t stream_tag, int32_t* tokens, int token_stride, int32_t* status,
                                 cudaStream_t st);
spec_status launch_argmax_rows(int rows, int V, const float* logits, size_t row_stride, int32_t* tokens, int token_stride,
                               cudaStream_t st);
spec_status launch_build_t2d(int V, int Vd, const int32_t* d2t, int32_t* t2d, cudaStream_t st);
spec_status launch_map_tokens(int B, const int32_t* src, int src_stride, const int32_t* d2t, int32_t* dst, int dst_stride,
                              cudaStream_t st);
int sampler_max_vocab();

// ops.cu: element-wise and bookkeeping kernels.  dtype = SPEC_DTYPE_* of the activation/weight/KV storage.
struct StepRows {            // per-row metadata of a forward over B sequences x R rows
    int32_t* token;          // [B*R] input token of each row
    int32_t* pos;            // [B*R] absolute position, or -1 for a row that does nothing
};
spec_status launch_verify_rows(int B, int R, const int32_t* seq_len, const int32_t* last_token,
                               const int32_t* draft_tokens, int draft_stride, int vocab, StepRows rows,
                               int32_t* status, cudaStream_t st);
spec_status launch_embed(int M, int d, const void* table, int dtype, const int32_t* token, float* x, cudaStream_t st);
// out[m][col0 .. col0+d) = RMSNorm(in[m]) * w, out row stride ld_out elements
spec_status launch_rmsnorm(int M, int d, const float* in, const float* w, float eps, void* out, int ld_out, int col0,
                           int dtype, cudaStream_t st);
// rotates q and k of qkv [M][(Hq+2Hkv)*dh] in place and writes k, v into the paged cache at the rows' positions
spec_status launch_rope_append(int B, int R, int Hq, int Hkv, int dh, float theta, void* qkv, const int32_t* pos,
                               void* k_pool, void* v_pool, const int32_t* block_table, int max_blocks,
                               int block_tokens, int dtype, cudaStream_t st, const float* rope_table = nullptr);   // rope_table: [dh/2][B*R] (cos, sin) of pos, or NULL
spec_status launch_swiglu(int M, int F, const void* gate_up, void* out, int dtype, cudaStream_t st);
// rows_valid: optional device-side count of the rows that hold data (the others are skipped)
spec_status launch_quantize_rows(int rows, int K, const void* x_bf16, void* codes, float* scales, cudaStream_t st,
                                 const int32_t* rows_valid = nullptr);
// RMSNorm of fp32 rows [M][d] + per-row e4m3 quantisation of the bf16-rounded result (same codes and scales as the two separate kernels).
spec_status launch_rmsnorm_quantize(int M, int d, const float* in, const float* w, float eps, void* codes, float* scales, cudaStream_t st);
spec_status launch_copy_rows_f32_to(int M, int d, const float* x, void* out, int ld_out, int col0, int dtype,
                                    cudaStream_t st);
// dst[b] = src[b*R + idx[b]-1] rows of width d (fp32); idx = rows valid per sequence
spec_status launch_gather_last_rows(int B, int R, int d, const float* src, const int32_t* n_valid, float* dst,
                                    cudaStream_t st);

// KV bookkeeping (single CTA, deterministic order)
spec_status launch_kv_reserve(int B, int k, int block_tokens, int max_blocks, const int32_t* seq_len,
                              int32_t* block_table, int32_t* owned, int32_t* free_stack, int32_t* free_top, int32_t* status,
                              cudaStream_t st);
struct CommitArgs {
    int B, k, block_tokens, max_blocks;
    const int32_t* force_n;       // nullable
    const int32_t* force_token;   // nullable
    const int32_t* verify_tokens; // [B][k+1] input tokens of the last verify (read by a forced commit)
    int32_t* n_emitted;           // [B] in: sampler's n+1 (ignored when forced); out: committed n+1
    int32_t* out_tokens;          // [B][k+1]
    int32_t* seq_len; int32_t* last_token; int32_t* block_table; int32_t* owned; int32_t* free_stack; int32_t* free_top;
    int32_t* pending_base;        // [B] first position committed by this step
    int32_t* history; int max_hist;            // nullable: token at every cached position, appended here
    uint32_t* step; long long* counters;   // counters: steps, emitted, accepted
    int32_t* status;
};
spec_status launch_kv_commit(const CommitArgs& a, cudaStream_t st);
spec_status launch_kv_replace(int n, const int32_t* slots, const int32_t* new_len, const int32_t* new_last, int bt,
                              int max_blocks, int32_t* seq_len, int32_t* last_token, int32_t* table, int32_t* owned,
                              int32_t* free_stack, int32_t* free_top, int32_t* n_emitted,
                              int32_t* pending_base, int32_t* status, cudaStream_t st);

spec_status launch_seq_compact(int n_keep, int B_old, const int32_t* keep, int max_blocks, int out_stride, int hist_len, int32_t* seq_len,
                               int32_t* last_token, int32_t* owned, int32_t* pending_base, int32_t* n_emitted, int32_t* table,
                               int32_t* out_tokens, float* out_logp, int32_t* history, cudaStream_t st);
spec_status launch_permute_rows(int n_keep, int R, size_t row_bytes, const int32_t* keep, const void* src, void* dst, cudaStream_t st);

// model-free drafting: continue the most recent earlier occurrence of the trailing n-gram of (history[0..len), last token)
spec_status launch_ngram_draft(int B, int k, int n_max, const int32_t* history, int max_hist, const int32_t* seq_len,
                               const int32_t* last_token, int32_t* draft_tokens, int draft_stride, cudaStream_t st);

// gemm_simt.cu / gemm_tc.cu: C[M][N] (+)= A[M][K] W[N][K]^T, fp32 accumulation
spec_status launch_gemm_simt(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int dtype_in,
                             int out_dtype, int accumulate, cudaStream_t st);
spec_status launch_gemm(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int dtype_in,
                        int out_dtype, int accumulate, cudaStream_t st);

// swiglu != 0: W holds [2F] rows per group in 256-row gate/up groups and C is the activation [rows][N/2] (bf16)
// 8-bit (e4m3) operands with per-row scales: plain (optionally with the LM head's row statistics), SwiGLU and QKV epilogues
spec_status launch_gemm8_tc(int M, int N, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale, void* C, int ldc,
                            int out_dtype, int accumulate, float temperature, float* part, size_t part_bytes, float* stats,
                            size_t stats_stride, int32_t* status, cudaStream_t st);
spec_status launch_gemm8_swiglu_tc(int M, int F, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale, void* act,
                                   int32_t* status, cudaStream_t st);
// very few rows (M <= 16): the weights are the MMA's M operand, one CTA per 32 weight rows (gemm_skinny.cu)
bool gemm_skinny_supported(int M, int N, int K, const void* A, int lda, const void* W, int dtype_in);
spec_status launch_gemm_skinny(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int out_dtype,
                               int accumulate, cudaStream_t st);
// 17..64 rows: the tensor-core kernel with the operands swapped (weights as the M operand, one narrow tile of activation rows)
bool gemm_tc_thin_supported(int M, int N, int K, const void* A, int lda, const void* W, const void* C, int ldc, int dtype_in, int out_dtype);
spec_status launch_gemm_lm_head_stats(int M, int N, int K, const void* A, int lda, const void* W, float* logits, int ldc, int dtype_in,
                                      float temperature, float* part, size_t part_bytes, float* stats, size_t stats_stride,
                                      int32_t* status, cudaStream_t st);
spec_status launch_gemm_grouped(int rows_total, int max_rows_per_group, int E, int N, int K, const void* A, const void* W,
                                void* C, int out_dtype, int swiglu, const int32_t* counts, const int32_t* offsets,
                                int32_t* status, cudaStream_t st);
spec_status launch_gemm_tc(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int out_dtype,
                           int accumulate, int32_t* status, cudaStream_t st);
bool gemm_tc_supported(int M, int N, int K, const void* A, int lda, const void* W, const void* C, int ldc, int dtype_in,
                       int out_dtype);
spec_status launch_gemm_swiglu_tc(int M, int F, int K, const void* A, int lda, const void* W, void* act, int32_t* status,
                                  cudaStream_t st);
struct QkvEpilogue {
    int Hq, Hkv, dh, R, max_blocks, block_tokens;
    const int32_t* pos; const int32_t* block_table;
    const float* rope;            // [dh/2][M][2] (cos, sin) of each row's position
    void* k_pool; void* v_pool;
    int kv_fp8 = 0;               // write e4m3 codes of k / k_scale and v / v_scale instead of bf16
    float k_scale = 1.f, v_scale = 1.f;
};
spec_status launch_gemm_qkv_tc(int M, int K, const void* A, int lda, const void* W, void* qkv, const QkvEpilogue& e,
                               int32_t* status, cudaStream_t st);
spec_status launch_gemm8_qkv_tc(int M, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale, void* qkv,
                                const QkvEpilogue& e, int32_t* status, cudaStream_t st);
spec_status launch_gemm8_grouped(int rows_total, int max_rows_per_group, int E, int N, int K, const void* a8, const float* a_scale,
                                 const void* w8, const float* w_scale, void* C, int out_dtype, int swiglu, const int32_t* counts,
                                 const int32_t* offsets, int32_t* status, cudaStream_t st);
// (cos, sin) table of the rows' positions for the fused QKV epilogue
spec_status launch_rope_table(int M, int dh, float theta, const int32_t* pos, float* table, cudaStream_t st);

// moe.cu: router top-k, permutation into expert order, weighted combination
spec_status launch_moe_route(int M, int E, int top_k, const float* logits, int32_t* ids, float* wts, cudaStream_t st);
spec_status launch_moe_rank(int n_entries, int E, const int32_t* ids, int32_t* rank, int32_t* counts, cudaStream_t st);
// h rows of d 16-bit elements (8-bit code rows: pass d / 2 and the rows' scales, which are then permuted along)
spec_status launch_moe_permute(int M, int E, int top_k, int d, const int32_t* ids, int32_t* rank, int32_t* counts,
                               int32_t* offsets, int32_t* inv, const void* h, void* a_perm, cudaStream_t st,
                               const float* row_scale = nullptr, float* perm_scale = nullptr);
spec_status launch_moe_combine(int M, int top_k, int d, const float* wts, const int32_t* inv, const float* out_perm,
                               float* x, cudaStream_t st);

// attention.cu
struct AttnArgs {
    int B, R, Hq, Hkv, dh, block_tokens, max_blocks;
    const void* q; int q_row_stride;   // q row (b, r) at q + (b*R + r) * q_row_stride elements, heads contiguous
    const void* k_pool; const void* v_pool;
    const int32_t* block_table;
    const int32_t* pos;                // [B*R] position of each query row (-1: skip, output zeros)
    void* out; int out_row_stride;
    int dtype;
    void* scratch; size_t scratch_bytes;
    int max_kv_len;
    int launch_index;                  // 0 plans the work units; later launches of the same step reuse the plan
    int32_t* status = nullptr;         // device status word for kernels with bounded waits (may be null)
    int kv_fp8 = 0;                    // the pools hold e4m3 codes of x / scale (one byte per element)
    float k_scale = 1.f, v_scale = 1.f;
};
spec_status launch_attention(const AttnArgs& a, cudaStream_t st);
size_t attention_scratch_bytes(int B, int R, int Hq, int Hkv, int dh, int max_kv_len);
bool attention_mma_supported(const AttnArgs& a);
size_t attention_mma_scratch_bytes(int B, int R, int Hq, int Hkv, int dh, int max_kv_len);
spec_status launch_attention_mma(const AttnArgs& a, cudaStream_t st);

}  // namespace spec
