/*
 * spec.h - C ABI of the speculative-decoding step library (CUDA, sm_100a).
 *
 * One speculation step of autoregressive rollout generation: a draft head proposes k tokens, the target
 * model verifies the k+1 positions in one forward against a paged KV cache, a lossless rejection sampler
 * keeps the target's output distribution, and the KV cache keeps the accepted slots (paper: Introduction,
 * third paragraph; Section 2.1 "rollouts follow the verifier policy by construction"; Section 2.2 "only the
 * autoregressive decode phase", "tokens produced per speculation step"; Section 2.3 the two drafting paths).
 *
 * Conventions for every function:
 *   - plain C types only; pointers named *_host are host pointers, every other pointer is a DEVICE pointer;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream);
 *   - the library never allocates or frees device memory: every buffer is caller-owned and must outlive
 *     the calls (and the context) that use it;
 *   - step functions only enqueue work on `stream`; they do not synchronise (spec_get_status does);
 *   - a host-detectable problem returns a negative spec_status and launches nothing; a problem found on
 *     the device is recorded in a status word (first error wins) and never traps;
 *   - a context is not thread-safe: serialise the calls on one context.  Different contexts may be driven from different
 *     host threads and on different devices of one process (one-time kernel set-up is kept per device); the stateless
 *     operators are reentrant.
 *
 * Layouts: a weight matrix is [out][in] row-major; token ids, lengths and tables are int32; logits and
 * probabilities are fp32; activations, weights and KV are bf16 (SPEC_DTYPE_BF16) or fp32 (SPEC_DTYPE_F32).
 */
#ifndef SPEC_H_
#define SPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPEC_ABI_VERSION 6u

typedef struct spec_ctx spec_ctx; /* opaque */

typedef enum {
    SPEC_OK = 0,
    /* detected on the host, returned immediately, nothing launched */
    SPEC_ERR_INVALID_ARG = -1,
    SPEC_ERR_SHAPE = -2,
    SPEC_ERR_UNSUPPORTED = -3,
    SPEC_ERR_STATE = -4,
    SPEC_ERR_CUDA = -5,
    /* detected on the device, reported through the status word / spec_get_status */
    SPEC_ERR_KV_EXHAUSTED = -16,
    SPEC_ERR_TOKEN_RANGE = -17,
    SPEC_ERR_BAD_PROB = -18,
    SPEC_ERR_TIMEOUT = -19,
    SPEC_ERR_EP_CAPACITY = -20
} spec_status;

enum { SPEC_DTYPE_BF16 = 0, SPEC_DTYPE_F32 = 1 };
enum { SPEC_KV_MODEL = 0, SPEC_KV_E4M3 = 1 };
enum { SPEC_W_MODEL = 0, SPEC_W_E4M3 = 1 };
enum { SPEC_DRAFT_NONE = 0, SPEC_DRAFT_EAGLE3 = 1, SPEC_DRAFT_MTP = 2, SPEC_DRAFT_NGRAM = 3 };

/* Model and run description.  n_experts = 0 selects the dense SwiGLU MLP. */
typedef struct {
    uint32_t struct_size, abi_version;
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t n_experts, experts_top_k, d_expert_ffn;
    float rms_eps, rope_theta;
    int32_t dtype;              /* SPEC_DTYPE_*: storage type of weights, KV and activations            */
    int32_t draft_kind;         /* SPEC_DRAFT_*; NONE = the caller supplies draft tokens and draft logits */
    int32_t draft_d_ffn;        /* FFN width of the draft head's layer                                   */
    int32_t n_taps, tap_layers[3]; /* residual-stream taps handed to the draft head: tap t = after t layers */
    int32_t k_max;              /* largest draft length used with this context (<= 7)                    */
    int32_t max_batch;
    int32_t kv_block_tokens;    /* tokens per KV block (16)                                              */
    int32_t kv_num_blocks;      /* physical blocks per layer pool                                        */
    int32_t max_blocks_per_seq;
    int32_t kv_layer_pools;     /* physical per-layer pools G <= n_layers; layer l uses pool l mod G.    */
                                /* G < n_layers aliases layers onto shared pools: a timing-only mode for  */
                                /* caches larger than the device; results are then not meaningful        */
    float temperature;          /* > 0; scales the logits of both models before the softmax              */
    uint64_t seed;              /* Philox key of every uniform the step draws                            */
    int32_t ngram_n;            /* SPEC_DRAFT_NGRAM: longest trailing n-gram looked up in the sequence's own   */
                                /* tokens (1..8); the model-free drafting the paper uses as a baseline (Table 2) */
    int32_t draft_greedy;       /* 1: the draft head proposes d_i = argmax of its logits (ties: lowest id)      */
                                /* and q_i is taken as one-hot(d_i): accept iff u < p_i(d_i), residual = p_i    */
                                /* without d_i's mass (the deterministic-draft special case of the rule)        */
    int32_t draft_vocab;        /* EAGLE3 only: 0 = the head's LM head covers the whole vocabulary; else its    */
                                /* number of rows (a multiple of 8, <= vocab): row r scores target token        */
                                /* D_D2T[r] (strictly increasing ids), q is zero outside that set                */
    int32_t kv_dtype;           /* SPEC_KV_MODEL: the cache holds `dtype`; SPEC_KV_E4M3: one byte per element, the e4m3    */
                                /* code (round to nearest even, saturating at 448) of x / scale, read back as code * scale */
                                /* (the precision of the paper's deployment simulator, Section 5.1).  bf16 models with     */
                                /* head_dim 128 and at most 16 query rows per KV head; a reduced-precision mode            */
    float kv_scale_k, kv_scale_v; /* > 0 with SPEC_KV_E4M3: one scale for all keys (after the rotary embedding), one for values */
    int32_t weight_dtype;       /* SPEC_W_MODEL: the projections run in `dtype`; SPEC_W_E4M3: the target's QKV, O, gate/up, down  */
                                /* and LM-head weights are stored as e4m3 codes with one fp32 scale per output row (the     */
                                /* *_SCALE tensors; code = round_e4m3(w / scale), scale = amax(row) / 448), activations are */
                                /* quantised the same way per row on the fly, and the products run on the 8-bit tensor-core */
                                /* path with fp32 accumulation (the precision of the paper's simulator, Section 5.1).       */
                                /* bf16 models (in a mixture-of-experts layer the router stays 16-bit, the experts' gate/up */
                                /* and down weights are 8-bit); the draft heads' own weights stay 16-bit (the MTP head scores with    */
                                /* the target's 8-bit LM head); a reduced-precision mode                                    */
} spec_config;

/* Byte sizes of the caller-owned device arenas for a configuration. */
typedef struct {
    size_t weights_bytes, draft_weights_bytes, kv_bytes, draft_kv_bytes, workspace_bytes, state_bytes;
} spec_sizes;

/* The arenas themselves (device pointers, each 256-byte aligned, at least the queried size). */
typedef struct {
    void *weights, *draft_weights, *kv, *draft_kv, *workspace, *state;
} spec_buffers;

/* Tensors addressable through spec_tensor. */
enum {
    /* target weights (arena `weights`); per-layer ones take the layer index */
    SPEC_T_EMBED = 0, SPEC_T_LM_HEAD, SPEC_T_FINAL_NORM,
    SPEC_T_ATTN_NORM, SPEC_T_WQKV, SPEC_T_WO, SPEC_T_MLP_NORM,
    SPEC_T_WGATEUP,             /* [2*d_ffn][d] in 256-row groups: gate rows 128g..128g+127, then up   */
                                /* rows 128g..128g+127 (d_ffn % 128 == 0)                              */
    SPEC_T_WDOWN,
    SPEC_T_ROUTER,              /* [n_experts][d]                                                      */
    SPEC_T_EXPERTS_GATEUP,      /* [n_experts][2*d_expert_ffn][d], each expert grouped like WGATEUP    */
    SPEC_T_EXPERTS_DOWN,        /* [n_experts][d][d_expert_ffn]                                        */
    /* SPEC_W_E4M3: fp32 [rows of the weight] scales; the weight tensors themselves then hold one byte per element */
    SPEC_T_LM_HEAD_SCALE = 16, SPEC_T_WQKV_SCALE, SPEC_T_WO_SCALE, SPEC_T_WGATEUP_SCALE, SPEC_T_WDOWN_SCALE,
    SPEC_T_EXPERTS_GATEUP_SCALE, /* [n_experts][2*d_expert_ffn] (the router stays 16-bit)                  */
    SPEC_T_EXPERTS_DOWN_SCALE,  /* [n_experts][d]                                                       */
    /* draft head weights (arena `draft_weights`) */
    SPEC_T_D_WFC = 32,          /* EAGLE3: [d][n_taps*d]                                               */
    SPEC_T_D_WPROJ,             /* MTP: [d][2d] acting on concat(norm_g(g), norm_e(e))                 */
    SPEC_T_D_NORM_E, SPEC_T_D_NORM_G, SPEC_T_D_NORM_F, SPEC_T_D_ATTN_NORM,
    SPEC_T_D_WQKV,              /* EAGLE3: [(Hq+2Hkv)dh][2d] acting on concat(norm_e(e), norm_g(g))    */
    SPEC_T_D_WO, SPEC_T_D_MLP_NORM, SPEC_T_D_WGATEUP, SPEC_T_D_WDOWN,
    SPEC_T_D_LM_HEAD,           /* EAGLE3: [draft_vocab or vocab][d]                                   */
    SPEC_T_D_D2T,               /* EAGLE3 with draft_vocab: [draft_vocab] int32 target id of each row  */
    /* caches: [block][n_kv_heads][kv_block_tokens][head_dim]; layer = pool index for the target */
    SPEC_T_KV_K = 64, SPEC_T_KV_V, SPEC_T_DRAFT_KV_K, SPEC_T_DRAFT_KV_V,
    /* state (int32) */
    SPEC_T_SEQ_LEN = 96,        /* [max_batch] valid KV entries per sequence                           */
    SPEC_T_LAST_TOKEN,          /* [max_batch] last committed token, not yet fed to the target         */
    SPEC_T_BLOCK_TABLE,         /* [max_batch][max_blocks_per_seq], -1 = none                          */
    SPEC_T_FREE_STACK,          /* [kv_num_blocks]                                                     */
    SPEC_T_FREE_TOP,            /* [1] number of free blocks                                           */
    SPEC_T_DRAFT_TOKENS,        /* [max_batch][k_max]                                                  */
    SPEC_T_OUT_TOKENS,          /* [max_batch][k_max+1], -1 padded                                     */
    SPEC_T_N_EMITTED,           /* [max_batch]                                                         */
    SPEC_T_STATUS,              /* [4] device status word: code, detail, 0, 0                          */
    SPEC_T_STEP,                /* [1] step counter = Philox counter word 0                            */
    SPEC_T_TOKEN_HISTORY,       /* [max_batch][max_blocks_per_seq*kv_block_tokens] token at every cached    */
                                /* position (SPEC_DRAFT_NGRAM only); commits append to it, the caller fills  */
                                /* it for positions that were cached before spec_seq_init                  */
    SPEC_T_OUT_LOGP,            /* [max_batch][k+1] fp32 log p_target(token) of the emitted tokens     */
                                /* (the verifier's log-probabilities an RL loss needs, Section 2.3)    */
    /* step results in the workspace */
    SPEC_T_LOGITS = 128,        /* [B][k+1][vocab] fp32 target logits of the last verify               */
    SPEC_T_DRAFT_LOGITS,        /* [B][k][draft_vocab or vocab] fp32 draft logits of the last draft    */
    SPEC_T_ROW_STATS,           /* [B*(k+1)][2] fp32 (max, sum exp) of the target rows                 */
    SPEC_T_DRAFT_ROW_STATS,     /* [B*k][2]                                                            */
    SPEC_T_TAPS,                /* [B][k+1][n_taps*d] tapped hidden states of the last verify          */
    SPEC_T_HIDDEN,              /* [B*(k+1)][d] fp32 residual stream after the last layer              */
    SPEC_T_MOE_LOGITS,          /* [B*(k+1)][n_experts] fp32 router logits of the last MoE layer run   */
    SPEC_T_MOE_IDS,             /* [B*(k+1)][experts_top_k] int32 selected experts, best first         */
    SPEC_T_MOE_WTS,             /* [B*(k+1)][experts_top_k] fp32 renormalised mixture weights          */
    /* SPEC_W_E4M3 only: the quantised rows a projection consumed in the last pass.  `layer` names the     */
    /* slot: 0 QKV, 1 O, 2 gate/up, 3 down (of the last layer that ran), 4 LM head (the last LM-head     */
    /* product: the target's, or an MTP head's last pass).  Row r of a slot has                            */
    /* K codes at byte r*K (K = that projection's input width) and its scale at ACT_SCALES[r].             */
    /* In a mixture-of-experts layer slots 2 and 3 hold the rows in expert order (top_k entries per row). */
    SPEC_T_ACT_CODES,           /* uint8 e4m3 codes, rows back to back                                 */
    SPEC_T_ACT_SCALES,          /* fp32 [rows]                                                         */
    SPEC_T_MOE_INV              /* [B*(k+1)][experts_top_k] int32: where (row, slot) sits in expert order */
};

/* Counters returned by spec_get_status (host struct). */
typedef struct {
    int32_t device_status;      /* SPEC_OK or the first device-detected error                          */
    int32_t device_detail;      /* sequence index or row the error refers to                           */
    int64_t steps;              /* commits since spec_seq_init                                         */
    int64_t emitted_tokens;     /* sum over sequences and steps of n+1                                 */
    int64_t accepted_drafts;    /* sum of n                                                            */
} spec_step_report;

/* ---- context -------------------------------------------------------------------------------------------- */

/* Arena sizes for `cfg`.  Errors: INVALID_ARG (NULL, wrong struct_size/abi_version), SHAPE, UNSUPPORTED. */
spec_status spec_query_sizes(const spec_config* cfg, spec_sizes* out);

/* Builds a context over caller-owned arenas (nothing is copied or allocated on the device; the context
 * itself is a small host object freed by spec_destroy).  The state arena must be zero-filled by the caller
 * or initialised with spec_seq_init before the first step. */
spec_status spec_create(const spec_config* cfg, const spec_buffers* buffers, spec_ctx** out);
spec_status spec_destroy(spec_ctx* ctx);

/* Address and byte size of a tensor inside the arenas, so the caller can write weights (also between
 * steps: overwriting them in place is how refreshed policy weights reach the step, Section 2.3) or cache
 * contents, and read results. */
spec_status spec_tensor(spec_ctx* ctx, int tensor_id, int layer, void** dev_ptr, size_t* bytes);

/* Starts B sequences: sequence b has seq_len_host[b] valid KV entries (the caller has filled or will fill
 * them) and last token last_token_host[b].  free_stack_host[kv_num_blocks] is the initial order of the free
 * stack (top = last element); blocks for the valid entries are popped in sequence order.  Resets the step
 * counter.  Errors: INVALID_ARG, SHAPE (B > max_batch, a length that does not fit), KV exhaustion (SHAPE). */
spec_status spec_seq_init(spec_ctx* ctx, int B, const int32_t* seq_len_host, const int32_t* last_token_host,
                          const int32_t* free_stack_host, void* stream);

/* Replaces finished sequences between steps: rollout responses end at very different lengths (the long tail
 * of Section 5.1) and a slot whose sequence is done takes the next prompt while the others keep decoding.
 * For i = 0..n-1, in list order: every block of slot slots_host[i] returns to the free stack (logical
 * order), blocks for seq_len_host[i] cached positions are popped (the caller fills them, or passes 0 and
 * prefills through forced verify steps), its last token becomes last_token_host[i] and the draft head has
 * no pending positions for it.  seq_len_host[i] < 0 retires the slot instead (no prompt left): it keeps
 * no block, its rows of later steps are inert (no cache access, nothing emitted: N_EMITTED 0, SEQ_LEN -1)
 * until it is replaced again.  The step counter and the other slots are untouched, so their random
 * streams continue.  Host arrays, n <= current batch; synchronises `stream`.
 * Errors: STATE (between verify and commit), INVALID_ARG (slot out of range or twice, bad token), SHAPE;
 * a free stack too small for the list leaves the state unchanged and sets the device status
 * SPEC_ERR_KV_EXHAUSTED. */
spec_status spec_seq_replace(spec_ctx* ctx, int n, const int32_t* slots_host, const int32_t* seq_len_host,
                             const int32_t* last_token_host, void* stream);

/* ---- one speculation step (Introduction, third paragraph) ------------------------------------------------- */

/* Renumbers the running sequences so that the batch shrinks: new slot j takes over everything of old slot
 * keep_slots_host[j] (strictly ascending old slots), every slot that is not listed is retired first (its blocks
 * go back to the free stack in slot order, logical block order, as spec_seq_replace does) and the context
 * continues with n_keep sequences - every later pass (projections, attention plan, sampler) then works on
 * n_keep * (k+1) rows instead of carrying the retired slots' inert rows: what the long tail of a rollout needs
 * (paper: Section 5.2, thin batches).  Between steps only.  The uniforms are drawn per slot, so a moved sequence
 * continues on its new slot's stream.  The logits and hidden-state tensors of the last step are not renumbered
 * (read them before); token, log-probability and block tables are.  The batch cannot grow again without
 * spec_seq_init.  Synchronises `stream`.  Errors: INVALID_ARG (order, range), SHAPE, STATE (a verified step is
 * waiting for its commit). */
spec_status spec_seq_compact(spec_ctx* ctx, int n_keep, const int32_t* keep_slots_host, void* stream);

/* S1 draft propose.  Runs the draft head: pass 0 consumes the (tapped hidden state, next token) pairs of the
 * positions committed by the previous step, passes 1..k-1 feed the head its own output; fills draft tokens
 * d_1..d_k (d_i drawn from q_i with the stream-1 uniforms), draft logits and their row statistics.
 * With draft_greedy = 1 the head's tokens are the arg-maxima of its logits and no draft uniform is consumed.
 * With SPEC_DRAFT_NGRAM no model runs: d_1..d_k continue the most recent earlier occurrence of the sequence's trailing
 * n-gram (n = ngram_n down to 1; without any match the last token is repeated), and q is one-hot.
 * Errors: STATE (no committed step to draft from, draft_kind NONE), SHAPE (k outside 1..k_max). */
spec_status spec_draft(spec_ctx* ctx, int k, void* stream);

/* S2 target verify.  One forward over the k+1 tokens [last token, d_1..d_k] of every sequence at positions
 * seq_len .. seq_len+k, causal among them, against the paged cache; appends their keys/values; writes the
 * logits of all k+1 positions, their row statistics and the tapped hidden states.  k = 0 is plain decode.
 * draft_tokens [B][k] overrides the context's draft tokens when not NULL (teacher forcing, external drafts). */
spec_status spec_verify(spec_ctx* ctx, int k, const int32_t* draft_tokens, void* stream);

/* S3+S4 fused vocabulary softmax and rejection sampling on the context's logits: accept_i = u_i <
 * min(1, p_i(d_i)/q_i(d_i)); n = accepted prefix length; token n+1 from norm(max(0, p_{n+1}-q_{n+1})) or,
 * when n = k, the bonus token from p_{k+1}; uniforms Philox(seed; step, sequence, slot 0..k, stream 0).
 * draft_logits [B][k][vocab] (always over the whole vocabulary) overrides the context's draft logits when not NULL.  With draft_kind NONE and
 * draft_logits NULL the drafts are taken as deterministic (n-gram lookup, greedy drafting): q = one-hot(d), i.e.
 * accept iff u < p(d), residual = p without the draft token's mass. */
spec_status spec_reject_sample(spec_ctx* ctx, int k, const float* draft_logits, void* stream);

/* S5 KV commit / rollback: seq_len += n+1, blocks past the new length return to the free stack, the last
 * token becomes the emitted token, the step counter advances.  force_n / force_token ([B] each, both or
 * neither) replace the sampler's n and token: teacher-forced prefill through the verify path; a negative
 * force_n[b] leaves sequence b to the sampler (a new prompt prefills while the other slots decode). */
spec_status spec_kv_commit(spec_ctx* ctx, const int32_t* force_n, const int32_t* force_token, void* stream);

/* Synchronises `stream`, reads the device status word and counters. */
spec_status spec_get_status(spec_ctx* ctx, spec_step_report* host_out, void* stream);
const char* spec_last_error(const spec_ctx* ctx);

/* ---- stateless entry points (same kernels, no context) ------------------------------------------------------ */

/* Row statistics and, optionally, probabilities of `rows` logit rows of width V:
 * m = max_v l_v, Z = sum_v exp((l_v - m)/T), p_v = exp((l_v - m)/T)/Z.  stats [rows][2] = (m, Z) and probs
 * [rows][V] may each be NULL. */
spec_status spec_softmax_rows(int rows, int V, const float* logits, float temperature, float* stats,
                              float* probs, void* stream);

/* Draws one token per row from fp32 probabilities (not necessarily normalised) by inverse CDF with the
 * uniform Philox(seed; step, row, slot, stream_tag); tokens [rows]. */
spec_status spec_sample_rows(int rows, int V, const float* probs, uint64_t seed, uint32_t step, uint32_t slot,
                             uint32_t stream_tag, int32_t* tokens, int32_t* status, void* stream);

/* Rejection sampling on given probabilities: p [B][k+1][V], q [B][k][V], draft [B][k] ->
 * out_tokens [B][k+1] (-1 padded), n_emitted [B] in 1..k+1.  status [4] int32 device status word (may be NULL).
 * q == NULL means deterministic drafts: q = one-hot(draft). */
spec_status spec_reject_sample_probs(int B, int k, int V, const float* p, const float* q, const int32_t* draft,
                                     uint64_t seed, uint32_t step, int32_t* out_tokens, int32_t* n_emitted,
                                     int32_t* status, void* stream);

/* The same from logits and their row statistics (p_stats [B*(k+1)][2], q_stats [B*k][2]), probabilities
 * formed on the fly and never written. */
spec_status spec_reject_sample_logits(int B, int k, int V, const float* p_logits, const float* p_stats,
                                      const float* q_logits, const float* q_stats, const int32_t* draft,
                                      float temperature, uint64_t seed, uint32_t step, int32_t* out_tokens,
                                      int32_t* n_emitted, int32_t* status, void* stream);

/* Philox uniforms u [n_seq][n_slots] of (seed, step, stream_tag), as the sampler draws them. */
spec_status spec_uniforms(uint64_t seed, uint32_t step, uint32_t stream_tag, int n_seq, int n_slots, float* u,
                          void* stream);

/* Per-row e4m3 quantisation of a bf16 matrix x [rows][K] (K % 16 == 0): scales [rows] = amax(row) / 448 (1 for a zero
 * row), codes [rows][K] = round_e4m3(x / scale), round to nearest even, saturating.  What SPEC_W_E4M3 contexts expect in
 * their weight tensors, and what they do to activations (the 8-bit precision the paper's large-scale projection assumes,
 * Section 5.1; the paper gives no scaling rule, this one is ours).  All pointers are device memory owned by the caller,
 * x and codes 16-byte aligned; rows == 0 is a no-op; a null pointer or K <= 0 returns SPEC_ERR_INVALID_ARG and
 * K % 8 != 0 SPEC_ERR_SHAPE, both before anything is launched. */
spec_status spec_quantize_rows(int rows, int K, const void* x_bf16, void* codes, float* scales, void* stream);

/* C[M][N] = A[M][K] * W[N][K]^T (+ C when accumulate != 0).  dtype_in selects bf16 (tensor-core path, fp32
 * accumulation) or fp32 inputs; out_dtype the type of C.  All leading dimensions are the natural ones.
 * bf16 requires K % 64 == 0 and N % 8 == 0. */
spec_status spec_gemm(int M, int N, int K, const void* A, const void* W, void* C, int dtype_in, int out_dtype,
                      int accumulate, void* stream);

/* The same product with 8-bit operands: a8 [M][K] and w8 [N][K] e4m3 codes (as spec_quantize_rows writes them), a_scale
 * [M] and w_scale [N] their row scales; C[m][n] (+)= a_scale[m] * w_scale[n] * sum_k a8[m][k] * w8[n][k], accumulated in
 * fp32 on the 8-bit tensor-core path.  K % 16 == 0, N % 8 == 0; pointers 16-byte aligned; C is fp32 or bf16 (out_dtype),
 * caller-owned device memory like the operands.  M == 0 or N == 0 is a no-op; a null pointer returns
 * SPEC_ERR_INVALID_ARG, a shape or alignment the kernel does not take SPEC_ERR_SHAPE, nothing launched in either case. */
spec_status spec_gemm_e4m3(int M, int N, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale,
                           void* C, int out_dtype, int accumulate, void* stream);

/* Paged attention of R = rows_per_seq query rows per sequence (query row i at position seq_len[b] + i sees
 * cache positions <= seq_len[b] + i), grouped-query heads.  q [B][R][Hq][dh], out the same shape and type;
 * k_pool / v_pool [blocks][Hkv][block_tokens][dh]; block_table [B][max_blocks]; scratch: see
 * spec_attention_scratch_bytes. */
spec_status spec_attention(int B, int R, int Hq, int Hkv, int dh, int block_tokens, int max_blocks,
                           const void* q, const void* k_pool, const void* v_pool, const int32_t* block_table,
                           const int32_t* seq_len, void* out, int dtype, void* scratch, size_t scratch_bytes,
                           void* stream);
size_t spec_attention_scratch_bytes(int B, int R, int Hq, int Hkv, int dh, int max_kv_len);

/* spec_attention for callers that cannot allocate device memory.  (The paper has no counterpart: this is a
 * convenience of the library.)  Some callers of this code run where cudaMalloc is off limits: inside a host
 * program that has handed all device memory to another allocator and forbids further driver allocations, in a
 * plug-in that may only enqueue work on a stream it is given, or in a latency-critical loop where an allocation
 * would serialise the device.  They cannot provide the scratch buffer spec_attention asks for, so this variant
 * keeps the scratch in a 32 MiB array built into the library image (every GPU that loads the library holds those
 * 32 MiB until the process exits).  Arguments, layouts and results are those of spec_attention; inputs and outputs
 * are still the caller's.
 *   - Sizes: returns SPEC_ERR_SHAPE, launching nothing, when spec_attention_scratch_bytes(B, R, Hq, Hkv, dh,
 *     max_blocks * block_tokens) exceeds 32 MiB (33554432 bytes); for the 8B head shape with k = 3 that allows,
 *     for example, 64 sequences of up to 16384 cached positions per call (24.4 MiB).
 *   - The first call on each device looks up the array's device address (with that device current); make that
 *     first call outside any stream capture.  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - All calls share the one array, which keeps whatever the last call left; every call rewrites what it reads
 *     (row positions, work counters, partial results), so results do not depend on earlier calls.  Two calls that
 *     overlap on the GPU (different streams, or different host threads) race on the array: serialise them.
 * Errors: INVALID_ARG, SHAPE (see above), CUDA. */
spec_status spec_attention_noalloc(int B, int R, int Hq, int Hkv, int dh, int block_tokens, int max_blocks,
                                   const void* q, const void* k_pool, const void* v_pool, const int32_t* block_table,
                                   const int32_t* seq_len, void* out, int dtype, void* stream);

/* ---- expert-parallel mixture-of-experts MLP (bf16) -----------------------------------------------------------
 *
 * The paper's largest configuration (Qwen3-235B-A22B, Section 5.1) does not fit one GPU: its experts are spread over
 * the GPUs of an NVLink domain while every GPU keeps its own sequences.  These three calls are one MoE MLP block
 * (router top-k, SwiGLU experts, weighted sum into the residual; the same arithmetic as the single-GPU block) for that
 * arrangement.  Rank r of ep_size owns the experts [r * n_experts / ep_size, (r + 1) * n_experts / ep_size) and holds
 * only their weights.  Data crosses between ranks by LOADS FROM PEER MEMORY inside the gather and combine kernels
 * (each rank pulls what it needs; nothing is pushed, no kernel waits on another rank):
 *
 *   spec_ep_route    (on every rank)  router logits, top-k, and the per-expert lists of this rank's entries; copies
 *                                     the rank's input rows into its window.  Reads and writes the own window only.
 *   -- barrier: every rank's route has completed --
 *   spec_ep_experts  (on every rank)  pulls the rows routed to the local experts out of all ranks' windows into local
 *                                     memory (expert ascending, source rank ascending, the source's entry order), runs
 *                                     the two grouped tensor-core GEMMs, leaves the expert outputs in the own window.
 *   -- barrier: every rank's experts pass has completed --
 *   spec_ep_combine  (on every rank)  for each own token pulls its top_k expert outputs from the owners' windows and
 *                                     adds them to the residual in slot order (x += sum_j w_j * y_j, fused multiply-adds).
 *   -- barrier before the next spec_ep_route reuses the windows --
 *
 * The barriers are the caller's (stream-ordered: a collective on the same stream, or a host barrier after a stream
 * synchronise); on one GPU with several windows, stream order alone is the barrier.  A WINDOW is a caller-owned device
 * buffer of spec_ep_sizes.window_bytes, 256-byte aligned, that the other ranks can address: peer_windows_host [ep_size]
 * holds, in rank order, the device addresses under which THIS process sees every rank's window (its own included), e.g.
 * from spec_ipc_open or from peer access between devices of one process.  scratch is private to the rank.
 * Results do not depend on ep_size: a token's output is bit-identical to what the single-rank call computes for it.
 *
 * status [4] int32 (device, may be NULL): SPEC_ERR_EP_CAPACITY when more rows were routed to this rank than
 * cap_rows (the surplus rows are dropped: their outputs are missing from the sums), SPEC_ERR_TIMEOUT from the GEMMs.
 * Host errors: INVALID_ARG (NULL pointers, rank out of range), SHAPE (n_experts % ep_size, n_experts > 256, top_k > 32,
 * d % 256, 2 * d_expert_ffn % 256, d_expert_ffn % 64, M > max_rows), UNSUPPORTED (ep_size > 16).  Every rank passes
 * the same spec_ep_config except for ep_rank (the window layout is derived from it). */
typedef struct spec_ep_config {
    int32_t ep_size, ep_rank;
    int32_t n_experts, top_k;
    int32_t d, d_expert_ffn;
    int32_t max_rows;           /* most rows (tokens) any rank routes per call                                          */
    int32_t cap_rows;           /* most rows this rank can receive; ep_size * max_rows * min(top_k, local experts) is safe */
} spec_ep_config;
typedef struct spec_ep_sizes { size_t window_bytes, scratch_bytes; } spec_ep_sizes;
enum {
    SPEC_EP_T_IDS = 0,          /* window: [M][top_k] int32 selected experts, best first                               */
    SPEC_EP_T_WTS,              /* window: [M][top_k] fp32 renormalised mixture weights                                 */
    SPEC_EP_T_COUNTS,           /* window: [n_experts] int32 entries of this rank per expert                            */
    SPEC_EP_T_RECV_OFF,         /* window: [local experts][ep_size] int32 first received row of each (expert, source)   */
    SPEC_EP_T_RECV_TOTAL,       /* window: [1] int32 rows received (before clamping to cap_rows)                        */
    SPEC_EP_T_EXPERT_OUT,       /* window: [cap_rows][d] fp32 expert outputs in receive order                           */
    SPEC_EP_T_RECV_ROWS         /* scratch: [cap_rows][d] bf16 received rows in receive order                           */
};
spec_status spec_ep_query_sizes(const spec_ep_config* cfg, spec_ep_sizes* out);
spec_status spec_ep_tensor(const spec_ep_config* cfg, void* window, void* scratch, int tensor_id, void** dev_ptr, size_t* bytes);
/* h [M][d] bf16: the block's (normed) input rows; router_w [n_experts][d] bf16. */
spec_status spec_ep_route(const spec_ep_config* cfg, void* window, void* scratch, int M, const void* h,
                          const void* router_w, void* stream);
/* w_gateup [local experts][2 * d_expert_ffn][d] (each expert grouped like SPEC_T_EXPERTS_GATEUP), w_down
 * [local experts][d][d_expert_ffn]: the LOCAL experts only. */
spec_status spec_ep_experts(const spec_ep_config* cfg, void* const* peer_windows_host, void* scratch,
                            const void* w_gateup, const void* w_down, int32_t* status, void* stream);
/* The block with 8-bit expert weights and 8-bit dispatch (the precision of the paper's large-scale projection, Section 5.1).
 * spec_ep_route_e4m3 is spec_ep_route that also publishes the rank's rows as e4m3 codes with one scale per row
 * (spec_quantize_rows' rule; d % 16 == 0), quantised once at their source.  spec_ep_experts_e4m3 pulls those codes and
 * scales (half the bytes of the 16-bit rows) and multiplies them with w_gateup / w_down given as e4m3 codes (one byte per
 * element, same shapes as above) and w_gateup_scale [local experts][2 * d_expert_ffn], w_down_scale [local experts][d] (one
 * fp32 scale per weight row; spec_quantize_rows produces both); the SwiGLU outputs are quantised per row on this rank.  A
 * row gives the same codes wherever its expert lives, so the result does not depend on ep_size.  Every rank of the group
 * must have routed with spec_ep_route_e4m3: a source that did not is reported as SPEC_ERR_STATE (detail = its rank) in
 * `status`.  spec_ep_combine is unchanged. */
spec_status spec_ep_route_e4m3(const spec_ep_config* cfg, void* window, void* scratch, int M, const void* h,
                               const void* router_w, void* stream);
spec_status spec_ep_experts_e4m3(const spec_ep_config* cfg, void* const* peer_windows_host, void* scratch,
                                 const void* w_gateup, const float* w_gateup_scale, const void* w_down,
                                 const float* w_down_scale, int32_t* status, void* stream);
/* x [M][d] fp32 residual of this rank's rows (M as given to spec_ep_route). */
spec_status spec_ep_combine(const spec_ep_config* cfg, void* const* peer_windows_host, int M, float* x, void* stream);

/* Plumbing for windows in other processes (CUDA inter-process memory handles; the device memory must come from a
 * plain device allocation).  spec_ipc_export fills handle_host [64] and the offset of dev_ptr inside its allocation;
 * spec_ipc_open maps the allocation of a handle exported by ANOTHER process and returns its base address (add the
 * offset); spec_ipc_close unmaps it.  Errors: INVALID_ARG, CUDA. */
spec_status spec_ipc_export(void* dev_ptr, unsigned char* handle_host, uint64_t* offset_host);
spec_status spec_ipc_open(const unsigned char* handle_host, void** base_dev_ptr);
spec_status spec_ipc_close(void* base_dev_ptr);

/* Optional per-pass device timing.  When enabled, the step functions bracket the passes selected by `mask` (bit 0
 * attention, bit 1 GEMMs, bit 2 softmax + sampling, bit 3 everything else) with CUDA events on the call's stream.
 * spec_get_timing synchronises `stream`, adds up the elapsed time per class since the last read (milliseconds) and
 * the number of bracketed passes, and resets the accumulation.  At most 8192 passes are recorded between reads;
 * later ones are dropped and counted in `dropped`.  Events are host-side objects; no device memory is allocated. */
typedef struct { float ms[4]; int32_t passes[4]; int32_t dropped; } spec_timing;
spec_status spec_set_timing(spec_ctx* ctx, uint32_t mask);
spec_status spec_get_timing(spec_ctx* ctx, spec_timing* host_out, void* stream);

/* Self-test of the bounded waits every tensor-core kernel uses: a one-thread kernel waits on a barrier that nothing
 * signals, gives up after about one millisecond, and records SPEC_ERR_TIMEOUT in status [4] (device) the way the
 * GEMM roles do; elapsed_kcycles [1] (device) receives the waited time in units of 1024 clock cycles.  Nothing
 * traps or hangs, and the device context stays usable. */
spec_status spec_selftest_bounded_wait(int32_t* status, int32_t* elapsed_kcycles, void* stream);

/* Number of kernels the library has launched in this process so far. */
int64_t spec_launch_count(void);

/* Version string of the library build. */
const char* spec_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPEC_H_ */
