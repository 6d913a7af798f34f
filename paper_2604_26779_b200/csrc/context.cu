// The context: arena layout over caller-owned device buffers and the host-side sequencing of one speculation step
// (draft propose -> target verify -> fused softmax + rejection sampling -> KV commit).  Host code only enqueues
// kernels; everything ragged (lengths, accepted counts, block tables) lives in device metadata, so a step is a fixed
// sequence of launches.
#include <string>
#include <vector>

#include "ops.cuh"

struct Loc { size_t off = 0, bytes = 0; };
constexpr int kActSlots = 5;         // quantised activation buffers of an 8-bit-weights context: QKV, O, gate/up, down, LM head

struct LayerLoc { Loc attn_norm, wqkv, wo, mlp_norm, wgateup, wdown, router, exp_gateup, exp_down, wqkv_s, wo_s, wgateup_s, wdown_s,
                  exp_gateup_s, exp_down_s; };

struct spec_ctx {
    spec_config cfg;
    spec_buffers buf;
    int Mmax;                       // max_batch * (k_max + 1)
    // weights
    Loc embed, lm_head, final_norm, lm_head_s;
    std::vector<LayerLoc> layers;
    size_t weights_bytes = 0;
    // draft weights
    Loc d_wfc, d_wproj, d_norm_e, d_norm_g, d_norm_f;
    LayerLoc d_layer;
    Loc d_lm_head, d_d2t;
    size_t draft_weights_bytes = 0;
    // caches
    size_t kv_pool_bytes = 0, kv_bytes = 0, draft_kv_bytes = 0;
    // state
    Loc seq_len, last_token, block_table, free_stack, free_top, draft_tokens, out_tokens, n_emitted, status, step,
        counters, pending_base, owned, out_logp, history, replace_args;
    size_t state_bytes = 0;
    // workspace
    Loc tokens_in, pos, x, h, qkv, attn_out, gu, act, logits, draft_logits, row_stats, draft_row_stats, taps,
        attn_scratch, dg, dx, d_hidden, d_tok, d_pos,
        moe_logits, moe_ids, moe_wts, moe_rank, moe_counts, moe_offsets, moe_inv, moe_a, moe_gu, moe_act, moe_out, rope, splitk,
        t2d, draft_red, a8, a8_scale;
    size_t workspace_bytes = 0;
    // host-side run state
    int B = 0;
    int k_last = -1;                // k of the last verify
    bool have_pending = false;      // a commit has happened since spec_seq_init
    bool verified = false;          // a verify has run since the last commit
    std::string err;
    // optional pass timing (host-side event pool)
    uint32_t timing_mask = 0;
    std::vector<cudaEvent_t> ev;    // pairs: start, stop
    std::vector<int> ev_cls;        // class of each recorded pair
    int ev_dropped = 0;
};

using namespace spec;

namespace {

struct Arena {
    size_t top = 0;
    Loc take(size_t bytes) { Loc l{top, bytes}; top = align_up(top + bytes, 256); return l; }
};

bool has_tap(const spec_config& c, int t)
{
    for (int i = 0; i < c.n_taps; ++i) if (c.tap_layers[i] == t) return true;
    return false;
}
int tap_slot(const spec_config& c, int t)
{
    for (int i = 0; i < c.n_taps; ++i) if (c.tap_layers[i] == t) return i;
    return -1;
}

spec_status check_config(const spec_config* c)
{
    if (c == nullptr || c->struct_size != sizeof(spec_config) || c->abi_version != SPEC_ABI_VERSION) return SPEC_ERR_INVALID_ARG;
    if (c->n_layers <= 0 || c->d_model <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0 || c->vocab <= 0)
        return SPEC_ERR_SHAPE;
    if (c->n_q_heads % c->n_kv_heads != 0 || c->d_model % 8 != 0 || c->head_dim % 8 != 0 || c->vocab % 4 != 0) return SPEC_ERR_SHAPE;
    if (c->n_experts == 0 && (c->d_ffn <= 0 || c->d_ffn % 128 != 0)) return SPEC_ERR_SHAPE;
    if (c->n_experts > 0 && (c->experts_top_k <= 0 || c->experts_top_k > c->n_experts || c->d_expert_ffn <= 0)) return SPEC_ERR_SHAPE;
    if (c->n_experts > 0 && (c->dtype != SPEC_DTYPE_BF16 || c->n_experts > 256 || c->experts_top_k > 32 ||
                             c->d_expert_ffn % 128 != 0 || c->d_model % 256 != 0)) return SPEC_ERR_UNSUPPORTED;
    if (c->dtype != SPEC_DTYPE_BF16 && c->dtype != SPEC_DTYPE_F32) return SPEC_ERR_UNSUPPORTED;
    if (c->draft_kind < SPEC_DRAFT_NONE || c->draft_kind > SPEC_DRAFT_NGRAM) return SPEC_ERR_UNSUPPORTED;
    if (c->draft_kind == SPEC_DRAFT_NGRAM && (c->ngram_n < 1 || c->ngram_n > 8)) return SPEC_ERR_SHAPE;
    if (c->k_max < 0 || c->k_max > 7 || c->max_batch <= 0) return SPEC_ERR_SHAPE;
    if (c->kv_block_tokens <= 0 || c->kv_num_blocks <= 0 || c->max_blocks_per_seq <= 0) return SPEC_ERR_SHAPE;
    if (c->kv_layer_pools <= 0 || c->kv_layer_pools > c->n_layers) return SPEC_ERR_SHAPE;
    if (c->n_taps < 0 || c->n_taps > 3) return SPEC_ERR_SHAPE;
    for (int i = 0; i < c->n_taps; ++i) if (c->tap_layers[i] < 0 || c->tap_layers[i] > c->n_layers) return SPEC_ERR_SHAPE;
    if (c->draft_kind == SPEC_DRAFT_EAGLE3 && (c->n_taps < 1 || c->draft_d_ffn <= 0 || c->draft_d_ffn % 128 != 0)) return SPEC_ERR_SHAPE;
    if (c->draft_kind == SPEC_DRAFT_MTP && (c->draft_d_ffn <= 0 || c->draft_d_ffn % 128 != 0)) return SPEC_ERR_SHAPE;
    if (!(c->temperature > 0.f) || !(c->rms_eps > 0.f) || !(c->rope_theta > 1.f)) return SPEC_ERR_UNSUPPORTED;
    if (c->vocab > sampler_max_vocab()) return SPEC_ERR_SHAPE;
    if (c->kv_dtype != SPEC_KV_MODEL && (c->kv_dtype != SPEC_KV_E4M3 || c->dtype != SPEC_DTYPE_BF16 || c->head_dim != 128 ||
                                         !(c->kv_scale_k > 0.f) || !(c->kv_scale_v > 0.f) ||
                                         (c->k_max + 1) * (c->n_q_heads / c->n_kv_heads) > 16)) return SPEC_ERR_UNSUPPORTED;
    if (c->weight_dtype != SPEC_W_MODEL &&
        (c->weight_dtype != SPEC_W_E4M3 || c->dtype != SPEC_DTYPE_BF16 ||
         c->d_model % 128 != 0 || (c->n_experts > 0 ? c->d_expert_ffn % 128 != 0 : c->d_ffn % 128 != 0) || (c->n_q_heads * c->head_dim) % 128 != 0 || (c->head_dim != 64 && c->head_dim != 128) ||
         c->vocab % 8 != 0))
        return SPEC_ERR_UNSUPPORTED;
    if (c->draft_vocab != 0 && (c->draft_kind != SPEC_DRAFT_EAGLE3 || c->draft_vocab < 8 || c->draft_vocab > c->vocab ||
                                c->draft_vocab % 8 != 0)) return SPEC_ERR_SHAPE;
    return SPEC_OK;
}

void build_layout(spec_ctx& x)
{
    const spec_config& c = x.cfg;
    const size_t es = dtype_bytes(c.dtype);
    const size_t d = c.d_model, qkv_n = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim, od = (size_t)c.n_q_heads * c.head_dim;
    x.Mmax = c.max_batch * (c.k_max + 1);
    {
        Arena a;
        const bool w8 = c.weight_dtype == SPEC_W_E4M3;        // 8-bit projections: one byte per weight + one fp32 scale per row
        const size_t ws = w8 ? 1 : es;
        x.embed = a.take((size_t)c.vocab * d * es);
        x.lm_head = a.take((size_t)c.vocab * d * ws);
        if (w8) x.lm_head_s = a.take((size_t)c.vocab * 4);
        x.final_norm = a.take(d * 4);
        x.layers.resize(c.n_layers);
        for (auto& L : x.layers) {
            L.attn_norm = a.take(d * 4);
            L.wqkv = a.take(qkv_n * d * ws);
            L.wo = a.take(d * od * ws);
            if (w8) { L.wqkv_s = a.take(qkv_n * 4); L.wo_s = a.take(d * 4); }
            L.mlp_norm = a.take(d * 4);
            if (c.n_experts > 0) {
                L.router = a.take((size_t)c.n_experts * d * es);
                L.exp_gateup = a.take((size_t)c.n_experts * 2 * c.d_expert_ffn * d * ws);     // the router stays 16-bit
                L.exp_down = a.take((size_t)c.n_experts * d * c.d_expert_ffn * ws);
                if (w8) { L.exp_gateup_s = a.take((size_t)c.n_experts * 2 * c.d_expert_ffn * 4); L.exp_down_s = a.take((size_t)c.n_experts * d * 4); }
            } else {
                L.wgateup = a.take((size_t)2 * c.d_ffn * d * ws);
                L.wdown = a.take(d * (size_t)c.d_ffn * ws);
                if (w8) { L.wgateup_s = a.take((size_t)2 * c.d_ffn * 4); L.wdown_s = a.take(d * 4); }
            }
        }
        x.weights_bytes = a.top;
    }
    {
        Arena a;
        if (c.draft_kind == SPEC_DRAFT_EAGLE3 || c.draft_kind == SPEC_DRAFT_MTP) {
            const size_t F = c.draft_d_ffn;
            x.d_norm_e = a.take(d * 4);
            x.d_norm_g = a.take(d * 4);
            x.d_layer.mlp_norm = a.take(d * 4);
            x.d_layer.wo = a.take(d * od * es);
            x.d_layer.wgateup = a.take(2 * F * d * es);
            x.d_layer.wdown = a.take(d * F * es);
            if (c.draft_kind == SPEC_DRAFT_EAGLE3) {
                x.d_wfc = a.take(d * (size_t)c.n_taps * d * es);
                x.d_norm_f = a.take(d * 4);
                x.d_layer.wqkv = a.take(qkv_n * 2 * d * es);
                x.d_lm_head = a.take((size_t)(c.draft_vocab ? c.draft_vocab : c.vocab) * d * es);
                if (c.draft_vocab) x.d_d2t = a.take((size_t)c.draft_vocab * 4);
            } else {
                x.d_wproj = a.take(d * 2 * d * es);
                x.d_layer.attn_norm = a.take(d * 4);
                x.d_layer.wqkv = a.take(qkv_n * d * es);
            }
        }
        x.draft_weights_bytes = a.top;
    }
    x.kv_pool_bytes = align_up((size_t)c.kv_num_blocks * c.n_kv_heads * c.kv_block_tokens * c.head_dim *
                               (c.kv_dtype == SPEC_KV_E4M3 ? 1 : es), 256);
    x.kv_bytes = x.kv_pool_bytes * 2 * c.kv_layer_pools;
    x.draft_kv_bytes = (c.draft_kind == SPEC_DRAFT_EAGLE3 || c.draft_kind == SPEC_DRAFT_MTP) ? x.kv_pool_bytes * 2 : 0;
    {
        Arena a;
        const size_t Bm = c.max_batch;
        x.seq_len = a.take(Bm * 4);
        x.last_token = a.take(Bm * 4);
        x.block_table = a.take(Bm * c.max_blocks_per_seq * 4);
        x.free_stack = a.take((size_t)c.kv_num_blocks * 4);
        x.free_top = a.take(4);
        x.draft_tokens = a.take(Bm * (size_t)(c.k_max > 0 ? c.k_max : 1) * 4);
        x.out_tokens = a.take(Bm * (c.k_max + 1) * 4);
        x.n_emitted = a.take(Bm * 4);
        x.status = a.take(16);
        x.step = a.take(4);
        x.counters = a.take(3 * 8);
        x.pending_base = a.take(Bm * 4);
        x.owned = a.take(Bm * 4);
        x.out_logp = a.take(Bm * (c.k_max + 1) * 4);
        if (c.draft_kind == SPEC_DRAFT_NGRAM) x.history = a.take(Bm * (size_t)c.max_blocks_per_seq * c.kv_block_tokens * 4);
        x.replace_args = a.take(3 * Bm * 4);
        x.state_bytes = a.top;
    }
    {
        Arena a;
        const size_t M = x.Mmax, Bm = c.max_batch;
        const size_t Fmax = (size_t)(c.d_ffn > c.draft_d_ffn ? c.d_ffn : c.draft_d_ffn);
        x.tokens_in = a.take(M * 4);
        x.pos = a.take(M * 4);
        x.x = a.take(M * d * 4);
        x.h = a.take(M * 2 * d * es);
        x.qkv = a.take(M * qkv_n * es);
        x.attn_out = a.take(M * od * es);
        x.gu = a.take(M * 2 * Fmax * es);
        x.act = a.take(M * Fmax * es);
        if (c.weight_dtype == SPEC_W_E4M3) {                  // activations as e4m3 codes + one scale per row, rewritten before every projection
            const size_t f8 = c.n_experts > 0 ? (size_t)c.d_expert_ffn : (size_t)c.d_ffn;
            const size_t kmax = (f8 > od ? f8 : od) > d ? (f8 > od ? f8 : od) : d;
            // a mixture-of-experts layer quantises its rows in expert order: top_k entries per row, + one tile of slack rows
            // for the last group's TMA box
            const size_t rows8 = c.n_experts > 0 ? M * c.experts_top_k + 128 : M;
            // five slots, one per projection of a layer (QKV, O, gate/up, down) and one for the LM head, so that what the last
            // layer and the LM head consumed stays readable after the pass (SPEC_T_ACT_CODES / SPEC_T_ACT_SCALES)
            x.a8 = a.take(kActSlots * rows8 * kmax);
            x.a8_scale = a.take(kActSlots * rows8 * 4);
        }
        x.logits = a.take(M * (size_t)c.vocab * 4);
        x.draft_logits = a.take(Bm * (size_t)(c.k_max > 0 ? c.k_max : 1) * c.vocab * 4);   // sized for the whole vocabulary
        if (c.draft_vocab) {
            x.t2d = a.take((size_t)c.vocab * 4);
            x.draft_red = a.take(Bm * (size_t)(c.k_max > 0 ? c.k_max : 1) * 4);
        }
        x.row_stats = a.take(M * 8);
        x.draft_row_stats = a.take(Bm * (size_t)(c.k_max > 0 ? c.k_max : 1) * 8);
        x.taps = a.take(M * (size_t)(c.n_taps > 0 ? c.n_taps : 1) * d * es);
        x.attn_scratch = a.take(attention_scratch_bytes(c.max_batch, c.k_max + 1, c.n_q_heads, c.n_kv_heads, c.head_dim,
                                                        c.max_blocks_per_seq * c.kv_block_tokens));
        x.dg = a.take(M * d * 4);
        x.dx = a.take(M * d * 4);
        x.d_hidden = a.take(Bm * d * 4);
        x.d_tok = a.take(M * 4);
        x.d_pos = a.take(M * 4);
        x.rope = a.take(M * (size_t)(c.head_dim / 2) * 8);
        x.splitk = a.take((size_t)32 << 20);
        if (c.n_experts > 0) {
            const size_t n = M * c.experts_top_k, E = c.n_experts, Fe = c.d_expert_ffn;
            x.moe_logits = a.take(M * E * 4);
            x.moe_ids = a.take(n * 4);
            x.moe_wts = a.take(n * 4);
            x.moe_rank = a.take(n * 4);
            x.moe_counts = a.take(E * 4);
            x.moe_offsets = a.take(E * 4);
            x.moe_inv = a.take(n * 4);
            x.moe_a = a.take((n + 128) * d * es);                // + one tile of slack rows for the last group's TMA box
            x.moe_gu = a.take(n * 2 * Fe * es);
            x.moe_act = a.take((n + 128) * Fe * es);
            x.moe_out = a.take(n * d * 4);
        }
        x.workspace_bytes = a.top;
    }
}

template <class T = void> T* at(void* base, const Loc& l) { return reinterpret_cast<T*>(static_cast<char*>(base) + l.off); }

struct LayerPtrs { const float* attn_norm; const void* wqkv; const void* wo; const float* mlp_norm; const void* wgateup; const void* wdown;
                   const void* router; const void* exp_gateup; const void* exp_down;
                   const float* wqkv_s; const float* wo_s; const float* wgateup_s; const float* wdown_s;       // 8-bit weights: row scales
                   const float* exp_gateup_s; const float* exp_down_s; };

LayerPtrs layer_ptrs(void* base, const LayerLoc& L)
{
    return {at<const float>(base, L.attn_norm), at<const void>(base, L.wqkv), at<const void>(base, L.wo),
            at<const float>(base, L.mlp_norm), at<const void>(base, L.wgateup), at<const void>(base, L.wdown),
            L.router.bytes ? at<const void>(base, L.router) : nullptr, at<const void>(base, L.exp_gateup),
            at<const void>(base, L.exp_down),
            L.wqkv_s.bytes ? at<const float>(base, L.wqkv_s) : nullptr, L.wo_s.bytes ? at<const float>(base, L.wo_s) : nullptr,
            L.wgateup_s.bytes ? at<const float>(base, L.wgateup_s) : nullptr, L.wdown_s.bytes ? at<const float>(base, L.wdown_s) : nullptr,
            L.exp_gateup_s.bytes ? at<const float>(base, L.exp_gateup_s) : nullptr,
            L.exp_down_s.bytes ? at<const float>(base, L.exp_down_s) : nullptr};
}

#define TRY(expr) do { spec_status s__ = (expr); if (s__ != SPEC_OK) return s__; } while (0)

// Records why a call was refused (read back with spec_last_error) and returns the code.
spec_status fail(spec_ctx* c, spec_status code, const char* why)
{
    if (c != nullptr) c->err = why;
    return code;
}

// Installs the context's split-K scratch for the duration of a step function.
struct ScratchScope {
    explicit ScratchScope(spec_ctx* c)
    {
        spec::gemm_scratch().ptr = static_cast<char*>(c->buf.workspace) + c->splitk.off;
        spec::gemm_scratch().bytes = c->splitk.bytes;
    }
    ~ScratchScope() { spec::gemm_scratch() = spec::GemmScratch{}; }
};

constexpr int kMaxTimedPasses = 8192;

// Brackets a pass with two events when its class is selected by the context's timing mask.
struct Timed {
    spec_ctx& c; cudaStream_t st; int idx = -1;
    Timed(spec_ctx& ctx, int cls, cudaStream_t s) : c(ctx), st(s)
    {
        if (!(c.timing_mask & (1u << cls))) return;
        if ((int)c.ev_cls.size() >= kMaxTimedPasses) { c.ev_dropped += 1; return; }
        idx = (int)c.ev_cls.size();
        c.ev_cls.push_back(cls);
        cudaEventRecord(c.ev[2 * idx], st);
    }
    ~Timed() { if (idx >= 0) cudaEventRecord(c.ev[2 * idx + 1], st); }
};
#define TIMED(ctx, cls, expr) do { Timed t__(ctx, cls, st); TRY(expr); } while (0)
enum { CLS_ATTN = 0, CLS_GEMM = 1, CLS_SAMPLE = 2, CLS_OTHER = 3 };

// attention + MLP of one decoder layer on the fp32 residual `res` [M][d].  `qkv_in` [M][qkv_k] is the already
// prepared input of the QKV projection.
spec_status run_layer_body(spec_ctx& c, const LayerPtrs& W, int d_ffn, float* res, const void* qkv_in, int qkv_k, int B, int R,
                           const int32_t* pos, void* k_pool, void* v_pool, int launch_index, cudaStream_t st)
{
    // `pos` rows have their (cos, sin) table in c.rope (filled by the caller for this forward)
    const spec_config& g = c.cfg;
    const int M = B * R, d = g.d_model, dh = g.head_dim, Hq = g.n_q_heads, Hkv = g.n_kv_heads;
    const int qkv_n = (Hq + 2 * Hkv) * dh, dt = g.dtype;
    void* ws = c.buf.workspace;
    int32_t* status_word = at<int32_t>(c.buf.state, c.status);
    const bool w8 = g.weight_dtype == SPEC_W_E4M3 && W.wqkv_s != nullptr;   // the target's layers with 8-bit weights (the draft head has none)
    // what the fused QKV epilogue needs (rotary table, cache slots), and the attention launch: the same for every weight format
    auto qkv_epilogue = [&]() {
        QkvEpilogue e{Hq, Hkv, dh, R, g.max_blocks_per_seq, g.kv_block_tokens, pos, at<int32_t>(c.buf.state, c.block_table),
                      at<float>(ws, c.rope), k_pool, v_pool};
        if (g.kv_dtype == SPEC_KV_E4M3) { e.kv_fp8 = 1; e.k_scale = g.kv_scale_k; e.v_scale = g.kv_scale_v; }
        return e;
    };
    auto attention = [&]() -> spec_status {
        AttnArgs a{B, R, Hq, Hkv, dh, g.kv_block_tokens, g.max_blocks_per_seq, at(ws, c.qkv), qkv_n, k_pool, v_pool,
                   at<int32_t>(c.buf.state, c.block_table), pos, at(ws, c.attn_out), Hq * dh, dt, at(ws, c.attn_scratch),
                   c.attn_scratch.bytes, g.max_blocks_per_seq * g.kv_block_tokens, launch_index};
        a.status = status_word;
        if (g.kv_dtype == SPEC_KV_E4M3) { a.kv_fp8 = 1; a.k_scale = g.kv_scale_k; a.v_scale = g.kv_scale_v; }
        Timed t__(c, CLS_ATTN, st);
        return launch_attention(a, st);
    };
    if (w8) {
        const size_t slot_bytes = c.a8.bytes / kActSlots, slot_rows = c.a8_scale.bytes / kActSlots / 4;
        auto a8_of = [&](int slot) { return at<unsigned char>(ws, c.a8) + slot * slot_bytes; };
        auto a8s_of = [&](int slot) { return at<float>(ws, c.a8_scale) + slot * slot_rows; };
        // every projection: its input rows to e4m3 with a scale per row, then the 8-bit tensor-core product; the epilogues
        // are the usual ones (rotary + cache append, residual add, SwiGLU) on the rescaled accumulators
        if (qkv_in == nullptr) TRY(launch_rmsnorm_quantize(M, d, res, W.attn_norm, g.rms_eps, a8_of(0), a8s_of(0), st));   // norm fused with the quantiser
        else TRY(launch_quantize_rows(M, qkv_k, qkv_in, a8_of(0), a8s_of(0), st));
        TIMED(c, CLS_GEMM, launch_gemm8_qkv_tc(M, qkv_k, a8_of(0), a8s_of(0), W.wqkv, W.wqkv_s, at(ws, c.qkv), qkv_epilogue(), status_word, st));
        TRY(attention());
        TRY(launch_quantize_rows(M, Hq * dh, at(ws, c.attn_out), a8_of(1), a8s_of(1), st));
        TIMED(c, CLS_GEMM, launch_gemm8_tc(M, d, Hq * dh, a8_of(1), a8s_of(1), W.wo, W.wo_s, res, d, SPEC_DTYPE_F32, 1, 1.f, nullptr, 0, nullptr, 0,
                                           status_word, st));
        if (W.router != nullptr) {
            // mixture of experts: the router decides on the 16-bit rows; the rows are quantised in expert order (slot 2), the
            // SwiGLU outputs again (slot 3); both grouped products run on the 8-bit path with the experts' row scales
            const int E = g.n_experts, tk = g.experts_top_k, Fe = g.d_expert_ffn, n = M * tk;
            TRY(launch_rmsnorm(M, d, res, W.mlp_norm, g.rms_eps, at(ws, c.h), d, 0, dt, st));
            TIMED(c, CLS_GEMM, launch_gemm(M, E, d, at(ws, c.h), d, W.router, at(ws, c.moe_logits), E, dt, SPEC_DTYPE_F32, 0, st));
            TRY(launch_moe_route(M, E, tk, at<float>(ws, c.moe_logits), at<int32_t>(ws, c.moe_ids), at<float>(ws, c.moe_wts), st));
            // the rows are quantised once (parked in slot 3, which the SwiGLU outputs take over later) and their codes and
            // scales permuted into expert order: the same codes as quantising every permuted copy, an eighth of the work
            TRY(launch_quantize_rows(M, d, at(ws, c.h), a8_of(3), a8s_of(3), st));
            TRY(launch_moe_permute(M, E, tk, d / 2, at<int32_t>(ws, c.moe_ids), at<int32_t>(ws, c.moe_rank), at<int32_t>(ws, c.moe_counts),
                                   at<int32_t>(ws, c.moe_offsets), at<int32_t>(ws, c.moe_inv), a8_of(3), a8_of(2), st, a8s_of(3), a8s_of(2)));
            TIMED(c, CLS_GEMM, launch_gemm8_grouped(n, M, E, 2 * Fe, d, a8_of(2), a8s_of(2), W.exp_gateup, W.exp_gateup_s, at(ws, c.moe_act), dt, 1,
                                                    at<int32_t>(ws, c.moe_counts), at<int32_t>(ws, c.moe_offsets), status_word, st));
            TRY(launch_quantize_rows(n, Fe, at(ws, c.moe_act), a8_of(3), a8s_of(3), st));
            TIMED(c, CLS_GEMM, launch_gemm8_grouped(n, M, E, d, Fe, a8_of(3), a8s_of(3), W.exp_down, W.exp_down_s, at(ws, c.moe_out), SPEC_DTYPE_F32, 0,
                                                    at<int32_t>(ws, c.moe_counts), at<int32_t>(ws, c.moe_offsets), status_word, st));
            TRY(launch_moe_combine(M, tk, d, at<float>(ws, c.moe_wts), at<int32_t>(ws, c.moe_inv), at<float>(ws, c.moe_out), res, st));
            return SPEC_OK;
        }
        TRY(launch_rmsnorm_quantize(M, d, res, W.mlp_norm, g.rms_eps, a8_of(2), a8s_of(2), st));
        TIMED(c, CLS_GEMM, launch_gemm8_swiglu_tc(M, d_ffn, d, a8_of(2), a8s_of(2), W.wgateup, W.wgateup_s, at(ws, c.act), status_word, st));
        TRY(launch_quantize_rows(M, d_ffn, at(ws, c.act), a8_of(3), a8s_of(3), st));
        TIMED(c, CLS_GEMM, launch_gemm8_tc(M, d, d_ffn, a8_of(3), a8s_of(3), W.wdown, W.wdown_s, res, d, SPEC_DTYPE_F32, 1, 1.f, nullptr, 0, nullptr, 0,
                                           status_word, st));
        return SPEC_OK;
    }
    const bool tc = gemm_tc_supported(M, qkv_n, qkv_k, qkv_in, qkv_k, W.wqkv, at(ws, c.qkv), qkv_n, dt, dt);
    // very few rows (the thin tail of a rollout): plain weight-streaming projections + the small element-wise kernels beat
    // the fused tensor-core epilogues, which have too few tiles to pull the weights at the HBM rate
    const bool thin = g.kv_dtype != SPEC_KV_E4M3 &&
                      (gemm_skinny_supported(M, qkv_n, qkv_k, qkv_in, qkv_k, W.wqkv, dt) ||
                       gemm_tc_thin_supported(M, qkv_n, qkv_k, qkv_in, qkv_k, W.wqkv, at(ws, c.qkv), qkv_n, dt, dt)) &&
                      (gemm_skinny_supported(M, 2 * d_ffn, d, at(ws, c.h), d, W.wgateup, dt) ||
                       gemm_tc_thin_supported(M, 2 * d_ffn, d, at(ws, c.h), d, W.wgateup, at(ws, c.gu), 2 * d_ffn, dt, dt));
    if (tc && !thin && (dh == 64 || dh == 128)) {
        // projection, rotary embedding and the append into the paged cache in one kernel
        TIMED(c, CLS_GEMM, launch_gemm_qkv_tc(M, qkv_k, qkv_in, qkv_k, W.wqkv, at(ws, c.qkv), qkv_epilogue(), status_word, st));
    } else {
        if (g.kv_dtype == SPEC_KV_E4M3) return SPEC_ERR_UNSUPPORTED;    // the 8-bit cache is written by the fused epilogue only
        TIMED(c, CLS_GEMM, launch_gemm(M, qkv_n, qkv_k, qkv_in, qkv_k, W.wqkv, at(ws, c.qkv), qkv_n, dt, dt, 0, st));
        TRY(launch_rope_append(B, R, Hq, Hkv, dh, g.rope_theta, at(ws, c.qkv), pos, k_pool, v_pool,
                               at<int32_t>(c.buf.state, c.block_table), g.max_blocks_per_seq, g.kv_block_tokens, dt, st,
                               at<float>(ws, c.rope)));
    }
    TRY(attention());
    TIMED(c, CLS_GEMM, launch_gemm(M, d, Hq * dh, at(ws, c.attn_out), Hq * dh, W.wo, res, d, dt, SPEC_DTYPE_F32, 1, st));
    TRY(launch_rmsnorm(M, d, res, W.mlp_norm, g.rms_eps, at(ws, c.h), d, 0, dt, st));
    if (W.router != nullptr) {
        // mixture of experts: router -> top-k -> permute into expert order -> grouped gate/up, SwiGLU, grouped down -> combine
        const int E = g.n_experts, tk = g.experts_top_k, Fe = g.d_expert_ffn, n = M * tk;
        int32_t* status = at<int32_t>(c.buf.state, c.status);
        TIMED(c, CLS_GEMM, launch_gemm(M, E, d, at(ws, c.h), d, W.router, at(ws, c.moe_logits), E, dt, SPEC_DTYPE_F32, 0, st));
        TRY(launch_moe_route(M, E, tk, at<float>(ws, c.moe_logits), at<int32_t>(ws, c.moe_ids), at<float>(ws, c.moe_wts), st));
        TRY(launch_moe_permute(M, E, tk, d, at<int32_t>(ws, c.moe_ids), at<int32_t>(ws, c.moe_rank), at<int32_t>(ws, c.moe_counts),
                               at<int32_t>(ws, c.moe_offsets), at<int32_t>(ws, c.moe_inv), at(ws, c.h), at(ws, c.moe_a), st));
        TIMED(c, CLS_GEMM, launch_gemm_grouped(n, M, E, 2 * Fe, d, at(ws, c.moe_a), W.exp_gateup, at(ws, c.moe_act), dt, 1,
                                               at<int32_t>(ws, c.moe_counts), at<int32_t>(ws, c.moe_offsets), status, st));
        TIMED(c, CLS_GEMM, launch_gemm_grouped(n, M, E, d, Fe, at(ws, c.moe_act), W.exp_down, at(ws, c.moe_out), SPEC_DTYPE_F32, 0,
                                               at<int32_t>(ws, c.moe_counts), at<int32_t>(ws, c.moe_offsets), status, st));
        TRY(launch_moe_combine(M, tk, d, at<float>(ws, c.moe_wts), at<int32_t>(ws, c.moe_inv), at<float>(ws, c.moe_out), res, st));
        return SPEC_OK;
    }
    if (!thin && gemm_tc_supported(M, 2 * d_ffn, d, at(ws, c.h), d, W.wgateup, at(ws, c.act), d_ffn, dt, dt)) {
        TIMED(c, CLS_GEMM, launch_gemm_swiglu_tc(M, d_ffn, d, at(ws, c.h), d, W.wgateup, at(ws, c.act), status_word, st));
    } else {
        TIMED(c, CLS_GEMM, launch_gemm(M, 2 * d_ffn, d, at(ws, c.h), d, W.wgateup, at(ws, c.gu), 2 * d_ffn, dt, dt, 0, st));
        TRY(launch_swiglu(M, d_ffn, at(ws, c.gu), at(ws, c.act), dt, st));
    }
    TIMED(c, CLS_GEMM, launch_gemm(M, d, d_ffn, at(ws, c.act), d_ffn, W.wdown, res, d, dt, SPEC_DTYPE_F32, 1, st));
    return SPEC_OK;
}

__global__ void draft_rows0_kernel(int B, int R, const int32_t* n_emitted, const int32_t* pending_base,
                                   const int32_t* out_tokens, int32_t* tok, int32_t* pos)
{
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= B * R) return;
    const int b = m / R, i = m % R;
    const bool valid = i < n_emitted[b];
    pos[m] = valid ? pending_base[b] + i : -1;
    tok[m] = valid ? out_tokens[m] : -1;
}

__global__ void draft_rows_kernel(int B, int j, const int32_t* seq_len, const int32_t* n_emitted, const int32_t* draft_tokens,
                                  int stride, int32_t* tok, int32_t* pos)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    // a slot that was just replaced has nothing committed to draft from: its rows are inert (zero hidden state, uniform
    // q) until its first commit, and touch no cache slot
    const bool fresh = n_emitted[b] == 0;
    pos[b] = fresh ? -1 : seq_len[b] - 1 + j;
    tok[b] = fresh ? -1 : draft_tokens[(size_t)b * stride + j - 1];
}

}  // namespace

extern "C" spec_status spec_query_sizes(const spec_config* cfg, spec_sizes* out)
{
    if (out == nullptr) return SPEC_ERR_INVALID_ARG;
    TRY(check_config(cfg));
    spec_ctx tmp;
    tmp.cfg = *cfg;
    build_layout(tmp);
    out->weights_bytes = tmp.weights_bytes;
    out->draft_weights_bytes = tmp.draft_weights_bytes;
    out->kv_bytes = tmp.kv_bytes;
    out->draft_kv_bytes = tmp.draft_kv_bytes;
    out->workspace_bytes = tmp.workspace_bytes;
    out->state_bytes = tmp.state_bytes;
    return SPEC_OK;
}

extern "C" spec_status spec_create(const spec_config* cfg, const spec_buffers* b, spec_ctx** out)
{
    if (out == nullptr || b == nullptr) return SPEC_ERR_INVALID_ARG;
    TRY(check_config(cfg));
    if (!b->weights || !b->kv || !b->workspace || !b->state) return SPEC_ERR_INVALID_ARG;
    if ((cfg->draft_kind == SPEC_DRAFT_EAGLE3 || cfg->draft_kind == SPEC_DRAFT_MTP) && (!b->draft_weights || !b->draft_kv))
        return SPEC_ERR_INVALID_ARG;
    const void* ptrs[] = {b->weights, b->draft_weights, b->kv, b->draft_kv, b->workspace, b->state};
    for (const void* p : ptrs) if ((reinterpret_cast<uintptr_t>(p) & 255u) != 0) return SPEC_ERR_INVALID_ARG;
    spec_ctx* c = new spec_ctx();
    c->cfg = *cfg;
    c->buf = *b;
    build_layout(*c);
    *out = c;
    return SPEC_OK;
}

extern "C" spec_status spec_destroy(spec_ctx* ctx)
{
    if (ctx == nullptr) return SPEC_ERR_INVALID_ARG;
    for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
    delete ctx;
    return SPEC_OK;
}

extern "C" const char* spec_last_error(const spec_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

extern "C" const char* spec_version(void) { return "spec-step 0.1 (sm_100a)"; }

extern "C" spec_status spec_tensor(spec_ctx* c, int id, int layer, void** dev_ptr, size_t* bytes)
{
    if (c == nullptr || dev_ptr == nullptr || bytes == nullptr) return SPEC_ERR_INVALID_ARG;
    const spec_config& g = c->cfg;
    void* base = nullptr;
    Loc l;
    auto layer_ok = [&]() { return layer >= 0 && layer < g.n_layers; };
    switch (id) {
    case SPEC_T_EMBED: base = c->buf.weights; l = c->embed; break;
    case SPEC_T_LM_HEAD: base = c->buf.weights; l = c->lm_head; break;
    case SPEC_T_FINAL_NORM: base = c->buf.weights; l = c->final_norm; break;
    case SPEC_T_ATTN_NORM: case SPEC_T_WQKV: case SPEC_T_WO: case SPEC_T_MLP_NORM: case SPEC_T_WGATEUP: case SPEC_T_WDOWN:
    case SPEC_T_ROUTER: case SPEC_T_EXPERTS_GATEUP: case SPEC_T_EXPERTS_DOWN: {
        if (!layer_ok()) return SPEC_ERR_INVALID_ARG;
        const LayerLoc& L = c->layers[layer];
        base = c->buf.weights;
        l = id == SPEC_T_ATTN_NORM ? L.attn_norm : id == SPEC_T_WQKV ? L.wqkv : id == SPEC_T_WO ? L.wo :
            id == SPEC_T_MLP_NORM ? L.mlp_norm : id == SPEC_T_WGATEUP ? L.wgateup : id == SPEC_T_WDOWN ? L.wdown :
            id == SPEC_T_ROUTER ? L.router : id == SPEC_T_EXPERTS_GATEUP ? L.exp_gateup : L.exp_down;
        break;
    }
    case SPEC_T_LM_HEAD_SCALE: base = c->buf.weights; l = c->lm_head_s; break;
    case SPEC_T_WQKV_SCALE: case SPEC_T_WO_SCALE: case SPEC_T_WGATEUP_SCALE: case SPEC_T_WDOWN_SCALE: {
        if (!layer_ok()) return SPEC_ERR_INVALID_ARG;
        const LayerLoc& L = c->layers[layer];
        base = c->buf.weights;
        l = id == SPEC_T_WQKV_SCALE ? L.wqkv_s : id == SPEC_T_WO_SCALE ? L.wo_s : id == SPEC_T_WGATEUP_SCALE ? L.wgateup_s : L.wdown_s;
        break;
    }
    case SPEC_T_D_WFC: base = c->buf.draft_weights; l = c->d_wfc; break;
    case SPEC_T_D_WPROJ: base = c->buf.draft_weights; l = c->d_wproj; break;
    case SPEC_T_D_NORM_E: base = c->buf.draft_weights; l = c->d_norm_e; break;
    case SPEC_T_D_NORM_G: base = c->buf.draft_weights; l = c->d_norm_g; break;
    case SPEC_T_D_NORM_F: base = c->buf.draft_weights; l = c->d_norm_f; break;
    case SPEC_T_D_ATTN_NORM: base = c->buf.draft_weights; l = c->d_layer.attn_norm; break;
    case SPEC_T_D_WQKV: base = c->buf.draft_weights; l = c->d_layer.wqkv; break;
    case SPEC_T_D_WO: base = c->buf.draft_weights; l = c->d_layer.wo; break;
    case SPEC_T_D_MLP_NORM: base = c->buf.draft_weights; l = c->d_layer.mlp_norm; break;
    case SPEC_T_D_WGATEUP: base = c->buf.draft_weights; l = c->d_layer.wgateup; break;
    case SPEC_T_D_WDOWN: base = c->buf.draft_weights; l = c->d_layer.wdown; break;
    case SPEC_T_D_LM_HEAD: base = c->buf.draft_weights; l = c->d_lm_head; break;
    case SPEC_T_D_D2T: base = c->buf.draft_weights; l = c->d_d2t; break;
    case SPEC_T_KV_K: case SPEC_T_KV_V:
        if (layer < 0 || layer >= g.kv_layer_pools) return SPEC_ERR_INVALID_ARG;
        base = c->buf.kv;
        l = Loc{((size_t)layer * 2 + (id == SPEC_T_KV_V ? 1 : 0)) * c->kv_pool_bytes, c->kv_pool_bytes};
        break;
    case SPEC_T_DRAFT_KV_K: case SPEC_T_DRAFT_KV_V:
        if (g.draft_kind != SPEC_DRAFT_EAGLE3 && g.draft_kind != SPEC_DRAFT_MTP) return SPEC_ERR_INVALID_ARG;
        base = c->buf.draft_kv;
        l = Loc{(id == SPEC_T_DRAFT_KV_V ? 1 : 0) * c->kv_pool_bytes, c->kv_pool_bytes};
        break;
    case SPEC_T_SEQ_LEN: base = c->buf.state; l = c->seq_len; break;
    case SPEC_T_LAST_TOKEN: base = c->buf.state; l = c->last_token; break;
    case SPEC_T_BLOCK_TABLE: base = c->buf.state; l = c->block_table; break;
    case SPEC_T_FREE_STACK: base = c->buf.state; l = c->free_stack; break;
    case SPEC_T_FREE_TOP: base = c->buf.state; l = c->free_top; break;
    case SPEC_T_DRAFT_TOKENS: base = c->buf.state; l = c->draft_tokens; break;
    case SPEC_T_OUT_TOKENS: base = c->buf.state; l = c->out_tokens; break;
    case SPEC_T_N_EMITTED: base = c->buf.state; l = c->n_emitted; break;
    case SPEC_T_STATUS: base = c->buf.state; l = c->status; break;
    case SPEC_T_STEP: base = c->buf.state; l = c->step; break;
    case SPEC_T_OUT_LOGP: base = c->buf.state; l = c->out_logp; break;
    case SPEC_T_TOKEN_HISTORY: base = c->buf.state; l = c->history; break;
    case SPEC_T_LOGITS: base = c->buf.workspace; l = c->logits; break;
    case SPEC_T_DRAFT_LOGITS: base = c->buf.workspace; l = c->draft_logits; break;
    case SPEC_T_ROW_STATS: base = c->buf.workspace; l = c->row_stats; break;
    case SPEC_T_DRAFT_ROW_STATS: base = c->buf.workspace; l = c->draft_row_stats; break;
    case SPEC_T_TAPS: base = c->buf.workspace; l = c->taps; break;
    case SPEC_T_HIDDEN: base = c->buf.workspace; l = c->x; break;
    case SPEC_T_MOE_LOGITS: base = c->buf.workspace; l = c->moe_logits; break;
    case SPEC_T_MOE_IDS: base = c->buf.workspace; l = c->moe_ids; break;
    case SPEC_T_MOE_WTS: base = c->buf.workspace; l = c->moe_wts; break;
    case SPEC_T_MOE_INV: base = c->buf.workspace; l = c->moe_inv; break;
    case SPEC_T_EXPERTS_GATEUP_SCALE: case SPEC_T_EXPERTS_DOWN_SCALE: {
        if (!layer_ok()) return SPEC_ERR_INVALID_ARG;
        base = c->buf.weights;
        l = id == SPEC_T_EXPERTS_GATEUP_SCALE ? c->layers[layer].exp_gateup_s : c->layers[layer].exp_down_s;
        break;
    }
    case SPEC_T_ACT_CODES: case SPEC_T_ACT_SCALES: {
        // `layer` selects the slot: 0 QKV, 1 O, 2 gate/up, 3 down (of the last layer run), 4 LM head
        if (layer < 0 || layer >= kActSlots) return SPEC_ERR_INVALID_ARG;
        const Loc& whole = id == SPEC_T_ACT_CODES ? c->a8 : c->a8_scale;
        base = c->buf.workspace;
        l.bytes = whole.bytes / kActSlots;
        l.off = whole.off + layer * l.bytes;
        break;
    }
    default: return SPEC_ERR_INVALID_ARG;
    }
    if (base == nullptr || l.bytes == 0) return SPEC_ERR_INVALID_ARG;
    *dev_ptr = static_cast<char*>(base) + l.off;
    *bytes = l.bytes;
    return SPEC_OK;
}

extern "C" spec_status spec_seq_init(spec_ctx* c, int B, const int32_t* seq_len_host, const int32_t* last_token_host,
                                     const int32_t* free_stack_host, void* stream)
{
    if (c == nullptr || B < 0 || (B > 0 && (!seq_len_host || !last_token_host)) || !free_stack_host) return SPEC_ERR_INVALID_ARG;
    const spec_config& g = c->cfg;
    if (B > g.max_batch) return fail(c, SPEC_ERR_SHAPE, "spec_seq_init: B exceeds max_batch");
    const int bt = g.kv_block_tokens, mb = g.max_blocks_per_seq, nb = g.kv_num_blocks;
    std::vector<int32_t> table((size_t)g.max_batch * mb, -1), stack(free_stack_host, free_stack_host + nb), owned(g.max_batch, 0);
    std::vector<char> seen(nb, 0);
    for (int i = 0; i < nb; ++i) {
        if (stack[i] < 0 || stack[i] >= nb || seen[stack[i]]) return fail(c, SPEC_ERR_INVALID_ARG, "spec_seq_init: free_stack_host is not a permutation of the block ids");
        seen[stack[i]] = 1;
    }
    int top = nb;
    for (int b = 0; b < B; ++b) {
        if (seq_len_host[b] < 0 || last_token_host[b] < 0 || last_token_host[b] >= g.vocab) return SPEC_ERR_INVALID_ARG;
        const int need = (seq_len_host[b] + bt - 1) / bt;
        if (need > mb || (seq_len_host[b] + g.k_max + 1 + bt - 1) / bt > mb)
            return fail(c, SPEC_ERR_SHAPE, "spec_seq_init: a sequence does not fit max_blocks_per_seq");
        if (need > top) return fail(c, SPEC_ERR_SHAPE, "spec_seq_init: not enough KV blocks for the initial lengths");
        for (int j = 0; j < need; ++j) table[(size_t)b * mb + j] = stack[--top];
        owned[b] = need;
    }
    cudaStream_t st = (cudaStream_t)stream;
    char* sb = static_cast<char*>(c->buf.state);
    SPEC_CUDA_OK(cudaMemsetAsync(sb, 0, c->state_bytes, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(sb + c->seq_len.off, seq_len_host, (size_t)B * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(sb + c->last_token.off, last_token_host, (size_t)B * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(sb + c->block_table.off, table.data(), table.size() * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(sb + c->free_stack.off, stack.data(), (size_t)nb * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(sb + c->free_top.off, &top, 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(sb + c->owned.off, owned.data(), owned.size() * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaStreamSynchronize(st));          // the host staging vectors go out of scope here
    c->B = B;
    c->k_last = -1;
    c->have_pending = false;
    c->verified = false;
    return SPEC_OK;
}

extern "C" spec_status spec_seq_replace(spec_ctx* c, int n, const int32_t* slots_host, const int32_t* seq_len_host,
                                        const int32_t* last_token_host, void* stream)
{
    if (c == nullptr || n < 0 || (n > 0 && (!slots_host || !seq_len_host || !last_token_host))) return SPEC_ERR_INVALID_ARG;
    const spec_config& g = c->cfg;
    if (c->verified) return fail(c, SPEC_ERR_STATE, "spec_seq_replace: a verified step is waiting for its commit");
    if (n > c->B) return fail(c, SPEC_ERR_SHAPE, "spec_seq_replace: more slots listed than sequences running");
    if (n == 0) return SPEC_OK;
    const int bt = g.kv_block_tokens, mb = g.max_blocks_per_seq;
    std::vector<char> seen(c->B, 0);
    for (int i = 0; i < n; ++i) {
        const int b = slots_host[i];
        if (b < 0 || b >= c->B || seen[b]) return fail(c, SPEC_ERR_INVALID_ARG, "spec_seq_replace: a slot is out of range or listed twice");
        seen[b] = 1;
        if (seq_len_host[i] < 0) continue;                  // retire: the slot stays empty until it is replaced again
        if (last_token_host[i] < 0 || last_token_host[i] >= g.vocab) return SPEC_ERR_INVALID_ARG;
        if ((seq_len_host[i] + g.k_max + 1 + bt - 1) / bt > mb)
            return fail(c, SPEC_ERR_SHAPE, "spec_seq_replace: a sequence does not fit max_blocks_per_seq");
    }
    cudaStream_t st = (cudaStream_t)stream;
    char* sb = static_cast<char*>(c->buf.state);
    int32_t* args = at<int32_t>(sb, c->replace_args);
    const size_t Bm = g.max_batch;
    SPEC_CUDA_OK(cudaMemcpyAsync(args, slots_host, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(args + Bm, seq_len_host, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(args + 2 * Bm, last_token_host, (size_t)n * 4, cudaMemcpyHostToDevice, st));
    TRY(launch_kv_replace(n, args, args + Bm, args + 2 * Bm, bt, mb, at<int32_t>(sb, c->seq_len), at<int32_t>(sb, c->last_token),
                          at<int32_t>(sb, c->block_table), at<int32_t>(sb, c->owned), at<int32_t>(sb, c->free_stack),
                          at<int32_t>(sb, c->free_top), at<int32_t>(sb, c->n_emitted), at<int32_t>(sb, c->pending_base),
                          at<int32_t>(sb, c->status), st));
    SPEC_CUDA_OK(cudaStreamSynchronize(st));          // the host lists may be reused by the caller from here on
    return SPEC_OK;
}

extern "C" spec_status spec_seq_compact(spec_ctx* c, int n_keep, const int32_t* keep_slots_host, void* stream)
{
    if (c == nullptr || n_keep < 0 || (n_keep > 0 && keep_slots_host == nullptr)) return SPEC_ERR_INVALID_ARG;
    const spec_config& g = c->cfg;
    if (c->verified) return fail(c, SPEC_ERR_STATE, "spec_seq_compact: a verified step is waiting for its commit");
    if (n_keep > c->B) return fail(c, SPEC_ERR_SHAPE, "spec_seq_compact: more slots listed than sequences running");
    for (int j = 0; j < n_keep; ++j)
        if (keep_slots_host[j] < 0 || keep_slots_host[j] >= c->B || (j > 0 && keep_slots_host[j] <= keep_slots_host[j - 1]))
            return fail(c, SPEC_ERR_INVALID_ARG, "spec_seq_compact: kept slots must be in range and strictly ascending");
    if (n_keep == c->B) return SPEC_OK;                     // ascending and complete: the identity
    const int B_old = c->B, bt = g.kv_block_tokens, mb = g.max_blocks_per_seq;
    const size_t Bm = g.max_batch;
    cudaStream_t st = (cudaStream_t)stream;
    char* sb = static_cast<char*>(c->buf.state);
    char* ws = static_cast<char*>(c->buf.workspace);
    int32_t* args = at<int32_t>(sb, c->replace_args);
    // 1. every slot that is not kept is retired (its blocks go back in slot order, logical block order)
    std::vector<int32_t> dropped, minus(B_old, -1), zeros(B_old, 0);
    for (int b = 0, j = 0; b < B_old; ++b) {
        if (j < n_keep && keep_slots_host[j] == b) { ++j; continue; }
        dropped.push_back(b);
    }
    const int nd = (int)dropped.size();
    SPEC_CUDA_OK(cudaMemcpyAsync(args, dropped.data(), (size_t)nd * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(args + Bm, minus.data(), (size_t)nd * 4, cudaMemcpyHostToDevice, st));
    SPEC_CUDA_OK(cudaMemcpyAsync(args + 2 * Bm, zeros.data(), (size_t)nd * 4, cudaMemcpyHostToDevice, st));
    TRY(launch_kv_replace(nd, args, args + Bm, args + 2 * Bm, bt, mb, at<int32_t>(sb, c->seq_len), at<int32_t>(sb, c->last_token),
                          at<int32_t>(sb, c->block_table), at<int32_t>(sb, c->owned), at<int32_t>(sb, c->free_stack),
                          at<int32_t>(sb, c->free_top), at<int32_t>(sb, c->n_emitted), at<int32_t>(sb, c->pending_base),
                          at<int32_t>(sb, c->status), st));
    // 2. per-slot state moves to the front
    SPEC_CUDA_OK(cudaMemcpyAsync(args, keep_slots_host, (size_t)n_keep * 4, cudaMemcpyHostToDevice, st));
    const int R = c->k_last >= 0 ? c->k_last + 1 : 1;
    const bool ngram = g.draft_kind == SPEC_DRAFT_NGRAM;
    TRY(launch_seq_compact(n_keep, B_old, args, mb, R, ngram ? mb * bt : 0, at<int32_t>(sb, c->seq_len), at<int32_t>(sb, c->last_token),
                           at<int32_t>(sb, c->owned), at<int32_t>(sb, c->pending_base), at<int32_t>(sb, c->n_emitted),
                           at<int32_t>(sb, c->block_table), at<int32_t>(sb, c->out_tokens), at<float>(sb, c->out_logp),
                           ngram ? at<int32_t>(sb, c->history) : nullptr, st));
    // 3. what the draft head absorbs from the last verify (EAGLE-3: the tapped hidden states; MTP: the last-layer residual),
    //    row blocks of R per slot; permuted through the logits buffer, which the next verify overwrites anyway
    if (c->have_pending && c->k_last >= 0 && n_keep > 0) {
        const size_t es = g.dtype == SPEC_DTYPE_F32 ? 4 : 2;
        void* tmp = ws + c->logits.off;
        if (g.draft_kind == SPEC_DRAFT_EAGLE3) {
            const size_t row = (size_t)g.n_taps * g.d_model * es;
            TRY(launch_permute_rows(n_keep, R, row, args, ws + c->taps.off, tmp, st));
            SPEC_CUDA_OK(cudaMemcpyAsync(ws + c->taps.off, tmp, (size_t)n_keep * R * row, cudaMemcpyDeviceToDevice, st));
        } else if (g.draft_kind == SPEC_DRAFT_MTP) {
            const size_t row = (size_t)g.d_model * 4;
            TRY(launch_permute_rows(n_keep, R, row, args, ws + c->x.off, tmp, st));
            SPEC_CUDA_OK(cudaMemcpyAsync(ws + c->x.off, tmp, (size_t)n_keep * R * row, cudaMemcpyDeviceToDevice, st));
        }
    }
    SPEC_CUDA_OK(cudaStreamSynchronize(st));          // the host lists go out of scope here
    c->B = n_keep;
    return SPEC_OK;
}

extern "C" spec_status spec_verify(spec_ctx* c, int k, const int32_t* draft_tokens, void* stream)
{
    if (c == nullptr) return SPEC_ERR_INVALID_ARG;
    const spec_config& g = c->cfg;
    if (k < 0 || k > g.k_max) return fail(c, SPEC_ERR_SHAPE, "spec_verify: k outside 0..k_max");
    if (k > 0 && draft_tokens == nullptr && g.draft_kind == SPEC_DRAFT_NONE)
        return fail(c, SPEC_ERR_INVALID_ARG, "spec_verify: draft_kind NONE needs draft_tokens");
    cudaStream_t st = (cudaStream_t)stream;
    const int B = c->B, R = k + 1, M = B * R, d = g.d_model, dt = g.dtype;
    if (B == 0) { c->k_last = k; c->verified = true; return SPEC_OK; }
    ScratchScope scratch_scope(c);
    void* ws = c->buf.workspace;
    char* sb = static_cast<char*>(c->buf.state);
    int32_t* status = at<int32_t>(sb, c->status);
    int32_t* seq_len = at<int32_t>(sb, c->seq_len);
    TRY(launch_kv_reserve(B, k, g.kv_block_tokens, g.max_blocks_per_seq, seq_len, at<int32_t>(sb, c->block_table), at<int32_t>(sb, c->owned),
                          at<int32_t>(sb, c->free_stack), at<int32_t>(sb, c->free_top), status, st));
    StepRows rows{at<int32_t>(ws, c->tokens_in), at<int32_t>(ws, c->pos)};
    const int32_t* dtok = draft_tokens ? draft_tokens : at<int32_t>(sb, c->draft_tokens);
    const int dstride = draft_tokens ? k : (g.k_max > 0 ? g.k_max : 1);
    TRY(launch_verify_rows(B, R, seq_len, at<int32_t>(sb, c->last_token), dtok, dstride, g.vocab, rows, status, st));
    float* x = at<float>(ws, c->x);
    TRY(launch_rope_table(M, g.head_dim, g.rope_theta, rows.pos, at<float>(ws, c->rope), st));
    TRY(launch_embed(M, d, at(c->buf.weights, c->embed), dt, rows.token, x, st));
    const int tapw = g.n_taps * d;
    if (has_tap(g, 0)) TRY(launch_copy_rows_f32_to(M, d, x, at(ws, c->taps), tapw, tap_slot(g, 0) * d, dt, st));
    for (int l = 0; l < g.n_layers; ++l) {
        const LayerPtrs W = layer_ptrs(c->buf.weights, c->layers[l]);
        const bool w8 = g.weight_dtype == SPEC_W_E4M3;       // 8-bit projections: the layer body norms and quantises x itself
        if (!w8) TRY(launch_rmsnorm(M, d, x, W.attn_norm, g.rms_eps, at(ws, c->h), d, 0, dt, st));
        const int pool = l % g.kv_layer_pools;
        char* kp = static_cast<char*>(c->buf.kv) + (size_t)pool * 2 * c->kv_pool_bytes;
        TRY(run_layer_body(*c, W, g.d_ffn, x, w8 ? nullptr : at(ws, c->h), d, B, R, rows.pos, kp, kp + c->kv_pool_bytes, l, st));
        if (has_tap(g, l + 1)) TRY(launch_copy_rows_f32_to(M, d, x, at(ws, c->taps), tapw, tap_slot(g, l + 1) * d, dt, st));
    }
    if (g.weight_dtype != SPEC_W_E4M3) TRY(launch_rmsnorm(M, d, x, at<const float>(c->buf.weights, c->final_norm), g.rms_eps, at(ws, c->h), d, 0, dt, st));
    // LM head with the row statistics taken in its epilogue; shapes the tile kernel does not take go the two-pass way
    spec_status fused = SPEC_ERR_UNSUPPORTED;
    if (g.weight_dtype == SPEC_W_E4M3) {
        unsigned char* a8 = at<unsigned char>(ws, c->a8) + (kActSlots - 1) * (c->a8.bytes / kActSlots);
        float* a8s = at<float>(ws, c->a8_scale) + (kActSlots - 1) * (c->a8_scale.bytes / kActSlots / 4);
        TRY(launch_rmsnorm_quantize(M, d, x, at<const float>(c->buf.weights, c->final_norm), g.rms_eps, a8, a8s, st));
        Timed t__(*c, CLS_GEMM, st);
        fused = launch_gemm8_tc(M, g.vocab, d, a8, a8s, at(c->buf.weights, c->lm_head), at<const float>(c->buf.weights, c->lm_head_s),
                                at(ws, c->logits), g.vocab, SPEC_DTYPE_F32, 0, g.temperature, at<float>(ws, c->splitk), c->splitk.bytes,
                                at<float>(ws, c->row_stats), 1, at<int32_t>(sb, c->status), st);
        if (fused == SPEC_ERR_UNSUPPORTED) {                  // logits are written; only the statistics still need their pass
            cudaGetLastError();
            fused = launch_softmax_rows(M, g.vocab, at<float>(ws, c->logits), (size_t)g.vocab, g.temperature, at<float>(ws, c->row_stats), 1,
                                        nullptr, st);
        }
    } else {
        Timed t__(*c, CLS_GEMM, st);
        fused = launch_gemm_lm_head_stats(M, g.vocab, d, at(ws, c->h), d, at(c->buf.weights, c->lm_head), at<float>(ws, c->logits), g.vocab, dt,
                                          g.temperature, at<float>(ws, c->splitk), c->splitk.bytes, at<float>(ws, c->row_stats), 1,
                                          at<int32_t>(sb, c->status), st);
    }
    if (fused == SPEC_ERR_UNSUPPORTED) {
        TIMED(*c, CLS_GEMM, launch_gemm(M, g.vocab, d, at(ws, c->h), d, at(c->buf.weights, c->lm_head), at(ws, c->logits), g.vocab, dt,
                                        SPEC_DTYPE_F32, 0, st));
        TIMED(*c, CLS_SAMPLE, launch_softmax_rows(M, g.vocab, at<float>(ws, c->logits), (size_t)g.vocab, g.temperature,
                                                  at<float>(ws, c->row_stats), 1, nullptr, st));
    } else {
        TRY(fused);
    }
    c->k_last = k;
    c->verified = true;
    return SPEC_OK;
}

extern "C" spec_status spec_reject_sample(spec_ctx* c, int k, const float* draft_logits, void* stream)
{
    if (c == nullptr) return SPEC_ERR_INVALID_ARG;
    const spec_config& g = c->cfg;
    if (!c->verified || k != c->k_last) return fail(c, SPEC_ERR_STATE, "spec_reject_sample: no verify with this k since the last commit");
    cudaStream_t st = (cudaStream_t)stream;
    const int B = c->B;
    if (B == 0) return SPEC_OK;
    void* ws = c->buf.workspace;
    char* sb = static_cast<char*>(c->buf.state);
    // no sampled draft and no draft logits given: the drafts are deterministic (n-gram lookup, greedy head), q = one-hot(d)
    const bool has_head = (g.draft_kind == SPEC_DRAFT_EAGLE3 || g.draft_kind == SPEC_DRAFT_MTP) && !g.draft_greedy;
    const float* ql = draft_logits ? draft_logits : (has_head ? at<float>(ws, c->draft_logits) : nullptr);
    float* qs = at<float>(ws, c->draft_row_stats);
    if (draft_logits != nullptr && k > 0)
        TRY(launch_softmax_rows(B * k, g.vocab, ql, (size_t)g.vocab, g.temperature, qs, 1, nullptr, st));
    // draft tokens: those the verify used (rows 1..k of its token list), so an external draft stays consistent
    // a draft head with its own smaller vocabulary: q rows are draft_vocab wide and looked up through the target-to-draft map
    const bool mapped = draft_logits == nullptr && has_head && g.draft_vocab != 0;
    TIMED(*c, CLS_SAMPLE, launch_reject_sample(true, B, k, g.vocab, at<float>(ws, c->logits), at<float>(ws, c->row_stats), ql, qs,
                                               mapped ? g.draft_vocab : g.vocab, mapped ? at<int32_t>(ws, c->t2d) : nullptr,
                                               at<int32_t>(ws, c->tokens_in) + 1, k + 1, g.temperature, g.seed,
                                               at<uint32_t>(sb, c->step), 0, at<int32_t>(sb, c->out_tokens),
                                               at<int32_t>(sb, c->n_emitted), at<int32_t>(sb, c->status), at<float>(sb, c->out_logp), st));
    return SPEC_OK;
}

extern "C" spec_status spec_kv_commit(spec_ctx* c, const int32_t* force_n, const int32_t* force_token, void* stream)
{
    if (c == nullptr || (force_n == nullptr) != (force_token == nullptr)) return SPEC_ERR_INVALID_ARG;
    if (!c->verified) return fail(c, SPEC_ERR_STATE, "spec_kv_commit: nothing verified since the last commit");
    const spec_config& g = c->cfg;
    char* sb = static_cast<char*>(c->buf.state);
    CommitArgs a{};
    a.B = c->B; a.k = c->k_last; a.block_tokens = g.kv_block_tokens; a.max_blocks = g.max_blocks_per_seq;
    a.force_n = force_n; a.force_token = force_token;
    a.verify_tokens = at<int32_t>(c->buf.workspace, c->tokens_in);
    a.n_emitted = at<int32_t>(sb, c->n_emitted);
    a.out_tokens = at<int32_t>(sb, c->out_tokens);
    a.seq_len = at<int32_t>(sb, c->seq_len);
    a.last_token = at<int32_t>(sb, c->last_token);
    a.block_table = at<int32_t>(sb, c->block_table);
    a.owned = at<int32_t>(sb, c->owned);
    a.free_stack = at<int32_t>(sb, c->free_stack);
    a.free_top = at<int32_t>(sb, c->free_top);
    a.pending_base = at<int32_t>(sb, c->pending_base);
    a.history = c->history.bytes ? at<int32_t>(sb, c->history) : nullptr;
    a.max_hist = g.max_blocks_per_seq * g.kv_block_tokens;
    a.step = at<uint32_t>(sb, c->step);
    a.counters = at<long long>(sb, c->counters);
    a.status = at<int32_t>(sb, c->status);
    TRY(launch_kv_commit(a, (cudaStream_t)stream));
    c->verified = false;
    c->have_pending = true;
    return SPEC_OK;
}

extern "C" spec_status spec_draft(spec_ctx* c, int k, void* stream)
{
    if (c == nullptr) return SPEC_ERR_INVALID_ARG;
    const spec_config& g = c->cfg;
    if (g.draft_kind == SPEC_DRAFT_NONE) return fail(c, SPEC_ERR_STATE, "spec_draft: the context has no draft head");
    if (g.draft_kind == SPEC_DRAFT_NGRAM) {
        if (c->verified) return fail(c, SPEC_ERR_STATE, "spec_draft: a verified step is waiting for its commit");
        if (k < 1 || k > g.k_max) return fail(c, SPEC_ERR_SHAPE, "spec_draft: k outside 1..k_max");
        char* sbn = static_cast<char*>(c->buf.state);
        return launch_ngram_draft(c->B, k, g.ngram_n, at<int32_t>(sbn, c->history), g.max_blocks_per_seq * g.kv_block_tokens,
                                  at<int32_t>(sbn, c->seq_len), at<int32_t>(sbn, c->last_token), at<int32_t>(sbn, c->draft_tokens),
                                  g.k_max, (cudaStream_t)stream);
    }
    if (!c->have_pending) return fail(c, SPEC_ERR_STATE, "spec_draft: no committed step to draft from (run one plain decode step first)");
    if (c->verified) return fail(c, SPEC_ERR_STATE, "spec_draft: a verified step is waiting for its commit");
    if (k < 1 || k > g.k_max) return fail(c, SPEC_ERR_SHAPE, "spec_draft: k outside 1..k_max");
    cudaStream_t st = (cudaStream_t)stream;
    const int B = c->B, d = g.d_model, dt = g.dtype, V = g.vocab;
    if (B == 0) return SPEC_OK;
    ScratchScope scratch_scope(c);
    void* ws = c->buf.workspace;
    void* dw = c->buf.draft_weights;
    char* sb = static_cast<char*>(c->buf.state);
    int32_t* status = at<int32_t>(sb, c->status);
    int32_t* seq_len = at<int32_t>(sb, c->seq_len);
    const bool eagle = g.draft_kind == SPEC_DRAFT_EAGLE3;
    TRY(launch_kv_reserve(B, k, g.kv_block_tokens, g.max_blocks_per_seq, seq_len, at<int32_t>(sb, c->block_table), at<int32_t>(sb, c->owned),
                          at<int32_t>(sb, c->free_stack), at<int32_t>(sb, c->free_top), status, st));
    const LayerPtrs W = layer_ptrs(dw, c->d_layer);
    char* kp = static_cast<char*>(c->buf.draft_kv);
    char* vp = kp + c->kv_pool_bytes;
    int32_t* tok = at<int32_t>(ws, c->d_tok);
    int32_t* pos = at<int32_t>(ws, c->d_pos);
    float* dg = at<float>(ws, c->dg);
    float* dx = at<float>(ws, c->dx);
    float* hid = at<float>(ws, c->d_hidden);
    float* dlog = at<float>(ws, c->draft_logits);
    float* dstats = at<float>(ws, c->draft_row_stats);
    int32_t* dtoks = at<int32_t>(sb, c->draft_tokens);
    const int kstride = g.k_max;
    const bool mapped = eagle && g.draft_vocab != 0;
    const int Vd = mapped ? g.draft_vocab : V;
    int32_t* dred = mapped ? at<int32_t>(ws, c->draft_red) : nullptr;
    if (mapped) TRY(launch_build_t2d(V, Vd, at<const int32_t>(dw, c->d_d2t), at<int32_t>(ws, c->t2d), st));

    for (int j = 0; j < k; ++j) {
        const int R = j == 0 ? c->k_last + 1 : 1;
        const int M = B * R;
        float* res = j == 0 ? dg : hid;                 // residual stream of this pass
        if (j == 0) draft_rows0_kernel<<<(M + 255) / 256, 256, 0, st>>>(B, R, at<int32_t>(sb, c->n_emitted), at<int32_t>(sb, c->pending_base),
                                                                        at<int32_t>(sb, c->out_tokens), tok, pos);
        else        draft_rows_kernel<<<(B + 255) / 256, 256, 0, st>>>(B, j, seq_len, at<int32_t>(sb, c->n_emitted), dtoks, kstride, tok, pos);
        TRY(launch_status());
        TRY(launch_rope_table(M, g.head_dim, g.rope_theta, pos, at<float>(ws, c->rope), st));
        TRY(launch_embed(M, d, at(c->buf.weights, c->embed), dt, tok, dx, st));
        if (eagle) {
            // a = concat(norm_e(e), norm_g(g)); g = W_fc taps (true slots) or the head's previous output
            if (j == 0) TRY(launch_gemm(M, d, g.n_taps * d, at(ws, c->taps), g.n_taps * d, at(dw, c->d_wfc), dg, d, dt, SPEC_DTYPE_F32, 0, st));
            TRY(launch_rmsnorm(M, d, dx, at<const float>(dw, c->d_norm_e), g.rms_eps, at(ws, c->h), 2 * d, 0, dt, st));
            TRY(launch_rmsnorm(M, d, res, at<const float>(dw, c->d_norm_g), g.rms_eps, at(ws, c->h), 2 * d, d, dt, st));
            TRY(run_layer_body(*c, W, g.draft_d_ffn, res, at(ws, c->h), 2 * d, B, R, pos, kp, vp, 0, st));
        } else {
            // h0 = W_proj concat(norm_g(g), norm_e(e)); g = the target's last-layer residual or the head's previous output
            const float* gsrc = j == 0 ? at<float>(ws, c->x) : hid;
            TRY(launch_rmsnorm(M, d, gsrc, at<const float>(dw, c->d_norm_g), g.rms_eps, at(ws, c->h), 2 * d, 0, dt, st));
            TRY(launch_rmsnorm(M, d, dx, at<const float>(dw, c->d_norm_e), g.rms_eps, at(ws, c->h), 2 * d, d, dt, st));
            TRY(launch_gemm(M, d, 2 * d, at(ws, c->h), 2 * d, at(dw, c->d_wproj), res, d, dt, SPEC_DTYPE_F32, 0, st));
            TRY(launch_rmsnorm(M, d, res, W.attn_norm, g.rms_eps, at(ws, c->h), d, 0, dt, st));
            TRY(run_layer_body(*c, W, g.draft_d_ffn, res, at(ws, c->h), d, B, R, pos, kp, vp, 0, st));
        }
        if (j == 0) TRY(launch_gather_last_rows(B, R, d, dg, at<int32_t>(sb, c->n_emitted), hid, st));
        // logits of this slot, their statistics, and the draft token d_{j+1} ~ q_{j+1} (stream-1 uniform, slot j)
        const float* nf = eagle ? at<const float>(dw, c->d_norm_f) : at<const float>(c->buf.weights, c->final_norm);
        const void* lm = eagle ? at<const void>(dw, c->d_lm_head) : at<const void>(c->buf.weights, c->lm_head);
        const bool lm8 = !eagle && g.weight_dtype == SPEC_W_E4M3;    // the MTP head scores with the target's (8-bit) LM head
        spec_status fused = SPEC_ERR_UNSUPPORTED;
        if (lm8) {
            unsigned char* a8 = at<unsigned char>(ws, c->a8) + (kActSlots - 1) * (c->a8.bytes / kActSlots);
            float* a8s = at<float>(ws, c->a8_scale) + (kActSlots - 1) * (c->a8_scale.bytes / kActSlots / 4);
            TRY(launch_rmsnorm_quantize(B, d, hid, nf, g.rms_eps, a8, a8s, st));
            fused = launch_gemm8_tc(B, Vd, d, a8, a8s, lm, at<const float>(c->buf.weights, c->lm_head_s), dlog + (size_t)j * Vd, k * Vd,
                                    SPEC_DTYPE_F32, 0, g.temperature, g.draft_greedy ? nullptr : at<float>(ws, c->splitk), c->splitk.bytes,
                                    dstats + 2 * j, k, status, st);
            if (fused != SPEC_OK && fused != SPEC_ERR_UNSUPPORTED) return fused;
            if (g.draft_greedy) fused = SPEC_ERR_UNSUPPORTED;        // no statistics wanted; the logits are written
        } else {
            TRY(launch_rmsnorm(B, d, hid, nf, g.rms_eps, at(ws, c->h), d, 0, dt, st));
        }
        if (!g.draft_greedy && !lm8)
            fused = launch_gemm_lm_head_stats(B, Vd, d, at(ws, c->h), d, lm, dlog + (size_t)j * Vd, k * Vd, dt, g.temperature,
                                              at<float>(ws, c->splitk), c->splitk.bytes, dstats + 2 * j, k, status, st);
        if (fused == SPEC_ERR_UNSUPPORTED) {
            if (!lm8) TRY(launch_gemm(B, Vd, d, at(ws, c->h), d, lm, dlog + (size_t)j * Vd, k * Vd, dt, SPEC_DTYPE_F32, 0, st));
        } else {
            TRY(fused);
        }
        int32_t* tok_out = mapped ? dred + j : dtoks + j;          // reduced ids first when the head has its own vocabulary
        if (g.draft_greedy) {
            TRY(launch_argmax_rows(B, Vd, dlog + (size_t)j * Vd, (size_t)k * Vd, tok_out, kstride, st));
        } else {
            if (fused == SPEC_ERR_UNSUPPORTED)
                TRY(launch_softmax_rows(B, Vd, dlog + (size_t)j * Vd, (size_t)k * Vd, g.temperature, dstats + 2 * j, k, nullptr, st));
            TRY(launch_sample_logits(B, Vd, dlog + (size_t)j * Vd, (size_t)k * Vd, dstats + 2 * j, k, g.temperature, g.seed,
                                     at<uint32_t>(sb, c->step), (uint32_t)j, 1u, tok_out, kstride, status, st));
        }
        if (mapped) TRY(launch_map_tokens(B, dred + j, kstride, at<const int32_t>(dw, c->d_d2t), dtoks + j, kstride, st));
    }
    return SPEC_OK;
}

extern "C" spec_status spec_get_status(spec_ctx* c, spec_step_report* out, void* stream)
{
    if (c == nullptr || out == nullptr) return SPEC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    SPEC_CUDA_OK(cudaStreamSynchronize(st));
    char* sb = static_cast<char*>(c->buf.state);
    int32_t status[4];
    long long counters[3];
    SPEC_CUDA_OK(cudaMemcpy(status, sb + c->status.off, sizeof(status), cudaMemcpyDeviceToHost));
    SPEC_CUDA_OK(cudaMemcpy(counters, sb + c->counters.off, sizeof(counters), cudaMemcpyDeviceToHost));
    out->device_status = status[0];
    out->device_detail = status[1];
    out->steps = counters[0];
    out->emitted_tokens = counters[1];
    out->accepted_drafts = counters[2];
    return SPEC_OK;
}

spec::GemmScratch& spec::gemm_scratch()
{
    static thread_local GemmScratch s;
    return s;
}

std::atomic<long long>& spec::launch_counter()
{
    static std::atomic<long long> n{0};
    return n;
}

extern "C" int64_t spec_launch_count(void) { return (int64_t)spec::launch_counter().load(std::memory_order_relaxed); }

extern "C" spec_status spec_set_timing(spec_ctx* c, uint32_t mask)
{
    if (c == nullptr || mask > 15u) return SPEC_ERR_INVALID_ARG;
    if (mask != 0 && c->ev.empty()) {
        c->ev.resize(2 * kMaxTimedPasses);
        for (auto& e : c->ev) if (cudaEventCreate(&e) != cudaSuccess) return SPEC_ERR_CUDA;
        c->ev_cls.reserve(kMaxTimedPasses);
    }
    c->timing_mask = mask;
    return SPEC_OK;
}

extern "C" spec_status spec_get_timing(spec_ctx* c, spec_timing* out, void* stream)
{
    if (c == nullptr || out == nullptr) return SPEC_ERR_INVALID_ARG;
    SPEC_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
    *out = spec_timing{};
    for (size_t i = 0; i < c->ev_cls.size(); ++i) {
        float ms = 0.f;
        SPEC_CUDA_OK(cudaEventElapsedTime(&ms, c->ev[2 * i], c->ev[2 * i + 1]));
        out->ms[c->ev_cls[i]] += ms;
        out->passes[c->ev_cls[i]] += 1;
    }
    out->dropped = c->ev_dropped;
    c->ev_cls.clear();
    c->ev_dropped = 0;
    return SPEC_OK;
}
