// Expert-parallel mixture-of-experts MLP: the experts of one block are spread over ep_size GPUs of an NVLink domain
// (the paper's 235B-A22B configuration, Section 5.1), every GPU routes its own rows.  Rows travel by loads from peer
// memory inside two kernels: ep_pull_kernel gathers the rows routed to the local experts straight out of the other ranks'
// windows into the local grouped-GEMM operand (dispatch + permutation in one pass), ep_combine_kernel fetches each token's
// expert outputs from their owners and accumulates them (return + weighted sum in one pass).  Nothing is pushed and no
// kernel waits on another rank; the three phases are separated by the caller's barriers.
//
// Everything is deterministic: receive order = (local expert, source rank, the source's entry order), the combination adds
// slots 0..top_k-1 in turn with fused multiply-adds exactly as the single-GPU block does, so a token's result does not
// depend on ep_size.
#include "ops.cuh"

#include <cuda.h>
#include <cstring>

namespace spec {
namespace {

constexpr int kMaxRanks = 16;
constexpr int kMaxExperts = 256;

struct Peers { unsigned char* win[kMaxRanks]; };

// Byte offsets inside a window / the scratch.  Every piece starts on a 256-byte boundary.
struct EpLayout {
    size_t hdr, h, h8, h8_scale, ids, wts, rank, src_of, counts, offsets, recv_off, y, window_bytes;
    size_t logits, a_perm, act, grp_counts, grp_offsets, a8, a8_scale, scratch_bytes;
};
enum { HDR_M = 0, HDR_RECV_TOTAL = 1, HDR_ROWS8 = 2 };   // HDR_ROWS8: 1 when the rows were also published as e4m3 codes

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

EpLayout make_layout(const spec_ep_config& c)
{
    EpLayout l{};
    const size_t n = (size_t)c.max_rows * c.top_k, E = c.n_experts, cap = c.cap_rows;
    size_t at = 0;
    auto take = [&](size_t bytes) { const size_t o = at; at = up256(at + bytes); return o; };
    l.hdr = take(64 * 4);
    l.h = take((size_t)c.max_rows * c.d * 2);
    l.h8 = take((size_t)c.max_rows * c.d);                   // the same rows as e4m3 codes + one scale each (spec_ep_route_e4m3)
    l.h8_scale = take((size_t)c.max_rows * 4);
    l.ids = take(n * 4);
    l.wts = take(n * 4);
    l.rank = take(n * 4);
    l.src_of = take(n * 4);
    l.counts = take(E * 4);
    l.offsets = take(E * 4);
    l.recv_off = take(E * 4);
    l.y = take(cap * c.d * 4);
    l.window_bytes = at;
    at = 0;
    l.logits = take((size_t)c.max_rows * E * 4);
    l.a_perm = take((cap + 128) * c.d * 2);                  // + one tile of rows for the last group's TMA box
    l.act = take((cap + 128) * c.d_expert_ffn * 2);
    l.grp_counts = take(E * 4);
    l.grp_offsets = take(E * 4);
    // 8-bit experts (spec_ep_experts_e4m3): the received rows, then the SwiGLU outputs, as e4m3 codes with one scale per row
    l.a8 = take((cap + 128) * (size_t)(c.d > c.d_expert_ffn ? c.d : c.d_expert_ffn));
    l.a8_scale = take((cap + 128) * 4);
    l.scratch_bytes = at;
    return l;
}

spec_status check(const spec_ep_config* c)
{
    if (c == nullptr) return SPEC_ERR_INVALID_ARG;
    if (c->ep_size < 1 || c->ep_rank < 0 || c->ep_rank >= c->ep_size || c->max_rows < 0 || c->cap_rows < 0) return SPEC_ERR_INVALID_ARG;
    if (c->ep_size > kMaxRanks) return SPEC_ERR_UNSUPPORTED;
    if (c->n_experts < 1 || c->n_experts > kMaxExperts || c->n_experts % c->ep_size != 0) return SPEC_ERR_SHAPE;
    if (c->top_k < 1 || c->top_k > 32 || c->top_k > c->n_experts) return SPEC_ERR_SHAPE;
    if (c->d < 64 || c->d % 64 != 0 || c->d_expert_ffn < 64 || c->d_expert_ffn % 64 != 0 || (2 * c->d_expert_ffn) % 256 != 0) return SPEC_ERR_SHAPE;
    if (c->d % 256 != 0) return SPEC_ERR_SHAPE;             // the down projection's N
    return SPEC_OK;
}

// After the ranking pass: offsets = exclusive scan of counts, src_of[offsets[e] + rank[i]] = i for every entry i (the
// rank's entries listed expert by expert, each expert's in entry order), header M.
__global__ void __launch_bounds__(256) ep_publish_kernel(int M, int E, int top_k, const int32_t* __restrict__ ids,
                                                         const int32_t* __restrict__ rank, const int32_t* __restrict__ counts,
                                                         int32_t* __restrict__ offsets, int32_t* __restrict__ src_of,
                                                         int32_t* __restrict__ hdr, int rows8)
{
    __shared__ int s_off[kMaxExperts];
    if (threadIdx.x == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) { s_off[e] = run; run += counts[e]; }
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        for (int e = threadIdx.x; e < E; e += blockDim.x) offsets[e] = s_off[e];
        if (threadIdx.x == 0) { hdr[HDR_M] = M; hdr[HDR_ROWS8] = rows8; }
    }
    const int n = M * top_k;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        src_of[s_off[ids[i]] + rank[i]] = i;
}

// Destination side of the dispatch.  Run u = (local expert el, source s), u = el * R + s, holds the entries that source s
// routed to expert e0 + el; the runs are laid out back to back in u order.  Every CTA rebuilds the small run table from
// the sources' published counts, then the CTAs copy rows: one row per CTA per turn, 16 bytes per thread per load.
__global__ void __launch_bounds__(256) ep_pull_kernel(Peers peers, EpLayout L, int R, int me, int E, int top_k, int d, int cap_rows,
                                                      __nv_bfloat16* __restrict__ a_perm, int32_t* __restrict__ grp_counts,
                                                      int32_t* __restrict__ grp_offsets, int32_t* status,
                                                      unsigned char* __restrict__ a8, float* __restrict__ a8_scale)
{
    // a8 != nullptr: pull the rows as e4m3 codes + scale (what spec_ep_route_e4m3 published) instead of the 16-bit rows
    __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts + 1], s_src_start[kMaxExperts];
    const int per = E / R, e0 = me * per;
    for (int u = threadIdx.x; u < E; u += blockDim.x) {
        const int el = u / R, s = u % R;
        const int32_t* counts = reinterpret_cast<const int32_t*>(peers.win[s] + L.counts);
        const int32_t* offsets = reinterpret_cast<const int32_t*>(peers.win[s] + L.offsets);
        s_cnt[u] = counts[e0 + el];
        s_src_start[u] = offsets[e0 + el];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int u = 0; u < E; ++u) { s_off[u] = run; run += s_cnt[u]; }
        s_off[E] = run;
    }
    __syncthreads();
    const int total = s_off[E];
    if (blockIdx.x == 0) {
        int32_t* own_recv_off = reinterpret_cast<int32_t*>(peers.win[me] + L.recv_off);
        for (int u = threadIdx.x; u < E; u += blockDim.x) own_recv_off[u] = s_off[u];
        for (int el = threadIdx.x; el < per; el += blockDim.x) {
            const int b = min(s_off[el * R], cap_rows), e = min(s_off[(el + 1) * R], cap_rows);
            grp_offsets[el] = b;
            grp_counts[el] = e - b;
        }
        if (threadIdx.x == 0) {
            reinterpret_cast<int32_t*>(peers.win[me] + L.hdr)[HDR_RECV_TOTAL] = total;
            if (total > cap_rows) set_status(status, SPEC_ERR_EP_CAPACITY, total);
            if (a8 != nullptr)                                       // every source must have published codes
                for (int s = 0; s < R; ++s)
                    if (reinterpret_cast<const int32_t*>(peers.win[s] + L.hdr)[HDR_ROWS8] != 1) set_status(status, SPEC_ERR_STATE, s);
        }
    }
    const int rows = min(total, cap_rows);
    for (int t = blockIdx.x; t < rows; t += gridDim.x) {
        // last run u with s_off[u] <= t (empty runs share their start with the next one and are skipped by taking the last)
        int lo = 0, hi = E - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (s_off[mid] <= t) lo = mid; else hi = mid - 1;
        }
        const int u = lo, s = u % R, j = t - s_off[u];
        const int32_t* src_of = reinterpret_cast<const int32_t*>(peers.win[s] + L.src_of);
        const int m = src_of[s_src_start[u] + j] / top_k;
        if (a8 != nullptr) {
            const uint4* src8 = reinterpret_cast<const uint4*>(peers.win[s] + L.h8 + (size_t)m * d);
            uint4* dst8 = reinterpret_cast<uint4*>(a8 + (size_t)t * d);
            for (int c = threadIdx.x; c < d / 16; c += blockDim.x) dst8[c] = src8[c];
            if (threadIdx.x == 0) a8_scale[t] = reinterpret_cast<const float*>(peers.win[s] + L.h8_scale)[m];
            continue;
        }
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(peers.win[s] + L.h) + (size_t)m * d);
        uint4* dst = reinterpret_cast<uint4*>(a_perm + (size_t)t * d);
        for (int c = threadIdx.x; c < d / 8; c += blockDim.x) dst[c] = src[c];
    }
}

// Source side of the return path: token m adds w_j * (row of expert output that owner(e_j) computed for entry (m, j)), j in
// slot order.  The row index is the owner's receive offset of (expert, this rank) plus the entry's rank among this rank's
// entries of that expert.  Loads of up to eight slots are issued together, then added in order.
__global__ void __launch_bounds__(256) ep_combine_kernel(Peers peers, EpLayout L, int R, int me, int E, int top_k, int d, int cap_rows,
                                                         float* __restrict__ x)
{
    __shared__ const float* s_row[32];
    __shared__ float s_w[32];
    const int m = blockIdx.x, per = E / R;
    if (threadIdx.x < top_k) {
        const int i = m * top_k + threadIdx.x;
        const int e = reinterpret_cast<const int32_t*>(peers.win[me] + L.ids)[i];
        const int owner = e / per, el = e % per;
        const int row = reinterpret_cast<const int32_t*>(peers.win[owner] + L.recv_off)[el * R + me] +
                        reinterpret_cast<const int32_t*>(peers.win[me] + L.rank)[i];
        s_row[threadIdx.x] = (row >= 0 && row < cap_rows) ? reinterpret_cast<const float*>(peers.win[owner] + L.y) + (size_t)row * d : nullptr;
        s_w[threadIdx.x] = reinterpret_cast<const float*>(peers.win[me] + L.wts)[i];
    }
    __syncthreads();
    for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
        float4 acc = *reinterpret_cast<const float4*>(x + (size_t)m * d + c);
        for (int j0 = 0; j0 < top_k; j0 += 8) {
            float4 v[8];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                v[jj] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j0 + jj < top_k && s_row[j0 + jj] != nullptr) v[jj] = *reinterpret_cast<const float4*>(s_row[j0 + jj] + c);
            }
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                if (j0 + jj < top_k && s_row[j0 + jj] != nullptr) {
                    const float w = s_w[j0 + jj];
                    acc.x = fmaf(w, v[jj].x, acc.x); acc.y = fmaf(w, v[jj].y, acc.y);
                    acc.z = fmaf(w, v[jj].z, acc.z); acc.w = fmaf(w, v[jj].w, acc.w);
                }
            }
        }
        *reinterpret_cast<float4*>(x + (size_t)m * d + c) = acc;
    }
}

bool fill_peers(const spec_ep_config& c, void* const* peer_windows_host, Peers& p)
{
    for (int r = 0; r < kMaxRanks; ++r) p.win[r] = nullptr;
    for (int r = 0; r < c.ep_size; ++r) {
        if (peer_windows_host[r] == nullptr) return false;
        p.win[r] = static_cast<unsigned char*>(peer_windows_host[r]);
    }
    return true;
}

}  // namespace
}  // namespace spec

using namespace spec;

extern "C" spec_status spec_ep_query_sizes(const spec_ep_config* cfg, spec_ep_sizes* out)
{
    if (out == nullptr) return SPEC_ERR_INVALID_ARG;
    const spec_status s = check(cfg);
    if (s != SPEC_OK) return s;
    const EpLayout l = make_layout(*cfg);
    out->window_bytes = l.window_bytes;
    out->scratch_bytes = l.scratch_bytes;
    return SPEC_OK;
}

extern "C" spec_status spec_ep_tensor(const spec_ep_config* cfg, void* window, void* scratch, int tensor_id, void** dev_ptr, size_t* bytes)
{
    if (dev_ptr == nullptr || bytes == nullptr || window == nullptr || scratch == nullptr) return SPEC_ERR_INVALID_ARG;
    const spec_status s = check(cfg);
    if (s != SPEC_OK) return s;
    const EpLayout l = make_layout(*cfg);
    const size_t n = (size_t)cfg->max_rows * cfg->top_k;
    unsigned char* w = static_cast<unsigned char*>(window);
    switch (tensor_id) {
    case SPEC_EP_T_IDS: *dev_ptr = w + l.ids; *bytes = n * 4; break;
    case SPEC_EP_T_WTS: *dev_ptr = w + l.wts; *bytes = n * 4; break;
    case SPEC_EP_T_COUNTS: *dev_ptr = w + l.counts; *bytes = (size_t)cfg->n_experts * 4; break;
    case SPEC_EP_T_RECV_OFF: *dev_ptr = w + l.recv_off; *bytes = (size_t)cfg->n_experts * 4; break;
    case SPEC_EP_T_RECV_TOTAL: *dev_ptr = w + l.hdr + HDR_RECV_TOTAL * 4; *bytes = 4; break;
    case SPEC_EP_T_EXPERT_OUT: *dev_ptr = w + l.y; *bytes = (size_t)cfg->cap_rows * cfg->d * 4; break;
    case SPEC_EP_T_RECV_ROWS: *dev_ptr = static_cast<unsigned char*>(scratch) + l.a_perm; *bytes = (size_t)cfg->cap_rows * cfg->d * 2; break;
    default: return SPEC_ERR_INVALID_ARG;
    }
    return SPEC_OK;
}

namespace {
spec_status ep_route(const spec_ep_config* cfg, void* window, void* scratch, int M, const void* h, const void* router_w, int rows8, void* stream)
{
    const spec_status s = check(cfg);
    if (s != SPEC_OK) return s;
    if (window == nullptr || scratch == nullptr || router_w == nullptr || M < 0 || (M > 0 && h == nullptr)) return SPEC_ERR_INVALID_ARG;
    if (M > cfg->max_rows) return SPEC_ERR_SHAPE;
    const EpLayout l = make_layout(*cfg);
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char* w = static_cast<unsigned char*>(window);
    unsigned char* sc = static_cast<unsigned char*>(scratch);
    const int E = cfg->n_experts, tk = cfg->top_k, d = cfg->d;
    if (M > 0 && cudaMemcpyAsync(w + l.h, h, (size_t)M * d * 2, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SPEC_ERR_CUDA;
    // always the tensor-core tile kernel, whatever M is: a row's router logits (and with them its mixture weights) must not
    // depend on how many other rows this rank happens to hold, or the block's output would change with ep_size
    spec_status r = gemm_tc_supported(M, E, d, w + l.h, d, router_w, sc + l.logits, E, SPEC_DTYPE_BF16, SPEC_DTYPE_F32)
                        ? launch_gemm_tc(M, E, d, w + l.h, d, router_w, sc + l.logits, E, SPEC_DTYPE_F32, 0, nullptr, st)
                        : launch_gemm(M, E, d, w + l.h, d, router_w, sc + l.logits, E, SPEC_DTYPE_BF16, SPEC_DTYPE_F32, 0, st);
    if (r != SPEC_OK) return r;
    r = launch_moe_route(M, E, tk, reinterpret_cast<const float*>(sc + l.logits), reinterpret_cast<int32_t*>(w + l.ids),
                         reinterpret_cast<float*>(w + l.wts), st);
    if (r != SPEC_OK) return r;
    r = launch_moe_rank(M * tk, E, reinterpret_cast<const int32_t*>(w + l.ids), reinterpret_cast<int32_t*>(w + l.rank),
                        reinterpret_cast<int32_t*>(w + l.counts), st);
    if (r != SPEC_OK) return r;
    const int n = M * tk;
    ep_publish_kernel<<<n > 0 ? (n + 255) / 256 : 1, 256, 0, st>>>(
        M, E, tk, reinterpret_cast<const int32_t*>(w + l.ids), reinterpret_cast<const int32_t*>(w + l.rank),
        reinterpret_cast<const int32_t*>(w + l.counts), reinterpret_cast<int32_t*>(w + l.offsets),
        reinterpret_cast<int32_t*>(w + l.src_of), reinterpret_cast<int32_t*>(w + l.hdr), rows8);
    r = launch_status();
    if (r != SPEC_OK || !rows8 || M == 0) return r;
    // 8-bit dispatch: a row is quantised once, here, and travels as codes + scale (half the bytes of the 16-bit row)
    return launch_quantize_rows(M, d, w + l.h, w + l.h8, reinterpret_cast<float*>(w + l.h8_scale), st);
}
}  // namespace

extern "C" spec_status spec_ep_route(const spec_ep_config* cfg, void* window, void* scratch, int M, const void* h,
                                     const void* router_w, void* stream)
{
    return ep_route(cfg, window, scratch, M, h, router_w, 0, stream);
}

extern "C" spec_status spec_ep_route_e4m3(const spec_ep_config* cfg, void* window, void* scratch, int M, const void* h,
                                          const void* router_w, void* stream)
{
    if (cfg != nullptr && cfg->d % 16 != 0) return SPEC_ERR_SHAPE;
    return ep_route(cfg, window, scratch, M, h, router_w, 1, stream);
}

namespace {
// Shared body of spec_ep_experts and spec_ep_experts_e4m3 (scales != nullptr: 8-bit expert weights).
spec_status ep_experts(const spec_ep_config* cfg, void* const* peer_windows_host, void* scratch, const void* w_gateup, const float* gateup_scale,
                       const void* w_down, const float* down_scale, int32_t* status, void* stream)
{
    const spec_status s = check(cfg);
    if (s != SPEC_OK) return s;
    if (peer_windows_host == nullptr || scratch == nullptr || w_gateup == nullptr || w_down == nullptr) return SPEC_ERR_INVALID_ARG;
    const bool w8 = gateup_scale != nullptr;
    if (w8 && (down_scale == nullptr || cfg->d % 16 != 0 || cfg->d_expert_ffn % 16 != 0)) return SPEC_ERR_INVALID_ARG;
    Peers peers;
    if (!fill_peers(*cfg, peer_windows_host, peers)) return SPEC_ERR_INVALID_ARG;
    const EpLayout l = make_layout(*cfg);
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char* sc = static_cast<unsigned char*>(scratch);
    const int R = cfg->ep_size, me = cfg->ep_rank, E = cfg->n_experts, per = E / R, d = cfg->d, Fe = cfg->d_expert_ffn;
    int32_t* gc = reinterpret_cast<int32_t*>(sc + l.grp_counts);
    int32_t* go = reinterpret_cast<int32_t*>(sc + l.grp_offsets);
    __nv_bfloat16* a_perm = reinterpret_cast<__nv_bfloat16*>(sc + l.a_perm);
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    const long long want = (long long)sms * 8;
    const int grid = (int)(want < cfg->cap_rows ? want : (cfg->cap_rows > 0 ? cfg->cap_rows : 1));
    ep_pull_kernel<<<grid, 256, 0, st>>>(peers, l, R, me, E, cfg->top_k, d, cfg->cap_rows, a_perm, gc, go, status,
                                         w8 ? sc + l.a8 : nullptr, w8 ? reinterpret_cast<float*>(sc + l.a8_scale) : nullptr);
    spec_status r = launch_status();
    if (r != SPEC_OK || cfg->cap_rows == 0) return r;      // capacity 0: the offsets and the status are published, nothing to compute
    const long long most = (long long)R * cfg->max_rows;
    const int max_per_group = (int)(most < cfg->cap_rows ? most : cfg->cap_rows);
    if (w8) {
        // the rows arrived as codes + scale, quantised once at their source: a row gives the same codes on whichever rank its
        // expert lives, and half the bytes cross between ranks
        unsigned char* a8 = sc + l.a8;
        float* a8s = reinterpret_cast<float*>(sc + l.a8_scale);
        const int32_t* n_recv = reinterpret_cast<const int32_t*>(peers.win[me] + l.hdr) + HDR_RECV_TOTAL;
        r = launch_gemm8_grouped(cfg->cap_rows, max_per_group, per, 2 * Fe, d, a8, a8s, w_gateup, gateup_scale, sc + l.act, SPEC_DTYPE_BF16, 1, gc, go,
                                 status, st);
        if (r != SPEC_OK) return r;
        r = launch_quantize_rows(cfg->cap_rows, Fe, sc + l.act, a8, a8s, st, n_recv);
        if (r != SPEC_OK) return r;
        return launch_gemm8_grouped(cfg->cap_rows, max_per_group, per, d, Fe, a8, a8s, w_down, down_scale, peers.win[me] + l.y, SPEC_DTYPE_F32, 0, gc, go,
                                    status, st);
    }
    r = launch_gemm_grouped(cfg->cap_rows, max_per_group, per, 2 * Fe, d, a_perm, w_gateup, sc + l.act, SPEC_DTYPE_BF16, 1, gc, go, status, st);
    if (r != SPEC_OK) return r;
    return launch_gemm_grouped(cfg->cap_rows, max_per_group, per, d, Fe, sc + l.act, w_down, peers.win[me] + l.y, SPEC_DTYPE_F32, 0, gc, go,
                               status, st);
}
}  // namespace

extern "C" spec_status spec_ep_experts(const spec_ep_config* cfg, void* const* peer_windows_host, void* scratch,
                                       const void* w_gateup, const void* w_down, int32_t* status, void* stream)
{
    return ep_experts(cfg, peer_windows_host, scratch, w_gateup, nullptr, w_down, nullptr, status, stream);
}

extern "C" spec_status spec_ep_experts_e4m3(const spec_ep_config* cfg, void* const* peer_windows_host, void* scratch,
                                            const void* w_gateup, const float* w_gateup_scale, const void* w_down,
                                            const float* w_down_scale, int32_t* status, void* stream)
{
    if (w_gateup_scale == nullptr || w_down_scale == nullptr) return SPEC_ERR_INVALID_ARG;
    return ep_experts(cfg, peer_windows_host, scratch, w_gateup, w_gateup_scale, w_down, w_down_scale, status, stream);
}

extern "C" spec_status spec_ep_combine(const spec_ep_config* cfg, void* const* peer_windows_host, int M, float* x, void* stream)
{
    const spec_status s = check(cfg);
    if (s != SPEC_OK) return s;
    if (peer_windows_host == nullptr || M < 0 || (M > 0 && x == nullptr)) return SPEC_ERR_INVALID_ARG;
    if (M > cfg->max_rows) return SPEC_ERR_SHAPE;
    Peers peers;
    if (!fill_peers(*cfg, peer_windows_host, peers)) return SPEC_ERR_INVALID_ARG;
    if (M == 0) return SPEC_OK;
    const EpLayout l = make_layout(*cfg);
    ep_combine_kernel<<<M, 256, 0, (cudaStream_t)stream>>>(peers, l, cfg->ep_size, cfg->ep_rank, cfg->n_experts, cfg->top_k, cfg->d,
                                                           cfg->cap_rows, x);
    return launch_status();
}

extern "C" spec_status spec_ipc_export(void* dev_ptr, unsigned char* handle_host, uint64_t* offset_host)
{
    if (dev_ptr == nullptr || handle_host == nullptr || offset_host == nullptr) return SPEC_ERR_INVALID_ARG;
    static_assert(sizeof(cudaIpcMemHandle_t) == 64, "handle size of the C ABI");
    cudaIpcMemHandle_t h;
    if (cudaIpcGetMemHandle(&h, dev_ptr) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    typedef CUresult (*RangeFn)(CUdeviceptr*, size_t*, CUdeviceptr);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &q) != cudaSuccess || fn == nullptr) return SPEC_ERR_CUDA;
    CUdeviceptr base = 0;
    size_t size = 0;
    if (reinterpret_cast<RangeFn>(fn)(&base, &size, (CUdeviceptr)(uintptr_t)dev_ptr) != CUDA_SUCCESS) return SPEC_ERR_CUDA;
    memcpy(handle_host, &h, 64);
    *offset_host = (uint64_t)((uintptr_t)dev_ptr - (uintptr_t)base);
    return SPEC_OK;
}

extern "C" spec_status spec_ipc_open(const unsigned char* handle_host, void** base_dev_ptr)
{
    if (handle_host == nullptr || base_dev_ptr == nullptr) return SPEC_ERR_INVALID_ARG;
    cudaIpcMemHandle_t h;
    memcpy(&h, handle_host, 64);
    if (cudaIpcOpenMemHandle(base_dev_ptr, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    return SPEC_OK;
}

extern "C" spec_status spec_ipc_close(void* base_dev_ptr)
{
    if (base_dev_ptr == nullptr) return SPEC_ERR_INVALID_ARG;
    if (cudaIpcCloseMemHandle(base_dev_ptr) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    return SPEC_OK;
}
