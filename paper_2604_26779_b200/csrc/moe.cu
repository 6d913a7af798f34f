// Mixture-of-experts MLP of a decoder layer: router softmax + top-k, token permutation into expert order, and the
// weighted combination of the experts' outputs.  (The expert projections themselves are the grouped tcgen05 GEMM.)
// Order is deterministic: within an expert, rows are sorted by (token, slot); the combination adds slots 0..k-1 in turn.
#include "ops.cuh"

namespace spec {
namespace {

// One warp per row: top_k largest router logits (ties: lower expert index), softmax weights renormalised over them.
__global__ void __launch_bounds__(128) moe_route_kernel(int M, int E, int top_k, const float* __restrict__ logits,
                                                        int32_t* __restrict__ ids, float* __restrict__ wts)
{
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= M) return;
    const float* l = logits + (size_t)row * E;
    constexpr int kMaxPer = 8;                                   // up to 256 experts
    float v[kMaxPer];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < kMaxPer; ++i) {
        const int e = lane + 32 * i;
        v[i] = e < E ? l[e] : -INFINITY;
        mx = fmaxf(mx, v[i]);
    }
    mx = warp_max(mx);
    float z = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxPer; ++i) z += (lane + 32 * i < E) ? expf(v[i] - mx) : 0.f;
    z = warp_sum(z);
    float sel_p = 0.f, sum_sel = 0.f;                            // lane j keeps the j-th selected probability
    int sel_e = -1;
    for (int j = 0; j < top_k; ++j) {
        // best remaining (value desc, index asc) in this lane, then across the warp
        float bv = -INFINITY; int be = 0x7fffffff;
#pragma unroll
        for (int i = 0; i < kMaxPer; ++i) {
            const int e = lane + 32 * i;
            if (e < E && (v[i] > bv || (v[i] == bv && e < be))) { bv = v[i]; be = e; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oe = __shfl_xor_sync(0xffffffffu, be, o);
            if (ov > bv || (ov == bv && oe < be)) { bv = ov; be = oe; }
        }
        const float p = expf(bv - mx) / z;
        if (lane == j) { sel_p = p; sel_e = be; }
        sum_sel += p;
        if ((be & 31) == lane) v[be >> 5] = -INFINITY;           // remove it (a lane owns experts lane, lane+32, ...)
    }
    if (lane < top_k) {
        ids[(size_t)row * top_k + lane] = sel_e;
        wts[(size_t)row * top_k + lane] = sel_p / sum_sel;
    }
}

// CTA e ranks the entries routed to expert e in entry order and counts them.
__global__ void __launch_bounds__(256) moe_rank_kernel(int n_entries, const int32_t* __restrict__ ids,
                                                       int32_t* __restrict__ rank, int32_t* __restrict__ counts)
{
    __shared__ int s_warp[8];
    __shared__ int s_base;
    const int e = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    for (int i0 = 0; i0 < n_entries; i0 += 256) {
        const int i = i0 + threadIdx.x;
        const bool hit = i < n_entries && ids[i] == e;
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (lane == 0) s_warp[warp] = __popc(m);
        __syncthreads();
        int before = s_base;
        for (int w = 0; w < warp; ++w) before += s_warp[w];
        if (hit) rank[i] = before + __popc(m & ((1u << lane) - 1u));
        __syncthreads();
        if (threadIdx.x == 0) { int t = 0; for (int w = 0; w < 8; ++w) t += s_warp[w]; s_base += t; }
        __syncthreads();
    }
    if (threadIdx.x == 0) counts[e] = s_base;
}

// Entry i = (token m, slot j) goes to row offsets[expert] + rank of the permuted activation matrix.
template <class T>
__global__ void __launch_bounds__(256) moe_gather_kernel(int E, int top_k, int d, const int32_t* __restrict__ ids,
                                                         const int32_t* __restrict__ rank, const int32_t* __restrict__ counts,
                                                         int32_t* __restrict__ offsets, int32_t* __restrict__ inv,
                                                         const T* __restrict__ h, T* __restrict__ a_perm,
                                                         const float* __restrict__ row_scale, float* __restrict__ perm_scale)
{
    __shared__ int s_off;
    const int i = blockIdx.x, e = ids[i];
    if (threadIdx.x < 32) {
        int part = 0;
        for (int x = threadIdx.x; x < e; x += 32) part += counts[x];
        part = (int)warp_sum((float)part);                       // counts are small integers: exact in fp32
        if (threadIdx.x == 0) s_off = part;
    }
    if (i == 0 && threadIdx.x == 64) {                            // the grouped GEMM's offsets array
        int run = 0;
        for (int x = 0; x < E; ++x) { offsets[x] = run; run += counts[x]; }
    }
    __syncthreads();
    const int pos = s_off + rank[i];
    if (threadIdx.x == 0) {
        inv[i] = pos;
        if (row_scale != nullptr) perm_scale[pos] = row_scale[i / top_k];   // 8-bit rows travel with their scale
    }
    const T* src = h + (size_t)(i / top_k) * d;
    T* dst = a_perm + (size_t)pos * d;
    for (int c = threadIdx.x * 8; c < d; c += 256 * 8)
        *reinterpret_cast<uint4*>(dst + c) = *reinterpret_cast<const uint4*>(src + c);
}

__global__ void __launch_bounds__(256) moe_combine_kernel(int top_k, int d, const float* __restrict__ wts,
                                                          const int32_t* __restrict__ inv, const float* __restrict__ out_perm,
                                                          float* __restrict__ x)
{
    const int m = blockIdx.x;
    for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
        float4 acc = *reinterpret_cast<const float4*>(x + (size_t)m * d + c);
        for (int j = 0; j < top_k; ++j) {
            const float w = wts[(size_t)m * top_k + j];
            const float4 v = *reinterpret_cast<const float4*>(out_perm + (size_t)inv[(size_t)m * top_k + j] * d + c);
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y); acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
        *reinterpret_cast<float4*>(x + (size_t)m * d + c) = acc;
    }
}

}  // namespace

spec_status launch_moe_route(int M, int E, int top_k, const float* logits, int32_t* ids, float* wts, cudaStream_t st)
{
    if (M == 0) return SPEC_OK;
    if (E > 256 || top_k > 32) return SPEC_ERR_SHAPE;
    moe_route_kernel<<<(M + 3) / 4, 128, 0, st>>>(M, E, top_k, logits, ids, wts);
    return launch_status();
}

// Ranks n_entries routed entries inside their experts (entry order) and counts them per expert; n_entries may be 0.
spec_status launch_moe_rank(int n_entries, int E, const int32_t* ids, int32_t* rank, int32_t* counts, cudaStream_t st)
{
    moe_rank_kernel<<<E, 256, 0, st>>>(n_entries, ids, rank, counts);
    return launch_status();
}

spec_status launch_moe_permute(int M, int E, int top_k, int d, const int32_t* ids, int32_t* rank, int32_t* counts,
                               int32_t* offsets, int32_t* inv, const void* h, void* a_perm, cudaStream_t st,
                               const float* row_scale, float* perm_scale)
{
    const int n = M * top_k;
    if (n == 0) return SPEC_OK;
    moe_rank_kernel<<<E, 256, 0, st>>>(n, ids, rank, counts);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    moe_gather_kernel<__nv_bfloat16><<<n, 256, 0, st>>>(E, top_k, d, ids, rank, counts, offsets, inv,
                                                       (const __nv_bfloat16*)h, (__nv_bfloat16*)a_perm, row_scale, perm_scale);
    return launch_status(2);
}

spec_status launch_moe_combine(int M, int top_k, int d, const float* wts, const int32_t* inv, const float* out_perm,
                               float* x, cudaStream_t st)
{
    if (M == 0) return SPEC_OK;
    moe_combine_kernel<<<M, 256, 0, st>>>(top_k, d, wts, inv, out_perm, x);
    return launch_status();
}

}  // namespace spec
