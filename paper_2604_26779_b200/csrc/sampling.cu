// Vocabulary softmax statistics, inverse-CDF sampling and lossless rejection sampling (steps S3 and S4 of the
// speculation step: accept_i = u_i < min(1, p_i(d_i)/q_i(d_i)); first rejected position resampled from
// norm(max(0, p - q)); bonus token from p_{k+1} when every draft token is accepted).
//
// All three passes are HBM-bound streams over fp32 rows of vocabulary width.  One CTA owns one row (softmax
// statistics) or one sequence (sampling); lanes read 16 bytes at consecutive addresses; the row of weights is
// reduced to one fp64 sum per 512-element chunk in shared memory, the chunk holding the u-quantile is found by a
// scan over those sums, and only that chunk is read a second time to locate the token.  So a draw costs one pass
// over the row(s) it samples from, not two.  With at most a few hundred sequences a cluster of four CTAs shares that pass
// (distributed shared memory carries the chunk sums to the CTA that scans them).
#include "ops.cuh"

namespace spec {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kChunk = 512;          // elements reduced to one fp64 partial sum (one warp, 4 x float4 per lane)
constexpr int kMaxChunks = 1024;     // rows up to 524288 wide

// Probability of one logit given the row statistics.  Every kernel that needs a probability goes through this one
// expression so that materialised and on-the-fly probabilities are the same fp32 numbers.
__device__ __forceinline__ float prob_from_logit(float l, float m, float inv_t, float inv_z)
{
    return __fmul_rn(__expf(__fmul_rn(__fsub_rn(l, m), inv_t)), inv_z);
}

// Loads 4 consecutive floats of a row starting at idx (a multiple of 4); elements past V read as `fill`.
__device__ __forceinline__ void load4(const float* __restrict__ row, int idx, int V, bool vec_ok, float fill,
                                      float (&out)[4])
{
    if (vec_ok && idx + 3 < V) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(row + idx));
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) out[e] = (idx + e < V) ? __ldg(row + idx + e) : fill;
    }
}

__device__ __forceinline__ bool row_vec_ok(const float* row, int V)
{
    return (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(row) & 15u) == 0);
}

// ---- weight functors: non-negative weights of the distribution a token is drawn from ---------------------------
struct ProbRow {                      // w = p
    const float* p; bool vec;
    __device__ void load(int idx, int V, float (&w)[4]) const { load4(p, idx, V, vec, 0.f, w); }
};
struct ResidualProbs {                // w = max(0, p - q)
    const float* p; const float* q; bool vec;
    __device__ void load(int idx, int V, float (&w)[4]) const
    {
        float a[4], b[4];
        load4(p, idx, V, vec, 0.f, a);
        load4(q, idx, V, vec, 0.f, b);
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = fmaxf(0.f, __fsub_rn(a[e], b[e]));
    }
};
struct LogitRow {                     // w = softmax(l / T)
    const float* l; float m, inv_z, inv_t; bool vec;
    __device__ void load(int idx, int V, float (&w)[4]) const
    {
        float a[4];
        load4(l, idx, V, vec, -INFINITY, a);
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = (idx + e < V) ? prob_from_logit(a[e], m, inv_t, inv_z) : 0.f;
    }
};
struct ResidualLogits {               // w = max(0, softmax(lp/T) - softmax(lq/T))
    LogitRow P, Q;
    __device__ void load(int idx, int V, float (&w)[4]) const
    {
        float a[4], b[4];
        P.load(idx, V, a);
        Q.load(idx, V, b);
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = fmaxf(0.f, __fsub_rn(a[e], b[e]));
    }
};

// A draft distribution over a subset of the vocabulary: q(x) = softmax(lq / T)[t2d[x]] where t2d[x] >= 0, else 0.
struct MappedLogitRow {
    LogitRow Q; const int32_t* t2d;
    __device__ void load(int idx, int V, float (&w)[4]) const
    {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int t = (idx + e < V) ? t2d[idx + e] : -1;
            w[e] = t >= 0 ? prob_from_logit(Q.l[t], Q.m, Q.inv_t, Q.inv_z) : 0.f;
        }
    }
};
struct ResidualLogitsMapped {
    LogitRow P; MappedLogitRow Q;
    __device__ void load(int idx, int V, float (&w)[4]) const
    {
        float a[4], b[4];
        P.load(idx, V, a);
        Q.load(idx, V, b);
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = fmaxf(0.f, __fsub_rn(a[e], b[e]));
    }
};

// Deterministic draft (q = one-hot(d)): the residual is p with the draft token's mass removed.
template <class Row>
struct ResidualOneHot {
    Row P; int d;
    __device__ void load(int idx, int V, float (&w)[4]) const
    {
        P.load(idx, V, w);
#pragma unroll
        for (int e = 0; e < 4; ++e) if (idx + e == d) w[e] = 0.f;
    }
};

struct InvCdfSmem {
    double chunk_sum[kMaxChunks];
    int token;
};

// Block-wide inverse CDF: the smallest v with  sum_{j<=v} w_j > u * sum_j w_j  (strict; a zero-weight bin is never
// chosen); if rounding leaves every prefix at or below the target, the last positive bin.  Returns -1 when the row
// has no positive finite mass.  All threads of the block must call it; all get the result.
// The fp64 sum of one 512-element chunk of weights (one warp; the same fp32 tree in every caller, so that whoever computes
// a chunk gets the same number).
template <class WF>
__device__ __forceinline__ double chunk_sum_of(const WF& wf, int V, int c, int lane)
{
    const int base = c * kChunk + lane * 4;
    float w[16];
#pragma unroll
    for (int s = 0; s < 4; ++s) wf.load(base + s * 128, V, *reinterpret_cast<float(*)[4]>(&w[4 * s]));
    float part[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) part[s] = (w[4 * s] + w[4 * s + 1]) + (w[4 * s + 2] + w[4 * s + 3]);
    return warp_sum((double)((part[0] + part[1]) + (part[2] + part[3])));
}

template <class WF> __device__ int invcdf_select(const WF& wf, int V, float u, InvCdfSmem& sm);

template <class WF>
__device__ int block_invcdf(const WF& wf, int V, float u, InvCdfSmem& sm)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunks = (V + kChunk - 1) / kChunk;
    __syncthreads();                                         // the shared buffer may still be in use by a previous draw
    // pass over the row: one fp64 sum per chunk
    for (int c = warp; c < nchunks; c += (int)(blockDim.x >> 5)) {
        const double d = chunk_sum_of(wf, V, c, lane);
        if (lane == 0) sm.chunk_sum[c] = d;
    }
    __syncthreads();
    return invcdf_select(wf, V, u, sm);
}

// ---- the same draw by a cluster of CTAs: with a few hundred sequences one CTA per sequence leaves most of the machine
// idle, so kClusterCtas CTAs share the pass over the row; each writes its chunk sums straight into the first CTA's table
// through distributed shared memory, and that CTA scans them and takes the second look.  The sums are the same numbers
// whoever computes them, so the drawn token does not depend on the cluster size.
constexpr int kClusterCtas = 4;
__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f64(uint32_t local_saddr, uint32_t target_rank, double v)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_saddr), "r"(target_rank));
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(remote), "d"(v) : "memory");
}
// All CTAs of the cluster must call it with the same functor; returns the token in the first CTA and -2 in the others
// (which have nothing left to do).
template <class WF>
__device__ int cluster_invcdf(const WF& wf, int V, float u, InvCdfSmem& sm)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunks = (V + kChunk - 1) / kChunk;
    const uint32_t rank = cluster_cta_rank();
    const uint32_t table = (uint32_t)__cvta_generic_to_shared(&sm.chunk_sum[0]);
    for (int c = (int)rank * kWarps + warp; c < nchunks; c += kClusterCtas * kWarps) {
        const double d = chunk_sum_of(wf, V, c, lane);
        if (lane == 0) st_cluster_f64(table + (uint32_t)c * 8u, 0u, d);
    }
    cluster_sync_all();                                      // every sum has landed in the first CTA's table
    if (rank != 0) return -2;
    return invcdf_select(wf, V, u, sm);
}

template <class WF>
__device__ int invcdf_select(const WF& wf, int V, float u, InvCdfSmem& sm)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunks = (V + kChunk - 1) / kChunk;
    if (warp == 0) {
        // scan of the chunk sums: every lane owns a contiguous range of chunks
        const int per = (nchunks + 31) / 32;
        const int c0 = min(lane * per, nchunks), c1 = min(c0 + per, nchunks);
        double loc = 0.0;
        for (int c = c0; c < c1; ++c) loc += sm.chunk_sum[c];
        const double incl = warp_inclusive_scan(loc, lane);
        double excl = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) excl = 0.0;
        const double S = __shfl_sync(0xffffffffu, incl, 31);
        int token = -1;
        if (S > 0.0 && S < 1.0e300) {
            const double target = (double)u * S;
            int found = -1, last_pos_chunk = -1;
            double before = 0.0, before_last = 0.0, run = excl;
            for (int c = c0; c < c1; ++c) {
                const double cs = sm.chunk_sum[c];
                const double nxt = run + cs;
                if (cs > 0.0) { last_pos_chunk = c; before_last = run; }
                if (found < 0 && nxt > target) { found = c; before = run; }
                run = nxt;
            }
            const unsigned hit = __ballot_sync(0xffffffffu, found >= 0);
            if (hit != 0u) {
                const int src = __ffs(hit) - 1;
                found = __shfl_sync(0xffffffffu, found, src);
                before = __shfl_sync(0xffffffffu, before, src);
            } else {                                          // shortfall by rounding: the last chunk with mass
                const unsigned pos = __ballot_sync(0xffffffffu, last_pos_chunk >= 0);
                const int src = 31 - __clz(pos);
                found = __shfl_sync(0xffffffffu, last_pos_chunk, src);
                before = __shfl_sync(0xffffffffu, before_last, src);
            }
            // second look at the one chunk that holds the quantile, in fp64 and in index order
            const int base = found * kChunk + lane * 4;
            float w[16];
#pragma unroll
            for (int s = 0; s < 4; ++s) wf.load(base + s * 128, V, *reinterpret_cast<float(*)[4]>(&w[4 * s]));
            double run2 = before;
            int last_pos = -1;
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                const double ls = (((double)w[4 * s] + (double)w[4 * s + 1]) + (double)w[4 * s + 2]) + (double)w[4 * s + 3];
                const double inc = warp_inclusive_scan(ls, lane);
                double exc = __shfl_up_sync(0xffffffffu, inc, 1);
                if (lane == 0) exc = 0.0;
                double r = run2 + exc;
                int mine = -1;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    r += (double)w[4 * s + e];
                    if (w[4 * s + e] > 0.f) {
                        last_pos = base + s * 128 + e;
                        if (mine < 0 && r > target) mine = base + s * 128 + e;
                    }
                }
                const unsigned hm = __ballot_sync(0xffffffffu, mine >= 0);
                if (token < 0 && hm != 0u) token = __shfl_sync(0xffffffffu, mine, __ffs(hm) - 1);
                run2 += __shfl_sync(0xffffffffu, inc, 31);
            }
            if (token < 0) token = warp_max(last_pos);
        }
        if (lane == 0) sm.token = token;
    }
    __syncthreads();
    return sm.token;
}

// ---- softmax statistics (and optionally probabilities) ----------------------------------------------------------
__global__ void __launch_bounds__(kThreads) softmax_rows_kernel(int rows, int V, const float* __restrict__ logits,
                                                                size_t row_stride, float inv_t,
                                                                float* __restrict__ stats, size_t stats_stride,
                                                                float* __restrict__ probs)
{
    const int row = blockIdx.x;
    const float* l = logits + (size_t)row * row_stride;
    const bool vec = row_vec_ok(l, V);
    __shared__ float s_m[kWarps], s_z[kWarps];
    __shared__ float s_fin[2];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // online maximum and sum of exponentials: z always refers to the current m
    float m = -INFINITY, z = 0.f;
    for (int base = threadIdx.x * 4; base < V; base += kThreads * 4 * 2) {
        float a[4], b[4];
        load4(l, base, V, vec, -INFINITY, a);
        load4(l, base + kThreads * 4, V, vec, -INFINITY, b);
        const float mx = fmaxf(fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3])), fmaxf(fmaxf(b[0], b[1]), fmaxf(b[2], b[3])));
        if (mx > m) { z *= __expf(__fmul_rn(__fsub_rn(m, mx), inv_t)); m = mx; }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            z += __expf(__fmul_rn(__fsub_rn(a[e], m), inv_t));
            z += __expf(__fmul_rn(__fsub_rn(b[e], m), inv_t));
        }
    }
    // combine (m, z) pairs: warp, then block
    const float wm = warp_max(m);
    z = (m == -INFINITY) ? 0.f : z * __expf(__fmul_rn(__fsub_rn(m, wm), inv_t));
    z = warp_sum(z);
    if (lane == 0) { s_m[warp] = wm; s_z[warp] = z; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float bm = s_m[0];
        for (int w = 1; w < kWarps; ++w) bm = fmaxf(bm, s_m[w]);
        float bz = 0.f;
        for (int w = 0; w < kWarps; ++w)
            bz += (s_m[w] == -INFINITY) ? 0.f : s_z[w] * __expf(__fmul_rn(__fsub_rn(s_m[w], bm), inv_t));
        s_fin[0] = bm; s_fin[1] = bz;
        if (stats) { stats[2 * (size_t)row * stats_stride] = bm; stats[2 * (size_t)row * stats_stride + 1] = bz; }
    }
    if (probs == nullptr) return;
    __syncthreads();
    const float bm = s_fin[0], inv_z = __frcp_rn(s_fin[1]);
    float* pr = probs + (size_t)row * V;
    const bool vec_out = vec && ((reinterpret_cast<uintptr_t>(pr) & 15u) == 0);
    for (int base = threadIdx.x * 4; base < V; base += kThreads * 4) {
        float a[4];
        load4(l, base, V, vec, -INFINITY, a);
        float o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e] = prob_from_logit(a[e], bm, inv_t, inv_z);
        if (vec_out && base + 3 < V) {
            *reinterpret_cast<float4*>(pr + base) = make_float4(o[0], o[1], o[2], o[3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) if (base + e < V) pr[base + e] = o[e];
        }
    }
}

// The same statistics (and probabilities) by a cluster of kStatCtas CTAs per row: with few rows (a thin batch) one CTA per
// row reads its 0.5 MB of logits far below the memory rate.  Every CTA reduces a quarter-aligned slice of the row, hands its
// (m, z) pair to the first CTA through distributed shared memory, and that one combines the pairs in rank order.
constexpr int kStatCtas = 8;
__global__ void __launch_bounds__(kThreads) softmax_rows_cluster_kernel(int rows, int V, const float* __restrict__ logits,
                                                                        size_t row_stride, float inv_t,
                                                                        float* __restrict__ stats, size_t stats_stride,
                                                                        float* __restrict__ probs)
{
    const int row = blockIdx.x / kStatCtas;
    const uint32_t rank = cluster_cta_rank();
    const float* l = logits + (size_t)row * row_stride;
    const bool vec = row_vec_ok(l, V);
    __shared__ float s_m[kWarps], s_z[kWarps];
    __shared__ float s_pair[2 * kStatCtas];                  // first CTA: (m, z) of every rank
    __shared__ float s_fin[2];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slice = (((V + kStatCtas - 1) / kStatCtas) + 3) & ~3;
    const int lo = min(V, (int)rank * slice), hi = min(V, lo + slice);

    float m = -INFINITY, z = 0.f;
    for (int base = lo + threadIdx.x * 4; base < hi; base += kThreads * 4) {
        float a[4];
        load4(l, base, hi, vec, -INFINITY, a);
        const float mx = fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
        if (mx > m) { z *= __expf(__fmul_rn(__fsub_rn(m, mx), inv_t)); m = mx; }
#pragma unroll
        for (int e = 0; e < 4; ++e) z += __expf(__fmul_rn(__fsub_rn(a[e], m), inv_t));
    }
    const float wm = warp_max(m);
    z = (m == -INFINITY) ? 0.f : z * __expf(__fmul_rn(__fsub_rn(m, wm), inv_t));
    z = warp_sum(z);
    if (lane == 0) { s_m[warp] = wm; s_z[warp] = z; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float bm = s_m[0];
        for (int w = 1; w < kWarps; ++w) bm = fmaxf(bm, s_m[w]);
        float bz = 0.f;
        for (int w = 0; w < kWarps; ++w)
            bz += (s_m[w] == -INFINITY) ? 0.f : s_z[w] * __expf(__fmul_rn(__fsub_rn(s_m[w], bm), inv_t));
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(&s_pair[2 * rank])), "r"(0));
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(bm) : "memory");
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote + 4u), "f"(bz) : "memory");
    }
    cluster_sync_all();
    if (rank == 0 && threadIdx.x == 0) {
        float bm = s_pair[0];
        for (int r = 1; r < kStatCtas; ++r) bm = fmaxf(bm, s_pair[2 * r]);
        float bz = 0.f;
        for (int r = 0; r < kStatCtas; ++r)
            bz += (s_pair[2 * r] == -INFINITY) ? 0.f : s_pair[2 * r + 1] * __expf(__fmul_rn(__fsub_rn(s_pair[2 * r], bm), inv_t));
        s_fin[0] = bm; s_fin[1] = bz;
        if (stats) { stats[2 * (size_t)row * stats_stride] = bm; stats[2 * (size_t)row * stats_stride + 1] = bz; }
    }
    if (probs == nullptr) return;                            // uniform over the cluster: no CTA waits below for one that left
    cluster_sync_all();
    float bm, bz;
    {
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(&s_fin[0])), "r"(0));
        asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(bm) : "r"(remote) : "memory");
        asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(bz) : "r"(remote + 4u) : "memory");
    }
    const float inv_z = __frcp_rn(bz);
    float* pr = probs + (size_t)row * V;
    const bool vec_out = vec && ((reinterpret_cast<uintptr_t>(pr) & 15u) == 0);
    for (int base = lo + threadIdx.x * 4; base < hi; base += kThreads * 4) {
        float a[4];
        load4(l, base, hi, vec, -INFINITY, a);
        float o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e] = prob_from_logit(a[e], bm, inv_t, inv_z);
        if (vec_out && base + 3 < hi) {
            *reinterpret_cast<float4*>(pr + base) = make_float4(o[0], o[1], o[2], o[3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) if (base + e < hi) pr[base + e] = o[e];
        }
    }
    cluster_sync_all();                                      // the first CTA's shared memory is read until here
}

// ---- one token per row by inverse CDF -----------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) sample_rows_kernel(int V, const float* __restrict__ probs, uint64_t seed,
                                                               uint32_t step, uint32_t slot, uint32_t stream_tag,
                                                               int32_t* __restrict__ tokens, int32_t* status)
{
    __shared__ InvCdfSmem sm;
    const int row = blockIdx.x;
    const float* p = probs + (size_t)row * V;
    const float u = philox_uniform(seed, step, (uint32_t)row, slot, stream_tag);
    int t = block_invcdf(ProbRow{p, row_vec_ok(p, V)}, V, u, sm);
    if (threadIdx.x == 0) {
        if (t < 0) { set_status(status, SPEC_ERR_BAD_PROB, row); t = 0; }
        tokens[row] = t;
    }
}

// one token per row from logits and their statistics (the draft head's d_i ~ q_i)
template <bool kCluster>
__global__ void __launch_bounds__(kThreads) sample_logits_kernel(int V, const float* __restrict__ logits, size_t row_stride,
                                                                 const float* __restrict__ stats, size_t stats_stride,
                                                                 float inv_t, uint64_t seed, const uint32_t* step_dev,
                                                                 uint32_t slot, uint32_t stream_tag,
                                                                 int32_t* __restrict__ tokens, int token_stride,
                                                                 int32_t* status)
{
    __shared__ InvCdfSmem sm;
    const int row = kCluster ? blockIdx.x / kClusterCtas : blockIdx.x;
    const float* l = logits + (size_t)row * row_stride;
    const float* st = stats + 2 * (size_t)row * stats_stride;
    const float u = philox_uniform(seed, *step_dev, (uint32_t)row, slot, stream_tag);
    const LogitRow wf{l, st[0], __frcp_rn(st[1]), inv_t, row_vec_ok(l, V)};
    int t;
    if constexpr (kCluster) {
        cluster_sync_all();                                  // the first CTA's table exists before anyone writes to it
        t = cluster_invcdf(wf, V, u, sm);
        if (t == -2) return;
    } else {
        t = block_invcdf(wf, V, u, sm);
    }
    if (threadIdx.x == 0) {
        if (t < 0) { set_status(status, SPEC_ERR_BAD_PROB, row); t = 0; }
        tokens[(size_t)row * token_stride] = t;
    }
}

// arg-maximum per row (greedy drafting): the largest logit, the lowest index among equals
__global__ void __launch_bounds__(kThreads) argmax_rows_kernel(int V, const float* __restrict__ logits, size_t row_stride,
                                                               int32_t* __restrict__ tokens, int token_stride)
{
    __shared__ float s_v[kThreads / 32];
    __shared__ int s_i[kThreads / 32];
    const float* l = logits + (size_t)blockIdx.x * row_stride;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int v = threadIdx.x; v < V; v += kThreads) {
        const float x = l[v];
        if (x > bv || (x == bv && v < bi)) { bv = x; bi = v; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { s_v[threadIdx.x >> 5] = bv; s_i[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kThreads / 32; ++w)
            if (s_v[w] > bv || (s_v[w] == bv && s_i[w] < bi)) { bv = s_v[w]; bi = s_i[w]; }
        tokens[(size_t)blockIdx.x * token_stride] = bi == 0x7fffffff ? 0 : bi;
    }
}

// ---- rejection sampling ---------------------------------------------------------------------------------------------
struct RejectArgs {
    int B, k, V;
    const float* p;            // [B][k+1][V] probabilities or logits
    const float* q;            // [B][k][V]
    const float* p_stats;      // [B*(k+1)][2] (max, sum exp) when logits, else unused
    const float* q_stats;      // [B*k][2]
    int Vq;                    // width of a q row (V unless the draft head has its own vocabulary)
    const int32_t* t2d;        // [V] target id -> column of q, -1 outside the draft vocabulary; nullptr: identity
    const int32_t* draft;      // d_i of sequence b at draft[b*draft_stride + i]
    int draft_stride;
    float inv_t;
    uint64_t seed;
    const uint32_t* step_dev;  // step counter on the device, or nullptr to use `step`
    uint32_t step;
    int32_t* out_tokens;       // [B][k+1]
    int32_t* n_emitted;        // [B]
    int32_t* status;
    float* out_logp;           // [B][k+1] log p_target(emitted token) under the verifier, or nullptr
};

template <bool kFromLogits, bool kCluster>
__global__ void __launch_bounds__(kThreads) reject_sample_kernel(const RejectArgs A)
{
    __shared__ InvCdfSmem sm;
    __shared__ int s_n;
    const int b = kCluster ? blockIdx.x / kClusterCtas : blockIdx.x, k = A.k, V = A.V;
    if constexpr (kCluster) cluster_sync_all();              // the first CTA's table exists before anyone writes to it
    // the first draw is shared by the CTAs of a cluster (every CTA takes the same branch: the accept tests below are
    // recomputed by each); whatever follows it is the first CTA's alone
    auto draw = [&](const auto& wf, float u) {
        if constexpr (kCluster) return cluster_invcdf(wf, V, u, sm);
        else                    return block_invcdf(wf, V, u, sm);
    };
    const uint32_t step = A.step_dev ? *A.step_dev : A.step;
    const float* prow0 = A.p + (size_t)b * (k + 1) * V;
    const int Vq = A.Vq;
    const float* qrow0 = A.q + (size_t)b * k * Vq;

    auto p_row = [&](int i) {
        const float* l = prow0 + (size_t)i * V;
        if constexpr (kFromLogits) {
            const float* st = A.p_stats + 2 * ((size_t)b * (k + 1) + i);
            return LogitRow{l, st[0], __frcp_rn(st[1]), A.inv_t, row_vec_ok(l, V)};
        } else {
            return ProbRow{l, row_vec_ok(l, V)};
        }
    };
    auto q_row = [&](int i) {
        const float* l = qrow0 + (size_t)i * Vq;
        if constexpr (kFromLogits) {
            const float* st = A.q_stats + 2 * ((size_t)b * k + i);
            return LogitRow{l, st[0], __frcp_rn(st[1]), A.inv_t, row_vec_ok(l, Vq)};
        } else {
            return ProbRow{l, row_vec_ok(l, V)};
        }
    };

    // accept tests: lane i decides position i+1 with its own (positional) uniform; the ratio test is taken in fp64
    if (threadIdx.x < 32) {
        const int i = threadIdx.x;
        bool acc = false;
        if (i < k) {
            const int d = A.draft[(size_t)b * A.draft_stride + i];
            if (d < 0 || d >= V) {
                set_status(A.status, SPEC_ERR_TOKEN_RANGE, b);
            } else {
                float pd, qd;
                if constexpr (kFromLogits) {
                    const auto P = p_row(i);
                    pd = prob_from_logit(P.l[d], P.m, P.inv_t, P.inv_z);
                    if (A.q != nullptr) {
                        const auto Q = q_row(i);
                        const int dq = A.t2d != nullptr ? A.t2d[d] : d;            // a token outside the draft vocabulary has q = 0
                        qd = dq >= 0 ? prob_from_logit(Q.l[dq], Q.m, Q.inv_t, Q.inv_z) : 0.f;
                    } else qd = 1.f;                                 // deterministic draft: q = one-hot(d)
                } else {
                    pd = prow0[(size_t)i * V + d];
                    qd = A.q != nullptr ? qrow0[(size_t)i * V + d] : 1.f;
                }
                const float u = philox_uniform(A.seed, step, (uint32_t)b, (uint32_t)i, 0u);
                double thr;
                if (qd > 0.f) thr = fmin(1.0, (double)pd / (double)qd);
                else          thr = pd > 0.f ? 1.0 : 0.0;
                acc = (double)u < thr;
            }
        }
        const unsigned mask = __ballot_sync(0xffffffffu, acc);
        if (threadIdx.x == 0) s_n = min(k, __ffs(~mask) - 1);   // length of the all-accepted prefix
    }
    __syncthreads();
    const int n = s_n;
    const float u_last = philox_uniform(A.seed, step, (uint32_t)b, (uint32_t)k, 0u);

    int token;
    if (n < k && A.q == nullptr) {
        const int dn = A.draft[(size_t)b * A.draft_stride + n];
        token = draw(ResidualOneHot<decltype(p_row(n))>{p_row(n), dn}, u_last);
        if (token == -2) return;
        if (token < 0) {
            if (threadIdx.x == 0) set_status(A.status, SPEC_ERR_BAD_PROB, b);
            token = block_invcdf(p_row(n), V, u_last, sm);
        }
    } else if (n < k) {
        if constexpr (kFromLogits) {
            if (A.t2d != nullptr) token = draw(ResidualLogitsMapped{p_row(n), MappedLogitRow{q_row(n), A.t2d}}, u_last);
            else                  token = draw(ResidualLogits{p_row(n), q_row(n)}, u_last);
        }
        else                       token = draw(ResidualProbs{prow0 + (size_t)n * V, qrow0 + (size_t)n * V,
                                                              row_vec_ok(prow0 + (size_t)n * V, V) &&
                                                              row_vec_ok(qrow0 + (size_t)n * V, V)}, u_last);
        if (token == -2) return;
        if (token < 0) {                                       // residual without mass: garbage input
            if (threadIdx.x == 0) set_status(A.status, SPEC_ERR_BAD_PROB, b);
            token = block_invcdf(p_row(n), V, u_last, sm);
        }
    } else {
        token = draw(p_row(k), u_last);
        if (token == -2) return;
    }
    if (token < 0) {
        if (threadIdx.x == 0) set_status(A.status, SPEC_ERR_BAD_PROB, b);
        token = 0;
    }
    if (threadIdx.x <= k) {
        const int i = threadIdx.x;
        A.out_tokens[(size_t)b * (k + 1) + i] = i < n ? A.draft[(size_t)b * A.draft_stride + i] : (i == n ? token : -1);
    }
    if (threadIdx.x == 0) A.n_emitted[b] = n + 1;
    // log-probability of every emitted token under the TARGET (the quantity an RL loss needs: never the draft's)
    if (A.out_logp != nullptr && threadIdx.x <= k) {
        const int i = threadIdx.x;
        float lp = 0.f;
        if (i <= n) {
            const int t = i < n ? A.draft[(size_t)b * A.draft_stride + i] : token;
            if constexpr (kFromLogits) {
                const auto P = p_row(i);
                lp = __fmul_rn(__fsub_rn(P.l[t], P.m), P.inv_t) - logf(A.p_stats[2 * ((size_t)b * (k + 1) + i) + 1]);
            } else {
                lp = logf(prow0[(size_t)i * V + t]);
            }
        }
        A.out_logp[(size_t)b * (k + 1) + i] = lp;
    }
}

__global__ void uniforms_kernel(uint64_t seed, uint32_t step, uint32_t stream_tag, int n_seq, int n_slots, float* u)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_seq * n_slots) u[i] = philox_uniform(seed, step, (uint32_t)(i / n_slots), (uint32_t)(i % n_slots), stream_tag);
}

}  // namespace

// ---- launchers used by the context and by the stateless entry points -------------------------------------------
spec_status launch_softmax_rows(int rows, int V, const float* logits, size_t row_stride, float temperature, float* stats,
                                size_t stats_stride, float* probs, cudaStream_t st)
{
    if (rows == 0) return SPEC_OK;
    if (rows <= 128 && V >= 8192) {                          // few rows: a cluster of CTAs per row
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)rows * kStatCtas); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute attr{};
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = kStatCtas; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr; cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, softmax_rows_cluster_kernel, rows, V, logits, row_stride, 1.0f / temperature, stats, stats_stride, probs) !=
            cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
        return launch_status();
    }
    softmax_rows_kernel<<<rows, kThreads, 0, st>>>(rows, V, logits, row_stride, 1.0f / temperature, stats, stats_stride, probs);
    return launch_status();
}

namespace {
constexpr int kClusterBatchLimit = 512;          // above this one CTA per sequence already fills the machine
template <class... KArgs, class... Args>
spec_status launch_clustered(void (*kernel)(KArgs...), int n_seq, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)n_seq * kClusterCtas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = kClusterCtas; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) != cudaSuccess) { cudaGetLastError(); return SPEC_ERR_CUDA; }
    return launch_status();
}
}  // namespace

spec_status launch_reject_sample(bool from_logits, int B, int k, int V, const float* p, const float* p_stats,
                                 const float* q, const float* q_stats, int q_width, const int32_t* t2d,
                                 const int32_t* draft, int draft_stride,
                                 float temperature, uint64_t seed, const uint32_t* step_dev, uint32_t step,
                                 int32_t* out_tokens, int32_t* n_emitted, int32_t* status, float* out_logp, cudaStream_t st)
{
    if (B == 0) return SPEC_OK;
    RejectArgs A{B, k, V, p, q, p_stats, q_stats, q_width, t2d, draft, draft_stride, 1.0f / temperature, seed, step_dev, step, out_tokens,
                 n_emitted, status, out_logp};
    // few sequences: a cluster of CTAs per sequence, so that the pass over the vocabulary uses the whole machine
    if (B <= kClusterBatchLimit) {
        if (from_logits) return launch_clustered(reject_sample_kernel<true, true>, B, st, A);
        return launch_clustered(reject_sample_kernel<false, true>, B, st, A);
    }
    if (from_logits) reject_sample_kernel<true, false><<<B, kThreads, 0, st>>>(A);
    else             reject_sample_kernel<false, false><<<B, kThreads, 0, st>>>(A);
    return launch_status();
}

spec_status launch_sample_logits(int rows, int V, const float* logits, size_t row_stride, const float* stats,
                                 size_t stats_stride, float temperature, uint64_t seed, const uint32_t* step_dev,
                                 uint32_t slot, uint32_t stream_tag, int32_t* tokens, int token_stride, int32_t* status,
                                 cudaStream_t st)
{
    if (rows == 0) return SPEC_OK;
    if (rows <= kClusterBatchLimit)
        return launch_clustered(sample_logits_kernel<true>, rows, st, V, logits, row_stride, stats, stats_stride, 1.0f / temperature,
                                seed, step_dev, slot, stream_tag, tokens, token_stride, status);
    sample_logits_kernel<false><<<rows, kThreads, 0, st>>>(V, logits, row_stride, stats, stats_stride, 1.0f / temperature, seed,
                                                           step_dev, slot, stream_tag, tokens, token_stride, status);
    return launch_status();
}

spec_status launch_argmax_rows(int rows, int V, const float* logits, size_t row_stride, int32_t* tokens, int token_stride,
                               cudaStream_t st)
{
    if (rows == 0) return SPEC_OK;
    argmax_rows_kernel<<<rows, kThreads, 0, st>>>(V, logits, row_stride, tokens, token_stride);
    return launch_status();
}

// target-to-draft map of a draft head with its own vocabulary: t2d[x] = r where d2t[r] = x, -1 elsewhere
__global__ void build_t2d_kernel(int V, int Vd, const int32_t* __restrict__ d2t, int32_t* __restrict__ t2d, int phase)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (phase == 0) { if (i < V) t2d[i] = -1; }
    else if (i < Vd) { const int x = d2t[i]; if (x >= 0 && x < V) t2d[x] = i; }
}
__global__ void map_tokens_kernel(int B, const int32_t* __restrict__ src, int src_stride, const int32_t* __restrict__ d2t,
                                  int32_t* __restrict__ dst, int dst_stride)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) dst[(size_t)b * dst_stride] = d2t[src[(size_t)b * src_stride]];
}

spec_status launch_build_t2d(int V, int Vd, const int32_t* d2t, int32_t* t2d, cudaStream_t st)
{
    build_t2d_kernel<<<(V + 255) / 256, 256, 0, st>>>(V, Vd, d2t, t2d, 0);
    build_t2d_kernel<<<(Vd + 255) / 256, 256, 0, st>>>(V, Vd, d2t, t2d, 1);
    return launch_status(2);
}

spec_status launch_map_tokens(int B, const int32_t* src, int src_stride, const int32_t* d2t, int32_t* dst, int dst_stride,
                              cudaStream_t st)
{
    if (B == 0) return SPEC_OK;
    map_tokens_kernel<<<(B + 255) / 256, 256, 0, st>>>(B, src, src_stride, d2t, dst, dst_stride);
    return launch_status();
}

int sampler_max_vocab() { return kMaxChunks * kChunk; }

}  // namespace spec

using namespace spec;

extern "C" spec_status spec_softmax_rows(int rows, int V, const float* logits, float temperature, float* stats,
                                         float* probs, void* stream)
{
    if (rows < 0 || V <= 0 || !(temperature > 0.f)) return SPEC_ERR_INVALID_ARG;
    if (rows == 0) return SPEC_OK;
    if (logits == nullptr) return SPEC_ERR_INVALID_ARG;
    return launch_softmax_rows(rows, V, logits, (size_t)V, temperature, stats, 1, probs, (cudaStream_t)stream);
}

extern "C" spec_status spec_sample_rows(int rows, int V, const float* probs, uint64_t seed, uint32_t step,
                                        uint32_t slot, uint32_t stream_tag, int32_t* tokens, int32_t* status,
                                        void* stream)
{
    if (rows < 0 || V <= 0) return SPEC_ERR_INVALID_ARG;
    if (rows == 0) return SPEC_OK;
    if (probs == nullptr || tokens == nullptr) return SPEC_ERR_INVALID_ARG;
    if (V > sampler_max_vocab()) return SPEC_ERR_SHAPE;
    sample_rows_kernel<<<rows, kThreads, 0, (cudaStream_t)stream>>>(V, probs, seed, step, slot, stream_tag, tokens, status);
    return launch_status();
}

extern "C" spec_status spec_reject_sample_probs(int B, int k, int V, const float* p, const float* q,
                                                const int32_t* draft, uint64_t seed, uint32_t step,
                                                int32_t* out_tokens, int32_t* n_emitted, int32_t* status, void* stream)
{
    if (B < 0 || k < 0 || k > 31 || V <= 0) return SPEC_ERR_INVALID_ARG;
    if (B == 0) return SPEC_OK;
    if (p == nullptr || out_tokens == nullptr || n_emitted == nullptr) return SPEC_ERR_INVALID_ARG;
    if (k > 0 && draft == nullptr) return SPEC_ERR_INVALID_ARG;       // q == NULL: deterministic drafts, q = one-hot(d)
    if (V > sampler_max_vocab()) return SPEC_ERR_SHAPE;
    return launch_reject_sample(false, B, k, V, p, nullptr, q, nullptr, V, nullptr, draft, k, 1.0f, seed, nullptr, step, out_tokens,
                                n_emitted, status, nullptr, (cudaStream_t)stream);
}

extern "C" spec_status spec_reject_sample_logits(int B, int k, int V, const float* p_logits, const float* p_stats,
                                                 const float* q_logits, const float* q_stats, const int32_t* draft,
                                                 float temperature, uint64_t seed, uint32_t step, int32_t* out_tokens,
                                                 int32_t* n_emitted, int32_t* status, void* stream)
{
    if (B < 0 || k < 0 || k > 31 || V <= 0 || !(temperature > 0.f)) return SPEC_ERR_INVALID_ARG;
    if (B == 0) return SPEC_OK;
    if (p_logits == nullptr || p_stats == nullptr || out_tokens == nullptr || n_emitted == nullptr)
        return SPEC_ERR_INVALID_ARG;
    if (k > 0 && (draft == nullptr || (q_logits != nullptr && q_stats == nullptr))) return SPEC_ERR_INVALID_ARG;
    if (V > sampler_max_vocab()) return SPEC_ERR_SHAPE;
    return launch_reject_sample(true, B, k, V, p_logits, p_stats, q_logits, q_stats, V, nullptr, draft, k, temperature, seed, nullptr,
                                step, out_tokens, n_emitted, status, nullptr, (cudaStream_t)stream);
}

extern "C" spec_status spec_uniforms(uint64_t seed, uint32_t step, uint32_t stream_tag, int n_seq, int n_slots,
                                     float* u, void* stream)
{
    if (n_seq < 0 || n_slots < 0 || u == nullptr) return SPEC_ERR_INVALID_ARG;
    const int n = n_seq * n_slots;
    if (n == 0) return SPEC_OK;
    uniforms_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>(seed, step, stream_tag, n_seq, n_slots, u);
    return launch_status();
}
