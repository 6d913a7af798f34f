// Element-wise, gather/scatter and bookkeeping kernels of the verify and draft forwards: row metadata, embedding
// gather, RMSNorm, rotary embedding + paged KV append, SwiGLU, tap copies, and the paged-KV reserve / commit pass
// (step S5: keep the accepted slots, return the blocks of rejected ones).  All HBM-bound and small next to the
// attention and GEMM passes; written for coalesced 16-byte accesses where the row width allows.
#include "ops.cuh"

namespace spec {
namespace {

template <class T> struct Vec4;     // 4 elements loaded/stored as one access
template <> struct Vec4<float> {
    static __device__ __forceinline__ void load(const float* p, float (&v)[4])
    {
        const float4 t = *reinterpret_cast<const float4*>(p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    static __device__ __forceinline__ void store(float* p, const float (&v)[4])
    {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct Vec4<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[4])
    {
        const uint2 t = *reinterpret_cast<const uint2*>(p);
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
        v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[4])
    {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
        uint2 t;
        t.x = *reinterpret_cast<uint32_t*>(&a);
        t.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(p) = t;
    }
};

// ---- row metadata of a verify forward: tokens [last, d_1..d_k] at positions len .. len+k --------------------------
__global__ void verify_rows_kernel(int B, int R, const int32_t* seq_len, const int32_t* last_token,
                                   const int32_t* draft, int draft_stride, int vocab, StepRows rows, int32_t* status)
{
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= B * R) return;
    const int b = m / R, i = m % R;
    if (seq_len[b] < 0) { rows.token[m] = 0; rows.pos[m] = -1; return; }     // retired slot: inert rows, no cache access
    int tok = (i == 0) ? last_token[b] : draft[(size_t)b * draft_stride + i - 1];
    if (tok < 0 || tok >= vocab) { set_status(status, SPEC_ERR_TOKEN_RANGE, b); tok = 0; }
    rows.token[m] = tok;
    rows.pos[m] = seq_len[b] + i;
}

template <class T>
__global__ void embed_kernel(int d, const T* __restrict__ table, const int32_t* __restrict__ token, float* __restrict__ x)
{
    const int m = blockIdx.x;
    const int tok = token[m];
    float* xr = x + (size_t)m * d;
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (tok >= 0) Vec4<T>::load(table + (size_t)tok * d + c, v);
        Vec4<float>::store(xr + c, v);
    }
}

template <class T>
__global__ void __launch_bounds__(256) rmsnorm_kernel(int d, const float* __restrict__ in, const float* __restrict__ w,
                                                      float eps, T* __restrict__ out, int ld_out, int col0)
{
    pdl_trigger();
    pdl_wait();
    const int m = blockIdx.x;
    const float* xr = in + (size_t)m * d;
    __shared__ float s_part[8];
    float ss = 0.f;
    for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
        float v[4];
        Vec4<float>::load(xr + c, v);
        ss += v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += s_part[i];
    const float r = rsqrtf(tot / (float)d + eps);
    T* orow = out + (size_t)m * ld_out + col0;
    for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
        float v[4], g[4];
        Vec4<float>::load(xr + c, v);
        Vec4<float>::load(w + c, g);
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = v[e] * r * g[e];
        Vec4<T>::store(orow + c, v);
    }
}

// ---- rotary embedding (half-split pairing (j, j+dh/2), angle pos * theta^(-2j/dh)) + paged KV append ------------
template <class T>
__global__ void __launch_bounds__(256) rope_append_kernel(int R, int Hq, int Hkv, int dh, float theta,
                                                          T* __restrict__ qkv, const int32_t* __restrict__ pos,
                                                          T* __restrict__ k_pool, T* __restrict__ v_pool,
                                                          const int32_t* __restrict__ block_table, int max_blocks,
                                                          int block_tokens, const float2* __restrict__ table, int M)
{
    pdl_trigger();
    pdl_wait();
    extern __shared__ float s_cs[];                       // cos [dh/2], sin [dh/2]
    const int m = blockIdx.x;
    const int p = pos[m];
    if (p < 0) return;
    const int b = m / R;
    const int half = dh / 2;
    for (int j = threadIdx.x; j < half; j += blockDim.x) {
        if (table != nullptr) {                           // the forward's (cos, sin) table [dh/2][M]: the same fp32 values
            const float2 t = table[(size_t)j * M + m];
            s_cs[j] = t.x; s_cs[half + j] = t.y;
            continue;
        }
        // the angle is formed in fp64: at positions of 10^4 an fp32 product would already be off by 10^-3 rad
        const double inv = exp2(-2.0 * (double)j / (double)dh * log2((double)theta));
        double s, c;
        sincos((double)p * inv, &s, &c);
        s_cs[j] = (float)c;
        s_cs[half + j] = (float)s;
    }
    __syncthreads();
    T* row = qkv + (size_t)m * (Hq + 2 * Hkv) * dh;
    const int blk = block_table[(size_t)b * max_blocks + p / block_tokens];
    const int slot = p % block_tokens;
    if constexpr (sizeof(T) == 2) {
        if (half % 8 == 0) {
            // bf16: eight pairs per thread, 16-byte loads and stores (the scalar loop below is latency-bound at small batch)
            const int vec = half / 8;
            for (int idx = threadIdx.x; idx < (Hq + Hkv) * vec; idx += blockDim.x) {
                const int h = idx / vec, j = (idx % vec) * 8;
                T* hp = row + (size_t)h * dh;
                uint4 ua = *reinterpret_cast<const uint4*>(hp + j), ub = *reinterpret_cast<const uint4*>(hp + j + half);
                T* pa = reinterpret_cast<T*>(&ua);
                T* pb = reinterpret_cast<T*>(&ub);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float a = to_f32(pa[e]), bb = to_f32(pb[e]);
                    const float c = s_cs[j + e], sn = s_cs[half + j + e];
                    pa[e] = from_f32<T>(a * c - bb * sn);
                    pb[e] = from_f32<T>(bb * c + a * sn);
                }
                T* dst = nullptr;
                if (h < Hq) dst = hp;
                else if (blk >= 0) dst = k_pool + (((size_t)blk * Hkv + (h - Hq)) * block_tokens + slot) * dh;
                if (dst != nullptr) {
                    *reinterpret_cast<uint4*>(dst + j) = ua;
                    *reinterpret_cast<uint4*>(dst + j + half) = ub;
                }
            }
            if (blk >= 0) {
                const T* vsrc = row + (size_t)(Hq + Hkv) * dh;
                for (int idx = threadIdx.x; idx < Hkv * dh / 8; idx += blockDim.x) {
                    const int h = (idx * 8) / dh, j = (idx * 8) % dh;
                    *reinterpret_cast<uint4*>(v_pool + (((size_t)blk * Hkv + h) * block_tokens + slot) * dh + j) =
                        *reinterpret_cast<const uint4*>(vsrc + (size_t)idx * 8);
                }
            }
            return;
        }
    }
    // q and k heads: rotate pairs
    for (int idx = threadIdx.x; idx < (Hq + Hkv) * half; idx += blockDim.x) {
        const int h = idx / half, j = idx % half;
        T* hp = row + (size_t)h * dh;
        const float a = to_f32(hp[j]), bb = to_f32(hp[j + half]);
        const float c = s_cs[j], s = s_cs[half + j];
        const T ra = from_f32<T>(a * c - bb * s), rb = from_f32<T>(bb * c + a * s);
        if (h < Hq) {
            hp[j] = ra; hp[j + half] = rb;
        } else if (blk >= 0) {
            T* dst = k_pool + (((size_t)blk * Hkv + (h - Hq)) * block_tokens + slot) * dh;
            dst[j] = ra; dst[j + half] = rb;
        }
    }
    if (blk >= 0) {
        const T* vsrc = row + (size_t)(Hq + Hkv) * dh;
        for (int idx = threadIdx.x; idx < Hkv * dh; idx += blockDim.x) {
            const int h = idx / dh, j = idx % dh;
            v_pool[(((size_t)blk * Hkv + h) * block_tokens + slot) * dh + j] = vsrc[idx];
        }
    }
}

// gate_up [M][2F] holds 256-column groups: 128 gate columns, then the matching 128 up columns
template <class T>
__global__ void swiglu_kernel(size_t total4, int F, const T* __restrict__ gu, T* __restrict__ out)
{
    pdl_trigger();
    pdl_wait();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total4) return;
    const size_t e = i * 4;
    const size_t m = e / F, c = e % F;
    const size_t gc = (c / 128) * 256 + c % 128;
    float g[4], u[4], o[4];
    Vec4<T>::load(gu + m * 2 * F + gc, g);
    Vec4<T>::load(gu + m * 2 * F + gc + 128, u);
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = g[j] / (1.f + __expf(-g[j])) * u[j];
    Vec4<T>::store(out + e, o);
}

// (cos, sin) of pos * theta^(-2j/dh), j < dh/2, per row, stored [dh/2][M]; formed in fp64 (see rope_append_kernel)
__global__ void rope_table_kernel(int M, int half, int dh, float theta, const int32_t* __restrict__ pos, float2* __restrict__ table)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * half) return;
    const int m = i / half, j = i % half;
    const int p = pos[m];
    double s = 0.0, c = 1.0;
    if (p >= 0) {
        const double inv = exp2(-2.0 * (double)j / (double)dh * log2((double)theta));
        sincos((double)p * inv, &s, &c);
    }
    table[(size_t)j * M + m] = make_float2((float)c, (float)s);      // [dh/2][M]: rows are the fast index, so the GEMM
                                                                    // epilogue (one row per lane) reads it coalesced
}

template <class T>
__global__ void copy_rows_kernel(int d, const float* __restrict__ x, T* __restrict__ out, int ld_out, int col0)
{
    pdl_trigger();
    pdl_wait();
    const int m = blockIdx.x;
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
        float v[4];
        Vec4<float>::load(x + (size_t)m * d + c, v);
        Vec4<T>::store(out + (size_t)m * ld_out + col0 + c, v);
    }
}

__global__ void gather_last_rows_kernel(int R, int d, const float* __restrict__ src, const int32_t* __restrict__ n_valid,
                                        float* __restrict__ dst)
{
    const int b = blockIdx.x;
    const int r = n_valid[b] - 1;
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
        float v[4] = {0.f, 0.f, 0.f, 0.f};                      // no valid row: a zero state, not a stale one
        if (r >= 0) Vec4<float>::load(src + ((size_t)b * R + r) * d + c, v);
        Vec4<float>::store(dst + (size_t)b * d + c, v);
    }
}

// ---- paged-KV bookkeeping: one CTA, sequences in index order, so the result does not depend on scheduling ------
constexpr int kBookThreads = 1024;

__device__ int block_exclusive_scan(int v, int* total, int* s_warp /*[33]*/)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = s_warp[lane];
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += t;
        }
        s_warp[lane] = winc - w;
        if (lane == 31) s_warp[32] = winc;
    }
    __syncthreads();
    *total = s_warp[32];
    return s_warp[warp] + inc - v;
}

__global__ void __launch_bounds__(kBookThreads) kv_reserve_kernel(int B, int k, int bt, int max_blocks,
                                                                  const int32_t* seq_len, int32_t* table, int32_t* owned,
                                                                  int32_t* free_stack, int32_t* free_top, int32_t* status)
{
    // owned[b] = number of logical blocks sequence b holds (always the prefix 0..owned-1 of its table row)
    __shared__ int s_warp[33];
    __shared__ int s_fail;
    if (threadIdx.x == 0) s_fail = 0;
    __syncthreads();
    const int top0 = *free_top;
    // first sweep: total demand (nothing is changed if it cannot be served)
    int demand = 0;
    for (int base = 0; base < B; base += kBookThreads) {
        const int b = base + threadIdx.x;
        int need_new = 0;
        if (b < B && seq_len[b] >= 0) {                           // a retired slot (negative length) asks for nothing
            const int need = (seq_len[b] + k + 1 + bt - 1) / bt;
            if (need > max_blocks) { s_fail = 1; set_status(status, SPEC_ERR_KV_EXHAUSTED, b); }
            else need_new = max(0, need - owned[b]);
        }
        int tot;
        block_exclusive_scan(need_new, &tot, s_warp);
        demand += tot;
    }
    __syncthreads();
    if (s_fail) return;
    if (demand > top0) { if (threadIdx.x == 0) set_status(status, SPEC_ERR_KV_EXHAUSTED, -1); return; }
    int carry = 0;
    for (int base = 0; base < B; base += kBookThreads) {
        const int b = base + threadIdx.x;
        int need = 0, have = 0;
        if (b < B && seq_len[b] >= 0) { need = (seq_len[b] + k + 1 + bt - 1) / bt; have = owned[b]; }
        int tot;
        int off = carry + block_exclusive_scan(max(0, need - have), &tot, s_warp);
        if (b < B && need > have) {
            for (int j = have; j < need; ++j) { table[(size_t)b * max_blocks + j] = free_stack[top0 - 1 - off]; ++off; }
            owned[b] = need;
        }
        carry += tot;
    }
    __syncthreads();
    if (threadIdx.x == 0) *free_top = top0 - carry;
}

__global__ void __launch_bounds__(kBookThreads) kv_commit_kernel(const CommitArgs a)
{
    __shared__ int s_warp[33];
    __shared__ long long s_cnt[2];
    if (threadIdx.x == 0) { s_cnt[0] = 0; s_cnt[1] = 0; }
    __syncthreads();
    const int top0 = *a.free_top;
    const int R = a.k + 1;
    int carry = 0;
    for (int base = 0; base < a.B; base += kBookThreads) {
        const int b = base + threadIdx.x;
        int freed = 0, keep = 0;
        if (b < a.B && a.seq_len[b] < 0) {                       // retired slot: nothing emitted, nothing kept
            a.n_emitted[b] = 0;
            for (int i = 0; i < R; ++i) a.out_tokens[(size_t)b * R + i] = -1;
        } else if (b < a.B) {
            int n1, last;
            if (a.force_n != nullptr && a.force_n[b] >= 0) {     // a negative entry leaves the sequence to the sampler
                n1 = min(max(a.force_n[b], 0), a.k) + 1;
                last = a.force_token[b];
                // the committed tokens of a forced step are the verified inputs d_1..d_n followed by the given token
                for (int i = 0; i < R; ++i)
                    a.out_tokens[(size_t)b * R + i] = i < n1 - 1 ? a.verify_tokens[(size_t)b * R + i + 1] : (i == n1 - 1 ? last : -1);
                a.n_emitted[b] = n1;
            } else {
                n1 = min(max(a.n_emitted[b], 1), R);
                last = a.out_tokens[(size_t)b * R + n1 - 1];
            }
            if (a.history != nullptr)            // the tokens whose cache entries this commit keeps: x_last, d_1..d_n
                for (int i = 0; i < n1 && a.seq_len[b] + i < a.max_hist; ++i)
                    a.history[(size_t)b * a.max_hist + a.seq_len[b] + i] = a.verify_tokens[(size_t)b * R + i];
            a.pending_base[b] = a.seq_len[b];
            const int len = a.seq_len[b] + n1;
            a.seq_len[b] = len;
            a.last_token[b] = last;
            keep = (len + a.block_tokens - 1) / a.block_tokens;
            freed = max(0, a.owned[b] - keep);
            atomicAdd((unsigned long long*)&s_cnt[0], (unsigned long long)n1);
            atomicAdd((unsigned long long*)&s_cnt[1], (unsigned long long)(n1 - 1));
        }
        int tot;
        int off = carry + block_exclusive_scan(freed, &tot, s_warp);
        if (b < a.B && freed > 0) {
            for (int j = keep; j < keep + freed; ++j) {
                int32_t* e = &a.block_table[(size_t)b * a.max_blocks + j];
                a.free_stack[top0 + off] = *e; ++off; *e = -1;
            }
            a.owned[b] = keep;
        }
        carry += tot;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        *a.free_top = top0 + carry;
        *a.step += 1u;
        a.counters[0] += 1;
        a.counters[1] += s_cnt[0];
        a.counters[2] += s_cnt[1];
    }
}

// One CTA per sequence.  Context t[0..L-1] = history[0..len-1] followed by the last token.  For n = n_max..1: the trailing
// n tokens are searched at every earlier start s (s + n <= L - 1, so that at least one token follows the match); the
// largest such s wins; the draft continues from t[s+n], and once it runs past the end it repeats its last token.
__global__ void __launch_bounds__(256) ngram_draft_kernel(int k, int n_max, const int32_t* __restrict__ history, int max_hist,
                                                          const int32_t* __restrict__ seq_len,
                                                          const int32_t* __restrict__ last_token,
                                                          int32_t* __restrict__ draft, int draft_stride)
{
    __shared__ int s_best;
    const int b = blockIdx.x;
    const int32_t* h = history + (size_t)b * max_hist;
    const int len = min(seq_len[b], max_hist), L = len + 1;
    const int last = last_token[b];
    auto tok = [&](int p) { return p < len ? h[p] : last; };
    int found_s = -1, found_n = 0;
    for (int n = min(n_max, L - 1); n >= 1 && found_s < 0; --n) {
        if (threadIdx.x == 0) s_best = -1;
        __syncthreads();
        for (int s = threadIdx.x; s + n <= L - 1; s += blockDim.x) {
            bool eq = true;
            for (int j = 0; j < n && eq; ++j) eq = tok(s + j) == tok(L - n + j);
            if (eq) atomicMax(&s_best, s);
        }
        __syncthreads();
        if (s_best >= 0) { found_s = s_best; found_n = n; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int prev = last;
        for (int i = 0; i < k; ++i) {
            const int p = found_s + found_n + i;
            const int t = (found_s >= 0 && p <= L - 1) ? tok(p) : prev;
            draft[(size_t)b * draft_stride + i] = t;
            prev = t;
        }
    }
}

// Slot replacement (finished sequences leave, new ones take their slots).  One thread, list order: the bookkeeping is a
// few integers per sequence and must be deterministic.
__global__ void kv_replace_kernel(int n, const int32_t* __restrict__ slots, const int32_t* __restrict__ new_len,
                                  const int32_t* __restrict__ new_last, int bt, int max_blocks, int32_t* seq_len,
                                  int32_t* last_token, int32_t* table, int32_t* owned, int32_t* free_stack, int32_t* free_top,
                                  int32_t* n_emitted, int32_t* pending_base, int32_t* status)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int top = *free_top;
    long avail = top, need = 0;
    for (int i = 0; i < n; ++i) { avail += owned[slots[i]]; need += new_len[i] < 0 ? 0 : (new_len[i] + bt - 1) / bt; }
    if (need > avail) { set_status(status, SPEC_ERR_KV_EXHAUSTED, -2); return; }
    for (int i = 0; i < n; ++i) {
        const int b = slots[i];
        int32_t* row = table + (size_t)b * max_blocks;
        for (int j = 0; j < owned[b]; ++j) { free_stack[top++] = row[j]; row[j] = -1; }
        const int blocks = new_len[i] < 0 ? 0 : (new_len[i] + bt - 1) / bt;      // negative: the slot is retired
        for (int j = 0; j < blocks; ++j) row[j] = free_stack[--top];
        owned[b] = blocks;
        seq_len[b] = new_len[i] < 0 ? -1 : new_len[i];
        last_token[b] = new_last[i];
        n_emitted[b] = 0;                                       // nothing pending for the draft head
        pending_base[b] = new_len[i] < 0 ? 0 : new_len[i];
    }
    *free_top = top;
}

// Renumbering of the running sequences (new slot j <- old slot keep[j], keep strictly ascending, so j <= keep[j] and a row
// is never overwritten before it has been read when the slots are walked in order).  One CTA: the scalars by one thread in
// slot order, the table / token rows slot by slot with the threads across a row.
struct CompactArgs {
    int n_keep, B_old, max_blocks, out_stride, hist_len;
    const int32_t* keep;
    int32_t *seq_len, *last_token, *owned, *pending_base, *n_emitted, *table, *out_tokens, *history;
    float* out_logp;
};
__global__ void __launch_bounds__(256) seq_compact_kernel(const CompactArgs a)
{
    if (threadIdx.x == 0) {
        for (int j = 0; j < a.n_keep; ++j) {
            const int s = a.keep[j];
            a.seq_len[j] = a.seq_len[s]; a.last_token[j] = a.last_token[s]; a.owned[j] = a.owned[s];
            a.pending_base[j] = a.pending_base[s]; a.n_emitted[j] = a.n_emitted[s];
        }
        for (int j = a.n_keep; j < a.B_old; ++j) {          // the vacated tail: retired, owning nothing
            a.seq_len[j] = -1; a.last_token[j] = 0; a.owned[j] = 0; a.pending_base[j] = 0; a.n_emitted[j] = 0;
        }
    }
    for (int j = 0; j < a.n_keep; ++j) {
        const int s = a.keep[j];
        if (s == j) continue;
        for (int c = threadIdx.x; c < a.max_blocks; c += blockDim.x) a.table[(size_t)j * a.max_blocks + c] = a.table[(size_t)s * a.max_blocks + c];
        for (int c = threadIdx.x; c < a.out_stride; c += blockDim.x) {
            a.out_tokens[(size_t)j * a.out_stride + c] = a.out_tokens[(size_t)s * a.out_stride + c];
            a.out_logp[(size_t)j * a.out_stride + c] = a.out_logp[(size_t)s * a.out_stride + c];
        }
        if (a.history != nullptr)
            for (int c = threadIdx.x; c < a.hist_len; c += blockDim.x) a.history[(size_t)j * a.hist_len + c] = a.history[(size_t)s * a.hist_len + c];
        __syncthreads();                                    // a later slot may read what this one's source row held: keep the order
    }
    __syncthreads();
    for (int j = a.n_keep + (int)(threadIdx.x / 32); j < a.B_old; j += blockDim.x / 32)
        for (int c = threadIdx.x % 32; c < a.max_blocks; c += 32) a.table[(size_t)j * a.max_blocks + c] = -1;
}
// dst row j*R + i <- src row keep[j]*R + i (16-byte pieces); dst and src do not overlap.
__global__ void __launch_bounds__(256) permute_rows_kernel(int R, size_t row_bytes, const int32_t* __restrict__ keep,
                                                           const unsigned char* __restrict__ src, unsigned char* __restrict__ dst)
{
    const int j = blockIdx.x / R, i = blockIdx.x % R;
    const uint4* s4 = reinterpret_cast<const uint4*>(src + ((size_t)keep[j] * R + i) * row_bytes);
    uint4* d4 = reinterpret_cast<uint4*>(dst + (size_t)blockIdx.x * row_bytes);
    for (size_t c = threadIdx.x; c < row_bytes / 16; c += blockDim.x) d4[c] = s4[c];
}

// Per-row e4m3 quantisation of a bf16 matrix: one CTA per row.  scale = amax / 448 in fp32 (1 for a zero row), codes =
// round_e4m3(x / scale) with an exact fp32 division, round to nearest even, saturating: the same steps as the oracle's.
template <int CHUNKS>
__global__ void __launch_bounds__(256) quantize_rows_kernel(int K, const __nv_bfloat16* __restrict__ x, unsigned char* __restrict__ codes,
                                                            float* __restrict__ scales, const int32_t* __restrict__ rows_valid)
{
    // rows_valid (may be null): a device-side count; rows at or past it are left alone
    // CHUNKS > 0: the row (K <= 256 * 8 * CHUNKS) stays in registers between the maximum and the conversion, one global read;
    // CHUNKS == 0: any K, the row is read twice (the second time from cache)
    pdl_trigger();
    pdl_wait();
    __shared__ float s_w[8];
    const int row = blockIdx.x;
    if (rows_valid != nullptr && row >= *rows_valid) return;
    const __nv_bfloat16* xr = x + (size_t)row * K;
    constexpr int NV = CHUNKS > 0 ? CHUNKS : 1;
    uint4 held[NV];
    float amax = 0.f;
    if constexpr (CHUNKS > 0) {
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
            const int i = (j * 256 + threadIdx.x) * 8;
            held[j] = i < K ? *reinterpret_cast<const uint4*>(xr + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
            const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&held[j]);
#pragma unroll
            for (int e = 0; e < 4; ++e) amax = fmaxf(amax, fmaxf(fabsf(__low2float(p[e])), fabsf(__high2float(p[e]))));
        }
    } else {
        for (int i = threadIdx.x * 8; i < K; i += 256 * 8) {
            const uint4 v = *reinterpret_cast<const uint4*>(xr + i);
            const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int e = 0; e < 4; ++e) amax = fmaxf(amax, fmaxf(fabsf(__low2float(p[e])), fabsf(__high2float(p[e]))));
        }
    }
    amax = warp_max(amax);
    if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = amax;
    __syncthreads();
    float m = s_w[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) m = fmaxf(m, s_w[w]);
    const float sc = m > 0.f ? __fdiv_rn(m, 448.f) : 1.f;
    if (threadIdx.x == 0) scales[row] = sc;
    unsigned char* cr = codes + (size_t)row * K;
    auto convert = [&](const uint4& v, int i) {
        const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
        uint32_t w[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            unsigned short lo, hi;                           // cvt packs its first source into the upper byte
            asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(__fdiv_rn(__high2float(p[2 * h]), sc)), "f"(__fdiv_rn(__low2float(p[2 * h]), sc)));
            asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(__fdiv_rn(__high2float(p[2 * h + 1]), sc)), "f"(__fdiv_rn(__low2float(p[2 * h + 1]), sc)));
            w[h] = (uint32_t)lo | ((uint32_t)hi << 16);
        }
        *reinterpret_cast<uint2*>(cr + i) = make_uint2(w[0], w[1]);
    };
    if constexpr (CHUNKS > 0) {
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
            const int i = (j * 256 + threadIdx.x) * 8;
            if (i < K) convert(held[j], i);
        }
    } else {
        for (int i = threadIdx.x * 8; i < K; i += 256 * 8) convert(*reinterpret_cast<const uint4*>(xr + i), i);
    }
}

// RMSNorm of an fp32 row followed by the per-row e4m3 quantisation of its bf16-rounded result, in one kernel: the same
// values, scale and codes as rmsnorm_kernel<bf16> followed by quantize_rows_kernel (the 16-bit row itself is not written:
// in a context with 8-bit projections nothing else reads it).  d % 4 == 0.
__global__ void __launch_bounds__(256) rmsnorm_quantize_kernel(int d, const float* __restrict__ in, const float* __restrict__ w, float eps,
                                                               unsigned char* __restrict__ codes, float* __restrict__ scales)
{
    pdl_trigger();
    pdl_wait();
    const int m = blockIdx.x;
    const float* xr = in + (size_t)m * d;
    __shared__ float s_part[8];
    __shared__ float s_max[8];
    float ss = 0.f;
    for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
        float v[4];
        Vec4<float>::load(xr + c, v);
        ss += v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += s_part[i];
    const float r = rsqrtf(tot / (float)d + eps);
    float amax = 0.f;
    for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
        float v[4], g[4];
        Vec4<float>::load(xr + c, v);
        Vec4<float>::load(w + c, g);
#pragma unroll
        for (int e = 0; e < 4; ++e) amax = fmaxf(amax, fabsf(__bfloat162float(__float2bfloat16_rn(v[e] * r * g[e]))));
    }
    amax = warp_max(amax);
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    float mx = s_max[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) mx = fmaxf(mx, s_max[i]);
    const float sc = mx > 0.f ? __fdiv_rn(mx, 448.f) : 1.f;
    if (threadIdx.x == 0) scales[m] = sc;
    unsigned char* cr = codes + (size_t)m * d;
    for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
        float v[4], g[4];
        Vec4<float>::load(xr + c, v);
        Vec4<float>::load(w + c, g);
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = __fdiv_rn(__bfloat162float(__float2bfloat16_rn(v[e] * r * g[e])), sc);
        unsigned short lo, hi;                               // cvt packs its first source into the upper byte
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(v[1]), "f"(v[0]));
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(v[3]), "f"(v[2]));
        *reinterpret_cast<uint32_t*>(cr + c) = (uint32_t)lo | ((uint32_t)hi << 16);
    }
}

}  // namespace

#define DISPATCH_T(dtype, ...)                                            \
    if ((dtype) == SPEC_DTYPE_F32) { using T = float; __VA_ARGS__; }      \
    else { using T = __nv_bfloat16; __VA_ARGS__; }

spec_status launch_verify_rows(int B, int R, const int32_t* seq_len, const int32_t* last_token,
                               const int32_t* draft_tokens, int draft_stride, int vocab, StepRows rows,
                               int32_t* status, cudaStream_t st)
{
    const int M = B * R;
    if (M == 0) return SPEC_OK;
    verify_rows_kernel<<<(M + 255) / 256, 256, 0, st>>>(B, R, seq_len, last_token, draft_tokens, draft_stride, vocab, rows, status);
    return launch_status();
}

spec_status launch_embed(int M, int d, const void* table, int dtype, const int32_t* token, float* x, cudaStream_t st)
{
    if (M == 0) return SPEC_OK;
    DISPATCH_T(dtype, embed_kernel<T><<<M, 256, 0, st>>>(d, (const T*)table, token, x));
    return launch_status();
}

spec_status launch_rmsnorm(int M, int d, const float* in, const float* w, float eps, void* out, int ld_out, int col0,
                           int dtype, cudaStream_t st)
{
    if (M == 0) return SPEC_OK;
    DISPATCH_T(dtype, launch_pdl(rmsnorm_kernel<T>, dim3(M), dim3(256), 0, st, d, in, w, eps, (T*)out, ld_out, col0));
    return launch_status();
}

spec_status launch_rope_append(int B, int R, int Hq, int Hkv, int dh, float theta, void* qkv, const int32_t* pos,
                               void* k_pool, void* v_pool, const int32_t* block_table, int max_blocks,
                               int block_tokens, int dtype, cudaStream_t st, const float* rope_table)
{
    if (B * R == 0) return SPEC_OK;
    DISPATCH_T(dtype, launch_pdl(rope_append_kernel<T>, dim3(B * R), dim3(256), dh * sizeof(float), st,
                          R, Hq, Hkv, dh, theta, (T*)qkv, pos, (T*)k_pool, (T*)v_pool, block_table, max_blocks, block_tokens,
                          reinterpret_cast<const float2*>(rope_table), B * R));
    return launch_status();
}

spec_status launch_swiglu(int M, int F, const void* gate_up, void* out, int dtype, cudaStream_t st)
{
    const size_t total4 = (size_t)M * F / 4;
    if (total4 == 0) return SPEC_OK;
    DISPATCH_T(dtype, launch_pdl(swiglu_kernel<T>, dim3((unsigned)((total4 + 255) / 256)), dim3(256), 0, st, total4, F, (const T*)gate_up, (T*)out));
    return launch_status();
}

spec_status launch_rope_table(int M, int dh, float theta, const int32_t* pos, float* table, cudaStream_t st)
{
    const int n = M * (dh / 2);
    if (n == 0) return SPEC_OK;
    rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(M, dh / 2, dh, theta, pos, reinterpret_cast<float2*>(table));
    return launch_status();
}

spec_status launch_copy_rows_f32_to(int M, int d, const float* x, void* out, int ld_out, int col0, int dtype,
                                    cudaStream_t st)
{
    if (M == 0) return SPEC_OK;
    DISPATCH_T(dtype, launch_pdl(copy_rows_kernel<T>, dim3(M), dim3(256), 0, st, d, x, (T*)out, ld_out, col0));
    return launch_status();
}

spec_status launch_gather_last_rows(int B, int R, int d, const float* src, const int32_t* n_valid, float* dst,
                                    cudaStream_t st)
{
    if (B == 0) return SPEC_OK;
    gather_last_rows_kernel<<<B, 256, 0, st>>>(R, d, src, n_valid, dst);
    return launch_status();
}

spec_status launch_kv_reserve(int B, int k, int block_tokens, int max_blocks, const int32_t* seq_len,
                              int32_t* block_table, int32_t* owned, int32_t* free_stack, int32_t* free_top, int32_t* status,
                              cudaStream_t st)
{
    if (B == 0) return SPEC_OK;
    kv_reserve_kernel<<<1, kBookThreads, 0, st>>>(B, k, block_tokens, max_blocks, seq_len, block_table, owned, free_stack, free_top, status);
    return launch_status();
}

spec_status launch_ngram_draft(int B, int k, int n_max, const int32_t* history, int max_hist, const int32_t* seq_len,
                               const int32_t* last_token, int32_t* draft_tokens, int draft_stride, cudaStream_t st)
{
    if (B == 0) return SPEC_OK;
    ngram_draft_kernel<<<B, 256, 0, st>>>(k, n_max, history, max_hist, seq_len, last_token, draft_tokens, draft_stride);
    return launch_status();
}

spec_status launch_kv_replace(int n, const int32_t* slots, const int32_t* new_len, const int32_t* new_last, int bt,
                              int max_blocks, int32_t* seq_len, int32_t* last_token, int32_t* table, int32_t* owned,
                              int32_t* free_stack, int32_t* free_top, int32_t* n_emitted,
                              int32_t* pending_base, int32_t* status, cudaStream_t st)
{
    if (n == 0) return SPEC_OK;
    kv_replace_kernel<<<1, 32, 0, st>>>(n, slots, new_len, new_last, bt, max_blocks, seq_len, last_token, table, owned,
                                        free_stack, free_top, n_emitted, pending_base, status);
    return launch_status();
}

spec_status launch_seq_compact(int n_keep, int B_old, const int32_t* keep, int max_blocks, int out_stride, int hist_len, int32_t* seq_len,
                               int32_t* last_token, int32_t* owned, int32_t* pending_base, int32_t* n_emitted, int32_t* table,
                               int32_t* out_tokens, float* out_logp, int32_t* history, cudaStream_t st)
{
    CompactArgs a{n_keep, B_old, max_blocks, out_stride, hist_len, keep, seq_len, last_token, owned, pending_base, n_emitted, table,
                  out_tokens, history, out_logp};
    seq_compact_kernel<<<1, 256, 0, st>>>(a);
    return launch_status();
}

spec_status launch_permute_rows(int n_keep, int R, size_t row_bytes, const int32_t* keep, const void* src, void* dst, cudaStream_t st)
{
    if (n_keep * R == 0 || row_bytes == 0) return SPEC_OK;
    if (row_bytes % 16 != 0) return SPEC_ERR_SHAPE;
    permute_rows_kernel<<<n_keep * R, 256, 0, st>>>(R, row_bytes, keep, (const unsigned char*)src, (unsigned char*)dst);
    return launch_status();
}

spec_status launch_quantize_rows(int rows, int K, const void* x_bf16, void* codes, float* scales, cudaStream_t st, const int32_t* rows_valid)
{
    if (rows == 0) return SPEC_OK;
    if (K <= 0 || K % 8 != 0) return SPEC_ERR_SHAPE;
    if (K <= 256 * 8 * 2)      launch_pdl(quantize_rows_kernel<2>, dim3(rows), dim3(256), 0, st, K, (const __nv_bfloat16*)x_bf16, (unsigned char*)codes, scales, rows_valid);
    else if (K <= 256 * 8 * 8) launch_pdl(quantize_rows_kernel<8>, dim3(rows), dim3(256), 0, st, K, (const __nv_bfloat16*)x_bf16, (unsigned char*)codes, scales, rows_valid);
    else                       launch_pdl(quantize_rows_kernel<0>, dim3(rows), dim3(256), 0, st, K, (const __nv_bfloat16*)x_bf16, (unsigned char*)codes, scales, rows_valid);
    return launch_status();
}

spec_status launch_rmsnorm_quantize(int M, int d, const float* in, const float* w, float eps, void* codes, float* scales, cudaStream_t st)
{
    if (M == 0) return SPEC_OK;
    if (d <= 0 || d % 4 != 0) return SPEC_ERR_SHAPE;
    launch_pdl(rmsnorm_quantize_kernel, dim3(M), dim3(256), 0, st, d, in, w, eps, (unsigned char*)codes, scales);
    return launch_status();
}

spec_status launch_kv_commit(const CommitArgs& a, cudaStream_t st)
{
    if (a.B == 0) return SPEC_OK;
    kv_commit_kernel<<<1, kBookThreads, 0, st>>>(a);
    return launch_status();
}

}  // namespace spec

extern "C" spec_status spec_quantize_rows(int rows, int K, const void* x_bf16, void* codes, float* scales, void* stream)
{
    if (rows < 0 || K <= 0) return SPEC_ERR_INVALID_ARG;
    if (rows == 0) return SPEC_OK;
    if (!x_bf16 || !codes || !scales) return SPEC_ERR_INVALID_ARG;
    return spec::launch_quantize_rows(rows, K, x_bf16, codes, scales, (cudaStream_t)stream, nullptr);
}
