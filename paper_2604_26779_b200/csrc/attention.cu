// Paged grouped-query attention of the verify / draft forwards: every sequence brings R query rows (k+1 positions)
// that are causal among themselves and see the whole cached prefix.
//
// This file holds the plain SIMT kernel (any element type, any head shape): the reference-precision path of fp32
// models and the fallback for shapes the tensor-core kernel does not take.
#include "attention_plan.cuh"

namespace spec {
namespace {

template <class T>
__global__ void __launch_bounds__(128) attn_simt_kernel(const AttnArgs a)
{
    extern __shared__ float smem[];
    const int m = blockIdx.x, h = blockIdx.y;
    const int dh = a.dh, bt = a.block_tokens;
    float* s_q = smem;                 // [dh]
    float* s_s = smem + dh;            // [n_vis]
    __shared__ float s_red[4];
    T* out = (T*)a.out + (size_t)m * a.out_row_stride + (size_t)h * dh;
    const int p = a.pos[m];
    if (p < 0) {
        for (int j = threadIdx.x; j < dh; j += 128) out[j] = from_f32<T>(0.f);
        return;
    }
    const int b = m / a.R, kvh = h / (a.Hq / a.Hkv), n_vis = p + 1;
    const T* q = (const T*)a.q + (size_t)m * a.q_row_stride + (size_t)h * dh;
    const float scale = rsqrtf((float)dh);
    for (int j = threadIdx.x; j < dh; j += 128) s_q[j] = to_f32(q[j]) * scale;
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t* table = a.block_table + (size_t)b * a.max_blocks;
    float mx = -INFINITY;
    for (int t = warp; t < n_vis; t += 4) {
        const int blk = table[t / bt];
        float acc = -INFINITY;                          // a position without a block (reserve failed) is masked
        if (blk >= 0) {
            const T* kp = (const T*)a.k_pool + (((size_t)blk * a.Hkv + kvh) * bt + t % bt) * dh;
            acc = 0.f;
            for (int j = lane; j < dh; j += 32) acc = fmaf(s_q[j], to_f32(kp[j]), acc);
            acc = warp_sum(acc);
        }
        if (lane == 0) s_s[t] = acc;
        mx = fmaxf(mx, acc);
    }
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
    __syncthreads();
    float sum = 0.f;
    for (int t = threadIdx.x; t < n_vis; t += 128) {
        const float e = expf(s_s[t] - mx);
        s_s[t] = e;
        sum += e;
    }
    sum = warp_sum(sum);
    if (lane == 0) s_red[warp] = sum;
    __syncthreads();
    const float inv = 1.f / (s_red[0] + s_red[1] + s_red[2] + s_red[3]);
    for (int j = threadIdx.x; j < dh; j += 128) {
        float acc = 0.f;
        for (int t = 0; t < n_vis; ++t) {
            const int blk = table[t / bt];
            if (blk >= 0)
                acc = fmaf(s_s[t], to_f32(((const T*)a.v_pool)[(((size_t)blk * a.Hkv + kvh) * bt + t % bt) * dh + j]), acc);
        }
        out[j] = from_f32<T>(acc * inv);
    }
}

__global__ void attn_rows_kernel(int B, int R, const int32_t* seq_len, int32_t* pos)
{
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m < B * R) pos[m] = seq_len[m / R] + m % R;
}

}  // namespace

spec_status launch_attention_simt(const AttnArgs& a, cudaStream_t st)
{
    const int M = a.B * a.R;
    if (M == 0) return SPEC_OK;
    const size_t smem = (size_t)(a.dh + a.max_kv_len + a.R + 8) * sizeof(float);
    if (smem > 200 * 1024) return SPEC_ERR_UNSUPPORTED;
    const dim3 grid(M, a.Hq);
    if (a.dtype == SPEC_DTYPE_F32) {
        if (smem > 48 * 1024) cudaFuncSetAttribute(attn_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attn_simt_kernel<float><<<grid, 128, smem, st>>>(a);
    } else {
        if (smem > 48 * 1024) cudaFuncSetAttribute(attn_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attn_simt_kernel<__nv_bfloat16><<<grid, 128, smem, st>>>(a);
    }
    return launch_status();
}

spec_status launch_attention(const AttnArgs& a, cudaStream_t st)
{
    if (a.kv_fp8) return attn::attention_fp8_supported(a) ? attn::launch_attention_fp8(a, st) : SPEC_ERR_UNSUPPORTED;
    if (attn::attention_tc_supported(a)) return attn::launch_attention_tc(a, st);
    if (attention_mma_supported(a)) return launch_attention_mma(a, st);
    return launch_attention_simt(a, st);
}

size_t attention_scratch_bytes(int B, int R, int Hq, int Hkv, int dh, int max_kv_len)
{
    return attention_mma_scratch_bytes(B, R, Hq, Hkv, dh, max_kv_len);
}

}  // namespace spec

namespace spec {
void launch_attn_rows(int B, int R, const int32_t* seq_len, int32_t* pos, cudaStream_t st)
{
    attn_rows_kernel<<<(B * R + 255) / 256, 256, 0, st>>>(B, R, seq_len, pos);
}
}  // namespace spec

using namespace spec;

extern "C" size_t spec_attention_scratch_bytes(int B, int R, int Hq, int Hkv, int dh, int max_kv_len)
{
    return align_up((size_t)B * R * sizeof(int32_t), 256) + attention_scratch_bytes(B, R, Hq, Hkv, dh, max_kv_len);
}


extern "C" spec_status spec_attention(int B, int R, int Hq, int Hkv, int dh, int block_tokens, int max_blocks,
                                      const void* q, const void* k_pool, const void* v_pool, const int32_t* block_table,
                                      const int32_t* seq_len, void* out, int dtype, void* scratch, size_t scratch_bytes,
                                      void* stream)
{
    if (B < 0 || R <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || dh <= 0 || dh % 8 != 0 || block_tokens <= 0 ||
        max_blocks <= 0)
        return SPEC_ERR_INVALID_ARG;
    if (B == 0) return SPEC_OK;
    if (!q || !k_pool || !v_pool || !block_table || !seq_len || !out || !scratch) return SPEC_ERR_INVALID_ARG;
    // the first B*R int32 of the scratch hold the row positions; the rest is the kernels' own
    const size_t pos_bytes = align_up((size_t)B * R * sizeof(int32_t), 256);
    if (scratch_bytes < pos_bytes + attention_scratch_bytes(B, R, Hq, Hkv, dh, max_blocks * block_tokens))
        return SPEC_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    launch_attn_rows(B, R, seq_len, (int32_t*)scratch, st);
    AttnArgs a{B, R, Hq, Hkv, dh, block_tokens, max_blocks, q, Hq * dh, k_pool, v_pool, block_table,
               (const int32_t*)scratch, out, Hq * dh, dtype, (char*)scratch + pos_bytes, scratch_bytes - pos_bytes,
               max_blocks * block_tokens, 0};
    return launch_attention(a, st);
}

// ---- attention without caller-provided scratch ------------------------------------------------------------------------
// Built-in scratch for spec_attention_noalloc: one array per GPU that loads the library, held until the process exits.
namespace {
constexpr size_t kBuiltinScratchBytes = (size_t)32 << 20;                 // 32 MiB
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];
constexpr int kMaxDevices = 64;
void* g_builtin_scratch_addr[kMaxDevices] = {};                          // device address of the array, per device
}  // namespace

extern "C" spec_status spec_attention_noalloc(int B, int R, int Hq, int Hkv, int dh, int block_tokens, int max_blocks,
                                              const void* q, const void* k_pool, const void* v_pool,
                                              const int32_t* block_table, const int32_t* seq_len, void* out, int dtype,
                                              void* stream)
{
    if (B < 0 || R <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || dh <= 0 || dh % 8 != 0 || block_tokens <= 0 ||
        max_blocks <= 0)
        return SPEC_ERR_INVALID_ARG;
    if (B == 0) return SPEC_OK;
    if (!q || !k_pool || !v_pool || !block_table || !seq_len || !out) return SPEC_ERR_INVALID_ARG;
    // what spec_attention would ask the caller for must fit the built-in array
    const size_t pos_bytes = align_up((size_t)B * R * sizeof(int32_t), 256);
    const size_t need = pos_bytes + attention_scratch_bytes(B, R, Hq, Hkv, dh, max_blocks * block_tokens);
    if (need > kBuiltinScratchBytes) return SPEC_ERR_SHAPE;
    // once per device, with that device current: the array's name is a host-side handle, not a device address
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPEC_ERR_CUDA;
    if (g_builtin_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_builtin_scratch) != cudaSuccess || p == nullptr) return SPEC_ERR_CUDA;
        g_builtin_scratch_addr[dev] = p;
    }
    char* scratch = static_cast<char*>(g_builtin_scratch_addr[dev]);
    cudaStream_t st = (cudaStream_t)stream;
    // the row positions are rewritten and the work counters re-zeroed by every call, so nothing depends on what the
    // previous call left in the array
    launch_attn_rows(B, R, seq_len, (int32_t*)scratch, st);
    AttnArgs a{B, R, Hq, Hkv, dh, block_tokens, max_blocks, q, Hq * dh, k_pool, v_pool, block_table,
               (const int32_t*)scratch, out, Hq * dh, dtype, scratch + pos_bytes, kBuiltinScratchBytes - pos_bytes,
               max_blocks * block_tokens, 0};
    return launch_attention(a, st);
}
