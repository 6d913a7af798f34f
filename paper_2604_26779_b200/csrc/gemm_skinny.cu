// C[M][N] (+)= A[M][K] W[N][K]^T for very few rows (M <= 16: the thin tail of a rollout, where a handful of long
// sequences finish alone - paper Section 5.2).  With so few rows a projection is a pure weight-streaming pass and the
// 128-row tensor-core tiles of the main GEMM are padding: it has fewer tiles than SMs and cannot pull the weights at the
// HBM rate.  Here the WEIGHT rows are the M operand of the MMA and the activation rows its (narrow) N operand:
//   * one CTA = 32 weight rows x the whole K; N / 32 CTAs, so even the smallest projection (N = 4096) spreads over 128 CTAs;
//   * stages of 256 k: 32 x 512 contiguous bytes of W (16-byte cp.async, XOR-swizzled) plus the matching slice of A (from L2);
//   * the four warps split each stage's k range (64 each), mma.sync m16n8k16 with fp32 accumulation, and add their partial
//     sums at the end through shared memory in warp order - deterministic, no partials in global memory;
//   * the 32 x M result is written row-contiguously (32 consecutive features per token), fp32 or bf16, optionally added to C.
// The fused epilogues of the main GEMM (rotary + cache append, SwiGLU) are not repeated here: at these sizes the callers use
// the plain projection followed by the small element-wise kernels.
#include "ops.cuh"

namespace spec {
namespace {

constexpr int kRows = 32;            // weight rows per CTA
constexpr int kStageK = 256;         // k per stage: 64 per warp
constexpr int kThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// NT: activation rows in units of 8 (M <= 8 NT).  A stage holds, per warp, a [32 weight rows][64 k] and a [8 NT rows][64 k]
// sub-tile, each row 128 bytes = eight 16-byte chunks, chunk c of row r stored at chunk c ^ (r & 7).
template <int NT, int STAGES>
__global__ void __launch_bounds__(kThreads) gemm_skinny_kernel(int M, int N, int K, const __nv_bfloat16* __restrict__ A, int lda,
                                                               const __nv_bfloat16* __restrict__ W, void* C, int ldc, int out_f32,
                                                               int accumulate)
{
    constexpr int TOK = 8 * NT;
    constexpr int W_SUB = kRows * 128, A_SUB = TOK * 128;
    constexpr int STAGE = 4 * (W_SUB + A_SUB);
    pdl_trigger();
    pdl_wait();
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t base = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * kRows;
    const int n_stages = K / kStageK;

    auto issue = [&](int s) {
        const uint32_t st = base + (uint32_t)(s % STAGES) * STAGE;
        const int k0 = s * kStageK;
        // weights: 32 rows x 32 chunks, consecutive threads on consecutive chunks of a row (512 contiguous bytes)
#pragma unroll
        for (int i = 0; i < kRows * 32 / kThreads; ++i) {
            const int c = i * kThreads + tid, row = c >> 5, kc = c & 31, sub = kc >> 3, cc = kc & 7;
            const bool ok = n0 + row < N;
            cp_async16(st + sub * W_SUB + row * 128 + ((cc ^ (row & 7)) << 4), W + (size_t)(ok ? n0 + row : 0) * K + k0 + kc * 8, ok ? 16 : 0);
        }
        // activations: TOK rows x 32 chunks; rows past M are zero-filled
#pragma unroll
        for (int i = 0; i < (TOK * 32 + kThreads - 1) / kThreads; ++i) {
            const int c = i * kThreads + tid;
            if (c < TOK * 32) {
                const int row = c >> 5, kc = c & 31, sub = kc >> 3, cc = kc & 7;
                const bool ok = row < M;
                cp_async16(st + 4 * W_SUB + sub * A_SUB + row * 128 + ((cc ^ (row & 7)) << 4), A + (size_t)(ok ? row : 0) * lda + k0 + kc * 8,
                           ok ? 16 : 0);
            }
        }
    };

    float acc[2][NT][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { acc[mt][nt][0] = acc[mt][nt][1] = acc[mt][nt][2] = acc[mt][nt][3] = 0.f; }

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) { if (s < n_stages) issue(s); cp_async_commit(); }

    for (int s = 0; s < n_stages; ++s) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        if (s + STAGES - 1 < n_stages) issue(s + STAGES - 1);
        cp_async_commit();
        const uint32_t st = base + (uint32_t)(s % STAGES) * STAGE;
        const uint32_t wsub = st + warp * W_SUB, asub = st + 4 * W_SUB + warp * A_SUB;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {                     // 16-wide k steps of this warp's 64
            uint32_t a[2][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const int row = mt * 16 + (lane & 15), ch = 2 * ks + (lane >> 4);
                ldmatrix_x4(a[mt], wsub + row * 128 + ((ch ^ (row & 7)) << 4));
            }
            if constexpr (NT == 1) {
                uint32_t b[2];
                const int row = lane & 7, ch = 2 * ks + ((lane >> 3) & 1);
                ldmatrix_x2(b, asub + row * 128 + ((ch ^ (row & 7)) << 4));
                mma_bf16(acc[0][0], a[0], b[0], b[1]);
                mma_bf16(acc[1][0], a[1], b[0], b[1]);
            } else {
#pragma unroll
                for (int np = 0; np < NT / 2; ++np) {        // two 8-row n-tiles per load
                    uint32_t b[4];
                    const int row = np * 16 + ((lane >> 4) << 3) + (lane & 7), ch = 2 * ks + ((lane >> 3) & 1);
                    ldmatrix_x4(b, asub + row * 128 + ((ch ^ (row & 7)) << 4));
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        mma_bf16(acc[mt][2 * np], a[mt], b[0], b[1]);
                        mma_bf16(acc[mt][2 * np + 1], a[mt], b[2], b[3]);
                    }
                }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();                                         // the stages are free: reuse them for the reduction over the warps

    float* red = reinterpret_cast<float*>(smem);             // [4 warps][32 rows][TOK]
    const int g4 = lane >> 2, q4 = lane & 3;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int row = mt * 16 + g4 + 8 * (e >> 1), tok = nt * 8 + 2 * q4 + (e & 1);
                red[((size_t)warp * kRows + row) * TOK + tok] = acc[mt][nt][e];
            }
    __syncthreads();
    const int row = tid & 31;
    if (n0 + row < N) {
        for (int tok = tid >> 5; tok < M; tok += kThreads / 32) {
            float v = red[((size_t)0 * kRows + row) * TOK + tok];
#pragma unroll
            for (int w = 1; w < 4; ++w) v += red[((size_t)w * kRows + row) * TOK + tok];
            const size_t at = (size_t)tok * ldc + n0 + row;
            if (out_f32) {
                float* c = static_cast<float*>(C);
                c[at] = accumulate ? c[at] + v : v;
            } else {
                __nv_bfloat16* c = static_cast<__nv_bfloat16*>(C);
                c[at] = __float2bfloat16_rn(accumulate ? __bfloat162float(c[at]) + v : v);
            }
        }
    }
}

template <int NT, int STAGES>
spec_status run_skinny(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int out_dtype, int accumulate,
                       cudaStream_t st)
{
    constexpr int smem = STAGES * 4 * (kRows * 128 + 8 * NT * 128);
    auto kern = gemm_skinny_kernel<NT, STAGES>;
    static PerDeviceOnce configured;
    int dev__ = 0;
    if (configured.needed(&dev__)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SPEC_ERR_CUDA;
        configured.done(dev__);
    }
    launch_pdl(kern, dim3((N + kRows - 1) / kRows), dim3(kThreads), (size_t)smem, st, M, N, K, (const __nv_bfloat16*)A, lda,
               (const __nv_bfloat16*)W, C, ldc, out_dtype == SPEC_DTYPE_F32 ? 1 : 0, accumulate);
    return launch_status();
}

}  // namespace

bool gemm_skinny_supported(int M, int N, int K, const void* A, int lda, const void* W, int dtype_in)
{
    // (17..32 rows measured slower than the tensor-core tile kernel in two forms - 32 weight rows per CTA, and 64 rows with two
    // CTAs of a cluster splitting K: at four token tiles per weight tile the legacy MMA path no longer hides behind the stream)
    return dtype_in == SPEC_DTYPE_BF16 && M >= 1 && M <= 16 && K >= kStageK && K % kStageK == 0 && lda % 8 == 0 && N >= 1 &&
           (reinterpret_cast<uintptr_t>(A) & 15u) == 0 && (reinterpret_cast<uintptr_t>(W) & 15u) == 0;
}

spec_status launch_gemm_skinny(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int out_dtype,
                               int accumulate, cudaStream_t st)
{
    if (M <= 8) return run_skinny<1, 4>(M, N, K, A, lda, W, C, ldc, out_dtype, accumulate, st);
    if (M <= 16) return run_skinny<2, 4>(M, N, K, A, lda, W, C, ldc, out_dtype, accumulate, st);
    return SPEC_ERR_UNSUPPORTED;                            // callers ask gemm_skinny_supported first
}

}  // namespace spec
