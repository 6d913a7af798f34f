// Plain SIMT GEMM  C[M][N] (+)= A[M][K] * W[N][K]^T  with fp32 accumulation, for fp32 models (where the reference
// precision is fp32 and the shapes are tiny) and as the fallback for shapes the tensor-core kernel does not take.
#include "ops.cuh"

namespace spec {
namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <class TA, class TW, class TC>
__global__ void __launch_bounds__(256) gemm_simt_kernel(int M, int N, int K, const TA* __restrict__ A, int lda,
                                                        const TW* __restrict__ W, TC* __restrict__ C, int ldc,
                                                        int accumulate)
{
    __shared__ float sA[TK][TM + 1];
    __shared__ float sW[TK][TN + 1];
    const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;      // 16 x 16 threads, 4 x 4 outputs each
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += TK) {
        for (int i = threadIdx.x; i < TM * TK; i += 256) {
            const int r = i / TK, c = i % TK;
            const int gm = m0 + r, gk = k0 + c;
            sA[c][r] = (gm < M && gk < K) ? to_f32(A[(size_t)gm * lda + gk]) : 0.f;
        }
        for (int i = threadIdx.x; i < TN * TK; i += 256) {
            const int r = i / TK, c = i % TK;
            const int gn = n0 + r, gk = k0 + c;
            sW[c][r] = (gn < N && gk < K) ? to_f32(W[(size_t)gn * K + gk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = sA[kk][ty * 4 + i]; w[i] = sW[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            TC* c = C + (size_t)gm * ldc + gn;
            const float v = accumulate ? acc[i][j] + to_f32(*c) : acc[i][j];
            *c = from_f32<TC>(v);
        }
    }
}

template <class TI>
spec_status run(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int out_dtype,
                int accumulate, cudaStream_t st)
{
    const dim3 grid((N + TN - 1) / TN, (M + TM - 1) / TM);
    if (out_dtype == SPEC_DTYPE_F32)
        gemm_simt_kernel<TI, TI, float><<<grid, 256, 0, st>>>(M, N, K, (const TI*)A, lda, (const TI*)W, (float*)C, ldc, accumulate);
    else
        gemm_simt_kernel<TI, TI, __nv_bfloat16><<<grid, 256, 0, st>>>(M, N, K, (const TI*)A, lda, (const TI*)W, (__nv_bfloat16*)C, ldc, accumulate);
    return launch_status();
}

}  // namespace

spec_status launch_gemm_simt(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int dtype_in,
                             int out_dtype, int accumulate, cudaStream_t st)
{
    if (M == 0 || N == 0) return SPEC_OK;
    if (dtype_in == SPEC_DTYPE_F32) return run<float>(M, N, K, A, lda, W, C, ldc, out_dtype, accumulate, st);
    return run<__nv_bfloat16>(M, N, K, A, lda, W, C, ldc, out_dtype, accumulate, st);
}

}  // namespace spec

