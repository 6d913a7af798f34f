// Paged grouped-query attention over an 8-bit (e4m3) KV cache, up to 16 query rows per KV head, head_dim 128.
//
// The cache holds one byte per element (code = round_e4m3(x / scale), one scale for keys and one for values), so the pass
// that dominates a verify forward moves half the bytes.  The kernel is the register-fragment kernel of the bf16 cache
// with the fragments taken straight from the code tiles: tiles of codes arrive by 16-byte cp.async (stages of 16 KB,
// 16-byte chunks XOR-swizzled by token), ldmatrix reads them as if two codes were one 16-bit element, and the codes are
// converted to fp16 - exactly - in registers; both MMAs run in fp16 (Q converted from bf16 once per unit, P packed to
// fp16) with fp32 accumulation.  Two index permutations make the register contents fit the MMA fragments:
//   keys    a thread's ldmatrix register holds four consecutive head_dim codes of one token, so inside every 16-wide
//           k-block the MMA's k index 2t, 2t+1, 2t+8, 2t+9 is mapped to head_dim 4t .. 4t+3 (Q is loaded the same way);
//   values  the transposing ldmatrix delivers codes (token 2t, dims 2g, 2g+1) and (token 2t+1, dims 2g, 2g+1); a byte
//           permute pairs equal dims of the two tokens, which makes one MMA n-tile the even dims of a 16-wide block and
//           the next one the odd dims; the accumulator columns are put back in order when the result is written.
// The scales never touch the tile: the key scale multiplies the softmax scale, the value scale the final normalisation.
// Work units, the atomic work counter and the merge pass are the bf16 kernel's.
#include <cuda_fp16.h>

#include "attention_plan.cuh"

namespace spec {
namespace attn {
namespace {

constexpr int kThreads = 128;

struct Fp8Args {
    const __nv_bfloat16* q; int q_row_stride;
    const unsigned char* k_pool; const unsigned char* v_pool;
    const int32_t* block_table; int max_blocks;
    const int32_t* pos;
    int R, group, Hkv;
    __nv_bfloat16* out; int out_row_stride;
    float scale_log2;                  // log2(e) / sqrt(head_dim) * key scale
    float v_scale;
    PlanView pv;
    int counter_index;
};

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
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w)
{
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&w);
    return pack_f16(__low2float(b), __high2float(b));
}
// four e4m3 codes (one 32-bit word, lowest address first) -> four fp16 values as two pairs
__device__ __forceinline__ void e4m3x4_to_f16x4(uint32_t w, uint32_t& lo, uint32_t& hi)
{
    const unsigned short a = (unsigned short)(w & 0xffffu), b = (unsigned short)(w >> 16);
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(lo) : "h"(a));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(hi) : "h"(b));
}
// One CTA = 4 warps, each taking one 16-token block of every 64-token tile (16 query rows per KV head at most).
template <int STAGES>
__global__ void __launch_bounds__(kThreads, 4) attn_fp8_kernel(const Fp8Args a)
{
    constexpr int DH = 128, WM = 1, WN = 4;
    constexpr int kCodeBlk = kBT * DH;                       // the same block as e4m3 codes
    constexpr int kStageBytes = 4 * kCodeBlk * 2;            // 4 blocks, K and V, as codes
    constexpr int ROWS = 16 * WM;
    constexpr int NT_O = DH / 8;                             // output n-tiles per warp
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ int s_unit;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wm = warp / WN, wn = warp % WN;
    const int g4 = lane >> 2, q4 = lane & 3;
    const uint32_t smem_base = smem_u32(smem);
    const int n_rows_valid = a.R * a.group;

    for (;;) {
        if (tid == 0) s_unit = atomicAdd(&a.pv.counters[a.counter_index], 1);
        __syncthreads();
        const int u = s_unit;
        const int n_units = *a.pv.n_entries * a.Hkv;
        if (u >= n_units) break;
        const Unit un = a.pv.entries[u / a.Hkv];
        const int g = u % a.Hkv, b = un.b, t0 = un.t0, t1 = un.t1;
        const int32_t* table = a.block_table + (size_t)b * a.max_blocks;

        // per-thread row limits (rows r0 = 16 wm + g4 and r0 + 8): last visible cache position of the row
        int lim[2];
        uint32_t qf[DH / 16][4];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = 16 * wm + g4 + 8 * hh;
            const bool valid = r < n_rows_valid;
            const int i = valid ? r / a.group : 0, j = valid ? r % a.group : 0;
            lim[hh] = valid ? a.pos[(size_t)b * a.R + i] : 0x7fffffff;
            const __nv_bfloat16* qp = a.q + ((size_t)b * a.R + i) * a.q_row_stride + (size_t)(g * a.group + j) * DH;
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
                // A fragment under the key permutation: regs {hh, hh+2} hold (row, head_dim 16 ks + 4 q4 + {0,1}) and (+ {2,3})
                qf[ks][hh] = valid ? bf16x2_to_f16x2(*reinterpret_cast<const uint32_t*>(qp + 16 * ks + 4 * q4)) : 0u;
                qf[ks][hh + 2] = valid ? bf16x2_to_f16x2(*reinterpret_cast<const uint32_t*>(qp + 16 * ks + 4 * q4 + 2)) : 0u;
            }
        }
        int min_lim = min(lim[0], lim[1]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) min_lim = min(min_lim, __shfl_xor_sync(0xffffffffu, min_lim, o));

        float o_acc[NT_O][4];
#pragma unroll
        for (int n = 0; n < NT_O; ++n) { o_acc[n][0] = o_acc[n][1] = o_acc[n][2] = o_acc[n][3] = 0.f; }
        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

        const int n_tiles = (t1 - t0 + kTileTok - 1) / kTileTok;
        auto issue_tile = [&](int j) {
            const uint32_t stage = smem_base + (uint32_t)(j % STAGES) * kStageBytes;
            const int blk0 = (t0 + j * kTileTok) / kBT;
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) {
                const int bi = blk0 + bb;
                const int phys = (bi * kBT < t1 && bi < a.max_blocks) ? table[bi] : -1;
                const size_t goff = ((size_t)(phys < 0 ? 0 : phys) * a.Hkv + g) * (size_t)kCodeBlk;      // bytes
                const int nbytes = phys < 0 ? 0 : 16;
                // 128 chunks of 16 codes per block: one per thread and tensor
                const uint32_t soff = (uint32_t)(bb * kCodeBlk + (tid >> 3) * 128 + (((tid & 7) ^ ((tid >> 3) & 7)) << 4));   // token tid/8, chunk tid%8
                cp_async16(stage + soff, a.k_pool + goff + (size_t)tid * 16, nbytes);
                cp_async16(stage + 4 * kCodeBlk + soff, a.v_pool + goff + (size_t)tid * 16, nbytes);
            }
        };

#pragma unroll
        for (int j = 0; j < STAGES - 1; ++j) { if (j < n_tiles) issue_tile(j); cp_async_commit(); }

        for (int j = 0; j < n_tiles; ++j) {
            cp_async_wait<STAGES - 2>();
            __syncthreads();
            if (j + STAGES - 1 < n_tiles) issue_tile(j + STAGES - 1);
            cp_async_commit();
            const uint32_t stage = smem_base + (uint32_t)(j % STAGES) * kStageBytes;
#pragma unroll
            for (int bb = wn; bb < 4; bb += WN) {
                const int tok0 = t0 + j * kTileTok + bb * kBT;
                if (tok0 >= t1) continue;
                const uint32_t kb_base = stage + bb * kCodeBlk, vb_base = kb_base + 4 * kCodeBlk;
                // this lane's row of the four 8 x 8 matrices an ldmatrix.x4 reads: matrix m = lane / 8 covers tokens
                // (m & 1) * 8 .. + 7 and the 16-code chunk (first chunk of the pair) + (m >> 1)
                const int l_tok = ((lane >> 3) & 1) * 8 + (lane & 7), l_chunk = lane >> 4;
                // S = Q K^T for 16 tokens
                float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                for (int kp = 0; kp < DH / 32; ++kp) {               // two 16-wide k-blocks per load
                    uint32_t kb[4];
                    ldmatrix_x4(kb, kb_base + l_tok * 128 + (((2 * kp + l_chunk) ^ (l_tok & 7)) << 4));
                    uint32_t b0, b1;
                    e4m3x4_to_f16x4(kb[0], b0, b1); mma_f16(s[0], qf[2 * kp], b0, b1);          // tokens 0..7, k-block 2 kp
                    e4m3x4_to_f16x4(kb[1], b0, b1); mma_f16(s[1], qf[2 * kp], b0, b1);          // tokens 8..15
                    e4m3x4_to_f16x4(kb[2], b0, b1); mma_f16(s[0], qf[2 * kp + 1], b0, b1);      // k-block 2 kp + 1
                    e4m3x4_to_f16x4(kb[3], b0, b1); mma_f16(s[1], qf[2 * kp + 1], b0, b1);
                }
                // causal limit of the new rows and the end of this unit's range
                if (tok0 + kBT - 1 > min_lim || tok0 + kBT > t1) {
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int t = tok0 + 8 * nt + 2 * q4 + (e & 1);
                            if (t > lim[e >> 1] || t >= t1) s[nt][e] = -INFINITY;
                        }
                }
                // online softmax (exp2 domain)
                float mx[2];
                mx[0] = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
                mx[1] = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
                    mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
                    mx[hh] *= a.scale_log2;          // scale > 0, -inf stays -inf
                }
                const bool grow = mx[0] > m_run[0] || mx[1] > m_run[1];
                if (__any_sync(0xffffffffu, grow)) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const float mnew = fmaxf(m_run[hh], mx[hh]);
                        const float alpha = (mnew == -INFINITY) ? 1.f : exp2f(m_run[hh] - mnew);
                        m_run[hh] = mnew;
                        l_run[hh] *= alpha;
#pragma unroll
                        for (int n = 0; n < NT_O; ++n) { o_acc[n][2 * hh] *= alpha; o_acc[n][2 * hh + 1] *= alpha; }
                    }
                }
                const float ms0 = m_run[0] == -INFINITY ? 0.f : m_run[0], ms1 = m_run[1] == -INFINITY ? 0.f : m_run[1];
                uint32_t pf[4];
                {
                    float p[2][4];
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        p[nt][0] = exp2f(fmaf(s[nt][0], a.scale_log2, -ms0));
                        p[nt][1] = exp2f(fmaf(s[nt][1], a.scale_log2, -ms0));
                        p[nt][2] = exp2f(fmaf(s[nt][2], a.scale_log2, -ms1));
                        p[nt][3] = exp2f(fmaf(s[nt][3], a.scale_log2, -ms1));
                        l_run[0] += p[nt][0] + p[nt][1];
                        l_run[1] += p[nt][2] + p[nt][3];
                    }
                    pf[0] = pack_f16(p[0][0], p[0][1]);
                    pf[1] = pack_f16(p[0][2], p[0][3]);
                    pf[2] = pack_f16(p[1][0], p[1][1]);
                    pf[3] = pack_f16(p[1][2], p[1][3]);
                }
                // O += P V: per 32 head dims one transposing load; even dims and odd dims of a 16-wide block are two n-tiles
#pragma unroll
                for (int dp = 0; dp < DH / 32; ++dp) {
                    uint32_t vb[4];
                    ldmatrix_x4_trans(vb, vb_base + l_tok * 128 + (((2 * dp + l_chunk) ^ (l_tok & 7)) << 4));
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2) {                  // block 2 dp + h2: registers vb[2 h2] (tokens 0..7) and vb[2 h2 + 1] (8..15)
                        uint32_t b0, b1;
                        e4m3x4_to_f16x4(__byte_perm(vb[2 * h2], vb[2 * h2 + 1], 0x6420), b0, b1);
                        mma_f16(o_acc[2 * (2 * dp + h2)], pf, b0, b1);                       // even dims
                        e4m3x4_to_f16x4(__byte_perm(vb[2 * h2], vb[2 * h2 + 1], 0x7531), b0, b1);
                        mma_f16(o_acc[2 * (2 * dp + h2) + 1], pf, b0, b1);                   // odd dims
                    }
                }
            }
        }
        cp_async_wait<0>();
        __syncthreads();                                   // every warp is done with the stages: reuse them for the merge

        // row sums across the quad
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
            l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
        }
        float* mrg_o = reinterpret_cast<float*>(smem);                      // [WN][ROWS][DH]
        float* mrg_ml = mrg_o + WN * ROWS * DH;                             // [WN][ROWS][2]
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = 16 * wm + g4 + 8 * hh;
            float* orow = mrg_o + ((size_t)wn * ROWS + r) * DH;
#pragma unroll
            for (int d = 0; d < NT_O / 2; ++d)        // block d: n-tile 2d holds dims 16 d + 4 q4 + {0, 2}, n-tile 2d + 1 the dims + {1, 3}
                *reinterpret_cast<float4*>(orow + 16 * d + 4 * q4) =
                    make_float4(o_acc[2 * d][2 * hh], o_acc[2 * d + 1][2 * hh], o_acc[2 * d][2 * hh + 1], o_acc[2 * d + 1][2 * hh + 1]);
            if (q4 == 0) { mrg_ml[((size_t)wn * ROWS + r) * 2] = m_run[hh]; mrg_ml[((size_t)wn * ROWS + r) * 2 + 1] = l_run[hh]; }
        }
        __syncthreads();
        const int slot = un.slot;
        for (int e = tid; e < ROWS * (DH / 4); e += kThreads) {
            const int r = e / (DH / 4), c4 = (e % (DH / 4)) * 4;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < WN; ++w) M = fmaxf(M, mrg_ml[((size_t)w * ROWS + r) * 2]);
            float L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int w = 0; w < WN; ++w) {
                const float mw = mrg_ml[((size_t)w * ROWS + r) * 2];
                const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
                L += mrg_ml[((size_t)w * ROWS + r) * 2 + 1] * f;
                const float4 v = *reinterpret_cast<const float4*>(mrg_o + ((size_t)w * ROWS + r) * DH + c4);
                acc[0] += v.x * f; acc[1] += v.y * f; acc[2] += v.z * f; acc[3] += v.w * f;
            }
            if (slot >= 0) {
                const size_t ps = (size_t)slot * a.Hkv + g;
                *reinterpret_cast<float4*>(a.pv.part_o + (ps * ROWS + r) * DH + c4) =
                    make_float4(acc[0] * a.v_scale, acc[1] * a.v_scale, acc[2] * a.v_scale, acc[3] * a.v_scale);
                if (c4 == 0) { a.pv.part_ml[(ps * ROWS + r) * 2] = M; a.pv.part_ml[(ps * ROWS + r) * 2 + 1] = L; }
            } else if (r < n_rows_valid) {
                const float inv = L > 0.f ? a.v_scale / L : 0.f;
                const int i = r / a.group, j = r % a.group;
                __nv_bfloat16* op = a.out + ((size_t)b * a.R + i) * a.out_row_stride + (size_t)(g * a.group + j) * DH + c4;
                uint2 pk;
                pk.x = pack_bf16(acc[0] * inv, acc[1] * inv);
                pk.y = pack_bf16(acc[2] * inv, acc[3] * inv);
                *reinterpret_cast<uint2*>(op) = pk;
            }
        }
        __syncthreads();
    }
}


}  // namespace

bool attention_fp8_supported(const AttnArgs& a)
{
    const int rows = a.R * (a.Hq / a.Hkv);
    return a.kv_fp8 && a.dtype == SPEC_DTYPE_BF16 && a.block_tokens == kBT && a.dh == 128 && rows <= 16 &&
           a.q_row_stride % 2 == 0 && a.out_row_stride % 4 == 0 && a.k_scale > 0.f && a.v_scale > 0.f;
}

spec_status launch_attention_fp8(const AttnArgs& a, cudaStream_t st)
{
    constexpr int STAGES = 3;
    constexpr int kStages = STAGES * (4 * kBT * 128 * 2), kMerge = 4 * 16 * 130 * 4;
    constexpr int smem = kStages > kMerge ? kStages : kMerge;      // code stages; the unit-end merge of the four warps reuses them
    const int group = a.Hq / a.Hkv;
    if (a.scratch_bytes < attention_mma_scratch_bytes(a.B, a.R, a.Hq, a.Hkv, a.dh, a.max_kv_len)) return SPEC_ERR_SHAPE;
    const int max_chunks = max_chunks_for(a.max_kv_len);
    const PlanView pv = carve_plan(a.scratch, a.B, a.Hkv, 16, a.dh, max_chunks);
    auto kern = attn_fp8_kernel<STAGES>;
    static PerDeviceOnce configured;
    int dev__ = 0;
    if (configured.needed(&dev__)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SPEC_ERR_CUDA;
        configured.done(dev__);
    }
    Fp8Args f{(const __nv_bfloat16*)a.q, a.q_row_stride, (const unsigned char*)a.k_pool, (const unsigned char*)a.v_pool,
              a.block_table, a.max_blocks, a.pos, a.R, group, a.Hkv, (__nv_bfloat16*)a.out, a.out_row_stride,
              1.4426950408889634f / sqrtf((float)a.dh) * a.k_scale, a.v_scale, pv, a.launch_index % kCounters};
    if (a.launch_index % kCounters == 0) {
        const spec_status s = launch_attn_plan(a.B, a.R, a.pos, a.Hkv, 4 * 148, max_chunks, pv, st);
        if (s != SPEC_OK) return s;
    }
    int sms = 0, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
    const int ctas_per_sm = (228 * 1024) / (smem + 2048);
    kern<<<sms * (ctas_per_sm < 1 ? 1 : ctas_per_sm), kThreads, smem, st>>>(f);
    if (launch_status() != SPEC_OK) return SPEC_ERR_CUDA;
    return launch_attn_merge128(a.B, 16, a.Hkv, a.R, group, a.out, a.out_row_stride, pv, st);
}

}  // namespace attn
}  // namespace spec
