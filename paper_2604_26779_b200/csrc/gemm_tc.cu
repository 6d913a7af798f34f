// bf16 GEMM on the 5th-generation tensor cores:  C[M][N] (+)= A[M][K] * W[N][K]^T, fp32 accumulation.
//
// The projections of the verify forward (QKV, O, gate/up, down, LM head) are dense contractions with M = B(k+1)
// rows, far above the ridge point, so they run on tcgen05:
//   - persistent CTAs, one per SM, walk 128 x 256 output tiles (tiles that share a weight tile run side by side, so
//     the weight tile crosses HBM once and the activations stay in L2);
//   - warp 0 streams A and W tiles of 64 k-columns with TMA (cp.async.bulk.tensor, 128-byte swizzle) into a 4-stage
//     shared-memory ring, signalled by mbarriers;
//   - warp 1 issues tcgen05.mma (M=128, N=256, K=16 per instruction) from one thread; the fp32 accumulator lives in
//     tensor memory, double-buffered (2 x 256 columns) so the epilogue of one tile overlaps the next tile's loads;
//   - warps 2-9 read the accumulator with tcgen05.ld (two warps per 32-lane quarter, half of the columns each) and store
//     fp32 / bf16, optionally adding to the fp32 residual stream; the epilogue is a serial ld -> convert -> store chain per
//     32 columns, so its length is what eight warps instead of four buy.
// Every mbarrier wait is bounded: on a timeout the CTA raises a flag, all roles leave their loops, outstanding
// tensor-core work is drained with a bounded wait, tensor memory is released and the kernel returns with
// SPEC_ERR_TIMEOUT in the status word.
#include <cuda.h>

#include "ops.cuh"
#include "tc_common.cuh"

namespace spec {
using namespace tc;
namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int kThreads = 320;          // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue (two per tensor-memory lane quarter)
constexpr int kEpiThreads = 256;
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxGroups = 256;          // grouped mode: most groups per launch
constexpr int kOutStageBytes = 32 * 128;  // per epilogue warp: 32 rows x 128 bytes, where a warp turns its row-per-thread
                                          // accumulator fragments into row-contiguous 128-byte pieces before they go to memory
constexpr int kSmemBytes = STAGES * STAGE_BYTES + (kEpiThreads / 32) * kOutStageBytes + 1024 + 128 + (kMaxGroups + 1) * 4;
static_assert(kSmemBytes <= 232448, "shared memory per CTA");
#define TRY_LAUNCH(expr) do { spec_status s__ = (expr); if (s__ != SPEC_OK) return s__; } while (0)

struct Ctl {
    uint64_t full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], drain;
    uint32_t tmem_base;
    int abort;
    int pref[kMaxGroups + 1];          // grouped mode: m-tiles of the groups before group e (pref[E] = all m-tiles)
};

// Shared-memory matrix descriptor of a K-major tile whose rows are 64 bf16 (128 bytes) wide, 128-byte swizzle:
// start address >> 4, leading byte offset 1 (unused for swizzled K-major), stride byte offset = 1024 bytes between
// 8-row groups, descriptor version 1, layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
// The same for e4m3 operands (format code 0 for A and B).
constexpr uint32_t kIdescF8 = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

struct TileCoord { int a_row, b_row, c_row, rows_valid, col, kb0, kb1, split; };

struct GemmArgs {
    int M, N, K;
    void* C; int ldc;
    int out_f32, accumulate;
    int32_t* status;
    // grouped mode (E > 0): E independent problems that share K and N.  Group e multiplies rows
    // [offsets[e], offsets[e] + counts[e]) of A by the weight rows [e*N, (e+1)*N) of W; counts/offsets live on the device.
    int E, max_m_tiles;
    const int32_t* counts; const int32_t* offsets;
    // split-K (splits > 1, plain epilogue only): work item = (tile, split); split s covers k-blocks [s*kb_per, (s+1)*kb_per)
    // and stores its fp32 partial at C + s * M * ldc (C is then a scratch buffer; a second kernel sums the splits in order)
    int splits, kb_per;
    // EPI_QKV: rotary embedding on q and k heads, k and v written straight into the paged cache
    int Hq, Hkv, dh, R, max_blocks, block_tokens;
    const int32_t* pos; const int32_t* block_table; const float2* rope;   // rope [dh/2][M] (cos, sin) of each row's position
    __nv_bfloat16* k_pool; __nv_bfloat16* v_pool;
    int kv_fp8; float k_scale, v_scale;           // 8-bit cache: k and v are stored as e4m3 codes of x / scale
    // EPI_THIN (17..64 activation rows): the operands are swapped - the WEIGHT rows are the MMA's M operand (M = features here),
    // the activation rows its N operand (N = tokens <= bn, bn = 32 or 64: one narrow n-tile) - and the epilogue writes the
    // transposed tile, C[token][feature]
    int bn;
    // plain epilogue with fp32 output (an LM head): every (row, 128-column piece) also leaves the pair (max, sum of
    // exp((l - max) * inv_t)) of its logits in stat_part [rows][stat_pairs][2], piece index = 2 * n-tile + column half;
    // a small kernel combines the pairs of a row, so the row statistics cost no second pass over the logits
    float* stat_part; int stat_pairs; float inv_t;
    // 8-bit operands (fp8 != 0): A and W hold e4m3 codes, one byte per element, a k-block is 128 elements (the same 128 bytes
    // per row as 64 bf16), K counts byte PAIRS of a row (elements / 2) so that the k-block arithmetic is unchanged, and every
    // accumulator is multiplied by a_scale[row] * w_scale[weight row] before the epilogue does anything else with it
    int fp8; const float* a_scale; const float* w_scale;
};

enum { EPI_PLAIN = 0, EPI_SWIGLU = 1, EPI_QKV = 2, EPI_THIN = 3 };

__device__ __forceinline__ void store_bf16x32(__nv_bfloat16* dst, const float (&f)[32])
{
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint4 o;
        __nv_bfloat162 t0 = __floats2bfloat162_rn(f[8 * j], f[8 * j + 1]), t1 = __floats2bfloat162_rn(f[8 * j + 2], f[8 * j + 3]);
        __nv_bfloat162 t2 = __floats2bfloat162_rn(f[8 * j + 4], f[8 * j + 5]), t3 = __floats2bfloat162_rn(f[8 * j + 6], f[8 * j + 7]);
        o.x = *reinterpret_cast<uint32_t*>(&t0); o.y = *reinterpret_cast<uint32_t*>(&t1);
        o.z = *reinterpret_cast<uint32_t*>(&t2); o.w = *reinterpret_cast<uint32_t*>(&t3);
        *reinterpret_cast<uint4*>(dst + 8 * j) = o;
    }
}

// 32 consecutive values as e4m3 codes (round to nearest even, saturating), 32 bytes.
__device__ __forceinline__ void store_e4m3x32(unsigned char* dst, const float (&f)[32], float scale)
{
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        unsigned short lo, hi;                       // cvt packs its first source into the upper byte
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(__fdiv_rn(f[4 * j + 1], scale)), "f"(__fdiv_rn(f[4 * j], scale)));
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(__fdiv_rn(f[4 * j + 3], scale)), "f"(__fdiv_rn(f[4 * j + 2], scale)));
        w[j] = (uint32_t)lo | ((uint32_t)hi << 16);
    }
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<uint4*>(dst + 16) = make_uint4(w[4], w[5], w[6], w[7]);
}

// Output staging.  After tcgen05.ld a thread holds 32 consecutive columns of ONE row, so a direct store makes every warp
// instruction touch 32 different lines, 16 bytes each.  Instead each thread writes its 128 bytes into the warp's staging
// area (16-byte pieces XOR-swizzled by the row, conflict-free both ways) and the warp reads it back four rows at a time,
// eight lanes per row: every store (and every residual load) instruction then covers four whole 128-byte lines.
__device__ __forceinline__ void stage_put(uint32_t stage, int lane, int piece, const uint4& v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage + lane * 128 + ((piece ^ (lane & 7)) << 4)),
                 "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 stage_get(uint32_t stage, int row, int piece)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(stage + row * 128 + ((piece ^ (row & 7)) << 4)) : "memory");
    return v;
}
__device__ __forceinline__ uint4 pack_bf16x8(const float* f)
{
    __nv_bfloat162 t0 = __floats2bfloat162_rn(f[0], f[1]), t1 = __floats2bfloat162_rn(f[2], f[3]);
    __nv_bfloat162 t2 = __floats2bfloat162_rn(f[4], f[5]), t3 = __floats2bfloat162_rn(f[6], f[7]);
    return make_uint4(*reinterpret_cast<uint32_t*>(&t0), *reinterpret_cast<uint32_t*>(&t1),
                      *reinterpret_cast<uint32_t*>(&t2), *reinterpret_cast<uint32_t*>(&t3));
}
// The 32 x 128-byte block of the residual that a staged block will be added to: this lane's eight 16-byte pieces.
__device__ __forceinline__ void residual_get(uint4 (&o)[8], int lane, const unsigned char* src, size_t row_stride_bytes, int rows_ok)
{
    const unsigned char* base = src + (lane & 7) * 16;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = i * 4 + (lane >> 3);
        if (r < rows_ok) o[i] = __ldcg(reinterpret_cast<const uint4*>(base + (size_t)r * row_stride_bytes));
    }
}
// Writes the staged 32 x 128-byte block: row r of the block goes to dst + r * row_stride_bytes; rows >= rows_ok are skipped.
// kAddF32: the block is fp32 and o (from residual_get on the same rows) is added first.
template <bool kAddF32>
__device__ __forceinline__ void stage_flush(uint32_t stage, int lane, unsigned char* dst, size_t row_stride_bytes, int rows_ok,
                                            const uint4 (&o)[8])
{
    __syncwarp();
    const int piece = lane & 7, r0 = lane >> 3;
    unsigned char* base = dst + piece * 16;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = i * 4 + r0;
        if (r < rows_ok) {
            uint4 v = stage_get(stage, r, piece);
            if (kAddF32) {
                v.x = __float_as_uint(__uint_as_float(v.x) + __uint_as_float(o[i].x));
                v.y = __float_as_uint(__uint_as_float(v.y) + __uint_as_float(o[i].y));
                v.z = __float_as_uint(__uint_as_float(v.z) + __uint_as_float(o[i].z));
                v.w = __float_as_uint(__uint_as_float(v.w) + __uint_as_float(o[i].w));
            }
            *reinterpret_cast<uint4*>(base + (size_t)r * row_stride_bytes) = v;
        }
    }
    __syncwarp();
}
__device__ __forceinline__ void stage_flush(uint32_t stage, int lane, unsigned char* dst, size_t row_stride_bytes, int rows_ok)
{
    uint4 none[8];
    stage_flush<false>(stage, lane, dst, row_stride_bytes, rows_ok, none);
}

// 8-bit operands: accumulator columns [w0, w0 + 32) of this thread's row times the row's activation scale and the weight
// rows' scales (weight rows past n_w get 0).
__device__ __forceinline__ void scale32(const GemmArgs& g, uint32_t (&v)[32], float row_scale, int w0, int n_w)
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float4 ws = make_float4(0.f, 0.f, 0.f, 0.f);
        if (w0 + 4 * j + 3 < n_w) ws = __ldg(reinterpret_cast<const float4*>(g.w_scale + w0) + j);
        else {
            if (w0 + 4 * j < n_w) ws.x = g.w_scale[w0 + 4 * j];
            if (w0 + 4 * j + 1 < n_w) ws.y = g.w_scale[w0 + 4 * j + 1];
            if (w0 + 4 * j + 2 < n_w) ws.z = g.w_scale[w0 + 4 * j + 2];
        }
        v[4 * j] = __float_as_uint(__uint_as_float(v[4 * j]) * (row_scale * ws.x));
        v[4 * j + 1] = __float_as_uint(__uint_as_float(v[4 * j + 1]) * (row_scale * ws.y));
        v[4 * j + 2] = __float_as_uint(__uint_as_float(v[4 * j + 2]) * (row_scale * ws.z));
        v[4 * j + 3] = __float_as_uint(__uint_as_float(v[4 * j + 3]) * (row_scale * ws.w));
    }
}

// Plain epilogue: C (+)= accumulator, fp32 or bf16, ragged N handled element-wise.
__device__ __forceinline__ void epilogue_plain(const GemmArgs& g, const TileCoord& tc, uint32_t t_row, int row, bool row_ok, int half,
                                               uint32_t stage, int lane, int rows_ok, uint4 (&resid)[8])
{
    // resid (fp32 output added to what C holds, whole 32-column blocks): the residual block of the first 32 columns, loaded by the caller before it
    // waited for the accumulator; each later block is requested as soon as the previous one has been stored
    const int row0 = row - lane;                            // first row of this warp's 32
    float sm = -INFINITY, sz = 0.f;                         // running (max, sum of exponentials) of this row's piece
#pragma unroll 1
    for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
        const int col = tc.col + c0;
        if (col >= g.N) break;                              // warp-uniform
        uint32_t v[32];
        tc_ld32(t_row + c0, v);
        if (!g.out_f32 && !g.accumulate && col + 64 <= g.N) {          // bf16: 64 columns = 128 bytes per row
            uint32_t v2[32];
            tc_ld32(t_row + c0 + 32, v2);
            tc_wait_ld();
            if (g.fp8) { const float rs = row_ok ? g.a_scale[row] : 0.f; const int wo = tc.b_row - tc.col; scale32(g, v, rs, wo + col, wo + g.N); scale32(g, v2, rs, wo + col + 32, wo + g.N); }
            float f[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[8 * j + e]);
                stage_put(stage, lane, j, pack_bf16x8(f));
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v2[8 * j + e]);
                stage_put(stage, lane, 4 + j, pack_bf16x8(f));
            }
            stage_flush(stage, lane, reinterpret_cast<unsigned char*>(static_cast<__nv_bfloat16*>(g.C) + (size_t)row0 * g.ldc + col),
                               (size_t)g.ldc * 2, rows_ok);
            c0 += 32;
            continue;
        }
        tc_wait_ld();
        if (g.fp8) scale32(g, v, row_ok ? g.a_scale[row] : 0.f, tc.b_row - tc.col + col, tc.b_row - tc.col + g.N);   // grouped: the group's weight rows
        if (g.stat_part != nullptr) {
            float cm = -INFINITY;
#pragma unroll
            for (int e = 0; e < 32; ++e) if (col + e < g.N) cm = fmaxf(cm, __uint_as_float(v[e]));
            if (cm > sm) { sz *= __expf(__fmul_rn(__fsub_rn(sm, cm), g.inv_t)); sm = cm; }
#pragma unroll
            for (int e = 0; e < 32; ++e) if (col + e < g.N) sz += __expf(__fmul_rn(__fsub_rn(__uint_as_float(v[e]), sm), g.inv_t));
        }
        if (g.out_f32 && col + 32 <= g.N) {                 // fp32: 32 columns = 128 bytes per row
#pragma unroll
            for (int j = 0; j < 8; ++j) stage_put(stage, lane, j, make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]));
            unsigned char* dst = reinterpret_cast<unsigned char*>(static_cast<float*>(g.C) + (size_t)row0 * g.ldc + col);
            if (g.accumulate) {
                stage_flush<true>(stage, lane, dst, (size_t)g.ldc * 4, rows_ok, resid);
                if (c0 + 32 < (half + 1) * (BN / 2) && col + 64 <= g.N) residual_get(resid, lane, dst + 128, (size_t)g.ldc * 4, rows_ok);
            } else {
                stage_flush(stage, lane, dst, (size_t)g.ldc * 4, rows_ok);
            }
            continue;
        }
        if (!row_ok) continue;
        if (g.out_f32) {
            float* cp = static_cast<float*>(g.C) + (size_t)row * g.ldc + col;
            if (col + 32 <= g.N) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float4 o = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                           __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                    if (g.accumulate) {
                        const float4 p = *reinterpret_cast<const float4*>(cp + 4 * j);
                        o.x += p.x; o.y += p.y; o.z += p.z; o.w += p.w;
                    }
                    *reinterpret_cast<float4*>(cp + 4 * j) = o;
                }
            } else {
                for (int j = 0; j < 32 && col + j < g.N; ++j)
                    cp[j] = __uint_as_float(v[j]) + (g.accumulate ? cp[j] : 0.f);
            }
        } else {
            __nv_bfloat16* cp = static_cast<__nv_bfloat16*>(g.C) + (size_t)row * g.ldc + col;
            if (col + 32 <= g.N) {
                float f[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
                if (g.accumulate) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint4 p = *reinterpret_cast<const uint4*>(cp + 8 * j);
                        const __nv_bfloat162* pp = reinterpret_cast<const __nv_bfloat162*>(&p);
#pragma unroll
                        for (int e = 0; e < 4; ++e) { f[8 * j + 2 * e] += __low2float(pp[e]); f[8 * j + 2 * e + 1] += __high2float(pp[e]); }
                    }
                }
                store_bf16x32(cp, f);
            } else {
                for (int j = 0; j < 32 && col + j < g.N; ++j)
                    cp[j] = __float2bfloat16_rn(__uint_as_float(v[j]) + (g.accumulate ? __bfloat162float(cp[j]) : 0.f));
            }
        }
    }
    if (g.stat_part != nullptr && row_ok) {
        float* sp = g.stat_part + ((size_t)row * g.stat_pairs + 2 * (tc.col / BN) + half) * 2;
        sp[0] = sm; sp[1] = sz;
    }
}

// SwiGLU epilogue: the tile's first 128 columns are gate rows, the last 128 the matching up rows (the stacked weight is
// stored in such 256-row groups); writes act = silu(gate) * up, bf16, [rows][N/2].
__device__ __forceinline__ void epilogue_swiglu(const GemmArgs& g, const TileCoord& tc, uint32_t t_row, int row, bool row_ok, int half,
                                                uint32_t stage, int lane, int rows_ok)
{
    static_assert(BN / 4 == 64, "one staging pass per warp: 64 bf16 outputs = 128 bytes per row");
    const int c_base = half * (BN / 4);
#pragma unroll
    for (int part = 0; part < 2; ++part) {
        const int c0 = c_base + 32 * part;
        uint32_t gv[32], uv[32];
        tc_ld32(t_row + c0, gv);
        tc_ld32(t_row + BN / 2 + c0, uv);
        tc_wait_ld();
        if (g.fp8) {
            const float rs = row_ok ? g.a_scale[row] : 0.f;
            scale32(g, gv, rs, tc.b_row + c0, 0x7fffffff);
            scale32(g, uv, rs, tc.b_row + BN / 2 + c0, 0x7fffffff);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float a = __uint_as_float(gv[8 * j + e]);
                f[e] = a / (1.f + __expf(-a)) * __uint_as_float(uv[8 * j + e]);
            }
            stage_put(stage, lane, 4 * part + j, pack_bf16x8(f));
        }
    }
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(g.C) + (size_t)(row - lane) * g.ldc + tc.col / 2 + c_base;
    stage_flush(stage, lane, reinterpret_cast<unsigned char*>(out), (size_t)g.ldc * 2, rows_ok);
}

// QKV epilogue: heads of width dh; q and k heads get the rotary embedding (pairs (j, j + dh/2)); q goes to C (bf16,
// [rows][N]), k and v go to the paged cache slot of the row's position.  Rows with a negative position write nothing.
__device__ __forceinline__ void epilogue_qkv(const GemmArgs& g, const TileCoord& tc, uint32_t t_row, int row, bool row_ok, int part,
                                             uint32_t stage, int lane)
{
    const int half = g.dh / 2;
    int p = -1, blk = -1, slot = 0;
    if (row_ok) {
        p = g.pos[row];
        if (p >= 0) { blk = g.block_table[(size_t)(row / g.R) * g.max_blocks + p / g.block_tokens]; slot = p % g.block_tokens; }
    }
    const float2* cs = g.rope + (row_ok ? row : 0);                      // table is [dh/2][M]: element j of this row at cs[j * M]
#pragma unroll 1
    for (int hb = part * (BN / 2); hb < (part + 1) * (BN / 2); hb += g.dh) {   // this warp's heads inside the tile
        const int col = tc.col + hb;
        if (col >= g.N) break;                                           // warp-uniform
        const int head = col / g.dh;
        // where this thread's row of the head goes (0: nowhere): q into C, k and v into the cache slot of the row's position
        const bool is_k = head < g.Hq + g.Hkv;
        unsigned long long dst = 0;
        if (p >= 0) {
            if (head < g.Hq) {
                dst = reinterpret_cast<unsigned long long>(static_cast<__nv_bfloat16*>(g.C) + (size_t)row * g.ldc + col);
            } else if (blk >= 0) {
                const int kh = is_k ? head - g.Hq : head - g.Hq - g.Hkv;
                const size_t at = (((size_t)blk * g.Hkv + kh) * g.block_tokens + slot) * g.dh;
                dst = g.kv_fp8 ? reinterpret_cast<unsigned long long>(reinterpret_cast<unsigned char*>(is_k ? g.k_pool : g.v_pool) + at)
                               : reinterpret_cast<unsigned long long>((is_k ? g.k_pool : g.v_pool) + at);
            }
        }
#pragma unroll 1
        for (int j0 = 0; j0 < half; j0 += 32) {
            uint32_t lo[32], hi[32];
            tc_ld32(t_row + hb + j0, lo);
            tc_ld32(t_row + hb + half + j0, hi);
            tc_wait_ld();
            if (g.fp8) {
                const float rs = row_ok ? g.a_scale[row] : 0.f;
                scale32(g, lo, rs, col + j0, g.N);
                scale32(g, hi, rs, col + half + j0, g.N);
            }
            float a[32], b[32];
            if (is_k) {                                                  // q and k heads: rotary embedding
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float2 t = cs[(size_t)(j0 + e) * g.M];
                    const float x = __uint_as_float(lo[e]), y = __uint_as_float(hi[e]);
                    a[e] = x * t.x - y * t.y;
                    b[e] = y * t.x + x * t.y;
                }
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) { a[e] = __uint_as_float(lo[e]); b[e] = __uint_as_float(hi[e]); }
            }
            if (g.kv_fp8 && head >= g.Hq) {
                if (dst) {
                    unsigned char* d8 = reinterpret_cast<unsigned char*>(dst);
                    const float sc = is_k ? g.k_scale : g.v_scale;
                    store_e4m3x32(d8 + j0, a, sc);
                    store_e4m3x32(d8 + half + j0, b, sc);
                }
                continue;
            }
            // bf16: the row's two 64-byte pieces (columns j0.. and half + j0..) side by side in the staging area, then four
            // rows per store instruction
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                stage_put(stage, lane, j, pack_bf16x8(a + 8 * j));
                stage_put(stage, lane, 4 + j, pack_bf16x8(b + 8 * j));
            }
            __syncwarp();
            const int piece = lane & 7;
            const int off = piece < 4 ? j0 + piece * 8 : half + j0 + (piece - 4) * 8;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = i * 4 + (lane >> 3);
                const unsigned long long rp = __shfl_sync(0xffffffffu, dst, r);
                if (rp) *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(rp) + off) = stage_get(stage, r, piece);
            }
            __syncwarp();
        }
    }
}

// Thin epilogue (operands swapped): this thread's tensor-memory lane is a FEATURE (weight row), the columns are tokens.
// For every token the warp's 32 lanes hold 32 consecutive features: each store (and residual load) instruction covers one
// contiguous piece of a row of C.  With split K the piece goes to partial s of the scratch, [splits][tokens][features] fp32.
__device__ __forceinline__ void epilogue_thin(const GemmArgs& g, const TileCoord& tc, uint32_t t_row, int feature, bool feature_ok, int half)
{
    const int tokens = g.N;
#pragma unroll 1
    for (int c0 = half * 32; c0 < g.bn; c0 += 64) {
        if (c0 >= tokens) break;                            // warp-uniform
        uint32_t v[32];
        tc_ld32(t_row + c0, v);
        tc_wait_ld();
        if (!feature_ok) continue;
        if (g.out_f32) {
            float* cp = static_cast<float*>(g.C) + (size_t)tc.split * tokens * g.ldc + (size_t)c0 * g.ldc + feature;
#pragma unroll
            for (int t = 0; t < 32; ++t)
                if (c0 + t < tokens) {
                    const float x = __uint_as_float(v[t]);
                    cp[(size_t)t * g.ldc] = g.accumulate ? cp[(size_t)t * g.ldc] + x : x;
                }
        } else {
            __nv_bfloat16* cp = static_cast<__nv_bfloat16*>(g.C) + (size_t)c0 * g.ldc + feature;
#pragma unroll
            for (int t = 0; t < 32; ++t)
                if (c0 + t < tokens) {
                    const float x = __uint_as_float(v[t]);
                    cp[(size_t)t * g.ldc] = __float2bfloat16_rn(g.accumulate ? __bfloat162float(cp[(size_t)t * g.ldc]) + x : x);
                }
        }
    }
}

// Decodes work item w into (m-tile, n-tile, group) and the tile's row window.  Returns false for an empty tile.
// Grouped mode enumerates only the m-tiles that exist (pref = running count of ceil(counts / BM)): group by group, within
// a group the n-tiles in turn, within an n-tile the group's m-tiles next to each other, so the CTAs that run at the same
// time share weight tiles (a group with several m-tiles reads its weights from memory once, not once per m-tile) and no
// CTA spends turns on tiles that do not exist.
__device__ __forceinline__ bool tile_coord(const GemmArgs& g, int w, int m_tiles, int n_tiles, const int* pref, TileCoord& t)
{
    const int kb_count = (g.K + BK - 1) / BK;
    t.kb0 = 0; t.kb1 = kb_count; t.split = 0;
    int split = 0;
    if (g.E > 0) {
        int lo = 0, hi = g.E - 1;                            // last group whose first item is <= w
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (pref[mid] * n_tiles <= w) lo = mid; else hi = mid - 1;
        }
        const int e = lo, mts = pref[e + 1] - pref[e], r = w - pref[e] * n_tiles;
        const int nt = r / mts, mt = r - nt * mts;
        const int cnt = g.counts[e], off = g.offsets[e];
        t.a_row = off + mt * BM; t.c_row = t.a_row; t.rows_valid = cnt - mt * BM;
        t.b_row = e * g.N + nt * BN;
        t.col = nt * BN;
        return true;
    }
    if (g.splits > 1) { split = w % g.splits; w /= g.splits; t.kb0 = split * g.kb_per; t.kb1 = min(kb_count, t.kb0 + g.kb_per); t.split = split; }
    const int mt = w % m_tiles, nt = (w / m_tiles) % n_tiles;
    t.a_row = mt * BM; t.c_row = t.a_row + split * g.M; t.rows_valid = g.M - mt * BM;
    t.b_row = nt * BN;
    t.col = nt * BN;
    return true;
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1) gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a,
                                                              const __grid_constant__ CUtensorMap map_b, const GemmArgs g)
{
    pdl_trigger();                                                        // the next kernel may be scheduled behind this one
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                        // 1024-byte aligned stage ring
    const uint32_t out_stage = tiles + STAGES * STAGE_BYTES;              // epilogue warps' staging areas
    Ctl* ctl = reinterpret_cast<Ctl*>(smem_raw + (tiles - raw) + STAGES * STAGE_BYTES + (kEpiThreads / 32) * kOutStageBytes);
    volatile int* abort_flag = &ctl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int m_tiles = (g.M + BM - 1) / BM, n_tiles = (g.N + BN - 1) / BN;
    if (g.E > 0) pdl_wait();                                // the counts are another kernel's output
    if (g.E > 0 && threadIdx.x == 64) {                     // grouped: the m-tile prefix table (counts live on the device)
        int run = 0;
        for (int e = 0; e < g.E; ++e) { ctl->pref[e] = run; run += (min(g.counts[e], g.max_m_tiles * BM) + BM - 1) / BM; }
        ctl->pref[g.E] = run;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&ctl->tmem_full[a]), 1); mbar_init(smem_u32(&ctl->tmem_empty[a]), kEpiThreads); }
        mbar_init(smem_u32(&ctl->drain), 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int* pref = ctl->pref;
    pdl_wait();                                                           // from here on global memory of the kernels in front is read
    const int n_work = g.E > 0 ? pref[g.E] * n_tiles : m_tiles * n_tiles * (g.splits > 1 ? g.splits : 1);

    if (warp == 0) {
        // ---- TMA producer ----
        if (lane == 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
                TileCoord tc;
                if (!tile_coord(g, w, m_tiles, n_tiles, pref, tc)) continue;
                for (int kb = tc.kb0; kb < tc.kb1; ++kb) {
                    if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t bar = smem_u32(&ctl->full[s]);
                    mbar_expect_tx(bar, EPI == EPI_THIN ? (uint32_t)(A_BYTES + g.bn * BK * 2) : (uint32_t)STAGE_BYTES);
                    const int kx = g.fp8 ? kb * BK * 2 : kb * BK;               // first element of the k-block (8-bit: 128 per block)
                    tma_load_2d(tiles + s * STAGE_BYTES, &map_a, kx, tc.a_row, bar);
                    tma_load_2d(tiles + s * STAGE_BYTES + A_BYTES, &map_b, kx, tc.b_row, bar);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {                                  // give copies in flight time to land before the CTA goes away
                const long long t0 = clock64();
                while (clock64() - t0 < 200000) { }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ----
        if (lane == 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            int it = 0;
            // instruction descriptor; the thin variant's n extent is the activation tile (32 or 64 rows)
            const uint32_t idesc = EPI == EPI_THIN ? ((kIdesc & ~(0x3fu << 17)) | ((uint32_t)(g.bn >> 3) << 17)) : g.fp8 ? kIdescF8 : kIdesc;
            for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
                TileCoord tc;
                if (!tile_coord(g, w, m_tiles, n_tiles, pref, tc)) continue;
                const uint32_t acc = it & 1, acc_ph = (it >> 1) & 1;
                ++it;
                if (!mbar_wait(smem_u32(&ctl->tmem_empty[acc]), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = tc.kb0; kb < tc.kb1; ++kb) {
                    if (!mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles + s * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        if (g.fp8) tc_mma_f8(d_tmem, smem_desc(sa + k * UMMA_K * 2), smem_desc(sb + k * UMMA_K * 2), idesc, (kb > tc.kb0 || k > 0) ? 1u : 0u);
                        else tc_mma(d_tmem, smem_desc(sa + k * UMMA_K * 2), smem_desc(sb + k * UMMA_K * 2), idesc, (kb > tc.kb0 || k > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&ctl->empty[s]));            // stage reusable once these MMAs have read it
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit(smem_u32(&ctl->tmem_full[acc]));  // accumulator complete
            }
            if (!ok) {                                  // drain issued tensor-core work before tensor memory is freed
                tc_commit(smem_u32(&ctl->drain));
                const long long t0 = clock64();
                while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && clock64() - t0 < kWaitLimit) { }
            }
        }
    } else {
        // ---- epilogue: warps 2..9; a warp may only touch the 32-lane quarter (warp % 4) of tensor memory, so two warps
        // share each quarter and split the tile's columns in halves ----
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        bool ok = true;
        int it = 0;
        for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
            TileCoord tc;
            if (!tile_coord(g, w, m_tiles, n_tiles, pref, tc)) continue;
            const uint32_t acc = it & 1, acc_ph = (it >> 1) & 1;
            ++it;
            const int row_in_tile = quarter * 32 + lane;
            const int row = tc.c_row + row_in_tile;
            const bool row_ok = row_in_tile < tc.rows_valid;
            const int rows_ok = min(32, tc.rows_valid - quarter * 32);       // valid rows among this warp's 32 (may be <= 0)
            uint4 resid[8];
            if constexpr (EPI == EPI_PLAIN) {
                // += residual in fp32: ask for the first block of the residual before waiting for the accumulator
                const int col = tc.col + half * (BN / 2);
                if (g.out_f32 && g.accumulate && col + 32 <= g.N)
                    residual_get(resid, lane, reinterpret_cast<const unsigned char*>(static_cast<const float*>(g.C) + (size_t)(row - lane) * g.ldc + col),
                                 (size_t)g.ldc * 4, rows_ok);
            }
            if (!mbar_wait(smem_u32(&ctl->tmem_full[acc]), acc_ph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
            const uint32_t stage = out_stage + (warp - 2) * kOutStageBytes;
            if constexpr (EPI == EPI_THIN) epilogue_thin(g, tc, t_row, tc.a_row + row_in_tile, row_ok, half);
            else if constexpr (EPI == EPI_SWIGLU) epilogue_swiglu(g, tc, t_row, row, row_ok, half, stage, lane, rows_ok);
            else if constexpr (EPI == EPI_QKV) epilogue_qkv(g, tc, t_row, row, row_ok, half, stage, lane);
            else epilogue_plain(g, tc, t_row, row, row_ok, half, stage, lane, rows_ok, resid);
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && ctl->abort) set_status(g.status, SPEC_ERR_TIMEOUT, (int)blockIdx.x);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// Self-test of the bounded wait: waits on an mbarrier that nothing ever arrives on, with a short limit, and reports the
// outcome exactly as the GEMM roles do (abort flag -> SPEC_ERR_TIMEOUT in the status word).  The context stays usable.
}  // namespace
__global__ void bounded_wait_probe_kernel(long long limit_cycles, int32_t* status, int32_t* elapsed_out)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const long long t0 = clock64();
        bool ok = mbar_try_wait(smem_u32(&bar), 0);
        while (!ok && clock64() - t0 <= limit_cycles) ok = mbar_try_wait(smem_u32(&bar), 0);
        if (!ok) { abort_flag = 1; set_status(status, SPEC_ERR_TIMEOUT, 0); }
        *elapsed_out = (int32_t)((clock64() - t0) >> 10);
    }
}
namespace {

// Sums the split-K partials in split order (deterministic) into C, optionally on top of C's previous contents.
template <class TC>
__global__ void splitk_reduce_kernel(int M, int N, int splits, const float* __restrict__ part, TC* __restrict__ C, int ldc,
                                     int accumulate)
{
    pdl_trigger();
    pdl_wait();
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= (size_t)M * N) return;
    const int m = (int)(i / N), n = (int)(i % N);
    float4 acc = *reinterpret_cast<const float4*>(part + i);
    for (int s = 1; s < splits; ++s) {
        const float4 v = *reinterpret_cast<const float4*>(part + (size_t)s * M * N + i);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    TC* c = C + (size_t)m * ldc + n;
    if (accumulate) { acc.x += to_f32(c[0]); acc.y += to_f32(c[1]); acc.z += to_f32(c[2]); acc.w += to_f32(c[3]); }
    c[0] = from_f32<TC>(acc.x); c[1] = from_f32<TC>(acc.y); c[2] = from_f32<TC>(acc.z); c[3] = from_f32<TC>(acc.w);
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
std::atomic<EncodeFn> g_encode{nullptr};
thread_local int g_sms = 0;          // SM count of the device the calling thread last initialised for

// Resolves the tensor-map encoder once per process and raises the kernels' dynamic shared memory limit once per device.
bool init_once()
{
    static PerDeviceOnce configured;
    static std::atomic<int> sms[64];
    int dev = 0;
    if (!configured.needed(&dev) && g_encode.load(std::memory_order_acquire) != nullptr) {
        g_sms = sms[dev & 63].load(std::memory_order_relaxed);
        return true;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr) return false;
    int n = 0;
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
    if (cudaFuncSetAttribute(gemm_tc_kernel<EPI_PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return false;
    if (cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return false;
    if (cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return false;
    if (cudaFuncSetAttribute(gemm_tc_kernel<EPI_THIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return false;
    sms[dev & 63].store(n, std::memory_order_relaxed);
    g_sms = n;
    g_encode.store(reinterpret_cast<EncodeFn>(fn), std::memory_order_release);
    configured.done(dev);
    return true;
}

spec_status run_kernel(int epi, const CUtensorMap& ma, const CUtensorMap& mb, const GemmArgs& g, long long n_work, cudaStream_t st)
{
    const int grid = n_work < g_sms ? (int)n_work : g_sms;
    if (epi == EPI_SWIGLU)   launch_pdl(gemm_tc_kernel<EPI_SWIGLU>, dim3(grid), dim3(kThreads), (size_t)kSmemBytes, st, ma, mb, g);
    else if (epi == EPI_QKV) launch_pdl(gemm_tc_kernel<EPI_QKV>, dim3(grid), dim3(kThreads), (size_t)kSmemBytes, st, ma, mb, g);
    else if (epi == EPI_THIN) launch_pdl(gemm_tc_kernel<EPI_THIN>, dim3(grid), dim3(kThreads), (size_t)kSmemBytes, st, ma, mb, g);
    else                     launch_pdl(gemm_tc_kernel<EPI_PLAIN>, dim3(grid), dim3(kThreads), (size_t)kSmemBytes, st, ma, mb, g);
    return launch_status();
}

// 2-D map over a row-major [rows][cols] matrix of e4m3 codes (bytes) with row pitch ld bytes; box = 128 columns x box_rows rows:
// the same 128-byte-wide, 128B-swizzled tile in shared memory as 64 bf16 columns.
bool make_map8(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows);
// 2-D map over a row-major [rows][cols] bf16 matrix with row pitch ld elements; box = 64 columns x box_rows rows.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows)
{
    const cuuint64_t gdim[2] = {cols, rows};
    const cuuint64_t gstride[1] = {ld * 2};
    const cuuint32_t box[2] = {BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode.load(std::memory_order_acquire)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_map8(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows)
{
    const cuuint64_t gdim[2] = {cols, rows};
    const cuuint64_t gstride[1] = {ld};
    const cuuint32_t box[2] = {2 * BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode.load(std::memory_order_acquire)(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tc::tc_make_map_2d(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_cols,
                        uint32_t box_rows)
{
    if (!init_once()) return false;
    const cuuint64_t gdim[2] = {cols, rows};
    const cuuint64_t gstride[1] = {ld * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode.load(std::memory_order_acquire)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int tc::tc_sm_count() { return init_once() ? g_sms : 148; }

bool gemm_tc_supported(int M, int N, int K, const void* A, int lda, const void* W, const void* C, int ldc, int dtype_in,
                       int out_dtype)
{
    (void)M;
    const int cal = out_dtype == SPEC_DTYPE_F32 ? 4 : 8;
    return dtype_in == SPEC_DTYPE_BF16 && K % 8 == 0 && lda % 8 == 0 && N % cal == 0 && ldc % cal == 0 &&
           (reinterpret_cast<uintptr_t>(A) & 15u) == 0 && (reinterpret_cast<uintptr_t>(W) & 15u) == 0 &&
           (reinterpret_cast<uintptr_t>(C) & 15u) == 0;
}

spec_status launch_gemm_tc(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int out_dtype,
                           int accumulate, int32_t* status, cudaStream_t st)
{
    if (M == 0 || N == 0) return SPEC_OK;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map(&ma, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM)) return SPEC_ERR_CUDA;
    if (!make_map(&mb, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    const int n_work = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
    GemmArgs g{};
    g.M = M; g.N = N; g.K = K; g.C = C; g.ldc = ldc; g.out_f32 = out_dtype == SPEC_DTYPE_F32 ? 1 : 0; g.accumulate = accumulate;
    g.status = status;
    // Few tiles and a long K (small-M projections: plain decode, draft passes): split K so that every SM streams weights.
    // Partials go to the caller-provided scratch and are summed in split order by a second kernel.
    const GemmScratch& sc = gemm_scratch();
    const int kb_count = (K + BK - 1) / BK;
    int splits = 1;
    if (sc.ptr != nullptr && n_work * 2 <= g_sms && N % 4 == 0) {
        splits = g_sms / n_work;
        if (splits > 8) splits = 8;
        while (splits > 1 && (kb_count / splits < 8 || (size_t)splits * M * N * 4 > sc.bytes)) --splits;
    }
    if (splits > 1) {
        g.C = sc.ptr; g.ldc = N; g.out_f32 = 1; g.accumulate = 0;
        g.splits = splits; g.kb_per = (kb_count + splits - 1) / splits;
        TRY_LAUNCH(run_kernel(EPI_PLAIN, ma, mb, g, (long long)n_work * splits, st));
        const size_t n4 = (size_t)M * N / 4;
        if (out_dtype == SPEC_DTYPE_F32)
            splitk_reduce_kernel<float><<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(M, N, splits, (const float*)sc.ptr, (float*)C, ldc, accumulate);
        else
            splitk_reduce_kernel<__nv_bfloat16><<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(M, N, splits, (const float*)sc.ptr, (__nv_bfloat16*)C, ldc, accumulate);
        return launch_status();
    }
    return run_kernel(EPI_PLAIN, ma, mb, g, n_work, st);
}

// 17..64 activation rows: operands swapped (see GemmArgs::bn).  One work item per 128 weight rows (x splits of K when that
// leaves SMs idle and the caller gave scratch; the partials are summed in split order by the reduction kernel).
bool gemm_tc_thin_supported(int M, int N, int K, const void* A, int lda, const void* W, const void* C, int ldc, int dtype_in, int out_dtype)
{
    return M > 16 && M <= 64 && K % BK == 0 && gemm_tc_supported(M, N, K, A, lda, W, C, ldc, dtype_in, out_dtype);
}

spec_status launch_gemm_tc_thin(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int out_dtype,
                                int accumulate, int32_t* status, cudaStream_t st)
{
    if (!init_once()) return SPEC_ERR_CUDA;
    const int bn = M <= 32 ? 32 : 64;
    CUtensorMap ma, mb;
    if (!make_map(&ma, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, BM)) return SPEC_ERR_CUDA;            // weights: the M operand
    if (!make_map(&mb, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, (uint32_t)bn)) return SPEC_ERR_CUDA;   // activations: the N operand
    const int n_work = (N + BM - 1) / BM, kb_count = K / BK;
    GemmArgs g{};
    g.M = N; g.N = M; g.K = K; g.C = C; g.ldc = ldc; g.out_f32 = out_dtype == SPEC_DTYPE_F32 ? 1 : 0; g.accumulate = accumulate;
    g.status = status; g.bn = bn;
    const GemmScratch& sc = gemm_scratch();
    int splits = 1;
    if (sc.ptr != nullptr && n_work * 2 <= g_sms && N % 4 == 0) {
        splits = g_sms / n_work;
        if (splits > 8) splits = 8;
        while (splits > 1 && (kb_count / splits < 8 || (size_t)splits * M * N * 4 > sc.bytes)) --splits;
    }
    if (splits > 1) {
        g.C = sc.ptr; g.ldc = N; g.out_f32 = 1; g.accumulate = 0;
        g.splits = splits; g.kb_per = (kb_count + splits - 1) / splits;
        TRY_LAUNCH(run_kernel(EPI_THIN, ma, mb, g, (long long)n_work * splits, st));
        const size_t n4 = (size_t)M * N / 4;
        if (out_dtype == SPEC_DTYPE_F32)
            splitk_reduce_kernel<float><<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(M, N, splits, (const float*)sc.ptr, (float*)C, ldc, accumulate);
        else
            splitk_reduce_kernel<__nv_bfloat16><<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(M, N, splits, (const float*)sc.ptr, (__nv_bfloat16*)C, ldc, accumulate);
        return launch_status();
    }
    return run_kernel(EPI_THIN, ma, mb, g, n_work, st);
}

// Row statistics from the pairs an LM-head launch left behind: (m, Z) with Z = sum_v exp((l_v - m) * inv_t), pairs merged in a
// fixed order (each lane takes every 32nd pair in turn, then a shuffle tree).
__global__ void __launch_bounds__(256) stat_combine_kernel(int rows, int pairs, const float* __restrict__ part, float inv_t,
                                                           float* __restrict__ stats, size_t stats_stride)
{
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= rows) return;
    const float* p = part + (size_t)row * pairs * 2;
    float m = -INFINITY, z = 0.f;
    for (int i = lane; i < pairs; i += 32) {
        const float pm = p[2 * i], pz = p[2 * i + 1];
        if (pm > m) { z *= __expf(__fmul_rn(__fsub_rn(m, pm), inv_t)); m = pm; }
        if (pm != -INFINITY) z += pz * __expf(__fmul_rn(__fsub_rn(pm, m), inv_t));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, o), oz = __shfl_xor_sync(0xffffffffu, z, o);
        const float nm = fmaxf(m, om);
        const float a = (m == -INFINITY) ? 0.f : z * __expf(__fmul_rn(__fsub_rn(m, nm), inv_t));
        const float b = (om == -INFINITY) ? 0.f : oz * __expf(__fmul_rn(__fsub_rn(om, nm), inv_t));
        // both lanes of a pair must form the same sum: add the lower lane's term first
        z = (lane & o) ? b + a : a + b;
        m = nm;
    }
    if (lane == 0) { stats[2 * (size_t)row * stats_stride] = m; stats[2 * (size_t)row * stats_stride + 1] = z; }
}

// LM head: logits [M][N] fp32 = A W^T and the row statistics (m, Z) of logits / temperature in stats [row * stats_stride][2],
// the statistics taken in the GEMM epilogue.  part: scratch of at least M * 2 * ceil(N / 256) * 8 bytes.  Returns
// SPEC_ERR_UNSUPPORTED (nothing launched) when the shape does not run on the tile kernel; the caller then takes the two-pass way.
spec_status launch_gemm_lm_head_stats(int M, int N, int K, const void* A, int lda, const void* W, float* logits, int ldc, int dtype_in,
                                      float temperature, float* part, size_t part_bytes, float* stats, size_t stats_stride,
                                      int32_t* status, cudaStream_t st)
{
    if (M == 0 || N == 0) return SPEC_OK;
    const int pairs = 2 * ((N + BN - 1) / BN);
    if (M <= 64 || part == nullptr || (size_t)M * pairs * 8 > part_bytes ||
        !gemm_tc_supported(M, N, K, A, lda, W, logits, ldc, dtype_in, SPEC_DTYPE_F32))
        return SPEC_ERR_UNSUPPORTED;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map(&ma, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM)) return SPEC_ERR_CUDA;
    if (!make_map(&mb, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    GemmArgs g{};
    g.M = M; g.N = N; g.K = K; g.C = logits; g.ldc = ldc; g.out_f32 = 1; g.status = status;
    g.stat_part = part; g.stat_pairs = pairs; g.inv_t = 1.0f / temperature;
    TRY_LAUNCH(run_kernel(EPI_PLAIN, ma, mb, g, (long long)((M + BM - 1) / BM) * ((N + BN - 1) / BN), st));
    launch_pdl(stat_combine_kernel, dim3((M + 7) / 8), dim3(256), 0, st, M, pairs, (const float*)part, g.inv_t, stats, stats_stride);
    return launch_status();
}

// gate/up projection with the SwiGLU applied in the epilogue: W [2F][K] stored in 256-row groups (128 gate rows, then the
// matching 128 up rows), act [M][F] bf16.
spec_status launch_gemm_swiglu_tc(int M, int F, int K, const void* A, int lda, const void* W, void* act, int32_t* status,
                                  cudaStream_t st)
{
    if (M == 0 || F == 0) return SPEC_OK;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map(&ma, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM)) return SPEC_ERR_CUDA;
    if (!make_map(&mb, W, (uint64_t)2 * F, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    GemmArgs g{};
    g.M = M; g.N = 2 * F; g.K = K; g.C = act; g.ldc = F; g.status = status;
    return run_kernel(EPI_SWIGLU, ma, mb, g, (long long)((M + BM - 1) / BM) * (2 * F / BN), st);
}

// QKV projection with rotary embedding and KV append in the epilogue.
spec_status launch_gemm_qkv_tc(int M, int K, const void* A, int lda, const void* W, void* qkv, const QkvEpilogue& e,
                               int32_t* status, cudaStream_t st)
{
    const int N = (e.Hq + 2 * e.Hkv) * e.dh;
    if (M == 0) return SPEC_OK;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map(&ma, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM)) return SPEC_ERR_CUDA;
    if (!make_map(&mb, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    GemmArgs g{};
    g.M = M; g.N = N; g.K = K; g.C = qkv; g.ldc = N; g.status = status;
    g.Hq = e.Hq; g.Hkv = e.Hkv; g.dh = e.dh; g.R = e.R; g.max_blocks = e.max_blocks; g.block_tokens = e.block_tokens;
    g.pos = e.pos; g.block_table = e.block_table; g.rope = reinterpret_cast<const float2*>(e.rope);
    g.k_pool = static_cast<__nv_bfloat16*>(e.k_pool); g.v_pool = static_cast<__nv_bfloat16*>(e.v_pool);
    g.kv_fp8 = e.kv_fp8; g.k_scale = e.k_scale; g.v_scale = e.v_scale;
    return run_kernel(EPI_QKV, ma, mb, g, (long long)((M + BM - 1) / BM) * ((N + BN - 1) / BN), st);
}

// ---- 8-bit (e4m3) operands: A [M][K] and W [N][K] are codes with one fp32 scale per row; K % 16 == 0 ------------------
namespace {
bool fp8_ok(int K, const void* a8, const void* w8) { return K % 16 == 0 && ((reinterpret_cast<uintptr_t>(a8) | reinterpret_cast<uintptr_t>(w8)) & 15u) == 0; }
void fp8_args(GemmArgs& g, int M, int N, int K, const float* a_scale, const float* w_scale, int32_t* status)
{
    g.M = M; g.N = N; g.K = K / 2;                          // K in byte pairs: ceil(g.K / 64) = ceil(K / 128) k-blocks
    g.status = status; g.fp8 = 1; g.a_scale = a_scale; g.w_scale = w_scale;
}
}  // namespace

// C (+)= (A W^T) scaled; with part != nullptr (fp32 logits) the row statistics go to stats as in launch_gemm_lm_head_stats.
spec_status launch_gemm8_tc(int M, int N, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale, void* C, int ldc,
                            int out_dtype, int accumulate, float temperature, float* part, size_t part_bytes, float* stats,
                            size_t stats_stride, int32_t* status, cudaStream_t st)
{
    if (M == 0 || N == 0) return SPEC_OK;
    if (!fp8_ok(K, a8, w8)) return SPEC_ERR_SHAPE;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map8(&ma, a8, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM)) return SPEC_ERR_CUDA;
    if (!make_map8(&mb, w8, (uint64_t)N, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    GemmArgs g{};
    fp8_args(g, M, N, K, a_scale, w_scale, status);
    g.C = C; g.ldc = ldc; g.out_f32 = out_dtype == SPEC_DTYPE_F32 ? 1 : 0; g.accumulate = accumulate;
    const int pairs = 2 * ((N + BN - 1) / BN);
    const bool with_stats = part != nullptr && g.out_f32 && (size_t)M * pairs * 8 <= part_bytes;
    if (with_stats) { g.stat_part = part; g.stat_pairs = pairs; g.inv_t = 1.0f / temperature; }
    TRY_LAUNCH(run_kernel(EPI_PLAIN, ma, mb, g, (long long)((M + BM - 1) / BM) * ((N + BN - 1) / BN), st));
    if (with_stats) {
        launch_pdl(stat_combine_kernel, dim3((M + 7) / 8), dim3(256), 0, st, M, pairs, (const float*)part, g.inv_t, stats, stats_stride);
        return launch_status();
    }
    return part != nullptr ? SPEC_ERR_UNSUPPORTED : SPEC_OK;   // statistics wanted but the scratch is too small: the caller falls back
}

spec_status launch_gemm8_swiglu_tc(int M, int F, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale, void* act,
                                   int32_t* status, cudaStream_t st)
{
    if (M == 0 || F == 0) return SPEC_OK;
    if (!fp8_ok(K, a8, w8)) return SPEC_ERR_SHAPE;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map8(&ma, a8, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM)) return SPEC_ERR_CUDA;
    if (!make_map8(&mb, w8, (uint64_t)2 * F, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    GemmArgs g{};
    fp8_args(g, M, 2 * F, K, a_scale, w_scale, status);
    g.C = act; g.ldc = F;
    return run_kernel(EPI_SWIGLU, ma, mb, g, (long long)((M + BM - 1) / BM) * (2 * F / BN), st);
}

spec_status launch_gemm8_qkv_tc(int M, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale, void* qkv,
                                const QkvEpilogue& e, int32_t* status, cudaStream_t st)
{
    const int N = (e.Hq + 2 * e.Hkv) * e.dh;
    if (M == 0) return SPEC_OK;
    if (!fp8_ok(K, a8, w8)) return SPEC_ERR_SHAPE;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map8(&ma, a8, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM)) return SPEC_ERR_CUDA;
    if (!make_map8(&mb, w8, (uint64_t)N, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    GemmArgs g{};
    fp8_args(g, M, N, K, a_scale, w_scale, status);
    g.C = qkv; g.ldc = N;
    g.Hq = e.Hq; g.Hkv = e.Hkv; g.dh = e.dh; g.R = e.R; g.max_blocks = e.max_blocks; g.block_tokens = e.block_tokens;
    g.pos = e.pos; g.block_table = e.block_table; g.rope = reinterpret_cast<const float2*>(e.rope);
    g.k_pool = static_cast<__nv_bfloat16*>(e.k_pool); g.v_pool = static_cast<__nv_bfloat16*>(e.v_pool);
    g.kv_fp8 = e.kv_fp8; g.k_scale = e.k_scale; g.v_scale = e.v_scale;
    return run_kernel(EPI_QKV, ma, mb, g, (long long)((M + BM - 1) / BM) * ((N + BN - 1) / BN), st);
}

// Grouped product on 8-bit operands: as launch_gemm_grouped with A [rows_total][K] and W [E][N][K] as e4m3 codes, a_scale one
// per row of A, w_scale [E][N].
spec_status launch_gemm8_grouped(int rows_total, int max_rows_per_group, int E, int N, int K, const void* a8, const float* a_scale,
                                 const void* w8, const float* w_scale, void* C, int out_dtype, int swiglu, const int32_t* counts,
                                 const int32_t* offsets, int32_t* status, cudaStream_t st)
{
    if (rows_total == 0 || E == 0) return SPEC_OK;
    if (N % BN != 0 || E > kMaxGroups || !fp8_ok(K, a8, w8)) return SPEC_ERR_SHAPE;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map8(&ma, a8, (uint64_t)rows_total, (uint64_t)K, (uint64_t)K, BM)) return SPEC_ERR_CUDA;
    if (!make_map8(&mb, w8, (uint64_t)E * N, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    const int max_m_tiles = (max_rows_per_group + BM - 1) / BM;
    GemmArgs g{};
    fp8_args(g, rows_total, N, K, a_scale, w_scale, status);
    g.C = C; g.ldc = swiglu ? N / 2 : N; g.out_f32 = out_dtype == SPEC_DTYPE_F32 ? 1 : 0;
    g.E = E; g.max_m_tiles = max_m_tiles; g.counts = counts; g.offsets = offsets;
    return run_kernel(swiglu ? EPI_SWIGLU : EPI_PLAIN, ma, mb, g, (long long)E * max_m_tiles * (N / BN), st);
}

// Grouped form: A [rows_total][K] holds the groups' rows back to back (group e at offsets[e], counts[e] rows, both on
// the device; no group has more than max_rows_per_group rows), W [E][N][K], C [rows_total][N].  N % 256 == 0.
spec_status launch_gemm_grouped(int rows_total, int max_rows_per_group, int E, int N, int K, const void* A, const void* W,
                                void* C, int out_dtype, int swiglu, const int32_t* counts, const int32_t* offsets,
                                int32_t* status, cudaStream_t st)
{
    if (rows_total == 0 || E == 0) return SPEC_OK;
    if (N % BN != 0 || K % 8 != 0 || E > kMaxGroups) return SPEC_ERR_SHAPE;
    if (!init_once()) return SPEC_ERR_CUDA;
    CUtensorMap ma, mb;
    if (!make_map(&ma, A, (uint64_t)rows_total, (uint64_t)K, (uint64_t)K, BM)) return SPEC_ERR_CUDA;
    if (!make_map(&mb, W, (uint64_t)E * N, (uint64_t)K, (uint64_t)K, BN)) return SPEC_ERR_CUDA;
    const int max_m_tiles = (max_rows_per_group + BM - 1) / BM;
    GemmArgs g{};
    g.M = rows_total; g.N = N; g.K = K; g.C = C; g.ldc = swiglu ? N / 2 : N; g.out_f32 = out_dtype == SPEC_DTYPE_F32 ? 1 : 0;
    g.status = status; g.E = E; g.max_m_tiles = max_m_tiles; g.counts = counts; g.offsets = offsets;
    return run_kernel(swiglu ? EPI_SWIGLU : EPI_PLAIN, ma, mb, g, (long long)E * max_m_tiles * (N / BN), st);
}

spec_status launch_gemm(int M, int N, int K, const void* A, int lda, const void* W, void* C, int ldc, int dtype_in,
                        int out_dtype, int accumulate, cudaStream_t st)
{
    if (gemm_skinny_supported(M, N, K, A, lda, W, dtype_in)) return launch_gemm_skinny(M, N, K, A, lda, W, C, ldc, out_dtype, accumulate, st);
    if (gemm_tc_thin_supported(M, N, K, A, lda, W, C, ldc, dtype_in, out_dtype))
        return launch_gemm_tc_thin(M, N, K, A, lda, W, C, ldc, out_dtype, accumulate, nullptr, st);
    if (gemm_tc_supported(M, N, K, A, lda, W, C, ldc, dtype_in, out_dtype))
        return launch_gemm_tc(M, N, K, A, lda, W, C, ldc, out_dtype, accumulate, nullptr, st);
    return launch_gemm_simt(M, N, K, A, lda, W, C, ldc, dtype_in, out_dtype, accumulate, st);
}

}  // namespace spec

extern "C" spec_status spec_selftest_bounded_wait(int32_t* status, int32_t* elapsed_kcycles, void* stream)
{
    if (status == nullptr || elapsed_kcycles == nullptr) return SPEC_ERR_INVALID_ARG;
    spec::bounded_wait_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(2000000LL, status, elapsed_kcycles);
    return spec::launch_status();
}

extern "C" spec_status spec_gemm(int M, int N, int K, const void* A, const void* W, void* C, int dtype_in, int out_dtype,
                                 int accumulate, void* stream)
{
    if (M < 0 || N < 0 || K <= 0) return SPEC_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return SPEC_OK;
    if (!A || !W || !C) return SPEC_ERR_INVALID_ARG;
    return spec::launch_gemm(M, N, K, A, K, W, C, N, dtype_in, out_dtype, accumulate, (cudaStream_t)stream);
}

extern "C" spec_status spec_gemm_e4m3(int M, int N, int K, const void* a8, const float* a_scale, const void* w8, const float* w_scale,
                                      void* C, int out_dtype, int accumulate, void* stream)
{
    if (M < 0 || N < 0 || K <= 0) return SPEC_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return SPEC_OK;
    if (!a8 || !a_scale || !w8 || !w_scale || !C) return SPEC_ERR_INVALID_ARG;
    if (N % 8 != 0 || (reinterpret_cast<uintptr_t>(C) & 15u) != 0) return SPEC_ERR_SHAPE;
    return spec::launch_gemm8_tc(M, N, K, a8, a_scale, w8, w_scale, C, N, out_dtype, accumulate, 1.0f, nullptr, 0, nullptr, 0, nullptr,
                                 (cudaStream_t)stream);
}
