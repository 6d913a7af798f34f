// Paged grouped-query attention for bf16 caches: the HBM-bound pass that dominates a verify forward.
//
// Work = (sequence, KV head, KV chunk) units.  A one-CTA planning kernel splits every sequence into equal chunks of
// at most kChunk (4096) tokens and writes the unit list; persistent CTAs (a multiple of the SM count) pull units from an
// atomic counter, so the long tail of sequence lengths is balanced at unit granularity.  All query rows that share a
// KV head (the k+1 positions x the group of query heads: 16 rows for 4 x 4) form the M dimension of
// mma.m16n8k16, so each K/V byte is read from HBM once per layer.  K/V tiles of 64 tokens are staged with 16-byte
// cp.async into XOR-swizzled shared memory, a 3-stage pipeline keeps ~64 KB per CTA in flight, fragments come from
// ldmatrix (transposed for V), softmax is online in fp32 (exp2 domain), and units of one sequence are merged by a
// log-sum-exp kernel (skipped for single-chunk sequences, which write their output directly).
// Causality among the new rows: row (i, head j) sees cache positions <= pos[b*R + i].
// This is the kernel for up to 16 query rows per KV head (and for head_dim 64); wider row groups at head_dim 128 go to the
// tcgen05 kernel, which shares the plan and the merge pass defined here.
#include "attention_plan.cuh"

namespace spec {
using namespace attn;
namespace {

constexpr int kThreads = 128;
constexpr int kPlanThreads = 1024;

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
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---- planning: one CTA, sequences in index order -------------------------------------------------------------------
__global__ void __launch_bounds__(kPlanThreads) attn_plan_kernel(int B, int R, const int32_t* __restrict__ pos, int Hkv, int n_ctas,
                                                                 int cap_entries, PlanView pv)
{
    __shared__ int s_warp[33];
    __shared__ long long s_tot[2];
    for (int i = threadIdx.x; i < kCounters; i += kPlanThreads) pv.counters[i] = 0;
    if (threadIdx.x == 0) { s_tot[0] = 0; s_tot[1] = 0; }
    __syncthreads();
    // Chunk length of this launch.  With a full batch there are far more units than CTAs and kChunk-token chunks are best; a
    // thin batch (the long tail of a rollout: most slots retired) would leave most CTAs without a unit, so the chunk is halved
    // while the unit count stays under two per CTA - as long as the unit list still fits what the scratch was sized for.
    {
        long long tok = 0, act = 0;
        for (int b = threadIdx.x; b < B; b += kPlanThreads) {
            int ntok = 0;
            for (int i = 0; i < R; ++i) ntok = max(ntok, pos[(size_t)b * R + i] + 1);
            tok += ntok; act += ntok > 0;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { tok += __shfl_xor_sync(0xffffffffu, tok, o); act += __shfl_xor_sync(0xffffffffu, act, o); }
        if ((threadIdx.x & 31) == 0) { atomicAdd(reinterpret_cast<unsigned long long*>(&s_tot[0]), (unsigned long long)tok);
                                       atomicAdd(reinterpret_cast<unsigned long long*>(&s_tot[1]), (unsigned long long)act); }
    }
    __syncthreads();
    int chunk = kChunk;
    {
        const long long tok = s_tot[0], act = s_tot[1];
        while (chunk > kChunkMin && (tok / chunk + act) * Hkv < 2LL * n_ctas && tok / (chunk / 2) + act <= cap_entries) chunk >>= 1;
    }
    int carry = 0;
    for (int base = 0; base < B; base += kPlanThreads) {
        const int b = base + threadIdx.x;
        int ntok = 0, nc = 0, per = 0;
        if (b < B) {
            for (int i = 0; i < R; ++i) ntok = max(ntok, pos[(size_t)b * R + i] + 1);
            // a few tokens past a multiple of the chunk length (the k+1 new rows on top of a round cache length) do not
            // open another chunk: a chunk may run up to kChunkSlack tokens over
            nc = ntok > 0 ? max(1, (ntok - kChunkSlack + chunk - 1) / chunk) : 0;
            if (nc > 0) {
                per = ((ntok + nc - 1) / nc + kTileTok - 1) / kTileTok * kTileTok;
                nc = (ntok + per - 1) / per;                 // <= ntok / chunk + 1, so the list holds at most tok / chunk + act units
            }
        }
        // exclusive scan of nc over the block
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        int inc = nc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
        __syncthreads();
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const int w = s_warp[lane];
            int winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, winc, o); if (lane >= o) winc += t; }
            s_warp[lane] = winc - w;
            if (lane == 31) s_warp[32] = winc;
        }
        __syncthreads();
        const int off = carry + s_warp[warp] + inc - nc;
        const int total = s_warp[32];
        if (b < B) {
            pv.first[b] = off;
            pv.nc[b] = nc;
            for (int c = 0; c < nc; ++c)
                pv.entries[off + c] = Unit{b, c * per, min(ntok, (c + 1) * per), nc > 1 ? off + c : -1};
        }
        carry += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) *pv.n_entries = carry;
}

struct MmaArgs {
    const __nv_bfloat16* q; int q_row_stride;
    const __nv_bfloat16* k_pool; const __nv_bfloat16* v_pool;
    const int32_t* block_table; int max_blocks;
    const int32_t* pos;
    int R, group, Hkv;
    __nv_bfloat16* out; int out_row_stride;
    float scale_log2;
    PlanView pv;
    int counter_index;
};

// One CTA = 4 warps arranged WM x WN: WM warp-rows of 16 query rows each, WN warps splitting the tokens of a tile.
template <int DH, int WM, int WN, int STAGES>
__global__ void __launch_bounds__(kThreads) attn_mma_kernel(const MmaArgs a)
{
    pdl_trigger();
    pdl_wait();
    static_assert(WM * WN == 4, "four warps");
    constexpr int CH = DH / 8;                               // 16-byte chunks per row
    constexpr int kBlkBytes = kBT * DH * 2;                  // one KV block of one head
    constexpr int kTileBytes = 4 * kBlkBytes * 2;            // 4 blocks, K and V
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
                // A fragment: regs {hh, hh+2} hold (row, k = 16 ks + 2 q4 + {0,1}) and (row, the same + 8)
                qf[ks][hh] = valid ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 2 * q4) : 0u;
                qf[ks][hh + 2] = valid ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 8 + 2 * q4) : 0u;
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
            const uint32_t stage = smem_base + (uint32_t)(j % STAGES) * kTileBytes;
            const int blk0 = (t0 + j * kTileTok) / kBT;
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) {
                const int bi = blk0 + bb;
                const int phys = (bi * kBT < t1 && bi < a.max_blocks) ? table[bi] : -1;
                const size_t goff = ((size_t)(phys < 0 ? 0 : phys) * a.Hkv + g) * (size_t)(kBT * DH);
                const int nbytes = phys < 0 ? 0 : 16;
#pragma unroll
                for (int hlf = 0; hlf < (16 * CH) / kThreads; ++hlf) {
                    const int idx = tid + kThreads * hlf;           // 16-byte chunk within the block
                    const int r = idx / CH, c = idx % CH;
                    const uint32_t soff = (uint32_t)(bb * kBlkBytes + r * (DH * 2) + (((c & ~7) | ((c ^ r) & 7)) << 4));
                    cp_async16(stage + soff, a.k_pool + goff + (size_t)idx * 8, nbytes);
                    cp_async16(stage + 4 * kBlkBytes + soff, a.v_pool + goff + (size_t)idx * 8, nbytes);
                }
            }
        };

#pragma unroll
        for (int j = 0; j < STAGES - 1; ++j) { if (j < n_tiles) issue_tile(j); cp_async_commit(); }

        for (int j = 0; j < n_tiles; ++j) {
            cp_async_wait<STAGES - 2>();
            __syncthreads();
            if (j + STAGES - 1 < n_tiles) issue_tile(j + STAGES - 1);
            cp_async_commit();
            const uint32_t stage = smem_base + (uint32_t)(j % STAGES) * kTileBytes;
#pragma unroll
            for (int bb = wn; bb < 4; bb += WN) {
                const int tok0 = t0 + j * kTileTok + bb * kBT;
                if (tok0 >= t1) continue;
                const uint32_t kb_base = stage + bb * kBlkBytes, vb_base = kb_base + 4 * kBlkBytes;
                // S = Q K^T for 16 tokens
                float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                {
                    const int mat = lane >> 3, rr = lane & 7;
                    const int row = rr + 8 * (mat >> 1);
#pragma unroll
                    for (int ks = 0; ks < DH / 16; ++ks) {
                        const int c = 2 * ks + (mat & 1);
                        uint32_t kb[4];
                        ldmatrix_x4(kb, kb_base + row * (DH * 2) + (((c & ~7) | ((c ^ row) & 7)) << 4));
                        mma_bf16(s[0], qf[ks], kb[0], kb[1]);
                        mma_bf16(s[1], qf[ks], kb[2], kb[3]);
                    }
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
                    pf[0] = pack_bf16(p[0][0], p[0][1]);
                    pf[1] = pack_bf16(p[0][2], p[0][3]);
                    pf[2] = pack_bf16(p[1][0], p[1][1]);
                    pf[3] = pack_bf16(p[1][2], p[1][3]);
                }
                // O += P V
                {
                    const int mat = lane >> 3, rr = lane & 7;
                    const int row = rr + 8 * (mat & 1);
#pragma unroll
                    for (int nd = 0; nd < DH / 16; ++nd) {
                        const int c = 2 * nd + (mat >> 1);
                        uint32_t vb[4];
                        ldmatrix_x4_trans(vb, vb_base + row * (DH * 2) + (((c & ~7) | ((c ^ row) & 7)) << 4));
                        mma_bf16(o_acc[2 * nd], pf, vb[0], vb[1]);
                        mma_bf16(o_acc[2 * nd + 1], pf, vb[2], vb[3]);
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
            for (int n = 0; n < NT_O; ++n)
                *reinterpret_cast<float2*>(orow + 8 * n + 2 * q4) = make_float2(o_acc[n][2 * hh], o_acc[n][2 * hh + 1]);
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
                *reinterpret_cast<float4*>(a.pv.part_o + (ps * ROWS + r) * DH + c4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                if (c4 == 0) { a.pv.part_ml[(ps * ROWS + r) * 2] = M; a.pv.part_ml[(ps * ROWS + r) * 2 + 1] = L; }
            } else if (r < n_rows_valid) {
                const float inv = L > 0.f ? 1.f / L : 0.f;
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

// Merges the chunks of multi-chunk sequences; writes zeros for sequences without any visible position.
template <int DH>
__global__ void __launch_bounds__(128) attn_merge_kernel(int B, int rows_alloc, const MmaArgs a)
{
    pdl_trigger();
    pdl_wait();
    // blockIdx.x = (sequence, KV head); blockIdx.y = a slice of 128 (row, 4-column) elements, so that a thin batch still
    // spreads over many SMs
    const int b = blockIdx.x / a.Hkv, g = blockIdx.x % a.Hkv;
    const int nc = a.pv.nc[b], first = a.pv.first[b];
    const int n_rows_valid = a.R * a.group;
    if (nc == 1) return;
    for (int e = blockIdx.y * 128 + threadIdx.x; e < n_rows_valid * (DH / 4); e += 128 * gridDim.y) {
        const int r = e / (DH / 4), c4 = (e % (DH / 4)) * 4;
        float acc[4] = {0.f, 0.f, 0.f, 0.f}, L = 0.f, M = -INFINITY;
#pragma unroll 4
        for (int c = 0; c < nc; ++c) M = fmaxf(M, a.pv.part_ml[(((size_t)(first + c) * a.Hkv + g) * rows_alloc + r) * 2]);
#pragma unroll 4
        for (int c = 0; c < nc; ++c) {                       // chunk order: the sum does not depend on who computed what when
            const size_t ps = ((size_t)(first + c) * a.Hkv + g) * rows_alloc + r;
            const float mw = a.pv.part_ml[ps * 2];
            const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
            L += a.pv.part_ml[ps * 2 + 1] * f;
            const float4 v = *reinterpret_cast<const float4*>(a.pv.part_o + ps * DH + c4);
            acc[0] += v.x * f; acc[1] += v.y * f; acc[2] += v.z * f; acc[3] += v.w * f;
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        const int i = r / a.group, j = r % a.group;
        __nv_bfloat16* op = a.out + ((size_t)b * a.R + i) * a.out_row_stride + (size_t)(g * a.group + j) * DH + c4;
        uint2 pk;
        pk.x = pack_bf16(acc[0] * inv, acc[1] * inv);
        pk.y = pack_bf16(acc[2] * inv, acc[3] * inv);
        *reinterpret_cast<uint2*>(op) = pk;
    }
}

int sm_count()
{
    static std::atomic<int> cached[64];                      // per device ordinal; 0 = not asked yet
    int dev = 0;
    cudaGetDevice(&dev);
    int n = cached[dev & 63].load(std::memory_order_relaxed);
    if (n == 0) {
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
        cached[dev & 63].store(n, std::memory_order_relaxed);
    }
    return n;
}

template <int DH, int WM, int WN>
spec_status run_mma(const MmaArgs& m, int B, bool plan, int max_chunks, cudaStream_t st)
{
    constexpr int STAGES = 3;
    constexpr int smem = STAGES * (4 * kBT * DH * 2 * 2);
    static_assert(smem >= WN * 16 * WM * (DH + 2) * 4, "merge buffer fits in the stages");
    auto kern = attn_mma_kernel<DH, WM, WN, STAGES>;
    static PerDeviceOnce configured;
    int dev__ = 0;
    if (configured.needed(&dev__)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SPEC_ERR_CUDA;
        configured.done(dev__);
    }
    if (plan) {
        attn_plan_kernel<<<1, kPlanThreads, 0, st>>>(B, m.R, m.pos, m.Hkv, 2 * sm_count(), B * max_chunks, m.pv);
        if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    }
    const int ctas_per_sm = (228 * 1024) / (smem + 2048);
    launch_pdl(kern, dim3(sm_count() * (ctas_per_sm < 1 ? 1 : ctas_per_sm)), dim3(kThreads), (size_t)smem, st, m);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    launch_pdl(attn_merge_kernel<DH>, dim3(B * m.Hkv, (m.R * m.group * (DH / 4) + 127) / 128), dim3(128), 0, st, B, 16 * WM, m);
    return launch_status(plan ? 3 : 2);
}

}  // namespace

bool attention_mma_supported(const AttnArgs& a)
{
    const int rows = a.R * (a.Hq / a.Hkv);
    return a.dtype == SPEC_DTYPE_BF16 && a.block_tokens == kBT && (a.dh == 128 || a.dh == 64) && rows <= 64 &&
           a.q_row_stride % 2 == 0 && a.out_row_stride % 4 == 0;
}

size_t attention_mma_scratch_bytes(int B, int R, int Hq, int Hkv, int dh, int max_kv_len)
{
    return plan_scratch_bytes(B, Hkv, rows_alloc_for(R * (Hq / Hkv)), dh, max_chunks_for(max_kv_len));
}

spec_status attn::launch_attn_plan(int B, int R, const int32_t* pos, int Hkv, int n_ctas, int max_chunks, const PlanView& pv, cudaStream_t st)
{
    attn_plan_kernel<<<1, kPlanThreads, 0, st>>>(B, R, pos, Hkv, n_ctas, B * max_chunks, pv);
    return launch_status();
}

spec_status attn::launch_attn_merge128(int B, int rows_alloc, int Hkv, int R, int group, void* out, int out_row_stride,
                                       const PlanView& pv, cudaStream_t st)
{
    MmaArgs m{};
    m.R = R; m.group = group; m.Hkv = Hkv; m.out = static_cast<__nv_bfloat16*>(out); m.out_row_stride = out_row_stride; m.pv = pv;
    launch_pdl(attn_merge_kernel<128>, dim3(B * Hkv, (R * group * 32 + 127) / 128), dim3(128), 0, st, B, rows_alloc, m);
    return launch_status();
}

spec_status launch_attention_mma(const AttnArgs& a, cudaStream_t st)
{
    const int group = a.Hq / a.Hkv, rows = a.R * group;
    const int rows_alloc = rows_alloc_for(rows);
    if (a.scratch_bytes < attention_mma_scratch_bytes(a.B, a.R, a.Hq, a.Hkv, a.dh, a.max_kv_len)) return SPEC_ERR_SHAPE;
    const int max_chunks = max_chunks_for(a.max_kv_len);
    const PlanView pv = carve_plan(a.scratch, a.B, a.Hkv, rows_alloc, a.dh, max_chunks);
    MmaArgs m{(const __nv_bfloat16*)a.q, a.q_row_stride, (const __nv_bfloat16*)a.k_pool, (const __nv_bfloat16*)a.v_pool,
              a.block_table, a.max_blocks, a.pos, a.R, group, a.Hkv, (__nv_bfloat16*)a.out, a.out_row_stride,
              1.4426950408889634f / sqrtf((float)a.dh), pv, a.launch_index % kCounters};
    const bool plan = a.launch_index % kCounters == 0;
    if (a.dh == 128) {
        if (rows_alloc == 16) return run_mma<128, 1, 4>(m, a.B, plan, max_chunks, st);
        if (rows_alloc == 32) return run_mma<128, 2, 2>(m, a.B, plan, max_chunks, st);
        return run_mma<128, 4, 1>(m, a.B, plan, max_chunks, st);
    }
    if (rows_alloc == 16) return run_mma<64, 1, 4>(m, a.B, plan, max_chunks, st);
    if (rows_alloc == 32) return run_mma<64, 2, 2>(m, a.B, plan, max_chunks, st);
    return run_mma<64, 4, 1>(m, a.B, plan, max_chunks, st);
}

}  // namespace spec
