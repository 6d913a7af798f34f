// Paged grouped-query attention on the 5th-generation tensor cores, for 17..128 query rows per KV head (head_dim 128).
//
// With more than 16 query rows per KV head (long drafts, wide query groups: 64 rows for a 16-head group at k = 3) the
// register-fragment kernel re-reads every K/V tile from shared memory once per 16 rows and runs out of shared-memory
// bandwidth and issue slots before it runs out of HBM.  Here the rows are the M dimension of tcgen05.mma, which reads
// its operands from shared memory once per tile whatever M is:
//   - work units (sequence, KV head, chunk of <= 4096 tokens) come from the same plan and atomic counter as the
//     register-fragment kernel; one persistent CTA per SM;
//   - warp 0 pulls units and streams their K and V tiles of 128 tokens with TMA straight from the paged pools: one
//     64-column x 16-row box per (block, half of head_dim), 128-byte swizzle, so a tile lands as [half][token][64] -
//     K-major for S = Q K^T and MN-major for O += P V - in two 2-stage rings (K and V are released separately);
//   - warp 1 issues the MMAs from one thread: S (128 x 128, fp32) into one of two tensor-memory buffers, O (128 x 128)
//     accumulated in a third;
//   - warps 2..5 are the softmax: thread = query row = tensor-memory lane (rows are dealt round-robin over the four
//     32-lane quarters so that few rows still use all four warps).  Row maximum and exponentials in the exp2 domain; the
//     running maximum is only raised when a tile exceeds it by more than 2^8 (the accumulator and the row sum are then
//     rescaled in tensor memory), otherwise the stale maximum is kept - the final division makes both exact; P is
//     written to shared memory as bf16 in the K-major swizzled layout the second MMA reads;
//   - per unit the softmax threads stage Q (zero-padded to 128 rows) and write the result: normalised bf16 for
//     single-chunk sequences, (max, sum, unnormalised fp32 row) partials for the merge kernel otherwise.
// Every mbarrier wait is bounded (abort flag -> SPEC_ERR_TIMEOUT, tensor memory released, kernel returns).
#include <cuda.h>

#include "attention_plan.cuh"
#include "tc_common.cuh"

namespace spec {
using namespace tc;
namespace attn {
namespace {

constexpr int DH = 128, T = 128;                  // head_dim; KV tokens per tile
constexpr int kThreadsTc = 192;
constexpr int kSoftmaxThreads = 128;
constexpr int kHalfBytes = 128 * 128;             // [128 rows][64 bf16], 128-byte rows, swizzled
constexpr int kTileBytes = 2 * kHalfBytes;        // Q, P, one K tile, one V tile
constexpr int kStages = 2;
constexpr int NQ = 4;                             // unit queue depth (the producer runs ahead of the consumers)
constexpr uint32_t kTmemCols = 512;               // S0 [0,128), S1 [128,256), O [256,384)
constexpr int kSmemTc = (2 + 2 * kStages) * kTileBytes + 1024 + 512;
constexpr float kRescaleGap = 8.f;                // log2 units

struct UnitMsg { int b, g, t0, t1, slot, pad0, pad1, pad2; };

struct Ctl {
    uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
    uint64_t s_full[2], s_empty[2], p_full, pv_done, q_ready, uq_full[NQ], uq_empty[NQ], drain;
    UnitMsg uq[NQ];
    uint32_t tmem_base;
    int abort;
};
static_assert(sizeof(Ctl) <= 512, "control block fits its slot");

struct TcArgs {
    const __nv_bfloat16* q; int q_row_stride;
    const int32_t* block_table; int max_blocks;
    const int32_t* pos;
    int R, group, Hkv, rows_alloc;
    __nv_bfloat16* out; int out_row_stride;
    float scale_log2;
    PlanView pv;
    int counter_index;
    int32_t* status;
};

// K-major or MN-major tile of 128-byte swizzled rows: start address >> 4, leading byte offset >> 4 at bit 16, stride
// byte offset >> 4 at bit 32, descriptor version 1 at bit 46, layout type 2 (SWIZZLE_128B) at bit 61.
__device__ __forceinline__ uint64_t tile_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// D fp32, A and B bf16, M = 128, N = 128; bit 16 set: B is MN-major (V tiles are [token][head_dim]).
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t kIdescPV = kIdescQK | (1u << 16);

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kThreadsTc, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap map_k,
                                                                const __grid_constant__ CUtensorMap map_v, const TcArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);
    const uint32_t q_s = base, p_s = base + kTileBytes, k_s = base + 2 * kTileBytes, v_s = k_s + kStages * kTileBytes;
    Ctl* ctl = reinterpret_cast<Ctl*>(base_ptr + (2 + 2 * kStages) * kTileBytes);
    volatile int* abort_flag = &ctl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // finite contents everywhere: masked probabilities are exact zeros, and 0 x (stale but finite) stays 0
    for (int i = threadIdx.x; i < (2 + 2 * kStages) * kTileBytes / 16; i += kThreadsTc)
        reinterpret_cast<uint4*>(base_ptr)[i] = make_uint4(0u, 0u, 0u, 0u);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&ctl->k_full[s]), 1); mbar_init(smem_u32(&ctl->k_empty[s]), 1);
            mbar_init(smem_u32(&ctl->v_full[s]), 1); mbar_init(smem_u32(&ctl->v_empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ctl->s_full[s]), 1); mbar_init(smem_u32(&ctl->s_empty[s]), kSoftmaxThreads); }
        mbar_init(smem_u32(&ctl->p_full), kSoftmaxThreads);
        mbar_init(smem_u32(&ctl->pv_done), 1);
        mbar_init(smem_u32(&ctl->q_ready), kSoftmaxThreads);
        for (int s = 0; s < NQ; ++s) { mbar_init(smem_u32(&ctl->uq_full[s]), 1); mbar_init(smem_u32(&ctl->uq_empty[s]), 5); }
        mbar_init(smem_u32(&ctl->drain), 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_proxy_async();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int rows_valid = a.R * a.group;

    if (warp == 0) {
        // ---- producer: unit queue + TMA ring ----
        if (lane == 0) {
            uint32_t ks = 0, kph = 0, vs = 0, vph = 0;
            bool ok = true;
            const int n_units = *a.pv.n_entries * a.Hkv;
            for (int n = 0; ok; ++n) {
                const int slot_q = n % NQ;
                if (!mbar_wait(smem_u32(&ctl->uq_empty[slot_q]), (((uint32_t)(n / NQ)) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                const int u = atomicAdd(&a.pv.counters[a.counter_index], 1);
                UnitMsg msg{0, 0, 0, -1, -1, 0, 0, 0};
                if (u < n_units) {
                    const Unit un = a.pv.entries[u / a.Hkv];
                    msg.b = un.b; msg.g = u % a.Hkv; msg.t0 = un.t0; msg.t1 = un.t1; msg.slot = un.slot;
                }
                ctl->uq[slot_q] = msg;
                mbar_arrive(smem_u32(&ctl->uq_full[slot_q]));
                if (msg.t1 < 0) break;
                const int32_t* table = a.block_table + (size_t)msg.b * a.max_blocks;
                const int n_tiles = (msg.t1 - msg.t0 + T - 1) / T;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const int blk0 = (msg.t0 + j * T) / kBT;
                    int phys[T / kBT];
                    int n_ok = 0;
#pragma unroll
                    for (int bb = 0; bb < T / kBT; ++bb) {
                        const int bi = blk0 + bb;
                        phys[bb] = (bi * kBT < msg.t1 && bi < a.max_blocks) ? table[bi] : -1;
                        n_ok += phys[bb] >= 0;
                    }
                    // K tile
                    if (!mbar_wait(smem_u32(&ctl->k_empty[ks]), kph ^ 1u, abort_flag)) { ok = false; break; }
                    {
                        const uint32_t bar = smem_u32(&ctl->k_full[ks]);
                        mbar_expect_tx(bar, (uint32_t)n_ok * 2u * (kBT * 128));
                        const uint32_t dst = k_s + ks * kTileBytes;
#pragma unroll
                        for (int bb = 0; bb < T / kBT; ++bb) {
                            if (phys[bb] < 0) continue;
                            const int row = (phys[bb] * a.Hkv + msg.g) * kBT;
                            tma_load_2d(dst + bb * (kBT * 128), &map_k, 0, row, bar);
                            tma_load_2d(dst + kHalfBytes + bb * (kBT * 128), &map_k, 64, row, bar);
                        }
                        if (++ks == kStages) { ks = 0; kph ^= 1u; }
                    }
                    // V tile
                    if (!mbar_wait(smem_u32(&ctl->v_empty[vs]), vph ^ 1u, abort_flag)) { ok = false; break; }
                    {
                        const uint32_t bar = smem_u32(&ctl->v_full[vs]);
                        mbar_expect_tx(bar, (uint32_t)n_ok * 2u * (kBT * 128));
                        const uint32_t dst = v_s + vs * kTileBytes;
#pragma unroll
                        for (int bb = 0; bb < T / kBT; ++bb) {
                            if (phys[bb] < 0) continue;
                            const int row = (phys[bb] * a.Hkv + msg.g) * kBT;
                            tma_load_2d(dst + bb * (kBT * 128), &map_v, 0, row, bar);
                            tma_load_2d(dst + kHalfBytes + bb * (kBT * 128), &map_v, 64, row, bar);
                        }
                        if (++vs == kStages) { vs = 0; vph ^= 1u; }
                    }
                }
            }
            if (!ok) {                                  // give copies in flight time to land before the CTA goes away
                const long long t0c = clock64();
                while (clock64() - t0c < 200000) { }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ----
        if (lane == 0) {
            uint32_t ks = 0, kph = 0, vs = 0, vph = 0;
            uint32_t n_qk = 0, n_pv = 0;              // running tile counters (phases of the S / P barriers)
            bool ok = true;
            const uint32_t o_tmem = tmem_base + 256;
            auto issue_qk = [&]() -> bool {
                const uint32_t buf = n_qk & 1u;
                if (!mbar_wait(smem_u32(&ctl->k_full[ks]), kph, abort_flag)) return false;
                if (!mbar_wait(smem_u32(&ctl->s_empty[buf]), ((n_qk >> 1) & 1u) ^ 1u, abort_flag)) return false;
                tc_fence_after();
                const uint32_t kb = k_s + ks * kTileBytes;
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        tc_mma(tmem_base + buf * 128, tile_desc(q_s + h * kHalfBytes + kk * 32, 16, 1024),
                               tile_desc(kb + h * kHalfBytes + kk * 32, 16, 1024), kIdescQK, (h | kk) ? 1u : 0u);
                tc_commit(smem_u32(&ctl->k_empty[ks]));
                tc_commit(smem_u32(&ctl->s_full[buf]));
                if (++ks == kStages) { ks = 0; kph ^= 1u; }
                ++n_qk;
                return true;
            };
            for (int n = 0; ok; ++n) {
                const int slot_q = n % NQ;
                if (!mbar_wait(smem_u32(&ctl->uq_full[slot_q]), ((uint32_t)(n / NQ)) & 1u, abort_flag)) { ok = false; break; }
                const int t0 = ctl->uq[slot_q].t0, t1 = ctl->uq[slot_q].t1;
                mbar_arrive(smem_u32(&ctl->uq_empty[slot_q]));
                if (t1 < 0) break;
                const int n_tiles = (t1 - t0 + T - 1) / T;
                if (!mbar_wait(smem_u32(&ctl->q_ready), (uint32_t)n & 1u, abort_flag)) { ok = false; break; }
                if (!issue_qk()) { ok = false; break; }
                for (int j = 0; j < n_tiles; ++j) {
                    if (j + 1 < n_tiles && !issue_qk()) { ok = false; break; }
                    if (!mbar_wait(smem_u32(&ctl->p_full), n_pv & 1u, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(smem_u32(&ctl->v_full[vs]), vph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t vb = v_s + vs * kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < T / 16; ++kk)      // 16 tokens per instruction: two 8-token groups of the V tile
                        tc_mma(o_tmem, tile_desc(p_s + (kk >> 2) * kHalfBytes + (kk & 3) * 32, 16, 1024),
                               tile_desc(vb + kk * 2048, kHalfBytes, 1024), kIdescPV, (j > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&ctl->v_empty[vs]));
                    tc_commit(smem_u32(&ctl->pv_done));
                    if (++vs == kStages) { vs = 0; vph ^= 1u; }
                    ++n_pv;
                }
            }
            if (!ok) {                                  // drain issued tensor-core work before tensor memory is freed
                tc_commit(smem_u32(&ctl->drain));
                const long long t0c = clock64();
                while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && clock64() - t0c < kWaitLimit) { }
            }
        }
    } else {
        // ---- softmax warps: thread = MMA row m = quarter * 32 + lane; query row r = lane * 4 + quarter ----
        const int quarter = warp & 3;
        const int m = quarter * 32 + lane;
        const int r = lane * 4 + quarter;
        const bool row_ok = r < rows_valid;
        const int ri = row_ok ? r / a.group : 0, rj = row_ok ? r % a.group : 0;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t o_tmem = t_lane + 256;
        uint32_t n_tile = 0;                          // running tile counter (same sequence as the MMA warp's)
        bool ok = true;
        for (int n = 0; ok; ++n) {
            const int slot_q = n % NQ;
            if (!mbar_wait(smem_u32(&ctl->uq_full[slot_q]), ((uint32_t)(n / NQ)) & 1u, abort_flag)) { ok = false; break; }
            const UnitMsg un = ctl->uq[slot_q];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->uq_empty[slot_q]));
            if (un.t1 < 0) break;
            const int n_tiles = (un.t1 - un.t0 + T - 1) / T;
            // stage Q: the previous unit's S tiles have all been read, so no MMA still reads the buffer
            int lim = -1;
            if (row_ok) {
                lim = a.pos[(size_t)un.b * a.R + ri];
                const uint4* qp = reinterpret_cast<const uint4*>(a.q + ((size_t)un.b * a.R + ri) * a.q_row_stride +
                                                                 (size_t)(un.g * a.group + rj) * DH);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const uint4 v = qp[c];
                    const uint32_t off = (uint32_t)((c >> 3) * kHalfBytes + m * 128 + (((c & 7) ^ (m & 7)) << 4));
                    *reinterpret_cast<uint4*>(base_ptr + off) = v;
                }
            }
            fence_proxy_async();
            mbar_arrive(smem_u32(&ctl->q_ready));

            float m_used = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_tiles; ++j, ++n_tile) {
                const uint32_t buf = n_tile & 1u;
                if (!mbar_wait(smem_u32(&ctl->s_full[buf]), (n_tile >> 1) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const int tok0 = un.t0 + j * T;
                const int vis = min(lim + 1, un.t1) - tok0;       // this row sees tile columns [0, vis)
                // pass 1: row maximum
                float mx = -INFINITY;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t v[32];
                    tc_ld32(t_lane + buf * 128 + c * 32, v);
                    tc_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (c * 32 + e < vis) mx = fmaxf(mx, __uint_as_float(v[e]));
                    }
                }
                mx *= a.scale_log2;                               // scale > 0; -inf stays -inf
                float alpha = 1.f;
                bool raise = false;
                if (row_ok && mx > -INFINITY && (m_used == -INFINITY || mx > m_used + kRescaleGap)) {
                    alpha = m_used == -INFINITY ? 0.f : exp2f(m_used - mx);
                    raise = j > 0;                                // the first tile overwrites the accumulator
                    m_used = mx;
                    l_run *= alpha;
                }
                const float ms = m_used == -INFINITY ? 0.f : m_used;
                // pass 2: probabilities, packed to bf16
                uint32_t pk[64];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t v[32];
                    tc_ld32(t_lane + buf * 128 + c * 32, v);
                    tc_wait_ld();
                    if (c == 3) { tc_fence_before(); mbar_arrive(smem_u32(&ctl->s_empty[buf])); }
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float p0 = 0.f, p1 = 0.f;
                        if (row_ok) {
                            if (c * 32 + e < vis) p0 = exp2f(fmaf(__uint_as_float(v[e]), a.scale_log2, -ms));
                            if (c * 32 + e + 1 < vis) p1 = exp2f(fmaf(__uint_as_float(v[e + 1]), a.scale_log2, -ms));
                        }
                        l_run += p0 + p1;
                        pk[c * 16 + e / 2] = pack2(p0, p1);
                    }
                }
                // the previous tile's P V has finished: P may be overwritten and the accumulator is at rest
                if (n_tile > 0 && !mbar_wait(smem_u32(&ctl->pv_done), (n_tile - 1u) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                if (__any_sync(0xffffffffu, raise)) {
                    const float f = raise ? alpha : 1.f;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t v[32];
                        tc_ld32(o_tmem + c * 32, v);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * f);
                        tc_st32(o_tmem + c * 32, v);
                    }
                    tc_wait_st();
                }
                if (row_ok) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) {                // 16-byte chunk c holds tokens 8c .. 8c+7
                        const uint32_t off = (uint32_t)(kTileBytes + (c >> 3) * kHalfBytes + m * 128 + (((c & 7) ^ (m & 7)) << 4));
                        *reinterpret_cast<uint4*>(base_ptr + off) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                    }
                }
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->p_full));
            }
            if (!ok) break;
            // ---- unit result ----
            if (!mbar_wait(smem_u32(&ctl->pv_done), (n_tile - 1u) & 1u, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            float* part = nullptr;
            __nv_bfloat16* op = nullptr;
            if (row_ok) {
                if (un.slot >= 0) {
                    const size_t ps = ((size_t)un.slot * a.Hkv + un.g) * a.rows_alloc + r;
                    part = a.pv.part_o + ps * DH;
                    a.pv.part_ml[ps * 2] = m_used;
                    a.pv.part_ml[ps * 2 + 1] = l_run;
                } else {
                    op = a.out + ((size_t)un.b * a.R + ri) * a.out_row_stride + (size_t)(un.g * a.group + rj) * DH;
                }
            }
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t v[32];
                tc_ld32(o_tmem + c * 32, v);
                tc_wait_ld();
                if (part != nullptr) {
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        *reinterpret_cast<float4*>(part + c * 32 + e) =
                            make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]), __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                } else if (op != nullptr) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 o;
                        o.x = pack2(__uint_as_float(v[e]) * inv, __uint_as_float(v[e + 1]) * inv);
                        o.y = pack2(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv);
                        o.z = pack2(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv);
                        o.w = pack2(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv);
                        *reinterpret_cast<uint4*>(op + c * 32 + e) = o;
                    }
                }
            }
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && ctl->abort) set_status(a.status, SPEC_ERR_TIMEOUT, (int)blockIdx.x);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

bool attention_tc_supported(const AttnArgs& a)
{
    const int rows = a.R * (a.Hq / a.Hkv);
    return a.dtype == SPEC_DTYPE_BF16 && a.block_tokens == kBT && a.dh == DH && rows > 16 && rows <= 128 &&
           a.q_row_stride % 8 == 0 && a.out_row_stride % 8 == 0 && (reinterpret_cast<uintptr_t>(a.q) & 15u) == 0 &&
           (reinterpret_cast<uintptr_t>(a.out) & 15u) == 0 && (reinterpret_cast<uintptr_t>(a.k_pool) & 15u) == 0 &&
           (reinterpret_cast<uintptr_t>(a.v_pool) & 15u) == 0;
}

spec_status launch_attention_tc(const AttnArgs& a, cudaStream_t st)
{
    const int group = a.Hq / a.Hkv, rows = a.R * group;
    const int rows_alloc = rows_alloc_for(rows);
    const int max_chunks = max_chunks_for(a.max_kv_len);
    if (a.scratch_bytes < attention_mma_scratch_bytes(a.B, a.R, a.Hq, a.Hkv, a.dh, a.max_kv_len)) return SPEC_ERR_SHAPE;
    const PlanView pv = carve_plan(a.scratch, a.B, a.Hkv, rows_alloc, a.dh, max_chunks);
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc) != cudaSuccess) return SPEC_ERR_CUDA;
        configured = true;
    }
    // the pools as matrices of 128-column rows ((block, head, token) flattened); one box = 64 columns x 16 tokens
    CUtensorMap mk, mv;
    const uint64_t pool_rows = 1ull << 31;
    if (!tc_make_map_2d(&mk, a.k_pool, pool_rows, DH, DH, 64, kBT)) return SPEC_ERR_CUDA;
    if (!tc_make_map_2d(&mv, a.v_pool, pool_rows, DH, DH, 64, kBT)) return SPEC_ERR_CUDA;
    TcArgs t{(const __nv_bfloat16*)a.q, a.q_row_stride, a.block_table, a.max_blocks, a.pos, a.R, group, a.Hkv, rows_alloc,
             (__nv_bfloat16*)a.out, a.out_row_stride, 1.4426950408889634f / sqrtf((float)a.dh), pv, a.launch_index % kCounters,
             a.status};
    if (a.launch_index % kCounters == 0) {
        spec_status s = launch_attn_plan(a.B, a.R, a.pos, max_chunks, pv, st);
        if (s != SPEC_OK) return s;
    }
    attn_tc_kernel<<<tc_sm_count(), kThreadsTc, kSmemTc, st>>>(mk, mv, t);
    if (launch_status() != SPEC_OK) return SPEC_ERR_CUDA;
    return launch_attn_merge128(a.B, rows_alloc, a.Hkv, a.R, group, a.out, a.out_row_stride, pv, st);
}

}  // namespace attn
}  // namespace spec
