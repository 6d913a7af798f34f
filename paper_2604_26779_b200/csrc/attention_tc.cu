// Paged grouped-query attention on the 5th-generation tensor cores, for 17..128 query rows per KV head (head_dim 128).
//
// With more than 16 query rows per KV head (long drafts, wide query groups: 64 rows for a 16-head group at k = 3) the
// register-fragment kernel re-reads every K/V tile from shared memory once per 16 rows and runs out of shared-memory
// bandwidth and issue slots before it runs out of HBM.  Here the rows are the M dimension of tcgen05.mma, which reads
// its operands once per tile whatever M is:
//   - work units (sequence, KV head, chunk of about 4096 tokens) come from the same plan and atomic counter as the
//     register-fragment kernel; one persistent CTA per SM;
//   - four producer warps stream the K and V tiles of 128 tokens with TMA straight from the paged pools: one 64-column
//     x 16-row box per (block, half of head_dim), 128-byte swizzle, so a tile lands as [half][token][64] - K-major for
//     S = Q K^T and MN-major for O += P V - in a 4-stage K ring and a 3-stage V ring, which is all that shared memory
//     holds; warp 0 also pulls the units and publishes them to the other roles through a small queue;
//   - warp 1 issues the MMAs from one thread: S (128 x 128, fp32) into one of two tensor-memory buffers, O (128 x 128)
//     accumulated in a third; both A operands, Q and P, are read from tensor memory (bf16 pairs);
//   - warps 2..5 are the softmax; query rows are dealt round-robin over the four 32-lane quarters of tensor memory and
//     the scores are read in the 16-lane fragment shape, so the 32 threads of a warp share the columns of 16 rows (the
//     exponentials, 4 per clock and scheduler whatever the number of active lanes, are what a tile costs).  Row maximum
//     and exponentials in the exp2 domain; the running maximum is only raised when a tile exceeds it by more than 2^8
//     (the accumulator and the row sum are then rescaled in tensor memory), otherwise the stale maximum is kept - the
//     final division makes both exact; P goes back to tensor memory with one store per 16 rows;
//   - per unit the softmax threads stage Q (zero-padded to 128 rows) in tensor memory and write the result: normalised
//     bf16 for single-chunk sequences, (max, sum, unnormalised fp32 row) partials for the merge kernel otherwise.
// Every mbarrier wait is bounded (abort flag -> SPEC_ERR_TIMEOUT, tensor memory released, kernel returns).
#include <cuda.h>

#include "attention_plan.cuh"
#include "tc_common.cuh"

namespace spec {
using namespace tc;
namespace attn {
namespace {

constexpr int DH = 128, T = 128;                  // head_dim; KV tokens per tile
constexpr int kThreadsTc = 416;                  // warps: 0, 7 K producers; 6, 8 V producers; 1 MMA; 2..5 and 9..12 softmax
constexpr int kSoftmaxThreads = 256;
constexpr int kHalfBytes = 128 * 128;             // [128 rows][64 bf16], 128-byte rows, swizzled
constexpr int kTileBytes = 2 * kHalfBytes;        // one K tile or one V tile of 128 tokens
constexpr int kStagesK = 3, kStagesV = 3;
constexpr int NQ = 4;                             // unit queue depth (the producer runs ahead of the consumers)
constexpr uint32_t kTmemCols = 512;               // S0 [0,128), S1 [128,256), O [256,384), Q [384,448) and P [448,512) as bf16 pairs
constexpr int kSmemTc = (kStagesK + kStagesV) * kTileBytes + 1024 + 4096;
constexpr float kRescaleGap = 8.f;                // log2 units

struct UnitMsg { int b, g, t0, t1, slot, pad0, pad1, pad2; };

struct Ctl {
    uint64_t k_full[kStagesK], k_empty[kStagesK], v_full[kStagesV], v_empty[kStagesV];
    uint64_t s_full[2], s_empty[2], p_full, pv_done, q_ready, uq_full[NQ], uq_empty[NQ], drain;
    UnitMsg uq[NQ];
    float xmax[2][4][2][2][16];      // [tile parity][quarter][side][half][row]: row maxima exchanged by the two sides
    float xsum[4][2][32];            // [quarter][side][lane]: row sums at the end of a unit
    uint32_t tmem_base;
    int abort;
};
static_assert(sizeof(Ctl) <= 4096, "control block fits its slot");

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

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int H>
__global__ void __launch_bounds__(kThreadsTc, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap map_k,
                                                                const __grid_constant__ CUtensorMap map_v, const TcArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - raw);
    const uint32_t k_s = base, v_s = k_s + kStagesK * kTileBytes;
    Ctl* ctl = reinterpret_cast<Ctl*>(base_ptr + (kStagesK + kStagesV) * kTileBytes);
    volatile int* abort_flag = &ctl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // finite contents everywhere: masked probabilities are exact zeros, and 0 x (stale but finite) stays 0
    for (int i = threadIdx.x; i < (kStagesK + kStagesV) * kTileBytes / 16; i += kThreadsTc)
        reinterpret_cast<uint4*>(base_ptr)[i] = make_uint4(0u, 0u, 0u, 0u);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesK; ++s) { mbar_init(smem_u32(&ctl->k_full[s]), 2); mbar_init(smem_u32(&ctl->k_empty[s]), 1); }
        for (int s = 0; s < kStagesV; ++s) { mbar_init(smem_u32(&ctl->v_full[s]), 2); mbar_init(smem_u32(&ctl->v_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ctl->s_full[s]), 1); mbar_init(smem_u32(&ctl->s_empty[s]), kSoftmaxThreads); }
        mbar_init(smem_u32(&ctl->p_full), kSoftmaxThreads);
        mbar_init(smem_u32(&ctl->pv_done), 1);
        mbar_init(smem_u32(&ctl->q_ready), kSoftmaxThreads);
        for (int s = 0; s < NQ; ++s) { mbar_init(smem_u32(&ctl->uq_full[s]), 1); mbar_init(smem_u32(&ctl->uq_empty[s]), 12); }
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

    if (warp == 0 || (warp >= 6 && warp <= 8)) {
        // ---- producers: one thread issues a TMA box in ~100 cycles and a tile needs 16 per operand, so four warps share
        // them: warps 0 and 7 the even and odd blocks of the K tiles, warps 6 and 8 those of the V tiles.  Warp 0 also pulls
        // the units and publishes them to everyone else. ----
        if (lane == 0) {
            const bool is_k = warp == 0 || warp == 7;
            const int parity_b = warp >= 7 ? 1 : 0;
            const CUtensorMap* map = is_k ? &map_k : &map_v;
            uint64_t* full = is_k ? ctl->k_full : ctl->v_full;
            uint64_t* empty = is_k ? ctl->k_empty : ctl->v_empty;
            const uint32_t ring = is_k ? k_s : v_s;
            uint32_t st = 0, ph = 0;
            bool ok = true;
            const int n_units = *a.pv.n_entries * a.Hkv;
            for (int n = 0; ok; ++n) {
                const int slot_q = n % NQ;
                UnitMsg msg{0, 0, 0, -1, -1, 0, 0, 0};
                if (warp == 0) {
                    if (!mbar_wait(smem_u32(&ctl->uq_empty[slot_q]), (((uint32_t)(n / NQ)) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    const int u = atomicAdd(&a.pv.counters[a.counter_index], 1);
                    if (u < n_units) {
                        const Unit un = a.pv.entries[u / a.Hkv];
                        msg.b = un.b; msg.g = u % a.Hkv; msg.t0 = un.t0; msg.t1 = un.t1; msg.slot = un.slot;
                    }
                    ctl->uq[slot_q] = msg;
                    mbar_arrive(smem_u32(&ctl->uq_full[slot_q]));
                } else {
                    if (!mbar_wait(smem_u32(&ctl->uq_full[slot_q]), ((uint32_t)(n / NQ)) & 1u, abort_flag)) { ok = false; break; }
                    msg = ctl->uq[slot_q];
                    mbar_arrive(smem_u32(&ctl->uq_empty[slot_q]));
                }
                if (msg.t1 < 0) break;
                const int32_t* table = a.block_table + (size_t)msg.b * a.max_blocks;
                const int n_tiles = (msg.t1 - msg.t0 + T - 1) / T;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const int blk0 = (msg.t0 + j * T) / kBT;
                    int phys[T / kBT / 2];
                    int n_ok = 0;
#pragma unroll
                    for (int hb = 0; hb < T / kBT / 2; ++hb) {
                        const int bi = blk0 + 2 * hb + parity_b;
                        phys[hb] = (bi * kBT < msg.t1 && bi < a.max_blocks) ? table[bi] : -1;
                        n_ok += phys[hb] >= 0;
                    }
                    if (!mbar_wait(smem_u32(&empty[st]), ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t bar = smem_u32(&full[st]);
                    mbar_expect_tx(bar, (uint32_t)n_ok * 2u * (kBT * 128));
                    const uint32_t dst = ring + st * kTileBytes;
#pragma unroll
                    for (int hb = 0; hb < T / kBT / 2; ++hb) {
                        if (phys[hb] < 0) continue;
                        const int bb = 2 * hb + parity_b;
                        const int row = (phys[hb] * a.Hkv + msg.g) * kBT;
                        tma_load_2d(dst + bb * (kBT * 128), map, 0, row, bar);
                        tma_load_2d(dst + kHalfBytes + bb * (kBT * 128), map, 64, row, bar);
                    }
                    if (++st == (is_k ? kStagesK : kStagesV)) { st = 0; ph ^= 1u; }
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
                        tc_mma_ta(tmem_base + buf * 128, tmem_base + 384 + (h * 4 + kk) * 8,
                                  tile_desc(kb + h * kHalfBytes + kk * 32, 16, 1024), kIdescQK, (h | kk) ? 1u : 0u);
                tc_commit(smem_u32(&ctl->k_empty[ks]));
                tc_commit(smem_u32(&ctl->s_full[buf]));
                if (++ks == kStagesK) { ks = 0; kph ^= 1u; }
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
                        tc_mma_ta(o_tmem, tmem_base + 448 + kk * 8, tile_desc(vb + kk * 2048, kHalfBytes, 1024), kIdescPV,
                                  (j > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&ctl->v_empty[vs]));
                    tc_commit(smem_u32(&ctl->pv_done));
                    if (++vs == kStagesV) { vs = 0; vph ^= 1u; }
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
        // ---- softmax warps: 2..5 (columns 0..63 of every score tile) and 9..12 (columns 64..127).  Query row r lives in MMA
        // row / tensor-memory lane (r % 4) * 32 + r / 4, so every 32-lane quarter - which one warp of each side may touch -
        // holds rows_valid / 4 rows in its first lanes.  The scores are read in the 16-lane fragment shape (16x256b: a row's
        // 8 consecutive columns over the 4 threads of a quad, rows g4 and g4 + 8 per thread, as in an mma accumulator), so
        // the 32 threads of a warp share its 64 columns of 16 rows: 32 scores per thread and tile with up to 64 query rows
        // (H = 1), 64 with up to 128 (H = 2: both 16-lane halves).  The two warps of a quarter exchange their row maxima
        // through shared memory (a 64-thread named barrier per tile) and otherwise work on their own columns of S, P and O.
        // The exponentials are what a tile costs: 4 per clock and scheduler whatever the number of active lanes.
        const int quarter = warp & 3;
        const int x = warp >= 9 ? 1 : 0;              // column half
        const int g4 = lane >> 2, q4 = lane & 3;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t o_tmem = t_lane + 256;
        // staging / result mapping: thread = tensor-memory lane, this side's half of the row
        const int r_st = lane * 4 + quarter;
        const bool st_ok = r_st < rows_valid;
        const int st_i = st_ok ? r_st / a.group : 0, st_j = st_ok ? r_st % a.group : 0;
        // score mapping: rows (h, hh) -> lane-in-quarter h * 16 + g4 + 8 * hh
        bool rok[H][2];
        int ri[H][2];
#pragma unroll
        for (int h = 0; h < H; ++h)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int r = (h * 16 + g4 + 8 * hh) * 4 + quarter;
                rok[h][hh] = r < rows_valid;
                ri[h][hh] = rok[h][hh] ? r / a.group : 0;
            }
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + quarter) : "memory"); };
        {   // rows without a query row hold zeros in Q and P for the whole launch
            uint32_t z[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) z[e] = 0u;
            tc_st32(t_lane + 384 + x * 32, z);
            tc_st32(t_lane + 448 + x * 32, z);
            tc_wait_st();
        }
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
            // stage this side's half of Q in tensor memory (the A operand of S = Q K^T): thread = row, 32 columns of bf16
            // pairs.  The previous unit's S tiles have all been read, so no MMA still reads it.
            {
                uint32_t qv[32];
                const uint4* qp = reinterpret_cast<const uint4*>(a.q + ((size_t)un.b * a.R + st_i) * a.q_row_stride +
                                                                 (size_t)(un.g * a.group + st_j) * DH) + x * 8;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 v = st_ok ? qp[c] : make_uint4(0u, 0u, 0u, 0u);
                    qv[c * 4] = v.x; qv[c * 4 + 1] = v.y; qv[c * 4 + 2] = v.z; qv[c * 4 + 3] = v.w;
                }
                tc_st32(t_lane + 384 + x * 32, qv);
                tc_wait_st();
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->q_ready));
            int lim[H][2];
            float m_used[H][2], l_run[H][2];          // l_run: this thread's share of the row sum (its columns)
#pragma unroll
            for (int h = 0; h < H; ++h)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    lim[h][hh] = rok[h][hh] ? a.pos[(size_t)un.b * a.R + ri[h][hh]] : -1;
                    m_used[h][hh] = -INFINITY;
                    l_run[h][hh] = 0.f;
                }

            for (int j = 0; j < n_tiles; ++j, ++n_tile) {
                const uint32_t buf = n_tile & 1u;
                if (!mbar_wait(smem_u32(&ctl->s_full[buf]), (n_tile >> 1) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const int tok0 = un.t0 + j * T;
                int vis[H][2];                                    // the row sees tile columns [0, vis)
                bool all_vis = true;
#pragma unroll
                for (int h = 0; h < H; ++h)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        vis[h][hh] = min(lim[h][hh] + 1, un.t1) - tok0;
                        all_vis = all_vis && (vis[h][hh] >= T || !rok[h][hh]);
                    }
                if (__all_sync(0xffffffffu, all_vis)) {           // most tiles need no masking: lift the limits out of reach
#pragma unroll
                    for (int h = 0; h < H; ++h) { vis[h][0] = 0x7fffffff; vis[h][1] = 0x7fffffff; }
                }
                // this side's 64 columns of every half, all loads before the one wait (a tensor-memory load takes a few
                // hundred cycles and this warp shares its scheduler with one other softmax warp at most)
                uint32_t v[H][32];
#pragma unroll
                for (int h = 0; h < H; ++h) tc_ld_16x256b_x8(t_lane + ((uint32_t)(h * 16) << 16) + buf * 128 + x * 64, v[h]);
                tc_wait_ld();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->s_empty[buf]));
                // row maxima: this thread's columns, the quad, then the other side's
                float mx[H][2];
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    mx[h][0] = -INFINITY; mx[h][1] = -INFINITY;
#pragma unroll
                    for (int jc = 0; jc < 8; ++jc)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int col = x * 64 + jc * 8 + 2 * q4 + (e & 1);
                            if (col >= vis[h][e >> 1]) v[h][4 * jc + e] = 0xff800000u;          // -inf: the exponential is an exact zero
                            mx[h][e >> 1] = fmaxf(mx[h][e >> 1], __uint_as_float(v[h][4 * jc + e]));
                        }
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        mx[h][hh] = fmaxf(mx[h][hh], __shfl_xor_sync(0xffffffffu, mx[h][hh], 1));
                        mx[h][hh] = fmaxf(mx[h][hh], __shfl_xor_sync(0xffffffffu, mx[h][hh], 2));
                        if (q4 == 0) ctl->xmax[buf][quarter][x][h][g4 + 8 * hh] = mx[h][hh];
                    }
                }
                pair_sync();
                uint32_t pk[H][16];                               // bf16 pairs: [2 * jc + hh]
                float alpha[H][2];
                bool raise = false;
#pragma unroll
                for (int h = 0; h < H; ++h) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        float m2 = fmaxf(mx[h][hh], ctl->xmax[buf][quarter][x ^ 1][h][g4 + 8 * hh]) * a.scale_log2;   // -inf stays -inf
                        alpha[h][hh] = 1.f;
                        if (rok[h][hh] && m2 > -INFINITY && (m_used[h][hh] == -INFINITY || m2 > m_used[h][hh] + kRescaleGap)) {
                            alpha[h][hh] = m_used[h][hh] == -INFINITY ? 0.f : exp2f(m_used[h][hh] - m2);
                            raise = raise || j > 0;               // the first tile overwrites the accumulator
                            m_used[h][hh] = m2;
                            l_run[h][hh] *= alpha[h][hh];
                        }
                    }
                    const float ms0 = m_used[h][0] == -INFINITY ? 0.f : m_used[h][0];
                    const float ms1 = m_used[h][1] == -INFINITY ? 0.f : m_used[h][1];
                    float l0 = 0.f, l1 = 0.f;
#pragma unroll
                    for (int jc = 0; jc < 8; ++jc) {
                        float p[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            p[e] = ex2_approx(fmaf(__uint_as_float(v[h][4 * jc + e]), a.scale_log2, (e >> 1) ? -ms1 : -ms0));
                        l0 += p[0] + p[1];
                        l1 += p[2] + p[3];
                        pk[h][2 * jc] = pack2(p[0], p[1]);
                        pk[h][2 * jc + 1] = pack2(p[2], p[3]);
                    }
                    l_run[h][0] += l0;
                    l_run[h][1] += l1;
                }
                // the previous tile's P V has finished: P may be overwritten and the accumulator is at rest
                if (n_tile > 0 && !mbar_wait(smem_u32(&ctl->pv_done), (n_tile - 1u) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                if (__any_sync(0xffffffffu, raise)) {             // this side's 64 columns of the accumulator
#pragma unroll
                    for (int h = 0; h < H; ++h) {
                        uint32_t o[32];
                        const uint32_t o_addr = o_tmem + ((uint32_t)(h * 16) << 16) + x * 64;
                        tc_ld_16x256b_x8(o_addr, o);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha[h][(e >> 1) & 1]);
                        tc_st_16x256b_x8(o_addr, o);
                    }
                    tc_wait_st();
                }
                // P goes to tensor memory as bf16 pairs (the A operand of O += P V): this side's 32 packed columns
#pragma unroll
                for (int h = 0; h < H; ++h) tc_st_16x128b_x8(t_lane + ((uint32_t)(h * 16) << 16) + 448 + x * 32, pk[h]);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->p_full));
            }
            if (!ok) break;
            // ---- unit result: thread = tensor-memory lane; the row's maximum and sum come from the quads that tracked it ----
            if (!mbar_wait(smem_u32(&ctl->pv_done), (n_tile - 1u) & 1u, abort_flag)) { ok = false; break; }
            tc_fence_after();
            float row_m = -INFINITY, row_l = 0.f;
#pragma unroll
            for (int h = 0; h < H; ++h)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    float l = l_run[h][hh];
                    l += __shfl_xor_sync(0xffffffffu, l, 1);
                    l += __shfl_xor_sync(0xffffffffu, l, 2);
                    const float tm = __shfl_sync(0xffffffffu, m_used[h][hh], 4 * (lane & 7));
                    const float tl = __shfl_sync(0xffffffffu, l, 4 * (lane & 7));
                    if ((lane >> 4) == h && ((lane >> 3) & 1) == hh) { row_m = tm; row_l = tl; }
                }
            ctl->xsum[quarter][x][lane] = row_l;                  // the row sum is the two sides' together
            pair_sync();
            row_l += ctl->xsum[quarter][x ^ 1][lane];
            const float inv = row_l > 0.f ? 1.f / row_l : 0.f;
            float* part = nullptr;
            __nv_bfloat16* op = nullptr;
            if (st_ok) {
                if (un.slot >= 0) {
                    const size_t ps = ((size_t)un.slot * a.Hkv + un.g) * a.rows_alloc + r_st;
                    part = a.pv.part_o + ps * DH + x * 64;
                    if (x == 0) { a.pv.part_ml[ps * 2] = row_m; a.pv.part_ml[ps * 2 + 1] = row_l; }
                } else {
                    op = a.out + ((size_t)un.b * a.R + st_i) * a.out_row_stride + (size_t)(un.g * a.group + st_j) * DH + x * 64;
                }
            }
            {
                uint32_t o[2][32];                    // this side's half of the row in one round trip to tensor memory
#pragma unroll
                for (int c = 0; c < 2; ++c) tc_ld32(o_tmem + x * 64 + c * 32, o[c]);
                tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    if (part != nullptr) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            *reinterpret_cast<float4*>(part + c * 32 + e) =
                                make_float4(__uint_as_float(o[c][e]), __uint_as_float(o[c][e + 1]), __uint_as_float(o[c][e + 2]),
                                            __uint_as_float(o[c][e + 3]));
                    } else if (op != nullptr) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint4 w;
                            w.x = pack2(__uint_as_float(o[c][e]) * inv, __uint_as_float(o[c][e + 1]) * inv);
                            w.y = pack2(__uint_as_float(o[c][e + 2]) * inv, __uint_as_float(o[c][e + 3]) * inv);
                            w.z = pack2(__uint_as_float(o[c][e + 4]) * inv, __uint_as_float(o[c][e + 5]) * inv);
                            w.w = pack2(__uint_as_float(o[c][e + 6]) * inv, __uint_as_float(o[c][e + 7]) * inv);
                            *reinterpret_cast<uint4*>(op + c * 32 + e) = w;
                        }
                    }
                }
            }
            pair_sync();                                          // the exchange slots are free for the next unit
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
    if (a.scratch_bytes < attention_mma_scratch_bytes(a.B, a.R, a.Hq, a.Hkv, a.dh, a.max_kv_len)) return SPEC_ERR_SHAPE;
    const int max_chunks = max_chunks_for(a.max_kv_len);
    const PlanView pv = carve_plan(a.scratch, a.B, a.Hkv, rows_alloc, a.dh, max_chunks);
    static PerDeviceOnce configured;
    int dev__ = 0;
    if (configured.needed(&dev__)) {
        if (cudaFuncSetAttribute(attn_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc) != cudaSuccess ||
            cudaFuncSetAttribute(attn_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc) != cudaSuccess)
            return SPEC_ERR_CUDA;
        configured.done(dev__);
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
        spec_status s = launch_attn_plan(a.B, a.R, a.pos, a.Hkv, tc_sm_count(), max_chunks, pv, st);
        if (s != SPEC_OK) return s;
    }
    if (rows <= 64) attn_tc_kernel<1><<<tc_sm_count(), kThreadsTc, kSmemTc, st>>>(mk, mv, t);
    else            attn_tc_kernel<2><<<tc_sm_count(), kThreadsTc, kSmemTc, st>>>(mk, mv, t);
    if (launch_status() != SPEC_OK) return SPEC_ERR_CUDA;
    return launch_attn_merge128(a.B, rows_alloc, a.Hkv, a.R, group, a.out, a.out_row_stride, pv, st);
}

}  // namespace attn
}  // namespace spec
