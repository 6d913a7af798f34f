// Work planning shared by the attention kernels: units of (sequence, KV chunk), their scratch layout, and the launchers
// of the planning and merge kernels.
#pragma once
#include "ops.cuh"

namespace spec {
namespace attn {

constexpr int kChunk = 4096;        // KV tokens per unit (upper bound); 4096 measured 3 % faster than 2048 and 1 % faster than 8192
constexpr int kChunkMin = 1024;     // thin batches cut finer, down to this (decided by the planning kernel)
constexpr int kChunkSlack = 128;    // ... plus this much, rather than opening one more chunk
constexpr int kTileTok = 64;        // chunk lengths are multiples of this
constexpr int kBT = 16;             // tokens per KV block
constexpr int kCounters = 64;

struct Unit { int b, t0, t1, slot; };      // slot: index of this (sequence, chunk) among all; -1 when the sequence has one chunk

struct PlanView {                    // carved out of the scratch buffer
    int* counters;                   // [kCounters] work counters, one per launch index
    int* n_entries;                  // [1]
    int* first;                      // [B] first entry of the sequence
    int* nc;                         // [B] number of chunks of the sequence
    Unit* entries;                   // [B * max_chunks]
    float* part_o;                   // [entries * Hkv][rows][dh]
    float* part_ml;                  // [entries * Hkv][rows][2]
};

inline int rows_alloc_for(int rows) { return rows <= 16 ? 16 : rows <= 32 ? 32 : rows <= 64 ? 64 : 128; }
inline int max_chunks_for(int max_kv_len) { return (max_kv_len + kTileTok + kChunk - 1) / kChunk + 1; }

// Bytes of scratch a plan with max_chunks chunks per sequence needs (the layout of carve_plan).
inline size_t plan_scratch_bytes(int B, int Hkv, int rows_alloc, int dh, int max_chunks)
{
    const size_t entries = (size_t)B * max_chunks;
    return align_up((size_t)kCounters * 4 + 4, 256) + 2 * align_up((size_t)B * 4, 256) + align_up(entries * sizeof(Unit), 256) +
           align_up(entries * Hkv * rows_alloc * dh * 4, 256) + align_up(entries * Hkv * rows_alloc * 8, 256);
}

inline PlanView carve_plan(void* scratch, int B, int Hkv, int rows_alloc, int dh, int max_chunks)
{
    const size_t entries = (size_t)B * max_chunks;
    char* p = static_cast<char*>(scratch);
    PlanView pv;
    pv.counters = reinterpret_cast<int*>(p);
    pv.n_entries = pv.counters + kCounters;
    p += align_up((size_t)kCounters * 4 + 4, 256);
    pv.first = reinterpret_cast<int*>(p); p += align_up((size_t)B * 4, 256);
    pv.nc = reinterpret_cast<int*>(p); p += align_up((size_t)B * 4, 256);
    pv.entries = reinterpret_cast<Unit*>(p); p += align_up(entries * sizeof(Unit), 256);
    pv.part_o = reinterpret_cast<float*>(p); p += align_up(entries * Hkv * rows_alloc * dh * 4, 256);
    pv.part_ml = reinterpret_cast<float*>(p);
    return pv;
}

// One CTA: picks the chunk length (kChunk, or finer when the batch is thin: n_ctas = CTAs of the attention launch), splits every
// sequence into equal chunks and writes the unit list (at most B * max_chunks units); resets the work counters.
spec_status launch_attn_plan(int B, int R, const int32_t* pos, int Hkv, int n_ctas, int max_chunks, const PlanView& pv, cudaStream_t st);
// Log-sum-exp merge of the chunks of multi-chunk sequences (head_dim 128); zeros for sequences without visible positions.
spec_status launch_attn_merge128(int B, int rows_alloc, int Hkv, int R, int group, void* out, int out_row_stride,
                                 const PlanView& pv, cudaStream_t st);

bool attention_fp8_supported(const AttnArgs& a);
spec_status launch_attention_fp8(const AttnArgs& a, cudaStream_t st);
bool attention_tc_supported(const AttnArgs& a);
spec_status launch_attention_tc(const AttnArgs& a, cudaStream_t st);

}  // namespace attn
}  // namespace spec
