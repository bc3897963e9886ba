// Shared host/device helpers of the AirCache sm_100a library: error plumbing, the workspace
// carve-up, argument checks and a few device intrinsics.  Nothing in here is used by the CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/aircache.h"

namespace aircache {

constexpr int kMaxWindow = 128;
constexpr int kMaxGroup = 16;         // query heads per KV head
constexpr int kMaxRegions = 1792;     // L * B (the decode kernel keeps the unit prefix of all regions in shared memory)
constexpr int kMaxDecodeCtas = 256;   // upper bound on the persistent decode grid (sizes the partial slots)
constexpr int kScoreKeyTile = 128;    // visual keys per CTA of the importance pass
constexpr float kLog2e = 1.4426950408889634f;
// status word left by aircache_compact when the device-side budgets / offsets / lists do not fit the buffers
// (waits that gave up leave small numbers that say which wait)
constexpr uint32_t kStatusInconsistent = 100;
constexpr int64_t kStatusBytes = 256 + (int64_t)kMaxRegions * 4;  // status word + tickets, at the start of the workspace
// Decode launches over few regions plan per warp, in registers (head-split launches: at least two KV heads per
// region, so at most kMaxDecodeCtas / 2 regions; by-region launches: up to 64 regions), and keep, per CTA, the
// plan of their last call: 16 words of outcome and the unit count of every region.
constexpr int kPlanRegionsPerLane = kMaxDecodeCtas / 2 / 32;
constexpr int kPlanMemoInts = 16 + 32 * kPlanRegionsPerLane;
constexpr int64_t kPlanMemoBytes = (int64_t)kMaxDecodeCtas * kPlanMemoInts * 4;
// what aircache_reset_status clears: status word, tickets and the kept plans, which follow them
constexpr int64_t kResetBytes = kStatusBytes + kPlanMemoBytes;

// ---------------------------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------------------------
void set_last_cuda_error(cudaError_t e);

#define AIRCACHE_CUDA_TRY(expr)                         \
    do {                                                \
        cudaError_t _e = (expr);                        \
        if (_e != cudaSuccess) {                        \
            ::aircache::set_last_cuda_error(_e);        \
            return AIRCACHE_ERR_CUDA;                   \
        }                                               \
    } while (0)

#define AIRCACHE_LAUNCH_CHECK()                         \
    do {                                                \
        cudaError_t _e = cudaGetLastError();            \
        if (_e != cudaSuccess) {                        \
            ::aircache::set_last_cuda_error(_e);        \
            return AIRCACHE_ERR_CUDA;                   \
        }                                               \
    } while (0)

// ---------------------------------------------------------------------------------------------
// shape helpers and the workspace carve-up (host arithmetic)
// ---------------------------------------------------------------------------------------------
int check_shape(const aircache_shape_t *s);
int check_full(const aircache_shape_t *s, const aircache_full_t *f);
int64_t kept_per_sequence(const aircache_shape_t *s, double ratio);

inline int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Cells per (layer, sequence): the units that get a budget, a kept set and a stretch of the ragged cache of their
// own - the KV heads in per-KV-head mode, else the region as a whole.  KV heads stored in one row of the cache.
inline int cells_of(const aircache_shape_t *s) { return s->per_kv_head ? s->n_kv_heads : 1; }
inline int row_heads_of(const aircache_shape_t *s) { return s->per_kv_head ? 1 : s->n_kv_heads; }
inline int64_t n_cells(const aircache_shape_t *s) { return (int64_t)s->n_layers * s->batch * cells_of(s); }

// Floats of one split-K partial slot of the decode kernel: [Hq, d] accumulator, Hq maxima, Hq sums, padded so
// that every slot starts on a 16-byte boundary.
__host__ __device__ inline int64_t partial_slot_floats(int n_q_heads, int head_dim) {
    return ((int64_t)n_q_heads * (head_dim + 2) + 3) / 4 * 4;
}

// Elite rows one KV group can have at most, padded to the MMA tile of 8 rows.
inline int score_row_cap(const aircache_shape_t *s) {
    int g = s->n_q_heads / s->n_kv_heads;
    return (int)align_up((int64_t)g * s->window, 16);
}

// Visual-key chunks of the statistics pass for a call that covers `groups` KV groups (a range of layers).  592
// CTAs run at a time on a B200 (four CTAs of 128 threads per SM); a CTA costs about as much fixed time (row
// table, query staging, reduction, ticket) as streaming 600 keys.  The chunk count minimises
// waves * (fixed + keys per chunk) under at least 256 keys per chunk.  A function of the shape and of the number
// of layers the call covers only, so results are reproducible.
inline int score_chunks(int n_visual, int64_t groups) {
    int64_t most = n_visual / 256;
    if (most > 64) most = 64;
    if (most < 1) most = 1;
    int best = 1;
    int64_t best_cost = -1;
    for (int c = 1; c <= most; ++c) {
        const int64_t waves = (groups * c + 591) / 592;
        const int64_t cost = waves * (600 + (n_visual + c - 1) / c);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = c; }
    }
    return best;
}

// One-pass scoring (both passes of Eq. 7 in one block, logits kept on chip between them): a block covers 1024
// keys of a KV group with up to 8 elite rows, 512 keys otherwise, and as few as 256 in calls over few groups;
// the workspace is laid out for 256.
constexpr int kOnePassMinKeys = 256;
constexpr int kOnePassMaxKeys = 1024;
inline int onepass_chunks(int n_visual) { return (n_visual + kOnePassMinKeys - 1) / kOnePassMinKeys; }

// The most (group, chunk) cells of statistics any call on this shape can have (it sizes the workspace).
inline int64_t score_chunk_cells(const aircache_shape_t *s) {
    int64_t most = (int64_t)s->n_layers * s->batch * s->n_kv_heads * onepass_chunks(s->n_visual);
    for (int layers = 1; layers <= s->n_layers; ++layers) {
        const int64_t groups = (int64_t)layers * s->batch * s->n_kv_heads;
        const int64_t cells = groups * score_chunks(s->n_visual, groups);
        if (cells > most) most = cells;
    }
    return most;
}

struct WsLayout {
    int64_t status;       // u32 status word (256 bytes reserved)
    int64_t tickets;      // i32  [kMaxRegions]        split-K tickets of the decode kernel, zero between calls
    int64_t plan_memo;    // i32  [kMaxDecodeCtas][kPlanMemoInts]  kept plans of the decode kernel, zero before first use
    int64_t row_count;    // i32  [L*B*Hkv]            elite rows of the KV group
    int64_t row_info;     // i32  [L*B*Hkv][cap]       (head within group << 8) | window slot
    int64_t row_coef;     // f32  [L*B*Hkv][cap]       1 / (|E_h| * Hq)
    int64_t row_text;     // f32x2[L*B*Hkv][cap]       (max, sum) of the visible elite text logits, log2 domain
    int64_t chunk_stats;  // f32x2[groups of the call][chunks][cap]  (max, sum) over one chunk of visual keys
    int64_t row_final;    // f32x2[L*B*Hkv][cap]       (max, weight / normaliser) after all chunks
    int64_t group_ticket; // u32  [L*B*Hkv]            chunks of the group done so far
    int64_t dispatch;     // u32                       blocks of the one-pass scoring kernel started so far
    int64_t imp_part;     // f32  [L*B*Hkv][Nv]        importance of one KV group before the sum over groups
    int64_t q_block;      // bf16 [L*B*Hkv][16][d]     the first 16 elite query rows of a group, gathered
    int64_t mom_strength; // f64  [cells]
    int64_t mom_skew;     // f64  [cells]
    int64_t kept;         // i32  [cells*Nv]           kept-token lists when the caller passes none
    int64_t partials;     // f32  [2*kMaxDecodeCtas][Hq*(d+2)]
    int64_t total;
};

WsLayout ws_layout(const aircache_shape_t *s);

template <typename T>
inline T *ws_ptr(void *ws, int64_t off) {
    return reinterpret_cast<T *>(reinterpret_cast<char *>(ws) + off);
}

// entry points implemented per translation unit
int launch_score(const aircache_shape_t *s, const aircache_full_t *f, const void *q_window, float alpha,
                 int layer_begin, int layer_count, float *scores, uint64_t *elite_mask, void *ws, cudaStream_t st);
int launch_budget(const aircache_shape_t *s, const float *scores, double ratio, int32_t mode, int32_t *budgets,
                  double *strength, double *skewness, aircache_ragged_t *layout, void *ws, cudaStream_t st);
int launch_compact(const aircache_shape_t *s, const aircache_full_t *f, const float *scores,
                   const int32_t *budgets, double ratio, aircache_ragged_t *out, int32_t *kept_idx, void *ws,
                   cudaStream_t st);
int launch_decode(const aircache_shape_t *s, const aircache_ragged_t *c, const void *q, const void *k_new,
                  const void *v_new, float *out, void *ws, cudaStream_t st);
int launch_decode_static(const aircache_shape_t *s, const aircache_ragged_t *c, const void *q, float *out,
                         cudaStream_t st);
int launch_selftest_timeout(void *ws, cudaStream_t st);
int launch_append(const aircache_shape_t *s, aircache_ragged_t *c, const void *k_new, const void *v_new,
                  int32_t appended, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float bf16lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16hi(uint32_t packed) { return __uint_as_float(packed & 0xffff0000u); }
__device__ __forceinline__ float bf16_to_f32(uint16_t h) { return __uint_as_float((uint32_t)h << 16); }

// D += A(16x16, bf16, row) * B(16x8, bf16, col), fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Merge two (max, sum-of-exp2) pairs of the same softmax row.
__device__ __forceinline__ void merge_stats(float &m, float &z, float m2, float z2) {
    float mn = fmaxf(m, m2);
    z = z * fast_exp2(m - mn) + z2 * fast_exp2(m2 - mn);
    m = mn;
}
#endif

}  // namespace aircache
