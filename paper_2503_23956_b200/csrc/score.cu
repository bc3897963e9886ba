// aircache_score: importance of every visual token seen from the elite observation window
// (Section 3.3, Eq. 4-8), all layers and sequences per launch.
//
// Kernels on one stream:
//   elite_kernel       one CTA per (layer, sequence, KV head): the W candidate keys and the last text query
//                      are staged in shared memory; Eq. 4 logits as fp64 dot products in element order (so
//                      the Eq. 5 decision does not depend on a summation order), the elite set of each
//                      query head, the table of elite rows (head, window slot) of the KV group, and each
//                      row's softmax statistics over the text keys it may see (elite, causal).
//                      It also leaves a gathered copy of the group's first 16 elite query rows.
//   onepass_kernel     Eq. 7 and Eq. 8 with one read of the visual keys: Q_tk K_v^T on tensor cores (keys on
//   + group_sum_kernel the M axis, elite rows on N), a chunk's logits kept in shared memory between the
//                      statistics and the probabilities; see the comment at the kernel.  The normal path.
//   stats_kernel       the same in two passes, for sequences too long for the one-pass kernel.  Pass one:
//   + importance_kernel running (max, sum of exp2) of every elite row over one chunk of visual keys; the CTA
//                      that finishes a KV group last (ticket) merges the chunks and the text statistics
//                      into one (max, weight / normaliser) pair per row.  Pass two recomputes the same
//                      tiles, turns logits into probabilities and sums the rows of all heads per key with
//                      weight 1 / (|E_h| Hq), KV heads in ascending order by one thread per key.
//   dense_*_kernel     alpha = 0 (every window query elite): both passes on tcgen05, see there.
//
// The mma.sync kernels read the keys straight from global memory into MMA fragments: every key byte is used
// once per CTA, so staging it in shared memory would only add a round trip.
#include <math.h>

#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace aircache {

namespace {

struct ScoreParams {
    const uint16_t *k;
    int64_t s_layer, s_batch, s_head, s_token;
    const uint16_t *qw;  // [L,B,W,Hq,d]
    float *scores;       // [L,B,Nv]
    uint64_t *elite_mask;
    int32_t *row_count;
    int32_t *row_info;
    float *row_coef;
    float2 *row_text;
    float2 *chunk_stats;
    float2 *row_final;   // (max, weight / normaliser) per elite row, written by the last stats CTA of a group
    uint32_t *group_ticket;
    uint32_t *dispatch;     // one-pass scoring: blocks started so far
    float *imp_part;        // one-pass scoring: [L*B*Hkv][Nv] importance of one KV group
    uint16_t *q_block;      // one-pass scoring: [L*B*Hkv][16][d] the first 16 elite query rows, gathered
    int op_chunks;      // numbers (blocks) per KV group in the one-pass grid
    int op_tile_cap;    // most 16-key tiles a warp of the one-pass kernel takes: 16, or fewer when the call is small
    int L, B, Hq, Hkv, G, d, Nv, Nt, W;
    int lb0, n_lb;   // the launch covers regions lb0 .. lb0 + n_lb - 1 (a range of layers)
    int per_head;    // scores are kept apart per KV group: [L,B,Hkv,Nv], Eq. 8 averaged over the group's heads only
    int cap, chunks, chunk_keys;
    float scale, sl2, ln_alpha;
    int keep_all;
    // one stats launch handles the KV groups with rows_lo < elite rows <= rows_hi
    int rows_lo, rows_hi;
    // dense (tcgen05) path: position of the token / head / sequence / layer coordinate in the key tensor map
    int pos_token, pos_head, pos_batch, pos_layer;
    uint32_t *status;
};

constexpr float kNegBig = -1.0e30f;

// ---------------------------------------------------------------------------------------------
// Eq. 4-5 and the elite-row table
// ---------------------------------------------------------------------------------------------
// QREG: the row's query is held in registers (64 of them at d = 128, two CTAs per SM) - worth it when a thread
// takes many rows against many text keys, i.e. when every candidate is elite (alpha = 0); otherwise the row is
// re-read from L1 per text key and six CTAs share an SM.
template <int D, bool QREG>
__global__ void __launch_bounds__(128, QREG ? 2 : 6) elite_kernel(ScoreParams p) {
    constexpr int KS = D + 8;   // padded row: 16-byte reads of consecutive rows fall into different banks
    extern __shared__ __align__(16) uint16_t s_dyn[];
    uint16_t *s_k = s_dyn;                 // [W][KS]   candidate keys
    uint16_t *s_ql = s_dyn + p.W * KS;     // [G][KS]   queries of the last text token
    __shared__ float s_logit[kMaxGroup * kMaxWindow];
    __shared__ uint64_t s_mask[kMaxGroup][2];   // candidate w is bit w % 64 of word w / 64
    __shared__ int s_first_row[kMaxGroup + 1];
    const int words = (p.W + 63) >> 6;

    const int grp = p.lb0 * p.Hkv + blockIdx.x;  // (l*B + b)*Hkv + g
    const int g = grp % p.Hkv;
    const int lb = grp / p.Hkv;
    const int l = lb / p.B, b = lb % p.B;
    const int N = p.Nv + p.Nt;
    const uint16_t *k_g = p.k + (int64_t)l * p.s_layer + (int64_t)b * p.s_batch + (int64_t)g * p.s_head;
    const uint16_t *k_cand = k_g + (int64_t)(N - p.W) * p.s_token;
    const uint16_t *q_lb = p.qw + (int64_t)lb * p.W * p.Hq * D;

    if (threadIdx.x == 0) {
        p.group_ticket[grp] = 0;   // the statistics pass counts its chunks here
        if (blockIdx.x == 0) *p.dispatch = 0;
    }
    for (int idx = threadIdx.x; idx < (p.W + p.G) * (D / 8); idx += blockDim.x) {
        const int row = idx / (D / 8), c = idx % (D / 8);
        const uint16_t *src = row < p.W ? k_cand + (int64_t)row * p.s_token
                                        : q_lb + ((int64_t)(p.W - 1) * p.Hq + g * p.G + (row - p.W)) * D;
        *reinterpret_cast<uint4 *>(s_dyn + row * KS + c * 8) = __ldg(reinterpret_cast<const uint4 *>(src) + c);
    }
    __syncthreads();

    // Eq. 4, last row only: logit of candidate w for head hl, fp64 dot product in element order.
    for (int idx = threadIdx.x; idx < p.G * p.W; idx += blockDim.x) {
        const int hl = idx / p.W, w = idx % p.W;
        const uint4 *q = reinterpret_cast<const uint4 *>(s_ql + hl * KS);
        const uint4 *kk = reinterpret_cast<const uint4 *>(s_k + w * KS);
        double acc = 0.0;
#pragma unroll 4
        for (int c = 0; c < D / 8; ++c) {
            const uint4 a = q[c], bb = kk[c];
            const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                // a product of two bf16 values is exact in fp64, so the fused form rounds exactly where the
                // separate multiply and add do
                acc = __fma_rn((double)bf16lo(av[e]), (double)bf16lo(bv[e]), acc);
                acc = __fma_rn((double)bf16hi(av[e]), (double)bf16hi(bv[e]), acc);
            }
        }
        s_logit[idx] = __fmul_rn((float)acc, p.scale);
    }
    __syncthreads();

    // Eq. 5: candidates within a factor alpha of the best one (compared in the log domain, fp32).
    if (threadIdx.x < p.G) {
        const int hl = threadIdx.x;
        const float *t = s_logit + hl * p.W;
        float tmax = -INFINITY;
        for (int w = 0; w < p.W; ++w) tmax = fmaxf(tmax, t[w]);
        uint64_t mask[2] = {0, 0};
        for (int w = 0; w < p.W; ++w) {
            const float diff = __fsub_rn(t[w], tmax);
            if (p.keep_all || diff >= p.ln_alpha) mask[w >> 6] |= (uint64_t)1 << (w & 63);
        }
        s_mask[hl][0] = mask[0];
        s_mask[hl][1] = mask[1];
        if (p.elite_mask)
            for (int j = 0; j < words; ++j) p.elite_mask[((int64_t)lb * p.Hq + g * p.G + hl) * words + j] = mask[j];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int r = 0;
        for (int hl = 0; hl < p.G; ++hl) {
            s_first_row[hl] = r;
            r += __popcll(s_mask[hl][0]) + __popcll(s_mask[hl][1]);
        }
        s_first_row[p.G] = r;
        p.row_count[grp] = r;
    }
    __syncthreads();

    // Row table: elite rows of head hl are consecutive, ascending window slot.
    int32_t *info = p.row_info + (int64_t)grp * p.cap;
    float *coef = p.row_coef + (int64_t)grp * p.cap;
    float2 *text = p.row_text + (int64_t)grp * p.cap;
    for (int idx = threadIdx.x; idx < p.G * p.W; idx += blockDim.x) {
        const int hl = idx / p.W, w = idx % p.W;
        const uint64_t m_lo = s_mask[hl][0], m_hi = s_mask[hl][1];
        auto elite = [&](int j) { return (((j < 64 ? m_lo : m_hi) >> (j & 63)) & 1) != 0; };
        if (!elite(w)) continue;
        // elite candidates in front of w
        const int before = w < 64 ? __popcll(m_lo & (((uint64_t)1 << w) - 1))
                                  : __popcll(m_lo) + __popcll(m_hi & (((uint64_t)1 << (w - 64)) - 1));
        const int r = s_first_row[hl] + before;
        info[r] = (hl << 8) | w;
        coef[r] = 1.0f / ((float)(__popcll(m_lo) + __popcll(m_hi)) * (float)(p.per_head ? p.G : p.Hq));
        // Eq. 6-7, text columns: row w sees the elite text keys w' <= w.  The keys come from shared memory, the
        // query row is re-read for every key (256 bytes that stay in L1) rather than held in 64 registers.
        const uint4 *qq = reinterpret_cast<const uint4 *>(q_lb + ((int64_t)w * p.Hq + g * p.G + hl) * D);
        if (r < 16) {   // the one-pass kernel stages the first 16 rows from this gathered copy
            uint4 *qb = reinterpret_cast<uint4 *>(p.q_block + ((int64_t)grp * 16 + r) * D);
#pragma unroll 4
            for (int c = 0; c < D / 8; ++c) qb[c] = __ldg(qq + c);
        }
        uint4 qr[QREG ? D / 8 : 1];
        if (QREG) {
#pragma unroll
            for (int c = 0; c < D / 8; ++c) qr[c] = __ldg(qq + c);
        }
        float m = kNegBig, z = 0.0f;
        for (int w2 = 0; w2 <= w; ++w2) {
            if (!elite(w2)) continue;
            const uint4 *kk = reinterpret_cast<const uint4 *>(s_k + w2 * KS);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll QREG ? D / 8 : 4
            for (int c = 0; c < D / 8; ++c) {
                const uint4 a = QREG ? qr[c] : __ldg(qq + c), bb = kk[c];
                a0 = fmaf(bf16lo(a.x), bf16lo(bb.x), a0); a1 = fmaf(bf16hi(a.x), bf16hi(bb.x), a1);
                a2 = fmaf(bf16lo(a.y), bf16lo(bb.y), a2); a3 = fmaf(bf16hi(a.y), bf16hi(bb.y), a3);
                a0 = fmaf(bf16lo(a.z), bf16lo(bb.z), a0); a1 = fmaf(bf16hi(a.z), bf16hi(bb.z), a1);
                a2 = fmaf(bf16lo(a.w), bf16lo(bb.w), a2); a3 = fmaf(bf16hi(a.w), bf16hi(bb.w), a3);
            }
            merge_stats(m, z, ((a0 + a1) + (a2 + a3)) * p.sl2, 1.0f);
        }
        text[r] = make_float2(m, z);
    }
}

// ---------------------------------------------------------------------------------------------
// Tensor-core tile shared by both passes.
//
// One warp computes S^T = K_tile (16 keys x d) * Q^T (d x 8*NT elite rows) with mma.m16n8k16.  The
// contraction index is permuted inside each block of 32 channels so that every thread feeds the MMA
// from one 16-byte load: thread t of a quad owns channels 8t..8t+7 of the block, both for the key rows
// (read straight from global memory) and for the query rows (shared memory).  A dot product does not
// depend on the order of its terms' indices as long as both operands use the same order.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void prefetch_l2(const void *ptr) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr) : "memory");
}

template <int D>
struct KeyFrag {
    uint4 lo[D / 32];  // key row gid
    uint4 hi[D / 32];  // key row gid + 8
};

template <int D>
__device__ __forceinline__ void load_keys(KeyFrag<D> &f, const uint16_t *row_lo, const uint16_t *row_hi, int t) {
#pragma unroll
    for (int kb = 0; kb < D / 32; ++kb) {
        f.lo[kb] = __ldg(reinterpret_cast<const uint4 *>(row_lo + kb * 32 + 8 * t));
        f.hi[kb] = __ldg(reinterpret_cast<const uint4 *>(row_hi + kb * 32 + 8 * t));
    }
}

template <int D>
__device__ __forceinline__ void tile_mma(float (&acc)[4], const KeyFrag<D> &f, const uint16_t *q_row, int t) {
    acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
#pragma unroll
    for (int kb = 0; kb < D / 32; ++kb) {
        const uint4 bq = *reinterpret_cast<const uint4 *>(q_row + kb * 32 + 8 * t);
        mma_bf16_16816(acc, f.lo[kb].x, f.hi[kb].x, f.lo[kb].y, f.hi[kb].y, bq.x, bq.y);
        mma_bf16_16816(acc, f.lo[kb].z, f.hi[kb].z, f.lo[kb].w, f.hi[kb].w, bq.z, bq.w);
    }
}

// The same tile with the contraction split over two accumulators (channels 0..d/2-1 and d/2..d-1) that are
// added at the end: half the dependent-MMA chain, for callers with few row tiles to interleave.
template <int D>
__device__ __forceinline__ void tile_mma_split(float (&acc)[4], const KeyFrag<D> &f, const uint16_t *q_row, int t) {
    constexpr int H = D / 64;
    float lo[4] = {0.f, 0.f, 0.f, 0.f}, hi[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int kb = 0; kb < H; ++kb) {
        const uint4 bq = *reinterpret_cast<const uint4 *>(q_row + kb * 32 + 8 * t);
        const uint4 bq2 = *reinterpret_cast<const uint4 *>(q_row + (kb + H) * 32 + 8 * t);
        mma_bf16_16816(lo, f.lo[kb].x, f.hi[kb].x, f.lo[kb].y, f.hi[kb].y, bq.x, bq.y);
        mma_bf16_16816(hi, f.lo[kb + H].x, f.hi[kb + H].x, f.lo[kb + H].y, f.hi[kb + H].y, bq2.x, bq2.y);
        mma_bf16_16816(lo, f.lo[kb].z, f.hi[kb].z, f.lo[kb].w, f.hi[kb].w, bq.z, bq.w);
        mma_bf16_16816(hi, f.lo[kb + H].z, f.hi[kb + H].z, f.lo[kb + H].w, f.hi[kb + H].w, bq2.z, bq2.w);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = lo[i] + hi[i];
}

// Copies up to 8*NT elite query rows (starting at row0) of one KV group into shared memory, zero padded.
template <int D>
__device__ __forceinline__ void stage_queries(uint16_t *s_q, const ScoreParams &p, int grp, int lb, int g,
                                              int row0, int n_rows_total, int rows_pad,
                                              const int32_t *staged_info = nullptr) {
    constexpr int QS = D + 32;
    // (head, slot) words of the rows: from the caller's copy in shared memory (rows row0.., row0 = 0) if it has one
    const int32_t *info = staged_info ? staged_info - row0 : p.row_info + (int64_t)grp * p.cap;
    const uint16_t *q_lb = p.qw + (int64_t)lb * p.W * p.Hq * D;
    for (int idx = threadIdx.x; idx < rows_pad * (D / 8); idx += blockDim.x) {
        const int r = idx / (D / 8), c = idx % (D / 8);
        uint4 v = make_uint4(0, 0, 0, 0);
        if (row0 + r < n_rows_total) {
            const int in = info[row0 + r];
            const int hl = in >> 8, w = in & 255;
            v = __ldg(reinterpret_cast<const uint4 *>(q_lb + ((int64_t)w * p.Hq + g * p.G + hl) * D) + c);
        }
        *reinterpret_cast<uint4 *>(s_q + r * QS + c * 8) = v;
    }
}

// Eq. 7, pass one.  grid = (chunks, L*B*Hkv), 128 threads.
template <int D, int NT>
__global__ void __launch_bounds__(128) stats_kernel(ScoreParams p) {
    constexpr int QS = D + 32;
    __shared__ __align__(16) uint16_t s_q[NT * 8 * QS];
    __shared__ float2 s_red[4][NT * 8];
    __shared__ int s_is_last;

    const int grp = p.lb0 * p.Hkv + blockIdx.y;
    const int g = grp % p.Hkv;
    const int lb = grp / p.Hkv;
    const int l = lb / p.B, b = lb % p.B;
    const int chunk = blockIdx.x;
    const int key0 = chunk * p.chunk_keys;
    const int key1 = min(p.Nv, key0 + p.chunk_keys);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, t = lane & 3;
    const uint16_t *k_g = p.k + (int64_t)l * p.s_layer + (int64_t)b * p.s_batch + (int64_t)g * p.s_head;
    const int n_rows = p.row_count[grp];
    if (n_rows <= p.rows_lo || n_rows > p.rows_hi) return;
    float2 *out = p.chunk_stats + ((int64_t)(grp - p.lb0 * p.Hkv) * p.chunks + chunk) * p.cap;

    for (int row0 = 0; row0 < n_rows; row0 += NT * 8) {
        const int nt_used = min(NT, (n_rows - row0 + 7) / 8);
        __syncthreads();
        stage_queries<D>(s_q, p, grp, lb, g, row0, n_rows, nt_used * 8);
        __syncthreads();

        float m[NT][2], z[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { m[nt][0] = m[nt][1] = kNegBig; z[nt][0] = z[nt][1] = 0.f; }

        // software pipeline: the next tile's keys are requested before this tile's MMAs
        auto fetch = [&](KeyFrag<D> &dst, int kt) {
            const int ka = kt + gid, kb = kt + gid + 8;
            load_keys<D>(dst, k_g + (int64_t)(ka < key1 ? ka : key1 - 1) * p.s_token,
                         k_g + (int64_t)(kb < key1 ? kb : key1 - 1) * p.s_token, t);
        };
        KeyFrag<D> f, f_next;
        if (key0 + warp * 16 < key1) fetch(f, key0 + warp * 16);
        for (int kt = key0 + warp * 16; kt < key1; kt += 64) {
            const int ka = kt + gid, kb = kt + gid + 8;
            const bool va = ka < key1, vb = kb < key1;
            if (kt + 64 < key1) fetch(f_next, kt + 64);
            // and the tile after that is asked into L2 (one 128-byte line per lane: 16 rows x D channels)
            if (kt + 128 < key1 && lane < 16 * (D * 2 / 128)) {
                const int kp = min(kt + 128 + lane / (D * 2 / 128), key1 - 1);
                prefetch_l2(k_g + (int64_t)kp * p.s_token + (lane % (D * 2 / 128)) * 64);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (nt < nt_used) {
                    float acc[4];
                    tile_mma<D>(acc, f, s_q + (nt * 8 + gid) * QS, t);
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const float xa = va ? acc[j] * p.sl2 : kNegBig;
                        const float xb = vb ? acc[j + 2] * p.sl2 : kNegBig;
                        const float mn = fmaxf(m[nt][j], fmaxf(xa, xb));
                        const float ea = va ? fast_exp2(xa - mn) : 0.f;
                        const float eb = vb ? fast_exp2(xb - mn) : 0.f;
                        z[nt][j] = z[nt][j] * fast_exp2(m[nt][j] - mn) + (ea + eb);
                        m[nt][j] = mn;
                    }
                }
            }
            if (kt + 64 < key1) f = f_next;
        }
        // combine the eight key lanes of a column, then the four warps, in a fixed order
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            if (nt < nt_used) {
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    float mm = m[nt][j], zz = z[nt][j];
#pragma unroll
                    for (int sh = 4; sh < 32; sh <<= 1) {
                        const float m2 = __shfl_xor_sync(0xffffffffu, mm, sh);
                        const float z2 = __shfl_xor_sync(0xffffffffu, zz, sh);
                        merge_stats(mm, zz, m2, z2);
                    }
                    if (gid == 0) s_red[warp][nt * 8 + 2 * t + j] = make_float2(mm, zz);
                }
            }
        }
        __syncthreads();
        for (int r = threadIdx.x; r < nt_used * 8; r += blockDim.x) {
            float2 a = s_red[0][r];
#pragma unroll
            for (int w2 = 1; w2 < 4; ++w2) merge_stats(a.x, a.y, s_red[w2][r].x, s_red[w2][r].y);
            if (row0 + r < n_rows) __stcg(out + row0 + r, a);
        }
    }

    // The CTA that finishes the group last merges text and chunk statistics, one warp per row: lanes take
    // chunks lane, lane + 32, ... in order, then a fixed xor tree.  (The ticket was zeroed by elite_kernel.)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        s_is_last = atomicAdd(p.group_ticket + grp, 1u) == (unsigned)p.chunks - 1;
        if (s_is_last) __threadfence();
    }
    __syncthreads();
    if (!s_is_last) return;
    for (int r = warp; r < n_rows; r += 4) {
        float mm = kNegBig, zz = 0.f;
        if (lane == 0) {
            const float2 tx = p.row_text[(int64_t)grp * p.cap + r];
            mm = tx.x; zz = tx.y;
        }
        for (int c = lane; c < p.chunks; c += 32) {
            const float2 cs = __ldcg(p.chunk_stats + ((int64_t)(grp - p.lb0 * p.Hkv) * p.chunks + c) * p.cap + r);
            merge_stats(mm, zz, cs.x, cs.y);
        }
#pragma unroll
        for (int sh = 1; sh < 32; sh <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, mm, sh);
            const float z2 = __shfl_xor_sync(0xffffffffu, zz, sh);
            merge_stats(mm, zz, m2, z2);
        }
        if (lane == 0) p.row_final[(int64_t)grp * p.cap + r] = make_float2(mm, p.row_coef[(int64_t)grp * p.cap + r] / zz);
    }
}

// Eq. 7 pass two and Eq. 8.  grid = (ceil(Nv / 128), L*B), 128 threads; each warp owns 32 keys.
template <int D, int NT>
__global__ void __launch_bounds__(128) importance_kernel(ScoreParams p) {
    constexpr int QS = D + 32;
    __shared__ __align__(16) uint16_t s_q[NT * 8 * QS];
    __shared__ float2 s_stat[NT * 8];  // (row max, weight / normaliser)
    // the row tables of all KV heads of the sequence, fetched in one go at the start: per head the first NT * 8
    // rows' (head, slot) words and statistics, so that the loop over the heads waits for the query rows only
    constexpr int kMaxKv = 8;
    __shared__ int s_rows[kMaxKv];
    __shared__ int32_t s_info_all[kMaxKv][NT * 8];
    __shared__ float2 s_stat_all[kMaxKv][NT * 8];

    const int lb = p.lb0 + blockIdx.y;
    const int l = lb / p.B, b = lb % p.B;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, t = lane & 3;
    const int kbase = blockIdx.x * kScoreKeyTile + warp * 32;
    float imp[2][2] = {{0.f, 0.f}, {0.f, 0.f}};  // [m-tile][key gid / gid+8]

    for (int i = threadIdx.x; i < p.Hkv * NT * 8; i += blockDim.x) {
        const int g = i / (NT * 8), r = i % (NT * 8);
        const int64_t at = (int64_t)(lb * p.Hkv + g) * p.cap + r;
        const bool inside = r < p.cap;
        s_info_all[g][r] = inside ? p.row_info[at] : 0;
        s_stat_all[g][r] = inside ? p.row_final[at] : make_float2(0.f, 0.f);
        if (r == 0) s_rows[g] = p.row_count[lb * p.Hkv + g];
    }
    __syncthreads();

    for (int g = 0; g < p.Hkv; ++g) {
        const int grp = lb * p.Hkv + g;
        const uint16_t *k_g = p.k + (int64_t)l * p.s_layer + (int64_t)b * p.s_batch + (int64_t)g * p.s_head;
        const int n_rows = s_rows[g];
        KeyFrag<D> f[2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int ka = kbase + mt * 16 + gid, kb = ka + 8;
            load_keys<D>(f[mt], k_g + (int64_t)(ka < p.Nv ? ka : p.Nv - 1) * p.s_token,
                         k_g + (int64_t)(kb < p.Nv ? kb : p.Nv - 1) * p.s_token, t);
        }
        for (int row0 = 0; row0 < n_rows; row0 += NT * 8) {
            const int nt_used = min(NT, (n_rows - row0 + 7) / 8);
            __syncthreads();
            stage_queries<D>(s_q, p, grp, lb, g, row0, n_rows, nt_used * 8, row0 == 0 ? s_info_all[g] : nullptr);
            for (int r = threadIdx.x; r < nt_used * 8; r += blockDim.x)
                s_stat[r] = row0 + r >= n_rows ? make_float2(0.f, 0.f)
                            : (row0 == 0 ? s_stat_all[g][r] : p.row_final[(int64_t)grp * p.cap + row0 + r]);
            __syncthreads();
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (nt < nt_used) {
                    const float2 s0 = s_stat[nt * 8 + 2 * t], s1 = s_stat[nt * 8 + 2 * t + 1];
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        float acc[4];
                        tile_mma<D>(acc, f[mt], s_q + (nt * 8 + gid) * QS, t);
                        imp[mt][0] += fast_exp2(acc[0] * p.sl2 - s0.x) * s0.y + fast_exp2(acc[1] * p.sl2 - s1.x) * s1.y;
                        imp[mt][1] += fast_exp2(acc[2] * p.sl2 - s0.x) * s0.y + fast_exp2(acc[3] * p.sl2 - s1.x) * s1.y;
                    }
                }
            }
        }
        if (p.per_head || g == p.Hkv - 1) {
            // the key's score is complete: of this KV group alone, or summed over all of them
            float *out = p.scores + (p.per_head ? (int64_t)grp : (int64_t)lb) * p.Nv;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    float v = imp[mt][j];
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    const int key = kbase + mt * 16 + gid + 8 * j;
                    if (t == 0 && key < p.Nv) out[key] = v;
                    imp[mt][j] = 0.f;
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Eq. 7 and Eq. 8 in ONE pass over the keys.
//
// The two kernels above read the keys from HBM twice when the cache is larger than L2.  Here a block owns a
// chunk of one KV group's keys and keeps the chunk's logits (fp32 MMA accumulators, up to 16 rows) in shared
// memory: pass one gives the chunk's (max, sum) per row; when all chunks of the group have published theirs,
// every block of the group merges them (same fixed order in every block: equal bits), turns its stored logits
// into probabilities and sums them per key - no second read of the keys, no second contraction.  A chunk is
// 1024 keys for a group of up to 8 elite rows and 512 keys beyond, so the stored logits fill the same 32 KB
// (five blocks per SM); the per-key sums of pass two go into slots of that buffer the warp has already read.
// Rows beyond 16 (wide windows, small alpha) are recomputed from the keys, which are still in L1/L2.
//
// Waiting inside a grid is safe here because a block draws its number from a counter when it STARTS: all
// lower numbers belong to blocks that are running or done.  Numbers are group-major, a group spans
// op_chunks numbers, and the host only takes this path when op_chunks is at most half of the blocks the GPU
// holds at once - so the blocks a waiting block depends on are always resident or next in line, and blocks
// of lower groups, which wait for nothing that has not started, always finish.  The wait is bounded all the same.
//
// The sum over the KV groups of a (layer, sequence) is a second, small kernel (fixed order g = 0, 1, ...).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *ptr) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

__device__ __forceinline__ int onepass_tiles(int n_rows, int cap) {   // 16-key tiles per warp
    return min(n_rows <= 8 ? 16 : 8, cap);
}

template <int D>
__global__ void __launch_bounds__(128, 5) onepass_kernel(ScoreParams p) {
    constexpr int NT = 2, QS = D + 32;
    extern __shared__ __align__(16) uint16_t s_dyn[];
    float4 *s_S = reinterpret_cast<float4 *>(s_dyn);        // [tile of the warp][row tile][thread]: 2048 x 16 B
    __shared__ __align__(16) uint16_t s_q[NT * 8 * QS];
    __shared__ float2 s_red[4][NT * 8];
    __shared__ float2 s_stat[NT * 8];
    __shared__ int s_flag;

    if (threadIdx.x == 0) s_flag = (int)atomicAdd(p.dispatch, 1u);
    __syncthreads();
    const int vid = s_flag;
    __syncthreads();

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 2, t = lane & 3;
    const int gi = vid / p.op_chunks, c = vid % p.op_chunks;
    if (gi >= p.n_lb * p.Hkv) return;
    const int grp = p.lb0 * p.Hkv + gi;
    const int g = grp % p.Hkv, lb = grp / p.Hkv, l = lb / p.B, b = lb % p.B;
    const int n_rows = p.row_count[grp];
    const int tpw = onepass_tiles(n_rows, p.op_tile_cap);
    const int KB = 64 * tpw;
    const int chunks_g = (p.Nv + KB - 1) / KB;
    if (c >= chunks_g) return;
    const int nt0 = min(NT, (n_rows + 7) >> 3);
    const uint16_t *k_g = p.k + (int64_t)l * p.s_layer + (int64_t)b * p.s_batch + (int64_t)g * p.s_head;
    const int key0 = c * KB, key1 = min(p.Nv, key0 + KB);
    const int wk0 = key0 + warp * tpw * 16, wk1 = min(key1, wk0 + tpw * 16);
    // the warp's first two tiles are asked into L2 now (HBM latency runs beside the query staging), every later
    // tile two tiles before its turn.  (Asking for the whole chunk at once measured 15 % slower: the burst
    // queues in front of the loads that are waited for.)
    constexpr int kAhead = 2 * 16;
    for (int i = lane; i < min(wk1 - wk0, kAhead) * (D * 2 / 128); i += 32)
        prefetch_l2(k_g + (int64_t)(wk0 + i / (D * 2 / 128)) * p.s_token + (i % (D * 2 / 128)) * 64);

    auto fetch = [&](KeyFrag<D> &dst, int kt) {
        const int ka = kt + gid, kb = kt + gid + 8;
        load_keys<D>(dst, k_g + (int64_t)(ka < wk1 ? ka : wk1 - 1) * p.s_token,
                     k_g + (int64_t)(kb < wk1 ? kb : wk1 - 1) * p.s_token, t);
    };
    // (max, weight / normaliser) of rows row0 .. row0 + n - 1 into s_stat: one thread per row merges the text
    // statistics and then the chunks' statistics in chunk order (all loads of a row are independent, one round
    // trip), the same order in every block
    auto merge_rows = [&](int row0, int n) {
        if (tid < n) {
            const int row = row0 + tid;
            float2 fin = make_float2(0.f, 0.f);
            if (row < n_rows) {
                const float2 *cs = p.chunk_stats + (int64_t)gi * p.op_chunks * p.cap + row;
                const float2 tx = p.row_text[(int64_t)grp * p.cap + row];
                const float coef = p.row_coef[(int64_t)grp * p.cap + row];
                float mm = tx.x, zz = tx.y;
                int cc = 0;
                for (; cc + 4 <= chunks_g; cc += 4) {
                    const float2 c0 = __ldcg(cs + (int64_t)cc * p.cap), c1 = __ldcg(cs + (int64_t)(cc + 1) * p.cap);
                    const float2 c2 = __ldcg(cs + (int64_t)(cc + 2) * p.cap), c3 = __ldcg(cs + (int64_t)(cc + 3) * p.cap);
                    merge_stats(mm, zz, c0.x, c0.y); merge_stats(mm, zz, c1.x, c1.y);
                    merge_stats(mm, zz, c2.x, c2.y); merge_stats(mm, zz, c3.x, c3.y);
                }
                for (; cc < chunks_g; ++cc) {
                    const float2 c0 = __ldcg(cs + (int64_t)cc * p.cap);
                    merge_stats(mm, zz, c0.x, c0.y);
                }
                fin = make_float2(mm, coef / zz);
            }
            s_stat[tid] = fin;
        }
    };

    // ---- pass one: statistics of the chunk, logits of the first 16 rows kept ----
    float2 *out = p.chunk_stats + ((int64_t)gi * p.op_chunks + c) * p.cap;
    for (int row0 = 0; row0 < n_rows; row0 += NT * 8) {
        const int nt_used = min(NT, (n_rows - row0 + 7) / 8);
        KeyFrag<D> f, f_next;
        if (wk0 < wk1) fetch(f, wk0);
        __syncthreads();
        if (row0 == 0) {
            const uint4 *qb = reinterpret_cast<const uint4 *>(p.q_block + (int64_t)grp * 16 * D);
            for (int idx = tid; idx < nt_used * 8 * (D / 8); idx += blockDim.x) {
                const int r = idx / (D / 8), cc = idx % (D / 8);
                *reinterpret_cast<uint4 *>(s_q + r * QS + cc * 8) = r < n_rows ? __ldg(qb + idx) : make_uint4(0, 0, 0, 0);
            }
        } else {
            stage_queries<D>(s_q, p, grp, lb, g, row0, n_rows, nt_used * 8);
        }
        __syncthreads();
        float m[NT][2], z[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { m[nt][0] = m[nt][1] = kNegBig; z[nt][0] = z[nt][1] = 0.f; }
        int slot = tid;   // (tile * nt_used + nt) * 128 + tid
        for (int kt = wk0; kt < wk1; kt += 16) {
            const int ka = kt + gid, kb = kt + gid + 8;
            const bool va = ka < wk1, vb = kb < wk1;
            if (kt + 16 < wk1) fetch(f_next, kt + 16);
            if (kt + kAhead < wk1 && lane < 16 * (D * 2 / 128)) {   // one 128-byte line per lane: 16 rows x d channels
                const int kp = min(kt + kAhead + lane / (D * 2 / 128), wk1 - 1);
                prefetch_l2(k_g + (int64_t)kp * p.s_token + (lane % (D * 2 / 128)) * 64);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (nt < nt_used) {
                    float acc[4];
                    tile_mma_split<D>(acc, f, s_q + (nt * 8 + gid) * QS, t);
                    if (row0 == 0) { s_S[slot] = make_float4(acc[0], acc[1], acc[2], acc[3]); slot += 128; }
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const float xa = va ? acc[j] * p.sl2 : kNegBig;
                        const float xb = vb ? acc[j + 2] * p.sl2 : kNegBig;
                        const float mn = fmaxf(m[nt][j], fmaxf(xa, xb));
                        const float ea = va ? fast_exp2(xa - mn) : 0.f;
                        const float eb = vb ? fast_exp2(xb - mn) : 0.f;
                        z[nt][j] = z[nt][j] * fast_exp2(m[nt][j] - mn) + (ea + eb);
                        m[nt][j] = mn;
                    }
                }
            }
            if (kt + 16 < wk1) f = f_next;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            if (nt < nt_used) {
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    float mm = m[nt][j], zz = z[nt][j];
#pragma unroll
                    for (int sh = 4; sh < 32; sh <<= 1) {
                        const float m2 = __shfl_xor_sync(0xffffffffu, mm, sh);
                        const float z2 = __shfl_xor_sync(0xffffffffu, zz, sh);
                        merge_stats(mm, zz, m2, z2);
                    }
                    if (gid == 0) s_red[warp][nt * 8 + 2 * t + j] = make_float2(mm, zz);
                }
            }
        }
        __syncthreads();
        for (int r = tid; r < nt_used * 8; r += blockDim.x) {
            float2 a = s_red[0][r];
#pragma unroll
            for (int w2 = 1; w2 < 4; ++w2) merge_stats(a.x, a.y, s_red[w2][r].x, s_red[w2][r].y);
            if (row0 + r < n_rows) __stcg(out + row0 + r, a);
        }
    }

    // ---- publish the chunk, wait until every chunk of the group is published ----
    __syncthreads();
    if (tid == 0) {
        __threadfence();   // the block's statistics (ordered before this by the barrier) before the ticket
        int ok = atomicAdd(p.group_ticket + grp, 1u) + 1u >= (unsigned)chunks_g;
        for (uint32_t i = 0; !ok && i < kSpinLimit; ++i) {
            __nanosleep(i < 64 ? 32 : 1000);
            ok = ld_acquire_u32(p.group_ticket + grp) >= (unsigned)chunks_g;
        }
        if (!ok) atomicExch(p.status, 8u);
        __threadfence();
        s_flag = ok;
    }
    __syncthreads();
    if (!s_flag) return;

    // ---- pass two: probabilities from the kept logits, summed over the rows of the group ----
    merge_rows(0, nt0 * 8);
    __syncthreads();
    {
        int slot = tid;
        float *imp_w = reinterpret_cast<float *>(s_S + warp * 32);   // + tile * nt0 * 512 floats: the warp's own slots of the tile
#pragma unroll 4
        for (int kt = wk0; kt < wk1; kt += 16, imp_w += nt0 * 512) {
            float a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (nt < nt0) {
                    const float4 v = s_S[slot]; slot += 128;
                    const float2 s0 = s_stat[nt * 8 + 2 * t], s1 = s_stat[nt * 8 + 2 * t + 1];
                    a0 += fast_exp2(v.x * p.sl2 - s0.x) * s0.y + fast_exp2(v.y * p.sl2 - s1.x) * s1.y;
                    a1 += fast_exp2(v.z * p.sl2 - s0.x) * s0.y + fast_exp2(v.w * p.sl2 - s1.x) * s1.y;
                }
            }
            a0 += __shfl_xor_sync(0xffffffffu, a0, 1); a0 += __shfl_xor_sync(0xffffffffu, a0, 2);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            if (t == 0) { imp_w[gid] = a0; imp_w[gid + 8] = a1; }
        }
    }
    // rows beyond 16: logits recomputed from the keys
    for (int row0 = NT * 8; row0 < n_rows; row0 += NT * 8) {
        const int nt_used = min(NT, (n_rows - row0 + 7) / 8);
        __syncthreads();
        stage_queries<D>(s_q, p, grp, lb, g, row0, n_rows, nt_used * 8);
        merge_rows(row0, nt_used * 8);
        __syncthreads();
        KeyFrag<D> f;
        float *imp_w = reinterpret_cast<float *>(s_S + warp * 32);
        for (int kt = wk0; kt < wk1; kt += 16, imp_w += nt0 * 512) {
            fetch(f, kt);
            float a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (nt < nt_used) {
                    float acc[4];
                    tile_mma_split<D>(acc, f, s_q + (nt * 8 + gid) * QS, t);
                    const float2 s0 = s_stat[nt * 8 + 2 * t], s1 = s_stat[nt * 8 + 2 * t + 1];
                    a0 += fast_exp2(acc[0] * p.sl2 - s0.x) * s0.y + fast_exp2(acc[1] * p.sl2 - s1.x) * s1.y;
                    a1 += fast_exp2(acc[2] * p.sl2 - s0.x) * s0.y + fast_exp2(acc[3] * p.sl2 - s1.x) * s1.y;
                }
            }
            a0 += __shfl_xor_sync(0xffffffffu, a0, 1); a0 += __shfl_xor_sync(0xffffffffu, a0, 2);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            if (t == 0) { imp_w[gid] += a0; imp_w[gid + 8] += a1; }
        }
    }
    __syncthreads();

    // ---- Eq. 8: the group's own score, or its part of the sum over the KV groups ----
    const int nkeys = key1 - key0;
    float *dst = (p.per_head ? p.scores : p.imp_part) + (int64_t)grp * p.Nv + key0;
    for (int i = tid; i < nkeys; i += blockDim.x) {
        const int w = i / (tpw * 16), rem = i % (tpw * 16);
        dst[i] = reinterpret_cast<const float *>(s_S + w * 32)[(rem >> 4) * nt0 * 512 + (rem & 15)];
    }
}

// Eq. 8, the mean over all query heads: the KV groups' parts added in the order g = 0, 1, ...
__global__ void __launch_bounds__(256) group_sum_kernel(ScoreParams p) {
    const int lb = p.lb0 + blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.Nv) return;
    const float *src = p.imp_part + (int64_t)lb * p.Hkv * p.Nv + i;
    float v = 0.f;
    for (int g = 0; g < p.Hkv; ++g) v += __ldcg(src + (int64_t)g * p.Nv);
    p.scores[(int64_t)lb * p.Nv + i] = v;
}

// Blocks of the one-pass kernel the device holds at once (0 if the kernel cannot run); asked once per device,
// under a lock.
template <int D>
int onepass_resident_blocks() {
    static std::mutex lock;
    static int cached[64];
    static bool have[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    std::lock_guard<std::mutex> guard(lock);
    if (!have[dev]) {
        int per_sm = 0, sms = 0;
        if (cudaFuncSetAttribute(onepass_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, onepass_kernel<D>, 128, 32768) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return 0;
        cached[dev] = per_sm * sms;
        have[dev] = true;
    }
    return cached[dev];
}

template <int D>
int launch_onepass(const ScoreParams &p, cudaStream_t st) {
    const int64_t blocks = (int64_t)p.n_lb * p.Hkv * p.op_chunks;
    onepass_kernel<D><<<(unsigned)blocks, 128, 32768, st>>>(p);
    AIRCACHE_LAUNCH_CHECK();
    if (!p.per_head) {
        group_sum_kernel<<<dim3((p.Nv + 255) / 256, (unsigned)p.n_lb), 256, 0, st>>>(p);
        AIRCACHE_LAUNCH_CHECK();
    }
    return AIRCACHE_OK;
}

// ---------------------------------------------------------------------------------------------
// Dense window (alpha = 0: every one of the G*W window queries is an elite row, Eq. 7 is a dense
// [G*W x N_v] contraction per KV head).  Same two passes on the 5th-generation tensor cores:
//   * key tiles of 128 tokens come in by TMA (5-D tensor map over the caller's strided cache, 128-byte
//     swizzle), query blocks of 128 rows are written into the same K-major swizzled layout by the threads;
//   * one thread issues tcgen05.mma (M = 128, N = 128, K = 16 per instruction), the accumulator lives in
//     tensor memory and is read back with tcgen05.ld, one accumulator row per thread;
//   * pass one puts the query rows on M, so a thread owns one softmax row and keeps its running (max, sum)
//     in two registers; pass two swaps the operands (the same two shared-memory tiles), so a thread owns one
//     key and sums the weighted probabilities of all rows - neither pass needs a cross-lane reduction.
// Every mbarrier wait is bounded (status word + CTA-wide abort flag, as in the decode kernel).
// ---------------------------------------------------------------------------------------------
template <int D>
struct DenseCfg {
    static constexpr int KSUB = D / 64;             // 64-channel sub-tiles: rows of 128 bytes
    static constexpr int SUB_BYTES = 128 * 128;     // 128 rows
    static constexpr int TILE_BYTES = KSUB * SUB_BYTES;
    static constexpr int NST = 2;                   // key tiles in flight (two CTAs share an SM)
    static constexpr int SMEM_STATS = 1024 + (NST + 1) * TILE_BYTES + 256;
    static constexpr int SMEM_IMP = 1024 + (NST + 1) * TILE_BYTES + 128 * 8 + 256;
};

// 128 query rows (row0 .. row0+127 of the group's table, zero beyond) into the swizzled K-major layout.
// 128 threads: thread t copies 16-byte chunk t % (D/8) of rows t / (D/8) + k * (1024 / D); all table entries are
// fetched first, then all query chunks, so the copy costs two memory round trips.
template <int D>
__device__ __forceinline__ void stage_queries_sw128(uint8_t *s_q, const ScoreParams &p, int grp, int lb, int g,
                                                    int row0, int n_rows) {
    constexpr int SUB = DenseCfg<D>::SUB_BYTES;
    constexpr int CPR = D / 8;            // 16-byte chunks per row
    constexpr int RPI = 128 / CPR;        // rows covered by the CTA per step
    constexpr int STEPS = 128 / RPI;
    const int32_t *info = p.row_info + (int64_t)grp * p.cap;
    const uint16_t *q_lb = p.qw + (int64_t)lb * p.W * p.Hq * D;
    const int c16 = threadIdx.x % CPR, r0 = threadIdx.x / CPR;
    int in[STEPS];
#pragma unroll
    for (int k = 0; k < STEPS; ++k) {
        const int r = row0 + r0 + k * RPI;
        in[k] = r < n_rows ? __ldg(info + r) : -1;
    }
    uint4 v[STEPS];
#pragma unroll
    for (int k = 0; k < STEPS; ++k) {
        v[k] = make_uint4(0, 0, 0, 0);
        if (in[k] >= 0) {
            const int hl = in[k] >> 8, w = in[k] & 255;
            v[k] = __ldg(reinterpret_cast<const uint4 *>(q_lb + ((int64_t)w * p.Hq + g * p.G + hl) * D) + c16);
        }
    }
    const int sub = c16 >> 3, cc = c16 & 7;
#pragma unroll
    for (int k = 0; k < STEPS; ++k) {
        const int r = r0 + k * RPI;
        *reinterpret_cast<uint4 *>(s_q + sub * SUB + r * 128 + ((cc ^ (r & 7)) << 4)) = v[k];
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes, read by the tensor core
}

// acc[128 x 128] = A[128 x D] * B[128 x D]^T, both tiles K-major swizzled at a_base / b_base.
template <int D>
__device__ __forceinline__ void issue_tile_mma(uint32_t tmem_d, uint32_t a_base, uint32_t b_base) {
    constexpr int SUB = DenseCfg<D>::SUB_BYTES;
    const uint32_t idesc = umma_idesc_bf16(128, 128);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (kk >> 2) * SUB + (kk & 3) * 32;
        umma_bf16(tmem_d, umma_desc_sw128(a_base + off), umma_desc_sw128(b_base + off), idesc, kk > 0 ? 1u : 0u);
    }
}

template <int D>
__device__ __forceinline__ void load_key_tile(uint32_t dst, const CUtensorMap *tm, const ScoreParams &p, int key,
                                              int g, int b, int l, uint32_t bar) {
    int c[5] = {0, 0, 0, 0, 0};
    c[p.pos_token] = key; c[p.pos_head] = g; c[p.pos_batch] = b; c[p.pos_layer] = l;
    mbar_expect_tx(bar, DenseCfg<D>::TILE_BYTES);
#pragma unroll
    for (int sub = 0; sub < DenseCfg<D>::KSUB; ++sub)
        tma_load_5d(dst + sub * DenseCfg<D>::SUB_BYTES, tm, sub * 64, c[1], c[2], c[3], c[4], bar);
}

// Both dense kernels are warp-specialised: two sets of four epilogue warps (warps 0-3 and 4-7; a thread owns one
// accumulator row, a tensor-memory lane) run the exponent arithmetic, one thread of warp 8 drives the copies
// and the tensor core.  Key tiles cycle through NST shared-memory stages (full: TMA landed; empty: the MMAs
// that read the stage have completed, by tcgen05.commit), accumulators through two halves of 256 tensor-memory
// columns (acc_full by tcgen05.commit, acc_empty by one arrival per warp of the set that read it).  Each set
// takes the tiles of one accumulator, so two tiles' logits are read back and exponentiated at a time while the
// MMAs of the next run.  Parities follow from running tile counts.  Every wait is bounded.
constexpr int kDenseThreads = 288;
constexpr int kDenseDriverWarp = 8;

template <int D>
struct DensePipe {
    using C = DenseCfg<D>;
    uint32_t full[C::NST], empty[C::NST], acc_full[2], acc_empty[2];   // shared-memory addresses of the mbarriers
    __device__ void init(uint64_t *s_bar) {
        for (int i = 0; i < C::NST; ++i) { full[i] = smem_u32(&s_bar[i]); empty[i] = smem_u32(&s_bar[C::NST + i]); }
        for (int a = 0; a < 2; ++a) { acc_full[a] = smem_u32(&s_bar[2 * C::NST + a]); acc_empty[a] = smem_u32(&s_bar[2 * C::NST + 2 + a]); }
    }
    __device__ void init_barriers() const {
        for (int i = 0; i < C::NST; ++i) { mbar_init(full[i], 1); mbar_init(empty[i], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(acc_full[a], 1); mbar_init(acc_empty[a], 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
};

// The driver thread's part for n_tiles key tiles starting at key0: `base` tiles went through the pipe before.
// a_is_query: the query block is the MMA's A operand (rows on M, pass one), else the key tile is (keys on M).
// The first key tiles of a block of work, issued by the driver thread while the other warps stage the query
// block: returns how many loads are under way (the stages are free: the previous block's MMAs have completed).
template <int D>
__device__ __forceinline__ int dense_first_loads(const DensePipe<D> &pp, const CUtensorMap *tm, const ScoreParams &p,
                                                 uint8_t *s_k, uint32_t base, int n_tiles, int key0, int g, int b, int l,
                                                 volatile int *s_abort, uint32_t code) {
    using C = DenseCfg<D>;
    int loaded = 0;
    while (loaded < n_tiles && loaded < C::NST) {
        const uint32_t il = base + loaded, ls = il % C::NST;
        if (!mbar_wait(pp.empty[ls], ((il / C::NST) & 1) ^ 1, s_abort, p.status, code)) break;
        load_key_tile<D>(smem_u32(s_k + ls * C::TILE_BYTES), tm, p, key0 + loaded * 128, g, b, l, pp.full[ls]);
        ++loaded;
    }
    return loaded;
}

template <int D, bool A_IS_QUERY>
__device__ __forceinline__ bool dense_drive(const DensePipe<D> &pp, const CUtensorMap *tm, const ScoreParams &p,
                                            uint32_t tmem, uint8_t *s_k, uint8_t *s_q, uint32_t base, int n_tiles,
                                            int loaded, int key0, int g, int b, int l, volatile int *s_abort,
                                            uint32_t code) {
    using C = DenseCfg<D>;
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
        while (ok && loaded < n_tiles && loaded < t + C::NST) {
            const uint32_t il = base + loaded, ls = il % C::NST;
            ok = mbar_wait(pp.empty[ls], ((il / C::NST) & 1) ^ 1, s_abort, p.status, code);
            if (ok) {
                load_key_tile<D>(smem_u32(s_k + ls * C::TILE_BYTES), tm, p, key0 + loaded * 128, g, b, l, pp.full[ls]);
                ++loaded;
            }
        }
        if (!ok) break;
        const uint32_t it = base + t, st = it % C::NST, a = it & 1;
        ok = mbar_wait(pp.full[st], (it / C::NST) & 1, s_abort, p.status, code) &&
             mbar_wait(pp.acc_empty[a], ((it >> 1) & 1) ^ 1, s_abort, p.status, code + 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t k_tile = smem_u32(s_k + st * C::TILE_BYTES), q_blk = smem_u32(s_q);
        issue_tile_mma<D>(tmem + a * 128, A_IS_QUERY ? q_blk : k_tile, A_IS_QUERY ? k_tile : q_blk);
        umma_commit(pp.empty[st]);      // the stage may be refilled
        umma_commit(pp.acc_full[a]);    // the accumulator may be read
    }
    return ok;
}

// Pass one, dense.  grid = (chunks, L*B*Hkv), 160 threads.
template <int D>
__global__ void __launch_bounds__(kDenseThreads, 2) dense_stats_kernel(const __grid_constant__ CUtensorMap tm_k, ScoreParams p) {
    using C = DenseCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *s_k = smem;                             // NST key tiles
    uint8_t *s_q = smem + C::NST * C::TILE_BYTES;    // one query block
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + (C::NST + 1) * C::TILE_BYTES);
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort, s_is_last;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int set = warp >> 2, row = (warp & 3) * 32 + lane;   // epilogue set and accumulator row (warps 0-7)
    __shared__ float2 s_mz[128];                               // the second set's (max, sum) of every row
    const int grp = p.lb0 * p.Hkv + blockIdx.y;
    const int g = grp % p.Hkv, lb = grp / p.Hkv;
    const int l = lb / p.B, b = lb % p.B;
    const int chunk = blockIdx.x;
    const int key0 = chunk * p.chunk_keys, key1 = min(p.Nv, key0 + p.chunk_keys);
    const int n_tiles = key1 > key0 ? (key1 - key0 + 127) / 128 : 0;
    const int n_rows = p.row_count[grp];
    float2 *out = p.chunk_stats + ((int64_t)(grp - p.lb0 * p.Hkv) * p.chunks + chunk) * p.cap;

    DensePipe<D> pp;
    pp.init(s_bar);
    if (tid == 0) {
        pp.init_barriers();
        s_abort = 0;
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
    }
    if (warp == kDenseDriverWarp) tmem_alloc(smem_u32(&s_tmem), 256);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    uint32_t base = 0;   // tiles that went through the pipe in earlier row blocks

    for (int row0 = 0; row0 < n_rows; row0 += 128) {
        __syncthreads();   // the previous block's MMAs have completed (their logits were read): the query block is free
        if (s_abort) break;
        int loaded = 0;
        if (tid < 128) stage_queries_sw128<D>(s_q, p, grp, lb, g, row0, n_rows);
        else if (tid == kDenseDriverWarp * 32) loaded = dense_first_loads<D>(pp, &tm_k, p, s_k, base, n_tiles, key0, g, b, l, &s_abort, 4);
        __syncthreads();
        float m_mine = kNegBig, z_mine = 0.f;
        bool ok_mine = true;
        if (warp == kDenseDriverWarp) {
            if (lane == 0)
                dense_drive<D, true>(pp, &tm_k, p, tmem, s_k, s_q, base, n_tiles, loaded, key0, g, b, l, &s_abort, 4);
        } else {
            float m = kNegBig, z = 0.f;
            bool ok = true;
            // one chunk of 32 logits of the thread's row: running (max, sum of exp2)
            auto chunk32 = [&](const uint32_t (&r)[32], int kbase) {
                float mn, sum = 0.f;
                if (kbase + 32 <= key1) {
                    // all 32 keys are real: the scale is positive, so the largest raw logit gives the largest
                    // scaled one, and the exponent's argument is one fused multiply-add.  Four interleaved
                    // partial maxima and sums keep the dependent chains short (two warps share a scheduler).
                    float mx[4], sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int j = 0; j < 4; ++j) mx[j] = __uint_as_float(r[j]);
#pragma unroll
                    for (int j = 4; j < 32; ++j) mx[j & 3] = fmaxf(mx[j & 3], __uint_as_float(r[j]));
                    mn = fmaxf(m, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * p.sl2);
#pragma unroll
                    for (int j = 0; j < 32; ++j) sm[j & 3] += fast_exp2(fmaf(__uint_as_float(r[j]), p.sl2, -mn));
                    sum = (sm[0] + sm[1]) + (sm[2] + sm[3]);
                } else {
                    float mx = kNegBig;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (kbase + j < key1) mx = fmaxf(mx, __uint_as_float(r[j]) * p.sl2);
                    mn = fmaxf(m, mx);
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        sum += kbase + j < key1 ? fast_exp2(fmaf(__uint_as_float(r[j]), p.sl2, -mn)) : 0.f;
                }
                z = z * fast_exp2(m - mn) + sum;
                m = mn;
            };
            // this set's tiles: those whose accumulator (running tile count, low bit) is the set's
            for (int t = (set - (int)base) & 1; t < n_tiles; t += 2) {
                const uint32_t it = base + t, a = it & 1;
                ok = mbar_wait(pp.acc_full[a], (it >> 1) & 1, &s_abort, p.status, 6);
                if (!ok) break;
                tc_fence_after();
                const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + a * 128;
                const int kbase = key0 + t * 128;
                uint32_t r0[32], r1[32];
                tmem_ld32_issue(taddr, r0);
                tmem_ld_wait(r0);
                tmem_ld32_issue(taddr + 32, r1);
                chunk32(r0, kbase);
                tmem_ld_wait(r1);
                tmem_ld32_issue(taddr + 64, r0);
                chunk32(r1, kbase + 32);
                tmem_ld_wait(r0);
                tmem_ld32_issue(taddr + 96, r1);
                chunk32(r0, kbase + 64);
                tmem_ld_wait(r1);
                // the whole accumulator is in registers: hand it back before the last chunk's arithmetic
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(pp.acc_empty[a]);
                chunk32(r1, kbase + 96);
            }
            if (set == 1) s_mz[row] = make_float2(m, z);
            m_mine = m; z_mine = z; ok_mine = ok;
        }
        __syncthreads();   // the second set's half of every row's statistics is in shared memory
        if (warp < 4 && ok_mine) {
            merge_stats(m_mine, z_mine, s_mz[row].x, s_mz[row].y);
            if (row0 + row < n_rows) __stcg(out + row0 + row, make_float2(m_mine, z_mine));
        }
        base += n_tiles;
    }
    __syncthreads();
    const bool ok = !s_abort;
    if (warp == kDenseDriverWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, 256);
    }
    if (!ok) return;

    // last CTA of the group: merge text and chunk statistics (same scheme as stats_kernel)
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        s_is_last = atomicAdd(p.group_ticket + grp, 1u) == (unsigned)p.chunks - 1;
        if (s_is_last) __threadfence();
    }
    __syncthreads();
    if (!s_is_last || warp >= 4) return;   // four warps merge
    for (int r = warp; r < n_rows; r += 4) {
        float mm = kNegBig, zz = 0.f;
        if (lane == 0) {
            const float2 tx = p.row_text[(int64_t)grp * p.cap + r];
            mm = tx.x; zz = tx.y;
        }
        for (int c = lane; c < p.chunks; c += 32) {
            const float2 cs = __ldcg(p.chunk_stats + ((int64_t)(grp - p.lb0 * p.Hkv) * p.chunks + c) * p.cap + r);
            merge_stats(mm, zz, cs.x, cs.y);
        }
#pragma unroll
        for (int sh = 1; sh < 32; sh <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, mm, sh);
            const float z2 = __shfl_xor_sync(0xffffffffu, zz, sh);
            merge_stats(mm, zz, m2, z2);
        }
        if (lane == 0) p.row_final[(int64_t)grp * p.cap + r] = make_float2(mm, p.row_coef[(int64_t)grp * p.cap + r] / zz);
    }
}

// Pass two, dense.  grid = (chunks, L*B*Hkv) like pass one, 160 threads; an epilogue thread owns one key per tile
// and adds the weighted probabilities of the group's rows.  The group's sums go to its row of the per-group
// buffer (group_sum_kernel adds the groups), or straight to the scores in per-KV-head mode.
template <int D>
__global__ void __launch_bounds__(kDenseThreads, 2) dense_importance_kernel(const __grid_constant__ CUtensorMap tm_k, ScoreParams p) {
    using C = DenseCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *s_k = smem;                             // NST key tiles
    uint8_t *s_q = smem + C::NST * C::TILE_BYTES;    // one query block
    float2 *s_stat = reinterpret_cast<float2 *>(smem + (C::NST + 1) * C::TILE_BYTES);   // (max, weight / normaliser)
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + (C::NST + 1) * C::TILE_BYTES + 128 * 8);
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int set = warp >> 2, row = (warp & 3) * 32 + lane;   // epilogue set and accumulator row (warps 0-7)
    const int grp = p.lb0 * p.Hkv + blockIdx.y;
    const int g = grp % p.Hkv, lb = grp / p.Hkv;
    const int l = lb / p.B, b = lb % p.B;
    const int key0 = blockIdx.x * p.chunk_keys, key1 = min(p.Nv, key0 + p.chunk_keys);
    const int n_tiles = key1 > key0 ? (key1 - key0 + 127) / 128 : 0;
    const int n_rows = p.row_count[grp];
    float *out = (p.per_head ? p.scores : p.imp_part) + (int64_t)grp * p.Nv;

    DensePipe<D> pp;
    pp.init(s_bar);
    if (tid == 0) {
        pp.init_barriers();
        s_abort = 0;
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
    }
    if (warp == kDenseDriverWarp) tmem_alloc(smem_u32(&s_tmem), 256);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    uint32_t base = 0;

    for (int row0 = 0; row0 < n_rows; row0 += 128) {
        __syncthreads();   // the previous block's MMAs have completed: query block and statistics are free
        if (s_abort) break;
        int loaded = 0;
        if (tid < 128) {
            stage_queries_sw128<D>(s_q, p, grp, lb, g, row0, n_rows);
            s_stat[tid] = row0 + tid < n_rows ? p.row_final[(int64_t)grp * p.cap + row0 + tid] : make_float2(0.f, 0.f);
        } else if (tid == kDenseDriverWarp * 32) {
            loaded = dense_first_loads<D>(pp, &tm_k, p, s_k, base, n_tiles, key0, g, b, l, &s_abort, 10);
        }
        __syncthreads();
        if (warp == kDenseDriverWarp) {
            if (lane == 0)
                dense_drive<D, false>(pp, &tm_k, p, tmem, s_k, s_q, base, n_tiles, loaded, key0, g, b, l, &s_abort, 10);
        } else {
            const int nch = (min(128, n_rows - row0) + 31) >> 5;   // chunks of 32 rows with a real row in them
            // 32 rows of the thread's key: probabilities weighted and summed
            auto chunk32 = [&](const uint32_t (&r)[32], int c0) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};   // interleaved partial sums: short dependent chains
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float2 sj = s_stat[c0 + j];
                    acc[j & 3] = fmaf(fast_exp2(fmaf(__uint_as_float(r[j]), p.sl2, -sj.x)), sj.y, acc[j & 3]);
                }
                return (acc[0] + acc[1]) + (acc[2] + acc[3]);
            };
            // this set's tiles: those whose accumulator (running tile count, low bit) is the set's
            for (int t = (set - (int)base) & 1; t < n_tiles; t += 2) {
                const uint32_t it = base + t, a = it & 1;
                if (!mbar_wait(pp.acc_full[a], (it >> 1) & 1, &s_abort, p.status, 12)) break;
                tc_fence_after();
                const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + a * 128;
                uint32_t r0[32], r1[32];
                float acc = 0.f;
                tmem_ld32_issue(taddr, r0);
                tmem_ld_wait(r0);
                if (nch > 1) tmem_ld32_issue(taddr + 32, r1);
                acc += chunk32(r0, 0);
                if (nch > 1) {
                    tmem_ld_wait(r1);
                    if (nch > 2) tmem_ld32_issue(taddr + 64, r0);
                    acc += chunk32(r1, 32);
                    if (nch > 2) {
                        tmem_ld_wait(r0);
                        if (nch > 3) tmem_ld32_issue(taddr + 96, r1);
                        acc += chunk32(r0, 64);
                        if (nch > 3) {
                            tmem_ld_wait(r1);
                            acc += chunk32(r1, 96);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(pp.acc_empty[a]);
                // the thread's key of this tile: first row block writes, later ones add (same thread every time)
                const int key = key0 + t * 128 + row;
                if (key < key1) out[key] = row0 == 0 ? acc : out[key] + acc;
            }
        }
        base += n_tiles;
    }
    __syncthreads();
    if (warp == kDenseDriverWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, 256);
    }
}

template <int D, int NT>
int launch_stats(ScoreParams p, int rows_lo, int rows_hi, cudaStream_t st) {
    p.rows_lo = rows_lo; p.rows_hi = rows_hi;
    stats_kernel<D, NT><<<dim3(p.chunks, (unsigned)((int64_t)p.n_lb * p.Hkv)), 128, 0, st>>>(p);
    AIRCACHE_LAUNCH_CHECK();
    return AIRCACHE_OK;
}

template <int D, int NT>
int launch_importance(const ScoreParams &p, cudaStream_t st) {
    importance_kernel<D, NT><<<dim3((p.Nv + kScoreKeyTile - 1) / kScoreKeyTile, (unsigned)p.n_lb), 128, 0,
                               st>>>(p);
    AIRCACHE_LAUNCH_CHECK();
    return AIRCACHE_OK;
}

// The number of elite rows of a KV group is known on the device only and is small for the paper's
// threshold (a few rows per head), far below the G*W the shape allows.  The statistics pass keeps per-row
// state in registers, so groups with at most 32 rows run in a 4-tile instantiation (more CTAs per SM); if
// the shape allows more rows, a second launch with the wide instantiation picks up the groups beyond 32
// rows and exits at once elsewhere.  The importance pass keeps no per-row state and runs once.
template <int D>
int launch_passes_d(const ScoreParams &p, cudaStream_t st) {
    const int nt_max = (p.G * p.W + 7) / 8;
    const int big = 1 << 30;
    int rc;
    if (nt_max <= 2) {
        if ((rc = launch_stats<D, 2>(p, 0, big, st))) return rc;
        return launch_importance<D, 2>(p, st);
    }
    if ((rc = launch_stats<D, 4>(p, 0, nt_max <= 4 ? big : 32, st))) return rc;
    if (nt_max > 4) {
        rc = nt_max <= 8 ? launch_stats<D, 8>(p, 32, big, st) : launch_stats<D, 16>(p, 32, big, st);
        if (rc) return rc;
    }
    return nt_max <= 4 ? launch_importance<D, 4>(p, st) : launch_importance<D, 8>(p, st);
}

// 5-D tensor map over the caller's key cache: channels innermost, then token / head / sequence / layer in
// the order of their strides (smallest first); one box = 64 channels x 128 tokens.
int make_key_map(CUtensorMap *tm, ScoreParams &p, const aircache_shape_t *s, const aircache_full_t *f) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return AIRCACHE_ERR_CUDA;
    struct Dim { int64_t size, stride; int which; };
    Dim dims[4] = {{(int64_t)s->n_visual + s->n_text, f->stride_token, 0}, {s->n_kv_heads, f->stride_head, 1},
                   {s->batch, f->stride_batch, 2}, {s->n_layers, f->stride_layer, 3}};
    for (int i = 0; i < 4; ++i)
        for (int j = i + 1; j < 4; ++j)
            if (dims[j].stride < dims[i].stride || (dims[j].stride == dims[i].stride && dims[j].size < dims[i].size)) {
                const Dim t = dims[i]; dims[i] = dims[j]; dims[j] = t;
            }
    cuuint64_t gdim[5] = {(cuuint64_t)s->head_dim, 1, 1, 1, 1};
    cuuint64_t gstr[4] = {0, 0, 0, 0};
    cuuint32_t box[5] = {64, 1, 1, 1, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    int pos[4] = {0, 0, 0, 0};
    for (int i = 0; i < 4; ++i) {
        gdim[i + 1] = (cuuint64_t)dims[i].size;
        // a dimension of extent 1 never moves; give it the smallest stride the encoder accepts
        gstr[i] = (cuuint64_t)(dims[i].stride > 0 ? dims[i].stride : s->head_dim) * 2;
        pos[dims[i].which] = i + 1;
        if (dims[i].which == 0) box[i + 1] = 128;
    }
    p.pos_token = pos[0]; p.pos_head = pos[1]; p.pos_batch = pos[2]; p.pos_layer = pos[3];
    const CUresult rc = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(f->k), gdim, gstr, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? AIRCACHE_OK : AIRCACHE_ERR_CUDA;
}

template <int D>
int launch_dense(ScoreParams &p, const CUtensorMap &tm, cudaStream_t st) {
    using C = DenseCfg<D>;
    AIRCACHE_CUDA_TRY(cudaFuncSetAttribute(dense_stats_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_STATS));
    AIRCACHE_CUDA_TRY(cudaFuncSetAttribute(dense_importance_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           C::SMEM_IMP));
    dense_stats_kernel<D><<<dim3(p.chunks, (unsigned)((int64_t)p.n_lb * p.Hkv)), kDenseThreads, C::SMEM_STATS, st>>>(tm, p);
    AIRCACHE_LAUNCH_CHECK();
    dense_importance_kernel<D><<<dim3(p.chunks, (unsigned)((int64_t)p.n_lb * p.Hkv)), kDenseThreads, C::SMEM_IMP, st>>>(tm, p);
    AIRCACHE_LAUNCH_CHECK();
    if (!p.per_head) {
        group_sum_kernel<<<dim3((p.Nv + 255) / 256, (unsigned)p.n_lb), 256, 0, st>>>(p);
        AIRCACHE_LAUNCH_CHECK();
    }
    return AIRCACHE_OK;
}

}  // namespace

int launch_score(const aircache_shape_t *s, const aircache_full_t *f, const void *q_window, float alpha,
                 int layer_begin, int layer_count, float *scores, uint64_t *elite_mask, void *ws, cudaStream_t st) {
    const WsLayout w = ws_layout(s);
    ScoreParams p;
    p.k = (const uint16_t *)f->k;
    p.s_layer = f->stride_layer; p.s_batch = f->stride_batch; p.s_head = f->stride_head; p.s_token = f->stride_token;
    p.qw = (const uint16_t *)q_window;
    p.scores = scores;
    p.elite_mask = elite_mask;
    p.row_count = ws_ptr<int32_t>(ws, w.row_count);
    p.row_info = ws_ptr<int32_t>(ws, w.row_info);
    p.row_coef = ws_ptr<float>(ws, w.row_coef);
    p.row_text = ws_ptr<float2>(ws, w.row_text);
    p.chunk_stats = ws_ptr<float2>(ws, w.chunk_stats);
    p.row_final = ws_ptr<float2>(ws, w.row_final);
    p.group_ticket = ws_ptr<uint32_t>(ws, w.group_ticket);
    p.dispatch = ws_ptr<uint32_t>(ws, w.dispatch);
    p.imp_part = ws_ptr<float>(ws, w.imp_part);
    p.q_block = ws_ptr<uint16_t>(ws, w.q_block);
    // A call over few KV groups (a layer at a time, a single short sequence) would leave SMs idle with 512- and
    // 1024-key blocks: while the blocks would fill less than half of the GPU, they take half the tiles per warp,
    // down to 256 keys per block (config 4 a layer at a time: 41 -> 33 us per layer).
    {
        const int resident = s->head_dim == 64 ? onepass_resident_blocks<64>() : onepass_resident_blocks<128>();
        const int64_t groups = (int64_t)layer_count * s->batch * s->n_kv_heads;
        auto numbers_per_group = [&](int cap) { const int k = 64 * (cap < 8 ? cap : 8); return (s->n_visual + k - 1) / k; };
        p.op_tile_cap = 16;
        while (p.op_tile_cap > 4 &&
               groups * ((s->n_visual + 64 * p.op_tile_cap - 1) / (64 * p.op_tile_cap)) * 2 < (int64_t)resident &&
               (int64_t)numbers_per_group(p.op_tile_cap / 2) * 2 <= resident)
            p.op_tile_cap >>= 1;
        p.op_chunks = numbers_per_group(p.op_tile_cap);
    }
    p.L = s->n_layers; p.B = s->batch; p.Hq = s->n_q_heads; p.Hkv = s->n_kv_heads;
    p.G = s->n_q_heads / s->n_kv_heads; p.d = s->head_dim; p.Nv = s->n_visual; p.Nt = s->n_text; p.W = s->window;
    p.per_head = s->per_kv_head;
    p.lb0 = layer_begin * s->batch;
    p.n_lb = layer_count * s->batch;
    p.cap = score_row_cap(s);
    p.chunks = score_chunks(s->n_visual, (int64_t)layer_count * s->batch * s->n_kv_heads);
    p.chunk_keys = (int)align_up((s->n_visual + p.chunks - 1) / p.chunks, 16);
    p.scale = s->scale;
    p.sl2 = s->scale * kLog2e;
    p.keep_all = alpha <= 0.0f;
    p.ln_alpha = p.keep_all ? 0.0f : (float)log((double)alpha);
    p.rows_lo = 0; p.rows_hi = 1 << 30;
    p.pos_token = p.pos_head = p.pos_batch = p.pos_layer = 0;
    p.status = ws_ptr<uint32_t>(ws, w.status);

    const int64_t groups = (int64_t)p.n_lb * p.Hkv;
    const size_t elite_smem = (size_t)(p.W + p.G) * (p.d + 8) * 2;
    if (p.keep_all) {
        if (s->head_dim == 64) elite_kernel<64, true><<<(unsigned)groups, 128, elite_smem, st>>>(p);
        else elite_kernel<128, true><<<(unsigned)groups, 128, elite_smem, st>>>(p);
    } else {
        if (s->head_dim == 64) elite_kernel<64, false><<<(unsigned)groups, 128, elite_smem, st>>>(p);
        else elite_kernel<128, false><<<(unsigned)groups, 128, elite_smem, st>>>(p);
    }
    AIRCACHE_LAUNCH_CHECK();
    // alpha = 0 keeps all G*W window queries: the dense contraction goes to tcgen05 (if a tensor map over the
    // caller's strides can be made; otherwise the mma.sync passes handle it as well)
#ifndef AIRCACHE_NO_DENSE
    if (p.keep_all && p.G * p.W >= 32) {
        CUtensorMap tm;
        if (make_key_map(&tm, p, s, f) == AIRCACHE_OK)
            return s->head_dim == 64 ? launch_dense<64>(p, tm, st) : launch_dense<128>(p, tm, st);
    }
#endif
    // one pass over the keys, if a group's blocks are sure to be resident together
    const int resident = s->head_dim == 64 ? onepass_resident_blocks<64>() : onepass_resident_blocks<128>();
    if ((int64_t)p.op_chunks * 2 <= resident && (int64_t)p.n_lb * p.Hkv * p.op_chunks < ((int64_t)1 << 31))
        return s->head_dim == 64 ? launch_onepass<64>(p, st) : launch_onepass<128>(p, st);
    return s->head_dim == 64 ? launch_passes_d<64>(p, st) : launch_passes_d<128>(p, st);
}

}  // namespace aircache
