// aircache_budget: strength and skewness of every region's importance distribution (Eq. 9-10), the
// layer-wise budget of Eq. 11 turned into integer row counts, and the row offsets of the ragged cache.
//
// One launch.  Every CTA reduces one cell (three fp64 block reductions over the fp32 scores, which it
// keeps in registers: sum; squared deviations; cubed standardised deviations; fixed reduction tree).  The
// CTA that finishes a SEQUENCE last (one ticket per sequence in the workspace, put back to zero for the next
// call) runs that sequence's allocation with one warp: sums over the cells taken by one lane in cell order
// and every fp64 operation individually rounded (no fused multiply-add), so that the integer budgets are
// the ones the sequential definition gives; divisions, floors and the ranking of the fractional parts run
// across the lanes.  The CTA that finishes the last sequence scans the region sizes into offsets.
#include <math.h>

#include "common.cuh"

namespace aircache {

namespace {

constexpr int kThreads = 512;
constexpr int kPerThread = 16;   // scores a thread keeps in registers (covers N_v <= 8192; beyond, re-read)

struct BudgetParams {
    const float *scores;     // [L*B, Nv]
    double *strength, *skewness;  // [L,B]
    int32_t *budgets;        // [L,B]
    int64_t *offsets;        // [L*B+1]
    int32_t *lens;           // [L*B]
    uint32_t *ticket;        // sequences allocated so far; zero between calls
    uint32_t *seq_ticket;    // [B] cells of the sequence reduced so far; zero between calls
    int L, B, Hc, Nv, Nt, slack, mode;   // Hc: cells per (layer, sequence) - the KV heads in per-KV-head mode, else 1
    long long total_kept;    // T per sequence
    long long first_row;     // rows of the shared buffers in front of this cache's first region
};

__device__ __forceinline__ double block_sum(double v, double *s_part) {
#pragma unroll
    for (int sh = 16; sh > 0; sh >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, sh));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) s_part[warp] = v;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) tot = __dadd_rn(tot, s_part[w]);
    return tot;
}

__device__ __forceinline__ double warp_bcast(double v, int src) {
    return __shfl_sync(0xffffffffu, v, src);
}

// Eq. 11 and the integer budgets of one sequence, by one warp.  st/sk/w/share/bud/act are arrays in shared memory
// over the sequence's cells - its layers, or its (layer, KV head) pairs in per-KV-head mode, layer-major -
// numbered l = 0 .. n - 1; act flags cells that still take part in the proportional split.
__device__ void allocate_sequence(const BudgetParams &p, int n, const double *st, const double *sk, double *w,
                                  double *share, unsigned char *act, int *bud) {
    const int L = n, lane = threadIdx.x & 31;
    // across-layer means: one lane, layer order (this fixes the rounding of the sums)
    double mean_t = 0.0, mean_k = 0.0;
    if (lane == 0) {
        for (int l = 0; l < L; ++l) {
            mean_t = __dadd_rn(mean_t, st[l]);
            const double s = sk[l];
            mean_k = __dadd_rn(mean_k, s > 0.0 ? s : 0.0);
        }
        mean_t = __ddiv_rn(mean_t, (double)L);
        mean_k = __ddiv_rn(mean_k, (double)L);
    }
    mean_t = warp_bcast(mean_t, 0);
    mean_k = warp_bcast(mean_k, 0);
    for (int l = lane; l < L; l += 32) {
        const double t = st[l];
        double s = sk[l];
        if (s < 0.0) s = 0.0;
        const double nt = mean_t > 0.0 ? __ddiv_rn(t, mean_t) : 1.0;
        const double nk = mean_k > 0.0 ? __ddiv_rn(s, mean_k) : 1.0;
        double ww;
        if (p.mode == 0) ww = __dmul_rn(0.5, __dadd_rn(nt, nk));
        else if (p.mode == 1) ww = nt;
        else if (p.mode == 2) ww = nk;
        else ww = 1.0;
        w[l] = ww;
        act[l] = 1;
    }
    __syncwarp();
    long long R = p.total_kept;
    // capped proportional split: a layer whose share reaches Nv keeps everything, the rest re-share
    for (;;) {
        double wsum = 0.0;
        int n_active = 0;
        if (lane == 0) {
            for (int l = 0; l < L; ++l)
                if (act[l]) { wsum = __dadd_rn(wsum, w[l]); ++n_active; }
        }
        wsum = warp_bcast(wsum, 0);
        n_active = __shfl_sync(0xffffffffu, n_active, 0);
        if (n_active == 0) break;
        int moved = 0;
        for (int l = lane; l < L; l += 32) {
            if (!act[l]) continue;
            const double sh = wsum > 0.0 ? __ddiv_rn(__dmul_rn((double)R, w[l]), wsum)
                                         : __ddiv_rn((double)R, (double)n_active);
            share[l] = sh;
            if (sh >= (double)p.Nv) {
                bud[l] = p.Nv;
                act[l] = 0;
                ++moved;
            }
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) moved += __shfl_xor_sync(0xffffffffu, moved, s);
        __syncwarp();
        if (moved == 0) break;
        R -= (long long)moved * p.Nv;
    }
    // floors, then the largest fractional parts (ties to the lower layer) take one more row each
    int given = 0;
    for (int l = lane; l < L; l += 32) {
        if (!act[l]) continue;
        const double sh = share[l];
        const int f = (int)floor(sh);
        bud[l] = f;
        given += f;
        share[l] = __dsub_rn(sh, (double)f);
    }
    long long given_all = given;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) given_all += __shfl_xor_sync(0xffffffffu, given_all, s);
    __syncwarp();
    const long long left = R - given_all;
    // a layer gets the extra row iff fewer than `left` active layers precede it in the order
    // (fraction descending, layer ascending): the same set the one-at-a-time selection picks
    for (int l = lane; l < L; l += 32) {
        if (!act[l]) continue;
        const double fr = share[l];
        long long rank = 0;
        for (int l2 = 0; l2 < L; ++l2) {
            if (!act[l2]) continue;
            const double f2 = share[l2];
            rank += (f2 > fr) || (f2 == fr && l2 < l);
        }
        if (rank < left) bud[l] += 1;
    }
    __syncwarp();
}

__global__ void __launch_bounds__(kThreads, 2) budget_kernel(BudgetParams p) {
    extern __shared__ __align__(16) unsigned char s_dyn[];
    __shared__ double s_part[kThreads / 32];
    __shared__ int s_is_last;
    const int tid = threadIdx.x;
    const int LB = p.L * p.B * p.Hc;   // cells

    // ---------------- Eq. 9 and Eq. 10 of cell blockIdx.x ----------------
    {
        const float *x = p.scores + (int64_t)blockIdx.x * p.Nv;
        const double n = (double)p.Nv;
        float v[kPerThread];
#pragma unroll
        for (int k = 0; k < kPerThread; ++k) {
            const int i = tid + k * kThreads;
            v[k] = i < p.Nv ? x[i] : 0.f;
        }
        const bool spill = p.Nv > kThreads * kPerThread;
        double s = 0.0;
#pragma unroll
        for (int k = 0; k < kPerThread; ++k)
            if (tid + k * kThreads < p.Nv) s = __dadd_rn(s, (double)v[k]);
        if (spill)
            for (int i = tid + kPerThread * kThreads; i < p.Nv; i += kThreads) s = __dadd_rn(s, (double)x[i]);
        s = block_sum(s, s_part);
        const double mu = __ddiv_rn(s, n);

        double ss = 0.0;
#pragma unroll
        for (int k = 0; k < kPerThread; ++k)
            if (tid + k * kThreads < p.Nv) { const double c = __dsub_rn((double)v[k], mu); ss = __dadd_rn(ss, __dmul_rn(c, c)); }
        if (spill)
            for (int i = tid + kPerThread * kThreads; i < p.Nv; i += kThreads) {
                const double c = __dsub_rn((double)x[i], mu);
                ss = __dadd_rn(ss, __dmul_rn(c, c));
            }
        ss = block_sum(ss, s_part);
        const double sigma = __dsqrt_rn(__ddiv_rn(ss, __dsub_rn(n, 1.0)));

        double cube = 0.0;
        if (sigma > 0.0) {
#pragma unroll
            for (int k = 0; k < kPerThread; ++k)
                if (tid + k * kThreads < p.Nv) {
                    const double zc = __ddiv_rn(__dsub_rn((double)v[k], mu), sigma);
                    cube = __dadd_rn(cube, __dmul_rn(__dmul_rn(zc, zc), zc));
                }
            if (spill)
                for (int i = tid + kPerThread * kThreads; i < p.Nv; i += kThreads) {
                    const double zc = __ddiv_rn(__dsub_rn((double)x[i], mu), sigma);
                    cube = __dadd_rn(cube, __dmul_rn(__dmul_rn(zc, zc), zc));
                }
        }
        cube = block_sum(cube, s_part);
        if (tid == 0) {
            const double pre = __ddiv_rn(n, __dmul_rn(__dsub_rn(n, 1.0), __dsub_rn(n, 2.0)));
            p.strength[blockIdx.x] = s;
            p.skewness[blockIdx.x] = sigma > 0.0 ? __dmul_rn(pre, cube) : 0.0;
            __threadfence();
            // cell index = (l * B + b) * Hc + g: the sequence is the middle coordinate
            const int b = (blockIdx.x / p.Hc) % p.B;
            const unsigned t = atomicAdd(p.seq_ticket + b, 1u);
            s_is_last = (t == (unsigned)(p.L * p.Hc) - 1);
            if (s_is_last) { p.seq_ticket[b] = 0; __threadfence(); }
        }
        __syncthreads();
        if (!s_is_last) return;
    }

    // ---------------- the sequence's last CTA: its allocation ----------------
    const int b = (blockIdx.x / p.Hc) % p.B;
    const int n = p.L * p.Hc;   // cells of the sequence
    double *st = reinterpret_cast<double *>(s_dyn);
    double *sk = st + n;
    double *w = sk + n;
    double *share = w + n;
    int *bud = reinterpret_cast<int *>(share + n);
    unsigned char *act = reinterpret_cast<unsigned char *>(bud + n);
    // cell l of the sequence sits at ((l / Hc) * B + b) * Hc + l % Hc
    auto at = [&](int l) { return ((l / p.Hc) * p.B + b) * p.Hc + l % p.Hc; };
    for (int l = tid; l < n; l += kThreads) {
        st[l] = __ldcg(p.strength + at(l));
        sk[l] = __ldcg(p.skewness + at(l));
    }
    __syncthreads();
    if (tid < 32) allocate_sequence(p, n, st, sk, w, share, act, bud);
    __syncthreads();
    for (int l = tid; l < n; l += kThreads) {
        __stcg(p.budgets + at(l), bud[l]);
        p.lens[at(l)] = bud[l] + p.Nt;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned t = atomicAdd(p.ticket, 1u);
        s_is_last = (t == (unsigned)p.B - 1);
        if (s_is_last) { *p.ticket = 0; __threadfence(); }
    }
    __syncthreads();
    if (!s_is_last) return;

    // ---------------- the last sequence's CTA: offsets = exclusive scan of (budget + Nt + slack) over the cells ----
    __shared__ long long s_warp[kThreads / 32];
    const int per = (LB + kThreads - 1) / kThreads;
    const int i0 = min(LB, tid * per), i1 = min(LB, i0 + per);
    long long local = 0;
    for (int i = i0; i < i1; ++i) local += __ldcg(p.budgets + i) + p.Nt + p.slack;
    long long incl = local;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
        const long long o = __shfl_up_sync(0xffffffffu, incl, sh);
        if (lane >= sh) incl += o;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        long long vv = lane < kThreads / 32 ? s_warp[lane] : 0;
#pragma unroll
        for (int sh = 1; sh < 32; sh <<= 1) {
            const long long o = __shfl_up_sync(0xffffffffu, vv, sh);
            if (lane >= sh) vv += o;
        }
        if (lane < kThreads / 32) s_warp[lane] = vv;
    }
    __syncthreads();
    long long run = p.first_row + incl - local + (warp > 0 ? s_warp[warp - 1] : 0);
    for (int i = i0; i < i1; ++i) {
        p.offsets[i] = run;
        run += __ldcg(p.budgets + i) + p.Nt + p.slack;
    }
    if (tid == kThreads - 1) p.offsets[LB] = p.first_row + s_warp[kThreads / 32 - 1];
}

}  // namespace

int launch_budget(const aircache_shape_t *s, const float *scores, double ratio, int32_t mode, int32_t *budgets,
                  double *strength, double *skewness, aircache_ragged_t *layout, void *ws, cudaStream_t st) {
    const WsLayout w = ws_layout(s);
    const int LB = (int)n_cells(s);
    BudgetParams p;
    p.scores = scores;
    p.strength = strength ? strength : ws_ptr<double>(ws, w.mom_strength);
    p.skewness = skewness ? skewness : ws_ptr<double>(ws, w.mom_skew);
    p.budgets = budgets;
    p.offsets = layout->offsets;
    p.lens = layout->lens;
    p.ticket = ws_ptr<uint32_t>(ws, w.status) + 2;   // second word pair of the status block
    // one ticket per sequence: the decode kernel's split-K tickets, which every user leaves at zero (calls that
    // share a workspace are ordered on one stream)
    p.seq_ticket = ws_ptr<uint32_t>(ws, w.tickets);
    p.L = s->n_layers; p.B = s->batch; p.Hc = cells_of(s); p.Nv = s->n_visual; p.Nt = s->n_text; p.slack = s->slack; p.mode = mode;
    p.total_kept = kept_per_sequence(s, ratio);
    p.first_row = layout->first_row;
    const size_t smem = (size_t)s->n_layers * cells_of(s) * (4 * 8 + 4 + 1) + 16;
    AIRCACHE_CUDA_TRY(cudaFuncSetAttribute(budget_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
    budget_kernel<<<LB, kThreads, smem, st>>>(p);
    AIRCACHE_LAUNCH_CHECK();
    return AIRCACHE_OK;
}

}  // namespace aircache
