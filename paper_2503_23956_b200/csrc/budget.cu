// aircache_budget: strength and skewness of every region's importance distribution (Eq. 9-10), the
// layer-wise budget of Eq. 11 turned into integer row counts, and the row offsets of the ragged cache.
//
//   moments_kernel   one CTA per region: three fp64 block reductions (sum; squared deviations; cubed
//                    standardised deviations) over the fp32 scores, fixed reduction tree.
//   allocate_kernel  one CTA: thread b walks the layers of sequence b in order and performs the capped
//                    proportional split with largest-remainder rounding in fp64, every operation
//                    individually rounded (no fused multiply-add), then all threads scan the region sizes.
#include <math.h>

#include "common.cuh"

namespace aircache {

namespace {

constexpr int kMomThreads = 256;

__device__ __forceinline__ double block_sum(double v, double *s_part) {
#pragma unroll
    for (int sh = 16; sh > 0; sh >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, sh));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) s_part[warp] = v;
    __syncthreads();
    double tot = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot = __dadd_rn(tot, s_part[w]);
    return tot;
}

// Eq. 9 and Eq. 10 (adjusted Fisher-Pearson coefficient, sample standard deviation).
__global__ void __launch_bounds__(kMomThreads) moments_kernel(const float *__restrict__ scores, int n_visual,
                                                              double *__restrict__ strength,
                                                              double *__restrict__ skewness) {
    __shared__ double s_part[kMomThreads / 32];
    const float *x = scores + (int64_t)blockIdx.x * n_visual;
    const double n = (double)n_visual;

    double s = 0.0;
    for (int i = threadIdx.x; i < n_visual; i += kMomThreads) s = __dadd_rn(s, (double)x[i]);
    s = block_sum(s, s_part);
    const double mu = __ddiv_rn(s, n);

    double ss = 0.0;
    for (int i = threadIdx.x; i < n_visual; i += kMomThreads) {
        const double c = __dsub_rn((double)x[i], mu);
        ss = __dadd_rn(ss, __dmul_rn(c, c));
    }
    ss = block_sum(ss, s_part);
    const double sigma = __dsqrt_rn(__ddiv_rn(ss, __dsub_rn(n, 1.0)));

    double cube = 0.0;
    if (sigma > 0.0) {
        for (int i = threadIdx.x; i < n_visual; i += kMomThreads) {
            const double zc = __ddiv_rn(__dsub_rn((double)x[i], mu), sigma);
            cube = __dadd_rn(cube, __dmul_rn(__dmul_rn(zc, zc), zc));
        }
    }
    cube = block_sum(cube, s_part);
    if (threadIdx.x == 0) {
        strength[blockIdx.x] = s;
        const double pre = __ddiv_rn(n, __dmul_rn(__dsub_rn(n, 1.0), __dsub_rn(n, 2.0)));
        skewness[blockIdx.x] = (sigma > 0.0) ? __dmul_rn(pre, cube) : 0.0;
    }
}

struct AllocParams {
    const double *strength, *skewness;  // [L,B]
    double *w, *share;                  // [L,B] scratch
    int32_t *active;                    // [L,B] scratch
    int32_t *budgets;                   // [L,B]
    int64_t *offsets;                   // [L*B+1]
    int32_t *lens;                      // [L*B]
    int L, B, Nv, Nt, slack, mode;
    long long total_kept;               // T per sequence
};

constexpr int kAllocThreads = 1024;

__global__ void __launch_bounds__(kAllocThreads) allocate_kernel(AllocParams p) {
    const int L = p.L, B = p.B;
    // ---- Eq. 11 + integer budgets, one thread per sequence ----
    for (int b = threadIdx.x; b < B; b += kAllocThreads) {
        double mean_t = 0.0, mean_k = 0.0;
        for (int l = 0; l < L; ++l) {
            mean_t = __dadd_rn(mean_t, p.strength[l * B + b]);
            const double sk = p.skewness[l * B + b];
            mean_k = __dadd_rn(mean_k, sk > 0.0 ? sk : 0.0);
        }
        mean_t = __ddiv_rn(mean_t, (double)L);
        mean_k = __ddiv_rn(mean_k, (double)L);
        for (int l = 0; l < L; ++l) {
            const double st = p.strength[l * B + b];
            double sk = p.skewness[l * B + b];
            if (sk < 0.0) sk = 0.0;
            const double nt = mean_t > 0.0 ? __ddiv_rn(st, mean_t) : 1.0;
            const double nk = mean_k > 0.0 ? __ddiv_rn(sk, mean_k) : 1.0;
            double w;
            if (p.mode == 0) w = __dmul_rn(0.5, __dadd_rn(nt, nk));
            else if (p.mode == 1) w = nt;
            else if (p.mode == 2) w = nk;
            else w = 1.0;
            p.w[l * B + b] = w;
            p.active[l * B + b] = 1;
        }
        long long R = p.total_kept;
        // capped proportional split: a layer whose share reaches Nv keeps everything, the rest re-share
        for (;;) {
            double wsum = 0.0;
            int n_active = 0;
            for (int l = 0; l < L; ++l)
                if (p.active[l * B + b]) { wsum = __dadd_rn(wsum, p.w[l * B + b]); ++n_active; }
            if (n_active == 0) break;
            for (int l = 0; l < L; ++l) {
                if (!p.active[l * B + b]) continue;
                p.share[l * B + b] = wsum > 0.0 ? __ddiv_rn(__dmul_rn((double)R, p.w[l * B + b]), wsum)
                                                : __ddiv_rn((double)R, (double)n_active);
            }
            bool moved = false;
            for (int l = 0; l < L; ++l) {
                if (p.active[l * B + b] && p.share[l * B + b] >= (double)p.Nv) {
                    p.budgets[l * B + b] = p.Nv;
                    p.active[l * B + b] = 0;
                    R -= p.Nv;
                    moved = true;
                }
            }
            if (!moved) break;
        }
        // floors, then the largest fractional parts (ties to the lower layer) take one more row each
        long long given = 0;
        for (int l = 0; l < L; ++l) {
            if (!p.active[l * B + b]) continue;
            const double sh = p.share[l * B + b];
            const int f = (int)floor(sh);
            p.budgets[l * B + b] = f;
            given += f;
            p.share[l * B + b] = __dsub_rn(sh, (double)f);
        }
        for (long long left = R - given; left > 0; --left) {
            int best = -1;
            double best_frac = 0.0;
            for (int l = 0; l < L; ++l) {
                if (!p.active[l * B + b]) continue;
                const double fr = p.share[l * B + b];
                if (best < 0 || fr > best_frac) { best = l; best_frac = fr; }
            }
            if (best < 0) break;
            p.budgets[best * B + b] += 1;
            p.active[best * B + b] = 0;
        }
    }
    __syncthreads();

    // ---- offsets: exclusive scan of (budget + Nt + slack) over r = l*B + b ----
    __shared__ long long s_warp[kAllocThreads / 32];
    const int n = L * B;
    const int per = (n + kAllocThreads - 1) / kAllocThreads;
    const int i0 = threadIdx.x * per, i1 = min(n, i0 + per);
    long long local = 0;
    for (int i = i0; i < i1; ++i) local += p.budgets[i] + p.Nt + p.slack;
    long long incl = local;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
        const long long o = __shfl_up_sync(0xffffffffu, incl, sh);
        if (lane >= sh) incl += o;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        long long v = s_warp[lane];
#pragma unroll
        for (int sh = 1; sh < 32; sh <<= 1) {
            const long long o = __shfl_up_sync(0xffffffffu, v, sh);
            if (lane >= sh) v += o;
        }
        s_warp[lane] = v;
    }
    __syncthreads();
    long long run = incl - local + (warp > 0 ? s_warp[warp - 1] : 0);
    for (int i = i0; i < i1; ++i) {
        p.offsets[i] = run;
        p.lens[i] = p.budgets[i] + p.Nt;
        run += p.budgets[i] + p.Nt + p.slack;
    }
    if (threadIdx.x == kAllocThreads - 1) p.offsets[n] = s_warp[kAllocThreads / 32 - 1];
}

}  // namespace

int launch_budget(const aircache_shape_t *s, const float *scores, double ratio, int32_t mode, int32_t *budgets,
                  double *strength, double *skewness, aircache_ragged_t *layout, void *ws, cudaStream_t st) {
    const WsLayout w = ws_layout(s);
    const int LB = s->n_layers * s->batch;
    double *d_st = strength ? strength : ws_ptr<double>(ws, w.mom_strength);
    double *d_sk = skewness ? skewness : ws_ptr<double>(ws, w.mom_skew);
    moments_kernel<<<LB, kMomThreads, 0, st>>>(scores, s->n_visual, d_st, d_sk);
    AIRCACHE_LAUNCH_CHECK();
    AllocParams p;
    p.strength = d_st; p.skewness = d_sk;
    p.w = ws_ptr<double>(ws, w.alloc_w);
    p.share = ws_ptr<double>(ws, w.alloc_share);
    p.active = ws_ptr<int32_t>(ws, w.alloc_active);
    p.budgets = budgets;
    p.offsets = layout->offsets;
    p.lens = layout->lens;
    p.L = s->n_layers; p.B = s->batch; p.Nv = s->n_visual; p.Nt = s->n_text; p.slack = s->slack; p.mode = mode;
    p.total_kept = kept_per_sequence(s, ratio);
    allocate_kernel<<<1, kAllocThreads, 0, st>>>(p);
    AIRCACHE_LAUNCH_CHECK();
    return AIRCACHE_OK;
}

}  // namespace aircache
