// aircache_compact: per-region top-k of the importance scores and the gather that packs the kept
// visual rows and all text rows into the ragged cache (Algorithm 1, second loop); aircache_append (Eq. 2).
//
//   select_kernel  one CTA per region.  Radix select, most significant byte first, on an order-preserving
//                  integer image of the fp32 score: four 256-bin histogram passes find the value of the
//                  k-th largest score and how many of its duplicates are needed; one ordered pass then
//                  emits the kept token indices in ascending order, duplicates of the threshold value
//                  taken from the lowest indices.
//   gather_kernel  one warp per output row [Hkv, d] of K' and of V': 16-byte loads along the source row's
//                  head slices, 16-byte stores to the packed row.  Region of a row by binary search in the
//                  offsets table.
#include "common.cuh"

namespace aircache {

namespace {

constexpr int kSelThreads = 512;
constexpr int kSelSmemKeys = 40960;  // scores kept in shared memory up to this many visual tokens

// Order-preserving integer image of a float: a > b as floats <=> key(a) > key(b), a == b <=> equal keys.  The
// two zeros compare equal as floats, so -0.0 takes the key of +0.0 (the lower index then wins among them).
__device__ __forceinline__ uint32_t order_key(float x) {
    uint32_t u = __float_as_uint(x);
    if ((u << 1) == 0u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive block scan of one int per thread; returns the exclusive prefix, total in *total.
__device__ __forceinline__ int block_excl_scan(int v, int *s_warp, int *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, sh);
        if (lane >= sh) incl += o;
    }
    __syncthreads();
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < (kSelThreads / 32) ? s_warp[lane] : 0;
#pragma unroll
        for (int sh = 1; sh < 32; sh <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, w, sh);
            if (lane >= sh) w += o;
        }
        if (lane < kSelThreads / 32) s_warp[lane] = w;
    }
    __syncthreads();
    *total = s_warp[kSelThreads / 32 - 1];
    return incl - v + (warp > 0 ? s_warp[warp - 1] : 0);
}

template <bool SMEM_KEYS>
__global__ void __launch_bounds__(kSelThreads) select_kernel(const float *__restrict__ scores,
                                                             const int32_t *__restrict__ budgets,
                                                             const int64_t *__restrict__ offsets, int n_visual,
                                                             int n_text, int slack, int64_t first_row,
                                                             int32_t *__restrict__ kept, int64_t kept_cap,
                                                             uint32_t *status) {
    extern __shared__ uint32_t s_keys[];
    __shared__ int s_hist[256];
    __shared__ int s_warp[kSelThreads / 32];
    __shared__ uint32_t s_prefix;
    __shared__ int s_remaining;

    // the gather kernel that follows may start its text rows now; it waits before it reads the lists
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.x;
    const int k = budgets[r];
    // the region's list starts after the kept rows of the regions before it; budgets and offsets come from
    // device memory, so a pair that does not fit the list buffer is reported instead of followed
    const int64_t start = offsets[r] - first_row - (int64_t)r * (n_text + slack);
    if (k < 0 || k > n_visual || start < 0 || start + k > kept_cap) {
        if (threadIdx.x == 0) atomicExch(status, kStatusInconsistent);
        return;
    }
    int32_t *out = kept + start;
    const float *x = scores + (int64_t)r * n_visual;
    if (k <= 0) return;
    if (k >= n_visual) {
        for (int i = threadIdx.x; i < n_visual; i += kSelThreads) out[i] = i;
        return;
    }
    if (SMEM_KEYS) {
        for (int i = threadIdx.x; i < n_visual; i += kSelThreads) s_keys[i] = order_key(x[i]);
    }
    auto key_at = [&](int i) -> uint32_t { return SMEM_KEYS ? s_keys[i] : order_key(x[i]); };

    if (threadIdx.x == 0) { s_prefix = 0; s_remaining = k; }
    uint32_t mask = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += kSelThreads) s_hist[i] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        // scores of one layer share most of their exponent, so the first passes put nearly every key into one
        // or two bins: a warp whose 32 keys share the digit adds them with one atomic
        for (int i0 = 0; i0 < n_visual; i0 += kSelThreads) {
            const int i = i0 + threadIdx.x;
            const uint32_t key = i < n_visual ? key_at(i) : 0u;
            const bool in = i < n_visual && (key & mask) == prefix;
            const int bin = in ? (int)((key >> shift) & 255) : -1;
            int same;
            __match_all_sync(0xffffffffu, bin, &same);
            if (same) {
                if (in && (threadIdx.x & 31) == 0) atomicAdd(&s_hist[bin], 32);
            } else if (in) {
                atomicAdd(&s_hist[bin], 1);
            }
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // warp 0: walk the bins from the largest digit down until `remaining` keys are covered
            const int lane = threadIdx.x;
            int remaining = s_remaining;
            int chosen = -1;
            for (int base = 224; base >= 0 && chosen < 0; base -= 32) {
                const int bin = base + 31 - lane;  // lane 0 holds the largest digit of the group
                const int c = s_hist[bin];
                int incl = c;
#pragma unroll
                for (int sh = 1; sh < 32; sh <<= 1) {
                    const int o = __shfl_up_sync(0xffffffffu, incl, sh);
                    if (lane >= sh) incl += o;
                }
                const unsigned hit = __ballot_sync(0xffffffffu, incl >= remaining);
                if (hit) {
                    const int src = __ffs(hit) - 1;
                    const int before = __shfl_sync(0xffffffffu, incl - c, src);
                    chosen = base + 31 - src;
                    remaining -= before;
                } else {
                    remaining -= __shfl_sync(0xffffffffu, incl, 31);
                }
            }
            if (lane == 0) {
                s_prefix = prefix | ((uint32_t)chosen << shift);
                s_remaining = remaining;
            }
        }
        mask |= 255u << shift;
        __syncthreads();
    }
    const uint32_t thr = s_prefix;   // image of the k-th largest score
    const int need_eq = s_remaining; // how many tokens equal to it are kept (lowest indices first)

    // ordered emit: thread t owns the contiguous index range [i0, i1)
    const int per = (n_visual + kSelThreads - 1) / kSelThreads;
    const int i0 = min(n_visual, (int)threadIdx.x * per), i1 = min(n_visual, i0 + per);
    int n_eq = 0, n_gt = 0;
    for (int i = i0; i < i1; ++i) {
        const uint32_t key = key_at(i);
        n_eq += key == thr;
        n_gt += key > thr;
    }
    int tot;
    const int eq_before = block_excl_scan(n_eq, s_warp, &tot);
    int take_eq = min(max(need_eq - eq_before, 0), n_eq);
    const int pos0 = block_excl_scan(n_gt + take_eq, s_warp, &tot);
    int pos = pos0;
    for (int i = i0; i < i1; ++i) {
        const uint32_t key = key_at(i);
        bool keep = key > thr;
        if (key == thr && take_eq > 0) { keep = true; --take_eq; }
        if (keep) out[pos++] = i;
    }
}

struct GatherParams {
    const uint16_t *k, *v;
    int64_t s_layer, s_batch, s_head, s_token;
    uint16_t *k_out, *v_out;
    const int64_t *offsets;
    const int32_t *lens;
    const int32_t *budgets;
    const int32_t *kept;
    int64_t rows_cap;  // rows covered by the launch
    int64_t total_rows;  // rows the output buffers hold
    int64_t kept_cap;    // entries the kept-list buffer holds
    uint32_t *status;
    int64_t first_row; // rows of the shared buffers in front of this cache's first region
    int L, B, Hkv, d, Nv, Nt, slack;
    int Hc;   // cells per (layer, sequence): 1, or the KV heads in per-KV-head mode (a row then holds one head)
};

constexpr int kGatherThreads = 256;
constexpr int kGatherRowsPerWarp = 4;

// Copies the rows of the ragged cache: for region r first the kept visual rows in ascending token order, then
// the text rows (Algorithm 1's C^l = Concat(K_v[kept], K_t)).  A warp moves four rows at a time.
// The text rows need no selection result - their place follows from the budgets alone - so they are copied
// before the kernel waits for its predecessor in the stream (the selection kernel, which releases its
// dependents at once): that part of the traffic runs beside the selection, which occupies one CTA per region
// and is bound by latency, not by bandwidth.
__global__ void __launch_bounds__(kGatherThreads, 4) gather_kernel(GatherParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kGatherThreads + threadIdx.x) >> 5;
    const int64_t row_step = (int64_t)gridDim.x * (kGatherThreads / 32) * kGatherRowsPerWarp;
    const int n_regions = p.L * p.B * p.Hc;       // cells
    const int row_heads = p.Hc > 1 ? 1 : p.Hkv;   // KV heads in one row of the ragged cache
    const int vec_per_head = p.d / 8;             // 16-byte vectors per head slice
    const int vec_per_row = row_heads * vec_per_head;
    // source offset of token `tok` of cell r (its first head's slice)
    auto src_of = [&](int r, int tok) {
        const int lb = r / p.Hc, g0 = r - lb * p.Hc;
        const int l = lb / p.B, b = lb - l * p.B;
        return (int64_t)l * p.s_layer + (int64_t)b * p.s_batch + (int64_t)g0 * p.s_head + (int64_t)tok * p.s_token;
    };

    auto copy_rows = [&](const int64_t (&src_off)[kGatherRowsPerWarp], const int64_t (&dst_row)[kGatherRowsPerWarp]) {
        for (int v0 = lane; v0 < vec_per_row; v0 += 32) {
            const int g = v0 / vec_per_head, c = v0 % vec_per_head;
            uint4 kk[kGatherRowsPerWarp], vv[kGatherRowsPerWarp];
#pragma unroll
            for (int i = 0; i < kGatherRowsPerWarp; ++i) {
                if (dst_row[i] < 0) continue;
                const int64_t so = src_off[i] + (int64_t)g * p.s_head + c * 8;
                kk[i] = __ldg(reinterpret_cast<const uint4 *>(p.k + so));
                vv[i] = __ldg(reinterpret_cast<const uint4 *>(p.v + so));
            }
#pragma unroll
            for (int i = 0; i < kGatherRowsPerWarp; ++i) {
                if (dst_row[i] < 0) continue;
                const int64_t dof = (dst_row[i] * row_heads + g) * p.d + c * 8;
                *reinterpret_cast<uint4 *>(p.k_out + dof) = kk[i];
                *reinterpret_cast<uint4 *>(p.v_out + dof) = vv[i];
            }
        }
    };

    // ---- text rows: row j of region r goes to offsets[r] + budgets[r] + j ----
    const int n_text_rows = n_regions * p.Nt;   // below 2^31: the cache has fewer rows than that
    for (int64_t first = warp0 * kGatherRowsPerWarp; first < n_text_rows; first += row_step) {
        int64_t src_off[kGatherRowsPerWarp], dst_row[kGatherRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kGatherRowsPerWarp; ++i) {
            const int idx = (int)first + i;
            dst_row[i] = -1;
            src_off[i] = 0;
            if (idx >= n_text_rows) continue;
            const int r = idx / p.Nt, j = idx - r * p.Nt;
            src_off[i] = src_of(r, p.Nv + j);
            const int64_t dst = p.offsets[r] + p.budgets[r] + j;
            if (dst < 0 || dst >= p.total_rows) atomicExch(p.status, kStatusInconsistent);   // not written
            else dst_row[i] = dst;
        }
        copy_rows(src_off, dst_row);
    }

    // ---- kept visual rows, once the selection has written its lists ----
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t per = p.Nt + p.slack;   // offsets[r] - first_row - r * per = kept rows of the regions before r
    int64_t n_kept = p.offsets[n_regions] - p.first_row - (int64_t)n_regions * per;
    if (n_kept < 0 || n_kept > p.kept_cap) {
        if (threadIdx.x == 0) atomicExch(p.status, kStatusInconsistent);
        n_kept = 0;
    }
    for (int64_t first = warp0 * kGatherRowsPerWarp; first < n_kept; first += row_step) {
        int64_t src_off[kGatherRowsPerWarp], dst_row[kGatherRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kGatherRowsPerWarp; ++i) {
            const int64_t idx = first + i;
            dst_row[i] = -1;
            src_off[i] = 0;
            if (idx >= n_kept) continue;
            // largest r with (kept rows before r) <= idx: regions without kept rows are passed over
            int lo = 0, hi = n_regions - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (p.offsets[mid] - p.first_row - (int64_t)mid * per <= idx) lo = mid; else hi = mid - 1;
            }
            const int r = lo;
            const int64_t base = p.offsets[r];
            const int j = (int)(idx - (base - p.first_row - (int64_t)r * per));
            const int tok = p.kept[idx];
            const int64_t dst = base + j;
            if (tok < 0 || tok >= p.Nv || dst < 0 || dst >= p.total_rows) {
                atomicExch(p.status, kStatusInconsistent);   // not copied
            } else {
                src_off[i] = src_of(r, tok);
                dst_row[i] = dst;
            }
        }
        copy_rows(src_off, dst_row);
    }
}

__global__ void append_kernel(uint16_t *k_out, uint16_t *v_out, const int64_t *offsets, int32_t *lens,
                              const uint16_t *k_new, const uint16_t *v_new, int row_elems) {
    const int r = blockIdx.x;
    const int64_t dst = (offsets[r] + lens[r]) * row_elems;
    const int64_t src = (int64_t)r * row_elems;
    for (int c = threadIdx.x * 8; c < row_elems; c += blockDim.x * 8) {
        *reinterpret_cast<uint4 *>(k_out + dst + c) = *reinterpret_cast<const uint4 *>(k_new + src + c);
        *reinterpret_cast<uint4 *>(v_out + dst + c) = *reinterpret_cast<const uint4 *>(v_new + src + c);
    }
    __syncthreads();
    if (threadIdx.x == 0) lens[r] += 1;
}

}  // namespace

int launch_compact(const aircache_shape_t *s, const aircache_full_t *f, const float *scores,
                   const int32_t *budgets, double ratio, aircache_ragged_t *out, int32_t *kept_idx, void *ws,
                   cudaStream_t st) {
    const WsLayout w = ws_layout(s);
    const int LB = (int)n_cells(s);
    int32_t *kept = kept_idx ? kept_idx : ws_ptr<int32_t>(ws, w.kept);
    uint32_t *status = ws_ptr<uint32_t>(ws, w.status);
    const int64_t kept_cap = (int64_t)s->batch * kept_per_sequence(s, ratio);
    if (s->n_visual <= kSelSmemKeys) {
        const size_t smem = (size_t)s->n_visual * 4;
        AIRCACHE_CUDA_TRY(cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               kSelSmemKeys * 4));
        select_kernel<true><<<LB, kSelThreads, smem, st>>>(scores, budgets, out->offsets, s->n_visual, s->n_text,
                                                           s->slack, out->first_row, kept, kept_cap, status);
    } else {
        select_kernel<false><<<LB, kSelThreads, 0, st>>>(scores, budgets, out->offsets, s->n_visual, s->n_text,
                                                         s->slack, out->first_row, kept, kept_cap, status);
    }
    AIRCACHE_LAUNCH_CHECK();

    GatherParams p;
    p.k = (const uint16_t *)f->k; p.v = (const uint16_t *)f->v;
    p.s_layer = f->stride_layer; p.s_batch = f->stride_batch; p.s_head = f->stride_head; p.s_token = f->stride_token;
    p.k_out = (uint16_t *)out->k; p.v_out = (uint16_t *)out->v;
    p.offsets = out->offsets; p.lens = out->lens; p.budgets = budgets; p.kept = kept;
    p.first_row = out->first_row;
    p.rows_cap = kept_cap + (int64_t)LB * (s->n_text + s->slack);
    p.total_rows = out->total_rows;
    p.kept_cap = kept_cap;
    p.status = status;
    p.Hc = cells_of(s);
    p.L = s->n_layers; p.B = s->batch; p.Hkv = s->n_kv_heads; p.d = s->head_dim;
    p.Nv = s->n_visual; p.Nt = s->n_text; p.slack = s->slack;
    const int64_t rows_per_block = (kGatherThreads / 32) * kGatherRowsPerWarp;
    const int64_t text_rows = (int64_t)LB * s->n_text;
    const int64_t kept_rows = p.rows_cap - (int64_t)LB * (s->n_text + s->slack);
    const int64_t most = text_rows > kept_rows ? text_rows : kept_rows;
    // One block per 32 rows of the longer phase (a grid limited to the resident blocks, each striding through
    // the rows, measured 20 % slower on the large configurations).  Blocks that start after the selection has
    // finished pass the wait at once.
    int64_t blocks = (most + rows_per_block - 1) / rows_per_block;
    if (blocks < 1) blocks = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kGatherThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    AIRCACHE_CUDA_TRY(cudaLaunchKernelEx(&cfg, gather_kernel, p));
    AIRCACHE_LAUNCH_CHECK();
    return AIRCACHE_OK;
}

int launch_append(const aircache_shape_t *s, aircache_ragged_t *c, const void *k_new, const void *v_new,
                  int32_t appended, cudaStream_t st) {
    (void)appended;
    append_kernel<<<(unsigned)n_cells(s), 64, 0, st>>>((uint16_t *)c->k, (uint16_t *)c->v, c->offsets, c->lens,
                                                       (const uint16_t *)k_new, (const uint16_t *)v_new,
                                                       row_heads_of(s) * s->head_dim);
    AIRCACHE_LAUNCH_CHECK();
    return AIRCACHE_OK;
}

}  // namespace aircache
