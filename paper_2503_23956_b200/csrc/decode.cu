// aircache_decode_attn: single-token attention over the ragged compressed cache (Section 3.1, token
// decoding), all layers and sequences in one persistent launch.
//
// Work decomposition.  A "unit" is CH consecutive rows of one region (all KV heads, K and V).  Region r
// has ceil(lens[r] / CH) units; the units of all regions form one list, and CTA c takes the contiguous
// range [c * upc, (c+1) * upc) of it, upc = ceil(total / CTAs): the load is balanced to one unit however
// ragged the regions are.  When there are few regions and cutting each one into pieces needs no more CTAs
// than the grid has, the pieces are aligned to regions instead (one query load and one flush per CTA).
// When even (region, KV head) pairs do not outnumber the CTAs, the launcher cuts by such pairs
// ("head-split": the one-KV-head instantiation, the head taken from the item index).  With many regions
// every CTA builds the unit prefix in shared memory (block-wide scan); with few, every warp derives the
// handful of numbers it needs in registers (plan_few_regions), rehearsed before the dependency wait and
// kept in the workspace between calls.  Consecutive units of one region accumulate in registers; a region
// that lies wholly inside one CTA's range is finished and written by that CTA, otherwise the CTA writes
// an unnormalised partial (running max, sum, accumulator) and takes a ticket of the region; the CTA that
// draws the last ticket merges the region's partials (split-K with a result that does not depend on who
// arrives last) and puts the ticket back to zero for the next call.  Nobody waits for anybody.
//
// Inside a CTA.  One producer warp streams units through a ring of shared-memory stages with TMA
// (cp.async.bulk.tensor, 128-byte swizzle, one box of CH rows x 64 channels per KV head and half of
// head_dim) and mbarriers.  Consumer warp (g, ks) owns KV head g and the 16-row block ks of every unit;
// both products are taken transposed, so that the 8 tile columns are the query heads of the KV group:
//   S^T = K Q_g^T   mma.m16n8k16: the 16 keys are the M rows (K fragments from ldmatrix on the swizzled
//                   tile), the G query heads the N columns (two column tiles for 9-16 heads)
//   online softmax in the exp2 domain, column maxima over the eight lanes that share a head pair
//   O^T += V^T P^T  P split into a bf16 head and a bf16 remainder (two MMAs per V fragment: a single bf16
//                   rounding of P costs up to 2^-9 relative, too close to the 2e-3 bar), moved into the
//                   operand layout with movmatrix; V^T fragments from ldmatrix.trans
// The G-fold reuse of every K/V row across the query heads of a group is what puts this on the tensor
// pipe: with plain FMAs the kernel would need about 7 flop per byte, more than half of the fp32 peak at
// full HBM rate.
//
// Every mbarrier wait is bounded: after kSpinLimit polls the waiter records a status word in the
// workspace, raises a CTA-wide abort flag and the kernel drains and returns.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace aircache {

namespace {

struct DecodeParams {
    const uint16_t *q;       // [L*B, Hq, D]
    float *out;              // [L*B, Hq, D]
    int32_t *plan_memo;    // [kMaxDecodeCtas][kPlanMemoInts] kept plans of the head-split launches, or null
    const int64_t *offsets;  // [L*B + 1]
    const int32_t *lens;     // [L*B]
    int32_t *tickets;        // [L*B] partials of the region written so far; zero between calls
    float *partials;         // [2 * CTAs][Hq * (D + 2)]
    uint32_t *status;
    int n_regions, Hq, G;
    const uint16_t *k_new, *v_new;   // Eq. 2: [L*B, Hkv, D] K and V of the token appended by this call, or NULL
    uint16_t *k_cache, *v_cache;     // the ragged cache, for the appended rows
    int32_t *lens_rw;                // lens, bumped by the last CTA when a token is appended
    int32_t *done_ticket;            // CTAs finished (append only); zero between calls
    int kv_heads;                    // KV heads of the cache
    int hs;                  // head-split mode: KV heads per region (items are (region, head) pairs); else 1
    float sl2;               // scale * log2(e)
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers (mbarrier, TMA: ptx.cuh)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// transposes an 8x8 matrix of 16-bit elements held one row (two elements per thread) per four lanes
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void consumer_bar(int n_threads) {
    asm volatile("bar.sync 1, %0;" ::"r"(n_threads) : "memory");
}
__device__ __forceinline__ float exp2_or_zero(float m, float m_new) {
    return m == -INFINITY ? 0.f : fast_exp2(m - m_new);
}

template <int D, int HKV, bool G_HI, bool HS>
struct DecodeCfg {
    static constexpr int NROW = G_HI ? 2 : 1;        // accumulator row groups in use (heads 0-7, heads 8-15)
    static constexpr int KSPLIT = HS ? 8 : ((8 / HKV) > 4 ? 4 : (8 / HKV));
    static constexpr int CH = 16 * KSPLIT;           // rows per unit
    static constexpr int CH_LOG2 = KSPLIT == 8 ? 7 : (KSPLIT == 4 ? 6 : (KSPLIT == 2 ? 5 : 4));
    static_assert((1 << CH_LOG2) == CH, "unit rows are a power of two");
    static constexpr int NCW = HKV * KSPLIT;         // consumer warps
    static constexpr int THREADS = (NCW + 1) * 32;
    static constexpr int HALVES = D / 64;
    static constexpr int SUBTILE = CH * 128;         // bytes of one (head, half) box
    static constexpr int KV_BYTES = HKV * HALVES * SUBTILE;
    static constexpr int STAGE_BYTES = 2 * KV_BYTES;
    static constexpr int MERGE_FLOATS_PER_WARP = 32 * (NROW * (D / 4 + 4));
    static constexpr int MERGE_SLOTS = KSPLIT / 2;     // tree merge: the upper half of the warps hands over to the lower
    static constexpr int MERGE_BYTES = HKV * MERGE_SLOTS * MERGE_FLOATS_PER_WARP * 4;
    // the prologue's scan scratch lives in the same bytes as the merge buffer (used before the first flush)
    static constexpr int SCAN_BYTES = THREADS * 4;
    static constexpr int MERGE_STAGE_BYTES = 16384;            // weights [partials][Hq] of the final merge
    static constexpr int SCRATCH_MIN = SCAN_BYTES > MERGE_STAGE_BYTES ? SCAN_BYTES : MERGE_STAGE_BYTES;
    static constexpr int SCRATCH_BYTES = ((MERGE_BYTES > SCRATCH_MIN ? MERGE_BYTES : SCRATCH_MIN) + 15) / 16 * 16;
    // (head-split launches have at most kMaxDecodeCtas items)
    static constexpr int TABLE_ENTRIES = HS ? kMaxDecodeCtas : kMaxRegions;
    static constexpr int PLAN_BYTES = (TABLE_ENTRIES + 2) * 4;   // unit prefix
    static constexpr int OFFS_BYTES = TABLE_ENTRIES * 4;         // first row of every region
    // ring depth: what fits beside the scratch and the tables in the 227 KB a CTA may use (1.5 KB are left
    // for static shared memory, 1 KB for the alignment slack), at most 4 stages
    static constexpr int FIT = (232448 - 1536 - 1024 - SCRATCH_BYTES - PLAN_BYTES - OFFS_BYTES - 256) / STAGE_BYTES;
    static constexpr int NSTAGE = FIT > 4 ? 4 : FIT;
    static_assert(NSTAGE >= 2, "decode pipeline needs two stages");
    static constexpr int SMEM_BYTES = 1024 + NSTAGE * STAGE_BYTES + SCRATCH_BYTES + PLAN_BYTES + OFFS_BYTES + 256;
};

// a / b for a >= 0, b > 0, through the fp32 divider when both are below 2^23 (an integer division by a run-time
// divisor costs several hundred cycles of the prologue otherwise)
__device__ __forceinline__ int small_div(int a, int b) {
    if (a >= (1 << 23) || b >= (1 << 23)) return a / b;
    int q = (int)__fdividef((float)a, (float)b);
    if (q * b > a) --q;
    if ((q + 1) * b <= a) ++q;
    return q;
}

// The same for operands known to be below 2^23: no integer-division fallback to schedule around.
__device__ __forceinline__ int small_div_unchecked(int a, int b) {
    int q = (int)__fdividef((float)a, (float)b);
    if (q * b > a) --q;
    if ((q + 1) * b <= a) ++q;
    return q;
}

// largest r with P[r] <= u (P non-decreasing, P[0] = 0, u < P[n])
__device__ __forceinline__ int find_region(const int *P, int n, int u) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (P[mid] <= u) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// The region-aligned cut for few regions, planned by one warp in registers (all warps of a CTA call this and
// get the same answer).  With no more items than CTAs a CTA needs five numbers of the cut: its item, the
// item's units and rows, its piece and the piece count.  Each lane takes rpl consecutive regions; sums and the
// prefix of the piece counts go through warp primitives, so no warp waits for another, no table is built, and
// the producer can issue its first loads one global round trip after the kernel may read memory.
// Returns 0 when the tables have to decide (empty regions, too many regions, no fitting cut), 2 when this CTA
// has no piece, 1 with plan = {item, rows of the item, first unit, end unit} and the item's table entries
// stored if `store` is set (units counted from the item's first one).
// With BALANCED set (the by-region kernels) a cut that does not fit is no reason to give up: the warp then
// writes the unit prefix and first row of every region into the shared tables itself (every warp writes the
// same values, none waits for another) and returns 3 with plan = {-1, total units, first unit, end unit} of the
// balanced schedule, CTA c taking units [c * upc, (c + 1) * upc) of the global list; `force_balanced` makes the
// rehearsal take that way.  RPL = regions a lane may hold.
//
// `memo` (may be null) points at this CTA's kPlanMemoInts words of global memory, zero before their first use.
// The cut depends on the regions' unit counts alone, and those change only every CH appended tokens, so the CTA
// keeps the unit counts it planned for and the outcome; when the counts read now equal the kept ones, the
// outcome is taken from there and the arithmetic (about a microsecond of dependent steps) is skipped.  A CTA
// reads and writes only its own words, and only after the kernel's dependency wait (the rehearsal passes words
// in shared memory, hence the plain loads).
//   words 0..4: n, hs, n_ctas, ch_log2, outcome (1 or 2);  8..13: item, first unit, end unit, units, first CTA of the
//   item, pieces;  14: region;  16..: unit count of every region
template <int RPL, bool BALANCED>
__device__ __forceinline__ int plan_few_regions(const int32_t *lens, const int64_t *offsets, int n, int hs, int n_ctas,
                                                int ch_log2, int c, bool store, bool force_balanced, int32_t *memo,
                                                int *s_P, int *s_off, int *s_Q, int4 *plan) {
    const int lane = threadIdx.x & 31;
    const int nr = n / hs;
    if (n > n_ctas || nr <= 0 || nr > 32 * RPL) return 0;
    const int rpl = (nr + 31) >> 5;
    int un[RPL], ln[RPL], of[RPL], kept_un[RPL];
    bool nonempty = true;
    int tot = 0;
    int memo_word = 0;
#pragma unroll
    for (int j = 0; j < RPL; ++j) {
        un[j] = ln[j] = of[j] = kept_un[j] = 0;
        const int reg = lane * rpl + j;
        if (j < rpl && reg < nr) {
            ln[j] = max(lens[reg], 0);
            of[j] = (int)offsets[reg];
            if (memo) kept_un[j] = memo[16 + reg];
        }
    }
    if (memo && lane < 16) memo_word = memo[lane];
#pragma unroll
    for (int j = 0; j < RPL; ++j) {
        const int reg = lane * rpl + j;
        if (j < rpl && reg < nr) {
            un[j] = (ln[j] + (1 << ch_log2) - 1) >> ch_log2;
            nonempty = nonempty && un[j] > 0;
            tot += un[j];
        }
    }
    if (memo) {
        const int expect = lane == 0 ? n : (lane == 1 ? hs : (lane == 2 ? n_ctas : ch_log2));
        bool same = lane >= 4 || memo_word == expect;
        if (lane == 4) same = memo_word == 1 || memo_word == 2;
#pragma unroll
        for (int j = 0; j < RPL; ++j) same = same && kept_un[j] == un[j];   // (both zero past the last region)
        if (__all_sync(0xffffffffu, same)) {
            if (__shfl_sync(0xffffffffu, memo_word, 4) == 2) return 2;
            const int item = __shfl_sync(0xffffffffu, memo_word, 8);
            const int first_unit = __shfl_sync(0xffffffffu, memo_word, 9);
            const int end_unit = __shfl_sync(0xffffffffu, memo_word, 10);
            const int units = __shfl_sync(0xffffffffu, memo_word, 11);
            const int q_first = __shfl_sync(0xffffffffu, memo_word, 12);
            const int pieces = __shfl_sync(0xffffffffu, memo_word, 13);
            const int reg = __shfl_sync(0xffffffffu, memo_word, 14);
            // rows and first row of that region as read now: they change with every appended token
            const int src = small_div_unchecked(reg, rpl), slot = reg - src * rpl;
            int rows = 0, first_row = 0;
#pragma unroll
            for (int j = 0; j < RPL; ++j)
                if (j == slot) { rows = ln[j]; first_row = of[j]; }
            rows = __shfl_sync(0xffffffffu, rows, src);
            first_row = __shfl_sync(0xffffffffu, first_row, src);
            *plan = make_int4(item, rows, first_unit, end_unit);
            if (lane == 0 && store) {
                s_P[item] = 0;
                s_P[item + 1] = units;
                s_off[item] = first_row;
                s_Q[item] = q_first;
                s_Q[item + 1] = q_first + pieces;
            }
            __syncwarp();
            return 1;
        }
    }
    // one warp of the CTA records what is planned below
    const bool record = memo != nullptr && store && threadIdx.x < 32;
    tot = __reduce_add_sync(0xffffffffu, tot);   // units of one head's items
    // (the bound keeps every dividend below 2^23 and units * pieces below 2^31)
    if (!__all_sync(0xffffffffu, nonempty) || tot >= (1 << 22) / hs) return 0;
    const int upc = max(1, small_div_unchecked(tot * hs + n_ctas - 1, n_ctas));
    // An item of at most `cap` units stays whole; a longer one is cut into pieces of at most cap - kSplitCost
    // units, because its CTAs also publish and merge partials, which takes them about as long as that many
    // units: the whole items then end the kernel, not the pieces.  Tried in turn: cap = upc + 1, upc + 2, and
    // upc + 2 with plain pieces of at most cap units (the one that needs the fewest CTAs).
    constexpr int kSplitCost = 2;
    const int cap0 = upc + 1, cap1 = upc + 2;
    const int cut0 = max(1, cap0 - kSplitCost), cut1 = max(1, cap1 - kSplitCost);
    int sum0 = 0, sum1 = 0, sum2 = 0;
    int pc0[RPL], pc1[RPL], pc2[RPL];
#pragma unroll
    for (int j = 0; j < RPL; ++j) {
        pc0[j] = pc1[j] = pc2[j] = 0;
        if (j < rpl) {
            sum0 += pc0[j] = un[j] <= cap0 ? 1 : small_div_unchecked(un[j] + cut0 - 1, cut0);
            sum1 += pc1[j] = un[j] <= cap1 ? 1 : small_div_unchecked(un[j] + cut1 - 1, cut1);
            sum2 += pc2[j] = small_div_unchecked(un[j] + cap1 - 1, cap1);
        }
    }
    sum0 = __reduce_add_sync(0xffffffffu, sum0);
    sum1 = __reduce_add_sync(0xffffffffu, sum1);
    sum2 = __reduce_add_sync(0xffffffffu, sum2);
    const int lim = n_ctas / hs;   // the sums count pieces per head
    if ((sum0 > lim && sum1 > lim && sum2 > lim) || (BALANCED && force_balanced)) {
        if (!BALANCED) return 0;
        // balanced schedule: exclusive prefix of the unit counts, written by every lane for its regions
        int mine_units = 0;
#pragma unroll
        for (int j = 0; j < RPL; ++j) mine_units += un[j];
        int incl_units = mine_units;
#pragma unroll
        for (int sh = 1; sh < 32; sh <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl_units, sh);
            if (lane >= sh) incl_units += o;
        }
        if (store) {
            int before = incl_units - mine_units;
#pragma unroll
            for (int j = 0; j < RPL; ++j) {
                const int reg = lane * rpl + j;
                if (j < rpl && reg < nr) {
                    s_P[reg] = before;
                    s_off[reg] = of[j];
                    before += un[j];
                    if (reg == nr - 1) s_P[nr] = before;
                }
            }
        }
        __syncwarp();
        const int u_first = min(tot, c * upc);
        *plan = make_int4(-1, tot, u_first, min(tot, u_first + upc));
        return 3;
    }
    int pc[RPL];
    int mine = 0;
#pragma unroll
    for (int j = 0; j < RPL; ++j) {
        pc[j] = sum0 <= lim ? pc0[j] : (sum1 <= lim ? pc1[j] : pc2[j]);
        mine += pc[j];
    }
    int incl = mine;
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, sh);
        if (lane >= sh) incl += o;
    }
    // the region whose CTAs [first * hs, (first + pieces) * hs) include this one
    int run = incl - mine;
    int v_reg = -1, v_first = 0, v_pc = 0, v_un = 0, v_ln = 0, v_of = 0;
#pragma unroll
    for (int j = 0; j < RPL; ++j) {
        if (j < rpl) {
            if (c >= run * hs && c < (run + pc[j]) * hs) {
                v_reg = lane * rpl + j; v_first = run; v_pc = pc[j]; v_un = un[j]; v_ln = ln[j]; v_of = of[j];
            }
            run += pc[j];
        }
    }
    const unsigned ball = __ballot_sync(0xffffffffu, v_reg >= 0);
    if (record) {
#pragma unroll
        for (int j = 0; j < RPL; ++j)
            if (j < rpl && lane * rpl + j < nr) __stcg(memo + 16 + lane * rpl + j, un[j]);
    }
    if (ball == 0) {   // more CTAs than pieces
        if (record && lane < 5) __stcg(memo + lane, lane == 0 ? n : (lane == 1 ? hs : (lane == 2 ? n_ctas : (lane == 3 ? ch_log2 : 2))));
        return 2;
    }
    const int src = __ffs(ball) - 1;
    v_reg = __shfl_sync(0xffffffffu, v_reg, src);
    v_first = __shfl_sync(0xffffffffu, v_first, src);
    v_pc = __shfl_sync(0xffffffffu, v_pc, src);
    v_un = __shfl_sync(0xffffffffu, v_un, src);
    v_ln = __shfl_sync(0xffffffffu, v_ln, src);
    v_of = __shfl_sync(0xffffffffu, v_of, src);
    const int rel = c - v_first * hs;
    int h = rel, j = 0, first_unit = 0, end_unit = v_un;
    if (v_pc > 1) {   // (most items are one piece: no division then)
        h = small_div_unchecked(rel, v_pc);
        j = rel - h * v_pc;
        // no overflow: the units of all regions together are below 2^22, the pieces at most 256
        first_unit = small_div(v_un * j, v_pc);
        end_unit = small_div(v_un * (j + 1), v_pc);
    }
    const int item = v_reg * hs + h;
    *plan = make_int4(item, v_ln, first_unit, end_unit);
    if (lane == 0 && store) {
        s_P[item] = 0;
        s_P[item + 1] = v_un;
        s_off[item] = v_of;
        s_Q[item] = v_first * hs + h * v_pc;
        s_Q[item + 1] = v_first * hs + (h + 1) * v_pc;
    }
    if (record && lane < 16) {
        const int head[5] = {n, hs, n_ctas, ch_log2, 1};
        const int body[7] = {item, first_unit, end_unit, v_un, v_first * hs + h * v_pc, v_pc, v_reg};
        int w = 0;
#pragma unroll
        for (int i = 0; i < 5; ++i) if (lane == i) w = head[i];
#pragma unroll
        for (int i = 0; i < 7; ++i) if (lane == 8 + i) w = body[i];
        __stcg(memo + lane, w);
    }
    __syncwarp();
    return 1;
}

template <int D, int HKV, bool G_HI, bool HS>
__global__ void __launch_bounds__(DecodeCfg<D, HKV, G_HI, HS>::THREADS, 1)
decode_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, DecodeParams p) {
    using C = DecodeCfg<D, HKV, G_HI, HS>;
    constexpr int KSPLIT = C::KSPLIT, CH = C::CH, NCW = C::NCW, NROW = C::NROW, kStages = C::NSTAGE;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *s_stage = smem;
    float *s_merge = reinterpret_cast<float *>(smem + kStages * C::STAGE_BYTES);
    int *s_part = reinterpret_cast<int *>(s_merge);   // scan scratch of the prologue, same bytes
    int *s_P = reinterpret_cast<int *>(smem + kStages * C::STAGE_BYTES + C::SCRATCH_BYTES);
    int *s_off = reinterpret_cast<int *>(smem + kStages * C::STAGE_BYTES + C::SCRATCH_BYTES + C::PLAN_BYTES);
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem + kStages * C::STAGE_BYTES + C::SCRATCH_BYTES + C::PLAN_BYTES +
                                                   C::OFFS_BYTES);
    __shared__ int s_Q[kMaxDecodeCtas + 1];   // region-aligned mode: first CTA of every region
    __shared__ int s_abort;
    __shared__ int s_last;
    __shared__ int s_aligned;

    const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
    const int n = p.n_regions;   // items: regions, or (region, KV head) pairs in head-split mode
    const int hs = HS ? p.hs : 1;
    const int n_ctas = (int)gridDim.x;
    // Programmatic dependent launch: the next kernel in the stream may be scheduled as soon as SMs free up,
    // and this one does everything that reads no global memory before it waits for its predecessor.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (wid == NCW && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_v)) : "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&s_bar[s]), 1);             // full: the producer's expect_tx arrival
            mbar_init(smem_u32(&s_bar[kStages + s]), NCW);  // empty: one arrival per consumer warp
        }
        mbar_init(smem_u32(&s_bar[2 * kStages]), 1);        // partials staged for the final merge
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s_abort = 0;
    }
    // made-up region lengths (one unit each), first rows and a kept plan that matches them, for the rehearsal of
    // the register plan below
    // (head-split launches have at least two heads per region; with more than 64 regions the by-region kernels
    // measured no faster through the registers than through the shared tables)
    constexpr int kPlanRpl = HS ? kPlanRegionsPerLane : 2;
    constexpr int kPlanRegions = 32 * kPlanRpl;
    int32_t *rehearsal_lens = reinterpret_cast<int32_t *>(s_part);
    int64_t *rehearsal_offsets = reinterpret_cast<int64_t *>(s_part + kPlanRegions);
    int32_t *rehearsal_memo = reinterpret_cast<int32_t *>(s_part + 3 * kPlanRegions);
    static_assert((3 * kPlanRegions + kPlanMemoInts) * 4 <= C::SCRATCH_BYTES, "rehearsal inputs fit the scratch area");
    for (int i = tid; i < kPlanRegions; i += C::THREADS) {
        rehearsal_lens[i] = CH;
        rehearsal_offsets[i] = 0;
        rehearsal_memo[16 + i] = i < n / hs ? 1 : 0;
        if (i < 16) {
            // n, hs, n_ctas, log2 CH, outcome 1 | item 0 = units [0, 1) of 1, first CTA 0, one piece, region 0
            const int words[16] = {n, hs, n_ctas, C::CH_LOG2, 1, 0, 0, 0, 0, 0, 1, 1, 0, 1, 0, 0};
            int w = 0;
#pragma unroll
            for (int k = 0; k < 16; ++k) if (i == k) w = words[k];
            rehearsal_memo[i] = w;
        }
    }
    // Ask for the lines the plan will read first (lengths, first rows, this CTA's kept plan) to be brought into
    // L2 meanwhile: a prefetch consumes no value, so it may precede the dependency wait, and the loads after the
    // wait then find L2 instead of HBM.
    if (wid == NCW) {
        const int n_reg = n / hs;
        const char *lines[3] = {reinterpret_cast<const char *>(p.lens), reinterpret_cast<const char *>(p.offsets),
                                reinterpret_cast<const char *>(p.plan_memo ? p.plan_memo + (size_t)blockIdx.x * kPlanMemoInts
                                                                           : nullptr)};
        const int bytes[3] = {n_reg * 4, n_reg * 8, HS || n_reg <= 64 ? (16 + n_reg) * 4 : 0};
#pragma unroll
        for (int a = 0; a < 3; ++a)
            if (lines[a] != nullptr && lane * 128 < bytes[a] && lane < 16)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(lines[a] + lane * 128) : "memory");
    }
    // The barriers are initialised before any warp goes its own way (nothing above read global memory).
    __syncthreads();

    int total = 0, upc = 1;
    bool aligned = false;
    int u0 = 0, u1 = 0;
    int r_own = -1, len_own = 0;   // the one item of this CTA and its rows, when the register plan found them
    // Eq. 2 bookkeeping: the CTA that finishes last adds the appended token to every region's length
    auto finish = [&](bool all_threads) {
        if (p.k_new == nullptr) return;
        if (tid == 0) {
            __threadfence();
            s_last = atomicAdd(p.done_ticket, 1) == n_ctas - 1;
            if (s_last) *p.done_ticket = 0;
        }
        if (all_threads) __syncthreads(); else consumer_bar(NCW * 32);
        if (s_last)
            for (int i = tid; i < n / hs; i += (all_threads ? C::THREADS : NCW * 32)) p.lens_rw[i] += 1;
    };

    // ---- few regions: every warp plans for itself, in registers; otherwise the tables below decide ----
    bool planned = false;
    {
        // The plan runs twice through the same instructions: first on the made-up lengths in shared memory (with a
        // kept plan that matches them, the usual case of a head-split launch; the by-region kernels rehearse the
        // balanced schedule), while the kernel may not read global memory yet, then on the real ones.  A kernel's
        // first pass through a stretch of code waits for its instructions line by line, which for this serial
        // stretch costs more than its arithmetic; the rehearsal moves that wait in front of the dependency wait,
        // where the CTA idles.
        int4 plan;
        int rc = 0;
        const bool few = n <= n_ctas && n / hs <= kPlanRegions;   // else only the wait remains of the loop below
#pragma unroll 1
        for (int pass = few ? 0 : 1; pass < 2; ++pass) {
            if (pass) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                if (!few) break;
            }
            rc = plan_few_regions<kPlanRpl, !HS>(
                pass ? p.lens : rehearsal_lens, pass ? p.offsets : rehearsal_offsets, n, hs, n_ctas, C::CH_LOG2,
                (int)blockIdx.x, pass != 0, pass == 0,
                !p.plan_memo ? nullptr
                             : (pass ? p.plan_memo + (size_t)blockIdx.x * kPlanMemoInts : (HS ? rehearsal_memo : nullptr)),
                s_P, s_off, s_Q, &plan);
        }
        if (rc == 2) { finish(true); return; }
        if (rc == 1) {
            planned = aligned = true;
            r_own = plan.x; len_own = plan.y; u0 = plan.z; u1 = plan.w;
        } else if (rc == 3) {
            planned = true;
            total = plan.y; u0 = plan.z; u1 = plan.w;
            upc = max(1, small_div(total + n_ctas - 1, n_ctas));
        }
    }
    if (!planned) {
        // ---- unit prefix and first row of all regions (every CTA computes the same tables) ----
        {
            const int per = (n + C::THREADS - 1) / C::THREADS;
            const int i0 = min(n, tid * per), i1 = min(n, i0 + per);
            int local = 0;
            for (int i = i0; i < i1; ++i) {
                local += (max(p.lens[i / hs], 0) + CH - 1) / CH;
                s_off[i] = (int)p.offsets[i / hs];
            }
            s_part[tid] = local;
            __syncthreads();
            if (wid == 0) {
                // warp 0 turns s_part into an exclusive prefix
                constexpr int PER_LANE = (C::THREADS + 31) / 32;
                int sum = 0;
                for (int j = 0; j < PER_LANE; ++j) {
                    const int idx = lane * PER_LANE + j;
                    if (idx < C::THREADS) sum += s_part[idx];
                }
                int incl = sum;
    #pragma unroll
                for (int sh = 1; sh < 32; sh <<= 1) {
                    const int o = __shfl_up_sync(0xffffffffu, incl, sh);
                    if (lane >= sh) incl += o;
                }
                int run = incl - sum;
                for (int j = 0; j < PER_LANE; ++j) {
                    const int idx = lane * PER_LANE + j;
                    if (idx < C::THREADS) { const int v = s_part[idx]; s_part[idx] = run; run += v; }
                }
            }
            __syncthreads();
            int run = s_part[tid];
            for (int i = i0; i < i1; ++i) {
                s_P[i] = run;
                run += (max(p.lens[i / hs], 0) + CH - 1) / CH;
            }
            if (i1 == n && i0 < n) s_P[n] = run;
            if (n == 0 && tid == 0) s_P[0] = 0;
            __syncthreads();
        }
        total = s_P[n];
        upc = max(1, small_div(total + n_ctas - 1, n_ctas));

        // ---- schedule.  Balanced mode: CTA c takes units [c * upc, (c+1) * upc) of the global list.
        // Region-aligned mode (few regions, each cut into pieces of at most upc units, if that needs no more
        // CTAs than there are): every CTA works on one region only, so it reloads no query and flushes once.
        if (wid == 0) {
            // Aligned pieces of at most upc_a units: upc_a is the smallest of upc, upc + 1, upc + 2 for which the
            // pieces need no more CTAs than the grid has (two more units on the longest CTA cost less than a
            // second flush and merge).  All items of a region have the same unit count, so the sums run over
            // regions; the three candidates are evaluated together.  Rolled loops: this runs once.
            // With more than half as many regions as CTAs an aligned cut would have to leave most regions
            // whole, which pieces of about total / CTAs units cannot do unless the regions are tiny: the search
            // is skipped there (it costs over a microsecond on a hundred regions) and the schedule is balanced.
            const bool few = n <= n_ctas && total > 0 && !(2 * n > n_ctas && upc > 4);
            const int nr = n / hs;
            int sum0 = 0, sum1 = 0, sum2 = 0;
    #pragma unroll 1
            for (int r = lane; few && r < nr; r += 32) {
                const int u = s_P[r * hs + 1] - s_P[r * hs];
                sum0 += small_div(u + upc - 1, upc);
                sum1 += small_div(u + upc, upc + 1);
                sum2 += small_div(u + upc + 1, upc + 2);
            }
    #pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) {
                sum0 += __shfl_xor_sync(0xffffffffu, sum0, sh);
                sum1 += __shfl_xor_sync(0xffffffffu, sum1, sh);
                sum2 += __shfl_xor_sync(0xffffffffu, sum2, sh);
            }
            const int lim = n_ctas / hs;   // the sums count pieces per head
            const bool found = few && (sum0 <= lim || sum1 <= lim || sum2 <= lim);
            const int upc_a = sum0 <= lim ? upc : (sum1 <= lim ? upc + 1 : upc + 2);
            int carry = 0;
    #pragma unroll 1
            for (int base = 0; found && base <= nr; base += 32) {
                const int r = base + lane;
                const int v = r < nr ? small_div(s_P[r * hs + 1] - s_P[r * hs] + upc_a - 1, upc_a) : 0;
                int incl = v;
    #pragma unroll
                for (int sh = 1; sh < 32; sh <<= 1) {
                    const int o = __shfl_up_sync(0xffffffffu, incl, sh);
                    if (lane >= sh) incl += o;
                }
                if (r < nr) {
    #pragma unroll 1
                    for (int h = 0; h < hs; ++h) s_Q[r * hs + h] = (carry + incl - v) * hs + h * v;
                } else if (r == nr) {
                    s_Q[n] = (carry + incl - v) * hs;
                }
                carry += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (lane == 0) s_aligned = found ? 1 : 0;
        }
        __syncthreads();
        aligned = s_aligned != 0;

        // an item without rows yields zeros - or, when a token is appended, that token's value (softmax over one key)
        for (int r = blockIdx.x; r < n; r += n_ctas) {
            if (s_P[r + 1] != s_P[r]) continue;
            const int reg = r / hs;
            for (int i = tid; i < p.Hq * D; i += C::THREADS) {
                float v = 0.f;
                if (p.k_new) {
                    const int kvh = HS ? r % hs : (i / D) / p.G;
                    v = bf16_to_f32(p.v_new[((int64_t)reg * p.kv_heads + kvh) * D + i % D]);
                }
                p.out[(int64_t)r * p.Hq * D + i] = v;
            }
            if (p.k_new) {
                const int heads = HS ? 1 : p.kv_heads, h0 = HS ? r % hs : 0;
                for (int i = tid; i < heads * D; i += C::THREADS) {
                    const int64_t src = ((int64_t)reg * p.kv_heads + h0) * D + i;
                    const int64_t dst = ((int64_t)s_off[r] * p.kv_heads + h0) * D + i;
                    p.k_cache[dst] = p.k_new[src];
                    p.v_cache[dst] = p.v_new[src];
                }
            }
        }
        if (aligned) {
            const int c = (int)blockIdx.x;
            if (c >= s_Q[n]) { finish(true); return; }
            const int r = find_region(s_Q, n, c);      // largest r with s_Q[r] <= c: the region this CTA cuts
            const int pieces = s_Q[r + 1] - s_Q[r], j = c - s_Q[r], units = s_P[r + 1] - s_P[r];
            u0 = s_P[r] + small_div(units * j, pieces);          // units * pieces < 2^24: both are at most a few thousand
            u1 = s_P[r] + small_div(units * (j + 1), pieces);
        } else {
            u0 = min(total, (int)blockIdx.x * upc);
            u1 = min(total, u0 + upc);
        }
    }
    if (u0 >= u1) { finish(true); return; }
    // CTAs that hold a piece of region r, and the partial slot CTA c uses for it
    auto span_of = [&](int r, int &c0, int &c1) {
        if (aligned) { c0 = s_Q[r]; c1 = s_Q[r + 1] - 1; }
        else { c0 = s_P[r] / upc; c1 = (s_P[r + 1] - 1) / upc; }
    };
    auto slot_of = [&](int c, int r) { return aligned ? 2 * c : 2 * c + ((s_P[r] <= c * upc) ? 0 : 1); };

    if (wid == NCW) {
        // =============================== producer warp ===============================
        if (lane == 0) {
            int r = r_own >= 0 ? r_own : find_region(s_P, n, u0);
            int row_base = s_off[r];
            int it = 0;
            bool ok = true;
            for (int u = u0; u < u1 && ok; ++u, ++it) {
                if (u >= s_P[r + 1]) {
                    while (u >= s_P[r + 1]) ++r;
                    row_base = s_off[r];
                }
                const int s = it % kStages;
                if (it >= kStages)
                    ok = mbar_wait(smem_u32(&s_bar[kStages + s]), ((it / kStages) & 1) ^ 1, &s_abort, p.status, 1);
                if (!ok) break;
                const int row0 = row_base + (u - s_P[r]) * CH;
                const uint32_t full = smem_u32(&s_bar[s]);
                mbar_expect_tx(full, C::STAGE_BYTES);
                const uint32_t dst = smem_u32(s_stage + s * C::STAGE_BYTES);
#pragma unroll
                for (int g = 0; g < HKV; ++g) {
#pragma unroll
                    for (int hf = 0; hf < C::HALVES; ++hf) {
                        const uint32_t off = (g * C::HALVES + hf) * C::SUBTILE;
                        const int head = HS ? r % hs : g;
                        tma_load_3d(dst + off, &tm_k, hf * 64, head, row0, full);
                        tma_load_3d(dst + C::KV_BYTES + off, &tm_v, hf * 64, head, row0, full);
                    }
                }
            }
            if (!ok) {
                // drain: wait (bounded) for the loads already in flight before the CTA may exit
                for (int j = max(0, it - kStages); j < it; ++j) {
                    const uint32_t bar = smem_u32(&s_bar[j % kStages]);
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_test(bar, (j / kStages) & 1); ++i) __nanosleep(40);
                }
            }
        }
        if (p.k_new != nullptr && r_own >= 0) {
            // Eq. 2 bookkeeping off the critical path: a CTA planned in registers needs lens no more (its row
            // count sits in registers), so its idle producer draws the ticket now instead of the consumers at
            // the end; lens is bumped by whoever draws the last ticket, when no CTA will read it again.
            int last = 0;
            if (lane == 0) {
                last = atomicAdd(p.done_ticket, 1) == n_ctas - 1;
                if (last) *p.done_ticket = 0;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last)
                for (int i = lane; i < n / hs; i += 32) p.lens_rw[i] += 1;
        }
        return;
    }

    // ================================= consumer warps =================================
    const int g = wid / KSPLIT, ks = wid % KSPLIT;
    const int gid = lane >> 2, t = lane & 3;
    const int G = p.G;

    int len = 0;      // rows of the item being processed
    // The block's products are taken transposed - S^T = K Q^T and O^T = V^T P^T - so that the 16 rows of the tensor
    // core tile are keys (respectively channels) and its 8 columns the query heads of the KV group: a group of up
    // to 8 heads fills one column tile, where heads as rows would leave half of a 16-row tile empty.
    // A thread holds, per column tile nt: heads nt*8 + 2t, +1 of keys gid, gid+8 (S^T) or of channels
    // mt*16 + gid, +8 (O^T).
    uint32_t qb[NROW][D / 16][2];     // Q^T as the right-hand operand: head nt*8 + gid, channels kk*16 + 2t.., +8
    float oacc[NROW][D / 16][4];
    float m_run[NROW][2], l_run[NROW][2];   // per head 2t, 2t+1; l_run is this thread's share until the flush

    auto load_q = [&](int r) {
#pragma unroll
        for (int nt = 0; nt < NROW; ++nt) {
            const int hl = nt * 8 + gid;
            const bool valid = hl < G;
            const uint16_t *qp = p.q + ((int64_t)r * p.Hq + g * G + (valid ? hl : 0)) * D;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                qb[nt][kk][0] = valid ? __ldg(reinterpret_cast<const uint32_t *>(qp + kk * 16 + 2 * t)) : 0u;
                qb[nt][kk][1] = valid ? __ldg(reinterpret_cast<const uint32_t *>(qp + kk * 16 + 8 + 2 * t)) : 0u;
            }
#pragma unroll
            for (int mt = 0; mt < D / 16; ++mt) oacc[nt][mt][0] = oacc[nt][mt][1] = oacc[nt][mt][2] = oacc[nt][mt][3] = 0.f;
            m_run[nt][0] = m_run[nt][1] = -INFINITY;
            l_run[nt][0] = l_run[nt][1] = 0.f;
        }
    };

    // One block of 16 keys at rows blk_row0.. of a (K, V) tile in shared memory; the block's first key is row j0
    // of the region, which has len rows.  sub_stride is the distance between the two 64-channel halves.
    auto process_block = [&](uint32_t k_base, uint32_t v_base, uint32_t sub_stride, int blk_row0, int j0, int len) {
        const int mi = lane >> 3, rr = lane & 7;

        // ---- S^T = K Q^T for 16 keys; two accumulators per tile halve the chain of dependent MMAs ----
        float sacc[NROW][2][4];
#pragma unroll
        for (int nt = 0; nt < NROW; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) sacc[nt][e][0] = sacc[nt][e][1] = sacc[nt][e][2] = sacc[nt][e][3] = 0.f;
        {
            const int row = blk_row0 + (mi & 1) * 8 + rr;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const int hf = kk >> 2, chunk = ((kk & 3) << 1) + (mi >> 1);
                uint32_t a[4];   // keys 0-7 / 8-15 of channels kk*16.., then of channels kk*16 + 8..
                ldmatrix_x4(a, k_base + hf * sub_stride + row * 128 + ((chunk ^ (row & 7)) << 4));
#pragma unroll
                for (int nt = 0; nt < NROW; ++nt)
                    mma_bf16_16816(sacc[nt][kk & 1], a[0], a[1], a[2], a[3], qb[nt][kk][0], qb[nt][kk][1]);
            }
        }
        // ---- online softmax (exp2 domain) ----
        const bool tail = j0 + 16 > len;
        const bool dead_lo = tail && j0 + gid >= len, dead_hi = tail && j0 + gid + 8 >= len;
        uint32_t pa[NROW][2], pb[NROW][2];  // P^T = pa + pb (bf16 head and bf16 remainder), as right-hand operands
        bool rescale = false;
        float corr[NROW][2];
#pragma unroll
        for (int nt = 0; nt < NROW; ++nt) {
            float x[4];   // keys gid (heads 2t, 2t+1), gid + 8 (heads 2t, 2t+1)
#pragma unroll
            for (int i = 0; i < 4; ++i) x[i] = (sacc[nt][0][i] + sacc[nt][1][i]) * p.sl2;
            if (dead_lo) x[0] = x[1] = -INFINITY;
            if (dead_hi) x[2] = x[3] = -INFINITY;
            float mx0 = fmaxf(x[0], x[2]), mx1 = fmaxf(x[1], x[3]);
#pragma unroll
            for (int sh = 4; sh < 32; sh <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
            }
            const float mn0 = fmaxf(m_run[nt][0], mx0), mn1 = fmaxf(m_run[nt][1], mx1);  // finite: key j0 is valid
            corr[nt][0] = exp2_or_zero(m_run[nt][0], mn0);
            corr[nt][1] = exp2_or_zero(m_run[nt][1], mn1);
            rescale = rescale || corr[nt][0] != 1.f || corr[nt][1] != 1.f;
            m_run[nt][0] = mn0;
            m_run[nt][1] = mn1;
            const float e0 = fast_exp2(x[0] - mn0), e1 = fast_exp2(x[1] - mn1);
            const float e2 = fast_exp2(x[2] - mn0), e3 = fast_exp2(x[3] - mn1);
            const uint32_t a_lo = pack_bf16(e0, e1), a_hi = pack_bf16(e2, e3);   // key gid, key gid + 8
            const uint32_t b_lo = pack_bf16(e0 - bf16lo(a_lo), e1 - bf16hi(a_lo));
            const uint32_t b_hi = pack_bf16(e2 - bf16lo(a_hi), e3 - bf16hi(a_hi));
            l_run[nt][0] = l_run[nt][0] * corr[nt][0] + (e0 + e2);
            l_run[nt][1] = l_run[nt][1] * corr[nt][1] + (e1 + e3);
            // (key gid; heads 2t, 2t+1) -> (keys 2t, 2t+1; head gid): the operand layout of the second product
            pa[nt][0] = movmatrix_trans(a_lo);
            pa[nt][1] = movmatrix_trans(a_hi);
            pb[nt][0] = movmatrix_trans(b_lo);
            pb[nt][1] = movmatrix_trans(b_hi);
        }
        if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
            for (int nt = 0; nt < NROW; ++nt)
#pragma unroll
                for (int mt = 0; mt < D / 16; ++mt) {
                    oacc[nt][mt][0] *= corr[nt][0]; oacc[nt][mt][1] *= corr[nt][1];
                    oacc[nt][mt][2] *= corr[nt][0]; oacc[nt][mt][3] *= corr[nt][1];
                }
        }
        // ---- O^T += V^T P^T ----
        uint32_t vmask0 = 0xffffffffu, vmask1 = 0xffffffffu;
        if (tail) {
            // rows past the region's end may hold anything (slack is never written): clear them so that
            // 0 * garbage cannot turn into NaN
            const int jk = j0 + 2 * t;
            vmask0 = (jk < len ? 0x0000ffffu : 0u) | (jk + 1 < len ? 0xffff0000u : 0u);
            vmask1 = (jk + 8 < len ? 0x0000ffffu : 0u) | (jk + 9 < len ? 0xffff0000u : 0u);
        }
        {
            const int row = blk_row0 + (mi >> 1) * 8 + rr;
#pragma unroll
            for (int mt = 0; mt < D / 16; ++mt) {
                const int cg = mt * 2 + (mi & 1);
                const int hf = cg >> 3, chunk = cg & 7;
                uint32_t a[4];   // channels mt*16.. / +8 of keys 2t, 2t+1, then of keys 2t+8, 2t+9
                ldmatrix_x4_trans(a, v_base + hf * sub_stride + row * 128 + ((chunk ^ (row & 7)) << 4));
                if (tail) { a[0] &= vmask0; a[1] &= vmask0; a[2] &= vmask1; a[3] &= vmask1; }
#pragma unroll
                for (int nt = 0; nt < NROW; ++nt) {
                    mma_bf16_16816(oacc[nt][mt], a[0], a[1], a[2], a[3], pa[nt][0], pa[nt][1]);
                    mma_bf16_16816(oacc[nt][mt], a[0], a[1], a[2], a[3], pb[nt][0], pb[nt][1]);
                }
            }
        }
    };

    // Writes the region's result (whole region inside this CTA) or an unnormalised partial.
    uint4 tok = make_uint4(0u, 0u, 0u, 0u);
    bool tok_ready = false;
    // 16 bytes of the appended token's row of item r: lanes 0-15 chunk c of K, lanes 16-31 chunk c of V
    auto load_token = [&](int r) {
        const int reg = r / hs, head = HS ? r % hs : g;
        const int64_t src = ((int64_t)reg * p.kv_heads + head) * D;
        const int c = lane & 15;
        const uint16_t *from = lane < 16 ? p.k_new : p.v_new;
        return c < D / 8 ? __ldg(reinterpret_cast<const uint4 *>(from + src) + c) : make_uint4(0u, 0u, 0u, 0u);
    };
    auto flush = [&](int r, int ustart, int uend) {
        if (p.k_new != nullptr && uend == s_P[r + 1]) {
            // Eq. 2: this CTA holds the item's last unit, so the appended token joins here.  Warp ks = 0 of every
            // head copies the token's K and V rows into a one-row tile in the scratch area (rows 1..15 of that
            // tile are whatever lies behind it: masked like any row past the end), stores them into the cache
            // and runs the block routine on it.
            if (ks == 0) {
                const int head = HS ? r % hs : g;
                uint8_t *area = reinterpret_cast<uint8_t *>(s_merge) + g * (4 * 128);
                const int64_t dst = (((int64_t)s_off[r] + len) * p.kv_heads + head) * D;
                const int c = lane & 15;
                const uint4 v = tok_ready ? tok : load_token(r);
                tok_ready = false;
                if (c < D / 8) {
                    uint16_t *to = lane < 16 ? p.k_cache : p.v_cache;
                    *reinterpret_cast<uint4 *>(area + (lane < 16 ? 0 : 2 * 128) + (c >> 3) * 128 + (c & 7) * 16) = v;
                    reinterpret_cast<uint4 *>(to + dst)[c] = v;
                }
                __syncwarp();
                process_block(smem_u32(area), smem_u32(area + 2 * 128), 128, 0, len, len + 1);
            }
            consumer_bar(NCW * 32);   // the scratch area becomes the merge buffer below
        }
#pragma unroll
        for (int nt = 0; nt < NROW; ++nt)
#pragma unroll
            for (int sh = 4; sh < 32; sh <<= 1) {
                l_run[nt][0] += __shfl_xor_sync(0xffffffffu, l_run[nt][0], sh);
                l_run[nt][1] += __shfl_xor_sync(0xffffffffu, l_run[nt][1], sh);
            }
        // the KSPLIT warps of a KV head merge their states pairwise: in every round the upper half of the
        // remaining warps hands its (max, sum, accumulator) to the lower half through shared memory
#pragma unroll
        for (int half = KSPLIT / 2; half >= 1; half >>= 1) {
            if (ks >= half && ks < 2 * half) {
                float *dst = s_merge + (size_t)(g * C::MERGE_SLOTS + ks - half) * C::MERGE_FLOATS_PER_WARP + lane;
                int c = 0;
#pragma unroll
                for (int nt = 0; nt < NROW; ++nt) {
                    dst[32 * c++] = m_run[nt][0];
                    dst[32 * c++] = m_run[nt][1];
                    dst[32 * c++] = l_run[nt][0];
                    dst[32 * c++] = l_run[nt][1];
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) dst[32 * c++] = oacc[nt][mt][i];
                }
            }
            consumer_bar(NCW * 32);
            if (ks < half) {
                const float *src = s_merge + (size_t)(g * C::MERGE_SLOTS + ks) * C::MERGE_FLOATS_PER_WARP + lane;
                int c = 0;
#pragma unroll
                for (int nt = 0; nt < NROW; ++nt) {
                    float a[2], b[2];
                    const float m2[2] = {src[32 * c], src[32 * (c + 1)]};
                    const float l2[2] = {src[32 * (c + 2)], src[32 * (c + 3)]};
                    c += 4;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float mn = fmaxf(m_run[nt][e], m2[e]);
                        a[e] = exp2_or_zero(m_run[nt][e], mn);
                        b[e] = exp2_or_zero(m2[e], mn);
                        l_run[nt][e] = l_run[nt][e] * a[e] + l2[e] * b[e];
                        m_run[nt][e] = mn;
                    }
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            oacc[nt][mt][i] = oacc[nt][mt][i] * a[i & 1] + src[32 * c++] * b[i & 1];
                }
            }
            consumer_bar(NCW * 32);
        }
        const bool whole = (ustart == s_P[r]) && (uend == s_P[r + 1]);
        if (ks == 0) {
            // this thread's values: heads nt*8 + 2t + e, channels mt*16 + gid and + 8 (the eight gid lanes of a
            // store instruction cover 32 consecutive bytes of a head's row)
#pragma unroll
            for (int nt = 0; nt < NROW; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int hl = nt * 8 + 2 * t + e;
                    if (hl >= G) continue;
                    const int h = g * G + hl;
                    if (whole) {
                        const float inv = l_run[nt][e] > 0.f ? 1.0f / l_run[nt][e] : 0.f;
                        float *o = p.out + ((int64_t)r * p.Hq + h) * D + gid;
#pragma unroll
                        for (int mt = 0; mt < D / 16; ++mt) {
                            o[mt * 16] = oacc[nt][mt][e] * inv;
                            o[mt * 16 + 8] = oacc[nt][mt][2 + e] * inv;
                        }
                    } else {
                        const int slot = slot_of((int)blockIdx.x, r);
                        float *base = p.partials + (size_t)slot * partial_slot_floats(p.Hq, D);
                        float *o = base + (size_t)h * D + gid;
#pragma unroll
                        for (int mt = 0; mt < D / 16; ++mt) {
                            __stcg(o + mt * 16, oacc[nt][mt][e]);
                            __stcg(o + mt * 16 + 8, oacc[nt][mt][2 + e]);
                        }
                        if (gid == 0) {
                            __stcg(base + (size_t)p.Hq * D + h, m_run[nt][e]);
                            __stcg(base + (size_t)p.Hq * (D + 1) + h, l_run[nt][e]);
                        }
                    }
                }
        }
        if (!whole) {
            // split-K combine without a second launch: publish the partial, draw a ticket; the CTA that draws
            // the region's last ticket merges all partials in CTA order
            __threadfence();
            consumer_bar(NCW * 32);
            int c0, c1;
            span_of(r, c0, c1);
            if (tid == 0) {
                const int tk = atomicAdd(p.tickets + r, 1);
                s_last = (tk == c1 - c0);
                if (s_last) __threadfence();
            }
            consumer_bar(NCW * 32);
            if (s_last) {
                if (tid == 0) p.tickets[r] = 0;   // ready for the next call
                const size_t slot_floats = (size_t)partial_slot_floats(p.Hq, D);
                const int items = p.Hq * D / 4;
                const int np = c1 - c0 + 1;
                float4 *o4 = reinterpret_cast<float4 *>(p.out + (int64_t)r * p.Hq * D);
                if (np == 2) {
                    // Two pieces: this CTA's half is still in the registers of its ks = 0 warps, so only the
                    // other half is fetched (one round trip).  Products first, then one addition: the result
                    // does not depend on which of the two CTAs came last.
                    if (ks == 0) {
                        const int other = (int)blockIdx.x == c0 ? c1 : c0;
                        const float *base = p.partials + (size_t)slot_of(other, r) * slot_floats;
#pragma unroll
                        for (int nt = 0; nt < NROW; ++nt)
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int hl = nt * 8 + 2 * t + e;
                                if (hl >= G) continue;
                                const int h = g * G + hl;
                                const float m2 = __ldcg(base + (size_t)p.Hq * D + h);
                                const float l2 = __ldcg(base + (size_t)p.Hq * (D + 1) + h);
                                float x[D / 16][2];
#pragma unroll
                                for (int mt = 0; mt < D / 16; ++mt) {
                                    x[mt][0] = __ldcg(base + (size_t)h * D + mt * 16 + gid);
                                    x[mt][1] = __ldcg(base + (size_t)h * D + mt * 16 + 8 + gid);
                                }
                                const float mn = fmaxf(m_run[nt][e], m2);
                                const float a = exp2_or_zero(m_run[nt][e], mn), b = exp2_or_zero(m2, mn);
                                const float den = __fadd_rn(__fmul_rn(l_run[nt][e], a), __fmul_rn(l2, b));
                                const float inv = den > 0.f ? 1.0f / den : 0.f;
                                float *o = p.out + ((int64_t)r * p.Hq + h) * D + gid;
#pragma unroll
                                for (int mt = 0; mt < D / 16; ++mt) {
                                    o[mt * 16] = __fmul_rn(
                                        __fadd_rn(__fmul_rn(oacc[nt][mt][e], a), __fmul_rn(x[mt][0], b)), inv);
                                    o[mt * 16 + 8] = __fmul_rn(
                                        __fadd_rn(__fmul_rn(oacc[nt][mt][2 + e], a), __fmul_rn(x[mt][1], b)), inv);
                                }
                            }
                    }
                } else if (uend == u1 && (size_t)np * slot_floats * 4 <= (size_t)kStages * C::STAGE_BYTES) {
                    // This CTA has no unit left, so the ring is empty: pull all partials of the region into it
                    // with bulk copies (one round trip for everything), then merge out of shared memory.  The
                    // loops below are rolled on purpose: the code runs once and cold instructions cost more
                    // than the arithmetic.
                    const uint32_t bar = smem_u32(&s_bar[2 * kStages]);
                    const uint32_t slot_bytes = (uint32_t)(slot_floats * 4);
                    if (tid == 0) {
                        asm volatile("fence.proxy.async;" ::: "memory");
                        mbar_expect_tx(bar, np * slot_bytes);
#pragma unroll 1
                        for (int c = 0; c < np; ++c)
                            bulk_load(smem_u32(s_stage) + c * slot_bytes, p.partials + slot_of(c0 + c, r) * slot_floats,
                                      slot_bytes, bar);
                    }
                    if (mbar_wait(bar, 0, &s_abort, p.status, 3)) {
                        const float *sp = reinterpret_cast<const float *>(s_stage);
                        float *wgt = s_merge;   // [np][Hq] weights exp2(m_c - M) / sum
#pragma unroll 1
                        for (int h = tid; h < p.Hq; h += NCW * 32) {
                            float M = -INFINITY, den = 0.f;
#pragma unroll 1
                            for (int c = 0; c < np; ++c) M = fmaxf(M, sp[c * slot_floats + p.Hq * D + h]);
#pragma unroll 1
                            for (int c = 0; c < np; ++c)
                                den += sp[c * slot_floats + p.Hq * (D + 1) + h] *
                                       exp2_or_zero(sp[c * slot_floats + p.Hq * D + h], M);
                            const float inv = den > 0.f ? 1.0f / den : 0.f;
#pragma unroll 1
                            for (int c = 0; c < np; ++c)
                                wgt[c * p.Hq + h] = exp2_or_zero(sp[c * slot_floats + p.Hq * D + h], M) * inv;
                        }
                        consumer_bar(NCW * 32);
#pragma unroll 1
                        for (int i = tid; i < items; i += NCW * 32) {
                            const int h = (i * 4) / D;
                            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
                            for (int c = 0; c < np; ++c) {
                                const float4 a = reinterpret_cast<const float4 *>(sp + c * slot_floats)[i];
                                const float w = wgt[c * p.Hq + h];
                                acc.x += a.x * w; acc.y += a.y * w; acc.z += a.z * w; acc.w += a.w * w;
                            }
                            o4[i] = acc;
                        }
                    }
                } else {
                    // Mid-stream (the ring is busy) or too many partials for it: online merge straight from
                    // global memory, eight partials' loads in flight per column.
#pragma unroll 1
                    for (int i = tid; i < items; i += NCW * 32) {
                        const int h = (i * 4) / D;
                        float M = -INFINITY, den = 0.f;
                        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
                        for (int cb = c0; cb <= c1; cb += 8) {
                            float mm[8], ll[8];
                            float4 aa[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float *base = p.partials + slot_of(min(cb + j, c1), r) * slot_floats;
                                mm[j] = __ldcg(base + (size_t)p.Hq * D + h);
                                ll[j] = __ldcg(base + (size_t)p.Hq * (D + 1) + h);
                                aa[j] = __ldcg(reinterpret_cast<const float4 *>(base) + i);
                            }
                            float mx = -INFINITY;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (cb + j > c1) mm[j] = -INFINITY;
                                mx = fmaxf(mx, mm[j]);
                            }
                            const float Mn = fmaxf(M, mx);
                            const float sc = exp2_or_zero(M, Mn);
                            num.x *= sc; num.y *= sc; num.z *= sc; num.w *= sc; den *= sc;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float w = exp2_or_zero(mm[j], Mn);
                                num.x += aa[j].x * w; num.y += aa[j].y * w; num.z += aa[j].z * w; num.w += aa[j].w * w;
                                den += ll[j] * w;
                            }
                            M = Mn;
                        }
                        const float inv = den > 0.f ? 1.0f / den : 0.f;
                        o4[i] = make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
                    }
                }
            }
        }
    };

    int r = r_own >= 0 ? r_own : find_region(s_P, n, u0);
    int seg_start = u0;
    len = r_own >= 0 ? len_own : p.lens[r / hs];
    load_q(r);
    // Eq. 2: when this CTA will flush the item's last unit, the appended token's K (lanes 0-15) and V (lanes 16-31)
    // are requested now, so that the flush does not wait for them
    if (p.k_new != nullptr && ks == 0 && r_own >= 0 && u1 == s_P[r + 1]) {
        tok = load_token(r);
        tok_ready = true;
    }
    int it = 0;
    bool ok = true;
    for (int u = u0; u < u1; ++u, ++it) {
        if (u >= s_P[r + 1]) {
            flush(r, seg_start, u);
            while (u >= s_P[r + 1]) ++r;
            seg_start = u;
            len = p.lens[r / hs];
            load_q(r);
        }
        const int s = it % kStages;
        ok = mbar_wait(smem_u32(&s_bar[s]), (it / kStages) & 1, &s_abort, p.status, 2);
        if (!ok) break;
        const int j0 = (u - s_P[r]) * CH + ks * 16;  // first row of this warp's block inside the region
        if (j0 < len) {
            const uint32_t k_base = smem_u32(s_stage + s * C::STAGE_BYTES) + g * C::HALVES * C::SUBTILE;
            process_block(k_base, k_base + C::KV_BYTES, C::SUBTILE, ks * 16, j0, len);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&s_bar[kStages + s]));
    }
    if (ok) flush(r, seg_start, u1);
    if (r_own < 0) finish(false);   // (else the producer warp has drawn the ticket already)
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
// bf16 [rows, Hkv, D] viewed as a 3-D tensor (D, Hkv, rows); one box = 64 channels x 1 head x ch rows.
int make_map(CUtensorMap *tm, const void *base, int D, int Hkv, int64_t rows, int ch) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) { set_last_cuda_error(cudaErrorSymbolNotFound); return AIRCACHE_ERR_CUDA; }
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)rows};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hkv * D * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)ch};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult rc = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) { set_last_cuda_error(cudaErrorInvalidValue); return AIRCACHE_ERR_CUDA; }
    return AIRCACHE_OK;
}

int sm_count(int *out) {
    int dev = 0;
    AIRCACHE_CUDA_TRY(cudaGetDevice(&dev));
    AIRCACHE_CUDA_TRY(cudaDeviceGetAttribute(out, cudaDevAttrMultiProcessorCount, dev));
    return AIRCACHE_OK;
}

template <int D, int HKV, bool G_HI, bool HS>
int launch_decode_t(const aircache_ragged_t *c, DecodeParams &p, int kv_heads, cudaStream_t st) {
    using C = DecodeCfg<D, HKV, G_HI, HS>;
    CUtensorMap tm_k, tm_v;
    int rc = make_map(&tm_k, c->k, D, kv_heads, c->total_rows, C::CH);
    if (rc) return rc;
    if ((rc = make_map(&tm_v, c->v, D, kv_heads, c->total_rows, C::CH))) return rc;
    int sms = 0;
    if ((rc = sm_count(&sms))) return rc;
    const int ctas = sms < kMaxDecodeCtas ? sms : kMaxDecodeCtas;
    AIRCACHE_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<D, HKV, G_HI, HS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           C::SMEM_BYTES));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    AIRCACHE_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_kernel<D, HKV, G_HI, HS>, tm_k, tm_v, p));
    return AIRCACHE_OK;
}

template <int D, int HKV>
int launch_decode_g(const aircache_ragged_t *c, DecodeParams &p, cudaStream_t st) {
    return p.G > 8 ? launch_decode_t<D, HKV, true, false>(c, p, HKV, st)
                   : launch_decode_t<D, HKV, false, false>(c, p, HKV, st);
}

// When there are so few regions that even (region, KV head) pairs do not outnumber the SMs, the cache is cut
// by such pairs instead of by regions: an item is then a quarter (an eighth) of a region, most items fit one
// CTA whole and need no split-K merge, and the partials of the rest are a head's worth.  All eight consumer
// warps work on the item's head, 128 rows per unit.  The kernel is the one-KV-head instantiation with the
// head taken from the item index.  With more items than SMs the by-region cut is faster (shorter units, all
// heads of a row in one contiguous read).
template <int D>
int launch_decode_d(const aircache_shape_t *s, const aircache_ragged_t *c, DecodeParams &p, cudaStream_t st) {
    const int hkv = s->n_kv_heads;
    int sms = 0;
    int rc = sm_count(&sms);
    if (rc) return rc;
    if (p.n_regions * hkv <= (sms < kMaxDecodeCtas ? sms : kMaxDecodeCtas)) {   // also with one KV head: an item is a region
        p.hs = hkv;
        p.n_regions *= hkv;
        p.Hq = p.G;
        return p.G > 8 ? launch_decode_t<D, 1, true, true>(c, p, hkv, st)
                       : launch_decode_t<D, 1, false, true>(c, p, hkv, st);
    }
    switch (hkv) {
        case 1: return launch_decode_g<D, 1>(c, p, st);
        case 2: return launch_decode_g<D, 2>(c, p, st);
        case 4: return launch_decode_g<D, 4>(c, p, st);
        case 8: return launch_decode_g<D, 8>(c, p, st);
        default: return AIRCACHE_ERR_UNSUPPORTED;
    }
}

// In per-KV-head mode every cell (layer, sequence, KV head) is a region of its own with one KV head and the G query
// heads that read it: q and out [L, B, Hq, d] are [cells, G, d] as they stand, the new token's rows [cells, 1, d].
// The kernel sees that shape; the workspace carve-up stays the caller's.
const aircache_shape_t *decode_view(const aircache_shape_t *s, DecodeParams &p, aircache_shape_t *view) {
    if (!s->per_kv_head) return s;
    *view = *s;
    view->n_layers = (int32_t)n_cells(s);
    view->batch = 1;
    view->n_q_heads = s->n_q_heads / s->n_kv_heads;
    view->n_kv_heads = 1;
    view->per_kv_head = 0;
    p.n_regions = view->n_layers;
    p.Hq = view->n_q_heads;
    p.kv_heads = 1;
    return view;
}

}  // namespace

int launch_decode(const aircache_shape_t *s, const aircache_ragged_t *c, const void *q, const void *k_new,
                  const void *v_new, float *out, void *ws, cudaStream_t st) {
    const WsLayout w = ws_layout(s);
    DecodeParams p;
    p.q = (const uint16_t *)q;
    p.out = out;
    p.offsets = c->offsets;
    p.lens = c->lens;
    p.tickets = ws_ptr<int32_t>(ws, w.tickets);
    p.plan_memo = ws_ptr<int32_t>(ws, w.plan_memo);
    p.partials = ws_ptr<float>(ws, w.partials);
    p.status = ws_ptr<uint32_t>(ws, w.status);
    p.k_new = (const uint16_t *)k_new;
    p.v_new = (const uint16_t *)v_new;
    p.k_cache = (uint16_t *)c->k;
    p.v_cache = (uint16_t *)c->v;
    p.lens_rw = c->lens;
    p.done_ticket = ws_ptr<int32_t>(ws, w.status) + 4;   // fifth word of the status block
    p.kv_heads = s->n_kv_heads;
    p.n_regions = s->n_layers * s->batch;
    p.Hq = s->n_q_heads;
    p.G = s->n_q_heads / s->n_kv_heads;
    p.sl2 = s->scale * kLog2e;
    p.hs = 1;
    aircache_shape_t view;
    s = decode_view(s, p, &view);
    return s->head_dim == 64 ? launch_decode_d<64>(s, c, p, st) : launch_decode_d<128>(s, c, p, st);
}

// ---------------------------------------------------------------------------------------------
// aircache_decode_attn_static: the same kernel with its scratch in a built-in device array
// ---------------------------------------------------------------------------------------------
// Status word, split-K tickets and partial slots of the decode kernel, for callers that bring no
// workspace.  Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[AIRCACHE_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char *g_static_ptr[kMaxDevices] = {};
}  // namespace

int launch_decode_static(const aircache_shape_t *s, const aircache_ragged_t *c, const void *q, float *out,
                         cudaStream_t st) {
    int dev = 0, sms = 0;
    AIRCACHE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return AIRCACHE_ERR_UNSUPPORTED;
    AIRCACHE_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int64_t ctas = sms < kMaxDecodeCtas ? sms : kMaxDecodeCtas;
    const int64_t need = kStatusBytes + 2 * ctas * partial_slot_floats(s->n_q_heads, s->head_dim) * 4;
    if (need > (int64_t)AIRCACHE_STATIC_SCRATCH_BYTES) return AIRCACHE_ERR_STATIC_SCRATCH;
    unsigned char *base = nullptr;
    {
        // In host code the array's name is only a handle; its device address on the current device comes
        // from the runtime, once per device.
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {
            void *ptr = nullptr;
            AIRCACHE_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
            g_static_ptr[dev] = static_cast<unsigned char *>(ptr);
        }
        base = g_static_ptr[dev];
    }
    // The array keeps whatever the previous call left: the status word and the tickets must start at zero.
    AIRCACHE_CUDA_TRY(cudaMemsetAsync(base, 0, kStatusBytes, st));
    DecodeParams p;
    p.q = (const uint16_t *)q;
    p.out = out;
    p.offsets = c->offsets;
    p.lens = c->lens;
    p.status = reinterpret_cast<uint32_t *>(base);
    p.plan_memo = nullptr;   // the built-in array keeps no plans: every call plans afresh
    p.k_new = p.v_new = nullptr;
    p.k_cache = p.v_cache = nullptr;
    p.lens_rw = nullptr;
    p.done_ticket = nullptr;
    p.kv_heads = s->n_kv_heads;
    p.tickets = reinterpret_cast<int32_t *>(base + 256);
    p.partials = reinterpret_cast<float *>(base + kStatusBytes);
    p.n_regions = s->n_layers * s->batch;
    p.Hq = s->n_q_heads;
    p.G = s->n_q_heads / s->n_kv_heads;
    p.sl2 = s->scale * kLog2e;
    p.hs = 1;
    aircache_shape_t view;
    s = decode_view(s, p, &view);
    return s->head_dim == 64 ? launch_decode_d<64>(s, c, p, st) : launch_decode_d<128>(s, c, p, st);
}

}  // namespace aircache
