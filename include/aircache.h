/*
 * aircache.h -- C ABI of the AirCache compress-then-decode hot path for NVIDIA B200 (sm_100a).
 *
 * AirCache (arXiv 2503.23956) compresses the visual part of a vision-language
 * model's KV cache once, after prefill:
 *   1. aircache_score    importance of every visual token seen from the elite
 *                        observation window                     (Section 3.3, Eq. 4-8)
 *   2. aircache_budget   per-layer token budgets from the strength and skewness
 *                        of the importance distribution         (Section 3.4, Eq. 9-11)
 *   3. aircache_compact  per-layer top-k and gather into one packed ragged
 *                        cache; text tokens are always kept     (Algorithm 1, second loop)
 *   4. aircache_decode_attn  single-token attention over that ragged cache
 *                        (Section 3.1, token decoding)
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 * Pointers.   Unless a parameter is marked HOST it is a DEVICE pointer into
 *             memory owned by the caller.  The library never allocates or frees
 *             device memory; scratch space is the caller's `workspace`
 *             (aircache_workspace_bytes() bytes, 256-byte aligned).  Structs are
 *             HOST memory and are read before the call returns.
 * Layout.     bf16 tensors are raw 16-bit patterns.  Token order inside one
 *             sequence is Concat(visual, text) (Eq. 3): tokens 0..n_visual-1 are
 *             visual, n_visual..n_visual+n_text-1 are text.  "Region" (l, b) has
 *             index r = l * batch + b.  Query head h reads KV head
 *             g = h / (n_q_heads / n_kv_heads).
 * Streams.    All work is enqueued on `cuda_stream` (a cudaStream_t passed as
 *             void*, NULL = the legacy default stream).  No entry point
 *             synchronises or copies device memory to the host, except
 *             aircache_check_status() and aircache_pipeline_host().
 * Errors.     Return value 0 = success, negative = an AIRCACHE_ERR_* code.  All
 *             argument checks run on the host before anything is launched, so a
 *             failing call has enqueued nothing (aircache_pipeline_host, which
 *             issues many copies and launches, is the exception: see there).
 *             No exception crosses the ABI.
 * Threads.    The library keeps no mutable global state apart from a per-thread
 *             copy of the last CUDA error code, the device address of the
 *             built-in array of aircache_decode_attn_static and the number of
 *             blocks of the scoring kernel a device holds at once (each looked
 *             up once per device, under a lock); calls that share a workspace
 *             must be ordered on one stream.
 * Determinism. Same inputs give the same output bits on every run.
 */
#ifndef AIRCACHE_H
#define AIRCACHE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AIRCACHE_VERSION 102

#define AIRCACHE_OK 0
#define AIRCACHE_ERR_INVALID_ARG (-1)          /* NULL pointer, negative size, ratio outside [0,1], ...        */
#define AIRCACHE_ERR_UNSUPPORTED (-2)          /* a shape the kernels do not cover (see aircache_shape_t)       */
#define AIRCACHE_ERR_ALIGNMENT (-3)            /* a pointer or stride that breaks the 16-byte rules             */
#define AIRCACHE_ERR_WORKSPACE_TOO_SMALL (-4)
#define AIRCACHE_ERR_CAPACITY (-5)             /* ragged cache smaller than aircache_total_rows()               */
#define AIRCACHE_ERR_CUDA (-6)                 /* a CUDA call failed; see aircache_last_cuda_error()            */
#define AIRCACHE_ERR_TIMEOUT (-7)              /* a bounded device-side wait gave up (aircache_check_status)    */
#define AIRCACHE_ERR_STATIC_SCRATCH (-8)       /* aircache_decode_attn_static: built-in scratch array too small */
#define AIRCACHE_ERR_INCONSISTENT (-9)         /* aircache_compact found budgets / offsets that do not fit the buffers (aircache_check_status) */

/* Size of the device array that aircache_decode_attn_static uses as scratch, per GPU. */
#define AIRCACHE_STATIC_SCRATCH_BYTES (12 * 1024 * 1024)

/* Problem shape, uniform over the batch. */
typedef struct {
    int32_t n_layers;    /* L >= 1                                                                   */
    int32_t batch;       /* B >= 1; L * B <= 1792 (L * B * Hkv <= 1792 with per_kv_head)             */
    int32_t n_q_heads;   /* Hq, a multiple of n_kv_heads with Hq / Hkv <= 16                         */
    int32_t n_kv_heads;  /* Hkv in {1, 2, 4, 8}                                                      */
    int32_t head_dim;    /* d in {64, 128}                                                           */
    int32_t n_visual;    /* Nv >= 3 visual tokens per sequence (Eq. 10 needs three)                  */
    int32_t n_text;      /* Nt >= 1 text tokens per sequence                                         */
    int32_t window;      /* W: the last W text tokens are the candidates of Eq. 5; 1 <= W <= min(128, Nt);
                            W = Nt is the paper's window (every text token a candidate)                */
    int32_t slack;       /* rows left free after each region for tokens appended while decoding, >= 0 */
    float scale;         /* softmax scale of Eq. 4 and Eq. 7, normally 1 / sqrt(head_dim)            */
    int32_t per_kv_head; /* 0: one budget and one kept set per (layer, sequence), shared by all KV heads
                            (the paper's method).  1: Eq. 8-11 and the top-k of Algorithm 1 applied to
                            every KV head on its own - see "Per-KV-head mode" below                  */
} aircache_shape_t;

/*
 * Per-KV-head mode (per_kv_head = 1), a refinement the paper does not evaluate.
 * The unit of compression is the cell (layer l, sequence b, KV head g), index
 * c = (l * B + b) * Hkv + g, instead of the region (l, b):
 *   scores    fp32 [L, B, Hkv, Nv]: Eq. 8 averaged over the query heads of group g only;
 *   budgets, strength, skewness  [L, B, Hkv]: Eq. 9-10 per cell; Eq. 11 normalises over the
 *             L * Hkv cells of a sequence, which share T = floor(ratio * Nv * L * Hkv + 0.5)
 *             rows (aircache_kept_per_sequence), ties to the lower cell;
 *   ragged cache: rows are single-head rows, k and v bf16 [total_rows, 1, d]; offsets
 *             [L*B*Hkv + 1] and lens [L*B*Hkv] are per cell; cell c keeps its own tokens;
 *   kept_idx  cell c's ascending list at offsets[c] - c * (Nt + slack);
 *   decode    query head h attends to the cell of its KV head; q and out stay [L, B, Hq, d];
 *   append    k_new, v_new stay [L, B, Hkv, d]: one row per cell.
 * Everything else (elite_mask, window queries, the full cache view) is unchanged.
 */

/*
 * Full (uncompressed) cache of the prefill: logical bf16 [L, B, Hkv, Nv+Nt, d]
 * addressed with element strides, head_dim contiguous.  Pointers 16-byte
 * aligned, every stride a multiple of 8 elements.  Read-only for the library.
 */
typedef struct {
    const void *k, *v;
    int64_t stride_layer, stride_batch, stride_head, stride_token;
} aircache_full_t;

/*
 * Compressed ragged cache (Algorithm 1's C^l = {K', V'}, a different length per
 * layer).  k and v are bf16 [total_rows, Hkv, d]; region r owns rows
 * offsets[r] .. offsets[r+1]-1, of which the first lens[r] hold
 * Concat(K_v[kept], K_t) in ascending token order and the rest is slack.
 * aircache_budget writes offsets and lens, aircache_compact writes k and v.
 * k and v must be 128-byte aligned.
 *
 * Several caches may share one pair of buffers, packed back to back (requests
 * whose sequences differ in N_v and N_t, hence in shape, compressed by separate
 * calls): each call gets the same k, v and total_rows, first_row = the rows
 * taken by the caches before it (the sum of their aircache_total_rows(), known
 * on the host), and offsets / lens pointing at its own stretch of two shared
 * arrays - stretch s starts where stretch s-1 holds its last offset, which is
 * the same number.  offsets are rows of the shared buffers, so one
 * aircache_decode_attn call (n_layers = number of all regions, batch = 1) then
 * attends over all of them.
 */
typedef struct {
    void *k, *v;
    int64_t *offsets;    /* [L*B + 1] rows */
    int32_t *lens;       /* [L*B]     rows in use */
    int64_t total_rows;  /* capacity of k and v in rows, >= first_row + aircache_total_rows() */
    int64_t first_row;   /* rows of k and v in front of this cache's first region; 0 for a cache of its own */
} aircache_ragged_t;

int aircache_version(void);

/* Static, NUL-terminated description of a return code (never freed). */
const char *aircache_strerror(int code);

/* cudaError_t of the most recent AIRCACHE_ERR_CUDA on the calling thread (0 if none). */
int aircache_last_cuda_error(void);

/*
 * Visual rows one sequence keeps over all layers: T = floor(ratio * Nv * L + 0.5)
 * (the total budget r of Algorithm 1 is preserved by the re-allocation of Eq. 11).
 * Host arithmetic only.
 */
int64_t aircache_kept_per_sequence(const aircache_shape_t *shape, double ratio);

/*
 * Rows the ragged cache needs: B * (T + L * (Nt + slack)).  Known before
 * anything runs because Eq. 11 only re-partitions T among the layers.
 * Host arithmetic only; negative = error code.
 */
int64_t aircache_total_rows(const aircache_shape_t *shape, double ratio);

/* Bytes of scratch any entry point may use for this shape.  Host arithmetic only; negative = error code. */
int64_t aircache_workspace_bytes(const aircache_shape_t *shape);

/*
 * Section 3.3, Eq. 4-8.  For every region and query head h: the last window
 * query scores the W candidate text keys (Eq. 4); candidates within a factor
 * alpha of the best form the elite set E_h (Eq. 5; alpha <= 0 keeps all W, the
 * decision is taken on fp32 logits computed from fp64 dot products).  Each elite
 * query w attends to all visual keys plus the elite text keys w' <= w (Eq. 6-7,
 * causal among text); the visual columns are averaged over the elite rows
 * (Eq. 8) and then over the Hq heads.
 *   q_window    bf16 [L, B, W, Hq, d]  queries of the W candidate text tokens (candidate w is
 *                                      text token Nt-W+w; the last one is the reference of Eq. 4)
 *   alpha       relevance threshold in [0, 1]
 *   scores      fp32 [L, B, Nv]        output I_v
 *   elite_mask  u64  [L, B, Hq, ceil(W/64)]  output, candidate w is elite <=> bit w % 64 of word w / 64 is
 *                                      set (one word per head up to W = 64, two beyond); may be NULL
 * The blocks of the scoring kernel that share a KV group wait for one another
 * (a bounded wait; safe because the library only lets them when at most half of
 * the blocks the GPU holds at once are involved).  If other work keeps most of
 * the GPU busy for the whole wait (a quarter of a second), the wait gives up,
 * the scores are incomplete and aircache_check_status() reports
 * AIRCACHE_ERR_TIMEOUT.
 */
int aircache_score(const aircache_shape_t *shape, const aircache_full_t *full, const void *q_window,
                   float alpha, float *scores, uint64_t *elite_mask, void *workspace, int64_t workspace_bytes,
                   void *cuda_stream);

/*
 * Algorithm 1, first loop, a range of its iterations: aircache_score for layers
 * layer_begin .. layer_begin + layer_count - 1 only.  The paper scores layer by
 * layer and keeps every layer's full cache until all are scored (Section 4.1
 * and the limitation noted in Appendix A); an engine calls this at the end of
 * each layer's prefill, while that layer's keys are still in L2, and runs
 * aircache_budget once after the last layer.  All arrays are the ones
 * aircache_score takes (indexed by absolute layer); only the given layers' keys
 * and window queries are read and only their rows of scores / elite_mask are
 * written.  A layer's scores equal those of aircache_score up to rounding
 * (into how many chunks a call cuts the keys, hence the order in which their
 * softmax statistics merge, depends on how many layers it covers); equal calls
 * give equal bits.  Calls that share a workspace must be ordered on one
 * stream.  layer_count = 0 is a no-op.
 */
int aircache_score_layers(const aircache_shape_t *shape, const aircache_full_t *full, const void *q_window,
                          float alpha, int32_t layer_begin, int32_t layer_count, float *scores,
                          uint64_t *elite_mask, void *workspace, int64_t workspace_bytes, void *cuda_stream);

/*
 * Section 3.4, Eq. 9-11 and the budget line of Algorithm 1.  Per region:
 * strength s_t = sum of I_v (Eq. 9) and skewness s_k = adjusted Fisher-Pearson
 * coefficient with the sample standard deviation (Eq. 10), both in fp64.  Per
 * sequence: both are divided by their mean over the layers (negative skewness
 * counts as 0, a zero mean makes the factor 1), w_l = (s't + s'k) / 2 (Eq. 11),
 * and T = aircache_kept_per_sequence() rows are split in proportion to w_l with
 * every layer capped at Nv (excess re-shared), floors first, the remaining rows
 * one each to the largest fractional parts, ties to the lower layer.
 *   mode      0: Eq. 11   1: strength only   2: skewness only   3: uniform
 *   budgets   i32 [L, B]  output n_{l,b}                       ([L, B, Hkv] in per-KV-head mode,
 *   strength, skewness  f64 [L, B]  outputs; either may be NULL  as are these)
 *   layout    offsets and lens are written (offsets[r+1] - offsets[r] = n_r + Nt + slack,
 *             lens[r] = n_r + Nt); k and v are not touched
 */
int aircache_budget(const aircache_shape_t *shape, const float *scores, double ratio, int32_t mode,
                    int32_t *budgets, double *strength, double *skewness, aircache_ragged_t *layout,
                    void *workspace, int64_t workspace_bytes, void *cuda_stream);

/*
 * Algorithm 1, second loop.  Per region: the n_r visual tokens of largest score
 * (radix select on the fp32 bit pattern; equal scores: the lower token index
 * wins), then K' = Concat(K_v[kept], K_t), V' = Concat(V_v[kept], V_t) are
 * gathered into the region's rows, kept tokens in ascending token order.
 * out->offsets and out->lens must hold what aircache_budget wrote for `budgets`.
 * Both live in device memory, so the host cannot check them: the kernels do.  A
 * budget outside [0, Nv], a kept list that would leave the list buffer, a row
 * that would land outside [0, out->total_rows) or a listed token outside
 * [0, Nv) is not followed - the entries and rows concerned stay unwritten - and
 * aircache_check_status() then reports AIRCACHE_ERR_INCONSISTENT.  (Values that
 * fit the buffers but do not belong together, such as regions that overlap,
 * cannot be told from a layout the caller meant.)
 *   ratio      the same ratio aircache_budget was given (sizes the launch; capacity check)
 *   kept_idx   i32, region r's ascending token list at position offsets[r] - r*(Nt+slack);
 *              B * T entries in total; may be NULL
 */
int aircache_compact(const aircache_shape_t *shape, const aircache_full_t *full, const float *scores,
                     const int32_t *budgets, double ratio, aircache_ragged_t *out, int32_t *kept_idx,
                     void *workspace, int64_t workspace_bytes, void *cuda_stream);

/*
 * Section 3.1, token decoding, over the compressed cache: for every region and
 * query head h,  out_h = sum_j softmax_j(scale * <q_h, K'_g[j]>) * V'_g[j]  over
 * the lens[r] rows of region r.  bf16 inputs, fp32 accumulation, fp32 output.
 * A region with lens[r] = 0 yields zeros.
 *   q    bf16 [L, B, Hq, d]   one query token per region
 *   out  fp32 [L, B, Hq, d]
 * Device-side waits are bounded; if one gives up, a status word in the workspace
 * is set and aircache_check_status() reports AIRCACHE_ERR_TIMEOUT.
 */
int aircache_decode_attn(const aircache_shape_t *shape, const aircache_ragged_t *cache, const void *q,
                         float *out, void *workspace, int64_t workspace_bytes, void *cuda_stream);

/*
 * One decode step with the KV append of Eq. 2 fused in: the new token's K and V
 * (bf16 [L, B, Hkv, d]) are stored in the first free slack row of every region,
 * take part in this call's attention together with the lens[r] cached rows, and
 * lens[r] grows by one when the call completes (same result as aircache_append
 * followed by aircache_decode_attn, in one launch).  `appended` as in
 * aircache_append; AIRCACHE_ERR_CAPACITY on the host when the slack is used up.
 */
int aircache_decode_step(const aircache_shape_t *shape, aircache_ragged_t *cache, const void *q, const void *k_new,
                         const void *v_new, int32_t appended, float *out, void *workspace, int64_t workspace_bytes,
                         void *cuda_stream);

/*
 * aircache_decode_attn for callers that cannot allocate device memory.  (An
 * addition of this library; the paper has no counterpart.)
 *
 * Some hosts of this code only ever borrow the GPU: a plug-in running inside
 * another engine's memory pool, a real-time loop that may not enter the
 * allocator after start-up, a process whose device memory is fully
 * pre-assigned.  They can hand over the cache, the query and the output, but
 * have nowhere to get the workspace that aircache_decode_attn wants.  This
 * entry point runs the same kernel and takes the kernel's scratch (status
 * word, split-K tickets, partial results) from an array of
 * AIRCACHE_STATIC_SCRATCH_BYTES bytes that is compiled into the library; every
 * GPU that loads the library holds that array until the process exits.  It
 * never calls cudaMalloc, cudaFree or any other allocating routine.
 *
 *   Arguments as in aircache_decode_attn, without the workspace.
 *   Limit.   7424 + 2 * min(SMs, 256) * 4 * (Hq * (d + 2) rounded up to a multiple of 4)
 *            bytes must fit in the array (7424 = 256 bytes of status + 1792 tickets;
 *            on a 148-SM B200: Hq * (d + 2) <= 10620, e.g. 80 heads of 128);
 *            larger problems get AIRCACHE_ERR_STATIC_SCRATCH and nothing is enqueued.
 *   Set-up.  The first call on each device looks up the array's device address
 *            (with that device current).  Make that first call before any
 *            stream capture is begun.
 *   Sharing. All calls on a device use the one array, and the array keeps what
 *            the last call left in it; each call therefore clears the status
 *            word and the tickets on the stream before its kernel.  Two calls
 *            that can overlap on the GPU (different streams without an ordering
 *            between them) race on the array and give wrong results: order them.
 *   Status.  The status word of the bounded waits lives inside the array and is
 *            not visible to aircache_check_status.
 */
int aircache_decode_attn_static(const aircache_shape_t *shape, const aircache_ragged_t *cache, const void *q,
                                float *out, void *cuda_stream);

/*
 * Eq. 2, KV append during decoding: writes one new token's K and V
 * (bf16 [L, B, Hkv, d]) into the first free slack row of every region and adds 1
 * to lens[r].  Fails on the host with AIRCACHE_ERR_CAPACITY when `appended`
 * (rows already appended since compaction, tracked by the caller) >= slack.
 */
int aircache_append(const aircache_shape_t *shape, aircache_ragged_t *cache, const void *k_new,
                    const void *v_new, int32_t appended, void *cuda_stream);

/*
 * Zeroes the head of a workspace (enqueued on the stream): the status word, the
 * tickets and the plans that decode launches keep from one call to the next
 * (about 150 KB in all).  Must be called once after allocating the workspace,
 * before its first use by aircache_budget or aircache_decode_attn, and again
 * after an AIRCACHE_ERR_TIMEOUT or AIRCACHE_ERR_INCONSISTENT.
 */
int aircache_reset_status(void *workspace, int64_t workspace_bytes, void *cuda_stream);

/*
 * Synchronises the stream, reads the workspace's status word and returns 0,
 * AIRCACHE_ERR_TIMEOUT (a bounded wait gave up) or AIRCACHE_ERR_INCONSISTENT
 * (aircache_compact met values that do not fit the buffers).  The only
 * device-to-host read in the library apart from
 * aircache_pipeline_host().
 */
int aircache_check_status(void *workspace, int64_t workspace_bytes, void *cuda_stream);

/*
 * Diagnostics: enqueues a one-CTA kernel whose threads wait, with the same
 * bounded wait the decode kernel uses, on a barrier that nothing completes.
 * The wait gives up after its poll limit (a fraction of a second), the kernel
 * returns normally and the workspace's status word is set, so a following
 * aircache_check_status() reports AIRCACHE_ERR_TIMEOUT; aircache_reset_status()
 * clears it.  Shows that a stuck wait ends in an error code, not in a hang.
 */
int aircache_selftest_wait_timeout(void *workspace, int64_t workspace_bytes, void *cuda_stream);

/*
 * 1 if the whole host range [host_ptr, host_ptr + bytes) is page-locked memory
 * that kernels on the current device can read in place, else 0 (pageable
 * memory, a null pointer, an empty range).  Host-side query, launches nothing.
 */
int aircache_host_range_is_mapped(const void *host_ptr, int64_t bytes);

/*
 * The whole path with HOST inputs and outputs: uploads the full cache and the
 * queries, runs score -> budget -> compact -> n_steps x decode_attn on the
 * stream, downloads the results and synchronises.  Every device buffer is still
 * the caller's (no device memory is allocated inside).  K is uploaded whole
 * (scoring reads all of it).  V is only ever read where a row
 * survives: if h_full->v is page-locked host memory that the GPU can address
 * (cudaHostAlloc / cudaHostRegister; aircache_host_range_is_mapped() tells),
 * compaction reads the kept and the text rows of V from it in place and
 * d_full_v stays untouched; otherwise V is uploaded whole like K.  The decode
 * queries are uploaded in groups of 16 rounds on a stream of their own, behind
 * the caches and beside the compression and the earlier rounds, and the outputs
 * of the decode rounds are copied back in groups of 4 rounds on another stream,
 * beside the later rounds (the call creates and destroys both streams); on
 * return every copy has completed.  The call clears the workspace's status
 * words itself.  If a copy or a launch fails after the first copy has been
 * enqueued, the call still drains all its streams before it returns the error, so
 * the host buffers are never touched after the return; the device buffers then
 * hold partial results.
 *   h_full       HOST view of the full cache (strides as in aircache_full_t)
 *   full_elems   elements (bf16) spanned by h_full->k and by h_full->v
 *   d_full_k/v   DEVICE buffers of full_elems bf16 each
 *   h_q_window   HOST bf16 [L, B, W, Hq, d];  d_q_window DEVICE, same size
 *   h_q_steps    HOST bf16 [n_steps, L, B, Hq, d];  d_q_steps DEVICE, same size
 *   d_scores     DEVICE fp32 [L, B, Nv];  d_budgets DEVICE i32 [L, B]
 *   d_cache      DEVICE ragged cache (k, v, offsets, lens, total_rows)
 *   d_out        DEVICE fp32 [n_steps, L, B, Hq, d];  h_out HOST, same size (output)
 *   h_budgets    HOST i32 [L, B] (output; [L, B, Hkv] in per-KV-head mode, like d_budgets)
 */
int aircache_pipeline_host(const aircache_shape_t *shape, const aircache_full_t *h_full, int64_t full_elems,
                           void *d_full_k, void *d_full_v, const void *h_q_window, void *d_q_window,
                           const void *h_q_steps, void *d_q_steps, int32_t n_steps, float alpha, double ratio,
                           int32_t mode, float *d_scores, int32_t *d_budgets, aircache_ragged_t *d_cache,
                           float *d_out, float *h_out, int32_t *h_budgets, void *workspace,
                           int64_t workspace_bytes, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* AIRCACHE_H */
